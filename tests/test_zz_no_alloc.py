"""dllm_attention_noalloc: the attention entry point for callers that cannot
allocate device memory (they hold raw buffers only, or run under a fixed memory
plan).  It must give what dllm_attention gives, call after call, although all
calls share one scratch array built into the library that still holds the
previous call's partial results.  Collected last on purpose: a failure here
cannot hide the result of any other test."""
import numpy as np
import pytest

from paper_2506_06295_b200 import synth
from tests.helpers import rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2506_06295_b200 import build as build_mod
    build_mod.build()
    from paper_2506_06295_b200 import dllm
    assert torch.cuda.is_available()
    return torch, dllm


def _inputs(torch, B, a, n, H, Hkv, hd, seed):
    q = synth.round_to_bf16(synth.random_normal((B * a, H * hd), seed=seed, std=1.3))
    k = synth.round_to_bf16(synth.random_normal((B, n, Hkv * hd), seed=seed + 1, std=1.3))
    v = synth.round_to_bf16(synth.random_normal((B, n, Hkv * hd), seed=seed + 2))
    return [torch.from_numpy(t).cuda().to(torch.bfloat16) for t in (q, k, v)]


def test_noalloc_matches_the_allocating_entry_point_on_two_calls_in_a_row(env):
    torch, dllm = env
    # every shape splits the key range into partials in scratch, so every call uses the built-in scratch: the
    # first two on the 64-row kernel with more splits than a cluster merges (21 and 10), the third on the 128-row
    # tcgen05 kernel (128 rows per KV head); each is differently laid out from the one before, so stale partials of
    # the previous call lie in and behind its own
    for i, shape in enumerate([(1, 36, 4128, 2, 2, 128), (2, 40, 2000, 2, 1, 64), (1, 128, 512, 8, 8, 128)]):
        B, a, n, H, Hkv, hd = shape
        assert dllm.lib.dllm_attention_scratch_bytes(B, a, n, H, Hkv, hd, dllm.BF16) > 0
        q, k, v = _inputs(torch, *shape, seed=100 + 10 * i)
        want = dllm.attention(q, k, v, B, a, n, H, Hkv, hd).to(torch.float32).cpu().numpy()
        out = torch.full_like(q, float("nan"))
        before = torch.cuda.memory_allocated()
        dllm.attention_noalloc(q, k, v, out, B, a, n, H, Hkv, hd)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before           # the binding created no tensor either
        got = out.to(torch.float32).cpu().numpy()
        assert np.isfinite(got).all()
        assert rel_l2(got, want) < 8e-3                            # the tolerance of the attention parity test
        assert np.array_equal(got, want)                           # same kernels, same plan: in fact identical


def test_noalloc_rejects_what_does_not_fit_its_scratch(env):
    torch, dllm = env
    # 256 rows per KV head (the tcgen05 kernel), 16 heads, 2048 keys: key splits with 16 MB of partials
    B, a, n, H, Hkv, hd = 1, 256, 2048, 16, 16, 128
    assert dllm.lib.dllm_attention_scratch_bytes(B, a, n, H, Hkv, hd, dllm.BF16) > 8 * 1024 * 1024
    q, k, v = _inputs(torch, B, a, n, H, Hkv, hd, seed=7)
    out = torch.zeros_like(q)
    with pytest.raises(dllm.DllmError) as e:
        dllm.attention_noalloc(q, k, v, out, B, a, n, H, Hkv, hd)
    assert e.value.status == dllm.UNSUPPORTED and "scratch" in str(e.value)
    assert float(out.abs().max()) == 0.0                           # nothing ran
    with pytest.raises(dllm.DllmError) as e:
        dllm.attention_noalloc(q, k, v, out, B, a, n, H, Hkv, 96)
    assert e.value.status == dllm.UNSUPPORTED
