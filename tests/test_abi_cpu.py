"""Host-only checks of the C ABI: the library loads without a GPU, exports every
symbol include/dllm.h declares, and its size / layout / argument logic is right.
No compute call is made here."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2506_06295_b200 import build as build_mod
from paper_2506_06295_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def dllm():
    build_mod.build()
    from paper_2506_06295_b200 import dllm as d
    return d


def declared_functions():
    text = open(os.path.join(ROOT, "include", "dllm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dllm_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(dllm):
    names = declared_functions()
    assert len(names) >= 30
    for name in names:
        assert hasattr(dllm.lib, name), f"{name} not exported"
        assert name in dllm.SIGNATURES, f"{name} has no Python signature"
    assert sorted(dllm.SIGNATURES) == names


def test_cache_bytes_is_four_tensors_per_layer(dllm):
    # Sec. A.9: 4 * tokens * d * layers elements (MHA), x2 bytes in bf16
    assert dllm.cache_bytes(synth.TINY, 1, 64, 32) == 4 * 96 * 256 * 2 * 4
    assert dllm.cache_bytes(synth.LLADA_8B, 1, 512, 256) == 805306368
    c = synth.DREAM_7B   # GQA: K and V are narrower
    assert dllm.cache_bytes(c, 1, 256, 256) == c.n_layers * 512 * (2 * 512 + 2 * 3584) * 2
    assert dllm.cache_bytes(synth.TINY, 0, 64, 32) == 0


def test_weight_blob_layout(dllm):
    for cfg in (synth.TINY, synth.small_bf16_model(), synth.small_bf16_model(gqa=True)):
        total = dllm.weights_bytes(cfg)
        es = 2 if cfg.dtype == "bf16" else 4
        spans = []
        for name, shape in synth.tensor_names(cfg):
            off, n = dllm.tensor_offset(cfg, name)
            assert n == int(np.prod(shape))
            size = n * (4 if name.endswith(("norm1", "norm2", "norm_f")) else es)
            rows, stride = dllm.tensor_blocks(cfg, name)
            assert off % 16 == 0
            if rows == 0:
                spans.append((off, off + size, name))
            else:   # row-blocked: one span per block
                blk = rows * cfg.d_model * es
                assert size % blk == 0 and stride >= blk
                spans += [(off + b * stride, off + b * stride + blk, name) for b in range(size // blk)]
        spans.sort()
        assert spans[-1][1] <= total
        for (a0, a1, an), (b0, b1, bn) in zip(spans, spans[1:]):
            assert a1 <= b0, f"{an} overlaps {bn}"
        # W_q, W_k, W_v are stacked contiguously (one GEMM for Q and K), so are W_gate, W_up
        q, nq = dllm.tensor_offset(cfg, "layers.1.wq")
        k, nk = dllm.tensor_offset(cfg, "layers.1.wk")
        v, _ = dllm.tensor_offset(cfg, "layers.1.wv")
        assert k == q + nq * es and v == k + nk * es
        # ... so are W_gate and W_up: one after the other, or (bf16, d_ffn % 64 == 0) alternating in blocks of 64 rows
        g, ng = dllm.tensor_offset(cfg, "layers.0.wg")
        u, _ = dllm.tensor_offset(cfg, "layers.0.wu")
        rows, stride = dllm.tensor_blocks(cfg, "layers.0.wg")
        if cfg.dtype == "bf16" and cfg.d_ffn % 64 == 0:
            assert (rows, stride) == (64, 128 * cfg.d_model * es) == dllm.tensor_blocks(cfg, "layers.0.wu")
            assert u == g + 64 * cfg.d_model * es
        else:
            assert rows == 0 and u == g + ng * es
        assert dllm.tensor_blocks(cfg, "layers.1.wq") == (0, 0) == dllm.tensor_blocks(cfg, "lm_head")


def test_llada_sizes_fit_one_gpu(dllm):
    cfg = synth.LLADA_8B
    w = dllm.weights_bytes(cfg)
    assert 15.9e9 < w < 16.2e9          # 8.0 B parameters in bf16
    ws = dllm.workspace_bytes(cfg, 16, 1024, 512)
    assert w + ws + dllm.cache_bytes(cfg, 16, 1024, 512) < 170e9


def test_invalid_arguments_are_rejected_without_a_gpu(dllm):
    bad = synth.ModelConfig(n_layers=0, d_model=256, n_heads=4, n_kv_heads=4, head_dim=64, d_ffn=688,
                            vocab=1024, mask_id=1023, dtype="fp32")
    assert dllm.weights_bytes(bad) == 0
    with pytest.raises(dllm.DllmError) as e:
        dllm.tensor_offset(synth.TINY, "layers.9.wq")
    assert e.value.status == dllm.INVALID_ARG and "unknown tensor" in str(e.value)
    h = C.c_void_p()
    cc = dllm.make_config(synth.TINY)
    assert dllm.lib.dllm_model_create(C.byref(cc), None, C.byref(h)) == dllm.INVALID_ARG
    assert not h.value
    odd = synth.ModelConfig(n_layers=1, d_model=100, n_heads=4, n_kv_heads=3, head_dim=64, d_ffn=688,
                            vocab=1024, mask_id=1023, dtype="fp32")
    cc = dllm.make_config(odd)
    assert dllm.lib.dllm_model_create(C.byref(cc), C.c_void_p(256), C.byref(h)) == dllm.INVALID_ARG
    assert "multiple of n_kv_heads" in dllm.last_error()
    for fn, args in (("dllm_step_full", (None, None)), ("dllm_sync", (None, None)),
                     ("dllm_remask_low_confidence", (None, 0, 1, 1, None)),
                     ("dllm_generate", (None, 8, 4, 2, 0.25, 0, 32, None))):
        assert getattr(dllm.lib, fn)(*args) == dllm.INVALID_ARG
    assert dllm.lib.dllm_gemm_bf16(None, None, None, 1, 1, 8, None, None) == dllm.INVALID_ARG
    assert dllm.lib.dllm_gemm_bf16_scratch_bytes(64, 4096, 4096) > 0
    assert dllm.lib.dllm_gemm_bf16_scratch_bytes(256, 126464, 4096) == 0      # enough tiles: no split


def test_timeline_build_exports_its_hooks_and_the_product_library_has_none(dllm):
    """The timeline variant is a separate library with the same ABI plus one pair of hooks per kernel file; the
    product library carries no instrumentation."""
    path = build_mod.build(timeline=True)
    assert path.endswith("libdllm_b200_timeline.so") and os.path.exists(path)
    tl = C.CDLL(path)
    from paper_2506_06295_b200 import timeline
    for stem in timeline.STEMS:
        assert hasattr(tl, "dllm_timeline_set_" + stem) and hasattr(tl, "dllm_timeline_count_" + stem)
        assert not hasattr(dllm.lib, "dllm_timeline_set_" + stem)
    for name in declared_functions():
        assert hasattr(tl, name)


def test_binding_has_no_fallback():
    src = open(os.path.join(ROOT, "paper_2506_06295_b200", "dllm.py")).read()
    assert "oracle" not in src.replace("no CPU or PyTorch fallback", "")
    for f in os.listdir(os.path.join(ROOT, "paper_2506_06295_b200", "csrc")):
        assert "oracle" not in open(os.path.join(ROOT, "paper_2506_06295_b200", "csrc", f)).read()
