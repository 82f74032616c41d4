"""Sessions with response-only AttnOut / FFNOut caches (DLLM_SESSION_COMPACT_CACHE) against the four-tensor
session (bit for bit: the same kernels compute the same rows, only the addresses differ) and against the
compact oracle, over every step kind; and the cache size against the storage count of Sec. A.9."""
import numpy as np
import pytest

from oracle import dllm_oracle as O
from paper_2506_06295_b200 import synth
from tests.helpers import rel_l2

pytestmark = pytest.mark.gpu

PLAN = [(False, False, 0.25), (False, False, 0.5), (False, True, 0.0), (True, False, 0.5), (False, False, 0.0),
        (True, True, 0.0), (False, False, 0.25)]


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2506_06295_b200 import build as build_mod
    build_mod.build()
    from paper_2506_06295_b200 import dllm
    assert torch.cuda.is_available()
    return torch, dllm


@pytest.mark.parametrize("which", ["tiny_fp32", "bf16_mha", "bf16_gqa", "bf16_many_rows", "fp32_many_rows"])
def test_compact_session_matches_the_four_tensor_session_and_the_compact_oracle(env, which):
    torch, dllm = env
    cfg = synth.TINY if which in ("tiny_fp32", "fp32_many_rows") else synth.small_bf16_model(gqa=which == "bf16_gqa")
    B, P, R = (2, 64, 32) if which == "tiny_fp32" else (2, 150, 72)
    if which.endswith("many_rows"):     # 1088 response rows: V-verify and the layer tail take their streaming forms
        B, P, R = 8, 40, 136
    tol = 1e-4 if cfg.dtype == "fp32" else 2e-2
    w = synth.make_weights(cfg)
    prompt = synth.make_prompt(cfg, B, P)
    orc = O.DLLMOracle(cfg, w, B, P, R, compact_prompt_outs=True)
    orc.set_prompt(prompt)
    model = dllm.Model(cfg).load(w)
    full = dllm.Session(model, B, P, R)
    comp = dllm.Session(model, B, P, R, compact_cache=True)
    for s in (full, comp):
        s.set_prompt(prompt)
    dkv, d, T = cfg.dkv, cfg.d_model, cfg.n_layers
    es = 4 if cfg.dtype == "fp32" else 2
    assert dllm.cache_bytes(cfg, B, P, R) == T * B * (P + R) * (2 * dkv + 2 * d) * es
    assert dllm.cache_bytes(cfg, B, P, R, dllm.SESSION_COMPACT_CACHE) == \
        dllm.cache_bytes(cfg, B, P, R) - 2 * P * d * T * B * es
    assert comp.cache.numel() == dllm.cache_bytes(cfg, B, P, R, dllm.SESSION_COMPACT_CACHE)

    for step, (rp, rr, rho) in enumerate([(True, True, 0.0)] + PLAN):
        if step:
            resp = orc.tokens[:, P:].copy()
            for b in range(B):
                j = (11 * step + 5 * b) % R
                resp[b, j] = (131 * j + step) % (cfg.vocab - 1)
            orc.tokens[:, P:] = resp
            for s in (full, comp):
                s.set_response_tokens(resp)
        r = orc.step(rp, rr, rho)
        for s in (full, comp):
            s.step_cached(rp, rr, rho) if step else s.step_full()
            s.sync()
        what = f"step {step} ({rp}, {rr}, {rho})"
        assert np.array_equal(full.hidden(), comp.hidden()), what
        assert all(np.array_equal(a, b) for a, b in zip(full.pred(), comp.pred())), what
        assert rel_l2(comp.hidden(), r.hidden) < tol, what
        for l in range(T):
            for c in (dllm.CACHE_K, dllm.CACHE_V):
                assert np.array_equal(full.get_cache(l, c), comp.get_cache(l, c)), what
            for c, ref in ((dllm.CACHE_ATTN, orc.Ac), (dllm.CACHE_FFN, orc.Fc)):
                got = comp.get_cache(l, c)
                assert got.shape == (B, R, d)
                assert np.array_equal(full.get_cache(l, c)[:, P:], got), what
                assert rel_l2(got, ref[l]) < tol, what
            if not rr and rho > 0:
                assert np.array_equal(full.selected(l)[0], comp.selected(l)[0]), what


def test_compact_generation_gives_the_same_tokens(env):
    torch, dllm = env
    wl = synth.WORKLOADS["tiny"]
    cfg = wl.model
    w = synth.make_weights(cfg)
    prompt = synth.make_prompt(cfg, wl.batch, wl.prompt_len)
    model = dllm.Model(cfg).load(w)
    out = []
    for compact in (False, True):
        ses = dllm.Session(model, wl.batch, wl.prompt_len, wl.gen_len, compact_cache=compact)
        ses.set_prompt(prompt)
        ses.generate(wl.steps, wl.Kp, wl.Kr, wl.rho, wl.block_len)
        ses.sync()
        out.append(ses.tokens())
    assert np.array_equal(out[0], out[1]) and (out[1] != cfg.mask_id).all()
    orc = O.DLLMOracle(cfg, w, wl.batch, wl.prompt_len, wl.gen_len, compact_prompt_outs=True)
    orc.set_prompt(prompt)
    assert np.array_equal(orc.generate(wl.steps, wl.Kp, wl.Kr, wl.rho, wl.block_len), out[1])
