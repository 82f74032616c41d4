"""Pins for the compact storage variant of the oracle (response-only AttnOut / FFNOut caches; the memory
limitation of Sec. A.10 item (1) and the storage count of Sec. A.9).  CPU only.

The variant rests on one claim: between prompt refreshes no step reads the prompt rows of AttnOut / FFNOut,
and a prompt refresh rewrites them before it reads them.  That claim is pinned on the FOUR-tensor oracle, by
poisoning those rows; the compact oracle is then pinned to the four-tensor one output by output."""
import numpy as np
import pytest

from oracle import dllm_oracle as O
from paper_2506_06295_b200 import synth
from tests.test_oracle_pins import GQA_TINY, unmask_some

PLAN = [(False, False, 0.25), (False, False, 0.5), (False, True, 0.0), (True, False, 0.5), (False, False, 0.0),
        (False, False, 1.0), (True, True, 0.0), (False, False, 0.25)]


def pair(cfg, B, P, R, scale=3.0):
    w = synth.make_weights(cfg)
    w = {k: (v * scale if v.ndim == 2 else v) for k, v in w.items()}
    a = O.DLLMOracle(cfg, w, B, P, R)
    b = O.DLLMOracle(cfg, w, B, P, R, compact_prompt_outs=True)
    prompt = synth.make_prompt(cfg, B, P)
    a.set_prompt(prompt)
    b.set_prompt(prompt)
    return a, b


def test_prompt_rows_of_attnout_and_ffnout_are_dead_in_the_four_tensor_oracle():
    cfg, B, P, R = GQA_TINY, 2, 12, 8
    clean, _ = pair(cfg, B, P, R)
    dirty, _ = pair(cfg, B, P, R)
    for o in (clean, dirty):
        o.step(True, True)
    for k, (rp, rr, rho) in enumerate(PLAN):
        for l in range(cfg.n_layers):           # poison what the compact variant does not keep
            dirty.Ac[l][:, :P] = np.nan
            dirty.Fc[l][:, :P] = np.nan
        for o in (clean, dirty):
            unmask_some(o, k)
        rc, rd = clean.step(rp, rr, rho), dirty.step(rp, rr, rho)
        assert np.array_equal(rc.hidden, rd.hidden) and np.array_equal(rc.x0, rd.x0)
        assert np.array_equal(rc.conf, rd.conf)
        fin = np.isfinite(rc.logits)
        assert np.array_equal(fin, np.isfinite(rd.logits)) and np.array_equal(rc.logits[fin], rd.logits[fin])
        for l in range(cfg.n_layers):
            assert np.array_equal(clean.Kc[l], dirty.Kc[l]) and np.array_equal(clean.Vc[l], dirty.Vc[l])
            assert np.array_equal(clean.Ac[l][:, P:], dirty.Ac[l][:, P:])
            assert np.array_equal(clean.Fc[l][:, P:], dirty.Fc[l][:, P:])
            if rp:   # a prompt refresh rewrites them (before reading them: the outputs above are NaN-free)
                assert np.isfinite(dirty.Ac[l]).all() and np.isfinite(dirty.Fc[l]).all()


@pytest.mark.parametrize("cfg", [synth.TINY, GQA_TINY], ids=["tiny_mha", "gqa"])
def test_compact_oracle_equals_the_four_tensor_oracle_on_every_step_kind(cfg):
    B, P, R = 2, 12, 8
    a, b = pair(cfg, B, P, R)
    ra, rb = a.step(True, True), b.step(True, True)
    for k, (rp, rr, rho) in enumerate([(True, True, 0.0)] + PLAN):
        if k:
            for o in (a, b):
                unmask_some(o, k)
            ra, rb = a.step(rp, rr, rho), b.step(rp, rr, rho)
        assert np.array_equal(ra.hidden, rb.hidden) and np.array_equal(ra.x0, rb.x0) and np.array_equal(ra.conf, rb.conf)
        for l in range(cfg.n_layers):
            assert np.array_equal(ra.selected[l], rb.selected[l])
            assert (ra.sim[l] is None) == (rb.sim[l] is None)
            if ra.sim[l] is not None:
                assert np.array_equal(ra.sim[l], rb.sim[l])
            assert np.array_equal(a.Kc[l], b.Kc[l]) and np.array_equal(a.Vc[l], b.Vc[l])
            assert b.Ac[l].shape == (B, R, cfg.d_model) and b.Fc[l].shape == (B, R, cfg.d_model)
            assert np.array_equal(a.Ac[l][:, P:], b.Ac[l]) and np.array_equal(a.Fc[l][:, P:], b.Fc[l])


def test_compact_generation_gives_the_same_tokens():
    wl = synth.WORKLOADS["tiny"]
    a, b = pair(wl.model, 1, wl.prompt_len, wl.gen_len, scale=1.0)
    ta = a.generate(wl.steps, wl.Kp, wl.Kr, wl.rho, wl.block_len)
    tb = b.generate(wl.steps, wl.Kp, wl.Kr, wl.rho, wl.block_len)
    assert np.array_equal(ta, tb) and (tb != wl.model.mask_id).all()


def test_compact_storage_is_the_four_tensor_count_minus_the_prompt_outputs():
    """Sec. A.9 counts 4 * tokens * d * layers elements for MHA; the compact variant stores
    2 * P * d * layers fewer per sequence."""
    cfg, B, P, R = synth.TINY, 3, 64, 32
    a, b = pair(cfg, B, P, R, scale=1.0)
    full = 4 * (P + R) * cfg.d_model * cfg.n_layers * B
    assert a.cache_elements() == full
    assert b.cache_elements() == full - 2 * P * cfg.d_model * cfg.n_layers * B
    # at the long-prompt benchmark shape (P = 4096, R = 32, LLaDA-8B widths, bf16) that is 2.15 of 4.33 GB
    big, Pl, Rl = synth.LLADA_8B, 4096, 32
    assert 2 * 2 * Pl * big.d_model * big.n_layers == 2147483648
    assert 2 * 4 * (Pl + Rl) * big.d_model * big.n_layers == 4328521728
