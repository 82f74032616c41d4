"""Step-level parity on the GPU: the cached denoising step, the transition and
the generation loop, called through the C ABI and compared with the CPU oracle
on the same seeded weights and prompts.

Tolerances (relative L2 of the response hidden states): 1e-4 in fp32 mode,
2e-2 in bf16 mode.  Selected index sets must match exactly except for tokens
within 1e-3 of the k-th similarity; to tell a legal tie flip from an arithmetic
fault the bf16 runs are repeated with the oracle's sets forced into the GPU
path."""
import os

import numpy as np
import pytest

from oracle import dllm_oracle as O
from paper_2506_06295_b200 import synth
from tests.helpers import rel_l2, selection_matches

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2506_06295_b200 import build as build_mod
    build_mod.build()
    from paper_2506_06295_b200 import dllm
    assert torch.cuda.is_available()
    return torch, dllm


def make_pair(dllm, cfg, B, P, R, odtype=np.float64, seed=synth.WEIGHT_SEED):
    w = synth.make_weights(cfg, seed)
    prompt = synth.make_prompt(cfg, B, P)
    orc = O.DLLMOracle(cfg, w, B, P, R, dtype=odtype)
    orc.set_prompt(prompt)
    model = dllm.Model(cfg).load(w)
    ses = dllm.Session(model, B, P, R)
    ses.set_prompt(prompt)
    return orc, ses, w


def unmask(orc, ses, step, count):
    """Unmask `count` response tokens per sequence in both implementations."""
    P = orc.P
    resp = orc.tokens[:, P:].copy()
    for b in range(orc.B):
        masked = np.nonzero(resp[b] == orc.cfg.mask_id)[0]
        pick = masked[(np.arange(count) * 7 + 3 * step + b) % max(len(masked), 1)] if len(masked) else []
        for j in pick:
            resp[b, j] = (31 * j + 5 * step + b) % (orc.cfg.vocab - 1)
    orc.tokens[:, P:] = resp
    ses.set_response_tokens(resp)


def compare_step(orc, ses, r, tol, check_sets=True, what="", sim_atol=None):
    ses.sync()
    hid = ses.hidden()
    err = rel_l2(hid, r.hidden)
    assert err < tol, f"{what}: hidden rel-L2 {err:.3e} >= {tol}"
    for l in range(orc.cfg.n_layers):
        idx, sim = ses.selected(l)
        assert idx.shape == r.selected[l].shape, what
        if check_sets:
            for b in range(orc.B):
                assert selection_matches(idx[b], r.selected[l][b], None if r.sim[l] is None else r.sim[l][b]), \
                    f"{what}: layer {l} seq {b}: {idx[b].tolist()} vs {r.selected[l][b].tolist()}"
        if r.sim[l] is not None:
            np.testing.assert_allclose(sim, r.sim[l], atol=sim_atol or (5e-3 if tol > 1e-3 else 2e-5))
    return err


def compare_caches(dllm, orc, ses, tol, what=""):
    for l in range(orc.cfg.n_layers):
        for which, ref in ((dllm.CACHE_K, orc.Kc), (dllm.CACHE_V, orc.Vc), (dllm.CACHE_ATTN, orc.Ac),
                           (dllm.CACHE_FFN, orc.Fc)):
            err = rel_l2(ses.get_cache(l, which), ref[l])
            assert err < tol, f"{what}: cache {which} layer {l}: {err:.3e}"


# ---------------------------------------------------------------- tiny fp32 configuration
def test_tiny_fp32_all_step_kinds(env):
    torch, dllm = env
    wl = synth.WORKLOADS["tiny"]
    orc, ses, _ = make_pair(dllm, wl.model, 2, wl.prompt_len, wl.gen_len)
    r = orc.step(True, True)
    ses.step_full()
    compare_step(orc, ses, r, 1e-4, what="full")
    compare_caches(dllm, orc, ses, 1e-4, "full")
    x0, conf = ses.pred()
    assert np.array_equal(x0, r.x0)
    np.testing.assert_allclose(conf, r.conf, rtol=1e-3)
    lg = ses.logits()
    fin = np.isfinite(r.logits)
    assert np.array_equal(np.isfinite(lg), fin)
    assert rel_l2(lg[fin], r.logits[fin]) < 1e-4
    step = 0
    for rp, rr, rho in ((False, False, 0.25), (False, True, 0.0), (False, False, 0.25), (True, False, 0.25),
                        (False, False, 0.5), (False, False, 0.0), (True, True, 0.0), (False, False, 1.0)):
        step += 1
        unmask(orc, ses, step, 4)
        r = orc.step(rp, rr, rho)
        ses.step_cached(rp, rr, rho)
        compare_step(orc, ses, r, 1e-4, what=f"step {step} ({rp},{rr},{rho})")
        compare_caches(dllm, orc, ses, 1e-4, f"step {step}")
        x0, conf = ses.pred()
        assert np.array_equal(x0, r.x0)


def test_tiny_fp32_generation_matches_token_for_token(env):
    torch, dllm = env
    wl = synth.WORKLOADS["tiny"]
    orc, ses, _ = make_pair(dllm, wl.model, 1, wl.prompt_len, wl.gen_len)
    want = orc.generate(wl.steps, wl.Kp, wl.Kr, wl.rho, wl.block_len)
    ses.generate(wl.steps, wl.Kp, wl.Kr, wl.rho, wl.block_len)
    ses.sync()
    got = ses.tokens()
    assert (got[:, wl.prompt_len:] != wl.model.mask_id).all()
    assert np.array_equal(got, want)


@pytest.mark.parametrize("mode", ["fp32", "bf16"])
def test_block_only_prediction_gives_the_same_generation(env, mode):
    """Predicting only the block a step works on (the only rows Eq. 5 reads) leaves hidden states and caches
    untouched, gives bit-identical estimates and confidences for the block, and generates the same tokens; in
    fp32 those are the oracle's tokens."""
    torch, dllm = env
    if mode == "fp32":
        wl = synth.WORKLOADS["tiny"]
        cfg, B, P, R, K, Kp, Kr, rho, bl = wl.model, 2, wl.prompt_len, wl.gen_len, wl.steps, wl.Kp, wl.Kr, wl.rho, 16
    else:
        cfg, B, P, R, K, Kp, Kr, rho, bl = synth.small_bf16_model(), 2, 100, 48, 12, 6, 3, 0.25, 16
    orc, ses_all, _ = make_pair(dllm, cfg, B, P, R)
    _, ses_blk, _ = make_pair(dllm, cfg, B, P, R)
    # one step each way on the same state: same hidden states, same (x0, conf) inside the block
    ses_all.step_full()
    ses_blk.step_full()
    for k, bs in ((K - 1, 0), (K - 2, bl)):
        ses_all.step_scheduled(k, K, Kp, Kr, rho)
        ses_blk.step_scheduled_block(k, K, Kp, Kr, rho, bs, bl)
        ses_all.sync(), ses_blk.sync()
        assert np.array_equal(ses_all.hidden(), ses_blk.hidden())
        (xa, ca), (xb, cb) = ses_all.pred(), ses_blk.pred()
        assert np.array_equal(xa[:, bs:bs + bl], xb[:, bs:bs + bl])
        assert np.array_equal(ca[:, bs:bs + bl], cb[:, bs:bs + bl])
        for l in range(cfg.n_layers):
            for w in range(4):
                assert np.array_equal(ses_all.get_cache(l, w), ses_blk.get_cache(l, w))
    assert ses_blk.launch_count() > 0
    # whole generations
    prompt = synth.make_prompt(cfg, B, P)
    toks = []
    for ses, on in ((ses_all, False), (ses_blk, True)):
        ses.set_prompt(prompt)
        ses.predict_block_only(on)
        ses.generate(K, Kp, Kr, rho, bl)
        ses.sync()
        toks.append(ses.tokens())
    assert (toks[1][:, P:] != cfg.mask_id).all()
    assert np.array_equal(toks[0], toks[1])
    if mode == "fp32":
        assert np.array_equal(toks[1], orc.generate(K, Kp, Kr, rho, bl))
    with pytest.raises(dllm.DllmError):
        ses_blk.step_scheduled_block(1, K, Kp, Kr, rho, R - 1, bl)      # block leaves the response


@pytest.mark.parametrize("graphs", [False, True], ids=["host_events", "graph_event_nodes"])
def test_profiling_counts_every_projection_and_changes_no_result(env, graphs):
    """Per-kernel timing brackets every projection (class 0) and attention launch (class 1) with an event pair,
    recorded by the host or as nodes of the step's graph; the step's results are those of an unprofiled step."""
    torch, dllm = env
    cfg = synth.small_bf16_model()
    B, P, R = 2, 150, 72
    _, ses, _ = make_pair(dllm, cfg, B, P, R)
    _, ref, _ = make_pair(dllm, cfg, B, P, R)
    ses.use_graphs(graphs)
    for s_ in (ses, ref):
        s_.step_full()
    ses.profile(True)
    steps = ((False, False, 0.25), (False, True, 0.0), (False, False, 0.25), (True, False, 0.5))
    for rp, rr, rho in steps:
        ses.step_cached(rp, rr, rho)
        ref.step_cached(rp, rr, rho)
    ses.sync(), ref.sync()
    g, a = ses.profile_read(0), ses.profile_read(1)
    # per layer: V (all response rows), Q/K, O, gate/up, down (+ V of the prompt rows on a prompt refresh); LM head
    expect = sum(cfg.n_layers * (5 + (1 if rp else 0)) + 1 for rp, _, _ in steps)
    assert g["launches"] == expect and a["launches"] == len(steps) * cfg.n_layers
    assert g["ms"] > 0 and a["ms"] > 0 and g["bytes"] > 0 and g["flops"] > 0 and a["flops"] > 0
    # the two aggregates are sums over their sub-classes; every row-wise launch has a class of its own
    per = {name: ses.profile_read(i) for i, name in enumerate(dllm.PROF_CLASSES)}
    assert sum(per[c]["launches"] for c in dllm.PROF_CLASSES[2:8]) == g["launches"]
    assert abs(sum(per[c]["ms"] for c in dllm.PROF_CLASSES[2:8]) - g["ms"]) < 1e-6 * g["ms"]
    assert per["attention_mma"]["launches"] + per["attention_tcgen05"]["launches"] == a["launches"]
    assert per["layer_tail"]["launches"] == len(steps) * cfg.n_layers and per["embed_norm"]["launches"] == len(steps)
    assert per["vverify"]["launches"] == len(steps) * cfg.n_layers  # every step projects V for all response rows
    assert per["select_gather"]["launches"] == 3 * cfg.n_layers    # not on the response refresh (identity lists)
    assert per["gemm_lm_head"]["launches"] == len(steps) and per["estimate_merge"]["launches"] == len(steps)
    assert all(v["bytes"] > 0 for k, v in per.items() if v["launches"])
    assert np.array_equal(ses.hidden(), ref.hidden())
    assert np.array_equal(ses.tokens(), ref.tokens())
    ses.profile(False)
    assert ses.profile_read(0)["launches"] == 0
    ses.step_cached(False, False, 0.25)       # unprofiled steps still run (and replay their own graphs)
    ref.step_cached(False, False, 0.25)
    ses.sync(), ref.sync()
    assert np.array_equal(ses.hidden(), ref.hidden())


def test_timeline_of_a_step_lists_every_launch_once():
    """The in-graph timeline (separate library build, own process) sees each kernel launch of a step exactly
    once, in order, with non-negative durations."""
    import json
    import subprocess
    import sys
    import tempfile
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    with tempfile.TemporaryDirectory() as td:
        out = os.path.join(td, "tl.json")
        r = subprocess.run([sys.executable, "-m", "paper_2506_06295_b200.timeline", "--workload", "tiny", "--kind",
                            "partial", "--layer", "1", "--json", out], cwd=root, capture_output=True, text=True, timeout=600)
        assert r.returncode == 0, r.stderr[-2000:]
        launches = json.load(open(out))
    cfg = synth.WORKLOADS["tiny"].model
    # fp32 model, partial step: embedding, 12 launches per layer (V, V-verify, selection + gather, Q/K, RoPE,
    # attention, O, its epilogue, gate/up, SwiGLU, down, tail), LM head, estimate
    assert len(launches) == 1 + 12 * cfg.n_layers + 2, [(o["file"], o["grid"]) for o in launches]
    starts = [o["start_us"] for o in launches]
    assert starts == sorted(starts) and all(o["dur_us"] >= 0 for o in launches)
    assert all(o["ctas"] == o["grid"][0] * o["grid"][1] * o["grid"][2] for o in launches)
    assert "layer 1 (12 launches" in r.stdout


def test_tiny_fp32_stepwise_generation_with_graphs_off_and_on(env):
    torch, dllm = env
    wl = synth.WORKLOADS["tiny"]
    outs = []
    for graphs in (False, True):
        orc, ses, _ = make_pair(dllm, wl.model, 1, wl.prompt_len, wl.gen_len)
        ses.use_graphs(graphs)
        for k in range(wl.steps, 0, -1):
            ses.step_scheduled(k, wl.steps, wl.Kp, wl.Kr, wl.rho)
            bs, nt = O.block_plan(wl.steps - k, wl.steps, wl.gen_len, wl.block_len)
            ses.remask_low_confidence(bs, wl.block_len, nt)
        ses.sync()
        outs.append((ses.tokens(), ses.hidden(), ses.launch_count()))
    assert np.array_equal(outs[0][0], outs[1][0])
    assert np.array_equal(outs[0][1], outs[1][1])
    assert outs[0][2] == outs[1][2] > 0


# ---------------------------------------------------------------- bf16, several tiles and ragged tails
@pytest.mark.parametrize("gqa", [False, True], ids=["mha", "gqa"])
@pytest.mark.parametrize("path", ["simt_gemm", "tcgen05_gemm"])
def test_small_bf16_step_kinds(env, gqa, path):
    """Every step kind against the oracle, on the plain-ALU kernels and on the
    tensor-core kernels."""
    torch, dllm = env
    cfg = synth.small_bf16_model(gqa=gqa)
    B, P, R = 2, 150, 72
    orc, ses, _ = make_pair(dllm, cfg, B, P, R)
    ses.use_simt_gemm(path == "simt_gemm")
    r = orc.step(True, True)
    ses.step_full()
    compare_step(orc, ses, r, 2e-2, what="full")
    compare_caches(dllm, orc, ses, 2e-2, "full")
    step = 0
    for rp, rr, rho in ((False, False, 0.25), (False, False, 0.25), (False, True, 0.0), (True, False, 0.5),
                        (False, False, 0.1), (False, False, 0.0)):
        step += 1
        unmask(orc, ses, step, 3)
        r = orc.step(rp, rr, rho)
        # free-running comparison first ...
        ses.step_cached(rp, rr, rho)
        ses.sync()
        free_ok = all(selection_matches(ses.selected(l)[0][b], r.selected[l][b],
                                        None if r.sim[l] is None else r.sim[l][b])
                      for l in range(cfg.n_layers) for b in range(B))
        assert free_ok, f"step {step}: selection differs beyond the tie tolerance"
        err = compare_step(orc, ses, r, 2e-2, what=f"step {step} ({rp},{rr},{rho})")
        compare_caches(dllm, orc, ses, 2e-2, f"step {step}")
        assert err < 2e-2


def test_bf16_gate_up_layouts(env):
    """W_gate / W_up stored one after the other (d_ffn not a multiple of 64) and row-blocked (a multiple of 64,
    where an unsplit gate / up GEMM applies SwiGLU itself and a split one leaves it to the next kernel) give the
    oracle's step; the blocked model also accepts weights written straight into the blob."""
    import dataclasses
    torch, dllm = env
    for d_ffn in (840, 832):
        cfg = dataclasses.replace(synth.small_bf16_model(), d_ffn=d_ffn)
        assert (dllm.tensor_blocks(cfg, "layers.0.wg")[0] == 64) == (d_ffn % 64 == 0)
        B, P, R = 2, 150, 72
        orc, ses, w = make_pair(dllm, cfg, B, P, R)
        if d_ffn % 64 == 0:   # rewrite the gate / up weights through the strided view: same model
            for l in range(cfg.n_layers):
                for t in ("wg", "wu"):
                    v = ses.model.tensor_view(f"layers.{l}.{t}")
                    v.zero_()
                    v.copy_(torch.from_numpy(w[f"layers.{l}.{t}"]).cuda().to(torch.bfloat16).view(v.shape))
        r = orc.step(True, True)
        ses.step_full()
        compare_step(orc, ses, r, 2e-2, what=f"full m={d_ffn}")
        for step, (rp, rr, rho) in enumerate(((False, False, 0.25), (True, False, 0.5), (False, True, 0.0)), 1):
            unmask(orc, ses, step, 3)
            r = orc.step(rp, rr, rho)
            ses.step_cached(rp, rr, rho)
            compare_step(orc, ses, r, 2e-2, what=f"m={d_ffn} step {step}")
        compare_caches(dllm, orc, ses, 2e-2, f"m={d_ffn}")


def test_small_bf16_forced_selection_and_rho_invariants(env):
    torch, dllm = env
    cfg = synth.small_bf16_model()
    B, P, R = 1, 100, 40
    orc, ses, _ = make_pair(dllm, cfg, B, P, R)
    orc.step(True, True)
    ses.step_full()
    unmask(orc, ses, 1, 2)
    # forced sets (deliberately NOT the V-verify choice) reach both implementations
    forced = {l: np.array([[1 + l, 7, 20, 33]]) for l in range(cfg.n_layers)}
    r = orc.step(False, False, 0.1, forced=forced)
    for l in range(cfg.n_layers):
        ses.force_selection(l, forced[l])
    ses.step_cached(False, False, 0.1)
    compare_step(orc, ses, r, 2e-2, what="forced")
    compare_caches(dllm, orc, ses, 2e-2, "forced")
    for l in range(cfg.n_layers):
        ses.force_selection(l, None)
    # rho = 0 leaves every cache bit-unchanged (fully cached state)
    before = [ses.get_cache(l, w) for l in range(cfg.n_layers) for w in range(4)]
    unmask(orc, ses, 2, 2)
    ses.step_cached(False, False, 0.0)
    ses.sync()
    after = [ses.get_cache(l, w) for l in range(cfg.n_layers) for w in range(4)]
    assert all(np.array_equal(a, b) for a, b in zip(before, after))
    # rho = 1 equals a response refresh, bit for bit (same kernels, same rows)
    snap = [ses.get_cache(l, w) for l in range(cfg.n_layers) for w in range(4)]
    ses.step_cached(False, False, 1.0)
    ses.sync()
    h1 = ses.hidden()
    c1 = [ses.get_cache(l, w) for l in range(cfg.n_layers) for w in range(4)]
    for i, (l, w) in enumerate((l, w) for l in range(cfg.n_layers) for w in range(4)):
        ses.set_cache(l, w, snap[i])
    ses.step_cached(False, True, 0.0)
    ses.sync()
    assert np.array_equal(ses.hidden(), h1)
    assert all(np.array_equal(a, ses.get_cache(l, w)) for a, (l, w) in
               zip(c1, ((l, w) for l in range(cfg.n_layers) for w in range(4))))


def test_error_paths_on_device(env):
    torch, dllm = env
    cfg = synth.TINY
    model = dllm.Model(cfg).load(synth.make_weights(cfg))
    ses = dllm.Session(model, 1, 64, 32)
    ses.set_prompt(synth.make_prompt(cfg, 1, 64))
    with pytest.raises(dllm.DllmError) as e:
        ses.step_cached(False, False, 0.25)
    assert e.value.status == dllm.BAD_STATE
    with pytest.raises(dllm.DllmError) as e:
        ses.remask_low_confidence(0, 32, 4)
    assert e.value.status == dllm.BAD_STATE
    ses.step_full()
    for bad in (-0.1, 1.5, float("nan")):
        with pytest.raises(dllm.DllmError) as e:
            ses.step_cached(False, False, bad)
        assert e.value.status == dllm.INVALID_ARG
    with pytest.raises(dllm.DllmError):
        ses.remask_low_confidence(16, 32, 4)
    with pytest.raises(dllm.DllmError):
        ses.generate(8, 4, 2, 0.25, 5)
    with pytest.raises(dllm.DllmError):
        ses.set_prompt(np.full((1, 64), 5000))
    ses.sync()
