"""Pins for the CPU oracle: everything here runs without a GPU and without the
CUDA library.  Each test ties the oracle to something other than itself: a
library routine, a closed form, an invariant the paper fixes, or brute force."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import dllm_oracle as O
from paper_2506_06295_b200 import synth

torch.set_num_threads(4)


# --------------------------------------------------------------------------
# an independent textbook forward (library routines only)
# --------------------------------------------------------------------------
def textbook_forward(cfg, w, tokens):
    """Uncached bidirectional transformer forward for ONE sequence in fp64,
    written with torch library routines (embedding, rms_norm, linear,
    scaled_dot_product_attention, silu) and complex-number rotary embedding."""
    t = {k: torch.from_numpy(np.asarray(v, dtype=np.float64)) for k, v in w.items()}
    tok = torch.from_numpy(np.asarray(tokens, dtype=np.int64))
    n = tok.shape[0]
    H, Hkv, hd, d = cfg.n_heads, cfg.n_kv_heads, cfg.head_dim, cfg.d_model
    half = hd // 2
    freqs = torch.arange(half, dtype=torch.float64) * 2.0 / hd
    ang = torch.arange(n, dtype=torch.float64)[:, None] * (cfg.rope_theta ** -freqs)[None, :]
    rot = torch.polar(torch.ones_like(ang), ang)[:, None, :]          # e^{i pos w_i}

    def rotary(v):                                                       # [n, heads, hd]
        z = torch.complex(v[..., :half], v[..., half:]) * rot
        return torch.cat([z.real, z.imag], dim=-1)

    x = F.embedding(tok, t["embed"])
    per_layer = []
    for l in range(cfg.n_layers):
        p = f"layers.{l}."
        u = F.rms_norm(x, (d,), t[p + "norm1"], cfg.rms_eps)
        q = rotary(F.linear(u, t[p + "wq"]).view(n, H, hd))
        k = rotary(F.linear(u, t[p + "wk"]).view(n, Hkv, hd))
        v = F.linear(u, t[p + "wv"]).view(n, Hkv, hd)
        kk = k.repeat_interleave(H // Hkv, dim=1)
        vv = v.repeat_interleave(H // Hkv, dim=1)
        o = F.scaled_dot_product_attention(q.transpose(0, 1)[None], kk.transpose(0, 1)[None],
                                           vv.transpose(0, 1)[None], is_causal=False)[0]
        a = F.linear(o.transpose(0, 1).reshape(n, H * hd), t[p + "wo"])
        h = x + a
        hn = F.rms_norm(h, (d,), t[p + "norm2"], cfg.rms_eps)
        f = F.linear(F.silu(F.linear(hn, t[p + "wg"])) * F.linear(hn, t[p + "wu"]), t[p + "wd"])
        x = h + f
        per_layer.append((k.reshape(n, -1).numpy(), v.reshape(n, -1).numpy(), a.numpy(), f.numpy()))
    logits = F.linear(F.rms_norm(x, (d,), t["norm_f"], cfg.rms_eps), t["lm_head"])
    return x.numpy(), logits.numpy(), per_layer


def rel_l2(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


GQA_TINY = synth.ModelConfig(n_layers=2, d_model=96, n_heads=6, n_kv_heads=2, head_dim=16,
                             d_ffn=160, vocab=211, mask_id=210, dtype="fp32")


def make(cfg, B=1, P=12, R=8, dtype=np.float64, seed=synth.WEIGHT_SEED, scale=1.0):
    w = synth.make_weights(cfg, seed)
    if scale != 1.0:   # larger weights make the caching error visible in tests
        w = {k: (v * scale if v.ndim == 2 else v) for k, v in w.items()}
    o = O.DLLMOracle(cfg, w, B, P, R, dtype=dtype)
    o.set_prompt(synth.make_prompt(cfg, B, P))
    return o, w


# --------------------------------------------------------------------------
# full step == uncached forward (the case that reduces to a plain definition)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("cfg", [synth.TINY, GQA_TINY], ids=["tiny_mha", "gqa"])
def test_full_step_equals_textbook_forward(cfg):
    P, R = (64, 32) if cfg is synth.TINY else (12, 8)
    o, w = make(cfg, B=2, P=P, R=R)
    # mix of masked and unmasked response tokens
    o.tokens[1, P + 1:P + 5] = [3, 7, 11, 13]
    r = o.step(True, True)
    for b in range(2):
        hid, logits, per_layer = textbook_forward(cfg, w, o.tokens[b])
        assert rel_l2(r.hidden[b], hid[P:]) < 1e-12
        lg = logits[P:].copy()
        lg[:, cfg.mask_id] = -np.inf
        fin = np.isfinite(lg)
        assert rel_l2(r.logits[b][fin], lg[fin]) < 1e-12
        assert np.array_equal(r.x0[b], lg.argmax(-1))
        ref_conf = torch.softmax(torch.from_numpy(lg), -1).max(-1).values.numpy()
        np.testing.assert_allclose(r.conf[b], ref_conf, rtol=1e-6)
        for l, (k, v, a, f) in enumerate(per_layer):
            assert rel_l2(o.Kc[l][b], k) < 1e-12
            assert rel_l2(o.Vc[l][b], v) < 1e-12
            assert rel_l2(o.Ac[l][b], a) < 1e-12
            assert rel_l2(o.Fc[l][b], f) < 1e-12


def test_full_step_float32_mode_close_to_float64():
    o64, _ = make(synth.TINY, P=64, R=32)
    o32, _ = make(synth.TINY, P=64, R=32, dtype=np.float32)
    r64, r32 = o64.step(True, True), o32.step(True, True)
    assert rel_l2(r32.hidden, r64.hidden) < 1e-5
    assert np.array_equal(r32.x0, r64.x0)


# --------------------------------------------------------------------------
# invariants of the caching rule
# --------------------------------------------------------------------------
def unmask_some(o, k):
    """Deterministically unmask a few tokens, as a sampler would between steps."""
    P = o.P
    for b in range(o.B):
        for j in range(k % 3, o.R, 5):
            if o.tokens[b, P + j] == o.cfg.mask_id:
                o.tokens[b, P + j] = (17 * j + 3 * k + b) % (o.cfg.vocab - 1)
                break


def test_Kp_Kr_one_is_the_uncached_model():
    """K_p = K_r = 1: every step refreshes everything (Sec. 3.2 items 1-2)."""
    cfg = GQA_TINY
    o, w = make(cfg, B=1)
    K = 4
    for k in range(K, 0, -1):
        r = o.step_scheduled(k, K, 1, 1, rho=0.3)
        hid, _, _ = textbook_forward(cfg, w, o.tokens[0])
        assert rel_l2(r.hidden[0], hid[o.P:]) < 1e-12
        unmask_some(o, k)


@pytest.mark.parametrize("refresh_prompt", [False, True])
def test_rho_one_equals_refresh(refresh_prompt):
    """All rows selected: the adaptive update is a response refresh; together
    with a prompt refresh it is the full step (Sec. 3.2.2)."""
    cfg = GQA_TINY
    a, _ = make(cfg, B=2)
    b, _ = make(cfg, B=2)
    for o in (a, b):
        o.step(True, True)
        unmask_some(o, 1)
    ra = a.step(refresh_prompt, False, rho=1.0)
    rb = b.step(refresh_prompt, True)
    assert rel_l2(ra.hidden, rb.hidden) < 1e-13
    for l in range(cfg.n_layers):
        for ca, cb in ((a.Kc, b.Kc), (a.Vc, b.Vc), (a.Ac, b.Ac), (a.Fc, b.Fc)):
            assert rel_l2(ca[l], cb[l]) < 1e-13
        assert np.array_equal(ra.selected[l], np.tile(np.arange(a.R), (2, 1)))


def test_rho_zero_leaves_caches_untouched():
    """Fully cached state (discussion of Fig. 8): nothing is projected, nothing
    is written; the output is the embeddings plus the cached layer outputs."""
    cfg = GQA_TINY
    o, w = make(cfg, B=1)
    o.step(True, True)
    unmask_some(o, 2)
    before = [[c[l].copy() for l in range(cfg.n_layers)] for c in (o.Kc, o.Vc, o.Ac, o.Fc)]
    macs_before = dict(o.macs)
    r = o.step(False, False, rho=0.0)
    for c, snap in zip((o.Kc, o.Vc, o.Ac, o.Fc), before):
        for l in range(cfg.n_layers):
            assert np.array_equal(c[l], snap[l])
    P = o.P
    x = w["embed"][o.tokens[0, P:]].astype(np.float64)
    for l in range(cfg.n_layers):
        x = (x + o.Ac[l][0, P:]) + o.Fc[l][0, P:]
    assert np.array_equal(r.hidden[0], x)
    assert all(o.macs[k] == macs_before[k] for k in ("proj", "attn", "ffn"))
    assert all(s is None for s in r.sim) and all(s.shape == (1, 0) for s in r.selected)


def test_idempotent_partial_step():
    """Unchanged tokens: every similarity is 1 and K / AttnOut / FFNOut stay."""
    cfg = GQA_TINY
    o, _ = make(cfg, B=1)
    o.step(True, True)
    before = [[c[l].copy() for l in range(cfg.n_layers)] for c in (o.Kc, o.Vc, o.Ac, o.Fc)]
    r = o.step(False, False, rho=0.25)
    for l in range(cfg.n_layers):
        np.testing.assert_allclose(r.sim[l], 1.0, atol=1e-6)
        assert np.array_equal(r.selected[l][0], np.arange(O.k_selected(0.25, o.R)))  # ties -> lowest index
    for c, snap in zip((o.Kc, o.Vc, o.Ac, o.Fc), before):
        for l in range(cfg.n_layers):
            assert rel_l2(c[l], snap[l]) < 1e-12


def test_partial_step_writes_V_everywhere_and_the_rest_only_at_selected_rows():
    cfg = GQA_TINY
    o, w = make(cfg, B=2, scale=3.0)
    o.step(True, True)
    unmask_some(o, 1)
    unmask_some(o, 2)
    before = [[c[l].copy() for l in range(cfg.n_layers)] for c in (o.Kc, o.Vc, o.Ac, o.Fc)]
    r = o.step(False, False, rho=0.5)
    P, R = o.P, o.R
    ksel = O.k_selected(0.5, R)
    for l in range(cfg.n_layers):
        for b in range(2):
            S = r.selected[l][b]
            assert len(S) == ksel and len(set(S.tolist())) == ksel
            rest = np.setdiff1d(np.arange(R), S)
            # prompt cache untouched
            for c, snap in zip((o.Kc, o.Vc, o.Ac, o.Fc), before):
                assert np.array_equal(c[l][b, :P], snap[l][b, :P])
            # K, AttnOut, FFNOut untouched outside S, changed inside S
            for c, snap in zip((o.Kc, o.Ac, o.Fc), (before[0], before[2], before[3])):
                assert np.array_equal(c[l][b, P + rest], snap[l][b, P + rest])
            # selection really is the lowest-similarity set
            s = r.sim[l][b]
            assert s[S].max() <= s[rest].min() + 2.0 ** -20
    # layer 0: cached V equals the fresh projection of ALL response rows
    for b in range(2):
        x = w["embed"][o.tokens[b, P:]].astype(np.float64)
        v = O.rmsnorm(x, np.ones(cfg.d_model), cfg.rms_eps) @ w["layers.0.wv"].astype(np.float64).T
        assert rel_l2(o.Vc[0][b, P:], v) < 1e-13
        changed = np.nonzero(np.abs(o.Vc[0][b, P:] - before[1][0][b, P:]).max(-1) > 0)[0]
        assert set(changed.tolist()) <= set(r.selected[0][b].tolist())  # at layer 0 only re-embedded rows move
        assert len(changed) == 2


def test_selected_queries_see_fresh_V_and_stale_K():
    """Cache writes precede attention (reading of Sec. 3.2.2): a recomputed row
    attends to the new V of all response rows, new K of selected rows, old K of
    the others, and the cached prompt K / V."""
    cfg = synth.ModelConfig(n_layers=1, d_model=96, n_heads=6, n_kv_heads=2, head_dim=16,
                            d_ffn=160, vocab=211, mask_id=210, dtype="fp32")
    o, w = make(cfg, B=1, scale=3.0)
    o.step(True, True)
    P, R, n = o.P, o.R, o.n
    o.tokens[0, P + 2] = 5
    o.tokens[0, P + 6] = 9
    K_old = o.Kc[0][0].copy()
    r = o.step(False, False, rho=0.25)         # k = 2 rows
    S = r.selected[0][0]
    assert sorted(S.tolist()) == [2, 6]
    x = w["embed"][o.tokens[0, P:]].astype(np.float64)
    u = O.rmsnorm(x, 1.0, cfg.rms_eps)
    wq, wk, wv, wo = (w["layers.0." + k].astype(np.float64) for k in ("wq", "wk", "wv", "wo"))
    Vmix = np.concatenate([o.Vc[0][0, :P], u @ wv.T])
    Kmix = K_old.copy()
    Kmix[P + S] = O.rope((u[S] @ wk.T).reshape(-1, 2, 16), P + S, cfg.rope_theta).reshape(len(S), -1)
    q = O.rope((u[S] @ wq.T).reshape(-1, 6, 16), P + S, cfg.rope_theta)
    tq = torch.from_numpy(q).transpose(0, 1)[None]
    tk = torch.from_numpy(Kmix.reshape(n, 2, 16)).repeat_interleave(3, 1).transpose(0, 1)[None]
    tv = torch.from_numpy(Vmix.reshape(n, 2, 16)).repeat_interleave(3, 1).transpose(0, 1)[None]
    att = F.scaled_dot_product_attention(tq, tk, tv)[0].transpose(0, 1).reshape(len(S), -1).numpy()
    assert rel_l2(o.Ac[0][0, P + S], att @ wo.T) < 1e-12


def test_prompt_isolation_until_next_prompt_refresh():
    """The prompt cache is reused between prompt refreshes (Sec. 3.2.1): editing
    prompt ids changes nothing until refresh_prompt is set."""
    cfg = GQA_TINY
    a, _ = make(cfg)
    b, _ = make(cfg)
    a.step(True, True)
    b.step(True, True)
    b.tokens[0, :b.P] = (b.tokens[0, :b.P] + 1) % (cfg.vocab - 1)
    for rp, rr, rho in ((False, False, 0.25), (False, True, 0.0)):
        ra, rb = a.step(rp, rr, rho), b.step(rp, rr, rho)
        assert np.array_equal(ra.hidden, rb.hidden)
    ra, rb = a.step(True, False, 0.25), b.step(True, False, 0.25)
    assert rel_l2(ra.hidden, rb.hidden) > 1e-3


def test_error_resets_at_joint_refresh():
    """Sec. A.8: the deviation from the uncached model is reset at a refresh
    (exactly, when the prompt cache is fresh too) and non-zero in between."""
    cfg = GQA_TINY
    o, w = make(cfg, scale=4.0)
    K, Kp, Kr = 8, 4, 2
    errs = {}
    for k in range(K, 0, -1):
        r = o.step_scheduled(k, K, Kp, Kr, rho=0.25)
        hid, _, _ = textbook_forward(cfg, w, o.tokens[0])
        errs[k] = rel_l2(r.hidden[0], hid[o.P:])
        unmask_some(o, k)
    assert errs[8] < 1e-12 and errs[4] < 1e-12
    assert all(errs[k] > 1e-6 for k in (7, 5, 3, 1))
    assert errs[6] > 1e-9          # response refreshed against a stale prompt cache: smaller, not zero
    assert errs[6] < errs[7] and errs[2] < errs[3]


# --------------------------------------------------------------------------
# selection (Sec. 3.2.2) against brute force
# --------------------------------------------------------------------------
def brute_force_lowest(sim, k):
    keys = [(int(round(float(np.float32(s)) * 2 ** 20)), j) for j, s in enumerate(sim)]
    return sorted(j for _, j in sorted(keys)[:k])


@pytest.mark.parametrize("seed", range(6))
def test_selection_matches_brute_force(seed):
    rng = np.random.default_rng(seed)
    R = int(rng.integers(1, 70))
    sim = rng.uniform(-1, 1, R).astype(np.float32)
    if seed % 2:                                   # engineered ties, incl. exact 1.0 and sub-quantum noise
        sim[rng.integers(0, R, R // 2)] = 1.0
        sim[rng.integers(0, R, R // 3)] = np.float32(1.0 - 2.0 ** -24)
        sim[rng.integers(0, R, 3)] = sim[0]
    for k in (0, 1, R // 4, R // 2, R):
        got = O.select_lowest(sim, k)
        assert got.tolist() == brute_force_lowest(sim, k)
        assert len(got) == k


def test_k_selected_floor_and_ceil():
    assert O.k_selected(0.25, 256) == 64
    assert O.k_selected(0.25, 32) == 8
    assert O.k_selected(0.1, 32) == 3 and O.k_selected(0.1, 32, "ceil") == 4
    assert O.k_selected(0.1, 512) == 51 and O.k_selected(0.1, 512, "ceil") == 52
    assert O.k_selected(0.5, 256, "ceil") == 128 and O.k_selected(0.3, 10) == 3   # 0.3*10 = 2.999.. in binary
    assert O.k_selected(0.0, 99) == 0 and O.k_selected(1.0, 99) == 99


# --------------------------------------------------------------------------
# schedule (Sec. 3.2) -- patterns of the five configurations
# --------------------------------------------------------------------------
def kinds(K, Kp, Kr):
    out = []
    for k in range(K, 0, -1):
        rp, rr = O.schedule(k, K, Kp, Kr)
        out.append("f" if rp and rr else "r" if rr else "m" if rp else "p")
    return "".join(out)


def test_schedule_patterns():
    assert kinds(8, 4, 2) == "fprpfprp"
    for (K, Kp, Kr), want in {(256, 100, 6): (1, 42, 2, 211), (256, 50, 8): (2, 30, 4, 220),
                              (32, 100, 4): (1, 7, 0, 24), (512, 100, 8): (3, 61, 3, 445)}.items():
        s = kinds(K, Kp, Kr)
        assert (s.count("f"), s.count("r"), s.count("m"), s.count("p")) == want
    assert kinds(5, 1, 1) == "fffff"
    # literal count-down residues of k (a count-up reading would give "fprpfpr")
    assert kinds(7, 4, 2) == "frpfprp"
    assert O.schedule(200, 256, 100, 6) == (True, False) and O.schedule(252, 256, 100, 6) == (False, True)


# --------------------------------------------------------------------------
# storage (Sec. A.9) and cost terms (Sec. A.7)
# --------------------------------------------------------------------------
def test_cache_storage_is_four_tensors_per_layer():
    cfg = synth.TINY
    o, _ = make(cfg, B=1, P=64, R=32)
    assert o.cache_elements() == 4 * (64 + 32) * cfg.d_model * cfg.n_layers
    big = synth.LLADA_8B
    n = 512 + 256
    assert 2 * 4 * big.n_layers * n * big.d_model == 805306368       # 0.81 GB in bf16, "<1 GB"


def test_mac_counts_match_closed_form_terms():
    """MHA model: counted multiply-accumulates x2 against Sec. A.7.  Two stated
    deltas: the paper's partial term counts V twice for selected rows
    (2 r d^2 + 8 rhat d^2), and no term has the LM head."""
    cfg = synth.ModelConfig(n_layers=3, d_model=64, n_heads=4, n_kv_heads=4, head_dim=16,
                            d_ffn=176, vocab=97, mask_id=96, dtype="fp32")
    P, R = 20, 12
    n, d, m, T = P + R, cfg.d_model, cfg.d_ffn, cfg.n_layers
    o, _ = make(cfg, P=P, R=R)

    def body():
        return 2 * (o.macs["proj"] + o.macs["attn"] + o.macs["ffn"])

    o.step(True, True)
    assert body() == O.flops_full_step(T, n, d, m)
    assert 2 * o.macs["lm_head"] == 2 * R * d * cfg.vocab
    o.macs = dict.fromkeys(o.macs, 0)
    o.step(False, True)
    assert body() == O.flops_response_refresh(T, n, R, d, m)
    o.macs = dict.fromkeys(o.macs, 0)
    o.step(False, False, rho=0.25)
    rhat = 3
    assert body() == O.flops_partial(T, n, R, rhat, d, m) - T * 2 * rhat * d * d


# --------------------------------------------------------------------------
# closed forms for the elementary operations
# --------------------------------------------------------------------------
def test_rmsnorm_closed_forms():
    x = np.full((3, 8), 2.0)
    np.testing.assert_allclose(O.rmsnorm(x, np.ones(8), 0.0), 1.0)
    np.testing.assert_allclose(O.rmsnorm(x, np.arange(8.0), 12.0), np.tile(np.arange(8.0) * 0.5, (3, 1)))
    y = np.random.default_rng(0).normal(size=(5, 16))
    ref = F.rms_norm(torch.from_numpy(y), (16,), torch.ones(16, dtype=torch.float64) * 1.5, 1e-5).numpy()
    np.testing.assert_allclose(O.rmsnorm(y, 1.5, 1e-5), ref, rtol=1e-13)


def test_rope_closed_forms():
    rng = np.random.default_rng(1)
    hd = 8
    q, k = rng.normal(size=(1, 1, hd)), rng.normal(size=(1, 1, hd))
    np.testing.assert_allclose(O.rope(q, np.array([0]), 10000.0), q)          # position 0: identity
    r = O.rope(q, np.array([5]), 10000.0)
    np.testing.assert_allclose(np.linalg.norm(r), np.linalg.norm(q))          # rotation
    # pair (0, hd/2) turns by `pos` radians, pair (i, i+hd/2) by pos * theta^(-2i/hd)
    for i in range(hd // 2):
        ang = 5 * 10000.0 ** (-2 * i / hd)
        want = np.array([[math.cos(ang), -math.sin(ang)], [math.sin(ang), math.cos(ang)]]) @ \
            np.array([q[0, 0, i], q[0, 0, i + hd // 2]])
        np.testing.assert_allclose([r[0, 0, i], r[0, 0, i + hd // 2]], want, rtol=1e-12)
    # scores depend on the position difference only
    d1 = (O.rope(q, np.array([7]), 100.0) * O.rope(k, np.array([3]), 100.0)).sum()
    d2 = (O.rope(q, np.array([14]), 100.0) * O.rope(k, np.array([10]), 100.0)).sum()
    np.testing.assert_allclose(d1, d2, rtol=1e-12)


def test_attention_closed_forms():
    rng = np.random.default_rng(2)
    n, Hkv, H, hd = 9, 2, 4, 8
    q = rng.normal(size=(3, H, hd))
    V = rng.normal(size=(n, Hkv, hd))
    K_same = np.tile(rng.normal(size=(1, Hkv, hd)), (n, 1, 1))
    out = O.attention(q, K_same, V, Hkv).reshape(3, H, hd)      # equal keys: uniform weights -> mean of V
    for h in range(H):
        np.testing.assert_allclose(out[:, h], np.tile(V[:, h // 2].mean(0), (3, 1)), rtol=1e-12)
    K = rng.normal(size=(n, Hkv, hd))
    K[4] *= 0
    K[4, :, 0] = 1e4                                            # one dominant key: output = its value
    q[..., 0] = 1.0
    out = O.attention(q, K, V, Hkv).reshape(3, H, hd)
    for h in range(H):
        np.testing.assert_allclose(out[:, h], np.tile(V[4, h // 2], (3, 1)), rtol=1e-9)


def test_cosine_closed_forms():
    a = np.array([[1.0, 0, 0], [1, 1, 0], [2, 0, 0], [1, 2, 3], [0, 0, 0]])
    b = np.array([[0.0, 1, 0], [1, 0, 0], [5, 0, 0], [-1, -2, -3], [1, 0, 0]])
    np.testing.assert_allclose(O.cosine_rows(a, b), [0, 1 / math.sqrt(2), 1, -1, 0], atol=1e-7)
    x = np.random.default_rng(3).normal(size=(4, 33))
    y = np.random.default_rng(4).normal(size=(4, 33))
    ref = F.cosine_similarity(torch.from_numpy(x), torch.from_numpy(y), dim=-1).numpy()
    np.testing.assert_allclose(O.cosine_rows(x, y), ref, rtol=1e-6)
    np.testing.assert_allclose(O.cosine_rows(3.0 * x, 0.5 * y), ref, rtol=1e-6)   # scale invariant


def test_silu():
    x = np.linspace(-6, 6, 25)
    np.testing.assert_allclose(O.silu(x), F.silu(torch.from_numpy(x)).numpy(), rtol=1e-13)


# --------------------------------------------------------------------------
# remasking (Eq. 5) and generation
# --------------------------------------------------------------------------
def test_remask_takes_highest_confidence_masked_positions_of_the_block():
    M = 99
    tok = np.array([M, 5, M, M, M, M, M, M])
    x0 = np.arange(10, 18)
    conf = np.array([0.9, 0.99, 0.2, 0.7, 0.7, 0.1, 0.95, 0.3], np.float32)
    out = O.remask_low_confidence(tok, x0, conf, M, 0, 6, 2)
    assert out.tolist() == [10, 5, M, 13, M, M, M, M]           # 0.9 and the FIRST 0.7; position 6 is outside
    out = O.remask_low_confidence(tok, x0, conf, M, 4, 4, 10)   # more than available: all four
    assert out.tolist() == [M, 5, M, M, 14, 15, 16, 17]
    assert O.remask_low_confidence(tok, x0, conf, M, 0, 8, 0).tolist() == tok.tolist()


def test_block_plan():
    assert [O.block_plan(t, 8, 32, 32) for t in range(8)] == [(0, 4)] * 8
    plan = [O.block_plan(t, 256, 256, 32) for t in range(256)]
    assert plan[0] == (0, 1) and plan[31] == (0, 1) and plan[32] == (32, 1) and plan[255] == (224, 1)
    plan = [O.block_plan(t, 6, 16, 8) for t in range(6)]         # 8 tokens over 3 steps: 3, 3, 2
    assert plan == [(0, 3), (0, 3), (0, 2), (8, 3), (8, 3), (8, 2)]


def test_generate_tiny_config_invariants():
    wl = synth.WORKLOADS["tiny"]
    o, _ = make(wl.model, B=1, P=wl.prompt_len, R=wl.gen_len)
    trace = []
    prompt = o.tokens[:, :wl.prompt_len].copy()
    out = o.generate(wl.steps, wl.Kp, wl.Kr, wl.rho, wl.block_len, trace=trace)
    M = wl.model.mask_id
    assert (out[:, wl.prompt_len:] != M).all()                  # K steps end mask-free
    assert np.array_equal(out[:, :wl.prompt_len], prompt)
    prev = np.full(wl.gen_len, M)
    for k, r, toks in trace:
        cur = toks[0, wl.prompt_len:]
        changed = np.nonzero(cur != prev)[0]
        assert len(changed) == 4                                 # 4 tokens per step
        assert (prev[changed] == M).all()                        # only masked positions change
        assert np.array_equal(cur[changed], r.x0[0][changed])
        still = np.nonzero(prev == M)[0]
        kept = np.setdiff1d(still, changed)
        if len(kept):
            assert r.conf[0][changed].min() >= r.conf[0][kept].max()
        prev = cur.copy()
    # per-layer selection sizes follow floor(rho * L) on adaptive steps
    for k, r, _ in trace:
        rp, rr = O.schedule(k, wl.steps, wl.Kp, wl.Kr)
        want = wl.gen_len if rr else 8
        assert all(s.shape == (1, want) for s in r.selected)


def test_cached_step_before_full_step_is_an_error():
    o, _ = make(GQA_TINY)
    with pytest.raises(RuntimeError):
        o.step(False, False, 0.25)
