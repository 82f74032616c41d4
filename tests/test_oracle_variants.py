"""Pins for the oracle's ablation variants of the adaptive step (Sec. 4.3 selection
strategies, Sec. A.5 selected-only V update, Sec. A.6 L2 metric).  CPU only.
Each variant is tied to what the paper fixes about it: which tensors may change
and where, what the refreshed tensor must equal, brute force for the choice."""
import numpy as np
import pytest

from oracle import dllm_oracle as O
from paper_2506_06295_b200 import synth
from tests.test_oracle_pins import GQA_TINY, make, rel_l2, unmask_some

VARIANTS = [dict(strategy="v_verify", metric="l2"), dict(strategy="v_verify", v_update="selected"),
            dict(strategy="k_verify"), dict(strategy="k_verify", metric="l2"), dict(strategy="random")]


def fresh(o, scores_seed=None):
    if scores_seed is None:
        return None
    return synth.random_uniform((o.cfg.n_layers, o.B, o.R), scores_seed)


def test_l2_score_is_the_negated_euclidean_distance():
    rng = np.random.default_rng(3)
    a, b = rng.standard_normal((5, 7)), rng.standard_normal((5, 7))
    s = O.l2_score_rows(a, b)
    assert s.dtype == np.float32
    assert np.allclose(s, -np.linalg.norm(a - b, axis=1), rtol=1e-6)
    assert O.l2_score_rows(a, a).max() == 0.0
    # the largest distance is selected first
    assert O.select_lowest(s, 1)[0] == int(np.argmax(np.linalg.norm(a - b, axis=1)))


@pytest.mark.parametrize("kw", VARIANTS, ids=lambda k: "-".join(f"{v}" for v in k.values()))
def test_every_variant_with_rho_one_equals_a_refresh(kw):
    cfg = GQA_TINY
    a, _ = make(cfg, B=2, scale=3.0)
    b, _ = make(cfg, B=2, scale=3.0)
    for o in (a, b):
        o.step(True, True)
        unmask_some(o, 1)
    sc = synth.random_uniform((cfg.n_layers, 2, a.R), 5) if kw.get("strategy") == "random" else None
    ra = a.step(False, False, rho=1.0, scores=sc, **kw)
    rb = b.step(False, True)
    assert rel_l2(ra.hidden, rb.hidden) < 1e-12
    for ca, cb in zip((a.Kc, a.Vc, a.Ac, a.Fc), (b.Kc, b.Vc, b.Ac, b.Fc)):
        for l in range(cfg.n_layers):
            assert rel_l2(ca[l], cb[l]) < 1e-12


@pytest.mark.parametrize("kw", VARIANTS, ids=lambda k: "-".join(f"{v}" for v in k.values()))
def test_variant_touches_only_what_it_may(kw):
    cfg = GQA_TINY
    o, w = make(cfg, B=2, scale=3.0)
    o.step(True, True)
    unmask_some(o, 1)
    unmask_some(o, 2)
    before = [[c[l].copy() for l in range(cfg.n_layers)] for c in (o.Kc, o.Vc, o.Ac, o.Fc)]
    strategy = kw.get("strategy", "v_verify")
    sc = synth.random_uniform((cfg.n_layers, 2, o.R), 11) if strategy == "random" else None
    r = o.step(False, False, rho=0.5, scores=sc, **kw)
    P, R = o.P, o.R
    ksel = O.k_selected(0.5, R)
    for l in range(cfg.n_layers):
        for b in range(2):
            S = r.selected[l][b]
            rest = np.setdiff1d(np.arange(R), S)
            assert len(set(S.tolist())) == ksel
            s = r.sim[l][b]
            assert s[S].max() <= s[rest].min() + 2.0 ** -20          # the lowest scores were taken
            if strategy == "random":
                assert np.array_equal(np.sort(np.argsort(sc[l][b], kind="stable")[:ksel]), S)
            for c, snap in zip((o.Kc, o.Vc, o.Ac, o.Fc), before):      # prompt cache untouched
                assert np.array_equal(c[l][b, :P], snap[l][b, :P])
            for c, snap in zip((o.Ac, o.Fc), (before[2], before[3])):  # outputs only at S
                assert np.array_equal(c[l][b, P + rest], snap[l][b, P + rest])
            whole_v = strategy == "v_verify" and kw.get("v_update", "all") == "all"
            if not whole_v:                                            # V only at the selected tokens
                assert np.array_equal(o.Vc[l][b, P + rest], before[1][l][b, P + rest])
            if strategy != "k_verify":                                 # K only at the selected tokens
                assert np.array_equal(o.Kc[l][b, P + rest], before[0][l][b, P + rest])
    # layer 0, where the input of every row is its embedding: what was refreshed equals the fresh projection
    for b in range(2):
        x = w["embed"][o.tokens[b, P:]].astype(np.float64)
        u = O.rmsnorm(x, np.ones(cfg.d_model), cfg.rms_eps)
        v = u @ w["layers.0.wv"].astype(np.float64).T
        k = O.rope((u @ w["layers.0.wk"].astype(np.float64).T).reshape(R, cfg.n_kv_heads, cfg.head_dim),
                   np.arange(P, P + R), cfg.rope_theta).reshape(R, -1)
        S = r.selected[0][b]
        assert rel_l2(o.Vc[0][b, P + S], v[S]) < 1e-13
        assert rel_l2(o.Kc[0][b, P + S], k[S]) < 1e-13
        if strategy == "k_verify":
            assert rel_l2(o.Kc[0][b, P:], k) < 1e-13                   # whole K_r overwritten


def test_k_verify_is_idempotent_and_scores_are_one():
    cfg = GQA_TINY
    o, _ = make(cfg, scale=3.0)
    o.step(True, True)
    unmask_some(o, 1)
    o.step(False, True)
    r = o.step(False, False, rho=0.25, strategy="k_verify")
    for l in range(cfg.n_layers):
        assert np.all(np.abs(r.sim[l] - 1.0) < 1e-6)
    r = o.step(False, False, rho=0.25, strategy="v_verify", metric="l2")
    for l in range(cfg.n_layers):
        assert np.all(np.abs(r.sim[l]) < 1e-6)


def test_selected_only_update_keeps_stale_values_for_the_next_check():
    """Sec. A.5: with the selected-only variant an unselected token keeps its old V,
    so its score at the next step is still measured against the stale vector."""
    cfg = GQA_TINY
    o, _ = make(cfg, scale=3.0)
    o.step(True, True)
    unmask_some(o, 1)
    unmask_some(o, 2)
    r1 = o.step(False, False, rho=0.125, strategy="v_verify", v_update="selected")
    r2 = o.step(False, False, rho=0.125, strategy="v_verify", v_update="selected")
    # layer 0: two rows changed their embedding, one was refreshed per step
    assert (r1.sim[0][0] < 1 - 1e-6).sum() == 2
    assert (r2.sim[0][0] < 1 - 1e-6).sum() == 1
    assert set(r1.selected[0][0].tolist()) != set(r2.selected[0][0].tolist())


def test_unknown_variant_is_rejected():
    o, _ = make(GQA_TINY)
    o.step(True, True)
    with pytest.raises(ValueError):
        o.step(False, False, 0.5, strategy="q_verify")


# ---- cross-layer allocation of the update ratio (Sec. A.4, Table 11) ---------------------------
def test_per_layer_rho_selects_floor_rho_l_R_rows_per_layer_and_uniform_list_equals_scalar():
    cfg = GQA_TINY
    a, _ = make(cfg, B=2, scale=3.0)
    b, _ = make(cfg, B=2, scale=3.0)
    for o in (a, b):
        o.step(True, True)
        unmask_some(o, 1)
    ra = a.step(False, False, rho=[0.5, 0.5])
    rb = b.step(False, False, rho=0.5)
    assert rel_l2(ra.hidden, rb.hidden) == 0.0
    unmask_some(a, 2)
    before = [[c[l].copy() for l in range(cfg.n_layers)] for c in (a.Kc, a.Ac, a.Fc)]
    r = a.step(False, False, rho=[0.375, 0.125])            # the front-heavy allocation of Table 11
    R, P = a.R, a.P
    for l, rho_l in enumerate((0.375, 0.125)):
        k = O.k_selected(rho_l, R)
        assert r.selected[l].shape == (2, k)
        for bb in range(2):
            rest = np.setdiff1d(np.arange(R), r.selected[l][bb])
            for c, snap in zip((a.Kc, a.Ac, a.Fc), before):
                assert np.array_equal(c[l][bb, P + rest], snap[l][bb, P + rest])
    with pytest.raises(ValueError):
        a.step(False, False, rho=[0.25])


def test_per_layer_rho_zero_layer_is_fully_cached():
    cfg = GQA_TINY
    o, _ = make(cfg, scale=3.0)
    o.step(True, True)
    unmask_some(o, 1)
    snap = [c[1].copy() for c in (o.Kc, o.Vc, o.Ac, o.Fc)]
    r = o.step(False, False, rho=[0.5, 0.0])
    assert r.sim[1] is None and r.selected[1].shape == (1, 0)
    for c, s0 in zip((o.Kc, o.Vc, o.Ac, o.Fc), snap):
        assert np.array_equal(c[1], s0)
