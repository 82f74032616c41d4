"""CPU oracle for the cached denoising step of a masked-diffusion transformer.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
CUDA library must compute.  Only the tests, the smoke check and the CPU-baseline
leg of the benchmark may import it; the product path never does.  It shares no
code with the CUDA path and imports nothing from it.

What it follows:
  * model:   "bidirectional Transformer" (Sec. 3.1) with SwiGLU FFN of three
             matmuls (Sec. A.7); pre-norm RMSNorm / RoPE architecture as the
             benchmark configurations state it.
  * sampler: Eqs. 2-5 (all-mask start, greedy estimate, transition S).
  * caching: Sec. 3.2 (workflow items (1)-(3)), Sec. 3.2.1 (prompt cache),
             Sec. 3.2.2 (response refresh, V-verify Eq. 6, bottom-floor(rho*L)
             selection, whole-V overwrite), Sec. A.4 (selection is per layer),
             Sec. A.5 (V overwrite), Sec. A.7 (cost terms), Sec. A.9 (storage).

The method is an approximation (Sec. A.10), so the cached step follows the
algorithm's steps in the paper's order; only the all-refresh step reduces to a
plain definition (the uncached forward), and the tests pin it to one.

Pins (tests/test_oracle_*.py, all CPU): textbook fp64 torch forward for the full
step; K_p = K_r = 1 equals the uncached model; rho = 1 equals a refresh; rho = 0
leaves the caches untouched; idempotence; V overwritten on all response rows, K /
AttnOut / FFNOut only on the selected ones; selection against brute-force
sorting; prompt isolation; storage count (Sec. A.9); multiply-accumulate counts
against the closed-form terms of Sec. A.7; error reset at joint refreshes
(Sec. A.8); remasking invariants; closed forms for RMSNorm, RoPE, softmax
attention and the cosine.  The paper prints no intermediate numeric value, so
beyond these the absolute numerics are "parity unpinned" by paper-printed data.

Arithmetic: numpy, compute type selectable (float64 default; float32 is the
type the benchmark's CPU baseline times).  Matrix products are numpy matmuls;
there is no blocking or fusion.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

SIM_QUANT = float(2 ** 20)   # selection key quantum (ties: see select_lowest)
COS_EPS = 1e-8


# --------------------------------------------------------------------------
# elementary operations
# --------------------------------------------------------------------------
def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """x / sqrt(mean(x^2) + eps) * gain, row-wise over the last axis."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding, rotate-half pairing: element i is paired with i + hd/2
    and the pair is rotated by the angle pos * theta^(-2i/hd).
    x: [rows, heads, hd]; pos: [rows] absolute position in [prompt; response]."""
    hd = x.shape[-1]
    half = hd // 2
    inv_freq = theta ** (-(np.arange(half, dtype=np.float64) * 2.0) / hd)
    ang = pos.astype(np.float64)[:, None] * inv_freq[None, :]
    c = np.cos(ang).astype(x.dtype)[:, None, :]
    s = np.sin(ang).astype(x.dtype)[:, None, :]
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, n_kv_heads: int) -> np.ndarray:
    """Non-causal softmax attention of a set of queries over ALL cached keys
    (Sec. A.7: the queries of the recomputed rows attend to the full sequence).
    q: [a, H, hd]; K, V: [n, Hkv, hd]; query head h uses KV head h // (H/Hkv).
    Returns [a, H*hd]."""
    a, H, hd = q.shape
    G = H // n_kv_heads
    out = np.empty((a, H, hd), dtype=q.dtype)
    scale = 1.0 / math.sqrt(hd)
    for h in range(H):
        kh = h // G
        s = (q[:, h, :] @ K[:, kh, :].T) * scale            # [a, n]
        s = s - s.max(axis=-1, keepdims=True)
        p = np.exp(s)
        p = p / p.sum(axis=-1, keepdims=True)
        out[:, h, :] = p @ V[:, kh, :]
    return out.reshape(a, H * hd)


def cosine_rows(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """Eq. 6: one scalar per token over the whole value vector (all KV heads
    concatenated).  Returned as float32, the precision the selection is taken in."""
    dot = np.sum(a * b, axis=-1)
    den = np.sqrt(np.sum(a * a, axis=-1) * np.sum(b * b, axis=-1))
    return (dot / np.maximum(den, COS_EPS)).astype(np.float32)


def l2_score_rows(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """The alternative metric of Sec. A.6: Euclidean distance between the new and
    the cached vector of a token.  Returned NEGATED (as float32) so that, as with
    the cosine, the least similar tokens have the lowest score."""
    diff = a - b
    return (-np.sqrt(np.sum(diff * diff, axis=-1))).astype(np.float32)


def k_selected(rho: float, R: int, kround: str = "floor") -> int:
    """Number of response tokens updated in an adaptive step: floor(rho * L)
    (Sec. 3.2.2).  'ceil' is the alternative wording of the benchmark statement."""
    if kround == "floor":
        k = int(math.floor(rho * R + 1e-6))
    elif kround == "ceil":
        k = int(math.ceil(rho * R - 1e-6))
    else:
        raise ValueError(kround)
    return max(0, min(R, k))


def select_lowest(sim: np.ndarray, k: int) -> np.ndarray:
    """The k tokens with the lowest similarity (Sec. 3.2.2), ascending index
    order.  The paper is silent on ties; the reading used everywhere here is:
    order by (round(sim * 2^20), index).  Unchanged rows reproduce their cached
    V exactly, so most similarities are 1 up to rounding, and without the
    quantisation rounding noise would decide the set."""
    sim = np.asarray(sim, dtype=np.float32)
    key = np.rint(sim.astype(np.float64) * SIM_QUANT).astype(np.int64)
    idx = np.arange(sim.shape[0])
    order = np.lexsort((idx, key))           # primary key, then index
    return np.sort(order[:k]).astype(np.int32)


def schedule(k: int, K: int, Kp: int, Kr: int) -> tuple[bool, bool]:
    """Which caches are refreshed at denoising step k (counting down K..1):
    everything at k = K (initialisation), the prompt when k = 0 mod K_p, the
    response when k = 0 mod K_r (Sec. 3.2 items (1)-(2), Sec. 3.2.2)."""
    return (k == K) or (k % Kp == 0), (k == K) or (k % Kr == 0)


def remask_low_confidence(tokens_resp: np.ndarray, x0: np.ndarray, conf: np.ndarray, mask_id: int,
                          block_start: int, block_len: int, n_transfer: int) -> np.ndarray:
    """Transition S (Eq. 5) with low-confidence remasking: among the still
    masked positions of the current block keep the n_transfer predictions with
    the highest confidence (ties: lowest position) and leave the rest masked.
    Works on one sequence's response tokens; returns the updated copy."""
    out = np.array(tokens_resp, copy=True)
    cand = [j for j in range(block_start, block_start + block_len) if out[j] == mask_id]
    cand.sort(key=lambda j: (-float(np.float32(conf[j])), j))
    for j in cand[:max(0, n_transfer)]:
        out[j] = x0[j]
    return out


def block_plan(t: int, K: int, R: int, block_len: int) -> tuple[int, int]:
    """Semi-autoregressive plan (Table 12 lists steps / block length / generation
    length): step index t = K - k works on block t // (K / blocks) and unmasks
    block_len / steps_per_block tokens, the remainder spread over the first steps
    of the block.  Returns (block_start, n_transfer)."""
    blocks = R // block_len
    spb = K // blocks
    blk = min(t // spb, blocks - 1)
    i = t - blk * spb
    n_transfer = block_len // spb + (1 if i < block_len % spb else 0)
    return blk * block_len, n_transfer


# --------------------------------------------------------------------------
# the model with its per-layer caches
# --------------------------------------------------------------------------
@dataclass
class StepResult:
    hidden: np.ndarray                  # [B, R, d] residual stream before the final norm
    logits: np.ndarray                  # [B, R, vocab], mask id set to -inf
    x0: np.ndarray                      # [B, R] greedy estimate (Eq. 4)
    conf: np.ndarray                    # [B, R] softmax probability of x0
    selected: list = field(default_factory=list)   # per layer: int32 [B, k] (response-relative)
    sim: list = field(default_factory=list)        # per layer: float32 [B, R] or None


class DLLMOracle:
    """Model p_theta with Prompt Cache C_p and Response Cache C_r (Sec. 3.2):
    per layer K, V [B, n, dkv] and AttnOut, FFNOut [B, n, d]; rows [0, P) are
    C_p, rows [P, n) are C_r.

    compact_prompt_outs=True is the storage variant that the memory limitation of
    Sec. A.10 item (1) invites: AttnOut and FFNOut are kept for the response rows
    only, [B, R, d].  The prompt's AttnOut / FFNOut are never read between prompt
    refreshes (the prompt's residual stream is not carried on those steps) and on
    a prompt refresh they are recomputed before they are used, so within a step
    they live in a temporary and are dropped at the end of the layer."""

    def __init__(self, cfg, weights: dict, batch: int, prompt_len: int, gen_len: int,
                 dtype=np.float64, compact_prompt_outs: bool = False):
        self.cfg = cfg
        self.dt = np.dtype(dtype)
        self.B, self.P, self.R = batch, prompt_len, gen_len
        self.n = prompt_len + gen_len
        self.w = {k: np.asarray(v) for k, v in weights.items()}
        c = cfg
        T, n = c.n_layers, self.n
        dkv, d = c.n_kv_heads * c.head_dim, c.d_model
        self.Kc = [np.zeros((batch, n, dkv), self.dt) for _ in range(T)]
        self.Vc = [np.zeros((batch, n, dkv), self.dt) for _ in range(T)]
        self.compact = bool(compact_prompt_outs)
        rows_out = gen_len if self.compact else n
        self.Ac = [np.zeros((batch, rows_out, d), self.dt) for _ in range(T)]
        self.Fc = [np.zeros((batch, rows_out, d), self.dt) for _ in range(T)]
        self.tokens = np.full((batch, n), c.mask_id, dtype=np.int64)
        self.valid = False
        self.macs = {"proj": 0, "attn": 0, "ffn": 0, "lm_head": 0}

    # -- bookkeeping -------------------------------------------------------
    def cache_elements(self) -> int:
        return sum(a.size for group in (self.Kc, self.Vc, self.Ac, self.Fc) for a in group)

    def set_prompt(self, prompt: np.ndarray) -> None:
        """tokens <- [prompt ; mask x R] (Eq. 2); caches become invalid."""
        prompt = np.asarray(prompt).reshape(self.B, self.P)
        self.tokens[:, :self.P] = prompt
        self.tokens[:, self.P:] = self.cfg.mask_id
        self.valid = False

    def _lin(self, x: np.ndarray, name: str, kind: str) -> np.ndarray:
        W = self.w[name]
        self.macs[kind] += x.shape[0] * W.shape[0] * W.shape[1]
        return x @ W.T.astype(self.dt, copy=False)

    # -- one denoising step --------------------------------------------------
    def step(self, refresh_prompt: bool, refresh_response: bool, rho: float = 0.0,
             kround: str = "floor", forced: dict | None = None, strategy: str = "v_verify",
             metric: str = "cosine", v_update: str = "all", scores=None) -> StepResult:
        """One forward pass under the caching rule.  (True, True) is the
        initialisation / full refresh.  `forced[(layer)] = int array [B, k]`
        replaces the V-verify choice of that layer (used to separate legal tie
        flips from arithmetic differences in parity tests).

        The paper's ablations of the adaptive step (Sec. 4.3, Sec. A.5, Sec. A.6):
          strategy  "v_verify" (default, Eq. 6 on V), "k_verify" (the same test on
                    the post-RoPE K; read symmetrically: K of ALL response rows is
                    projected and overwritten, V only at the selected rows), or
                    "random" (no projection over all rows: the lowest of the given
                    `scores` [T, B, R] are taken, V only at the selected rows);
          metric    "cosine" (default) or "l2" (Sec. A.6);
          v_update  "all" (default: whole V_r overwritten) or "selected" (Sec. A.5:
                    only the selected tokens' V)."""
        if strategy not in ("v_verify", "k_verify", "random") or metric not in ("cosine", "l2") \
                or v_update not in ("all", "selected"):
            raise ValueError("unknown selection variant")
        score_rows = cosine_rows if metric == "cosine" else l2_score_rows
        c, B, P, R, n = self.cfg, self.B, self.P, self.R, self.n
        if not self.valid and not (refresh_prompt and refresh_response):
            raise RuntimeError("cached step before any full step")
        H, Hkv, hd, d = c.n_heads, c.n_kv_heads, c.head_dim, c.d_model
        # rho may be one ratio or one per layer (the cross-layer allocation of Sec. A.4, Table 11)
        rhos = [float(rho)] * c.n_layers if np.ndim(rho) == 0 else [float(r) for r in rho]
        if len(rhos) != c.n_layers:
            raise ValueError("one rho per layer expected")
        ksels = [R if refresh_response else k_selected(r, R, kround) for r in rhos]
        res = StepResult(hidden=np.zeros((B, R, d), self.dt), logits=None, x0=None, conf=None)
        res.selected = [np.zeros((B, ksels[l]), np.int32) for l in range(c.n_layers)]
        res.sim = [np.zeros((B, R), np.float32) if (not refresh_response and ksels[l] > 0) else None
                   for l in range(c.n_layers)]
        logits = np.zeros((B, R, c.vocab), self.dt)

        for b in range(B):
            # 1. carried rows: the response always, the prompt on a prompt refresh
            carried = np.arange(0 if refresh_prompt else P, n)
            E = self.w["embed"]
            x = np.zeros((n, d), self.dt)
            x[carried] = E[self.tokens[b, carried]].astype(self.dt)
            for l in range(c.n_layers):
                p = f"layers.{l}."
                ksel = ksels[l]
                Kc, Vc, Ac, Fc = self.Kc[l][b], self.Vc[l][b], self.Ac[l][b], self.Fc[l][b]
                if self.compact:
                    # the layer works on full-height temporaries whose response rows are the stored ones; the
                    # prompt rows hold nothing until (and unless) this step recomputes them
                    Ac_resp, Fc_resp = Ac, Fc
                    Ac, Fc = np.zeros((n, d), self.dt), np.zeros((n, d), self.dt)
                    Ac[P:], Fc[P:] = Ac_resp, Fc_resp
                # a. pre-attention norm of the carried rows
                u = np.zeros((n, d), self.dt)
                u[carried] = rmsnorm(x[carried], self.w[p + "norm1"].astype(self.dt), c.rms_eps)
                # b-d. which response rows are recomputed
                have_v = np.zeros(n, bool)
                if refresh_response:
                    S = np.arange(R)
                elif ksel == 0:
                    S = np.zeros(0, np.int64)            # fully cached: nothing projected
                elif strategy == "v_verify":
                    v_new = self._lin(u[P:], p + "wv", "proj")          # all R rows
                    s = score_rows(v_new, Vc[P:])                          # Eq. 6 (or Sec. A.6)
                    res.sim[l][b] = s
                    S = select_lowest(s, ksel)
                    if v_update == "all":
                        Vc[P:] = v_new                                      # whole V_r overwritten
                        have_v[P:] = True
                    else:                                                   # Sec. A.5 variant
                        Vc[P + S] = v_new[S]
                        have_v[P + S] = True
                elif strategy == "k_verify":
                    k_new = self._lin(u[P:], p + "wk", "proj").reshape(-1, Hkv, hd)
                    k_new = rope(k_new, np.arange(P, n), c.rope_theta).reshape(R, Hkv * hd)
                    s = score_rows(k_new, Kc[P:])                          # the test of Eq. 6 on K
                    res.sim[l][b] = s
                    S = select_lowest(s, ksel)
                    Kc[P:] = k_new                                          # whole K_r overwritten
                else:                                                       # random selection
                    s = np.asarray(scores[l][b], dtype=np.float32)
                    res.sim[l][b] = s
                    S = select_lowest(s, ksel)
                if forced is not None and l in forced and not refresh_response and ksel > 0:
                    S = np.sort(np.asarray(forced[l])[b].astype(np.int64))
                res.selected[l][b, :len(S)] = S
                # e. active rows: Q, K (and V where not yet projected); caches written first
                act = np.concatenate([np.arange(P) if refresh_prompt else np.zeros(0, np.int64),
                                      P + np.asarray(S, np.int64)]).astype(np.int64)
                if act.size:
                    ua = u[act]
                    q = self._lin(ua, p + "wq", "proj").reshape(-1, H, hd)
                    k = self._lin(ua, p + "wk", "proj").reshape(-1, Hkv, hd)
                    q = rope(q, act, c.rope_theta)
                    k = rope(k, act, c.rope_theta)
                    Kc[act] = k.reshape(-1, Hkv * hd)
                    need_v = act[~have_v[act]]
                    if need_v.size:
                        Vc[need_v] = self._lin(u[need_v], p + "wv", "proj")
                    # f. attention over the UPDATED caches, then O-proj and FFN
                    self.macs["attn"] += 2 * act.size * n * H * hd
                    o = attention(q, Kc.reshape(n, Hkv, hd), Vc.reshape(n, Hkv, hd), Hkv)
                    Ac[act] = self._lin(o, p + "wo", "proj")
                    h = x[act] + Ac[act]
                    hn = rmsnorm(h, self.w[p + "norm2"].astype(self.dt), c.rms_eps)
                    g = self._lin(hn, p + "wg", "ffn")
                    up = self._lin(hn, p + "wu", "ffn")
                    Fc[act] = self._lin(silu(g) * up, p + "wd", "ffn")
                # g. every carried row continues with the available feature version
                x[carried] = (x[carried] + Ac[carried]) + Fc[carried]
                if self.compact:
                    Ac_resp[...], Fc_resp[...] = Ac[P:], Fc[P:]      # the prompt rows are dropped
            # 3. prediction at the response rows (Eqs. 3-4)
            res.hidden[b] = x[P:]
            z = rmsnorm(x[P:], self.w["norm_f"].astype(self.dt), c.rms_eps)
            lg = self._lin(z, "lm_head", "lm_head")
            lg[:, c.mask_id] = -np.inf                   # the estimate is never [MASK]
            logits[b] = lg
        res.logits = logits
        res.x0 = np.argmax(logits, axis=-1).astype(np.int64)          # lowest id on ties
        mx = logits.max(axis=-1, keepdims=True)
        pexp = np.exp(logits - mx)
        res.conf = (1.0 / pexp.sum(axis=-1)).astype(np.float32)       # softmax prob of the argmax
        self.valid = True
        self.last = res
        return res

    def step_scheduled(self, k: int, K: int, Kp: int, Kr: int, rho: float,
                       kround: str = "floor", forced=None) -> StepResult:
        rp, rr = schedule(k, K, Kp, Kr)
        return self.step(rp, rr, rho, kround, forced)

    def remask(self, block_start: int, block_len: int, n_transfer: int) -> None:
        r = self.last
        for b in range(self.B):
            self.tokens[b, self.P:] = remask_low_confidence(
                self.tokens[b, self.P:], r.x0[b], r.conf[b], self.cfg.mask_id,
                block_start, block_len, n_transfer)

    def generate(self, K: int, Kp: int, Kr: int, rho: float, block_len: int,
                 kround: str = "floor", trace: list | None = None) -> np.ndarray:
        """K forward passes at k = K, K-1, ..., 1, each followed by the transition."""
        for k in range(K, 0, -1):
            r = self.step_scheduled(k, K, Kp, Kr, rho, kround)
            bs, nt = block_plan(K - k, K, self.R, block_len)
            self.remask(bs, block_len, nt)
            if trace is not None:
                trace.append((k, r, self.tokens.copy()))
        return self.tokens.copy()


# --------------------------------------------------------------------------
# closed-form cost terms of Sec. A.7 (for the multiply-accumulate pin)
# --------------------------------------------------------------------------
def flops_full_step(T, n, d, m):
    return T * (8 * n * d * d + 4 * n * n * d + 6 * n * d * m)


def flops_response_refresh(T, n, r, d, m):
    return T * (8 * r * d * d + 4 * r * n * d + 6 * r * d * m)


def flops_partial(T, n, r, rhat, d, m):
    return T * (2 * r * d * d + 8 * rhat * d * d + 4 * rhat * n * d + 6 * rhat * d * m)
