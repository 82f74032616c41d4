"""Shared helpers for the parity tests (no arithmetic of the method)."""
import numpy as np


def rel_l2(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def row_rel_max(a, b):
    """Largest per-row relative L2 error over the last axis: one bad row among hundreds moves the global
    figure by little, this one by its full error."""
    a = np.asarray(a, np.float64).reshape(-1, np.shape(a)[-1])
    b = np.asarray(b, np.float64).reshape(-1, np.shape(b)[-1])
    num = np.linalg.norm(a - b, axis=-1)
    den = np.maximum(np.linalg.norm(b, axis=-1), 1e-300)
    return float((num / den).max())


def bf16_round_torch(t):
    import torch
    return t.to(torch.bfloat16).to(torch.float32)


def selection_matches(got_idx, want_idx, sim_oracle, tol=1e-3):
    """Index sets must be equal, except for tokens whose similarity lies within
    `tol` of the k-th threshold (those may legally flip)."""
    got, want = set(np.asarray(got_idx).tolist()), set(np.asarray(want_idx).tolist())
    if got == want:
        return True
    if len(got) != len(want) or sim_oracle is None:
        return False
    s = np.asarray(sim_oracle, np.float64)
    thr = np.sort(s)[len(want) - 1] if len(want) else -np.inf
    diff = got ^ want
    return all(abs(s[j] - thr) <= tol for j in diff)
