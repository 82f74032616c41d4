"""Seeded synthetic inputs: model shapes, random-init weights, prompts.

This module holds no arithmetic of the method.  It only draws numbers and
describes shapes, so that the CPU oracle and the CUDA library can be fed the
same buffers.  Neither of them generates its own inputs.

The workloads stand in for the paper's evaluation (Sec. 4.1, Table 12): real
LLaDA-8B / Dream-7B weights and benchmark prompts are not available, so every
matrix is i.i.d. N(0, 0.02^2), norm gains are 1, prompt ids are uniform and
the response starts fully masked (Eq. 2).
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass, asdict, replace

import numpy as np

WEIGHT_SEED = 20250606
WEIGHT_STD = 0.02


@dataclass(frozen=True)
class ModelConfig:
    """Architecture of a bidirectional pre-norm transformer (Sec. A.7 names the
    terms: T layers, hidden d, SwiGLU width m)."""
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    mask_id: int
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0
    dtype: str = "bf16"  # storage type of weights and caches: "fp32" | "bf16"

    @property
    def dq(self) -> int:
        return self.n_heads * self.head_dim

    @property
    def dkv(self) -> int:
        return self.n_kv_heads * self.head_dim

    def as_dict(self) -> dict:
        return asdict(self)

    def with_layers(self, n_layers: int) -> "ModelConfig":
        return replace(self, n_layers=n_layers)


@dataclass(frozen=True)
class Workload:
    """One decoding job: shapes plus the caching hyper-parameters (K_p, K_r, rho)."""
    name: str
    model: ModelConfig
    batch: int
    prompt_len: int
    gen_len: int
    block_len: int
    steps: int
    Kp: int
    Kr: int
    rho: float


TINY = ModelConfig(n_layers=2, d_model=256, n_heads=4, n_kv_heads=4, head_dim=64,
                   d_ffn=688, vocab=1024, mask_id=1023, dtype="fp32")
LLADA_8B = ModelConfig(n_layers=32, d_model=4096, n_heads=32, n_kv_heads=32, head_dim=128,
                       d_ffn=12288, vocab=126464, mask_id=126463, dtype="bf16")
DREAM_7B = ModelConfig(n_layers=28, d_model=3584, n_heads=28, n_kv_heads=4, head_dim=128,
                       d_ffn=18944, vocab=152064, mask_id=152063, dtype="bf16")

WORKLOADS = {
    # the five benchmark configurations, in order
    "tiny": Workload("tiny", TINY, 1, 64, 32, 32, 8, 4, 2, 0.25),
    "llada8b": Workload("llada8b", LLADA_8B, 1, 512, 256, 32, 256, 100, 6, 0.25),
    "dream7b": Workload("dream7b", DREAM_7B, 1, 256, 256, 256, 256, 50, 8, 0.5),
    "long": Workload("long", LLADA_8B, 1, 4096, 32, 32, 32, 100, 4, 0.1),
    "batch16": Workload("batch16", LLADA_8B, 16, 1024, 512, 64, 512, 100, 8, 0.25),
}


def small_bf16_model(n_layers: int = 2, gqa: bool = False) -> ModelConfig:
    """A bf16 model small enough for the oracle to run in seconds but spanning
    several 128-wide GEMM tiles with ragged tails (d and m are not multiples of
    128; 320 = 5*64)."""
    if gqa:
        return ModelConfig(n_layers=n_layers, d_model=448, n_heads=7, n_kv_heads=1, head_dim=64,
                           d_ffn=1216, vocab=2176, mask_id=2175, dtype="bf16")
    return ModelConfig(n_layers=n_layers, d_model=320, n_heads=5, n_kv_heads=5, head_dim=64,
                       d_ffn=832, vocab=1536, mask_id=1535, dtype="bf16")


def tensor_names(cfg: ModelConfig) -> list[tuple[str, tuple[int, ...]]]:
    """Every weight tensor with its shape.  Linear maps are stored
    [out_features, in_features] and applied as y = x W^T."""
    out = [("embed", (cfg.vocab, cfg.d_model)),
           ("lm_head", (cfg.vocab, cfg.d_model)),
           ("norm_f", (cfg.d_model,))]
    for l in range(cfg.n_layers):
        p = f"layers.{l}."
        out += [(p + "norm1", (cfg.d_model,)),
                (p + "wq", (cfg.dq, cfg.d_model)),
                (p + "wk", (cfg.dkv, cfg.d_model)),
                (p + "wv", (cfg.dkv, cfg.d_model)),
                (p + "wo", (cfg.d_model, cfg.dq)),
                (p + "norm2", (cfg.d_model,)),
                (p + "wg", (cfg.d_ffn, cfg.d_model)),
                (p + "wu", (cfg.d_ffn, cfg.d_model)),
                (p + "wd", (cfg.d_model, cfg.d_ffn))]
    return out


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """float32 array -> float32 array whose values are exactly representable in
    bfloat16 (round to nearest even on the upper 16 bits)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 array (already bf16-representable or not) -> uint16 bit patterns."""
    return (round_to_bf16(a).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def make_tensor(cfg: ModelConfig, name: str, shape: tuple[int, ...], seed: int = WEIGHT_SEED) -> np.ndarray:
    """One weight tensor as float32 (bf16-representable when cfg.dtype == 'bf16').
    Each tensor has its own counter-based stream, so any subset can be drawn
    without drawing the rest."""
    if name.endswith(("norm1", "norm2", "norm_f")):
        return np.ones(shape, dtype=np.float32)
    key = zlib.crc32(name.encode()) & 0xFFFFFFFF
    rng = np.random.Generator(np.random.Philox(key=[seed, key]))
    w = rng.standard_normal(shape, dtype=np.float32) * np.float32(WEIGHT_STD)
    if cfg.dtype == "bf16":
        w = round_to_bf16(w)
    return w


def make_weights(cfg: ModelConfig, seed: int = WEIGHT_SEED) -> dict[str, np.ndarray]:
    return {name: make_tensor(cfg, name, shape, seed) for name, shape in tensor_names(cfg)}


def make_prompt(cfg: ModelConfig, batch: int, prompt_len: int, seed: int = 1) -> np.ndarray:
    """int32 [batch, prompt_len], ids uniform on [0, vocab-2]; the mask id
    (vocab-1 in every configuration here) never appears in a prompt."""
    rows = []
    for b in range(batch):
        rng = np.random.Generator(np.random.Philox(key=[seed + b, 0x70726F6D]))
        hi = cfg.vocab - 1 if cfg.mask_id == cfg.vocab - 1 else cfg.vocab
        ids = rng.integers(0, hi, size=prompt_len, dtype=np.int64)
        if cfg.mask_id != cfg.vocab - 1:
            ids = np.where(ids == cfg.mask_id, (ids + 1) % cfg.vocab, ids)
        rows.append(ids.astype(np.int32))
    return np.stack(rows)


def random_uniform(shape, seed: int, lo: float = 0.0, hi: float = 1.0) -> np.ndarray:
    """Plain seeded uniforms for kernel-level tests."""
    rng = np.random.Generator(np.random.Philox(key=[seed, 0x756E6966]))
    return (rng.random(shape, dtype=np.float32) * np.float32(hi - lo) + np.float32(lo)).astype(np.float32)


def random_normal(shape, seed: int, std: float = 1.0) -> np.ndarray:
    rng = np.random.Generator(np.random.Philox(key=[seed, 0x6E6F726D]))
    return rng.standard_normal(shape, dtype=np.float32) * np.float32(std)
