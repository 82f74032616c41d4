"""ctypes binding of libdllm_b200.so (the C ABI of include/dllm.h).

Argument marshalling only: every step of the method runs inside the library's
CUDA kernels.  torch is used to allocate device memory and to provide the CUDA
stream.  Importing this module fails loudly if the library has not been built
(`python -m paper_2506_06295_b200.build`); there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# DLLM_B200_LIB names another build of the same library (the timeline build of timeline.py)
LIB_PATH = os.environ.get("DLLM_B200_LIB") or os.path.join(_HERE, "libdllm_b200.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2506_06295_b200.build` "
                      "(there is no CPU or PyTorch fallback for the CUDA path)")
lib = C.CDLL(LIB_PATH)

OK, INVALID_ARG, BAD_STATE, UNSUPPORTED, OUT_OF_MEMORY, CUDA_ERROR, TIMEOUT = range(7)
STATUS_NAMES = ["OK", "INVALID_ARG", "BAD_STATE", "UNSUPPORTED", "OUT_OF_MEMORY", "CUDA_ERROR", "TIMEOUT"]
FP32, BF16 = 0, 1
K_FLOOR, K_CEIL = 0, 1
CACHE_K, CACHE_V, CACHE_ATTN, CACHE_FFN = range(4)
SESSION_DEFAULT, SESSION_COMPACT_CACHE = 0, 1
# classes of dllm_session_profile_read (DLLM_PROF_*), in the header's order
PROF_CLASSES = ["gemm", "attention", "gemm_v", "gemm_qk", "gemm_o", "gemm_gate_up", "gemm_down", "gemm_lm_head",
                "attention_mma", "attention_tcgen05", "vverify", "select_gather", "rope_kscatter", "oproj_epilogue",
                "silu_mul", "layer_tail", "embed_norm", "estimate_merge", "v_scatter"]


class Config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("d_ffn", C.c_int32),
                ("vocab", C.c_int32), ("mask_id", C.c_int32), ("rms_eps", C.c_float),
                ("rope_theta", C.c_float), ("dtype", C.c_int32)]


# every symbol include/dllm.h declares, with its C signature
_P, _I, _F, _SZ = C.c_void_p, C.c_int, C.c_float, C.c_size_t
SIGNATURES = {
    "dllm_last_error": (C.c_char_p, [_P]),
    "dllm_weights_bytes": (_SZ, [C.POINTER(Config)]),
    "dllm_cache_bytes": (_SZ, [C.POINTER(Config), _I, _I, _I]),
    "dllm_workspace_bytes": (_SZ, [C.POINTER(Config), _I, _I, _I]),
    "dllm_cache_bytes_ex": (_SZ, [C.POINTER(Config), _I, _I, _I, _I]),
    "dllm_workspace_bytes_ex": (_SZ, [C.POINTER(Config), _I, _I, _I, _I]),
    "dllm_session_create_ex": (_I, [_P, _I, _I, _I, _I, _P, _P, _P, C.POINTER(_P)]),
    "dllm_tensor_offset": (_I, [C.POINTER(Config), C.c_char_p, C.POINTER(_SZ), C.POINTER(_SZ)]),
    "dllm_step_scheduled_block": (_I, [_P, _I, _I, _I, _I, _F, _I, _I, _I, _P]),
    "dllm_session_predict_block_only": (_I, [_P, _I]),
    "dllm_tensor_blocks": (_I, [C.POINTER(Config), C.c_char_p, C.POINTER(_SZ), C.POINTER(_SZ)]),
    "dllm_model_create": (_I, [C.POINTER(Config), _P, C.POINTER(_P)]),
    "dllm_model_set_tensor": (_I, [_P, C.c_char_p, _P, _SZ]),
    "dllm_model_destroy": (_I, [_P]),
    "dllm_session_create": (_I, [_P, _I, _I, _I, _P, _P, _P, C.POINTER(_P)]),
    "dllm_session_destroy": (_I, [_P]),
    "dllm_session_set_prompt": (_I, [_P, _P, _P]),
    "dllm_step_full": (_I, [_P, _P]),
    "dllm_step_cached": (_I, [_P, _I, _I, _F, _I, _P]),
    "dllm_step_cached_layers": (_I, [_P, _I, _I, _P, _I, _I, _P]),
    "dllm_step_scheduled": (_I, [_P, _I, _I, _I, _I, _F, _I, _P]),
    "dllm_remask_low_confidence": (_I, [_P, _I, _I, _I, _P]),
    "dllm_generate": (_I, [_P, _I, _I, _I, _F, _I, _I, _P]),
    "dllm_sync": (_I, [_P, _P]),
    "dllm_get_tokens": (_I, [_P, _P, _P]),
    "dllm_set_response_tokens": (_I, [_P, _P, _P]),
    "dllm_get_hidden": (_I, [_P, _P, _P]),
    "dllm_get_pred": (_I, [_P, _P, _P, _P]),
    "dllm_get_logits": (_I, [_P, _P, _P]),
    "dllm_get_selected": (_I, [_P, _I, _P, _P, C.POINTER(_I), _P]),
    "dllm_get_cache": (_I, [_P, _I, _I, _P, _P]),
    "dllm_set_cache": (_I, [_P, _I, _I, _P, _P]),
    "dllm_force_selection": (_I, [_P, _I, _P, _I]),
    "dllm_session_set_selection": (_I, [_P, _I, _I, _I]),
    "dllm_set_scores": (_I, [_P, _I, _P, _P]),
    "dllm_launch_count": (C.c_uint64, [_P]),
    "dllm_session_use_graphs": (_I, [_P, _I]),
    "dllm_session_use_simt_gemm": (_I, [_P, _I]),
    "dllm_session_use_pdl": (_I, [_P, _I]),
    "dllm_session_profile": (_I, [_P, _I]),
    "dllm_session_profile_read": (_I, [_P, _I, C.POINTER(C.c_double), C.POINTER(C.c_uint64),
                                       C.POINTER(C.c_double), C.POINTER(C.c_double)]),
    "dllm_gemm_bf16_scratch_bytes": (_SZ, [_I, _I, _I]),
    "dllm_gemm_bf16": (_I, [_P, _P, _P, _I, _I, _I, _P, _P]),
    "dllm_gemm_bf16_planned_scratch_bytes": (_SZ, [_I, _I, _I, _I, _I]),
    "dllm_gemm_bf16_planned": (_I, [_P, _P, _P, _I, _I, _I, _I, _I, _I, _P, _SZ, _P]),
    "dllm_gemm_bf16_pair_scratch_bytes": (_SZ, [_I, _I, _I, _I, _I]),
    "dllm_gemm_bf16_pair": (_I, [_P, _P, _P, _I, _I, _I, _I, _I, _I, _P, _SZ, _P]),
    "dllm_ffn_gate_up_bf16": (_I, [_P, _P, _P, _I, _I, _I, _I, _I, _P]),
    "dllm_gemm_simt": (_I, [_P, _P, _P, _I, _I, _I, _I, _P]),
    "dllm_attention_scratch_bytes": (_SZ, [_I, _I, _I, _I, _I, _I, _I]),
    "dllm_attention": (_I, [_P, _P, _P, _P, _I, _I, _I, _I, _I, _I, _I, _P, _SZ, _P]),
    "dllm_vverify_select": (_I, [_P, _P, _P, _P, _I, _I, _I, _I, _I, _P]),
    "dllm_attention_noalloc": (_I, [_P, _P, _P, _P, _I, _I, _I, _I, _I, _I, _P]),
    "dllm_kernel_status": (_I, [_P]),
    "dllm_debug_set_wait_limit_ns": (_I, [C.c_uint64]),
    "dllm_debug_skip_one_load": (_I, [_I]),
    "dllm_debug_attention_plan": (_I, [_I, _I, _I, _I]),
    "dllm_debug_gemm_plan": (_I, [_I]),
}
for _name, (_res, _args) in SIGNATURES.items():
    _fn = getattr(lib, _name)
    _fn.restype = _res
    _fn.argtypes = _args


class DllmError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"{STATUS_NAMES[status] if 0 <= status < 7 else status}: {msg}")
        self.status = status


def last_error() -> str:
    return (lib.dllm_last_error(None) or b"").decode()


def _check(status: int) -> None:
    if status != OK:
        raise DllmError(status, last_error())


def make_config(cfg) -> Config:
    """From any object with the architecture fields (e.g. synth.ModelConfig)."""
    return Config(cfg.n_layers, cfg.d_model, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim, cfg.d_ffn,
                  cfg.vocab, cfg.mask_id, cfg.rms_eps, cfg.rope_theta, BF16 if cfg.dtype == "bf16" else FP32)


def weights_bytes(cfg) -> int:
    return lib.dllm_weights_bytes(C.byref(make_config(cfg)))


def cache_bytes(cfg, B, P, R, flags: int = 0) -> int:
    return lib.dllm_cache_bytes_ex(C.byref(make_config(cfg)), B, P, R, flags)


def workspace_bytes(cfg, B, P, R, flags: int = 0) -> int:
    return lib.dllm_workspace_bytes_ex(C.byref(make_config(cfg)), B, P, R, flags)


def tensor_offset(cfg, name: str) -> tuple[int, int]:
    off, n = _SZ(), _SZ()
    _check(lib.dllm_tensor_offset(C.byref(make_config(cfg)), name.encode(), C.byref(off), C.byref(n)))
    return off.value, n.value


def tensor_blocks(cfg, name: str) -> tuple[int, int]:
    """(rows per block, bytes between block starts); (0, 0) for a contiguous tensor."""
    rows, stride = _SZ(), _SZ()
    _check(lib.dllm_tensor_blocks(C.byref(make_config(cfg)), name.encode(), C.byref(rows), C.byref(stride)))
    return rows.value, stride.value


def _stream_ptr(stream) -> int:
    if stream is None:
        return 0
    return int(stream.cuda_stream)


def _np_ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


class Model:
    """p_theta bound to a device weight blob (a torch uint8 tensor this object owns)."""

    def __init__(self, cfg, device="cuda:0"):
        import torch
        self.cfg = cfg
        self.ccfg = make_config(cfg)
        self.device = torch.device(device)
        nbytes = weights_bytes(cfg)
        if nbytes == 0:
            raise DllmError(INVALID_ARG, "invalid configuration")
        self.blob = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        h = _P()
        _check(lib.dllm_model_create(C.byref(self.ccfg), C.c_void_p(self.blob.data_ptr()), C.byref(h)))
        self.handle = h

    def set_tensor(self, name: str, values: np.ndarray) -> None:
        a = np.ascontiguousarray(values, dtype=np.float32)
        _check(lib.dllm_model_set_tensor(self.handle, name.encode(), _np_ptr(a), a.size))

    def load(self, weights: dict) -> "Model":
        for name, w in weights.items():
            self.set_tensor(name, w)
        return self

    def tensor_view(self, name: str):
        """torch view of one tensor inside the blob (for filling weights on the device): flat for a
        contiguous tensor, [blocks, rows per block, d_model] (strided) for a row-blocked one."""
        import torch
        off, n = tensor_offset(self.cfg, name)
        is_f32 = name.endswith(("norm1", "norm2", "norm_f")) or self.cfg.dtype != "bf16"
        dt, es = (torch.float32, 4) if is_f32 else (torch.bfloat16, 2)
        rows, stride = tensor_blocks(self.cfg, name)
        if rows == 0:
            return self.blob[off:off + n * es].view(dt)
        d = self.cfg.d_model
        nb = n // (rows * d)
        span = self.blob[off:off + (nb - 1) * stride + rows * d * es].view(dt)
        return span.as_strided((nb, rows, d), (stride // es, d, 1))

    def random_init_on_device(self, seed: int, std: float = 0.02) -> "Model":
        """N(0, std^2) weights and unit norm gains drawn with torch on the device
        (for shapes too large to generate on the host)."""
        import torch
        from .synth import tensor_names
        gen = torch.Generator(device=self.device)
        gen.manual_seed(seed)
        for name, _shape in tensor_names(self.cfg):
            v = self.tensor_view(name)
            if name.endswith(("norm1", "norm2", "norm_f")):
                v.fill_(1.0)
            else:
                per = v[0].numel() if v.dim() > 1 else 1      # a blocked tensor is filled block by block
                chunk = max(1, (1 << 26) // per)
                for s in range(0, v.shape[0], chunk):
                    e = min(v.shape[0], s + chunk)
                    r = torch.randn((e - s) * per, generator=gen, device=self.device, dtype=torch.float32) * std
                    v[s:e] = r.to(v.dtype).view(v[s:e].shape)
        return self

    def close(self):
        if self.handle:
            lib.dllm_model_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Session:
    """Tokens (c, y^(k)) plus the per-layer caches C_p, C_r for B sequences."""

    def __init__(self, model: Model, B: int, P: int, R: int, stream=None, compact_cache: bool = False):
        """compact_cache: AttnOut / FFNOut caches for the response rows only (same results, smaller cache)."""
        import torch
        self.model, self.B, self.P, self.R, self.n = model, B, P, R, P + R
        self.cfg = model.cfg
        self.compact = bool(compact_cache)
        flags = SESSION_COMPACT_CACHE if self.compact else SESSION_DEFAULT
        with torch.cuda.device(model.device):
            self.stream = stream if stream is not None else torch.cuda.Stream(device=model.device)
            cb, wb = cache_bytes(self.cfg, B, P, R, flags), workspace_bytes(self.cfg, B, P, R, flags)
        self.sp = C.c_void_p(_stream_ptr(self.stream))
        if cb == 0 or wb == 0:
            raise DllmError(INVALID_ARG, "B, P and R must be positive")
        self.cache = torch.empty(cb, dtype=torch.uint8, device=model.device)
        self.workspace = torch.empty(wb, dtype=torch.uint8, device=model.device)
        torch.cuda.synchronize(model.device)
        h = _P()
        _check(lib.dllm_session_create_ex(model.handle, B, P, R, flags, C.c_void_p(self.cache.data_ptr()),
                                          C.c_void_p(self.workspace.data_ptr()), self.sp, C.byref(h)))
        self.handle = h

    # -- the calls of the method ------------------------------------------
    def set_prompt(self, prompt: np.ndarray) -> None:
        a = np.ascontiguousarray(prompt, dtype=np.int32).reshape(self.B, self.P)
        _check(lib.dllm_session_set_prompt(self.handle, _np_ptr(a), self.sp))

    def step_full(self) -> None:
        _check(lib.dllm_step_full(self.handle, self.sp))

    def step_cached(self, refresh_prompt: bool, refresh_response: bool, rho: float, kround: int = K_FLOOR) -> None:
        _check(lib.dllm_step_cached(self.handle, int(refresh_prompt), int(refresh_response), rho, kround, self.sp))

    def step_cached_layers(self, refresh_prompt: bool, refresh_response: bool, rhos, kround: int = K_FLOOR) -> None:
        """step_cached with one update ratio per layer (Sec. A.4, Table 11)."""
        a = np.ascontiguousarray(rhos, dtype=np.float32)
        _check(lib.dllm_step_cached_layers(self.handle, int(refresh_prompt), int(refresh_response), _np_ptr(a),
                                           int(a.size), kround, self.sp))

    def step_scheduled(self, k: int, K: int, Kp: int, Kr: int, rho: float, kround: int = K_FLOOR) -> None:
        _check(lib.dllm_step_scheduled(self.handle, k, K, Kp, Kr, rho, kround, self.sp))

    def step_scheduled_block(self, k: int, K: int, Kp: int, Kr: int, rho: float, block_start: int, block_len: int,
                             kround: int = K_FLOOR) -> None:
        """step_scheduled with logits / estimate / confidence only for one block of the response."""
        _check(lib.dllm_step_scheduled_block(self.handle, k, K, Kp, Kr, rho, kround, block_start, block_len, self.sp))

    def predict_block_only(self, on: bool) -> None:
        """generate() predicts only the block each step works on (same tokens, smaller LM head)."""
        _check(lib.dllm_session_predict_block_only(self.handle, int(on)))

    def remask_low_confidence(self, block_start: int, block_len: int, n_transfer: int) -> None:
        _check(lib.dllm_remask_low_confidence(self.handle, block_start, block_len, n_transfer, self.sp))

    def generate(self, K: int, Kp: int, Kr: int, rho: float, block_len: int, kround: int = K_FLOOR) -> None:
        _check(lib.dllm_generate(self.handle, K, Kp, Kr, rho, kround, block_len, self.sp))

    def sync(self) -> None:
        _check(lib.dllm_sync(self.handle, self.sp))

    # -- inspection --------------------------------------------------------
    def tokens(self) -> np.ndarray:
        out = np.empty((self.B, self.n), np.int32)
        _check(lib.dllm_get_tokens(self.handle, _np_ptr(out), self.sp))
        return out

    def set_response_tokens(self, tok: np.ndarray) -> None:
        a = np.ascontiguousarray(tok, dtype=np.int32).reshape(self.B, self.R)
        _check(lib.dllm_set_response_tokens(self.handle, _np_ptr(a), self.sp))

    def hidden(self) -> np.ndarray:
        out = np.empty((self.B, self.R, self.cfg.d_model), np.float32)
        _check(lib.dllm_get_hidden(self.handle, _np_ptr(out), self.sp))
        return out

    def pred(self) -> tuple[np.ndarray, np.ndarray]:
        x0 = np.empty((self.B, self.R), np.int32)
        conf = np.empty((self.B, self.R), np.float32)
        _check(lib.dllm_get_pred(self.handle, _np_ptr(x0), _np_ptr(conf), self.sp))
        return x0, conf

    def logits(self) -> np.ndarray:
        out = np.empty((self.B, self.R, self.cfg.vocab), np.float32)
        _check(lib.dllm_get_logits(self.handle, _np_ptr(out), self.sp))
        return out

    def selected(self, layer: int) -> tuple[np.ndarray, np.ndarray]:
        k = C.c_int()
        _check(lib.dllm_get_selected(self.handle, layer, None, None, C.byref(k), self.sp))
        idx = np.empty((self.B, k.value), np.int32)
        sim = np.empty((self.B, self.R), np.float32)
        _check(lib.dllm_get_selected(self.handle, layer, _np_ptr(idx) if k.value else None, _np_ptr(sim),
                                     C.byref(k), self.sp))
        return idx, sim

    def get_cache(self, layer: int, which: int) -> np.ndarray:
        width = self.cfg.dkv if which in (CACHE_K, CACHE_V) else self.cfg.d_model
        rows = self.R if (self.compact and which in (CACHE_ATTN, CACHE_FFN)) else self.n
        out = np.empty((self.B, rows, width), np.float32)
        _check(lib.dllm_get_cache(self.handle, layer, which, _np_ptr(out), self.sp))
        return out

    def set_cache(self, layer: int, which: int, values: np.ndarray) -> None:
        a = np.ascontiguousarray(values, dtype=np.float32)
        _check(lib.dllm_set_cache(self.handle, layer, which, _np_ptr(a), self.sp))

    def force_selection(self, layer: int, idx) -> None:
        if idx is None:
            _check(lib.dllm_force_selection(self.handle, layer, None, -1))
            return
        a = np.ascontiguousarray(idx, dtype=np.int32).reshape(self.B, -1)
        _check(lib.dllm_force_selection(self.handle, layer, _np_ptr(a), a.shape[1]))

    def set_selection(self, strategy: str = "v_verify", metric: str = "cosine", v_update: str = "all") -> None:
        """Ablation variants of the adaptive step (Sec. 4.3, Sec. A.5, Sec. A.6)."""
        st = {"v_verify": 0, "k_verify": 1, "random": 2}[strategy]
        me = {"cosine": 0, "l2": 1}[metric]
        _check(lib.dllm_session_set_selection(self.handle, st, me, int(v_update == "selected")))

    def set_scores(self, layer: int, scores: np.ndarray) -> None:
        a = np.ascontiguousarray(scores, dtype=np.float32).reshape(self.B, self.R)
        _check(lib.dllm_set_scores(self.handle, layer, _np_ptr(a), self.sp))

    def launch_count(self) -> int:
        return int(lib.dllm_launch_count(self.handle))

    def use_graphs(self, enable: bool) -> None:
        _check(lib.dllm_session_use_graphs(self.handle, int(enable)))

    def use_pdl(self, enable: bool) -> None:
        _check(lib.dllm_session_use_pdl(self.handle, int(enable)))

    def use_simt_gemm(self, enable: bool) -> None:
        _check(lib.dllm_session_use_simt_gemm(self.handle, int(enable)))

    def profile(self, enable: bool) -> None:
        _check(lib.dllm_session_profile(self.handle, int(enable)))

    def profile_read(self, cls: int) -> dict:
        ms, by, fl, cnt = C.c_double(), C.c_double(), C.c_double(), C.c_uint64()
        _check(lib.dllm_session_profile_read(self.handle, cls, C.byref(ms), C.byref(cnt), C.byref(by), C.byref(fl)))
        return {"ms": ms.value, "launches": cnt.value, "bytes": by.value, "flops": fl.value}

    def close(self):
        if getattr(self, "handle", None):
            lib.dllm_session_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# -- kernel-level entry points (device pointers come from torch tensors) -----
def gemm_bf16(A, W, stream=None):
    """C = A @ W.T for torch bf16 CUDA tensors A [M,K], W [N,K]; returns fp32 [M,N]."""
    import torch
    M, K = A.shape
    N = W.shape[0]
    Cm = torch.empty((M, N), dtype=torch.float32, device=A.device)
    sb = lib.dllm_gemm_bf16_scratch_bytes(M, N, K)
    scratch = torch.empty(max(sb, 16), dtype=torch.uint8, device=A.device)
    sp = _stream_ptr(stream if stream is not None else torch.cuda.current_stream(A.device))
    _check(lib.dllm_gemm_bf16(C.c_void_p(A.data_ptr()), C.c_void_p(W.data_ptr()), C.c_void_p(Cm.data_ptr()), M, N, K,
                              C.c_void_p(scratch.data_ptr()), C.c_void_p(sp)))
    return Cm


def gemm_bf16_planned(A, W, act_tile=0, splits=0, stages=0, out=None, scratch=None, stream=None, reduce=True):
    """gemm_bf16 with an explicit launch plan (tuning hook); `out` / `scratch` may be preallocated.
    reduce=False with a split plan leaves the split-K slabs unreduced in `scratch`."""
    import torch
    M, K = A.shape
    N = W.shape[0]
    Cm = out if out is not None else torch.empty((M, N), dtype=torch.float32, device=A.device)
    sb = lib.dllm_gemm_bf16_planned_scratch_bytes(M, N, K, act_tile, splits)
    if scratch is None:
        scratch = torch.empty(max(sb, 16), dtype=torch.uint8, device=A.device)
    sp = _stream_ptr(stream if stream is not None else torch.cuda.current_stream(A.device))
    cptr = Cm.data_ptr() if (reduce or sb == 0) else None
    _check(lib.dllm_gemm_bf16_planned(C.c_void_p(A.data_ptr()), C.c_void_p(W.data_ptr()), C.c_void_p(cptr),
                                      M, N, K, act_tile, splits, stages, C.c_void_p(scratch.data_ptr()),
                                      scratch.numel(), C.c_void_p(sp)))
    return Cm


def gemm_bf16_pair(A, W, act_tile=256, splits=0, stages=0, out=None, scratch=None, stream=None):
    """gemm_bf16 by CTA pairs (cta_group::2); N % 256 == 0."""
    import torch
    M, K = A.shape
    N = W.shape[0]
    Cm = out if out is not None else torch.empty((M, N), dtype=torch.float32, device=A.device)
    sb = lib.dllm_gemm_bf16_pair_scratch_bytes(M, N, K, act_tile, splits)
    if scratch is None:
        scratch = torch.empty(max(sb, 16), dtype=torch.uint8, device=A.device)
    sp = _stream_ptr(stream if stream is not None else torch.cuda.current_stream(A.device))
    _check(lib.dllm_gemm_bf16_pair(C.c_void_p(A.data_ptr()), C.c_void_p(W.data_ptr()), C.c_void_p(Cm.data_ptr()),
                                   M, N, K, act_tile, splits, stages, C.c_void_p(scratch.data_ptr()), scratch.numel(),
                                   C.c_void_p(sp)))
    return Cm


def ffn_gate_up_bf16(A, Wgu, act_tile=0, stages=0, stream=None):
    """silu(A Wg^T) * (A Wu^T) as bf16 [M, d_ffn]; Wgu [2 d_ffn, K] alternates 64 rows of Wg and 64 of Wu."""
    import torch
    M, K = A.shape
    m = Wgu.shape[0] // 2
    out = torch.empty((M, m), dtype=torch.bfloat16, device=A.device)
    sp = _stream_ptr(stream if stream is not None else torch.cuda.current_stream(A.device))
    _check(lib.dllm_ffn_gate_up_bf16(C.c_void_p(A.data_ptr()), C.c_void_p(Wgu.data_ptr()), C.c_void_p(out.data_ptr()),
                                     M, m, K, act_tile, stages, C.c_void_p(sp)))
    return out


def gemm_simt(A, W, stream=None):
    import torch
    M, K = A.shape
    N = W.shape[0]
    Cm = torch.empty((M, N), dtype=torch.float32, device=A.device)
    sp = _stream_ptr(stream if stream is not None else torch.cuda.current_stream(A.device))
    dt = BF16 if A.dtype == torch.bfloat16 else FP32
    _check(lib.dllm_gemm_simt(C.c_void_p(A.data_ptr()), C.c_void_p(W.data_ptr()), C.c_void_p(Cm.data_ptr()), M, N, K,
                              dt, C.c_void_p(sp)))
    return Cm


def attention(q, k, v, B, a, n, H, Hkv, hd, stream=None, split=True):
    """q [B*a, H*hd], k/v [B, n, Hkv*hd] torch CUDA tensors (fp32 or bf16); returns o like q.
    split=False withholds the scratch buffer, so the key range is processed by one CTA per row tile."""
    import torch
    o = torch.empty_like(q)
    sp = _stream_ptr(stream if stream is not None else torch.cuda.current_stream(q.device))
    dt = BF16 if q.dtype == torch.bfloat16 else FP32
    sb = lib.dllm_attention_scratch_bytes(B, a, n, H, Hkv, hd, dt) if split else 0
    scratch = torch.empty(max(sb, 16), dtype=torch.uint8, device=q.device)
    _check(lib.dllm_attention(C.c_void_p(q.data_ptr()), C.c_void_p(k.data_ptr()), C.c_void_p(v.data_ptr()),
                              C.c_void_p(o.data_ptr()), B, a, n, H, Hkv, hd, dt, C.c_void_p(scratch.data_ptr()), sb,
                              C.c_void_p(sp)))
    return o


def attention_noalloc(q, k, v, o, B, a, n, H, Hkv, hd, stream=None):
    """bf16 attention into the caller's output tensor `o` without any device
    allocation: the binding creates no tensor and the library takes its scratch
    from an 8 MiB array built into the shared object (see include/dllm.h).
    For callers that hold only raw buffers and may not allocate.  Calls that
    overlap on the GPU share that scratch and race; keep them on one stream."""
    import torch
    sp = _stream_ptr(stream if stream is not None else torch.cuda.current_stream(q.device))
    _check(lib.dllm_attention_noalloc(C.c_void_p(q.data_ptr()), C.c_void_p(k.data_ptr()), C.c_void_p(v.data_ptr()),
                                      C.c_void_p(o.data_ptr()), B, a, n, H, Hkv, hd, C.c_void_p(sp)))
    return o


def vverify_select(vnew, vcache, k, stream=None):
    """vnew, vcache [B, R, width] torch CUDA tensors; overwrites vcache; returns (sim [B,R], idx [B,k])."""
    import torch
    B, R, width = vnew.shape
    sim = torch.empty((B, R), dtype=torch.float32, device=vnew.device)
    idx = torch.empty((B, max(k, 1)), dtype=torch.int32, device=vnew.device)
    sp = _stream_ptr(stream if stream is not None else torch.cuda.current_stream(vnew.device))
    dt = BF16 if vnew.dtype == torch.bfloat16 else FP32
    _check(lib.dllm_vverify_select(C.c_void_p(vnew.data_ptr()), C.c_void_p(vcache.data_ptr()),
                                   C.c_void_p(sim.data_ptr()), C.c_void_p(idx.data_ptr()), B, R, width, k, dt,
                                   C.c_void_p(sp)))
    return sim, idx[:, :k]


def kernel_status(stream=None) -> None:
    """Raises DllmError(TIMEOUT) if a bounded wait of a kernel-level call gave up since the last read."""
    import torch
    sp = _stream_ptr(stream if stream is not None else torch.cuda.current_stream())
    _check(lib.dllm_kernel_status(C.c_void_p(sp)))


def debug_set_wait_limit_ns(ns: int) -> None:
    """Test hook: limit of the device-side waits (0 restores the 2 s default)."""
    _check(lib.dllm_debug_set_wait_limit_ns(int(ns)))


def debug_skip_one_load(enable: bool) -> None:
    """Test hook: the first CTA of every one-CTA bf16 GEMM launch leaves out one tile copy (its waits run out)."""
    _check(lib.dllm_debug_skip_one_load(int(enable)))
