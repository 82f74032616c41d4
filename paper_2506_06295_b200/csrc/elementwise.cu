// Memory-bound kernels of the cached denoising step: embedding, RMSNorm,
// V-verify (Eq. 6) with the whole-V overwrite, bottom-k selection, row gather,
// RoPE + K scatter, cache scatters, SwiGLU gate, residual assembly, greedy
// estimate with confidence (Eq. 4) and the low-confidence transition (Eq. 5).
//
// All of them are one pass over their rows with 16-byte vector accesses, fp32
// arithmetic and warp-shuffle reductions.  Split-K partial sums of the
// preceding GEMM are reduced here, in slab order, so the GEMM never needs
// atomics and every row's value is independent of which other rows were in the
// same launch.
#include <algorithm>

#include "internal.h"
#include "tma.cuh"

namespace dllm {

#define DLLM_DISPATCH(dtype, ...)                 \
  do {                                            \
    if ((dtype) == 0) {                           \
      using T = float;                            \
      __VA_ARGS__;                                \
    } else {                                      \
      using T = __nv_bfloat16;                    \
      __VA_ARGS__;                                \
    }                                             \
  } while (0)

// ------------------------------------------------------------------ four-wide helpers
template <typename T>
__device__ __forceinline__ void store4(T* p, const float (&v)[4]);
template <>
__device__ __forceinline__ void store4<float>(float* p, const float (&v)[4]) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
template <>
__device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16* p, const float (&v)[4]) {
  const __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
  *reinterpret_cast<uint2*>(p) = make_uint2(*reinterpret_cast<const uint32_t*>(&a), *reinterpret_cast<const uint32_t*>(&b));
}
// Sum of the slabs of four consecutive columns, slab 0 first; up to four loads in flight.
__device__ __forceinline__ void sum_partials4(const Partials& part, int row, int col, float (&v)[4]) {
  const int n = part.count(row, col);
  const float* base = part.p + (size_t)row * part.N + col;
  v[0] = v[1] = v[2] = v[3] = 0.f;
  for (int s = 0; s < n; s += 4) {
    float4 t[4];
#pragma unroll
    for (int q = 0; q < 4; ++q)
      t[q] = __ldcg(reinterpret_cast<const float4*>(base + (size_t)min(s + q, n - 1) * part.split_stride));
#pragma unroll
    for (int q = 0; q < 4; ++q)
      if (s + q < n) {
        v[0] += t[q].x; v[1] += t[q].y; v[2] += t[q].z; v[3] += t[q].w;
      }
  }
}

// ------------------------------------------------------------------ streaming forms for many rows
// With thousands of carried rows (batched serving) the one-row-per-CTA kernels above leave HBM idle while a CTA
// reduces and stores: two rows per SM in flight, nothing requested meanwhile.  The streaming forms run one CTA
// per SM for the whole launch: a producer thread fetches the rows of the CTA (blockIdx.x, + gridDim.x, ...) by
// untiled bulk copies into a ring of shared-memory stages, ahead of four consumer warps that each take a whole
// row (no block barrier: lane-local sums and one warp reduction per row) and write its results straight to
// global memory.  Split-K slabs are not supported here (S = 1: with this many rows no projection is split).
constexpr int STREAM_CONSUMERS = 4;                 // warps 1..4; warp 0 produces
constexpr int STREAM_THREADS = 32 * (1 + STREAM_CONSUMERS);
constexpr int STREAM_MAX_STAGES = 12;

// End of a layer, streaming: see tail_kernel.  Stage = [x row fp32 | AttnOut row | FFN row (fp32 projection
// result of an active row, or the cached row)].
template <typename T>
__global__ void __launch_bounds__(STREAM_THREADS, 1)
    tail_stream_kernel(const float* __restrict__ part, const int32_t* __restrict__ inv, float* __restrict__ x,
                       OutRows Ac, OutRows Fc, const float* __restrict__ gain, T* __restrict__ u, Geo g, int c0, int c1,
                       float eps, int stages, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[STREAM_MAX_STAGES], empty_bar[STREAM_MAX_STAGES];
  __shared__ int meta[STREAM_MAX_STAGES];
  __shared__ int abort_flag;
  const int d = g.d, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t xb = (uint32_t)d * 4, ab = (uint32_t)d * sizeof(T), fb = (uint32_t)d * 4;
  const uint32_t stage_bytes = xb + ab + fb;
  const uint32_t base = (smem_u32(smem_raw) + 127u) & ~127u;
  uint8_t* base_gen = smem_raw + (base - smem_u32(smem_raw));
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    mbar_fence_init();
  }
  __syncthreads();
  pdl_wait();
  pdl_trigger();
  volatile int* abortp = &abort_flag;
  const int n_rows = c1 - c0;
  const int my_rows = (int)blockIdx.x < n_rows ? (n_rows - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  bool ok = true;
  if (warp == 0) {
    if (lane == 0) {
      for (int i = 0; i < my_rows; ++i) {
        const int s = i % stages, c = c0 + blockIdx.x + i * gridDim.x;
        if (i >= stages && !mbar_wait(smem_u32(&empty_bar[s]), (uint32_t)(i / stages - 1) & 1u, abortp)) {
          ok = false;
          break;
        }
        const int r = inv ? inv[c] : -1;
        meta[s] = r;
        const uint32_t dst = base + s * stage_bytes, bar = smem_u32(&full_bar[s]);
        mbar_expect_tx(bar, xb + ab + (r >= 0 ? fb : ab));
        bulk_load_1d(dst, x + (size_t)c * d, xb, bar);
        bulk_load_1d(dst + xb, Ac.row<T>(c, g), ab, bar);
        if (r >= 0)
          bulk_load_1d(dst + xb + ab, part + (size_t)r * d, fb, bar);
        else
          bulk_load_1d(dst + xb + ab, Fc.row<T>(c, g), ab, bar);
      }
    }
  } else {
    const int w = warp - 1;
    for (int i = w; i < my_rows; i += STREAM_CONSUMERS) {
      const int s = i % stages, c = c0 + blockIdx.x + i * gridDim.x;
      ok = mbar_wait(smem_u32(&full_bar[s]), (uint32_t)(i / stages) & 1u, abortp);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const int r = meta[s];
      float* xs = reinterpret_cast<float*>(base_gen + (size_t)s * stage_bytes);
      const T* as = reinterpret_cast<const T*>(base_gen + (size_t)s * stage_bytes + xb);
      const uint8_t* fs = base_gen + (size_t)s * stage_bytes + xb + ab;
      float* xr = x + (size_t)c * d;
      T* frow = Fc.row<T>(c, g);
      float ss = 0.f;
      for (int j = lane * 8; j < d; j += 256) {
        float xv[8], a[8], f[8];
        Vec8<float>::load(xs + j, xv);
        Vec8<T>::load(as + j, a);
        if (r >= 0) {
          Vec8<float>::load(reinterpret_cast<const float*>(fs) + j, f);
          Vec8<T>::store(frow + j, f);
#pragma unroll
          for (int t = 0; t < 8; ++t) f[t] = Vec8<T>::round(f[t]);
        } else {
          Vec8<T>::load(reinterpret_cast<const T*>(fs) + j, f);
        }
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          xv[t] = (xv[t] + a[t]) + f[t];
          ss += xv[t] * xv[t];
        }
        Vec8<float>::store(xr + j, xv);
        Vec8<float>::store(xs + j, xv);   // kept for the second pass
      }
      ss = warp_sum(ss);
      const float rs = rsqrtf(ss / (float)d + eps);
      T* orow = u + (size_t)c * d;
      for (int j = lane * 8; j < d; j += 256) {
        float v[8], gv[8];
        Vec8<float>::load(xs + j, v);
        Vec8<float>::load(gain + j, gv);
#pragma unroll
        for (int t = 0; t < 8; ++t) v[t] = v[t] * rs * gv[t];
        Vec8<T>::store(orow + j, v);
      }
      // the stage was written by this warp through the generic proxy; the next bulk copy goes through the async one
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&empty_bar[s]));
    }
  }
  ok = __syncthreads_and(ok);
  if (!ok) {
    if (threadIdx.x == 0 && status) atomicCAS(status, ST_OK, ST_TIMEOUT_ROWS_TAIL);
    drain_delay();
  }
}

// V-verify (Eq. 6) + V overwrite, streaming: see vverify_kernel.  Stage = [projected row fp32 | cached row].
template <typename T>
__global__ void __launch_bounds__(STREAM_THREADS, 1)
    vverify_stream_kernel(const float* __restrict__ part, T* __restrict__ Vc, float* __restrict__ sim, Geo g, int dkv,
                          int metric, int write_v, IdentityLists id, int stages, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[STREAM_MAX_STAGES], empty_bar[STREAM_MAX_STAGES];
  __shared__ int abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t nb_ = (uint32_t)dkv * 4, cb = (uint32_t)dkv * sizeof(T), stage_bytes = nb_ + cb;
  const uint32_t base = (smem_u32(smem_raw) + 127u) & ~127u;
  uint8_t* base_gen = smem_raw + (base - smem_u32(smem_raw));
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    mbar_fence_init();
  }
  __syncthreads();
  pdl_wait();
  pdl_trigger();
  volatile int* abortp = &abort_flag;
  const int n_rows = g.B * g.R;
  const int my_rows = (int)blockIdx.x < n_rows ? (n_rows - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  auto cache_row = [&](int c) {
    const int b = c / g.R, j = c - b * g.R;
    return Vc + ((size_t)b * g.n + g.P + j) * dkv;
  };
  bool ok = true;
  if (warp == 0) {
    if (lane == 0) {
      for (int i = 0; i < my_rows; ++i) {
        const int s = i % stages, c = blockIdx.x + i * gridDim.x;
        if (i >= stages && !mbar_wait(smem_u32(&empty_bar[s]), (uint32_t)(i / stages - 1) & 1u, abortp)) {
          ok = false;
          break;
        }
        const uint32_t dst = base + s * stage_bytes, bar = smem_u32(&full_bar[s]);
        mbar_expect_tx(bar, stage_bytes);
        bulk_load_1d(dst, part + (size_t)c * dkv, nb_, bar);
        bulk_load_1d(dst + nb_, cache_row(c), cb, bar);
      }
    }
  } else {
    const int w = warp - 1;
    for (int i = w; i < my_rows; i += STREAM_CONSUMERS) {
      const int s = i % stages, c = blockIdx.x + i * gridDim.x;
      ok = mbar_wait(smem_u32(&full_bar[s]), (uint32_t)(i / stages) & 1u, abortp);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const float* ns = reinterpret_cast<const float*>(base_gen + (size_t)s * stage_bytes);
      const T* cs = reinterpret_cast<const T*>(base_gen + (size_t)s * stage_bytes + nb_);
      T* vrow = cache_row(c);
      float dot = 0.f, na = 0.f, nb = 0.f;
      for (int j = lane * 8; j < dkv; j += 256) {
        float vn[8], vo[8];
        Vec8<float>::load(ns + j, vn);
        Vec8<T>::load(cs + j, vo);
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          vn[t] = Vec8<T>::round(vn[t]);  // compare what the cache will hold
          if (metric == 0) {
            dot += vn[t] * vo[t];
            na += vn[t] * vn[t];
            nb += vo[t] * vo[t];
          } else {
            const float df = vn[t] - vo[t];
            dot += df * df;
          }
        }
        if (write_v) Vec8<T>::store(vrow + j, vn);
      }
      dot = warp_sum(dot);
      na = warp_sum(na);
      nb = warp_sum(nb);
      if (lane == 0) {
        sim[c] = metric == 0 ? dot / fmaxf(sqrtf(na * nb), 1e-8f) : -sqrtf(dot);
        if (id.act) {  // a response refresh recomputes every response row, in carried order: identity lists
          id.sel[c] = c % g.R;
          id.act[c] = c;
          id.inv[c] = c;
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&empty_bar[s]));
    }
  }
  ok = __syncthreads_and(ok);
  if (!ok) {
    if (threadIdx.x == 0 && status) atomicCAS(status, ST_OK, ST_TIMEOUT_ROWS_VVERIFY);
    drain_delay();
  }
}

// After the O projection, streaming: see oproj_epilogue_kernel.  Stage = [projected row fp32 | x row fp32] of
// active row r (carried row act[r]).
template <typename T>
__global__ void __launch_bounds__(STREAM_THREADS, 1)
    oproj_stream_kernel(const float* __restrict__ part, const int32_t* __restrict__ act, const float* __restrict__ x,
                        const float* __restrict__ gain2, OutRows Ac, T* __restrict__ hn, Geo g, int Ma, float eps,
                        int stages, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[STREAM_MAX_STAGES], empty_bar[STREAM_MAX_STAGES];
  __shared__ int meta[STREAM_MAX_STAGES];
  __shared__ int abort_flag;
  const int d = g.d, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rb = (uint32_t)d * 4, stage_bytes = 2 * rb;
  const uint32_t base = (smem_u32(smem_raw) + 127u) & ~127u;
  uint8_t* base_gen = smem_raw + (base - smem_u32(smem_raw));
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    mbar_fence_init();
  }
  __syncthreads();
  pdl_wait();
  pdl_trigger();
  volatile int* abortp = &abort_flag;
  const int my_rows = (int)blockIdx.x < Ma ? (Ma - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  bool ok = true;
  if (warp == 0) {
    if (lane == 0) {
      for (int i = 0; i < my_rows; ++i) {
        const int s = i % stages, r = blockIdx.x + i * gridDim.x;
        if (i >= stages && !mbar_wait(smem_u32(&empty_bar[s]), (uint32_t)(i / stages - 1) & 1u, abortp)) {
          ok = false;
          break;
        }
        const int c = act[r];
        meta[s] = c;
        const uint32_t dst = base + s * stage_bytes, bar = smem_u32(&full_bar[s]);
        mbar_expect_tx(bar, stage_bytes);
        bulk_load_1d(dst, part + (size_t)r * d, rb, bar);
        bulk_load_1d(dst + rb, x + (size_t)c * d, rb, bar);
      }
    }
  } else {
    const int w = warp - 1;
    for (int i = w; i < my_rows; i += STREAM_CONSUMERS) {
      const int s = i % stages, r = blockIdx.x + i * gridDim.x;
      ok = mbar_wait(smem_u32(&full_bar[s]), (uint32_t)(i / stages) & 1u, abortp);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const int c = meta[s];
      const float* ps = reinterpret_cast<const float*>(base_gen + (size_t)s * stage_bytes);
      float* xs = reinterpret_cast<float*>(base_gen + (size_t)s * stage_bytes + rb);
      T* arow = Ac.row<T>(c, g);
      float ss = 0.f;
      for (int j = lane * 8; j < d; j += 256) {
        float a[8], xv[8];
        Vec8<float>::load(ps + j, a);
        Vec8<float>::load(xs + j, xv);
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          a[t] = Vec8<T>::round(a[t]);
          xv[t] += a[t];
          ss += xv[t] * xv[t];
        }
        Vec8<T>::store(arow + j, a);
        Vec8<float>::store(xs + j, xv);   // kept for the second pass
      }
      ss = warp_sum(ss);
      const float rs = rsqrtf(ss / (float)d + eps);
      T* out = hn + (size_t)r * d;
      for (int j = lane * 8; j < d; j += 256) {
        float v[8], gv[8];
        Vec8<float>::load(xs + j, v);
        Vec8<float>::load(gain2 + j, gv);
#pragma unroll
        for (int t = 0; t < 8; ++t) v[t] = v[t] * rs * gv[t];
        Vec8<T>::store(out + j, v);
      }
      // the stage was written by this warp through the generic proxy; the next bulk copy goes through the async one
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&empty_bar[s]));
    }
  }
  ok = __syncthreads_and(ok);
  if (!ok) {
    if (threadIdx.x == 0 && status) atomicCAS(status, ST_OK, ST_TIMEOUT_ROWS_OEPI);
    drain_delay();
  }
}

// RoPE + K scatter, streaming: see qk_rope_kernel.  Stage = the projected [Q | K] row (fp32) of active row r.  A
// consumer warp rotates a whole row: hd / 8 lanes cover the hd / 2 pairs of a head four at a time (element i with
// i + hd / 2), so a warp takes 256 / hd heads per trip; the row's cos / sin values are read once.
template <typename T>
__global__ void __launch_bounds__(STREAM_THREADS, 1)
    qk_rope_stream_kernel(const float* __restrict__ part, const int32_t* __restrict__ act,
                          const float* __restrict__ rope_tab, T* __restrict__ qbuf, T* __restrict__ Kc, Geo g, int Ma,
                          int H, int Hkv, int hd, int stages, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[STREAM_MAX_STAGES], empty_bar[STREAM_MAX_STAGES];
  __shared__ int meta[STREAM_MAX_STAGES];
  __shared__ int abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int dq = H * hd, dkv = Hkv * hd, width = dq + dkv, half = hd >> 1;
  const uint32_t stage_bytes = (uint32_t)width * 4;
  const uint32_t base = (smem_u32(smem_raw) + 127u) & ~127u;
  uint8_t* base_gen = smem_raw + (base - smem_u32(smem_raw));
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    mbar_fence_init();
  }
  __syncthreads();
  pdl_wait();
  pdl_trigger();
  volatile int* abortp = &abort_flag;
  const int my_rows = (int)blockIdx.x < Ma ? (Ma - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  bool ok = true;
  if (warp == 0) {
    if (lane == 0) {
      for (int i = 0; i < my_rows; ++i) {
        const int s = i % stages, r = blockIdx.x + i * gridDim.x;
        if (i >= stages && !mbar_wait(smem_u32(&empty_bar[s]), (uint32_t)(i / stages - 1) & 1u, abortp)) {
          ok = false;
          break;
        }
        meta[s] = act[r];
        const uint32_t bar = smem_u32(&full_bar[s]);
        mbar_expect_tx(bar, stage_bytes);
        bulk_load_1d(base + s * stage_bytes, part + (size_t)r * width, stage_bytes, bar);
      }
    }
  } else {
    const int w = warp - 1;
    const int lph = hd >> 3;                 // lanes per head: four pairs each
    const int hpt = 32 / lph;                // heads per trip of a warp
    const int hl = lane / lph, i0 = (lane - hl * lph) * 4;
    for (int i = w; i < my_rows; i += STREAM_CONSUMERS) {
      const int s = i % stages, r = blockIdx.x + i * gridDim.x;
      ok = mbar_wait(smem_u32(&full_bar[s]), (uint32_t)(i / stages) & 1u, abortp);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      int b, pos;
      carried_to_pos(meta[s], g, b, pos);
      const float* row = reinterpret_cast<const float*>(base_gen + (size_t)s * stage_bytes);
      const float* tab = rope_tab + (size_t)pos * hd;  // [cos(half) | sin(half)]
      const float4 cs = *reinterpret_cast<const float4*>(tab + i0);
      const float4 sn = *reinterpret_cast<const float4*>(tab + half + i0);
      const float cc[4] = {cs.x, cs.y, cs.z, cs.w}, ss[4] = {sn.x, sn.y, sn.z, sn.w};
      T* qrow = qbuf + (size_t)r * dq;
      T* krow = Kc + ((size_t)b * g.n + pos) * dkv;
      for (int h0 = 0; h0 < H + Hkv; h0 += hpt) {
        const int head = h0 + hl;
        if (head >= H + Hkv) break;          // the last trip may be partly empty
        const float4 lo4 = *reinterpret_cast<const float4*>(row + head * hd + i0);
        const float4 hi4 = *reinterpret_cast<const float4*>(row + head * hd + half + i0);
        const float lo[4] = {lo4.x, lo4.y, lo4.z, lo4.w}, hi[4] = {hi4.x, hi4.y, hi4.z, hi4.w};
        float o_lo[4], o_hi[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          o_lo[t] = lo[t] * cc[t] - hi[t] * ss[t];
          o_hi[t] = hi[t] * cc[t] + lo[t] * ss[t];
        }
        T* dst = head < H ? qrow + head * hd : krow + (head - H) * hd;
        store4<T>(dst + i0, o_lo);
        store4<T>(dst + i0 + half, o_hi);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&empty_bar[s]));
    }
  }
  ok = __syncthreads_and(ok);
  if (!ok) {
    if (threadIdx.x == 0 && status) atomicCAS(status, ST_OK, ST_TIMEOUT_ROWS_ROPE);
    drain_delay();
  }
}

// Rows from which the streaming forms are taken (a property of the session's response rows, so that every
// step kind of a session reduces a row in the same order).
constexpr int STREAM_MIN_ROWS = 1024;
static int stream_stages(size_t stage_bytes) {
  const size_t fit = (227 * 1024 - 2048) / stage_bytes;
  return (int)(fit < (size_t)STREAM_MAX_STAGES ? fit : (size_t)STREAM_MAX_STAGES);
}

// ------------------------------------------------------------------ rmsnorm
template <typename T>
__global__ void rmsnorm_kernel(const float* __restrict__ x, const float* __restrict__ gain, T* __restrict__ out, int d,
                               float eps, int c0) {
  pdl_wait();
  pdl_trigger();
  __shared__ float red[32];
  const size_t row = (size_t)(c0 + blockIdx.x);
  const float* xr = x + row * d;
  float ss = 0.f;
  for (int i = threadIdx.x * 8; i < d; i += blockDim.x * 8) {
    float v[8];
    Vec8<float>::load(xr + i, v);
#pragma unroll
    for (int j = 0; j < 8; ++j) ss += v[j] * v[j];
  }
  ss = block_sum(ss, red);
  const float r = rsqrtf(ss / (float)d + eps);
  T* orow = out + row * d;
  for (int i = threadIdx.x * 8; i < d; i += blockDim.x * 8) {
    float v[8], gv[8];
    Vec8<float>::load(xr + i, v);
    Vec8<float>::load(gain + i, gv);
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = v[j] * r * gv[j];
    Vec8<T>::store(orow + i, v);
  }
}

void launch_rmsnorm(const Launch& L, int dtype, const float* x, const float* gain, void* out, int d, float eps, int c0,
                    int c1) {
  if (c1 <= c0) return;
  DLLM_DISPATCH(dtype, (launch_k(L, rmsnorm_kernel<T>, dim3(c1 - c0), dim3(row_threads(d)), 0, x, gain, (T*)out, d, eps, c0)));
  L.count();
}

// ------------------------------------------------------------------ selection inside a kernel
// Bottom-k selection of sequence b by the whole CTA (R <= 1024: R^2 comparisons out of shared memory, 13 R + 16
// bytes at `keys`).  Fills slot[j] = position of response row j among the selected rows, or -1; with `write` the
// CTA also writes the index list, the active list (np prompt rows first) and its inverse.
// mode 0: every row; 1: the ksel lowest scores (Sec. 3.2.2); 2: the forced list.  Ends with a barrier.
__device__ __forceinline__ int32_t* select_sequence(unsigned long long* keys, const float* __restrict__ sim,
                                                    const int32_t* __restrict__ forced, int mode, int ksel,
                                                    int32_t* __restrict__ sel, int32_t* __restrict__ act,
                                                    int32_t* __restrict__ inv, const Geo& g, int np, int b, bool write) {
  const int R = g.R;
  int32_t* slot = reinterpret_cast<int32_t*>(keys + R);
  uint32_t* words = reinterpret_cast<uint32_t*>(slot + R);  // one ballot word per 32 rows
  const int a_seq = np + ksel;
  if (mode == 0) {
    for (int j = threadIdx.x; j < R; j += blockDim.x) slot[j] = j;
  } else if (mode == 2) {
    for (int j = threadIdx.x; j < R; j += blockDim.x) slot[j] = -1;
    __syncthreads();
    for (int r = threadIdx.x; r < ksel; r += blockDim.x) slot[forced[(size_t)b * R + r]] = r;
  } else {
    for (int j = threadIdx.x; j < R; j += blockDim.x) {
      const float s = __ldcg(sim + (size_t)b * R + j);
      // key = round(s * 2^20), offset into 1 .. 2^32 - 1 (scores beyond +-2047 saturate); NaN sorts first
      const float qf = fminf(fmaxf(rintf(s * 1048576.0f), -2147483520.0f), 2147483520.0f);
      const long long q = (s == s) ? (long long)qf + (1ll << 31) : 0ll;
      keys[j] = ((unsigned long long)q << 32) | (unsigned)j;
    }
    __syncthreads();
    // rank of every key (two keys per shared-memory load); a row is selected iff its rank is below ksel
    const int Rw = (R + 31) & ~31;
    for (int j = threadIdx.x; j < Rw; j += blockDim.x) {
      bool f = false;
      if (j < R) {
        const unsigned long long kj = keys[j];
        int rank = 0;
#pragma unroll 4
        for (int i = 0; i + 1 < R; i += 2) {
          const ulonglong2 kk = *reinterpret_cast<const ulonglong2*>(keys + i);
          rank += (kk.x < kj) + (kk.y < kj);
        }
        if (R & 1) rank += (keys[R - 1] < kj);
        f = rank < ksel;
      }
      const unsigned bal = __ballot_sync(0xffffffffu, f);
      if ((threadIdx.x & 31) == 0) words[j >> 5] = bal;
    }
    __syncthreads();
    for (int j = threadIdx.x; j < R; j += blockDim.x) {
      const unsigned wj = words[j >> 5];
      int r = -1;
      if ((wj >> (j & 31)) & 1u) {
        r = __popc(wj & ((1u << (j & 31)) - 1u));
        for (int w = 0; w < (j >> 5); ++w) r += __popc(words[w]);
      }
      slot[j] = r;
    }
  }
  __syncthreads();
  if (write) {
    for (int j = threadIdx.x; j < R; j += blockDim.x) {
      const int r = slot[j];
      inv[(size_t)b * R + j] = r >= 0 ? b * a_seq + np + r : -1;
      if (r >= 0) {
        sel[(size_t)b * R + r] = j;
        act[(size_t)b * a_seq + np + r] = b * R + j;
      }
    }
    for (int i = threadIdx.x; i < np; i += blockDim.x) {
      act[(size_t)b * a_seq + i] = g.B * R + b * g.P + i;
      inv[(size_t)g.B * R + (size_t)b * g.P + i] = b * a_seq + i;
    }
  }
  __syncthreads();
  return slot;
}

// ------------------------------------------------------------------ V-verify (Eq. 6) + V overwrite
// metric 0: cosine (Eq. 6); 1: negated Euclidean distance (Sec. A.6), so that the
// least similar rows have the lowest score either way.  write_v 0: the cache is
// left as it is (the selected-only variant of Sec. A.5 writes the selected rows later).
// The launch before this one is the V projection, which writes nothing but `part`: a row that fits one pass
// fetches its cached V row before the dependency wait, while the projection still runs.
template <typename T>
__global__ void __launch_bounds__(512, 2) vverify_kernel(Partials part, T* __restrict__ Vc, float* __restrict__ sim,
                                                         Geo g, int dkv, int metric, int write_v, IdentityLists id) {
  __shared__ float red[96];
  const int c = blockIdx.x;  // response row, carried order
  const int b = c / g.R, j = c - b * g.R;
  T* vrow = Vc + ((size_t)b * g.n + g.P + j) * dkv;
  const bool one_trip = dkv <= (int)blockDim.x * 8;
  float vo0[8];
  if (one_trip && (int)threadIdx.x * 8 < dkv) Vec8<T>::load_cg(vrow + threadIdx.x * 8, vo0);
  pdl_wait();
  pdl_trigger();
  float dot = 0.f, na = 0.f, nb = 0.f;
  for (int i = threadIdx.x * 8; i < dkv; i += blockDim.x * 8) {
    float vn[8], vo[8];
    sum_partials8(part.p, part.split_stride, part.count(c, i), (size_t)c * part.N + i, vn);
    if (one_trip) {
#pragma unroll
      for (int t = 0; t < 8; ++t) vo[t] = vo0[t];
    } else {
      Vec8<T>::load(vrow + i, vo);
    }
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      vn[t] = Vec8<T>::round(vn[t]);  // compare what the cache will hold
      if (metric == 0) {
        dot += vn[t] * vo[t];
        na += vn[t] * vn[t];
        nb += vo[t] * vo[t];
      } else {
        const float df = vn[t] - vo[t];
        dot += df * df;
      }
    }
    if (write_v) Vec8<T>::store(vrow + i, vn);
  }
  block_sum3(dot, na, nb, red);
  if (threadIdx.x == 0) sim[c] = metric == 0 ? dot / fmaxf(sqrtf(na * nb), 1e-8f) : -sqrtf(dot);
  // a response refresh recomputes every response row, in carried order: the lists are the identity
  if (id.act && threadIdx.x == 0) {
    id.sel[c] = j;
    id.act[c] = c;
    id.inv[c] = c;
  }
}

void launch_vverify(const Launch& L, int dtype, Partials part, void* Vc_layer, float* sim, Geo g, int dkv, int metric,
                    int write_v, const IdentityLists* lists) {
  const int rows = g.B * g.R;
  const IdentityLists id = lists ? *lists : IdentityLists{};
  const size_t es = dtype == 0 ? 4 : 2, stage = (size_t)dkv * (4 + es);
  if (rows >= STREAM_MIN_ROWS && part.S == 1 && part.upc == 0 && stream_stages(stage) >= STREAM_CONSUMERS + 1) {
    const int stages = stream_stages(stage);
    const size_t smem = (size_t)stages * stage + 128;
    const int ctas = std::min(rows, sm_count());
    DLLM_DISPATCH(dtype, {
      static DeviceOnce once;
      cudaError_t e0 = once.run([] {
        return cudaFuncSetAttribute(vverify_stream_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 1024);
      });
      if (e0 == cudaSuccess)
        launch_k(L, vverify_stream_kernel<T>, dim3(ctas), dim3(STREAM_THREADS), smem, part.p, (T*)Vc_layer, sim, g, dkv,
                 metric, write_v, id, stages, L.d_status);
    });
    L.count();
    return;
  }
  DLLM_DISPATCH(dtype, (launch_k(L, vverify_kernel<T>, dim3(rows), dim3(row_threads(dkv)), 0, part, (T*)Vc_layer, sim, g, dkv,
                                 metric, write_v, id)));
  L.count();
}

// ------------------------------------------------------------------ K-verify: the same test on the post-RoPE K
// One block per response row: slab sum of the K projection, RoPE at the row's
// position, rounding to the cache dtype, score against the cached K row, and
// the whole-K overwrite (the symmetric reading of the K-verify ablation, Sec. 4.3).
template <typename T>
__global__ void kverify_kernel(Partials part, T* __restrict__ Kc, float* __restrict__ sim,
                               const float* __restrict__ rope_tab, Geo g, int Hkv, int hd, int metric) {
  pdl_wait();
  pdl_trigger();
  __shared__ float red[32];
  const int c = blockIdx.x;
  const int b = c / g.R, j = c - b * g.R, pos = g.P + j;
  const int half = hd >> 1, q4 = half >> 2, dkv = Hkv * hd;
  T* krow = Kc + ((size_t)b * g.n + pos) * dkv;
  const float* tab = rope_tab + (size_t)pos * hd;
  float dot = 0.f, na = 0.f, nb = 0.f;
  for (int gidx = threadIdx.x; gidx < Hkv * q4; gidx += blockDim.x) {
    const int head = gidx / q4, i0 = (gidx - head * q4) * 4, col0 = head * hd;
    float lo[4], hi[4], o_lo[4], o_hi[4], c_lo[4], c_hi[4];
    sum_partials4(part, c, col0 + i0, lo);
    sum_partials4(part, c, col0 + i0 + half, hi);
    const float4 cs = *reinterpret_cast<const float4*>(tab + i0);
    const float4 sn = *reinterpret_cast<const float4*>(tab + half + i0);
    const float cc[4] = {cs.x, cs.y, cs.z, cs.w}, ss[4] = {sn.x, sn.y, sn.z, sn.w};
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      o_lo[t] = Vec8<T>::round(lo[t] * cc[t] - hi[t] * ss[t]);
      o_hi[t] = Vec8<T>::round(hi[t] * cc[t] + lo[t] * ss[t]);
      c_lo[t] = to_f32<T>(krow[col0 + i0 + t]);
      c_hi[t] = to_f32<T>(krow[col0 + i0 + half + t]);
    }
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      if (metric == 0) {
        dot += o_lo[t] * c_lo[t] + o_hi[t] * c_hi[t];
        na += o_lo[t] * o_lo[t] + o_hi[t] * o_hi[t];
        nb += c_lo[t] * c_lo[t] + c_hi[t] * c_hi[t];
      } else {
        const float d0 = o_lo[t] - c_lo[t], d1 = o_hi[t] - c_hi[t];
        dot += d0 * d0 + d1 * d1;
      }
    }
    store4<T>(krow + col0 + i0, o_lo);
    store4<T>(krow + col0 + i0 + half, o_hi);
  }
  dot = block_sum(dot, red);
  if (metric == 0) {
    na = block_sum(na, red);
    nb = block_sum(nb, red);
  }
  if (threadIdx.x == 0) sim[c] = metric == 0 ? dot / fmaxf(sqrtf(na * nb), 1e-8f) : -sqrtf(dot);
}

void launch_kverify(const Launch& L, int dtype, Partials part, void* Kc_layer, float* sim, const float* rope_tab, Geo g,
                    int Hkv, int hd, int metric) {
  const int rows = g.B * g.R;
  DLLM_DISPATCH(dtype, (launch_k(L, kverify_kernel<T>, dim3(rows), dim3(256), 0, part, (T*)Kc_layer, sim, rope_tab, g,
                                 Hkv, hd, metric)));
  L.count();
}

// standalone form used by the kernel-level entry point: v_new given as a tensor
template <typename T>
__global__ void vverify_rows_kernel(const T* __restrict__ vnew, T* __restrict__ vcache, float* __restrict__ sim,
                                    int width) {
  pdl_wait();
  pdl_trigger();
  __shared__ float red[32];
  const size_t row = blockIdx.x;
  const T* a = vnew + row * width;
  T* bb = vcache + row * width;
  float dot = 0.f, na = 0.f, nb = 0.f;
  for (int i = threadIdx.x * 8; i < width; i += blockDim.x * 8) {
    float vn[8], vo[8];
    Vec8<T>::load(a + i, vn);
    Vec8<T>::load(bb + i, vo);
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      dot += vn[t] * vo[t];
      na += vn[t] * vn[t];
      nb += vo[t] * vo[t];
    }
    Vec8<T>::store(bb + i, vn);
  }
  dot = block_sum(dot, red);
  na = block_sum(na, red);
  nb = block_sum(nb, red);
  if (threadIdx.x == 0) sim[row] = dot / fmaxf(sqrtf(na * nb), 1e-8f);
}

void launch_vverify_rows(const Launch& L, int dtype, const void* vnew, void* vcache, float* sim, int rows, int width) {
  if (rows <= 0) return;
  DLLM_DISPATCH(dtype, (launch_k(L, vverify_rows_kernel<T>, dim3(rows), dim3(128), 0, (const T*)vnew, (T*)vcache, sim, width)));
  L.count();
}

// ------------------------------------------------------------------ bottom-k selection
// One block per sequence.  Keys are unique (the index is part of the key), so
// the rank of a key among all R keys is its position in sorted order; a row is
// selected iff rank < k.  R^2 comparisons out of shared memory: R <= 8192.
__global__ void select_kernel(const float* __restrict__ sim, const int32_t* __restrict__ forced, int mode, int ksel,
                              int32_t* __restrict__ sel, int sel_stride, int32_t* __restrict__ act,
                              int32_t* __restrict__ inv, Geo g, int refresh_prompt) {
  pdl_wait();
  pdl_trigger();
  extern __shared__ unsigned long long keys[];  // R keys, then R flags (as bytes)
  unsigned char* flag = reinterpret_cast<unsigned char*>(keys + g.R);
  const int b = blockIdx.x;
  const int R = g.R;
  const int a_seq = (refresh_prompt ? g.P : 0) + ksel;
  int32_t* act_b = act ? act + (size_t)b * a_seq : nullptr;
  int32_t* sel_b = sel + (size_t)b * sel_stride;
  const int np = refresh_prompt ? g.P : 0;
  if (refresh_prompt && act)
    for (int i = threadIdx.x; i < g.P; i += blockDim.x) {
      act_b[i] = g.B * R + b * g.P + i;
      if (inv) inv[(size_t)g.B * R + (size_t)b * g.P + i] = b * a_seq + i;
    }
  int32_t* act_r = act ? act_b + np : nullptr;
  if (mode == 0) {
    for (int j = threadIdx.x; j < R; j += blockDim.x) {
      sel_b[j] = j;
      if (act_r) act_r[j] = b * R + j;
      if (inv) inv[(size_t)b * R + j] = b * a_seq + np + j;
    }
    return;
  }
  if (mode == 2) {
    if (inv) {
      for (int j = threadIdx.x; j < R; j += blockDim.x) inv[(size_t)b * R + j] = -1;
      __syncthreads();
    }
    for (int r = threadIdx.x; r < ksel; r += blockDim.x) {
      const int j = forced[(size_t)b * R + r];
      sel_b[r] = j;
      if (act_r) act_r[r] = b * R + j;
      if (inv) inv[(size_t)b * R + j] = b * a_seq + np + r;
    }
    return;
  }
  for (int j = threadIdx.x; j < R; j += blockDim.x) {
    const float s = sim[(size_t)b * R + j];
    // key = round(s * 2^20), offset into 1 .. 2^32 - 1 (scores beyond +-2047 saturate); NaN sorts first
    const float qf = fminf(fmaxf(rintf(s * 1048576.0f), -2147483520.0f), 2147483520.0f);
    const long long q = (s == s) ? (long long)qf + (1ll << 31) : 0ll;
    keys[j] = ((unsigned long long)q << 32) | (unsigned)j;
    flag[j] = 0;
  }
  __syncthreads();
  for (int j = threadIdx.x; j < R; j += blockDim.x) {
    const unsigned long long kj = keys[j];
    int rank = 0;
    for (int i = 0; i < R; ++i) rank += (keys[i] < kj);
    flag[j] = (rank < ksel);
  }
  __syncthreads();
  for (int j = threadIdx.x; j < R; j += blockDim.x) {
    if (!flag[j]) {
      if (inv) inv[(size_t)b * R + j] = -1;
      continue;
    }
    int r = 0;
    for (int i = 0; i < j; ++i) r += flag[i];
    sel_b[r] = j;
    if (act_r) act_r[r] = b * R + j;
    if (inv) inv[(size_t)b * R + j] = b * a_seq + np + r;
  }
}

cudaError_t launch_select(const Launch& L, const float* sim, const int32_t* forced, int mode, int ksel, int32_t* sel,
                          int sel_stride, int32_t* act, int32_t* inv, Geo g, int refresh_prompt) {
  // 9 bytes per response row: beyond 48 KB (R > 5459) the kernel needs the opt-in for large dynamic shared memory
  constexpr int MAX_R = 8192;
  if (g.R > MAX_R) return cudaErrorInvalidValue;
  static DeviceOnce once;
  cudaError_t e = once.run([] {
    return cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_R * 9 + 16);
  });
  if (e != cudaSuccess) return e;
  const size_t smem = (size_t)g.R * 9 + 16;
  // one key per thread up to 1024 response rows (the rank of a key costs R comparisons of its thread)
  const int threads = g.R <= 256 ? 256 : g.R >= 1024 ? 1024 : (g.R + 31) / 32 * 32;
  e = launch_k(L, select_kernel, dim3(g.B), dim3(threads), smem, sim, forced, mode, ksel, sel, sel_stride, act, inv, g,
               refresh_prompt);
  L.count();
  return e;
}

// ------------------------------------------------------------------ gather
template <typename T>
__global__ void gather_rows_kernel(const T* __restrict__ src, const int32_t* __restrict__ act, T* __restrict__ dst,
                                   int d) {
  pdl_wait();
  pdl_trigger();
  const size_t r = blockIdx.x;
  copy_row16(reinterpret_cast<const uint4*>(src + (size_t)act[r] * d), reinterpret_cast<uint4*>(dst + r * d),
             d * (int)sizeof(T) / 16);
}

void launch_gather_rows(const Launch& L, int dtype, const void* src, const int32_t* act, void* dst, int rows, int d) {
  if (rows <= 0) return;
  DLLM_DISPATCH(dtype, (launch_k(L, gather_rows_kernel<T>, dim3(rows), dim3(128), 0, (const T*)src, act, (T*)dst, d)));
  L.count();
}

// ------------------------------------------------------------------ RoPE + K scatter
// One thread per (active row, HP consecutive heads, four rotation pairs).  Rotate-half pairing:
// element i with i + hd/2, angle pos * theta^(-2i/hd) from a table built on the host.  HP = 2 (the heads of a
// thread share the row's position and rotation values) halves the CTAs when there are several per SM slot, so
// that all of them are resident, and have fetched those values, before the projection ahead of them ends.
template <typename T, int HP>
__global__ void qk_rope_kernel(Partials part, const int32_t* __restrict__ act, const float* __restrict__ rope_tab,
                               T* __restrict__ qbuf, T* __restrict__ Kc, Geo g, int Ma, int H, int Hkv, int hd) {
  // The launch before this one is the Q / K projection, which writes nothing but `part`: the row's position and
  // its cos / sin values are fetched before the dependency wait, while the projection still runs.
  const int half = hd >> 1, q4 = half >> 2;
  const int heads = H + Hkv, hgroups = (heads + HP - 1) / HP;
  const int groups = hgroups * q4;
  const long w = (long)blockIdx.x * blockDim.x + threadIdx.x;
  const bool live = w < (long)Ma * groups;
  const int r = live ? (int)(w / groups) : 0, gidx = live ? (int)(w - (long)r * groups) : 0;
  const int hg = gidx / q4, i0 = (gidx - hg * q4) * 4;
  int b, pos;
  carried_to_pos(__ldcg(act + r), g, b, pos);
  const int dq = H * hd, dkv = Hkv * hd;
  const float* tab = rope_tab + (size_t)pos * hd;  // [cos(half) | sin(half)]
  const float4 cs = *reinterpret_cast<const float4*>(tab + i0);
  const float4 sn = *reinterpret_cast<const float4*>(tab + half + i0);
  pdl_wait();
  pdl_trigger();
  if (!live) return;
  const float cc[4] = {cs.x, cs.y, cs.z, cs.w}, ss[4] = {sn.x, sn.y, sn.z, sn.w};
  float lo[HP][4], hi[HP][4];
#pragma unroll
  for (int u = 0; u < HP; ++u) {
    const int head = hg * HP + u;
    if (head >= heads) break;
    const int col0 = head < H ? head * hd : dq + (head - H) * hd;
    sum_partials4(part, r, col0 + i0, lo[u]);
    sum_partials4(part, r, col0 + i0 + half, hi[u]);
  }
#pragma unroll
  for (int u = 0; u < HP; ++u) {
    const int head = hg * HP + u;
    if (head >= heads) break;
    T* dst = head < H ? qbuf + (size_t)r * dq + head * hd : Kc + ((size_t)b * g.n + pos) * dkv + (head - H) * hd;
    float o_lo[4], o_hi[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      o_lo[t] = lo[u][t] * cc[t] - hi[u][t] * ss[t];
      o_hi[t] = hi[u][t] * cc[t] + lo[u][t] * ss[t];
    }
    store4<T>(dst + i0, o_lo);
    store4<T>(dst + i0 + half, o_hi);
  }
}

void launch_qk_rope(const Launch& L, int dtype, Partials part, const int32_t* act, const float* rope_tab, void* qbuf,
                    void* Kc_layer, Geo g, int Ma, int H, int Hkv, int hd) {
  if (Ma <= 0) return;
  const size_t stage = (size_t)(H + Hkv) * hd * 4;
  // streaming form: unsplit slabs, a head size whose pairs a group of lanes covers exactly (a power of two, 32..256)
  if (g.B * g.R >= STREAM_MIN_ROWS && part.S == 1 && part.upc == 0 && hd >= 32 && hd <= 256 && (hd & (hd - 1)) == 0 &&
      stream_stages(stage) >= STREAM_CONSUMERS + 1) {
    const int stages = stream_stages(stage);
    const size_t smem = (size_t)stages * stage + 128;
    const int ctas = std::min(Ma, sm_count());
    DLLM_DISPATCH(dtype, {
      static DeviceOnce once;
      cudaError_t e0 = once.run([] {
        return cudaFuncSetAttribute(qk_rope_stream_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 1024);
      });
      if (e0 == cudaSuccess)
        launch_k(L, qk_rope_stream_kernel<T>, dim3(ctas), dim3(STREAM_THREADS), smem, part.p, act, rope_tab, (T*)qbuf,
                 (T*)Kc_layer, g, Ma, H, Hkv, hd, stages, L.d_status);
    });
    L.count();
    return;
  }
  const long total = (long)Ma * (H + Hkv) * (hd >> 3);
  const long blocks1 = (total + 255) / 256;
  if (blocks1 > 2L * sm_count()) {   // two heads per thread: half the CTAs
    const long total2 = (long)Ma * ((H + Hkv + 1) / 2) * (hd >> 3);
    DLLM_DISPATCH(dtype, (launch_k(L, qk_rope_kernel<T, 2>, dim3((unsigned)((total2 + 255) / 256)), dim3(256), 0, part, act,
                                   rope_tab, (T*)qbuf, (T*)Kc_layer, g, Ma, H, Hkv, hd)));
  } else {
    DLLM_DISPATCH(dtype, (launch_k(L, qk_rope_kernel<T, 1>, dim3((unsigned)blocks1), dim3(256), 0, part, act, rope_tab,
                                   (T*)qbuf, (T*)Kc_layer, g, Ma, H, Hkv, hd)));
  }
  L.count();
}

// ------------------------------------------------------------------ scatter rows into a cache tensor
template <typename T>
__global__ void scatter_rows_kernel(Partials part, const int32_t* __restrict__ act, int c_base, T* __restrict__ cache,
                                    Geo g, int width) {
  pdl_wait();
  pdl_trigger();
  const int r = blockIdx.x;
  const int c = act ? act[r] : c_base + r;
  int b, pos;
  carried_to_pos(c, g, b, pos);
  T* dst = cache + ((size_t)b * g.n + pos) * width;
  for (int i = threadIdx.x * 8; i < width; i += blockDim.x * 8) {
    float v[8];
    sum_partials8(part.p, part.split_stride, part.count(r, i), (size_t)r * part.N + i, v);
    Vec8<T>::store(dst + i, v);
  }
}

void launch_scatter_rows(const Launch& L, int dtype, Partials part, const int32_t* act, int c_base, void* cache_layer,
                         Geo g, int rows, int width) {
  if (rows <= 0) return;
  DLLM_DISPATCH(dtype,
                (launch_k(L, scatter_rows_kernel<T>, dim3(rows), dim3(row_threads(width)), 0, part, act, c_base, (T*)cache_layer, g, width)));
  L.count();
}

// ------------------------------------------------------------------ O-proj epilogue
// AttnOut row -> cache (rounded to the cache dtype); h = x + AttnOut (the
// rounded value, so a later step that reads the cache sees the same h);
// hn = rmsnorm(h) * gain2.
template <typename T>
__global__ void oproj_epilogue_kernel(Partials part, const int32_t* __restrict__ act, const float* __restrict__ x,
                                      const float* __restrict__ gain2, OutRows Ac, T* __restrict__ hn, Geo g,
                                      float eps) {
  // The launch before this one is the O projection, which writes nothing but `part`: the row's place (act), its x
  // row and the gain are fetched before the dependency wait, while the projection still runs.
  extern __shared__ float hrow[];
  __shared__ float red[32];
  const int r = blockIdx.x;
  const int d = g.d;
  const bool one_trip = d <= (int)blockDim.x * 8;  // the row fits one pass: it stays in registers
  const int i0 = threadIdx.x * 8;
  float hv[8], gv[8], x0[8];
  const int c = __ldcg(act + r);
  T* arow = Ac.row<T>(c, g);
  const float* xr = x + (size_t)c * d;
  if (one_trip && i0 < d) {
    Vec8<float>::load(gain2 + i0, gv);
    Vec8<float>::load_cg(xr + i0, x0);
  }
  pdl_wait();
  pdl_trigger();
  float ss = 0.f;
  for (int i = i0; i < d; i += blockDim.x * 8) {
    float a[8], xv[8];
    sum_partials8(part.p, part.split_stride, part.count(r, i), (size_t)r * part.N + i, a);
    if (one_trip) {
#pragma unroll
      for (int t = 0; t < 8; ++t) xv[t] = x0[t];
    } else {
      Vec8<float>::load(xr + i, xv);
    }
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      a[t] = Vec8<T>::round(a[t]);
      xv[t] += a[t];
      ss += xv[t] * xv[t];
      hv[t] = xv[t];
    }
    Vec8<T>::store(arow + i, a);
    if (!one_trip) Vec8<float>::store(hrow + i, xv);
  }
  ss = block_sum(ss, red);
  const float rs = rsqrtf(ss / (float)d + eps);
  T* out = hn + (size_t)r * d;
  if (one_trip) {
    if (i0 < d) {
#pragma unroll
      for (int t = 0; t < 8; ++t) hv[t] = hv[t] * rs * gv[t];
      Vec8<T>::store(out + i0, hv);
    }
    return;
  }
  for (int i = i0; i < d; i += blockDim.x * 8) {
    float v[8];
    Vec8<float>::load(hrow + i, v);
    Vec8<float>::load(gain2 + i, gv);
#pragma unroll
    for (int t = 0; t < 8; ++t) v[t] = v[t] * rs * gv[t];
    Vec8<T>::store(out + i, v);
  }
}

void launch_oproj_epilogue(const Launch& L, int dtype, Partials part, const int32_t* act, const float* x,
                           const float* gain2, OutRows Ac_layer, void* hn, Geo g, int Ma, float eps) {
  if (Ma <= 0) return;
  const size_t stage = (size_t)g.d * 8;
  if (g.B * g.R >= STREAM_MIN_ROWS && part.S == 1 && part.upc == 0 && (g.d & 7) == 0 &&
      stream_stages(stage) >= STREAM_CONSUMERS + 1) {
    const int stages = stream_stages(stage);
    const size_t smem = (size_t)stages * stage + 128;
    const int ctas = std::min(Ma, sm_count());
    DLLM_DISPATCH(dtype, {
      static DeviceOnce once;
      cudaError_t e0 = once.run([] {
        return cudaFuncSetAttribute(oproj_stream_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 1024);
      });
      if (e0 == cudaSuccess)
        launch_k(L, oproj_stream_kernel<T>, dim3(ctas), dim3(STREAM_THREADS), smem, part.p, act, x, gain2, Ac_layer,
                 (T*)hn, g, Ma, eps, stages, L.d_status);
    });
    L.count();
    return;
  }
  const int threads = row_threads(g.d);
  const size_t smem = g.d <= threads * 8 ? 0 : (size_t)g.d * sizeof(float);  // staging only if a row takes several passes
  DLLM_DISPATCH(dtype, (launch_k(L, oproj_epilogue_kernel<T>, dim3(Ma), dim3(threads), smem, part, act, x, gain2, Ac_layer,
                                 (T*)hn, g, eps)));
  L.count();
}

// ------------------------------------------------------------------ SwiGLU gate
template <typename T>
__global__ void silu_mul_kernel(Partials part, T* __restrict__ out, int Ma, int m, int interleaved) {
  pdl_wait();
  pdl_trigger();
  const int mv = m >> 3;
  const size_t total = (size_t)Ma * mv;
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
    const int r = (int)(idx / mv), j = (int)(idx - (size_t)r * mv) * 8;
    float gt[8], up[8];
    const int cg = interleaved ? (j >> 6) * 128 + (j & 63) : j, cu = interleaved ? cg + 64 : m + j;
    sum_partials8(part.p, part.split_stride, part.count(r, cg), (size_t)r * part.N + cg, gt);
    sum_partials8(part.p, part.split_stride, part.count(r, cu), (size_t)r * part.N + cu, up);
#pragma unroll
    for (int t = 0; t < 8; ++t) gt[t] = __fdividef(gt[t], 1.f + __expf(-gt[t])) * up[t];  // as in the GEMM epilogue
    Vec8<T>::store(out + (size_t)r * m + j, gt);
  }
}

void launch_silu_mul(const Launch& L, int dtype, Partials part, void* out, int Ma, int m, int interleaved) {
  if (Ma <= 0) return;
  const size_t total = (size_t)Ma * (m >> 3);
  const int blocks = (int)((total + 255) / 256 < 148 * 8 ? (total + 255) / 256 : 148 * 8);
  DLLM_DISPATCH(dtype, (launch_k(L, silu_mul_kernel<T>, dim3(blocks), dim3(256), 0, part, (T*)out, Ma, m, interleaved)));
  L.count();
}

// ------------------------------------------------------------------ embedding + first RMSNorm
// x[c] = E[token(c)], u[c] = rmsnorm(x[c]) * gain for carried rows c0 <= c < c1.
template <typename T>
__global__ void embed_norm_kernel(const T* __restrict__ E, const int32_t* __restrict__ tokens, float* __restrict__ x,
                                  const float* __restrict__ gain, T* __restrict__ u, Geo g, int c0, float eps) {
  pdl_wait();
  pdl_trigger();
  __shared__ float red[32];
  const int c = c0 + blockIdx.x;
  int b, pos;
  carried_to_pos(c, g, b, pos);
  const int tok = tokens[(size_t)b * g.n + pos];
  const T* src = E + (size_t)tok * g.d;
  float* xr = x + (size_t)c * g.d;
  float ss = 0.f;
  for (int i = threadIdx.x * 8; i < g.d; i += blockDim.x * 8) {
    float v[8];
    Vec8<T>::load(src + i, v);
    Vec8<float>::store(xr + i, v);
#pragma unroll
    for (int j = 0; j < 8; ++j) ss += v[j] * v[j];
  }
  ss = block_sum(ss, red);
  const float r = rsqrtf(ss / (float)g.d + eps);
  T* orow = u + (size_t)c * g.d;
  for (int i = threadIdx.x * 8; i < g.d; i += blockDim.x * 8) {
    float v[8], gv[8];
    Vec8<T>::load(src + i, v);
    Vec8<float>::load(gain + i, gv);
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = v[j] * r * gv[j];
    Vec8<T>::store(orow + i, v);
  }
}

void launch_embed_norm(const Launch& L, int dtype, const void* E, const int32_t* tokens, float* x, const float* gain,
                       void* u, Geo g, int c0, int c1, float eps) {
  if (c1 <= c0) return;
  DLLM_DISPATCH(dtype, (launch_k(L, embed_norm_kernel<T>, dim3(c1 - c0), dim3(row_threads(g.d)), 0, (const T*)E, tokens, x, gain,
                                 (T*)u, g, c0, eps)));
  L.count();
}

// ------------------------------------------------------------------ layer tail
// For every carried row: the FFNOut row of an active row (inv[c] >= 0: its
// position in the active list, whose slabs `part` holds) goes to the cache,
// rounded to the cache dtype; x <- (x + AttnOut) + FFNOut from the caches
// (Sec. 3.2 item (3)); u = rmsnorm(x) * gain, the next layer's first norm (the
// final norm after the last layer).  inv == nullptr: no row is active.
// With active rows (inv != nullptr) the launch before this one is the down projection, which writes nothing but
// `part`; everything else a row needs (its place in the active list, x, AttnOut, a cached FFNOut row, the gain) was
// written by launches that had completed before that projection passed its own dependency wait.  A one-pass row
// therefore fetches all of it BEFORE the wait, while the projection still runs, and only the projection result
// (active rows) after it.
template <typename T, bool EARLY>
__global__ void __launch_bounds__(512, 2) tail_kernel(Partials part, const int32_t* __restrict__ inv, float* __restrict__ x,
                            OutRows Ac, OutRows Fc, const float* __restrict__ gain,
                            T* __restrict__ u, Geo g, int c0, float eps) {
  extern __shared__ float hrow[];
  __shared__ float red[32];
  const int c = c0 + blockIdx.x;
  const int d = g.d;
  const T* arow = Ac.row<T>(c, g);
  T* frow = Fc.row<T>(c, g);
  const bool one_trip = d <= (int)blockDim.x * 8;  // the row fits one pass: it stays in registers
  const int i0 = threadIdx.x * 8;
  float* xr = x + (size_t)c * d;
  float hv[8], gv[8];
  int r = -1;
  if constexpr (EARLY) {   // the host passes EARLY only with inv != nullptr and a one-pass row
    float ae[8], fe[8];
    r = __ldcg(inv + c);
    if (i0 < d) {
      Vec8<float>::load(gain + i0, gv);
      Vec8<float>::load_cg(xr + i0, hv);
      Vec8<T>::load_cg(arow + i0, ae);
      if (r < 0) Vec8<T>::load_cg(frow + i0, fe);
    }
    pdl_wait();
    pdl_trigger();
    float ss = 0.f;
    if (i0 < d) {
      if (r >= 0) {
        sum_partials8(part.p, part.split_stride, part.count(r, i0), (size_t)r * part.N + i0, fe);
        Vec8<T>::store(frow + i0, fe);
#pragma unroll
        for (int t = 0; t < 8; ++t) fe[t] = Vec8<T>::round(fe[t]);
      }
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        hv[t] = (hv[t] + ae[t]) + fe[t];
        ss += hv[t] * hv[t];
      }
      Vec8<float>::store(xr + i0, hv);
    }
    ss = block_sum(ss, red);
    const float rs = rsqrtf(ss / (float)d + eps);
    if (i0 < d) {
#pragma unroll
      for (int t = 0; t < 8; ++t) hv[t] = hv[t] * rs * gv[t];
      Vec8<T>::store(u + (size_t)c * d + i0, hv);
    }
    return;
  }
  pdl_wait();
  pdl_trigger();
  if (one_trip && i0 < d) Vec8<float>::load(gain + i0, gv);
  r = inv ? inv[c] : -1;
  float ss = 0.f;
  for (int i = i0; i < d; i += blockDim.x * 8) {
    float xv[8], a[8], f[8];
    Vec8<float>::load(xr + i, xv);
    Vec8<T>::load(arow + i, a);
    if (r >= 0) {
      sum_partials8(part.p, part.split_stride, part.count(r, i), (size_t)r * part.N + i, f);
      Vec8<T>::store(frow + i, f);
#pragma unroll
      for (int t = 0; t < 8; ++t) f[t] = Vec8<T>::round(f[t]);
    } else {
      Vec8<T>::load(frow + i, f);
    }
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      xv[t] = (xv[t] + a[t]) + f[t];
      ss += xv[t] * xv[t];
      hv[t] = xv[t];
    }
    Vec8<float>::store(xr + i, xv);
    if (!one_trip) Vec8<float>::store(hrow + i, xv);
  }
  ss = block_sum(ss, red);
  const float rs = rsqrtf(ss / (float)d + eps);
  T* orow = u + (size_t)c * d;
  if (one_trip) {
    if (i0 < d) {
#pragma unroll
      for (int t = 0; t < 8; ++t) hv[t] = hv[t] * rs * gv[t];
      Vec8<T>::store(orow + i0, hv);
    }
    return;
  }
  for (int i = i0; i < d; i += blockDim.x * 8) {
    float v[8];
    Vec8<float>::load(hrow + i, v);
    Vec8<float>::load(gain + i, gv);
#pragma unroll
    for (int t = 0; t < 8; ++t) v[t] = v[t] * rs * gv[t];
    Vec8<T>::store(orow + i, v);
  }
}

void launch_tail(const Launch& L, int dtype, Partials part, const int32_t* inv, float* x, OutRows Ac_layer,
                 OutRows Fc_layer, const float* gain, void* u, Geo g, int c0, int c1, float eps) {
  if (c1 <= c0) return;
  {
    const size_t es = dtype == 0 ? 4 : 2, stage = (size_t)g.d * (8 + es);
    if (g.B * g.R >= STREAM_MIN_ROWS && part.S == 1 && part.upc == 0 && stream_stages(stage) >= STREAM_CONSUMERS + 1) {
      const int stages = stream_stages(stage);
      const size_t smem_s = (size_t)stages * stage + 128;
      const int ctas = std::min(c1 - c0, sm_count());
      DLLM_DISPATCH(dtype, {
        static DeviceOnce once;
        cudaError_t e0 = once.run([] {
          return cudaFuncSetAttribute(tail_stream_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 1024);
        });
        if (e0 == cudaSuccess)
          launch_k(L, tail_stream_kernel<T>, dim3(ctas), dim3(STREAM_THREADS), smem_s, part.p, inv, x, Ac_layer, Fc_layer,
                   gain, (T*)u, g, c0, c1, eps, stages, L.d_status);
      });
      L.count();
      return;
    }
  }
  const int threads = row_threads(g.d);
  const size_t smem = g.d <= threads * 8 ? 0 : (size_t)g.d * sizeof(float);  // staging only if a row takes several passes
  if (inv != nullptr && smem == 0)
    DLLM_DISPATCH(dtype, (launch_k(L, tail_kernel<T, true>, dim3(c1 - c0), dim3(threads), smem, part, inv, x, Ac_layer,
                                   Fc_layer, gain, (T*)u, g, c0, eps)));
  else
    DLLM_DISPATCH(dtype, (launch_k(L, tail_kernel<T, false>, dim3(c1 - c0), dim3(threads), smem, part, inv, x, Ac_layer,
                                   Fc_layer, gain, (T*)u, g, c0, eps)));
  L.count();
}

// ------------------------------------------------------------------ selection + gather in one launch
// grid (a_seq, B): CTA (i, b) produces row i of sequence b's active list and
// copies that row of u into ua.  Rows below the prompt length (on a prompt
// refresh) are the prompt rows; the others are the selected response rows, for
// which every CTA repeats the bottom-k selection of its sequence instead of
// waiting for another launch.  CTA (0, b) writes the index list, the active
// list and its inverse.
template <typename T>
__global__ void select_gather_kernel(const float* __restrict__ sim, const int32_t* __restrict__ forced, int mode,
                                     int ksel, int32_t* __restrict__ sel, int32_t* __restrict__ act,
                                     int32_t* __restrict__ inv, const T* __restrict__ u, T* __restrict__ ua, Geo g,
                                     int refresh_prompt) {
  pdl_wait();
  pdl_trigger();
  extern __shared__ unsigned long long keys[];  // R keys, R slots (int), R / 8 bytes of ballot words
  const int R = g.R, b = blockIdx.y, ridx = blockIdx.x;
  __shared__ int my_j;
  const int np = refresh_prompt ? g.P : 0;
  const int a_seq = np + ksel;
  const bool leader = ridx == 0;
  if (mode == 1 && R <= (int)blockDim.x && (ridx >= np || leader)) {
    // One key per thread (the usual case, R <= 256): key -> shared memory, rank against all keys, one ballot
    // word per warp, position among the selected rows from the ballot words: three barriers in all.
    uint32_t* words = reinterpret_cast<uint32_t*>(keys + R);
    const int j = threadIdx.x;
    unsigned long long kj = ~0ull;
    if (j < R) {
      const float s = __ldcg(sim + (size_t)b * R + j);
      const float qf = fminf(fmaxf(rintf(s * 1048576.0f), -2147483520.0f), 2147483520.0f);
      const long long q = (s == s) ? (long long)qf + (1ll << 31) : 0ll;
      kj = ((unsigned long long)q << 32) | (unsigned)j;
      keys[j] = kj;
    }
    __syncthreads();
    int rank = 0;
    if (j < R) {
#pragma unroll 8
      for (int i = 0; i + 1 < R; i += 2) {
        const ulonglong2 kk = *reinterpret_cast<const ulonglong2*>(keys + i);
        rank += (kk.x < kj) + (kk.y < kj);
      }
      if (R & 1) rank += (keys[R - 1] < kj);
    }
    const bool f = j < R && rank < ksel;
    const unsigned bal = __ballot_sync(0xffffffffu, f);
    if ((j & 31) == 0) words[j >> 5] = bal;
    __syncthreads();
    int r = -1;
    if (f) {
      r = __popc(bal & ((1u << (j & 31)) - 1u));
      for (int w = 0; w < (j >> 5); ++w) r += __popc(words[w]);
      if (r == ridx - np) my_j = j;
    }
    if (leader) {
      if (j < R) {
        inv[(size_t)b * R + j] = r >= 0 ? b * a_seq + np + r : -1;
        if (r >= 0) {
          sel[(size_t)b * R + r] = j;
          act[(size_t)b * a_seq + np + r] = b * R + j;
        }
      }
      for (int i = threadIdx.x; i < np; i += blockDim.x) {
        act[(size_t)b * a_seq + i] = g.B * R + b * g.P + i;
        inv[(size_t)g.B * R + (size_t)b * g.P + i] = b * a_seq + i;
      }
    }
    __syncthreads();
  } else if (ridx >= np || leader) {
    const int32_t* slot = select_sequence(keys, sim, forced, mode, ksel, sel, act, inv, g, np, b, leader);
    if (ridx >= np)
      for (int j = threadIdx.x; j < R; j += blockDim.x)
        if (slot[j] == ridx - np) my_j = j;
    __syncthreads();
  }
  const int c = ridx < np ? g.B * R + b * g.P + ridx : b * R + my_j;
  copy_row16(reinterpret_cast<const uint4*>(u + (size_t)c * g.d),
             reinterpret_cast<uint4*>(ua + ((size_t)b * a_seq + ridx) * g.d), g.d * (int)sizeof(T) / 16);
}

void launch_select_gather(const Launch& L, int dtype, const float* sim, const int32_t* forced, int mode, int ksel,
                          int32_t* sel, int32_t* act, int32_t* inv, const void* u, void* ua, Geo g,
                          int refresh_prompt) {
  const int a_seq = (refresh_prompt ? g.P : 0) + ksel;
  if (a_seq <= 0) return;
  const size_t smem = (size_t)g.R * 13 + 16;
  DLLM_DISPATCH(dtype, (launch_k(L, select_gather_kernel<T>, dim3(a_seq, g.B), dim3(256), smem, sim, forced, mode, ksel,
                                 sel, act, inv, (const T*)u, (T*)ua, g, refresh_prompt)));
  L.count();
}

// ------------------------------------------------------------------ greedy estimate + confidence (Eq. 4)
// Online (max, argmax, sum exp) per thread, merged across the block.  Ties go
// to the lowest id.  The mask id is skipped: the estimate is never [MASK].
// blk_len > 0: logits row r belongs to response row blk_start + r % blk_len of sequence r / blk_len (the rows
// of one generation block); otherwise logits row r is carried response row r.
__global__ void argmax_conf_kernel(const float* __restrict__ logits, int vocab, int mask_id, int32_t* __restrict__ x0,
                                   float* __restrict__ conf, int R, int blk_start, int blk_len) {
  pdl_wait();
  pdl_trigger();
  __shared__ MaxSum sh[32];
  const size_t row = blockIdx.x;
  const float* lr = logits + row * vocab;
  MaxSum t{-INFINITY, 0.f, 0x7fffffff};
  // 16 floats per thread and trip (four 16-byte loads in flight); rows are 16-byte aligned when vocab % 4 == 0
  const int v16 = ((vocab & 3) == 0) ? vocab / 16 * 16 : 0;
  for (int i0 = threadIdx.x * 4; i0 < v16; i0 += blockDim.x * 16) {
    float4 q[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int i = i0 + k * blockDim.x * 4;
      q[k] = i < v16 ? *reinterpret_cast<const float4*>(lr + i) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int i = i0 + k * blockDim.x * 4;
      if (i >= v16) continue;
      const float e[4] = {q[k].x, q[k].y, q[k].z, q[k].w};
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (i + j != mask_id) online_add(t, e[j], i + j);
    }
  }
  for (int i = v16 + threadIdx.x; i < vocab; i += blockDim.x)
    if (i != mask_id) online_add(t, lr[i], i);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    MaxSum q;
    q.m = __shfl_xor_sync(0xffffffffu, t.m, o);
    q.s = __shfl_xor_sync(0xffffffffu, t.s, o);
    q.a = __shfl_xor_sync(0xffffffffu, t.a, o);
    t = merge(t, q);
  }
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (lane == 0) sh[w] = t;
  __syncthreads();
  if (w == 0) {
    const int nw = blockDim.x >> 5;
    t = (lane < nw) ? sh[lane] : MaxSum{-INFINITY, 0.f, 0x7fffffff};
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      MaxSum q;
      q.m = __shfl_xor_sync(0xffffffffu, t.m, o);
      q.s = __shfl_xor_sync(0xffffffffu, t.s, o);
      q.a = __shfl_xor_sync(0xffffffffu, t.a, o);
      t = merge(t, q);
    }
    if (lane == 0) {
      const size_t out = blk_len > 0 ? (row / blk_len) * R + blk_start + row % blk_len : row;
      x0[out] = t.a;
      conf[out] = 1.f / t.s;
    }
  }
}

void launch_argmax_conf(const Launch& L, const float* logits, int rows, int vocab, int mask_id, int32_t* x0,
                        float* conf, int R, int blk_start, int blk_len) {
  if (rows <= 0) return;
  launch_k(L, argmax_conf_kernel, dim3(rows), dim3(512), 0, logits, vocab, mask_id, x0, conf, R, blk_start, blk_len);
  L.count();
}

// Merge of the per-tile (max, argmax, sum exp) records the LM-head projection writes from its epilogue
// (records [rows][n_tiles] of {max, sum, argmax bits, -}): one warp per row, tiles in a fixed order.
__global__ void estimate_merge_kernel(const float4* __restrict__ rec, int rows, int n_tiles, int32_t* __restrict__ x0,
                                      float* __restrict__ conf, int R, int blk_start, int blk_len) {
  pdl_wait();
  pdl_trigger();
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= rows) return;
  MaxSum t{-INFINITY, 0.f, 0x7fffffff};
  for (int i0 = lane; i0 < n_tiles; i0 += 32 * 8) {  // eight records in flight per lane
    float4 q[8];
#pragma unroll
    for (int k = 0; k < 8; ++k)
      if (i0 + 32 * k < n_tiles) q[k] = __ldcg(rec + (size_t)row * n_tiles + i0 + 32 * k);
#pragma unroll
    for (int k = 0; k < 8; ++k)
      if (i0 + 32 * k < n_tiles) t = merge(t, MaxSum{q[k].x, q[k].y, __float_as_int(q[k].z)});
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    MaxSum q;
    q.m = __shfl_xor_sync(0xffffffffu, t.m, o);
    q.s = __shfl_xor_sync(0xffffffffu, t.s, o);
    q.a = __shfl_xor_sync(0xffffffffu, t.a, o);
    t = merge(t, q);
  }
  if (lane == 0) {
    const size_t out = blk_len > 0 ? (size_t)(row / blk_len) * R + blk_start + row % blk_len : (size_t)row;
    x0[out] = t.a;
    conf[out] = 1.f / t.s;
  }
}

void launch_estimate_merge(const Launch& L, const float* records, int rows, int n_tiles, int32_t* x0, float* conf,
                           int R, int blk_start, int blk_len) {
  if (rows <= 0) return;
  // two rows per CTA: 256 rows spread over 128 SMs (each warp walks its row's records in a few round trips)
  launch_k(L, estimate_merge_kernel, dim3((rows + 1) / 2), dim3(64), 0, reinterpret_cast<const float4*>(records), rows,
           n_tiles, x0, conf, R, blk_start, blk_len);
  L.count();
}

// ------------------------------------------------------------------ rows of one generation block, all sequences
// dst[b * len + i] = src[b * R + start + i] (rows of d elements): the final-norm rows the LM head needs when only
// the block a step works on is predicted.
template <typename T>
__global__ void gather_block_rows_kernel(const T* __restrict__ src, T* __restrict__ dst, int R, int start, int len,
                                         int d) {
  pdl_wait();
  pdl_trigger();
  const int r = blockIdx.x, b = r / len, i = r - b * len;
  copy_row16(reinterpret_cast<const uint4*>(src + ((size_t)b * R + start + i) * d),
             reinterpret_cast<uint4*>(dst + (size_t)r * d), d * (int)sizeof(T) / 16);
}

void launch_gather_block_rows(const Launch& L, int dtype, const void* src, void* dst, int B, int R, int start, int len,
                              int d) {
  if (B * len <= 0) return;
  DLLM_DISPATCH(dtype, (launch_k(L, gather_block_rows_kernel<T>, dim3(B * len), dim3(128), 0, (const T*)src, (T*)dst, R,
                                 start, len, d)));
  L.count();
}

// ------------------------------------------------------------------ low-confidence transition (Eq. 5)
// One block per sequence.  Candidates: masked positions of the block.  Rank by
// (confidence descending, position ascending); the first n_transfer are unmasked.
__global__ void remask_kernel(int32_t* __restrict__ tokens, const int32_t* __restrict__ x0,
                              const float* __restrict__ conf, Geo g, int mask_id, int block_start, int block_len,
                              int n_transfer) {
  pdl_wait();
  pdl_trigger();
  extern __shared__ unsigned long long keys[];
  const int b = blockIdx.x;
  int32_t* tok = tokens + (size_t)b * g.n + g.P;
  const float* cf = conf + (size_t)b * g.R;
  for (int t = threadIdx.x; t < block_len; t += blockDim.x) {
    const int j = block_start + t;
    unsigned long long k = ~0ull;
    if (tok[j] == mask_id) {
      const float c = cf[j];
      const unsigned bits = (c == c) ? __float_as_uint(fmaxf(c, 0.f)) : 0u;  // conf >= 0: bit order = value order
      k = ((unsigned long long)(0xFFFFFFFFu - bits) << 32) | (unsigned)t;
    }
    keys[t] = k;
  }
  __syncthreads();
  for (int t = threadIdx.x; t < block_len; t += blockDim.x) {
    const unsigned long long kt = keys[t];
    if (kt == ~0ull) continue;
    int rank = 0;
    for (int i = 0; i < block_len; ++i) rank += (keys[i] < kt);
    if (rank < n_transfer) tok[block_start + t] = x0[(size_t)b * g.R + block_start + t];
  }
}

void launch_remask(const Launch& L, int32_t* tokens, const int32_t* x0, const float* conf, Geo g, int mask_id,
                   int block_start, int block_len, int n_transfer) {
  launch_k(L, remask_kernel, dim3(g.B), dim3(256), (size_t)block_len * 8, tokens, x0, conf, g, mask_id, block_start, block_len,
                                                               n_transfer);
  L.count();
}

// ------------------------------------------------------------------ misc
__global__ void reduce_partials_kernel(Partials part, float* __restrict__ C, size_t total) {
  pdl_wait();
  pdl_trigger();
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    float v = part.p[i];
    const int n_slabs = part.count((int)(i / part.N), (int)(i % part.N));
    for (int s = 1; s < n_slabs; ++s) v += part.p[(size_t)s * part.split_stride + i];
    C[i] = v;
  }
}

void launch_reduce_partials(const Launch& L, Partials part, float* C, int M) {
  const size_t total = (size_t)M * part.N;
  if (!total) return;
  const int blocks = (int)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
  launch_k(L, reduce_partials_kernel, dim3(blocks), dim3(256), 0, part, C, total);
  L.count();
}

template <typename T>
__global__ void to_f32_kernel(const T* __restrict__ src, float* __restrict__ dst, size_t n) {
  pdl_wait();
  pdl_trigger();
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    dst[i] = to_f32<T>(src[i]);
}
template <typename T>
__global__ void from_f32_kernel(const float* __restrict__ src, T* __restrict__ dst, size_t n) {
  pdl_wait();
  pdl_trigger();
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    dst[i] = from_f32<T>(src[i]);
}

void launch_convert_to_f32(const Launch& L, int dtype, const void* src, float* dst, size_t n) {
  if (!n) return;
  const int blocks = (int)((n + 255) / 256 < 148 * 16 ? (n + 255) / 256 : 148 * 16);
  DLLM_DISPATCH(dtype, (launch_k(L, to_f32_kernel<T>, dim3(blocks), dim3(256), 0, (const T*)src, dst, n)));
  L.count();
}
void launch_convert_from_f32(const Launch& L, int dtype, const float* src, void* dst, size_t n) {
  if (!n) return;
  const int blocks = (int)((n + 255) / 256 < 148 * 16 ? (n + 255) / 256 : 148 * 16);
  DLLM_DISPATCH(dtype, (launch_k(L, from_f32_kernel<T>, dim3(blocks), dim3(256), 0, src, (T*)dst, n)));
  L.count();
}

__global__ void mask_column_kernel(float* logits, int rows, int vocab, int mask_id) {
  pdl_wait();
  pdl_trigger();
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r < rows) logits[(size_t)r * vocab + mask_id] = -INFINITY;
}
void launch_mask_column(const Launch& L, float* logits, int rows, int vocab, int mask_id) {
  if (rows <= 0) return;
  launch_k(L, mask_column_kernel, dim3((rows + 127) / 128), dim3(128), 0, logits, rows, vocab, mask_id);
  L.count();
}

}  // namespace dllm

DLLM_TIMELINE_HOOKS(elementwise)
