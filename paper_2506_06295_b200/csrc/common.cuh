// Shared device helpers for the dLLM cached-step kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace dllm {

// Row geometry of a session.  The residual stream and the normalised
// activations are kept in "carried" order: all response rows first
// (c = b*R + j), then all prompt rows (c = B*R + b*P + i), so that the rows
// every step touches (the response) are contiguous for any batch size.
struct Geo {
  int B, P, R, n, d;
};

__host__ __device__ inline void carried_to_pos(int c, const Geo& g, int& b, int& pos) {
  const int BR = g.B * g.R;
  if (c < BR) {
    b = c / g.R;
    pos = g.P + (c - b * g.R);
  } else {
    const int t = c - BR;
    b = t / g.P;
    pos = t - b * g.P;
  }
}

// Where the AttnOut / FFNOut row of a carried row lives.  Four-tensor layout (compact == 0): `base` is the
// layer's [B, n, d] tensor and the row of carried row c sits at its (sequence, position).  Compact layout
// (compact == 1): `base` is the layer's response-only tensor [B, R, d], which is carried order itself, and
// the prompt rows (alive only inside a prompt-refresh step) sit in `prompt`, [B, P, d] in carried order.
struct OutRows {
  void* base;
  void* prompt;
  int compact;
  template <typename T>
  __device__ __forceinline__ T* row(int c, const Geo& g) const {
    if (compact) {
      const int BR = g.B * g.R;
      return c < BR ? static_cast<T*>(base) + (size_t)c * g.d : static_cast<T*>(prompt) + (size_t)(c - BR) * g.d;
    }
    int b, pos;
    carried_to_pos(c, g, b, pos);
    return static_cast<T*>(base) + ((size_t)b * g.n + pos) * g.d;
  }
};

// device status word codes
enum : int {
  ST_OK = 0,
  ST_TIMEOUT_TMA = 101, ST_TIMEOUT_MMA = 102, ST_TIMEOUT_EPI = 103,  // GEMM: operand copies, MMA issuer, epilogue
  ST_TIMEOUT_GRID = 104,
  ST_TIMEOUT_ATTN = 111, ST_TIMEOUT_ATTN_FEW = 112, ST_TIMEOUT_ATTN_UMMA = 113,  // attention: 64-row, few-rows, tcgen05
  ST_TIMEOUT_ROWS_TAIL = 121, ST_TIMEOUT_ROWS_VVERIFY = 122, ST_TIMEOUT_ROWS_OEPI = 123,
  ST_TIMEOUT_ROWS_ROPE = 124,  // streaming row kernels
  ST_RANGE = 201
};

// Programmatic dependent launch.  pdl_wait(): blocks until the preceding grid
// in the stream has completed and its writes are visible (returns at once for
// a launch without the attribute).  pdl_trigger(): lets the next grid become
// resident once every CTA of this grid has called it.
#ifndef DLLM_TIMELINE
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#define DLLM_TIMELINE_HOOKS(stem)
__device__ __forceinline__ void timeline_mark(int) {}
#else
// Timeline build (python -m paper_2506_06295_b200.timeline): thread 0 of every CTA records the global timer
// before and after the dependency wait, so that a replayed CUDA graph yields, per kernel, when its CTAs became
// resident and when its predecessor had completed -- the time a kernel really takes inside the step, which
// neither serialised profiler runs nor event pairs around single launches show.  Records: {grid | block << 48,
// t_resident, t_released, SM id | CTA << 32}, one array and one cursor per translation unit.
static __device__ unsigned long long* g_timeline;
static __device__ unsigned int g_timeline_n;
static __device__ int g_timeline_marks = 1;  // 0: only the launches are recorded, the marks inside kernels are not
constexpr unsigned int TIMELINE_CAP = 1u << 20;
__device__ __forceinline__ unsigned long long timeline_now() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void pdl_wait() {
  const bool rec = threadIdx.x == 0 && g_timeline != nullptr;
  unsigned long long t0 = 0;
  if (rec) t0 = timeline_now();
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (rec) {
    const unsigned long long t1 = timeline_now();
    const unsigned int i = atomicAdd(&g_timeline_n, 1u);
    if (i < TIMELINE_CAP) {
      unsigned int smid;
      asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
      g_timeline[4 * i] = (unsigned long long)gridDim.x | ((unsigned long long)gridDim.y << 16) |
                          ((unsigned long long)gridDim.z << 32) | ((unsigned long long)blockDim.x << 48);
      g_timeline[4 * i + 1] = t0;
      g_timeline[4 * i + 2] = t1;
      g_timeline[4 * i + 3] = smid | ((unsigned long long)(blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z)) << 32);
    }
  }
}
// A point inside a kernel (called by one thread per CTA): the same record with the mark in the top four bits of
// the first word and the time in the second and third.
__device__ __forceinline__ void timeline_mark(int id) {
  if (g_timeline == nullptr || !g_timeline_marks) return;
  const unsigned long long t = timeline_now();
  const unsigned int i = atomicAdd(&g_timeline_n, 1u);
  if (i < TIMELINE_CAP) {
    g_timeline[4 * i] = (unsigned long long)gridDim.x | ((unsigned long long)gridDim.y << 16) |
                        ((unsigned long long)gridDim.z << 32) | ((unsigned long long)(blockDim.x & 0xfff) << 48) |
                        ((unsigned long long)id << 60);
    g_timeline[4 * i + 1] = t;
    g_timeline[4 * i + 2] = t;
    g_timeline[4 * i + 3] = (unsigned long long)(blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z)) << 32;
  }
}
// Host entry points per translation unit: set the record array (device, 32 bytes x 2^20; NULL = off) and clear
// the cursor; read the cursor; switch the marks inside kernels on or off (each costs an atomic and four stores,
// which a figure of what the launches cost should not contain).
#define DLLM_TIMELINE_HOOKS(stem)                                              \
  extern "C" int dllm_timeline_marks_##stem(int on) {                          \
    return (int)cudaMemcpyToSymbol(dllm::g_timeline_marks, &on, sizeof on);    \
  }                                                                            \
  extern "C" int dllm_timeline_set_##stem(unsigned long long* d_records) {     \
    unsigned int zero = 0;                                                     \
    cudaError_t e = cudaMemcpyToSymbol(dllm::g_timeline, &d_records, sizeof d_records); \
    if (e == cudaSuccess) e = cudaMemcpyToSymbol(dllm::g_timeline_n, &zero, sizeof zero); \
    return (int)e;                                                             \
  }                                                                            \
  extern "C" unsigned int dllm_timeline_count_##stem() {                       \
    unsigned int n = 0;                                                        \
    cudaMemcpyFromSymbol(&n, dllm::g_timeline_n, sizeof n);                    \
    return n < dllm::TIMELINE_CAP ? n : dllm::TIMELINE_CAP;                    \
  }
#endif
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename T>
struct Vec8;  // eight consecutive elements, 16-byte (bf16) or 32-byte (fp32) aligned

template <>
struct Vec8<float> {
  static __device__ __forceinline__ void load(const float* p, float (&v)[8]) {
    const float4 a = *reinterpret_cast<const float4*>(p);
    const float4 b = *reinterpret_cast<const float4*>(p + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  }
  // the same through L2 only (data another CTA of the running grid may have written)
  static __device__ __forceinline__ void load_cg(const float* p, float (&v)[8]) {
    const float4 a = __ldcg(reinterpret_cast<const float4*>(p));
    const float4 b = __ldcg(reinterpret_cast<const float4*>(p + 4));
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  }
  static __device__ __forceinline__ void store(float* p, const float (&v)[8]) {
    *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(p + 4) = make_float4(v[4], v[5], v[6], v[7]);
  }
  static __device__ __forceinline__ float round(float x) { return x; }
};

template <>
struct Vec8<__nv_bfloat16> {
  static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&v)[8]) {
    const uint4 u = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
  static __device__ __forceinline__ void load_cg(const __nv_bfloat16* p, float (&v)[8]) {
    const uint4 u = __ldcg(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
  static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&v)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
      w[i] = *reinterpret_cast<const uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  }
  static __device__ __forceinline__ float round(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }
};

template <typename T>
__device__ __forceinline__ float to_f32(T x);
template <>
__device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T>
__device__ __forceinline__ T from_f32(float x);
template <>
__device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Sum over the block; every thread gets the result.  `red` holds >= 32 floats.
__device__ __forceinline__ float block_sum(float v, float* red) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) red[w] = v;
  __syncthreads();
  float t = (lane < nw) ? red[lane] : 0.f;
  return warp_sum(t);
}

// Online (max, argmax, sum exp) for the greedy estimate and its confidence (Eq. 4).  Ties go to the lowest id.
struct MaxSum {
  float m, s;
  int a;
};
__device__ __forceinline__ MaxSum merge(MaxSum p, MaxSum q) {
  if (q.m > p.m || (q.m == p.m && q.a < p.a)) {
    MaxSum t = p;
    p = q;
    q = t;
  }
  if (q.m > -INFINITY) p.s += q.s * expf(q.m - p.m);
  return p;
}
__device__ __forceinline__ void online_add(MaxSum& t, float v, int i) {
  if (v > t.m) {
    t.s = t.s * expf(t.m - v) + 1.f;
    t.m = v;
    t.a = i;
  } else {
    t.s += expf(v - t.m);
  }
}

// Copy of one row of nvec 16-byte words by the whole block: four loads in flight per thread before the first
// store (a plain load-store loop waits a memory round trip per trip).
__device__ __forceinline__ void copy_row16(const uint4* __restrict__ src, uint4* __restrict__ dst, int nvec) {
  for (int i = threadIdx.x; i < nvec; i += blockDim.x * 4) {
    uint4 v[4];
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (i + k * (int)blockDim.x < nvec) v[k] = src[i + k * blockDim.x];
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (i + k * (int)blockDim.x < nvec) dst[i + k * blockDim.x] = v[k];
  }
}

// Three sums over the block at once (one pair of barriers); `red` holds >= 96 floats.
__device__ __forceinline__ void block_sum3(float& a, float& b, float& c, float* red) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  a = warp_sum(a);
  b = warp_sum(b);
  c = warp_sum(c);
  __syncthreads();
  if (lane == 0) {
    red[w] = a;
    red[32 + w] = b;
    red[64 + w] = c;
  }
  __syncthreads();
  a = warp_sum(lane < nw ? red[lane] : 0.f);
  b = warp_sum(lane < nw ? red[32 + lane] : 0.f);
  c = warp_sum(lane < nw ? red[64 + lane] : 0.f);
}

// Threads for a kernel that walks one row of `width` elements eight at a time: one trip when the row fits
// (all loads of a row in flight at once), at most 512.
inline int row_threads(int width) {
  const int t = ((width + 7) / 8 + 31) / 32 * 32;
  return t < 64 ? 64 : t > 512 ? 512 : t;
}

// Sum of n_slabs partial results for eight consecutive columns, slab 0 first.
// The loads of up to four slabs are issued together so that their latencies
// overlap; the adds keep the slab order.
__device__ __forceinline__ void sum_partials8(const float* part, size_t split_stride, int n_slabs, size_t off,
                                              float (&v)[8]) {
  Vec8<float>::load_cg(part + off, v);
  int s = 1;
  for (; s + 4 <= n_slabs; s += 4) {
    float t[4][8];
#pragma unroll
    for (int q = 0; q < 4; ++q) Vec8<float>::load_cg(part + (size_t)(s + q) * split_stride + off, t[q]);
#pragma unroll
    for (int q = 0; q < 4; ++q)
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] += t[q][i];
  }
  if (s < n_slabs) {  // up to three left: loaded together (index clamped, the surplus is not added)
    float t[3][8];
#pragma unroll
    for (int q = 0; q < 3; ++q)
      Vec8<float>::load_cg(part + (size_t)min(s + q, n_slabs - 1) * split_stride + off, t[q]);
#pragma unroll
    for (int q = 0; q < 3; ++q)
      if (s + q < n_slabs) {
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] += t[q][i];
      }
  }
}

}  // namespace dllm
