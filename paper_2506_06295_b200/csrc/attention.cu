// Non-causal attention of the active query rows over ALL n cached keys of their
// sequence (Sec. A.7: the recomputed rows attend to the full sequence), with
// grouped KV heads (query head h reads KV head h / (H/Hkv)).
//
// attn_simt_kernel: fp32 arithmetic on the plain ALUs for any storage type.
// One CTA = 16 query rows of one sequence x one query head; keys and values
// are staged 32 rows at a time in shared memory; each warp owns 4 queries,
// lane = key for the scores, lane = output column for P*V; online softmax.
#include <stdio.h>

#include <mutex>

#include "../../include/dllm.h"
#include "internal.h"
#include "tma.cuh"

namespace dllm {

namespace {

constexpr int TQ = 16;   // queries per CTA
constexpr int KC = 32;   // keys per chunk
constexpr int HD_MAX = 128;

template <typename T>
__global__ void __launch_bounds__(128) attn_simt_kernel(const T* __restrict__ q, const T* __restrict__ Kc,
                                                        const T* __restrict__ Vc, T* __restrict__ o, int a_seq, int n,
                                                        int H, int Hkv, int hd, float scale) {
  __shared__ float qs[TQ][HD_MAX];
  __shared__ float Ks[KC][HD_MAX + 1];
  __shared__ float Vs[KC][HD_MAX];
  __shared__ float ps[4][4][KC];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q0 = blockIdx.x * TQ, h = blockIdx.y, b = blockIdx.z;
  const int kh = h / (H / Hkv);
  const int dq = H * hd, dkv = Hkv * hd;
  const int nd = hd >> 5;  // output columns per lane
  pdl_wait();
  pdl_trigger();

  for (int e = threadIdx.x; e < TQ * hd; e += blockDim.x) {
    const int r = e / hd, c = e - r * hd;
    const int qi = q0 + r;
    qs[r][c] = (qi < a_seq) ? to_f32<T>(q[((size_t)b * a_seq + qi) * dq + h * hd + c]) * scale : 0.f;
  }
  float m_run[4], l_run[4], acc[4][HD_MAX / 32];
#pragma unroll
  for (int t = 0; t < 4; ++t) {
    m_run[t] = -INFINITY;
    l_run[t] = 0.f;
#pragma unroll
    for (int dd = 0; dd < HD_MAX / 32; ++dd) acc[t][dd] = 0.f;
  }
  const T* Kb = Kc + (size_t)b * n * dkv + kh * hd;
  const T* Vb = Vc + (size_t)b * n * dkv + kh * hd;

  for (int k0 = 0; k0 < n; k0 += KC) {
    __syncthreads();
    for (int e = threadIdx.x; e < KC * hd; e += blockDim.x) {
      const int r = e / hd, c = e - r * hd;
      const int key = k0 + r;
      const bool in = key < n;
      Ks[r][c] = in ? to_f32<T>(Kb[(size_t)key * dkv + c]) : 0.f;
      Vs[r][c] = in ? to_f32<T>(Vb[(size_t)key * dkv + c]) : 0.f;
    }
    __syncthreads();
    float s[4] = {0.f, 0.f, 0.f, 0.f};
    for (int c = 0; c < hd; ++c) {
      const float kv = Ks[lane][c];
#pragma unroll
      for (int t = 0; t < 4; ++t) s[t] = fmaf(qs[warp * 4 + t][c], kv, s[t]);
    }
    const bool valid = (k0 + lane) < n;
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const float sv = valid ? s[t] : -INFINITY;
      const float m_new = fmaxf(m_run[t], warp_max(sv));
      const float corr = expf(m_run[t] - m_new);   // first chunk: exp(-inf) = 0
      const float p = valid ? expf(sv - m_new) : 0.f;
      l_run[t] = l_run[t] * corr + warp_sum(p);
      m_run[t] = m_new;
#pragma unroll
      for (int dd = 0; dd < HD_MAX / 32; ++dd) acc[t][dd] *= corr;
      ps[warp][t][lane] = p;
    }
    __syncwarp();
    for (int key = 0; key < KC; ++key) {
      float vv[HD_MAX / 32];
#pragma unroll
      for (int dd = 0; dd < HD_MAX / 32; ++dd) vv[dd] = (dd < nd) ? Vs[key][lane + 32 * dd] : 0.f;
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const float p = ps[warp][t][key];
#pragma unroll
        for (int dd = 0; dd < HD_MAX / 32; ++dd) acc[t][dd] = fmaf(p, vv[dd], acc[t][dd]);
      }
    }
    __syncwarp();
  }
#pragma unroll
  for (int t = 0; t < 4; ++t) {
    const int qi = q0 + warp * 4 + t;
    if (qi >= a_seq) continue;
    const float inv = 1.f / l_run[t];
    T* orow = o + ((size_t)b * a_seq + qi) * dq + h * hd;
#pragma unroll
    for (int dd = 0; dd < HD_MAX / 32; ++dd)
      if (dd < nd) orow[lane + 32 * dd] = from_f32<T>(acc[t][dd] * inv);
  }
}


// ============================================================================
// attn_mma_kernel (bf16): flash-style attention on the tensor cores.
//
// One CTA = 64 "virtual rows" of one (sequence, KV head) x one split of the key
// range.  A virtual row is a (query, query-head-of-the-group) pair, so with
// grouped KV heads the G query heads that share a KV head are packed along the
// row dimension and every K/V tile is loaded once for all of them.  K and V
// tiles of 64 keys arrive by TMA (3-D map [B, n, dkv], 128-byte swizzle, keys
// beyond n zero-filled) into a two-stage ring; each of the 4 warps owns 16 rows
// and runs mma.sync m16n8k16 for S = Q K^T and O += P V with the online softmax
// in fp32 registers (exp2 with the scale folded in).  When few rows are active
// the key range is split over blockIdx.z so that >= 148 CTAs read K/V; splits
// write unnormalised partial outputs plus (max, sum) and attn_combine_kernel
// merges them.
// ============================================================================
constexpr int AT_ROWS = 64;   // virtual rows per CTA
constexpr int AT_KEYS = 64;   // keys per tile

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}
// Byte offset of the 16-byte chunk `dc` (8 bf16) of row `row` in a tile stored
// as panels of 64 columns: panel = [rows][128 bytes], chunk index XOR (row % 8).
template <int ROWS>
__device__ __forceinline__ uint32_t tile_off(int row, int dc) {
  return (uint32_t)((dc >> 3) * (ROWS * 128) + row * 128 + (((dc & 7) ^ (row & 7)) << 4));
}

template <int HD>
__global__ void __launch_bounds__(128) attn_mma_kernel(const __grid_constant__ CUtensorMap tmK,
                                                       const __grid_constant__ CUtensorMap tmV,
                                                       const __nv_bfloat16* __restrict__ q,
                                                       __nv_bfloat16* __restrict__ o, float* __restrict__ o_part,
                                                       float* __restrict__ ml_part, int a_seq, int n, int H, int Hkv,
                                                       int S, int keys_per_split, float scale_log2,
                                                       int* __restrict__ status) {
  constexpr int PANELS = HD / 64;
  constexpr uint32_t TILE_BYTES = AT_KEYS * HD * 2;   // one K or V tile
  constexpr uint32_t STAGE_BYTES = 2 * TILE_BYTES;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[2];
  __shared__ int abort_flag;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t q_s = base;                         // [64 rows][HD] in panels
  const uint32_t kv_s = base + AT_ROWS * HD * 2;     // 2 stages x (K tile, V tile)
  uint8_t* q_gen = smem_raw + (base - smem_u32(smem_raw));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = H / Hkv;
  const int kh = blockIdx.y;
  const int b = blockIdx.z / S, split = blockIdx.z - b * S;
  const int row0 = blockIdx.x * AT_ROWS;
  const int n_rows = a_seq * G;
  const int key_lo = split * keys_per_split;
  const int key_hi = min(n, key_lo + keys_per_split);
  const int n_tiles = (key_hi - key_lo + AT_KEYS - 1) / AT_KEYS;   // >= 1 by construction
  const int dq = H * HD;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&full_bar[0]), 1);
    mbar_init(smem_u32(&full_bar[1]), 1);
    mbar_fence_init();
  }
  __syncthreads();
  auto issue = [&](int t) {
    const int st = t & 1;
    const uint32_t fb = smem_u32(&full_bar[st]);
    mbar_expect_tx(fb, STAGE_BYTES);
    const uint32_t dst = kv_s + st * STAGE_BYTES;
    const int key0 = key_lo + t * AT_KEYS;
#pragma unroll
    for (int p = 0; p < PANELS; ++p) {
      tma_load_3d(dst + p * (AT_KEYS * 128), &tmK, fb, kh * HD + p * 64, key0, b);
      tma_load_3d(dst + TILE_BYTES + p * (AT_KEYS * 128), &tmV, fb, kh * HD + p * 64, key0, b);
    }
  };
  pdl_wait();  // K, V and Q come from the preceding kernels
  pdl_trigger();
  if (threadIdx.x == 0) {
    issue(0);
    if (n_tiles > 1) issue(1);
  }
  // Q tile: plain 16-byte loads into the swizzled layout (rows of other heads /
  // past the end are zero)
  for (int e = threadIdx.x; e < AT_ROWS * (HD / 8); e += blockDim.x) {
    const int r = e / (HD / 8), dc = e - r * (HD / 8);
    const int vr = row0 + r;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (vr < n_rows) {
      const int qi = vr / G, g = vr - qi * G;
      v = *reinterpret_cast<const uint4*>(q + ((size_t)b * a_seq + qi) * dq + (kh * G + g) * HD + dc * 8);
    }
    *reinterpret_cast<uint4*>(q_gen + tile_off<AT_ROWS>(r, dc)) = v;
  }
  __syncthreads();
  // Q fragments of this warp's 16 rows stay in registers
  uint32_t qf[HD / 16][4];
#pragma unroll
  for (int ks = 0; ks < HD / 16; ++ks) {
    const int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
    const int dc = ks * 2 + (lane >> 4);
    ldsm_x4(q_s + tile_off<AT_ROWS>(row, dc), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
  }
  float oacc[HD / 8][4];
#pragma unroll
  for (int i = 0; i < HD / 8; ++i) oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  bool ok = true;

  for (int t = 0; t < n_tiles; ++t) {
    const int st = t & 1;
    ok = mbar_wait(smem_u32(&full_bar[st]), (uint32_t)(t >> 1) & 1u, &abort_flag);
    ok = __syncthreads_and(ok);               // CTA-uniform: nobody is left behind at a barrier
    if (!ok) break;
    const uint32_t k_s = kv_s + st * STAGE_BYTES, v_s = k_s + TILE_BYTES;
    // ---- S = Q K^T for 16 rows x 64 keys
    float sacc[AT_KEYS / 8][4];
#pragma unroll
    for (int i = 0; i < AT_KEYS / 8; ++i) sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < HD / 16; ++ks) {
#pragma unroll
      for (int jp = 0; jp < AT_KEYS / 16; ++jp) {
        const int key = jp * 16 + (lane & 7) + (lane >> 4) * 8;
        const int dc = ks * 2 + ((lane >> 3) & 1);
        uint32_t r0, r1, r2, r3;
        ldsm_x4(k_s + tile_off<AT_KEYS>(key, dc), r0, r1, r2, r3);
        mma_bf16_16816(sacc[2 * jp], qf[ks], r0, r1);
        mma_bf16_16816(sacc[2 * jp + 1], qf[ks], r2, r3);
      }
    }
    // ---- online softmax (rows lane/4 and lane/4 + 8)
    const int key_base = key_lo + t * AT_KEYS + 2 * (lane & 3);
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nb = 0; nb < AT_KEYS / 8; ++nb) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int key = key_base + nb * 8 + (c & 1);
        const float v = (key < key_hi) ? sacc[nb][c] * scale_log2 : -INFINITY;
        sacc[nb][c] = v;
        mx[c >> 1] = fmaxf(mx[c >> 1], v);
      }
    }
    float corr[2];
#pragma unroll
    for (int h2 = 0; h2 < 2; ++h2) {
      mx[h2] = fmaxf(mx[h2], __shfl_xor_sync(0xffffffffu, mx[h2], 1));
      mx[h2] = fmaxf(mx[h2], __shfl_xor_sync(0xffffffffu, mx[h2], 2));
      const float m_new = fmaxf(m_run[h2], mx[h2]);      // finite: every tile has a valid key
      corr[h2] = exp2f(m_run[h2] - m_new);
      m_run[h2] = m_new;
      l_run[h2] *= corr[h2];
    }
#pragma unroll
    for (int nb = 0; nb < AT_KEYS / 8; ++nb) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const float p = exp2f(sacc[nb][c] - m_run[c >> 1]);
        sacc[nb][c] = p;
        l_run[c >> 1] += p;
      }
    }
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) {
      oacc[i][0] *= corr[0];
      oacc[i][1] *= corr[0];
      oacc[i][2] *= corr[1];
      oacc[i][3] *= corr[1];
    }
    // ---- O += P V
#pragma unroll
    for (int kk = 0; kk < AT_KEYS / 16; ++kk) {
      uint32_t pf[4];
      pf[0] = pack_bf16(sacc[2 * kk][0], sacc[2 * kk][1]);
      pf[1] = pack_bf16(sacc[2 * kk][2], sacc[2 * kk][3]);
      pf[2] = pack_bf16(sacc[2 * kk + 1][0], sacc[2 * kk + 1][1]);
      pf[3] = pack_bf16(sacc[2 * kk + 1][2], sacc[2 * kk + 1][3]);
#pragma unroll
      for (int dp = 0; dp < HD / 16; ++dp) {
        const int key = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        const int dc = dp * 2 + (lane >> 4);
        uint32_t r0, r1, r2, r3;
        ldsm_x4_trans(v_s + tile_off<AT_KEYS>(key, dc), r0, r1, r2, r3);
        mma_bf16_16816(oacc[2 * dp], pf, r0, r1);
        mma_bf16_16816(oacc[2 * dp + 1], pf, r2, r3);
      }
    }
    __syncthreads();                         // every warp is done with stage st
    if (threadIdx.x == 0 && t + 2 < n_tiles) issue(t + 2);
  }
  if (!ok) {
    if (threadIdx.x == 0 && status) atomicCAS(status, ST_OK, ST_TIMEOUT_TMA);
    drain_delay();
    return;
  }
  // ---- epilogue
#pragma unroll
  for (int h2 = 0; h2 < 2; ++h2) {
    l_run[h2] += __shfl_xor_sync(0xffffffffu, l_run[h2], 1);
    l_run[h2] += __shfl_xor_sync(0xffffffffu, l_run[h2], 2);
  }
#pragma unroll
  for (int h2 = 0; h2 < 2; ++h2) {
    const int vr = row0 + warp * 16 + (lane >> 2) + h2 * 8;
    if (vr >= n_rows) continue;
    const int qi = vr / G, g = vr - qi * G;
    const size_t orow = ((size_t)b * a_seq + qi) * H + (kh * G + g);   // (row, head) index
    if (S == 1) {
      const float inv = 1.f / l_run[h2];
      __nv_bfloat16* dst = o + orow * HD + 2 * (lane & 3);
#pragma unroll
      for (int i = 0; i < HD / 8; ++i)
        *reinterpret_cast<uint32_t*>(dst + i * 8) = pack_bf16(oacc[i][2 * h2] * inv, oacc[i][2 * h2 + 1] * inv);
    } else {
      const size_t total = (size_t)gridDim.z / S * a_seq * H;           // (row, head) pairs
      float* dst = o_part + ((size_t)split * total + orow) * HD + 2 * (lane & 3);
#pragma unroll
      for (int i = 0; i < HD / 8; ++i)
        *reinterpret_cast<float2*>(dst + i * 8) = make_float2(oacc[i][2 * h2], oacc[i][2 * h2 + 1]);
      if ((lane & 3) == 0) {
        float* ml = ml_part + ((size_t)split * total + orow) * 2;
        ml[0] = m_run[h2];
        ml[1] = l_run[h2];
      }
    }
  }
}

// Merges the key-range splits: out = sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s.
__global__ void attn_combine_kernel(const float* __restrict__ o_part, const float* __restrict__ ml_part,
                                    __nv_bfloat16* __restrict__ o, size_t total, int S, int hd) {
  pdl_wait();
  pdl_trigger();
  const size_t rh = blockIdx.x;
  float M = -INFINITY;
  for (int s = 0; s < S; ++s) M = fmaxf(M, ml_part[((size_t)s * total + rh) * 2]);
  float L = 0.f;
  for (int s = 0; s < S; ++s) {
    const float* ml = ml_part + ((size_t)s * total + rh) * 2;
    L += exp2f(ml[0] - M) * ml[1];
  }
  const float inv = 1.f / L;
  for (int d = threadIdx.x; d < hd; d += blockDim.x) {
    float acc = 0.f;
    for (int s = 0; s < S; ++s)
      acc += exp2f(ml_part[((size_t)s * total + rh) * 2] - M) * o_part[((size_t)s * total + rh) * hd + d];
    o[rh * hd + d] = __float2bfloat16_rn(acc * inv);
  }
}

template <int HD>
cudaError_t launch_mma(const Launch& L, const CUtensorMap& tmK, const CUtensorMap& tmV, const void* q, void* o,
                       float* scratch, int B, int a_seq, int n, int H, int Hkv, int S, int keys_per_split) {
  constexpr int SMEM = AT_ROWS * HD * 2 + 2 * 2 * AT_KEYS * HD * 2 + 1024;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(attn_mma_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  const int G = H / Hkv;
  const size_t total = (size_t)B * a_seq * H;
  float* o_part = scratch;
  float* ml_part = scratch ? scratch + (size_t)S * total * HD : nullptr;
  dim3 grid((a_seq * G + AT_ROWS - 1) / AT_ROWS, Hkv, B * S);
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)HD);
  launch_k(L, attn_mma_kernel<HD>, dim3(grid), dim3(128), SMEM, tmK, tmV, (const __nv_bfloat16*)q, (__nv_bfloat16*)o, o_part,
                                                     ml_part, a_seq, n, H, Hkv, S, keys_per_split, scale_log2,
                                                     L.d_status);
  L.count();
  if (S > 1) {
    launch_k(L, attn_combine_kernel, dim3((unsigned)total), dim3(HD / 2), 0, o_part, ml_part, (__nv_bfloat16*)o, total, S, HD);
    L.count();
  }
  return cudaGetLastError();
}

}  // namespace

// Key-range splits for the tensor-core kernel: enough CTAs to cover the SMs
// when few rows are active, whole 64-key tiles per split.
AttnPlan plan_attention(int B, int a_seq, int n, int H, int Hkv) {
  AttnPlan p;
  const int G = H / Hkv;
  const long tiles = (long)((a_seq * G + AT_ROWS - 1) / AT_ROWS) * Hkv * B;
  int S = 1;
  if (tiles < 148) S = (int)((148 + tiles - 1) / tiles);
  const int key_tiles = (n + AT_KEYS - 1) / AT_KEYS;
  if (S > key_tiles) S = key_tiles;
  const int tiles_per_split = (key_tiles + S - 1) / S;
  p.keys_per_split = tiles_per_split * AT_KEYS;
  p.S = (key_tiles + tiles_per_split - 1) / tiles_per_split;
  p.scratch_floats = p.S > 1 ? (size_t)p.S * B * a_seq * H * (128 + 2) : 0;
  return p;
}

cudaError_t launch_attention(const Launch& L, int dtype, const void* q, const void* Kc, const void* Vc, void* o, int B,
                             int a_seq, int n, int H, int Hkv, int hd, float* scratch, size_t scratch_floats,
                             bool force_simt) {
  if (B <= 0 || a_seq <= 0) return cudaSuccess;
  if (hd > HD_MAX || (hd & 31) || H % Hkv) return cudaErrorInvalidValue;
  const bool tensor = dtype == 1 && !force_simt && (hd == 64 || hd == 128) && ((Hkv * hd) % 8 == 0);
  if (tensor) {
    AttnPlan p = plan_attention(B, a_seq, n, H, Hkv);
    if (p.S > 1 && (!scratch || scratch_floats < p.scratch_floats)) {   // no room for partials: one split
      p.S = 1;
      p.keys_per_split = ((n + AT_KEYS - 1) / AT_KEYS) * AT_KEYS;
    }
    CUtensorMap tmK, tmV;
    if (!get_tensor_map_3d(Kc, (uint64_t)B, (uint64_t)n, (uint64_t)Hkv * hd, AT_KEYS, &tmK) ||
        !get_tensor_map_3d(Vc, (uint64_t)B, (uint64_t)n, (uint64_t)Hkv * hd, AT_KEYS, &tmV))
      return cudaErrorInvalidValue;
    return hd == 64 ? launch_mma<64>(L, tmK, tmV, q, o, scratch, B, a_seq, n, H, Hkv, p.S, p.keys_per_split)
                    : launch_mma<128>(L, tmK, tmV, q, o, scratch, B, a_seq, n, H, Hkv, p.S, p.keys_per_split);
  }
  const float scale = 1.0f / sqrtf((float)hd);
  dim3 grid((a_seq + TQ - 1) / TQ, H, B);
  if (dtype == 0)
    launch_k(L, attn_simt_kernel<float>, dim3(grid), dim3(128), 0, (const float*)q, (const float*)Kc, (const float*)Vc,
                                                        (float*)o, a_seq, n, H, Hkv, hd, scale);
  else
    launch_k(L, attn_simt_kernel<__nv_bfloat16>, dim3(grid), dim3(128), 0, (const __nv_bfloat16*)q, (const __nv_bfloat16*)Kc,
                                                                (const __nv_bfloat16*)Vc, (__nv_bfloat16*)o, a_seq, n,
                                                                H, Hkv, hd, scale);
  L.count();
  return cudaGetLastError();
}

}  // namespace dllm

// ============================================================================
// dllm_attention_noalloc: the tensor-core attention with its split-range
// scratch inside the library image.
//
// Who needs this: code that is not allowed to create device allocations at the
// point where it calls attention -- for example a host thread that only ever
// received raw pointers to Q, K, V and O from another component and has no
// allocator of its own, a caller running while memory is being accounted by
// someone else (a serving process with a fixed memory plan), or a context in
// which cudaMalloc would synchronise the device and stall other streams.  Such
// a caller still passes inputs and the output buffer; only the scratch for the
// partial results of split key ranges comes from the array below.
//
// The array is a file-scope __device__ array: every GPU that loads this
// library holds NOALLOC_SCRATCH_BYTES of it from load until the process exits.
// Its name is only a host-side handle here; the device address is looked up
// once per device with cudaGetSymbolAddress and handed to the kernels.
// ============================================================================
namespace dllm {
namespace {
constexpr size_t NOALLOC_SCRATCH_FLOATS = (size_t)2 * 1024 * 1024;          // 8 MiB
constexpr size_t NOALLOC_SCRATCH_BYTES = NOALLOC_SCRATCH_FLOATS * sizeof(float);
constexpr int NOALLOC_MAX_DEVICES = 64;
static __device__ __align__(256) float g_noalloc_scratch[NOALLOC_SCRATCH_FLOATS];

// Device address of the scratch array on the CURRENT device; looked up on the
// first call per device.
cudaError_t noalloc_scratch(float** out) {
  static std::mutex mu;
  static float* per_device[NOALLOC_MAX_DEVICES] = {};
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(mu);
  if (!per_device[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    if (!p) return cudaErrorInvalidSymbol;
    per_device[dev] = static_cast<float*>(p);
  }
  *out = per_device[dev];
  return cudaSuccess;
}
}  // namespace
}  // namespace dllm

extern "C" dllm_status dllm_attention_noalloc(const void* d_q, const void* d_k, const void* d_v, void* d_o, int B,
                                              int a, int n, int H, int Hkv, int hd, void* stream) {
  using namespace dllm;
  if (!d_q || !d_k || !d_v || !d_o || B <= 0 || a <= 0 || n <= 0 || H <= 0 || Hkv <= 0 || H % Hkv) {
    set_last_error("dllm_attention_noalloc: bad arguments");
    return DLLM_INVALID_ARG;
  }
  if (hd != 64 && hd != 128) {
    set_last_error("dllm_attention_noalloc: bf16 tensor-core path only, head_dim must be 64 or 128");
    return DLLM_UNSUPPORTED;
  }
  const AttnPlan plan = plan_attention(B, a, n, H, Hkv);
  if (plan.scratch_floats > NOALLOC_SCRATCH_FLOATS) {
    char msg[256];
    snprintf(msg, sizeof msg,
             "dllm_attention_noalloc: this shape splits the key range %d ways and needs %zu bytes of scratch, the "
             "built-in array holds %zu; use dllm_attention with a caller-owned scratch buffer",
             plan.S, plan.scratch_floats * sizeof(float), NOALLOC_SCRATCH_BYTES);
    set_last_error(msg);
    return DLLM_UNSUPPORTED;
  }
  float* scratch = nullptr;
  cudaError_t e = noalloc_scratch(&scratch);
  if (e != cudaSuccess) {
    set_last_error(cudaGetErrorString(e));
    return DLLM_CUDA_ERROR;
  }
  // Nothing in the scratch has to start at zero: every partial (output, max,
  // sum) that attn_combine_kernel reads is written by this call's attn_mma_kernel first.
  Launch L{(cudaStream_t)stream, nullptr, nullptr};
  e = launch_attention(L, DLLM_BF16, d_q, d_k, d_v, d_o, B, a, n, H, Hkv, hd, scratch, NOALLOC_SCRATCH_FLOATS, false);
  if (e != cudaSuccess) {
    set_last_error(cudaGetErrorString(e));
    return DLLM_CUDA_ERROR;
  }
  return DLLM_OK;
}

