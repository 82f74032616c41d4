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
#include "attention_core.cuh"

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
// attn_mma_kernel (bf16): one CTA of 128 threads runs one attn_tile (see
// attention_core.cuh): 64 (query, head-of-group) rows of one (sequence, KV
// head) over one split of the key range.  When few rows are active the key
// range is split over blockIdx.z so that >= 148 CTAs read K/V; splits write
// unnormalised partial outputs plus (max, sum) and attn_combine_kernel merges
// them.
// ============================================================================
template <int HD>
__global__ void __launch_bounds__(128) attn_mma_kernel(const __grid_constant__ CUtensorMap tmK,
                                                       const __grid_constant__ CUtensorMap tmV,
                                                       const __grid_constant__ CUtensorMap tmQ, int q_by_tma,
                                                       const __nv_bfloat16* __restrict__ q,
                                                       __nv_bfloat16* __restrict__ o, float* __restrict__ o_part,
                                                       float* __restrict__ ml_part, int a_seq, int n, int H, int Hkv,
                                                       int S, int keys_per_split, float scale_log2, int k_static,
                                                       int v_static, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[2];
  __shared__ int abort_flag;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&full_bar[0]), 1);
    mbar_init(smem_u32(&full_bar[1]), 1);
    mbar_fence_init();
    prefetch_tensormap(&tmK);  // the descriptors are fetched while the predecessor still runs
    prefetch_tensormap(&tmV);
    if (q_by_tma) prefetch_tensormap(&tmQ);
  }
  __syncthreads();
  uint32_t kv_iter = 0;   // (attn_tile waits for the launch before this one and releases the dependents)
  const bool ok = attn_tile<HD>((int)threadIdx.x, smem_raw + (base - smem_u32(smem_raw)), base, full_bar, kv_iter,
                                &abort_flag, &tmK, &tmV, q, o, o_part, ml_part, a_seq, n, H, Hkv, S, keys_per_split,
                                scale_log2, (int)gridDim.z / S, (int)blockIdx.x, (int)blockIdx.y, (int)blockIdx.z,
                                q_by_tma ? &tmQ : nullptr, k_static, v_static);
  if (!ok && threadIdx.x == 0 && status) atomicCAS(status, ST_OK, ST_TIMEOUT_ATTN);
}

// ============================================================================
// attn_mma_few_kernel (bf16): the same attention when a KV head has at most 16 * RG (query, head-of-group) rows
// (RG = 1 or 2: a few selected rows against a long prompt).  A CTA holds RG * KW warps: warp (rg, kw) works on
// rows 16 rg .. 16 rg + 15 and on the key tiles kw, kw + KW, ... of the CTA's split, so KW tiles are in the
// load -> QK^T -> softmax -> PV chain at once instead of one; every way kw has its own one-stage K/V buffer and
// barrier, refilled by its first warp.  The ways are merged through shared memory in way order.  Splits over
// CTAs, partials and the merge kernel as in attn_mma_kernel.
// ============================================================================
template <int HD, int RG, int KW>
__global__ void __launch_bounds__(32 * RG * KW, RG == 2 ? 2 : 1)
    attn_mma_few_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                        const __nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ o,
                        float* __restrict__ o_part, float* __restrict__ ml_part, int a_seq, int n, int H, int Hkv,
                        int S, int keys_per_split, float scale_log2, int k_static, int v_static,
                        int* __restrict__ status) {
  constexpr uint32_t Q_BYTES = AT_ROWS * HD * 2;          // the tile layout of the 64-row kernel; RG * 16 rows used
  constexpr uint32_t TILE_BYTES = AT_KEYS * HD * 2, STAGE_BYTES = 2 * TILE_BYTES;
  constexpr int ROWS = 16 * RG, NT = 32 * RG * KW, PANELS = HD / 64;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[KW];
  __shared__ float ml_s[KW > 1 ? KW - 1 : 1][RG][32][4];
  __shared__ int abort_flag;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_gen = smem_raw + (base - smem_u32(smem_raw));
  const int warp = (int)threadIdx.x >> 5, lane = (int)threadIdx.x & 31;
  const int rg = warp % RG, kw = warp / RG;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int w = 0; w < KW; ++w) mbar_init(smem_u32(&full_bar[w]), 1);
    mbar_fence_init();
    prefetch_tensormap(&tmK);
    prefetch_tensormap(&tmV);
  }
  __syncthreads();

  const int G = H / Hkv, kh = blockIdx.y;
  const int b = blockIdx.z / S, split = blockIdx.z - b * S;
  const int row0 = blockIdx.x * ROWS, n_rows = a_seq * G, dq = H * HD;
  const int key_lo = split * keys_per_split, key_hi = min(n, key_lo + keys_per_split);
  const int n_tiles = (key_hi - key_lo + AT_KEYS - 1) / AT_KEYS;   // >= 1 by construction of the plan
  const uint32_t q_s = base, kv_s = base + Q_BYTES + (uint32_t)kw * STAGE_BYTES;
  volatile int* abortp = &abort_flag;

  // key tile t of the split into this way's buffer; what: 1 = the K tile, 2 = the V tile, 4 = arm the barrier
  auto issue = [&](int t, int what) {
    const uint32_t fb = smem_u32(&full_bar[kw]);
    if (what & 4) mbar_expect_tx(fb, STAGE_BYTES);
    const int key0 = key_lo + t * AT_KEYS;
#pragma unroll
    for (int p = 0; p < PANELS; ++p) {
      if (what & 1) tma_load_3d(kv_s + p * (AT_KEYS * 128), &tmK, fb, kh * HD + p * 64, key0, b);
      if (what & 2) tma_load_3d(kv_s + TILE_BYTES + p * (AT_KEYS * 128), &tmV, fb, kh * HD + p * 64, key0, b);
    }
  };
  // The way's first tile: what only holds rows older than the launch before this one (see launch_attention) is
  // requested ahead of the dependency wait, the rest after it.
  const bool issuer = rg == 0 && lane == 0 && kw < n_tiles;
  int early = 0;
  if (issuer) {
    const int hi = min(key_lo + (kw + 1) * AT_KEYS, n);
    early = (hi <= k_static ? 1 : 0) | (hi <= v_static ? 2 : 0);
    if (early) issue(kw, early | 4);
  }
  pdl_wait();  // Q and the newest K rows come from the launch before this one
  pdl_trigger();
  if (issuer && early != 3) issue(kw, (3 & ~early) | (early ? 0 : 4));
  // Q rows of the tile: 16-byte loads into the swizzled layout (rows past the end are zero)
  {
    constexpr int CHUNKS = ROWS * (HD / 8);
    constexpr int PER = (CHUNKS + NT - 1) / NT;
    uint4 qv[PER];
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      const int e = (int)threadIdx.x + i * NT;
      const int r = e / (HD / 8), dc = e - r * (HD / 8);
      const int vr = row0 + r;
      qv[i] = make_uint4(0, 0, 0, 0);
      if (e < CHUNKS && vr < n_rows) {
        const int qi = vr / G, g = vr - qi * G;
        qv[i] = __ldcg(reinterpret_cast<const uint4*>(q + ((size_t)b * a_seq + qi) * dq + (kh * G + g) * HD + dc * 8));
      }
    }
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      const int e = (int)threadIdx.x + i * NT;
      const int r = e / (HD / 8), dc = e - r * (HD / 8);
      if (e < CHUNKS) *reinterpret_cast<uint4*>(base_gen + tile_off<AT_ROWS>(r, dc)) = qv[i];
    }
  }
  __syncthreads();

  AttnAcc<HD> acc;
  attn_acc_clear(acc);
  bool ok = true;
  int it = 0;
  for (int t = kw; t < n_tiles; t += KW, ++it) {
    ok = mbar_wait(smem_u32(&full_bar[kw]), (uint32_t)it & 1u, abortp);
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) break;
    attn_warp_tile<HD>(lane, rg, q_s, kv_s, kv_s + TILE_BYTES, key_lo + t * AT_KEYS, key_hi, scale_log2, acc);
    if (t + KW < n_tiles) {
      // every warp of the way has read the buffer before its first warp asks for the next tile
      if constexpr (RG > 1)
        asm volatile("bar.sync %0, %1;" ::"r"(1 + kw), "n"(32 * RG) : "memory");
      else
        __syncwarp();
      if (rg == 0 && lane == 0) issue(t + KW, 1 | 2 | 4);
    }
  }
  attn_warp_finish(acc);

  // ---- merge of the ways, in way order, through each way's own (drained) buffer
  if constexpr (KW > 1) {
    float* o_s = reinterpret_cast<float*>(base_gen + Q_BYTES + (size_t)kw * STAGE_BYTES) + rg * (HD / 2) * 32;
    if (kw > 0) {
      if constexpr (RG > 1)
        asm volatile("bar.sync %0, %1;" ::"r"(1 + kw), "n"(32 * RG) : "memory");  // the way is done with its tiles
      else
        __syncwarp();
      if (ok) {
#pragma unroll
        for (int i = 0; i < HD / 8; ++i)
#pragma unroll
          for (int c = 0; c < 4; ++c) o_s[(i * 4 + c) * 32 + lane] = acc.o[i][c];
        ml_s[kw - 1][rg][lane][0] = acc.m[0];
        ml_s[kw - 1][rg][lane][1] = acc.m[1];
        ml_s[kw - 1][rg][lane][2] = acc.l[0];
        ml_s[kw - 1][rg][lane][3] = acc.l[1];
      }
    }
    ok = __syncthreads_and(ok);
    if (ok && kw == 0) {
      float M[2] = {acc.m[0], acc.m[1]};
#pragma unroll
      for (int w = 1; w < KW; ++w) {
        M[0] = fmaxf(M[0], ml_s[w - 1][rg][lane][0]);
        M[1] = fmaxf(M[1], ml_s[w - 1][rg][lane][1]);
      }
      const float w0[2] = {exp2f(acc.m[0] - M[0]), exp2f(acc.m[1] - M[1])};  // way 0 always has a tile: finite
      acc.l[0] *= w0[0];
      acc.l[1] *= w0[1];
#pragma unroll
      for (int i = 0; i < HD / 8; ++i) {
        acc.o[i][0] *= w0[0];
        acc.o[i][1] *= w0[0];
        acc.o[i][2] *= w0[1];
        acc.o[i][3] *= w0[1];
      }
#pragma unroll
      for (int w = 1; w < KW; ++w) {
        const float* ow = reinterpret_cast<const float*>(base_gen + Q_BYTES + (size_t)w * STAGE_BYTES) + rg * (HD / 2) * 32;
        const float ww[2] = {exp2f(ml_s[w - 1][rg][lane][0] - M[0]), exp2f(ml_s[w - 1][rg][lane][1] - M[1])};  // no tile: 0
        acc.l[0] += ww[0] * ml_s[w - 1][rg][lane][2];
        acc.l[1] += ww[1] * ml_s[w - 1][rg][lane][3];
#pragma unroll
        for (int i = 0; i < HD / 8; ++i)
#pragma unroll
          for (int c = 0; c < 4; ++c) acc.o[i][c] += ww[c >> 1] * ow[(i * 4 + c) * 32 + lane];
      }
      acc.m[0] = M[0];
      acc.m[1] = M[1];
    }
  } else {
    ok = __syncthreads_and(ok);
  }
  if (!ok) {
    if (threadIdx.x == 0 && status) atomicCAS(status, ST_OK, ST_TIMEOUT_ATTN_FEW);
    drain_delay();
    return;
  }
  if (kw != 0) return;

  // ---- way 0 writes the CTA's rows: final output, or the split's unnormalised partial with (max, sum)
#pragma unroll
  for (int h2 = 0; h2 < 2; ++h2) {
    const int vr = row0 + rg * 16 + (lane >> 2) + h2 * 8;
    if (vr >= n_rows) continue;
    const int qi = vr / G, g = vr - qi * G;
    const size_t orow = ((size_t)b * a_seq + qi) * H + (kh * G + g);   // (row, head) index
    if (S == 1) {
      const float inv = 1.f / acc.l[h2];
      __nv_bfloat16* dst = o + orow * HD + 2 * (lane & 3);
#pragma unroll
      for (int i = 0; i < HD / 8; ++i)
        *reinterpret_cast<uint32_t*>(dst + i * 8) = pack_bf16(acc.o[i][2 * h2] * inv, acc.o[i][2 * h2 + 1] * inv);
    } else {
      const size_t total = (size_t)(gridDim.z / S) * a_seq * H;           // (row, head) pairs
      float* dst = o_part + ((size_t)split * total + orow) * HD + 2 * (lane & 3);
#pragma unroll
      for (int i = 0; i < HD / 8; ++i)
        *reinterpret_cast<float2*>(dst + i * 8) = make_float2(acc.o[i][2 * h2], acc.o[i][2 * h2 + 1]);
      if ((lane & 3) == 0) {
        float* ml = ml_part + ((size_t)split * total + orow) * 2;
        ml[0] = acc.m[h2];
        ml[1] = acc.l[h2];
      }
    }
  }
}

// Merges the key-range splits: out = sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s,
// splits in index order.  One warp per (row, head); the (max, sum) pairs of all
// splits are fetched together, then the partial outputs.
template <int MAXS>
__device__ __forceinline__ void combine_row(const float* __restrict__ o_part, const float* __restrict__ ml_part,
                                            __nv_bfloat16* __restrict__ o, size_t total, size_t rh, int S, int hd,
                                            int lane) {
  float2 ml[MAXS];
  float wgt[MAXS];
#pragma unroll
  for (int s = 0; s < MAXS; ++s)
    ml[s] = *reinterpret_cast<const float2*>(ml_part + ((size_t)min(s, S - 1) * total + rh) * 2);
  float M = -INFINITY, L = 0.f;
#pragma unroll
  for (int s = 0; s < MAXS; ++s)
    if (s < S) M = fmaxf(M, ml[s].x);
#pragma unroll
  for (int s = 0; s < MAXS; ++s) {
    wgt[s] = s < S ? exp2f(ml[s].x - M) : 0.f;
    if (s < S) L += wgt[s] * ml[s].y;
  }
  const float inv = 1.f / L;
  // hd <= 128: up to four trips; the partial outputs of all of them are fetched before the first store
  float v[4][MAXS];
#pragma unroll
  for (int t = 0; t < 4; ++t) {
    const int d = lane + 32 * t;
#pragma unroll
    for (int s = 0; s < MAXS; ++s) v[t][s] = d < hd ? o_part[((size_t)min(s, S - 1) * total + rh) * hd + d] : 0.f;
  }
#pragma unroll
  for (int t = 0; t < 4; ++t) {
    const int d = lane + 32 * t;
    float acc = 0.f;
#pragma unroll
    for (int s = 0; s < MAXS; ++s)
      if (s < S) acc += wgt[s] * v[t][s];
    if (d < hd) o[rh * hd + d] = __float2bfloat16_rn(acc * inv);
  }
}

// MAXS: 4, 8 or 16 splits held in registers (one instantiation each, so that few splits cost few registers and
// every CTA of a large merge is resident at once); 0: any number of splits, one at a time.
template <int MAXS>
__global__ void __launch_bounds__(256) attn_combine_kernel(const float* __restrict__ o_part,
                                                           const float* __restrict__ ml_part,
                                                           __nv_bfloat16* __restrict__ o, size_t total, int S, int hd) {
  pdl_wait();
  pdl_trigger();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const size_t rh = (size_t)blockIdx.x * 8 + warp;
  if (rh >= total) return;
  if constexpr (MAXS > 0) {
    combine_row<MAXS>(o_part, ml_part, o, total, rh, S, hd, lane);
  } else {
    float M = -INFINITY, L = 0.f;
    for (int s = 0; s < S; ++s) M = fmaxf(M, ml_part[((size_t)s * total + rh) * 2]);
    for (int s = 0; s < S; ++s) {
      const float* ml = ml_part + ((size_t)s * total + rh) * 2;
      L += exp2f(ml[0] - M) * ml[1];
    }
    const float inv = 1.f / L;
    for (int d = lane; d < hd; d += 32) {
      float acc = 0.f;
      for (int s = 0; s < S; ++s)
        acc += exp2f(ml_part[((size_t)s * total + rh) * 2] - M) * o_part[((size_t)s * total + rh) * hd + d];
      o[rh * hd + d] = __float2bfloat16_rn(acc * inv);
    }
  }
}

cudaError_t launch_combine(const Launch& L, const float* o_part, const float* ml_part, __nv_bfloat16* o, size_t total,
                           int S, int hd) {
  const dim3 grid((unsigned)((total + 7) / 8)), block(256);
  cudaError_t e;
  if (S <= 4) e = launch_k(L, attn_combine_kernel<4>, grid, block, 0, o_part, ml_part, o, total, S, hd);
  else if (S <= 8) e = launch_k(L, attn_combine_kernel<8>, grid, block, 0, o_part, ml_part, o, total, S, hd);
  else if (S <= 16) e = launch_k(L, attn_combine_kernel<16>, grid, block, 0, o_part, ml_part, o, total, S, hd);
  else e = launch_k(L, attn_combine_kernel<0>, grid, block, 0, o_part, ml_part, o, total, S, hd);
  L.count();
  return e;
}

template <int HD>
cudaError_t launch_mma(const Launch& L, const CUtensorMap& tmK, const CUtensorMap& tmV, const void* q, void* o,
                       float* scratch, int B, int a_seq, int n, int H, int Hkv, int S, int keys_per_split, int k_static,
                       int v_static) {
  constexpr int SMEM = AT_ROWS * HD * 2 + 2 * 2 * AT_KEYS * HD * 2 + 1024;
  static DeviceOnce once;
  cudaError_t e0 = once.run(
      [] { return cudaFuncSetAttribute(attn_mma_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM); });
  if (e0 != cudaSuccess) return e0;
  const int G = H / Hkv;
  const size_t total = (size_t)B * a_seq * H;
  float* o_part = scratch;
  float* ml_part = scratch ? scratch + (size_t)S * total * HD : nullptr;
  dim3 grid((a_seq * G + AT_ROWS - 1) / AT_ROWS, Hkv, B * S);
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)HD);
  // with one query head per KV head a row tile is 64 consecutive rows of q: fetched by TMA
  CUtensorMap tmQ = tmK;
  const int q_by_tma = H == Hkv && ((uintptr_t)q & 15) == 0 &&
                       get_tensor_map_2d(q, (uint64_t)B * a_seq, (uint64_t)H * HD, AT_ROWS, &tmQ);
  cudaError_t e = launch_k(L, attn_mma_kernel<HD>, dim3(grid), dim3(128), SMEM, tmK, tmV, tmQ, q_by_tma,
                           (const __nv_bfloat16*)q, (__nv_bfloat16*)o, o_part, ml_part, a_seq, n, H, Hkv, S,
                           keys_per_split, scale_log2, k_static, v_static, L.d_status);
  L.count();
  if (e == cudaSuccess && S > 1) e = launch_combine(L, o_part, ml_part, (__nv_bfloat16*)o, total, S, HD);
  return e != cudaSuccess ? e : cudaGetLastError();
}


}  // namespace

namespace {
template <int HD, int RG, int KW>
cudaError_t launch_few(const Launch& L, const CUtensorMap& tmK, const CUtensorMap& tmV, const void* q, void* o,
                       float* scratch, int B, int a_seq, int n, int H, int Hkv, int S, int keys_per_split, int k_static,
                       int v_static) {
  constexpr int SMEM = AT_ROWS * HD * 2 + KW * 2 * AT_KEYS * HD * 2 + 1024;
  static_assert(SMEM <= 227 * 1024, "the ways' buffers do not fit the shared memory of a CTA");
  static_assert(RG * 32 * (HD / 2) * 4 <= 2 * AT_KEYS * HD * 2, "a way's buffer must hold its warps' outputs");
  static DeviceOnce once;
  cudaError_t e0 = once.run([] {
    return cudaFuncSetAttribute(attn_mma_few_kernel<HD, RG, KW>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
  });
  if (e0 != cudaSuccess) return e0;
  const int G = H / Hkv;
  const size_t total = (size_t)B * a_seq * H;
  float* o_part = scratch;
  float* ml_part = scratch ? scratch + (size_t)S * total * HD : nullptr;
  dim3 grid((a_seq * G + 16 * RG - 1) / (16 * RG), Hkv, B * S);
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)HD);
  cudaError_t e = launch_k(L, attn_mma_few_kernel<HD, RG, KW>, grid, dim3(32 * RG * KW), SMEM, tmK, tmV,
                           (const __nv_bfloat16*)q, (__nv_bfloat16*)o, o_part, ml_part, a_seq, n, H, Hkv, S,
                           keys_per_split, scale_log2, k_static, v_static, L.d_status);
  L.count();
  if (e == cudaSuccess && S > 1) e = launch_combine(L, o_part, ml_part, (__nv_bfloat16*)o, total, S, HD);
  return e != cudaSuccess ? e : cudaGetLastError();
}
}  // namespace

// tuning override of the key-range split count of both tensor-core kernels (0 = automatic), see
// dllm_debug_attention_plan
int g_attn_force_splits = 0;
// (query, head-of-group) rows per KV head from which a bf16 shape takes the 128-row tcgen05 kernel
int g_attn_umma_min_rows = AT_ROWS + 1;
// 0: shapes with very few rows per KV head stay on the 64-row kernel (tuning / test switch)
int g_attn_few_rows = 1;
// 128-row tiles per CTA of the tcgen05 kernel: 0 = the plan's choice, 1 or 2 forced (tuning / test switch)
int g_attn_umma_row_tiles = 0;

// Key-range splits of the 64-row kernel, whole 64-key tiles per split: enough CTAs to cover the SMs when few
// rows are active (every split costs the merge a partial per row and head, so no more than that), and two CTAs
// per SM (what the shared memory of an SM holds) when a split would otherwise be left with more than eight key
// tiles to work through one after the other (a few queries against thousands of keys), but never fewer than
// three key tiles per split.  From sweeps on B200: 64 rows x 768 keys x 32 heads is fastest with 4 splits, 36
// rows x 4128 keys x 32 heads with 9 or 10, 56 rows x 2048 keys x 4 KV heads with 8 to 10 (11.8 us; 32: 36 us).
static void finish_plan(AttnPlan& p, int B, int a_seq, int n, int H, int S) {
  const int key_tiles = (n + AT_KEYS - 1) / AT_KEYS;
  if (S > key_tiles) S = key_tiles;
  if (S < 1) S = 1;
  const int tiles_per_split = (key_tiles + S - 1) / S;
  p.keys_per_split = tiles_per_split * AT_KEYS;
  p.S = (key_tiles + tiles_per_split - 1) / tiles_per_split;
  p.scratch_floats = p.S > 1 ? (size_t)p.S * B * a_seq * H * (128 + 2) : 0;
}

AttnPlan plan_attention(int B, int a_seq, int n, int H, int Hkv) {
  AttnPlan p;
  const int G = H / Hkv, sms = sm_count();
  // At most 32 rows per KV head against at least 16 key tiles: the kernel whose warps share the rows and take
  // different key tiles (6 ways of one 16-row warp, or 3 ways of two).  One wave of CTAs: as many splits as
  // keep the CTA count within the SM count (sweeps: 3 x 4128 x 32 heads 18.6 us with 4 splits against 25.0 on the
  // 64-row kernel, 25.6 with 5; 32 rows 23.7 against 26.2; four sequences 46 against 73), two tiles per way at least.
  if (a_seq * G <= 32 && (n + AT_KEYS - 1) / AT_KEYS >= 16 && g_attn_few_rows) {
    const int key_tiles = (n + AT_KEYS - 1) / AT_KEYS;
    p.few_rg = a_seq * G <= 16 ? 1 : 2;
    const int ways = p.few_rg == 1 ? 6 : 3;
    const long ctas = (long)Hkv * B;
    int S = (int)(sms / ctas);
    if (S > key_tiles / (2 * ways)) S = key_tiles / (2 * ways);
    if (g_attn_force_splits > 0) S = g_attn_force_splits;
    finish_plan(p, B, a_seq, n, H, S);
    return p;
  }
  const long tiles = (long)((a_seq * G + AT_ROWS - 1) / AT_ROWS) * Hkv * B;
  int S = 1;
  if (tiles < sms) {
    S = (int)((sms + tiles - 1) / tiles);
    const int key_tiles = (n + AT_KEYS - 1) / AT_KEYS;
    if ((key_tiles + S - 1) / S > 8) S = (int)((2L * sms + tiles - 1) / tiles);
    if (S > key_tiles / 3) S = key_tiles / 3 > 1 ? key_tiles / 3 : 1;  // three key tiles per split at least
  }
  if (g_attn_force_splits > 0) S = g_attn_force_splits;
  finish_plan(p, B, a_seq, n, H, S);
  return p;
}

// Which tensor-core kernel a bf16 shape takes, and its plan when the caller offers `scratch_floats` floats of
// scratch (SIZE_MAX: as much as the plan would like).  The 64-row mma.sync kernel never shrinks its plan: without
// room for the partials it runs one split.  The 128-row tcgen05 kernel lowers its split count to what fits.
AttnChoice choose_attention(int B, int a_seq, int n, int H, int Hkv, size_t scratch_floats) {
  AttnChoice c;
  c.umma = a_seq * (H / Hkv) >= g_attn_umma_min_rows;
  if (c.umma) {
    c.plan = plan_attention_umma(B, a_seq, n, H, Hkv, scratch_floats);
  } else {
    c.plan = plan_attention(B, a_seq, n, H, Hkv);
    if (c.plan.S > 1 && scratch_floats < c.plan.scratch_floats) finish_plan(c.plan, B, a_seq, n, H, 1);  // no room
    // (finish_plan keeps the kernel choice p.few_rg)
  }
  return c;
}

cudaError_t launch_attention(const Launch& L, int dtype, const void* q, const void* Kc, const void* Vc, void* o, int B,
                             int a_seq, int n, int H, int Hkv, int hd, float* scratch, size_t scratch_floats,
                             bool force_simt, int k_static, int v_static) {
  if (B <= 0 || a_seq <= 0) return cudaSuccess;
  if (hd > HD_MAX || (hd & 31) || H % Hkv) return cudaErrorInvalidValue;
  const bool tensor = dtype == 1 && !force_simt && (hd == 64 || hd == 128) && ((Hkv * hd) % 8 == 0);
  const AttnChoice ch = tensor ? choose_attention(B, a_seq, n, H, Hkv, scratch ? scratch_floats : 0) : AttnChoice{};
  if (tensor && ch.umma) {
    // many active rows per KV head: 128-row tiles on tcgen05
    int S = 1;
    cudaError_t e = launch_attention_umma(L, q, Kc, Vc, o, B, a_seq, n, H, Hkv, hd, scratch, scratch_floats, &S);
    if (e != cudaSuccess) return e;
    if (S > 1) {
      const size_t total = (size_t)B * a_seq * H;
      e = launch_combine(L, scratch, scratch + (size_t)S * total * hd, (__nv_bfloat16*)o, total, S, hd);
    }
    return e != cudaSuccess ? e : cudaGetLastError();
  }
  if (tensor) {
    const AttnPlan p = ch.plan;
    CUtensorMap tmK, tmV;
    if (!get_tensor_map_3d(Kc, (uint64_t)B, (uint64_t)n, (uint64_t)Hkv * hd, AT_KEYS, &tmK) ||
        !get_tensor_map_3d(Vc, (uint64_t)B, (uint64_t)n, (uint64_t)Hkv * hd, AT_KEYS, &tmV))
      return cudaErrorInvalidValue;
    const int S = p.S, kps = p.keys_per_split, ks = k_static, vs = v_static;
    if (p.few_rg == 1)
      return hd == 64 ? launch_few<64, 1, 6>(L, tmK, tmV, q, o, scratch, B, a_seq, n, H, Hkv, S, kps, ks, vs)
                      : launch_few<128, 1, 6>(L, tmK, tmV, q, o, scratch, B, a_seq, n, H, Hkv, S, kps, ks, vs);
    if (p.few_rg == 2)
      return hd == 64 ? launch_few<64, 2, 3>(L, tmK, tmV, q, o, scratch, B, a_seq, n, H, Hkv, S, kps, ks, vs)
                      : launch_few<128, 2, 3>(L, tmK, tmV, q, o, scratch, B, a_seq, n, H, Hkv, S, kps, ks, vs);
    return hd == 64 ? launch_mma<64>(L, tmK, tmV, q, o, scratch, B, a_seq, n, H, Hkv, S, kps, ks, vs)
                    : launch_mma<128>(L, tmK, tmV, q, o, scratch, B, a_seq, n, H, Hkv, S, kps, ks, vs);
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
  // the plan the kernels would take with unlimited scratch: the call must run exactly what dllm_attention runs
  // with a buffer of dllm_attention_scratch_bytes(), so a plan that does not fit the array is refused, not shrunk
  const AttnChoice want = choose_attention(B, a, n, H, Hkv, SIZE_MAX);
  if (want.plan.scratch_floats > NOALLOC_SCRATCH_FLOATS) {
    char msg[256];
    snprintf(msg, sizeof msg,
             "dllm_attention_noalloc: this shape splits the key range %d ways (%d-row tiles) and needs %zu bytes of "
             "scratch, the built-in array holds %zu; use dllm_attention with a caller-owned scratch buffer",
             want.plan.S, want.umma ? 128 : 64, want.plan.scratch_floats * sizeof(float), NOALLOC_SCRATCH_BYTES);
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
  // sum) that attn_combine_kernel reads is written by this call's attention kernel first.
  Launch L{(cudaStream_t)stream, kernel_status_word(), nullptr};
  e = launch_attention(L, DLLM_BF16, d_q, d_k, d_v, d_o, B, a, n, H, Hkv, hd, scratch, NOALLOC_SCRATCH_FLOATS, false);
  if (e != cudaSuccess) {
    set_last_error(cudaGetErrorString(e));
    return DLLM_CUDA_ERROR;
  }
  return DLLM_OK;
}

extern "C" dllm_status dllm_debug_attention_plan(int splits, int tcgen05_min_rows, int few_rows_kernel,
                                                 int tcgen05_row_tiles) {
  if (splits < 0 || tcgen05_min_rows < 0 || tcgen05_row_tiles < 0 || tcgen05_row_tiles > 2) {
    dllm::set_last_error("dllm_debug_attention_plan: arguments must not be negative, row tiles 0, 1 or 2");
    return DLLM_INVALID_ARG;
  }
  dllm::g_attn_force_splits = splits;
  if (tcgen05_min_rows > 0) dllm::g_attn_umma_min_rows = tcgen05_min_rows;
  dllm::g_attn_few_rows = few_rows_kernel != 0;
  dllm::g_attn_umma_row_tiles = tcgen05_row_tiles;
  return DLLM_OK;
}

DLLM_TIMELINE_HOOKS(attention)
DLLM_WAIT_LIMIT_HOOK(attention)
