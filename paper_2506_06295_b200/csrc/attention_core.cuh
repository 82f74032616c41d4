// Flash-style attention tile on the tensor cores (bf16, mma.sync), written as a
// device function of 128 cooperating threads so that the stand-alone attention
// kernel and the persistent layer kernel run the same code.
//
// One call = 64 "virtual rows" of one (sequence, KV head) x one split of the key
// range.  A virtual row is a (query, query-head-of-the-group) pair, so with
// grouped KV heads the G query heads that share a KV head are packed along the
// row dimension and every K/V tile is loaded once for all of them.  K and V
// tiles of 64 keys arrive by TMA (3-D map [B, n, dkv], 128-byte swizzle, keys
// beyond n zero-filled) into a two-stage ring; each of the 4 warps owns 16 rows
// and runs mma.sync m16n8k16 for S = Q K^T and O += P V with the online softmax
// in fp32 registers (exp2 with the scale folded in).  Splits write unnormalised
// partial outputs plus (max, sum); attn_combine merges them.
#pragma once
#include "common.cuh"
#include "tma.cuh"

namespace dllm {

// The 128 threads of a tile synchronise on named barrier 1, so the function can
// run inside a larger block whose other warps do something else.
__device__ __forceinline__ void at_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ bool at_sync_and(bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.and.pred p, 1, 128, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"((uint32_t)pred)
      : "memory");
  return r != 0;
}

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
// 2^x on the special-function unit (ex2.approx: relative error about 2^-22, far below the bf16 rounding of P;
// 2^-inf = 0)
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Online-softmax update of one warp's 16 x 64 score fragment (rows lane / 4 and lane / 4 + 8; raw scores in,
// probabilities out): new running maxima m (in log2 units of the scaled scores), the factors `corr` by which the
// sums and outputs so far shrink, and the row sums l advanced by this tile's (per-lane partial) sums.  The scale
// is folded into the exponent's multiply-add; keys at or past key_hi count for nothing (only a sequence's last
// tile has any: a warp-uniform test).  key_base: the first of this lane's keys.
__device__ __forceinline__ void softmax_tile(float (&sacc)[8][4], int key_base, int key_hi, int lane, float scale_log2,
                                             float (&m)[2], float (&l)[2], float (&corr)[2]) {
  if (key_base - 2 * (lane & 3) + 64 > key_hi) {
#pragma unroll
    for (int nb = 0; nb < 8; ++nb)
#pragma unroll
      for (int c = 0; c < 4; ++c)
        if (key_base + nb * 8 + (c & 1) >= key_hi) sacc[nb][c] = -INFINITY;
  }
  float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
  for (int nb = 0; nb < 8; ++nb)
#pragma unroll
    for (int c = 0; c < 4; ++c) mx[c >> 1] = fmaxf(mx[c >> 1], sacc[nb][c]);
#pragma unroll
  for (int h2 = 0; h2 < 2; ++h2) {
    mx[h2] = fmaxf(mx[h2], __shfl_xor_sync(0xffffffffu, mx[h2], 1));
    mx[h2] = fmaxf(mx[h2], __shfl_xor_sync(0xffffffffu, mx[h2], 2));
    const float m_new = fmaxf(m[h2], mx[h2] * scale_log2);  // finite: every tile has a valid key; scale_log2 > 0
    corr[h2] = fast_exp2(m[h2] - m_new);                      // first tile: 2^-inf = 0
    m[h2] = m_new;
    l[h2] *= corr[h2];
  }
#pragma unroll
  for (int nb = 0; nb < 8; ++nb)
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const float p = fast_exp2(fmaf(sacc[nb][c], scale_log2, -m[c >> 1]));
      sacc[nb][c] = p;
      l[c >> 1] += p;
    }
}

// Byte offset of the 16-byte chunk `dc` (8 bf16) of row `row` in a tile stored
// as panels of 64 columns: panel = [rows][128 bytes], chunk index XOR (row % 8).
template <int ROWS>
__device__ __forceinline__ uint32_t tile_off(int row, int dc) {
  return (uint32_t)((dc >> 3) * (ROWS * 128) + row * 128 + (((dc & 7) ^ (row & 7)) << 4));
}

template <int HD>
struct AttnSmem {
  static constexpr int BYTES = AT_ROWS * HD * 2 + 2 * 2 * AT_KEYS * HD * 2;  // Q tile + two (K, V) stages
};

// tid: 0..127.  smem_gen / smem_sh: generic pointer and shared-window address of
// the same 1024-byte aligned region of AttnSmem<HD>::BYTES bytes.  full_bar: two
// initialised mbarriers (count 1).  kv_iter: tiles this ring has carried so far
// (stage and phase parity continue across calls); advanced by the tiles of this
// call.  (bx, by, bz) play the role of the block index of a grid
// (row tiles, KV heads, B * S).  Returns false if a wait gave up.
// The function itself waits for the launch before this one (griddepcontrol.wait) and releases the dependents.
// k_static / v_static: the first so many keys of every sequence hold K / V rows that no launch since the one
// BEFORE the previous launch has written (0: none); tiles made of such rows only are requested ahead of the wait,
// while the previous launch (which writes Q and the newest K rows) still runs.
template <int HD>
__device__ __forceinline__ bool attn_tile(int tid, uint8_t* smem_gen, uint32_t smem_sh, uint64_t* full_bar,
                                          uint32_t& kv_iter, volatile int* abort_flag, const CUtensorMap* tmK,
                                          const CUtensorMap* tmV, const __nv_bfloat16* __restrict__ q,
                                          __nv_bfloat16* __restrict__ o, float* __restrict__ o_part,
                                          float* __restrict__ ml_part, int a_seq, int n, int H, int Hkv, int S,
                                          int keys_per_split, float scale_log2, int B, int bx, int by, int bz,
                                          const CUtensorMap* tmQ, int k_static, int v_static) {

  constexpr int PANELS = HD / 64;
  constexpr uint32_t TILE_BYTES = AT_KEYS * HD * 2;   // one K or V tile
  constexpr uint32_t STAGE_BYTES = 2 * TILE_BYTES;
  const uint32_t base = smem_sh;
  const uint32_t q_s = base;                         // [64 rows][HD] in panels
  const uint32_t kv_s = base + AT_ROWS * HD * 2;     // 2 stages x (K tile, V tile)
  uint8_t* q_gen = smem_gen;

  const int warp = tid >> 5, lane = tid & 31;
  const int G = H / Hkv;
  const int kh = by;
  const int b = bz / S, split = bz - b * S;
  const int row0 = bx * AT_ROWS;
  const int n_rows = a_seq * G;
  const int key_lo = split * keys_per_split;
  const int key_hi = min(n, key_lo + keys_per_split);
  const int n_tiles = (key_hi - key_lo + AT_KEYS - 1) / AT_KEYS;   // >= 1 by construction
  const int dq = H * HD;

  const uint32_t it0 = kv_iter;
  kv_iter += (uint32_t)n_tiles;
  at_sync();  // the previous tile's readers are done with the Q and K/V regions
  // tmQ (one query head per KV head, so a row tile is AT_ROWS consecutive rows of q): the Q tile arrives by TMA
  // together with the first K/V tile, on that tile's barrier; rows past the sequence's end belong to no live row
  const bool q_tma = tmQ != nullptr;
  // what: 1 = the K tile, 2 = the V tile, 4 = arm the stage's barrier with everything that will arrive on it
  // (K, V and, for the first tile, the Q tile by TMA), 8 = the Q tile
  auto issue = [&](int t, int what) {
    const int st = (int)((it0 + (uint32_t)t) & 1u);
    const uint32_t fb = smem_u32(&full_bar[st]);
    if (what & 4) mbar_expect_tx(fb, STAGE_BYTES + ((q_tma && t == 0) ? AT_ROWS * HD * 2 : 0));
    if ((what & 8) && q_tma && t == 0) {
#pragma unroll
      for (int p = 0; p < PANELS; ++p) tma_load_2d(q_s + p * (AT_ROWS * 128), tmQ, fb, kh * HD + p * 64, b * a_seq + row0);
    }
    const uint32_t dst = kv_s + st * STAGE_BYTES;
    const int key0 = key_lo + t * AT_KEYS;
#pragma unroll
    for (int p = 0; p < PANELS; ++p) {
      if (what & 1) tma_load_3d(dst + p * (AT_KEYS * 128), tmK, fb, kh * HD + p * 64, key0, b);
      if (what & 2) tma_load_3d(dst + TILE_BYTES + p * (AT_KEYS * 128), tmV, fb, kh * HD + p * 64, key0, b);
    }
  };
  int early[2] = {0, 0};  // what of the first two tiles was requested ahead of the dependency wait
  if (tid == 0) {
    for (int t = 0; t < 2 && t < n_tiles; ++t) {
      const int hi = min(key_lo + (t + 1) * AT_KEYS, n);  // one past the tile's last existing key
      early[t] = (hi <= k_static ? 1 : 0) | (hi <= v_static ? 2 : 0);
      if (early[t]) issue(t, early[t] | 4);
    }
  }
  pdl_wait();  // Q and the newest K rows come from the launch before this one
  pdl_trigger();
  if (tid == 0) {
    for (int t = 0; t < 2 && t < n_tiles; ++t) issue(t, (3 & ~early[t]) | (early[t] ? 0 : 4) | 8);
  }
  // Q tile: plain 16-byte loads into the swizzled layout (rows of other heads /
  // past the end are zero)
  if (q_tma) {
    mbar_wait(smem_u32(&full_bar[(int)(it0 & 1u)]), (it0 >> 1) & 1u, abort_flag);  // the loop checks the outcome again
  } else {
    constexpr int PER = AT_ROWS * (HD / 8) / 128;  // 16-byte chunks per thread: all loads first, then the stores
    uint4 qv[PER];
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      const int e = tid + i * 128;
      const int r = e / (HD / 8), dc = e - r * (HD / 8);
      const int vr = row0 + r;
      qv[i] = make_uint4(0, 0, 0, 0);
      if (vr < n_rows) {
        const int qi = vr / G, g = vr - qi * G;
        qv[i] = __ldcg(reinterpret_cast<const uint4*>(q + ((size_t)b * a_seq + qi) * dq + (kh * G + g) * HD + dc * 8));
      }
    }
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      const int e = tid + i * 128;
      const int r = e / (HD / 8), dc = e - r * (HD / 8);
      *reinterpret_cast<uint4*>(q_gen + tile_off<AT_ROWS>(r, dc)) = qv[i];
    }
  }
  at_sync();
  if (tid == 0) timeline_mark(1);  // Q staged
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
    const int st = (int)((it0 + (uint32_t)t) & 1u);
    ok = mbar_wait(smem_u32(&full_bar[st]), ((it0 + (uint32_t)t) >> 1) & 1u, abort_flag);
    ok = at_sync_and(ok);                     // uniform over the 128 threads: nobody is left behind at a barrier
    if (!ok) break;
    if (tid == 0) timeline_mark(2 + (t < 5 ? t : 5));  // K/V tile t has landed
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
    float corr[2];
    softmax_tile(sacc, key_lo + t * AT_KEYS + 2 * (lane & 3), key_hi, lane, scale_log2, m_run, l_run, corr);
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
    at_sync();                               // every warp is done with stage st
    if (tid == 0 && t + 2 < n_tiles) issue(t + 2, 1 | 2 | 4);
  }
  if (!ok) {
    drain_delay();
    return false;
  }
  if (tid == 0) timeline_mark(8);  // all tiles done
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
      const size_t total = (size_t)B * a_seq * H;           // (row, head) pairs
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
  return true;
}

// ---------------------------------------------------------------------------------------------------------
// The same arithmetic for ONE warp and ONE 64-key tile, used by the kernel for very few query rows, where the
// warps of a CTA share their 16 rows and take different key tiles (the chain load -> QK^T -> softmax -> PV of
// a tile takes a warp about as long whether its row tile is full or nearly empty, so with 3 or 30 rows it pays
// to work on several tiles at once).  q_s: the CTA's Q tile (swizzled panels of AT_ROWS rows); rg: which 16
// rows of it; k_s / v_s: the tile; keys [key0, key_hi) of it count.  acc carries (o, m, l) across the warp's
// tiles; l holds per-lane partial sums until attn_warp_finish.
template <int HD>
struct AttnAcc {
  float o[HD / 8][4];
  float m[2], l[2];
};
template <int HD>
__device__ __forceinline__ void attn_acc_clear(AttnAcc<HD>& acc) {
#pragma unroll
  for (int i = 0; i < HD / 8; ++i) acc.o[i][0] = acc.o[i][1] = acc.o[i][2] = acc.o[i][3] = 0.f;
  acc.m[0] = acc.m[1] = -INFINITY;
  acc.l[0] = acc.l[1] = 0.f;
}
template <int HD>
__device__ __forceinline__ void attn_warp_tile(int lane, int rg, uint32_t q_s, uint32_t k_s, uint32_t v_s, int key0,
                                               int key_hi, float scale_log2, AttnAcc<HD>& acc) {
  // ---- S = Q K^T for 16 rows x 64 keys
  float sacc[AT_KEYS / 8][4];
#pragma unroll
  for (int i = 0; i < AT_KEYS / 8; ++i) sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f;
#pragma unroll
  for (int ks = 0; ks < HD / 16; ++ks) {
    uint32_t qf[4];
    {
      const int row = rg * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
      const int dc = ks * 2 + (lane >> 4);
      ldsm_x4(q_s + tile_off<AT_ROWS>(row, dc), qf[0], qf[1], qf[2], qf[3]);
    }
#pragma unroll
    for (int jp = 0; jp < AT_KEYS / 16; ++jp) {
      const int key = jp * 16 + (lane & 7) + (lane >> 4) * 8;
      const int dc = ks * 2 + ((lane >> 3) & 1);
      uint32_t r0, r1, r2, r3;
      ldsm_x4(k_s + tile_off<AT_KEYS>(key, dc), r0, r1, r2, r3);
      mma_bf16_16816(sacc[2 * jp], qf, r0, r1);
      mma_bf16_16816(sacc[2 * jp + 1], qf, r2, r3);
    }
  }
  // ---- online softmax (rows lane/4 and lane/4 + 8)
  float corr[2];
  softmax_tile(sacc, key0 + 2 * (lane & 3), key_hi, lane, scale_log2, acc.m, acc.l, corr);
#pragma unroll
  for (int i = 0; i < HD / 8; ++i) {
    acc.o[i][0] *= corr[0];
    acc.o[i][1] *= corr[0];
    acc.o[i][2] *= corr[1];
    acc.o[i][3] *= corr[1];
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
      mma_bf16_16816(acc.o[2 * dp], pf, r0, r1);
      mma_bf16_16816(acc.o[2 * dp + 1], pf, r2, r3);
    }
  }
}
// the row sums are spread over the four lanes of a row
template <int HD>
__device__ __forceinline__ void attn_warp_finish(AttnAcc<HD>& acc) {
#pragma unroll
  for (int h2 = 0; h2 < 2; ++h2) {
    acc.l[h2] += __shfl_xor_sync(0xffffffffu, acc.l[h2], 1);
    acc.l[h2] += __shfl_xor_sync(0xffffffffu, acc.l[h2], 2);
  }
}

}  // namespace dllm
