// Flash-style attention tile on the tensor cores (bf16, mma.sync), written as a
// device function of one GROUP of 128 cooperating threads; a CTA runs one to
// four groups side by side on consecutive parts of its key range.
//
// One call = 64 "virtual rows" of one (sequence, KV head) x one range of keys.
// A virtual row is a (query, query-head-of-the-group) pair, so with grouped KV
// heads the G query heads that share a KV head are packed along the row
// dimension and every K/V tile is loaded once for all of them.  K and V tiles
// of 64 keys arrive by TMA (3-D map [B, n, dkv], 128-byte swizzle, keys beyond
// n zero-filled) into the group's own ring of one or two stages; each of the 4
// warps owns 16 rows and runs mma.sync m16n8k16 for S = Q K^T and O += P V with
// the online softmax in fp32 registers (exp2 with the scale folded in).  The
// result stays in registers (unnormalised output, row maximum, row sum); the
// kernel merges the groups of a CTA through shared memory, and attn_combine
// merges the key-range splits of different CTAs.
#pragma once
#include "common.cuh"
#include "tma.cuh"

namespace dllm {

// The 128 threads of a group synchronise on their own named barrier (1 + group index), so the groups of a CTA
// never wait for one another while they work through their keys.
__device__ __forceinline__ void at_sync(int bar_id) { asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory"); }
__device__ __forceinline__ bool at_sync_and(int bar_id, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.and.pred p, %2, 128, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"((uint32_t)pred), "r"(bar_id)
      : "memory");
  return r != 0;
}

constexpr int AT_ROWS = 64;   // virtual rows per CTA
constexpr int AT_KEYS = 64;   // keys per tile
constexpr int AT_MAX_GROUPS = 3;  // groups of 128 threads per CTA: 384 threads at up to 170 registers fill the file

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

// What a group holds for its 64 rows after its keys: thread (warp w, lane) has rows w * 16 + lane / 4 (index 0)
// and + 8 (index 1); o[i][2 * h2 + {0, 1}] are columns i * 8 + 2 * (lane % 4) + {0, 1} of row index h2.
// m is the row maximum in log2 units (scale folded in), l the sum of 2^(s - m) over the group's keys, o the
// unnormalised output.  A group without keys has m = -inf, l = 0, o = 0.
template <int HD>
struct AttnAcc {
  float o[HD / 8][4];
  float m[2], l[2];
};

// tid: 0..127 within the group.  q_s: shared-window address of the CTA's Q tile ([64 rows][HD] in swizzled
// panels, complete and visible before the call).  kv_s: shared-window address of the group's ring, `stages`
// (1 or 2) x (K tile, V tile), 1024-byte aligned.  full_bar: the group's `stages` mbarriers (count 1, fresh:
// phase 0).  Keys [key_lo, key_hi), key_lo a multiple of 64; an empty range returns the neutral element.
// stage_q(): called by every thread of every group once the group's first K/V requests are out; it brings the
// Q tile into shared memory (it may contain a CTA-wide barrier).  Returns false if a wait gave up.
template <int HD, typename StageQ>
__device__ __forceinline__ bool attn_group(int tid, int bar_id, uint32_t q_s, uint32_t kv_s, int stages,
                                           uint64_t* full_bar, volatile int* abort_flag, const CUtensorMap* tmK,
                                           const CUtensorMap* tmV, int kh, int b, int key_lo, int key_hi,
                                           float scale_log2, AttnAcc<HD>& acc, StageQ&& stage_q) {
  constexpr int PANELS = HD / 64;
  constexpr uint32_t TILE_BYTES = AT_KEYS * HD * 2;   // one K or V tile
  constexpr uint32_t STAGE_BYTES = 2 * TILE_BYTES;
  const int warp = tid >> 5, lane = tid & 31;
#pragma unroll
  for (int i = 0; i < HD / 8; ++i) acc.o[i][0] = acc.o[i][1] = acc.o[i][2] = acc.o[i][3] = 0.f;
  acc.m[0] = acc.m[1] = -INFINITY;
  acc.l[0] = acc.l[1] = 0.f;
  const int n_tiles = key_hi > key_lo ? (key_hi - key_lo + AT_KEYS - 1) / AT_KEYS : 0;

  auto issue = [&](int t) {
    const int st = t % stages;
    const uint32_t fb = smem_u32(&full_bar[st]);
    mbar_expect_tx(fb, STAGE_BYTES);
    const uint32_t dst = kv_s + st * STAGE_BYTES;
    const int key0 = key_lo + t * AT_KEYS;
#pragma unroll
    for (int p = 0; p < PANELS; ++p) {
      tma_load_3d(dst + p * (AT_KEYS * 128), tmK, fb, kh * HD + p * 64, key0, b);
      tma_load_3d(dst + TILE_BYTES + p * (AT_KEYS * 128), tmV, fb, kh * HD + p * 64, key0, b);
    }
  };
  if (tid == 0 && n_tiles > 0) {
    issue(0);
    if (n_tiles > 1 && stages > 1) issue(1);
  }
  stage_q();
  bool ok = true;
  for (int t = 0; t < n_tiles; ++t) {
    const int st = t % stages;
    ok = mbar_wait(smem_u32(&full_bar[st]), (uint32_t)(t / stages) & 1u, abort_flag);
    ok = at_sync_and(bar_id, ok);             // uniform over the group: nobody is left behind at a barrier
    if (!ok) break;
    if (tid == 0) timeline_mark(2 + (t < 5 ? t : 5));  // K/V tile t has landed
    const uint32_t k_s = kv_s + st * STAGE_BYTES, v_s = k_s + TILE_BYTES;
    // ---- S = Q K^T for 16 rows x 64 keys (the Q fragments are re-read per k-step: they are used once per tile
    // and a group mostly sees one or two tiles, so holding them would only cost registers)
    float sacc[AT_KEYS / 8][4];
#pragma unroll
    for (int i = 0; i < AT_KEYS / 8; ++i) sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < HD / 16; ++ks) {
      uint32_t qf[4];
      {
        const int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
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
      const float m_new = fmaxf(acc.m[h2], mx[h2]);      // finite: every tile has a valid key
      corr[h2] = exp2f(acc.m[h2] - m_new);
      acc.m[h2] = m_new;
      acc.l[h2] *= corr[h2];
    }
#pragma unroll
    for (int nb = 0; nb < AT_KEYS / 8; ++nb) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const float p = exp2f(sacc[nb][c] - acc.m[c >> 1]);
        sacc[nb][c] = p;
        acc.l[c >> 1] += p;
      }
    }
    if (t > 0) {
#pragma unroll
      for (int i = 0; i < HD / 8; ++i) {
        acc.o[i][0] *= corr[0];
        acc.o[i][1] *= corr[0];
        acc.o[i][2] *= corr[1];
        acc.o[i][3] *= corr[1];
      }
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
    if (t + stages < n_tiles) {
      at_sync(bar_id);                         // every warp of the group is done with stage st
      if (tid == 0) issue(t + stages);
    }
  }
  if (!ok) return false;
  // the row sums are spread over the four lanes of a row
#pragma unroll
  for (int h2 = 0; h2 < 2; ++h2) {
    acc.l[h2] += __shfl_xor_sync(0xffffffffu, acc.l[h2], 1);
    acc.l[h2] += __shfl_xor_sync(0xffffffffu, acc.l[h2], 2);
  }
  return true;
}

}  // namespace dllm
