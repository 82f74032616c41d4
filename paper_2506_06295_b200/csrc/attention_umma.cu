// Flash-style attention on the 5th-generation tensor cores (tcgen05) for the
// steps with many active rows (response refresh, full steps, batched serving):
// non-causal attention of the active query rows over ALL n cached keys of
// their sequence (Sec. A.7), grouped KV heads packed along the row dimension.
//
// One CTA = TWO tiles of 128 "virtual rows" ((query, head-of-group) pairs) of
// one (sequence, KV head) x one split of the key range, key tiles of 64, ten
// warps with fixed roles:
//   warp 9           TMA: K/V tiles into a six-stage ring (all that shared memory holds)
//   warp 8           issues every tcgen05.mma of the CTA
//   warps 0-3, 4-7   the softmax group of row tile 0 resp. 1 (one row per thread)
// Per key tile t and row tile i:
//   S_i = Q_i K^T     tcgen05.mma, M = 128 rows, N = 64 keys, contraction HD; Q_i is
//                     the A operand in tensor memory (written there once by its
//                     group), K in shared memory (K-major, 128-byte swizzle)
//   softmax           TMEM lane = row, so every thread of group i owns one row: it
//                     loads its 64 scores with tcgen05.ld, takes max / exp2 / sum
//                     locally (no shuffles) and writes P_i as bf16 pairs over the
//                     first 32 score columns: the A operand of the next product
//   O_i += P_i V      tcgen05.mma, M = 128 rows, N = HD, contraction 64 keys; V is
//                     used as stored ([key][hd], "MN-major" B operand); O_i
//                     accumulates in TMEM and is rescaled (tcgen05.ld / st) only
//                     when a row's maximum has grown by more than 2^8 since its
//                     reference was set
// The MMA warp issues O_i += P_i V of tile t and, right behind it, S_i of tile
// t+1, alternating between the row tiles: while one group is in its softmax the
// tensor pipe works for the other, and both row tiles read every K/V tile that
// arrives once.  A CTA with ONE live row tile (at most 128 rows per KV head, the
// odd last tile, or a plan of one-tile CTAs) gives both groups that tile's rows:
// group 0 takes the even key tiles of the CTA's range and group 1 the odd ones,
// each with its own scores, running maximum, sum and output accumulator, and the
// two halves are merged through shared memory at the end (group 1's first).
// Key-range splits write unnormalised partials plus (max, sum) exactly like the
// mma.sync kernel, and the same merge kernel finishes them.  Every mbarrier wait
// is bounded.
#include "attention_core.cuh"
#include "internal.h"
#include "tma.cuh"
#include "umma.cuh"

namespace dllm {

namespace {

constexpr int UA_ROWS = 128;   // virtual rows per row tile (UMMA M); a CTA works on two row tiles
constexpr int UA_TILES = 2;
constexpr int UA_KEYS = 64;    // keys per tile
constexpr int UA_STAGES = 6;   // K/V ring
constexpr int UA_THREADS = 320;  // two softmax groups of 128, one MMA warp, one TMA warp
// key tiles from which a CTA with one live row tile shares them between its two softmax groups: the exchange and
// merge of the two halves at the end cost about as much as the overlap saves on eight tiles (B200: 24 tiles per CTA
// 135 -> 114 us at 16 x 128 rows x 1536 keys; 3-4 tiles per CTA 13.8 -> 15.0 us at 128 rows x 768 keys)
constexpr int UA_KPAR_MIN_TILES = 8;

// MN-major operand ([k][mn] rows of 64 mn-elements = 128 bytes, 128-byte swizzle,
// panels of 64 mn-elements): lbo = bytes between panels along MN, sbo = bytes
// between groups of 8 k-rows.
__device__ __forceinline__ uint64_t make_smem_desc_mn(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
        "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}


template <int HD>
struct UaSmem {
  static constexpr uint32_t KV_TILE = UA_KEYS * HD * 2;          // one K or V tile
  static constexpr uint32_t STAGE = 2 * KV_TILE;                 // K then V
  static constexpr uint32_t TOTAL = UA_STAGES * STAGE + 1024;    // shared memory holds nothing but the K/V ring
  // Tensor memory, 128 lanes = the rows of a tile: Q_i as bf16 pairs (HD / 2 columns each), the scores S_i (64
  // fp32 columns each; the probabilities P_i overwrite the first 32 of them as bf16 pairs), the outputs O_i.
  static constexpr uint32_t Q_COL = 0, S_COL = UA_TILES * (HD / 2), O_COL = S_COL + UA_TILES * UA_KEYS;
  static constexpr uint32_t TMEM_COLS = 512;
  static_assert(O_COL + UA_TILES * HD <= TMEM_COLS, "tensor memory holds 512 columns");
};

template <int HD>
__global__ void __launch_bounds__(UA_THREADS, 1)
    attn_umma_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                     const __nv_bfloat16* __restrict__ q,
                     __nv_bfloat16* __restrict__ o, float* __restrict__ o_part, float* __restrict__ ml_part, int a_seq,
                     int n, int H, int Hkv, int S, int keys_per_split, int row_tiles_per_cta, float scale_log2,
                     int* __restrict__ status) {
  using SM = UaSmem<HD>;
  constexpr int PANELS = HD / 64;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t kv_full[UA_STAGES], kv_empty[UA_STAGES];
  __shared__ __align__(8) uint64_t s_full[UA_TILES], p_full[UA_TILES], o_full[UA_TILES], q_bar;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t kv_s = base;
  volatile int* abortp = &abort_flag;

  const int G = H / Hkv;
  const int kh = blockIdx.y;
  const int b = blockIdx.z / S, split = blockIdx.z - b * S;
  // row_tiles_per_cta = 1: every CTA takes one 128-row tile only (its second softmax group idles); the plan
  // asks for that when two-tile CTAs would be too few to fill the GPU
  const int row0 = blockIdx.x * (row_tiles_per_cta * UA_ROWS);
  const int n_rows = a_seq * G;
  const int live = (row_tiles_per_cta > 1 && row0 + UA_ROWS < n_rows) ? 2 : 1;  // row tiles of this CTA that hold rows
  const int key_lo = split * keys_per_split;
  const int key_hi = min(n, key_lo + keys_per_split);
  const int n_tiles = (key_hi - key_lo + UA_KEYS - 1) / UA_KEYS;  // >= 1 by construction of the plan
  const int dq = H * HD;
  // one live row tile and enough key tiles: both softmax groups work on that tile's rows, group i on the key
  // tiles t with t % 2 == i
  const bool kpar = live == 1 && n_tiles >= UA_KPAR_MIN_TILES;

  if (tid == 0) {
    abort_flag = 0;
    for (int i = 0; i < UA_STAGES; ++i) {
      mbar_init(smem_u32(&kv_full[i]), 1);
      mbar_init(smem_u32(&kv_empty[i]), 1);
    }
    for (int i = 0; i < UA_TILES; ++i) {
      mbar_init(smem_u32(&s_full[i]), 1);
      mbar_init(smem_u32(&p_full[i]), UA_ROWS / 32);  // one arrival per warp of the tile's softmax group
      mbar_init(smem_u32(&o_full[i]), 1);
    }
    mbar_init(smem_u32(&q_bar), UA_TILES * UA_ROWS / 32);  // one arrival per softmax warp
    mbar_fence_init();
    prefetch_tensormap(&tmK);
    prefetch_tensormap(&tmV);
  }
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                 "r"(SM::TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = tmem_slot;
  pdl_wait();  // Q, K and V come from the preceding kernels
  pdl_trigger();
  bool ok = true;

  if (warp == 9) {
    // ---------------- TMA producer: the K/V tiles of the key range ----------------
    if (lane == 0) {
      for (int t = 0; t < n_tiles; ++t) {
        const int st = t % UA_STAGES;
        if (t >= UA_STAGES && !mbar_wait(smem_u32(&kv_empty[st]), (uint32_t)(t / UA_STAGES - 1) & 1u, abortp)) {
          ok = false;
          break;
        }
        const uint32_t fb = smem_u32(&kv_full[st]);
        mbar_expect_tx(fb, SM::STAGE);
        const uint32_t dst = kv_s + st * SM::STAGE;
        const int key0 = key_lo + t * UA_KEYS;
#pragma unroll
        for (int p = 0; p < PANELS; ++p) {
          tma_load_3d(dst + p * (UA_KEYS * 128), &tmK, fb, kh * HD + p * 64, key0, b);
          tma_load_3d(dst + SM::KV_TILE + p * (UA_KEYS * 128), &tmV, fb, kh * HD + p * 64, key0, b);
        }
      }
    }
  } else if (warp == 8) {
    // ---------------- MMA issuer ----------------
    // Per key tile t and row tile i:  S_i(t) = Q_i K(t)^T  ->  [softmax group i]  ->  O_i += P_i(t) V(t), and right
    // behind it S_i(t+1), so that the tensor pipe works on one row tile while the other is in its softmax.  Q_i
    // and P_i are A operands in tensor memory (P_i in the columns its scores came from), so shared memory is
    // read for K and V only.  A commit covers every MMA issued before it, so when s_full[i] flips for tile t+1
    // the product O_i += P_i V of tile t has completed too: the group may then rescale O_i.
    if (lane == 0) {
      constexpr uint32_t idesc_s = make_idesc(UA_ROWS, UA_KEYS);
      constexpr uint32_t idesc_o = make_idesc(UA_ROWS, HD) | (1u << 16);  // B operand (V) is MN-major
      auto issue_s = [&](int i, int st) {
        const uint32_t k_s = kv_s + st * SM::STAGE;
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
          const uint32_t koff = (ks >> 2) * (UA_KEYS * 128) + (ks & 3) * 32;  // panel, then 32 bytes per k-step
          // A = 16 dimensions of Q_i from tensor memory (8 columns of bf16 pairs per k-step)
          umma_bf16_ta(tmem + SM::S_COL + (uint32_t)(i * UA_KEYS), tmem + SM::Q_COL + (uint32_t)(i * (HD / 2) + ks * 8),
                       make_smem_desc(k_s + koff), idesc_s, ks > 0 ? 1u : 0u);
        }
        umma_commit(smem_u32(&s_full[i]));
      };
      ok = mbar_wait(smem_u32(&q_bar), 0u, abortp) && mbar_wait(smem_u32(&kv_full[0]), 0u, abortp);
      if (ok && kpar) {
        // group i owns key tiles i, i + 2, ...: S_0(0), S_1(1); then per tile t (group i = t % 2):
        // O_i += P_i(t) V(t) and right behind it S_i(t + 2)
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        issue_s(0, 0);
        ok = mbar_wait(smem_u32(&kv_full[1]), 0u, abortp);
        if (ok) {
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          issue_s(1, 1);
        }
        for (int t = 0; t < n_tiles && ok; ++t) {
          const int i = t & 1, u = t >> 1;
          const int st = t % UA_STAGES;
          const uint32_t v_s = kv_s + st * SM::STAGE + SM::KV_TILE;
          ok = mbar_wait(smem_u32(&p_full[i]), (uint32_t)u & 1u, abortp);
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
          for (int ks = 0; ks < UA_KEYS / 16; ++ks)
            umma_bf16_ta(tmem + SM::O_COL + (uint32_t)(i * HD), tmem + SM::S_COL + (uint32_t)(i * UA_KEYS + ks * 8),
                         make_smem_desc_mn(v_s + ks * (16 * 128), UA_KEYS * 128, 1024), idesc_o,
                         (u > 0 || ks > 0) ? 1u : 0u);
          if (t + 2 < n_tiles) {
            const int st2 = (t + 2) % UA_STAGES;
            ok = mbar_wait(smem_u32(&kv_full[st2]), (uint32_t)((t + 2) / UA_STAGES) & 1u, abortp);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            issue_s(i, st2);
          } else {
            umma_commit(smem_u32(&o_full[i]));  // the group's last tile: O_i is final when this fires
          }
          umma_commit(smem_u32(&kv_empty[st]));  // only group i reads tile t
        }
      } else if (ok) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        for (int i = 0; i < live; ++i) issue_s(i, 0);
      }
      for (int t = 0; t < n_tiles && ok && !kpar; ++t) {
        const int st = t % UA_STAGES, st_next = (t + 1) % UA_STAGES;
        const uint32_t v_s = kv_s + st * SM::STAGE + SM::KV_TILE;
        bool next_ready = t + 1 >= n_tiles;
        for (int i = 0; i < live && ok; ++i) {
          ok = mbar_wait(smem_u32(&p_full[i]), (uint32_t)t & 1u, abortp);
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
          for (int ks = 0; ks < UA_KEYS / 16; ++ks)   // A = 16 keys of P_i from tensor memory; V: 16 key rows of 128 bytes
            umma_bf16_ta(tmem + SM::O_COL + (uint32_t)(i * HD), tmem + SM::S_COL + (uint32_t)(i * UA_KEYS + ks * 8),
                         make_smem_desc_mn(v_s + ks * (16 * 128), UA_KEYS * 128, 1024), idesc_o,
                         (t > 0 || ks > 0) ? 1u : 0u);
          if (t + 1 < n_tiles) {
            if (!next_ready) {
              ok = mbar_wait(smem_u32(&kv_full[st_next]), (uint32_t)((t + 1) / UA_STAGES) & 1u, abortp);
              if (!ok) break;
              asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
              next_ready = true;
            }
            issue_s(i, st_next);
          } else {
            umma_commit(smem_u32(&o_full[i]));  // last tile: O_i is final when this fires
          }
        }
        if (ok) umma_commit(smem_u32(&kv_empty[st]));  // the stage may be refilled once these MMAs have read it
      }
    }
  } else {
    // ---------------- softmax groups: warps 0-3 own row tile 0, warps 4-7 row tile 1 ----------------
    const int i = warp >> 2;                                  // row tile
    const int row = (warp & 3) * 32 + lane;                   // row of the tile = TMEM lane
    const uint32_t row_lane = ((uint32_t)((warp & 3) * 32)) << 16;
    const uint32_t s_col = SM::S_COL + (uint32_t)(i * UA_KEYS), o_col = SM::O_COL + (uint32_t)(i * HD);
    const int gtid = tid & 127;
    {
      // Q_i: every thread fetches its own row (HD bf16 = HD / 8 16-byte words, zero past the last row) and
      // writes it to its TMEM lane as bf16 pairs; all loads of a thread are in flight before the first use
      const int vr = row0 + (kpar ? 0 : i * UA_ROWS) + row;
      uint4 qv[HD / 8];
#pragma unroll
      for (int w = 0; w < HD / 8; ++w) qv[w] = make_uint4(0, 0, 0, 0);
      if (vr < n_rows && (i < live || kpar)) {
        const int qi = vr / G, g = vr - qi * G;
        const uint4* src = reinterpret_cast<const uint4*>(q + ((size_t)b * a_seq + qi) * dq + (kh * G + g) * HD);
#pragma unroll
        for (int w = 0; w < HD / 8; ++w) qv[w] = __ldcg(src + w);
      }
#pragma unroll
      for (int c = 0; c < HD / 2; c += 32) {
        uint32_t r[32];
#pragma unroll
        for (int w = 0; w < 8; ++w) {
          r[4 * w] = qv[c / 4 + w].x;
          r[4 * w + 1] = qv[c / 4 + w].y;
          r[4 * w + 2] = qv[c / 4 + w].z;
          r[4 * w + 3] = qv[c / 4 + w].w;
        }
        tmem_st32(tmem + row_lane + SM::Q_COL + (uint32_t)(i * (HD / 2) + c), r);  // waits for the store
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&q_bar));
    }
    if (gtid == 0 && i == 0) timeline_mark(1);  // Q in tensor memory

    constexpr float RESCALE_STEP = 8.f;  // log2 units a row's maximum may exceed its reference before O is rescaled
    // m_ref: the maximum the exponentials of this row refer to; it follows the true running maximum lazily (O in
    // TMEM is only rescaled when the maximum has grown by more than RESCALE_STEP, which keeps every exponential
    // below 2^8)
    float m_ref = -INFINITY, l_run = 0.f;
    if (i < live || kpar) {
      // u counts this group's tiles; with kpar they are the key tiles i, i + 2, ...
      const int t_step = kpar ? 2 : 1;
      for (int t = kpar ? i : 0, u = 0; t < n_tiles; t += t_step, ++u) {
        ok = mbar_wait(smem_u32(&s_full[i]), (uint32_t)u & 1u, abortp);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (gtid == 0 && i == 0) timeline_mark(2 + (u < 5 ? u : 5));  // scores of this group's tile u complete
        // ---- this thread's row of scores (raw: the scale is folded into the exponent's multiply-add)
        const int valid = key_hi - (key_lo + t * UA_KEYS);  // >= 1
        float sv[UA_KEYS];
        float mx;
        {
          uint32_t r0[32], r1[32];  // both loads in flight, one wait
          tmem_ld32(tmem + row_lane + s_col, r0);
          tmem_ld32(tmem + row_lane + s_col + 32u, r1);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            sv[j] = __uint_as_float(r0[j]);
            sv[32 + j] = __uint_as_float(r1[j]);
          }
          if (valid < UA_KEYS) {  // the ragged last tile of the sequence: keys past the end count for nothing
#pragma unroll
            for (int j = 0; j < UA_KEYS; ++j)
              if (j >= valid) sv[j] = -INFINITY;
          }
          float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};  // four chains instead of one of 64 steps
#pragma unroll
          for (int j = 0; j < UA_KEYS; ++j) mx4[j & 3] = fmaxf(mx4[j & 3], sv[j]);
          mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * scale_log2;  // scale_log2 > 0
        }
        // ---- lazy rescale of O (warp-uniform branch: the TMEM accesses are warp-collective)
        const bool grow = mx > m_ref + RESCALE_STEP;
        if (__any_sync(0xffffffffu, grow)) {
          const float corr = grow ? exp2f(m_ref - mx) : 1.f;  // first tile: exp2(-inf) = 0, O is not read (u == 0)
          if (grow) {
            m_ref = mx;
            l_run *= corr;
          }
          if (u > 0) {
#pragma unroll
            for (int c = 0; c < HD; c += 32) {
              uint32_t r[32];
              tmem_ld32(tmem + row_lane + o_col + (uint32_t)c, r);
              tmem_ld_wait();
#pragma unroll
              for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * corr);
              tmem_st32(tmem + row_lane + o_col + (uint32_t)c, r);
            }
          }
        }
        // ---- probabilities -> tensor memory as bf16 pairs (the A operand of O_i += P_i V), over the first 32 of
        // the columns this thread has just read its scores from
        float p_sum4[4] = {0.f, 0.f, 0.f, 0.f};
        uint32_t pk[UA_KEYS / 2];
#pragma unroll
        for (int c2 = 0; c2 < UA_KEYS / 2; ++c2) {
          const float p0 = fast_exp2(fmaf(sv[2 * c2], scale_log2, -m_ref));
          const float p1 = fast_exp2(fmaf(sv[2 * c2 + 1], scale_log2, -m_ref));
          p_sum4[c2 & 1] += p0;
          p_sum4[2 + (c2 & 1)] += p1;
          pk[c2] = pack_bf16(p0, p1);
        }
        l_run += (p_sum4[0] + p_sum4[1]) + (p_sum4[2] + p_sum4[3]);
        tmem_st32(tmem + row_lane + s_col, pk);  // waits for the store
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&p_full[i]));
      }
      if (ok) ok = mbar_wait(smem_u32(&o_full[i]), 0u, abortp);
      ok = __all_sync(0xffffffffu, ok);  // the TMEM loads below are warp-collective
      // ---- one live row tile shared by the groups: group 1 hands its half (max, sum, unnormalised output) to
      // group 0 through the K/V ring, which nothing reads any more once both groups' last products are complete
      constexpr int XS = HD + 4;  // floats per exchanged row: 16-byte aligned, rows 4 banks apart
      float* xo = reinterpret_cast<float*>(smem_raw + (base - smem_u32(smem_raw)));
      float* xml = xo + UA_ROWS * XS;
      float w_self = 1.f, w_peer = 0.f;  // weights of this group's and the other group's half in the merged row
      bool peer = false, write_out = ok;
      if (kpar) {
        static_assert((UA_ROWS * XS + 2 * UA_ROWS) * 4 <= UA_STAGES * SM::STAGE, "the exchange area must fit the ring");
        {  // both groups are past their last product (or gave up): all 256 threads agree
          uint32_t r;
          asm volatile(
              "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.and.pred p, 2, 256, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
              : "=r"(r)
              : "r"((uint32_t)ok)
              : "memory");
          ok = r != 0;
        }
        if (ok && i == 1) {
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
          for (int c = 0; c < HD; c += 32) {
            uint32_t r[32];
            tmem_ld32(tmem + row_lane + o_col + (uint32_t)c, r);
            tmem_ld_wait();
#pragma unroll
            for (int k = 0; k < 32; k += 4)
              *reinterpret_cast<uint4*>(xo + row * XS + c + k) = make_uint4(r[k], r[k + 1], r[k + 2], r[k + 3]);
          }
          xml[2 * row] = m_ref;
          xml[2 * row + 1] = l_run;
        }
        asm volatile("bar.sync 2, 256;" ::: "memory");
        write_out = ok && i == 0;  // group 0 writes the merged rows
        if (write_out) {
          const float m1 = xml[2 * row], l1 = xml[2 * row + 1];
          const float M = fmaxf(m_ref, m1);
          w_self = exp2f(m_ref - M);
          w_peer = exp2f(m1 - M);
          l_run = w_self * l_run + w_peer * l1;
          m_ref = M;
          peer = true;
        }
      }
      if (write_out) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (gtid == 0 && i == 0) timeline_mark(8);  // O complete
        const int vr = row0 + (kpar ? 0 : i * UA_ROWS) + row;
        const bool is_live = vr < n_rows;
        const int qi = is_live ? vr / G : 0, g = is_live ? vr - qi * G : 0;
        const size_t orow = ((size_t)b * a_seq + qi) * H + (kh * G + g);  // (row, head) index
        const float inv = 1.f / l_run;
        const size_t total = (size_t)gridDim.z / S * a_seq * H;
#pragma unroll
        for (int c = 0; c < HD; c += 32) {
          uint32_t r[32];
          tmem_ld32(tmem + row_lane + o_col + (uint32_t)c, r);  // warp-collective: every lane takes part
          tmem_ld_wait();
          if (!is_live) continue;
          if (peer) {
#pragma unroll
            for (int k = 0; k < 32; k += 4) {
              const float4 x = *reinterpret_cast<const float4*>(xo + row * XS + c + k);
              r[k] = __float_as_uint(w_self * __uint_as_float(r[k]) + w_peer * x.x);
              r[k + 1] = __float_as_uint(w_self * __uint_as_float(r[k + 1]) + w_peer * x.y);
              r[k + 2] = __float_as_uint(w_self * __uint_as_float(r[k + 2]) + w_peer * x.z);
              r[k + 3] = __float_as_uint(w_self * __uint_as_float(r[k + 3]) + w_peer * x.w);
            }
          }
          if (S == 1) {
            __nv_bfloat16* dst = o + orow * HD + c;
#pragma unroll
            for (int k = 0; k < 32; k += 8)
              *reinterpret_cast<uint4*>(dst + k) = make_uint4(
                  pack_bf16(__uint_as_float(r[k]) * inv, __uint_as_float(r[k + 1]) * inv),
                  pack_bf16(__uint_as_float(r[k + 2]) * inv, __uint_as_float(r[k + 3]) * inv),
                  pack_bf16(__uint_as_float(r[k + 4]) * inv, __uint_as_float(r[k + 5]) * inv),
                  pack_bf16(__uint_as_float(r[k + 6]) * inv, __uint_as_float(r[k + 7]) * inv));
          } else {
            float* dst = o_part + ((size_t)split * total + orow) * HD + c;
#pragma unroll
            for (int k = 0; k < 32; k += 4)
              *reinterpret_cast<uint4*>(dst + k) = make_uint4(r[k], r[k + 1], r[k + 2], r[k + 3]);
          }
        }
        if (is_live && S > 1) {
          float* ml = ml_part + ((size_t)split * total + orow) * 2;
          ml[0] = m_ref;
          ml[1] = l_run;
        }
      }
    }
  }
  // a wait that gave up anywhere in the CTA: record it once, let copies in flight land
  ok = __syncthreads_and(ok);
  if (!ok) {
    if (tid == 0 && status) atomicCAS(status, ST_OK, ST_TIMEOUT_ATTN_UMMA);
    drain_delay();
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 9) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(SM::TMEM_COLS) : "memory");
  }
}

template <int HD>
cudaError_t launch_umma(const Launch& L, const CUtensorMap& tmK, const CUtensorMap& tmV, const void* q, void* o,
                        float* scratch, int B, int a_seq, int n, int H, int Hkv, int S, int keys_per_split,
                        int row_tiles_per_cta) {
  constexpr int SMEM = (int)UaSmem<HD>::TOTAL;
  static DeviceOnce once;
  cudaError_t e0 = once.run(
      [] { return cudaFuncSetAttribute(attn_umma_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM); });
  if (e0 != cudaSuccess) return e0;
  const int G = H / Hkv;
  const size_t total = (size_t)B * a_seq * H;
  float* o_part = scratch;
  float* ml_part = scratch ? scratch + (size_t)S * total * HD : nullptr;
  const int rows_per_cta = row_tiles_per_cta * UA_ROWS;
  dim3 grid((a_seq * G + rows_per_cta - 1) / rows_per_cta, Hkv, B * S);
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)HD);
  cudaError_t e = launch_k(L, attn_umma_kernel<HD>, grid, dim3(UA_THREADS), SMEM, tmK, tmV, (const __nv_bfloat16*)q,
                           (__nv_bfloat16*)o, o_part, ml_part, a_seq, n, H, Hkv, S, keys_per_split, row_tiles_per_cta,
                           scale_log2, L.d_status);
  L.count();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

// Key-range splits for CTAs of two 128-row tiles, whole 64-key tiles per split, no more splits than the scratch
// holds.  A split shortens the key range a CTA walks through but adds a partial result per (row, head) pair that
// the merge has to write and read, and a CTA with one row tile instead of two doubles the CTAs but loses the
// overlap of the two softmax groups, so both are what a small cost model likes best (microseconds, fitted to
// sweeps on B200: per key tile of a CTA 1.76 us with two row tiles, 1.36 us with one and 1.15 us with one whose
// groups share the key tiles, one CTA per SM at a time, 4 us of fixed cost, and for a merge 2.5 us plus 1040 bytes
// per pair and split at 5 TB/s).
AttnPlan plan_attention_umma(int B, int a_seq, int n, int H, int Hkv, size_t scratch_floats) {
  AttnPlan p;
  const int G = H / Hkv, sms = sm_count();
  const int key_tiles = (n + UA_KEYS - 1) / UA_KEYS;
  const size_t per_split = (size_t)B * a_seq * H * (128 + 2);
  const double pairs = (double)B * a_seq * H;
  int best_s = 1, best_rt = UA_TILES;
  double best_us = -1.0;
  for (int rt = UA_TILES; rt >= 1; --rt) {   // row tiles per CTA: two (the groups overlap), or one (twice the CTAs)
    if (g_attn_umma_row_tiles && rt != g_attn_umma_row_tiles) continue;
    const long ctas = (long)((a_seq * G + rt * UA_ROWS - 1) / (rt * UA_ROWS)) * Hkv * B;
    for (int S = 1; S <= key_tiles && S <= 16; ++S) {
      if (S > 1 && (size_t)S * per_split > scratch_floats) break;
      const int tps = (key_tiles + S - 1) / S;
      // a key tile of a CTA, from 16 x 512 x 1536 and 16 x 128 x 1536 (the latter with and without the two groups
      // sharing the key tiles)
      const double tile_us = rt == 2 ? 1.76 : tps >= UA_KPAR_MIN_TILES ? 1.15 : 1.36;
      if (S > 1 && (key_tiles + tps - 1) / tps != S) continue;  // the same tiles per split as a smaller count
      const double waves = (double)((ctas * S + sms - 1) / sms);
      const double us = 4.0 + waves * tps * tile_us + (S > 1 ? 2.5 + S * pairs * 1040.0 / 5.0e6 : 0.0);
      if (best_us < 0.0 || us < best_us) {
        best_s = S;
        best_rt = rt;
        best_us = us;
      }
    }
  }
  int S = g_attn_force_splits > 0 ? g_attn_force_splits : best_s;
  if (S > key_tiles) S = key_tiles;
  if (S > 1 && (size_t)S * per_split > scratch_floats) S = (int)(scratch_floats / per_split);
  if (S < 1) S = 1;
  const int tiles_per_split = (key_tiles + S - 1) / S;
  p.keys_per_split = tiles_per_split * UA_KEYS;
  p.S = (key_tiles + tiles_per_split - 1) / tiles_per_split;
  p.scratch_floats = p.S > 1 ? (size_t)p.S * per_split : 0;
  p.row_tiles = a_seq * G <= UA_ROWS ? 1 : best_rt;
  return p;
}

cudaError_t launch_attention_umma(const Launch& L, const void* q, const void* Kc, const void* Vc, void* o, int B,
                                  int a_seq, int n, int H, int Hkv, int hd, float* scratch, size_t scratch_floats,
                                  int* S_out) {
  const AttnPlan p = plan_attention_umma(B, a_seq, n, H, Hkv, scratch ? scratch_floats : 0);
  CUtensorMap tmK, tmV;
  if (!get_tensor_map_3d(Kc, (uint64_t)B, (uint64_t)n, (uint64_t)Hkv * hd, 64, &tmK) ||
      !get_tensor_map_3d(Vc, (uint64_t)B, (uint64_t)n, (uint64_t)Hkv * hd, 64, &tmV))
    return cudaErrorInvalidValue;
  if (S_out) *S_out = p.S;
  return hd == 64
             ? launch_umma<64>(L, tmK, tmV, q, o, scratch, B, a_seq, n, H, Hkv, p.S, p.keys_per_split, p.row_tiles)
             : launch_umma<128>(L, tmK, tmV, q, o, scratch, B, a_seq, n, H, Hkv, p.S, p.keys_per_split, p.row_tiles);
}

}  // namespace dllm

DLLM_TIMELINE_HOOKS(attention_umma)
DLLM_WAIT_LIMIT_HOOK(attention_umma)
