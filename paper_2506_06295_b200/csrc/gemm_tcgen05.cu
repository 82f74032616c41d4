// bf16 GEMM for sm_100a:  part[z][M][N] (fp32) = A[M, Kz] * W[N, Kz]^T
//
// Every projection of the cached step (V for all response rows; Q/K, O and the
// SwiGLU matrices for the gathered active rows; the LM head) is
// "few activation rows x a large weight matrix".  With M between 3 and a few
// hundred rows the product is bound by streaming W from HBM once, so the kernel
// is laid out around the weight stream:
//
//   * the WEIGHT tile (128 rows of W, 64 k) is the M-side operand of
//     tcgen05.mma (UMMA M = 128) and the ACTIVATION tile (BN = 32..256 rows of
//     A, 64 k) is the N-side operand, so small row counts cost no padding of
//     the 128-row dimension and the accumulator D[128 weight rows][BN act rows]
//     sits in BN TMEM columns;
//   * both tiles arrive by TMA (128-byte swizzle) into a ring of shared-memory
//     stages guarded by full/empty mbarriers; one thread issues the copies,
//     one thread issues the MMAs, tcgen05.commit releases a stage;
//   * TMEM lane = output column n, so for a fixed activation row the 32 lanes
//     of a warp store 32 consecutive floats: the epilogue writes row-major
//     [M, N] coalesced straight from tcgen05.ld registers;
//   * split-K over blockIdx.z puts >= 148 CTAs on the weight stream when N/128
//     is small; every split writes its own slab and the consumer kernel adds
//     the slabs in order (no atomics, bit-reproducible);
//   * weight tiles are requested before griddepcontrol.wait: with programmatic
//     dependent launch the ring fills while the kernel that produces the
//     activation rows is still running; the activation tile of a stage follows
//     after the wait and the stage's barrier completes when both have landed;
//   * rows of A beyond M and k beyond K are zero-filled by TMA.
//
// Every wait on an mbarrier is bounded (2 s of %globaltimer); on expiry the
// CTA records a code in the status word, skips its epilogue, lets copies in
// flight land, frees its TMEM and returns.
#include <algorithm>
#include <mutex>
#include <unordered_map>

#include "../../include/dllm.h"
#include "internal.h"
#include "tma.cuh"
#include "umma.cuh"

namespace dllm {

namespace {

constexpr int TILE_W = 128;  // weight rows per CTA (UMMA M)
constexpr int TILE_K = 64;   // k per stage: 64 bf16 = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr uint32_t W_STAGE_BYTES = TILE_W * TILE_K * 2;

// Test hook for the bounded waits: while non-zero, the TMA producer of CTA (0, 0, 0) of every launch of the
// one-CTA kernel leaves out the activation tile of its first k-block, so that stage's barrier never completes
// and the CTA's waits run into their limit (it then records a status code and returns; nothing faults).
static __device__ int g_debug_skip_act_load = 0;

constexpr int MAX_STAGES = 12;
constexpr int RASTER = 16;     // activation tiles per group of the launch-order remap

template <int BN>
struct SmemLayout {
  static constexpr uint32_t A_STAGE_BYTES = BN * TILE_K * 2;
  static constexpr uint32_t STAGE_BYTES = W_STAGE_BYTES + A_STAGE_BYTES;
  static constexpr uint32_t total(int stages) { return (uint32_t)stages * STAGE_BYTES + 1024; }  // + slack to align the base to 1024
};

// Epilogue of one tile by 128 threads: the accumulator, TMEM lanes = 128 weight rows from n0 (tile number
// tile_y), columns = BN activation rows from m0, goes to the fp32 slab (coalesced: lane = output column) or,
// with act_out, through the SwiGLU combination.  `ex`: at least min(BN, 64) * 528 bytes of shared memory that
// nothing else uses meanwhile.  tl = 0..127 identifies the thread: it works on TMEM lane tl, so its warp must be
// the one allowed to touch lanes 32 * (tl / 32) .. + 31 (warp index % 4 == tl / 32).  NAMED_BAR == 0: the 128
// threads are the whole CTA (__syncthreads); otherwise they meet on that named barrier.
template <int NAMED_BAR>
__device__ __forceinline__ void epilogue_sync() {
  if constexpr (NAMED_BAR == 0)
    __syncthreads();
  else
    asm volatile("bar.sync %0, 128;" ::"n"(NAMED_BAR) : "memory");
}
template <int BN, int NAMED_BAR = 0>
__device__ __forceinline__ void gemm_epilogue(uint32_t tmem_d, float* ex, int tl, int m0, int n0, int tile_y, int M,
                                              int N, float* __restrict__ slab, __nv_bfloat16* __restrict__ act_out,
                                              int m_ffn) {
  const int warp = tl >> 5, lane = tl & 31;
  if (m_ffn < 0) {
    // Estimate epilogue of the LM head (no split-K, act_out == nullptr, m_ffn = -1 - mask id): instead of 128
    // logits per row the CTA writes one record per activation row, {max, sum exp(v - max), argmax, -} over its
    // 128 vocabulary columns (Eq. 4; the mask id and columns past N are skipped); a merge over the tiles
    // follows.  Staged like the SwiGLU epilogue; two threads share a row, 64 columns each.
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    constexpr int EXS = 132;
    constexpr int CH = BN < 64 ? BN : 64;
    const int mask_id = -1 - m_ffn, n_tiles = (N + TILE_W - 1) / TILE_W;
    float4* rec = reinterpret_cast<float4*>(slab);
    const int rr = tl >> 1, half = tl & 1;
#pragma unroll 1
    for (int c0 = 0; c0 < BN; c0 += CH) {
      if (m0 + c0 >= M) break;  // uniform across the CTA
      {  // all TMEM loads of the chunk in flight, one wait (a load-wait-store loop pays the TMEM latency per trip)
        uint32_t r[CH / 16][16];
#pragma unroll
        for (int c = 0; c < CH; c += 16) tmem_ld16(tmem_d + ((uint32_t)(warp * 32) << 16) + (uint32_t)(c0 + c), r[c / 16]);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int c = 0; c < CH; c += 16)
#pragma unroll
          for (int j = 0; j < 16; ++j) ex[(c + j) * EXS + tl] = __uint_as_float(r[c / 16][j]);
      }
      epilogue_sync<NAMED_BAR>();
      MaxSum t{-INFINITY, 0.f, 0x7fffffff};
      if (rr < CH) {
        // two passes over the thread's 64 columns: maximum and its first index, then the exponentials as four
        // independent sums (one serial chain of dependent exponentials would dominate the epilogue)
        const float* row = ex + rr * EXS + half * 64;
        const int nb = n0 + half * 64;
#pragma unroll 4
        for (int j = 0; j < 64; j += 4) {
          const float4 v = *reinterpret_cast<const float4*>(row + j);
          const float e[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int n = nb + j + q;
            if (n < N && n != mask_id && e[q] > t.m) {
              t.m = e[q];
              t.a = n;
            }
          }
        }
        if (t.m > -INFINITY) {
          float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
          for (int j = 0; j < 64; j += 4) {
            const float4 v = *reinterpret_cast<const float4*>(row + j);
            const float e[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const int n = nb + j + q;
              s4[q] += (n < N && n != mask_id) ? expf(e[q] - t.m) : 0.f;
            }
          }
          t.s = (s4[0] + s4[1]) + (s4[2] + s4[3]);
        }
      }
      MaxSum o;
      o.m = __shfl_xor_sync(0xffffffffu, t.m, 1);
      o.s = __shfl_xor_sync(0xffffffffu, t.s, 1);
      o.a = __shfl_xor_sync(0xffffffffu, t.a, 1);
      t = merge(t, o);
      const int m = m0 + c0 + rr;
      if (rr < CH && half == 0 && m < M)
        rec[(size_t)m * n_tiles + tile_y] = make_float4(t.m, t.s, __int_as_float(t.a), 0.f);
      epilogue_sync<NAMED_BAR>();
    }
  } else if (act_out) {
    // SwiGLU epilogue (no split-K): the tile's 128 weight rows are 64 gate rows followed by the 64 up rows
    // of the same FFN columns, so TMEM lanes 0..63 hold gate and 64..127 hold up.  The accumulator goes
    // through shared memory (every MMA has completed) 64 activation rows at a time, transposed to
    // [row][weight row], and comes back as silu(gate) * up in bf16, 8 bytes per thread.
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    constexpr int EXS = 132;   // floats per staged row: 16-byte aligned, rows 4 banks apart
    constexpr int CH = BN < 64 ? BN : 64;
    const int q = tl & 15, rsub = tl >> 4;  // 4 FFN columns, 8 rows per pass
    const int col = tile_y * 64 + 4 * q;
#pragma unroll 1
    for (int c0 = 0; c0 < BN; c0 += CH) {
      if (m0 + c0 >= M) break;  // uniform across the CTA
      {  // all TMEM loads of the chunk in flight, one wait (a load-wait-store loop pays the TMEM latency per trip)
        uint32_t r[CH / 16][16];
#pragma unroll
        for (int c = 0; c < CH; c += 16) tmem_ld16(tmem_d + ((uint32_t)(warp * 32) << 16) + (uint32_t)(c0 + c), r[c / 16]);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int c = 0; c < CH; c += 16)
#pragma unroll
          for (int j = 0; j < 16; ++j) ex[(c + j) * EXS + tl] = __uint_as_float(r[c / 16][j]);
      }
      epilogue_sync<NAMED_BAR>();
#pragma unroll
      for (int rr = rsub; rr < CH; rr += 8) {
        const int m = m0 + c0 + rr;
        const float4 gt = *reinterpret_cast<const float4*>(ex + rr * EXS + 4 * q);
        const float4 up = *reinterpret_cast<const float4*>(ex + rr * EXS + 64 + 4 * q);
        if (m < M && col < m_ffn) {
          // silu(g) * u with the fast exponential and division (relative error ~1e-6, far below the bf16 rounding
          // of the result)
          const __nv_bfloat162 lo = __floats2bfloat162_rn(__fdividef(gt.x, 1.f + __expf(-gt.x)) * up.x,
                                                          __fdividef(gt.y, 1.f + __expf(-gt.y)) * up.y);
          const __nv_bfloat162 hi = __floats2bfloat162_rn(__fdividef(gt.z, 1.f + __expf(-gt.z)) * up.z,
                                                          __fdividef(gt.w, 1.f + __expf(-gt.w)) * up.w);
          uint2 pk;
          pk.x = *reinterpret_cast<const uint32_t*>(&lo);
          pk.y = *reinterpret_cast<const uint32_t*>(&hi);
          *reinterpret_cast<uint2*>(act_out + (size_t)m * m_ffn + col) = pk;
        }
      }
      epilogue_sync<NAMED_BAR>();
    }
  } else {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const int n = n0 + warp * 32 + lane;
    float* out = slab + n;
    constexpr int CH = BN < 64 ? BN : 64;  // columns (activation rows) per trip: their TMEM loads are in flight together
#pragma unroll 1
    for (int c0 = 0; c0 < BN; c0 += CH) {
      if (m0 + c0 >= M) break;  // uniform across the CTA
      uint32_t r[CH / 16][16];
#pragma unroll
      for (int c = 0; c < CH; c += 16) tmem_ld16(tmem_d + ((uint32_t)(warp * 32) << 16) + (uint32_t)(c0 + c), r[c / 16]);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      if (n < N) {
#pragma unroll
        for (int c = 0; c < CH; c += 16)
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int m = m0 + c0 + c + j;
            if (m < M) out[(size_t)m * N] = __uint_as_float(r[c / 16][j]);
          }
      }
    }
  }
}

template <int BN>
__global__ void __launch_bounds__(128) gemm_bf16_tcgen05_kernel(const __grid_constant__ CUtensorMap tmW,
                                                                const __grid_constant__ CUtensorMap tmA,
                                                                float* __restrict__ part, int M, int N, int num_kb,
                                                                int kb_per_split, size_t split_stride, int STAGES,
                                                                __nv_bfloat16* __restrict__ act_out, int m_ffn,
                                                                int* __restrict__ status) {
  using SL = SmemLayout<BN>;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t empty_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t accum_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Tile of this CTA.  With many activation tiles, CTAs that run together (consecutive in x-major launch order)
  // take RASTER activation tiles times a few weight tiles, so that their operands stay in L2 while the other
  // dimension is swept; otherwise every sweep over the weight tiles would re-read all activations from HBM.
  int mt = blockIdx.x, nt = blockIdx.y;
  if (gridDim.x > RASTER) {
    const int lin = blockIdx.x + gridDim.x * blockIdx.y, per = RASTER * gridDim.y;
    const int grp = lin / per, within = lin - grp * per;
    const int wide = min(RASTER, (int)gridDim.x - grp * RASTER);
    nt = within / wide;
    mt = grp * RASTER + within - nt * wide;
  }
  const int m0 = mt * BN;       // activation rows
  const int n0 = nt * TILE_W;   // weight rows = output columns
  const int kb0 = blockIdx.z * kb_per_split;
  const int kb1 = min(num_kb, kb0 + kb_per_split);
  const int nkb = kb1 - kb0;            // >= 1 by construction of the plan

  const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;

  int pre = 0;  // stages whose weight tile was requested before the dependency wait
  int dbg_skip = 0;
  if (threadIdx.x == 0) {
    dbg_skip = g_debug_skip_act_load;  // read here, long before it is used: not on the path behind the dependency wait
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    mbar_init(smem_u32(&accum_bar), 1);
    mbar_fence_init();
    prefetch_tensormap(&tmW);
    prefetch_tensormap(&tmA);
    pre = min(STAGES, nkb);  // weights are written by no kernel: stream them ahead of the dependency
    for (int i = 0; i < pre; ++i) {
      const uint32_t fb = smem_u32(&full_bar[i]);
      mbar_expect_tx(fb, SL::STAGE_BYTES);
      tma_load_2d(tiles + i * SL::STAGE_BYTES, &tmW, fb, (kb0 + i) * TILE_K, n0);
    }
  }
  if (warp == 1) {  // TMEM: BN fp32 columns x 128 lanes
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"((uint32_t)BN)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_d = tmem_base_slot;
  volatile int* abortp = &abort_flag;
  pdl_wait();     // the activation rows and the slab buffer belong to the preceding kernels
  pdl_trigger();

  if (warp == 0 && lane == 0) {
    // ---------------- TMA producer ----------------
    int s = 0;
    uint32_t ph = 0;
    for (int i = 0; i < nkb; ++i) {
      const uint32_t fb = smem_u32(&full_bar[s]);
      const uint32_t dstW = tiles + s * SL::STAGE_BYTES;
      const int kc = (kb0 + i) * TILE_K;
      if (i >= pre) {
        if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, abortp)) {
          if (status) atomicCAS(status, ST_OK, ST_TIMEOUT_TMA);
          break;
        }
        mbar_expect_tx(fb, SL::STAGE_BYTES);
        tma_load_2d(dstW, &tmW, fb, kc, n0);
      }
      const bool skip = i == 0 && dbg_skip != 0 && (blockIdx.x | blockIdx.y | blockIdx.z) == 0;
      if (!skip) tma_load_2d(dstW + W_STAGE_BYTES, &tmA, fb, kc, m0);
      if (++s == STAGES) {
        s = 0;
        ph ^= 1u;
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ---------------- MMA issuer ----------------
    constexpr uint32_t idesc = make_idesc(TILE_W, BN);
    bool ok = true;
    int s = 0;
    uint32_t ph = 0;
    for (int i = 0; i < nkb && ok; ++i) {
      if (!mbar_wait(smem_u32(&full_bar[s]), ph, abortp)) {
        if (status) atomicCAS(status, ST_OK, ST_TIMEOUT_MMA);
        ok = false;
        break;
      }
      if (i == 0) timeline_mark(1);                    // first stage complete: activations have arrived
      else if (i == STAGES) timeline_mark(2);          // first stage whose weights were not requested ahead of the wait
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t sW = tiles + s * SL::STAGE_BYTES;
      const uint64_t dW = make_smem_desc(sW);
      const uint64_t dA = make_smem_desc(sW + W_STAGE_BYTES);
#pragma unroll
      for (int k = 0; k < TILE_K / UMMA_K; ++k) {
        // advance 32 bytes (16 bf16) along K inside the swizzle row: +2 in 16-byte units
        umma_bf16(tmem_d, dW + (uint64_t)(2 * k), dA + (uint64_t)(2 * k), idesc, (i > 0 || k > 0) ? 1u : 0u);
      }
      umma_commit(smem_u32(&empty_bar[s]));  // stage reusable once these MMAs have read it
      if (++s == STAGES) {
        s = 0;
        ph ^= 1u;
      }
    }
    if (ok) umma_commit(smem_u32(&accum_bar));
  }
  __syncwarp();

  // ---------------- epilogue: TMEM -> registers -> global (all four warps) ----------------
  const bool have = mbar_wait(smem_u32(&accum_bar), 0u, abortp);
  if (!have && threadIdx.x == 0 && status) atomicCAS(status, ST_OK, ST_TIMEOUT_EPI);
  if (threadIdx.x == 0) timeline_mark(3);              // accumulator complete
  // the whole warp must agree before the warp-collective TMEM loads
  bool warp_ok = __all_sync(0xffffffffu, have);
  if (act_out || m_ffn < 0) warp_ok = __syncthreads_and(warp_ok);  // these epilogues exchange data between warps
  if (warp_ok) {
    float* ex = reinterpret_cast<float*>(smem_raw + (tiles - smem_u32(smem_raw)));  // the drained ring
    gemm_epilogue<BN>(tmem_d, ex, (int)threadIdx.x, m0, n0, nt, M, N, part + (size_t)blockIdx.z * split_stride, act_out,
                      m_ffn);
    if (threadIdx.x == 0) timeline_mark(4);            // this thread's part of the epilogue written
  } else {
    drain_delay();  // gave up: let copies in flight land before shared memory is released
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"((uint32_t)BN) : "memory");
  }
}

// ---------------------------------------------------------------- persistent kernel (many tiles, no split-K)
// The same product for shapes with more tiles than SMs (many active rows: batched serving, full steps): one
// CTA per SM walks through tiles blockIdx.x, blockIdx.x + gridDim.x, ... with fixed roles -- warp 0 requests
// the operand tiles of one tile after the other without a gap, warp 1 issues the MMAs into one of TWO
// accumulators in tensor memory, warps 2-5 run the epilogue of the accumulator that has just been completed --
// so the epilogue of a tile (TMEM -> registers -> global, or the SwiGLU / estimate forms) runs under the main
// loop of the next one and the operand stream never drains between tiles.  Tile order is the launch order of
// the one-tile kernel including its remap, so CTAs that run together share operands in L2.  The k loop of a
// tile is the same as in the one-tile kernel: results are bit-identical to it.
constexpr int PERSIST_THREADS = 192;
template <int BN>
struct PersistLayout {
  static constexpr uint32_t STAGE_BYTES = W_STAGE_BYTES + BN * TILE_K * 2;
  static constexpr uint32_t EX_BYTES = 64 * 132 * 4;  // staging of the SwiGLU / estimate epilogues
  static constexpr uint32_t total(int stages, bool staged) {
    return (uint32_t)stages * STAGE_BYTES + (staged ? EX_BYTES : 0) + 1024;
  }
};

template <int BN>
__global__ void __launch_bounds__(PERSIST_THREADS, 1)
    gemm_bf16_persistent_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmA,
                                float* __restrict__ part, int M, int N, int num_kb, int m_tiles, int n_tiles,
                                int STAGES, __nv_bfloat16* __restrict__ act_out, int m_ffn, int* __restrict__ status) {
  using PL = PersistLayout<BN>;
  static_assert(2 * BN <= 512, "two accumulators must fit the 512 columns of tensor memory");
  // column distance of the two accumulators: an allocation is a power of two, so 192-row tiles sit 256 apart
  constexpr uint32_t ACC = BN > 128 ? 256 : BN > 64 ? 128 : BN > 32 ? 64 : 32;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t empty_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t acc_full[2], acc_empty[2];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tiles_s = (smem_u32(smem_raw) + 1023u) & ~1023u;
  float* ex = reinterpret_cast<float*>(smem_raw + (tiles_s - smem_u32(smem_raw)) + (size_t)STAGES * PL::STAGE_BYTES);
  const int total_tiles = m_tiles * n_tiles;
  // tile L of the walk -> (activation tile, weight tile): groups of RASTER activation tiles, weight tiles inside
  auto tile_of = [&](int L, int& mt, int& nt) {
    const int per = RASTER * n_tiles, grp = L / per, within = L - grp * per;
    const int wide = min(RASTER, m_tiles - grp * RASTER);
    nt = within / wide;
    mt = grp * RASTER + within - nt * wide;
  };

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&acc_full[a]), 1);
      mbar_init(smem_u32(&acc_empty[a]), 128);  // every epilogue thread arrives once it has read its part
    }
    mbar_fence_init();
    prefetch_tensormap(&tmW);
    prefetch_tensormap(&tmA);
  }
  if (warp == 1) {  // TMEM: two accumulators of BN fp32 columns x 128 lanes
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"(2u * ACC)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_d = tmem_base_slot;
  volatile int* abortp = &abort_flag;
  pdl_wait();     // the activation rows and the output buffer belong to the preceding kernels
  pdl_trigger();
  bool ok = true;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      for (int L = blockIdx.x; L < total_tiles && ok; L += gridDim.x) {
        int mt, nt;
        tile_of(L, mt, nt);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, abortp)) {
            if (status) atomicCAS(status, ST_OK, ST_TIMEOUT_TMA);
            ok = false;
            break;
          }
          const uint32_t fb = smem_u32(&full_bar[s]);
          const uint32_t dst = tiles_s + s * PL::STAGE_BYTES;
          mbar_expect_tx(fb, PL::STAGE_BYTES);
          tma_load_2d(dst, &tmW, fb, kb * TILE_K, nt * TILE_W);
          tma_load_2d(dst + W_STAGE_BYTES, &tmA, fb, kb * TILE_K, mt * BN);
          if (++s == STAGES) {
            s = 0;
            ph ^= 1u;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(TILE_W, BN);
      int s = 0, j = 0;
      uint32_t ph = 0;
      for (int L = blockIdx.x; L < total_tiles && ok; L += gridDim.x, ++j) {
        const int a = j & 1;
        // the epilogue of the tile that used this accumulator two tiles ago has read it
        if (!mbar_wait(smem_u32(&acc_empty[a]), ((uint32_t)(j >> 1) & 1u) ^ 1u, abortp)) {
          if (status) atomicCAS(status, ST_OK, ST_TIMEOUT_MMA);
          ok = false;
          break;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(smem_u32(&full_bar[s]), ph, abortp)) {
            if (status) atomicCAS(status, ST_OK, ST_TIMEOUT_MMA);
            ok = false;
            break;
          }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t sW = tiles_s + s * PL::STAGE_BYTES;
          const uint64_t dW = make_smem_desc(sW);
          const uint64_t dA = make_smem_desc(sW + W_STAGE_BYTES);
#pragma unroll
          for (int k = 0; k < TILE_K / UMMA_K; ++k)
            umma_bf16(tmem_d + (uint32_t)a * ACC, dW + (uint64_t)(2 * k), dA + (uint64_t)(2 * k), idesc,
                      (kb > 0 || k > 0) ? 1u : 0u);
          umma_commit(smem_u32(&empty_bar[s]));  // stage reusable once these MMAs have read it
          if (++s == STAGES) {
            s = 0;
            ph ^= 1u;
          }
        }
        if (ok) umma_commit(smem_u32(&acc_full[a]));
      }
    }
  } else {
    // ---------------- epilogue warps 2..5: TMEM lanes 32 * (warp % 4) .. + 31 ----------------
    const int tl = (warp & 3) * 32 + lane;
    int j = 0;
    for (int L = blockIdx.x; L < total_tiles; L += gridDim.x, ++j) {
      const int a = j & 1;
      int mt, nt;
      tile_of(L, mt, nt);
      bool have = mbar_wait(smem_u32(&acc_full[a]), (uint32_t)(j >> 1) & 1u, abortp);
      // the 128 epilogue threads agree (the TMEM loads are warp-collective and the staged forms exchange data)
      {
        uint32_t r;
        asm volatile(
            "{\n\t.reg .pred p, q;\n\t"
            "setp.ne.u32 q, %1, 0;\n\t"
            "bar.red.and.pred p, 1, 128, q;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(r)
            : "r"((uint32_t)have)
            : "memory");
        have = r != 0;
      }
      if (!have) {
        if (tl == 0 && status) atomicCAS(status, ST_OK, ST_TIMEOUT_EPI);
        ok = false;
        break;
      }
      gemm_epilogue<BN, 1>(tmem_d + (uint32_t)a * ACC, ex, tl, mt * BN, nt * TILE_W, nt, M, N, part, act_out, m_ffn);
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      mbar_arrive(smem_u32(&acc_empty[a]));
    }
  }
  ok = __syncthreads_and(ok);
  if (!ok) drain_delay();  // gave up: let copies in flight land before shared memory is released
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(2u * ACC) : "memory");
  }
}

// ---------------------------------------------------------------- CTA-pair kernel
// The same product with cta_group::2: two CTAs of a cluster (consecutive weight tiles, blockIdx.x = 2p, 2p + 1)
// work on one 256 x BN tile.  Each stages its own 128 weight rows and HALF of the activation tile, the first CTA
// of the pair issues MMAs that read both CTAs' shared memory, and each CTA ends with its own 128 x BN
// accumulator in its own TMEM.  Against the one-CTA kernel the activation tile crosses the L2 -> SM fabric once
// per 256 weight rows instead of once per 128, which is what bounds the product from about 128 activation rows
// on.  Loads carry no multicast: every byte is requested by the CTA that stages it.
template <int BN>
struct PairLayout {
  static constexpr uint32_t A_HALF_BYTES = (BN / 2) * TILE_K * 2;
  static constexpr uint32_t STAGE_BYTES = W_STAGE_BYTES + A_HALF_BYTES;
  static constexpr uint32_t total(int stages) { return (uint32_t)stages * STAGE_BYTES + 1024; }
};

template <int BN>
__global__ void __launch_bounds__(128) gemm_bf16_pair_kernel(const __grid_constant__ CUtensorMap tmW,
                                                             const __grid_constant__ CUtensorMap tmA,
                                                             float* __restrict__ part, int M, int N, int num_kb,
                                                             int kb_per_split, size_t split_stride, int STAGES,
                                                             __nv_bfloat16* __restrict__ act_out, int m_ffn,
                                                             int* __restrict__ status) {
  using PL = PairLayout<BN>;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[MAX_STAGES];   // used in the pair's first CTA: bytes of both CTAs
  __shared__ __align__(8) uint64_t empty_bar[MAX_STAGES];  // in each CTA: its stage may be refilled
  __shared__ __align__(8) uint64_t accum_bar;              // in each CTA: the accumulator is complete
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const int m0 = blockIdx.y * BN;
  const int n0 = blockIdx.x * TILE_W;  // the pair: blockIdx.x = 2p, 2p + 1
  const int kb0 = blockIdx.z * kb_per_split;
  const int kb1 = min(num_kb, kb0 + kb_per_split);
  const int nkb = kb1 - kb0;
  const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    mbar_init(smem_u32(&accum_bar), 1);
    mbar_fence_init();
    prefetch_tensormap(&tmW);
    prefetch_tensormap(&tmA);
  }
  if (warp == 1) {  // the same warp of both CTAs: BN fp32 columns x 128 lanes in each CTA's TMEM
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"((uint32_t)BN)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync();  // both CTAs' barriers exist before either signals the other's
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_d = tmem_base_slot;
  volatile int* abortp = &abort_flag;

  int pre = 0;
  if (threadIdx.x == 0) {
    pre = min(STAGES, nkb);  // weights are written by no kernel: stream them ahead of the dependency
    for (int i = 0; i < pre; ++i) {
      if (leader) mbar_expect_tx(smem_u32(&full_bar[i]), 2 * PL::STAGE_BYTES);
      tma_load_2d_pair(tiles + i * PL::STAGE_BYTES, &tmW, cluster_addr(smem_u32(&full_bar[i]), 0), (kb0 + i) * TILE_K, n0);
    }
  }
  pdl_wait();     // the activation rows and the slab buffer belong to the preceding kernels
  pdl_trigger();

  if (warp == 0 && lane == 0) {
    // ---------------- TMA producer (both CTAs) ----------------
    int s = 0;
    uint32_t ph = 0;
    for (int i = 0; i < nkb; ++i) {
      const uint32_t fb = cluster_addr(smem_u32(&full_bar[s]), 0);
      const uint32_t dstW = tiles + s * PL::STAGE_BYTES;
      const int kc = (kb0 + i) * TILE_K;
      if (i >= pre) {
        if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, abortp)) {
          if (status) atomicCAS(status, ST_OK, ST_TIMEOUT_TMA);
          break;
        }
        if (leader) mbar_expect_tx(smem_u32(&full_bar[s]), 2 * PL::STAGE_BYTES);
        tma_load_2d_pair(dstW, &tmW, fb, kc, n0);
      }
      tma_load_2d_pair(dstW + W_STAGE_BYTES, &tmA, fb, kc, m0 + (int)rank * (BN / 2));
      if (++s == STAGES) {
        s = 0;
        ph ^= 1u;
      }
    }
  } else if (leader && warp == 1 && lane == 0) {
    // ---------------- MMA issuer (first CTA of the pair) ----------------
    constexpr uint32_t idesc = make_idesc(2 * TILE_W, BN);
    bool ok = true;
    int s = 0;
    uint32_t ph = 0;
    for (int i = 0; i < nkb && ok; ++i) {
      if (!mbar_wait(smem_u32(&full_bar[s]), ph, abortp)) {
        if (status) atomicCAS(status, ST_OK, ST_TIMEOUT_MMA);
        ok = false;
        break;
      }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t sW = tiles + s * PL::STAGE_BYTES;
      const uint64_t dW = make_smem_desc(sW);
      const uint64_t dA = make_smem_desc(sW + W_STAGE_BYTES);
#pragma unroll
      for (int k = 0; k < TILE_K / UMMA_K; ++k)
        umma_bf16_pair(tmem_d, dW + (uint64_t)(2 * k), dA + (uint64_t)(2 * k), idesc, (i > 0 || k > 0) ? 1u : 0u);
      umma_commit_pair(smem_u32(&empty_bar[s]));  // both CTAs may refill the stage once these MMAs have read it
      if (++s == STAGES) {
        s = 0;
        ph ^= 1u;
      }
    }
    if (ok) umma_commit_pair(smem_u32(&accum_bar));
  }
  __syncwarp();

  // ---------------- epilogue: each CTA writes its own 128 output columns ----------------
  const bool have = mbar_wait(smem_u32(&accum_bar), 0u, abortp);
  if (!have && threadIdx.x == 0 && status) atomicCAS(status, ST_OK, ST_TIMEOUT_EPI);
  bool warp_ok = __all_sync(0xffffffffu, have);
  if (act_out || m_ffn < 0) warp_ok = __syncthreads_and(warp_ok);
  if (warp_ok) {
    float* ex = reinterpret_cast<float*>(smem_raw + (tiles - smem_u32(smem_raw)));  // the drained ring
    gemm_epilogue<BN>(tmem_d, ex, (int)threadIdx.x, m0, n0, (int)blockIdx.x, M, N,
                      part + (size_t)blockIdx.z * split_stride, act_out, m_ffn);
  } else {
    drain_delay();
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync();  // neither CTA leaves, nor is TMEM freed, while the other may still use this one's memory
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"((uint32_t)BN) : "memory");
  }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

struct MapKey {
  const void* base;
  uint64_t batch, rows, cols;
  uint32_t box_rows;
  int device;  // a map is encoded in the context of the device that was current
  bool operator==(const MapKey& o) const {
    return base == o.base && batch == o.batch && rows == o.rows && cols == o.cols && box_rows == o.box_rows &&
           device == o.device;
  }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    size_t h = std::hash<const void*>()(k.base);
    h ^= std::hash<uint64_t>()(k.rows * 1315423911ull + k.cols + k.batch * 2654435761ull) + 0x9e3779b97f4a7c15ull +
         (h << 6) + (h >> 2);
    return h ^ (k.box_rows * 2654435761u) ^ ((size_t)k.device << 56);
  }
};

bool get_map(const MapKey& key, CUtensorMap* out) {
  static std::unordered_map<MapKey, CUtensorMap, MapKeyHash> cache;
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  auto it = cache.find(key);
  if (it != cache.end()) {
    *out = it->second;
    return true;
  }
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return false;
  const bool three = key.batch > 0;
  cuuint64_t dims[3] = {key.cols, key.rows, three ? key.batch : 1};
  cuuint64_t strides[2] = {key.cols * 2, key.rows * key.cols * 2};
  cuuint32_t box[3] = {(cuuint32_t)TILE_K, key.box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUtensorMap tm;
  CUresult r = enc(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, three ? 3 : 2, const_cast<void*>(key.base), dims, strides,
                   box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  if (cache.size() > 8192) cache.clear();
  cache.emplace(key, tm);
  *out = tm;
  return true;
}

// Most stages whose ring fits the 227 KB of shared memory one CTA may use.
constexpr int max_stages(int bn) {
  const int fit = (227 * 1024 - 1024 - 256) / (int)(W_STAGE_BYTES + bn * TILE_K * 2);
  return fit < MAX_STAGES ? fit : MAX_STAGES;
}

template <int BN>
cudaError_t launch_one(const Launch& L, const CUtensorMap& tmW, const CUtensorMap& tmA, float* part, int M, int N,
                       int num_kb, const GemmPlan& plan, void* act_out, int m_ffn) {
  using SL = SmemLayout<BN>;
  static DeviceOnce once;
  cudaError_t e0 = once.run([] {
    return cudaFuncSetAttribute(gemm_bf16_tcgen05_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)SL::total(max_stages(BN)));
  });
  if (e0 != cudaSuccess) return e0;
  const int stages = plan.stages < 2 ? 2 : plan.stages > max_stages(BN) ? max_stages(BN) : plan.stages;
  dim3 grid((M + BN - 1) / BN, (N + TILE_W - 1) / TILE_W, plan.S_max);
  cudaError_t e = launch_k(L, gemm_bf16_tcgen05_kernel<BN>, grid, dim3(128), SL::total(stages), tmW, tmA, part, M, N,
                           num_kb, plan.upc, (size_t)M * N, stages, (__nv_bfloat16*)act_out, m_ffn, L.d_status);
  L.count();
  return e != cudaSuccess ? e : cudaGetLastError();
}

template <int BN>
cudaError_t launch_persistent(const Launch& L, const CUtensorMap& tmW, const CUtensorMap& tmA, float* part, int M,
                              int N, int num_kb, const GemmPlan& plan, void* act_out, int m_ffn) {
  using PL = PersistLayout<BN>;
  const bool staged = act_out != nullptr || m_ffn < 0;
  const int fit = (227 * 1024 - 1024 - 512 - (staged ? (int)PL::EX_BYTES : 0)) / (int)PL::STAGE_BYTES;
  const int stages = fit < MAX_STAGES ? fit : MAX_STAGES;
  static DeviceOnce once;
  cudaError_t e0 = once.run([] {
    return cudaFuncSetAttribute(gemm_bf16_persistent_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                227 * 1024 - 512);
  });
  if (e0 != cudaSuccess) return e0;
  const int n_tiles = (N + TILE_W - 1) / TILE_W, m_tiles = (M + BN - 1) / BN;
  const int ctas = std::min(m_tiles * n_tiles, sm_count());
  cudaError_t e = launch_k(L, gemm_bf16_persistent_kernel<BN>, dim3(ctas), dim3(PERSIST_THREADS),
                           PL::total(stages, staged), tmW, tmA, part, M, N, num_kb, m_tiles, n_tiles, stages,
                           (__nv_bfloat16*)act_out, m_ffn, L.d_status);
  L.count();
  return e != cudaSuccess ? e : cudaGetLastError();
}

template <int BN>
cudaError_t launch_pair(const Launch& L, const CUtensorMap& tmW, const CUtensorMap& tmA, float* part, int M, int N,
                        int num_kb, const GemmPlan& plan, void* act_out, int m_ffn) {
  using PL = PairLayout<BN>;
  constexpr int fit = (227 * 1024 - 1024 - 256) / (int)PL::STAGE_BYTES;
  constexpr int most = fit < MAX_STAGES ? fit : MAX_STAGES;
  static DeviceOnce once;
  cudaError_t e0 = once.run([] {
    return cudaFuncSetAttribute(gemm_bf16_pair_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)PL::total(most));
  });
  if (e0 != cudaSuccess) return e0;
  const int stages = plan.stages < 2 ? 2 : plan.stages > most ? most : plan.stages;
  dim3 grid(N / TILE_W, (M + BN - 1) / BN, plan.S_max);  // pairs along x
  cudaError_t e = launch_k_cluster(L, gemm_bf16_pair_kernel<BN>, grid, dim3(128), PL::total(stages), dim3(2, 1, 1), tmW,
                                   tmA, part, M, N, num_kb, plan.upc, (size_t)M * N, stages, (__nv_bfloat16*)act_out,
                                   m_ffn, L.d_status);
  L.count();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

static int current_device() {
  int dev = 0;
  return cudaGetDevice(&dev) == cudaSuccess ? dev : -1;
}
bool get_tensor_map_2d(const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows, CUtensorMap* out) {
  return get_map(MapKey{base, 0, rows, cols, box_rows, current_device()}, out);
}
bool get_tensor_map_3d(const void* base, uint64_t batch, uint64_t rows, uint64_t cols, uint32_t box_rows,
                       CUtensorMap* out) {
  return get_map(MapKey{base, batch, rows, cols, box_rows, current_device()}, out);
}

int sm_count() {
  static std::atomic<int> per_device[64];  // zero-initialised: not yet asked
  int dev = 0, v = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;  // no device visible (host-only size queries): a B200's count
  const bool tracked = dev >= 0 && dev < 64;
  if (tracked && (v = per_device[dev].load(std::memory_order_relaxed)) > 0) return v;
  if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
  if (tracked) per_device[dev].store(v, std::memory_order_relaxed);
  return v;
}

// tuning / test override of the kernel choice for unsplit plans with 256-row tiles: 0 automatic, 1 always the
// persistent kernel, -1 never (see dllm_debug_gemm_plan)
int g_gemm_force_persistent = 0;

Partials make_partials(const float* p, int M, int N, const GemmPlan& plan) {
  return Partials{p, (size_t)M * N, plan.S_max, N};  // every element has S_max slabs
}

// Tile shape, ring depth and split-K factor, from sweeps on B200: up to 256
// activation rows the product is bound by streaming W, so k ranges are split
// until at least one CTA per SM (two with 128-row tiles) streams weights.
GemmPlan plan_gemm_bf16(int M, int N, int K, int force_split, int force_stages, int force_bn, int force_pair,
                        int force_persistent) {
  GemmPlan p;
  const int sms = sm_count();
  const long n_tiles = (N + TILE_W - 1) / TILE_W;
  p.BN = M <= 32 ? 32 : M <= 64 ? 64 : M <= 256 ? 128 : 256;
  p.pair = 0;
  int pair_stages = 3;
  const bool automatic = force_pair == 0 && force_bn == 0 && force_split == 0;
  const long tiles64 = n_tiles * ((M + 63) / 64), tiles128 = n_tiles * ((M + 127) / 128);
  const long tiles256 = n_tiles * ((M + 255) / 256);
  if (automatic && M > 64 && M <= 128 && tiles64 <= sms) {
    // 65..128 rows against few weight tiles (the product will be split): two 64-row tiles per weight tile put
    // twice the CTAs on the weight stream (128 x 4096 x 4096: 14.9 against 17.8 us, 128 x 4096 x 3584: 10.0
    // against 11.8 us; with many weight tiles the 128-row tile stays: every weight tile crosses the fabric once)
    p.BN = 64;
  } else if (automatic && M > 128 && M <= 256 && tiles64 <= sms && (K + TILE_K - 1) / TILE_K <= 64) {
    // 129..256 rows against few weight tiles and a short k range (256 x 4096 x 4096, the V projection of every
    // cached step): four 64-row tiles per weight tile with two splits take as long as two 128-row tiles with four
    // (15.3 against 15.6 us) and leave the consumer half the slabs to sum (19.4 against 20.9 us with the
    // reduction); with a long k range the doubled weight traffic through the L2 -> SM fabric costs more (256 x
    // 4096 x 12288: 36.8 against 32.6 us)
    p.BN = 64;
  } else if (automatic && M > 256 && M <= 1024 && 2L * sms / tiles128 >= 2) {
    // so few 128-row tiles that they fill the SMs only when the k range is split: 320 x 4096 x 12288 43.8 against
    // 66.4 us without a split, 384 x 3584 x 18944 53.8 against 96.0 us, 512 x 4096 x 3584 20.0 against 24.4 us
    p.BN = 128;
  } else if (force_pair == 0 && force_bn == 0 && force_split <= 1 && N % (2 * TILE_W) == 0) {
    // CTA pairs where they measured faster (B200): products that need no split between 129 and 1024 activation
    // rows, where the activation tile's trips through the L2 -> SM fabric bound the one-CTA kernel.
    if (M > 128 && M <= 256 && n_tiles >= sms) {   // (65..128 rows: one-CTA 128-row tiles measured 10 % faster)
      p.pair = 1;
      p.BN = 256;
    } else if (M > 256 && M <= 1024 && 4 * tiles128 <= 11L * sms) {
      // pairs on 128-row tiles up to 2.75 tiles per SM: 768 x 8192 x 4096 44.4 us against 48.3 on 256-row pair
      // tiles and 52.7 on the persistent kernel (192 tiles of 256 rows are 1.3 waves of its CTAs)
      p.pair = 1;
      p.BN = 128;
      pair_stages = tiles128 <= 2L * sms ? 4 : 3;  // all 128-row pair tiles resident at once: a deeper ring
    } else if (M > 256 && M <= 1024 && tiles256 <= 2L * sms) {
      // (with more 256-row tiles than that the persistent kernel below measured faster: gate / up at 512, 768 and
      // 1024 rows 114 -> 91, 136 -> 127, 181 -> 162 us)
      p.pair = 1;
      p.BN = 256;
    }
  }
  // 192-row tiles (persistent kernel only) where they leave at least 15 % fewer padded activation rows than
  // 256-row tiles: the 576 rows of a mixed step (prompt refresh + adaptive response update) are 3 x 192, not 3 x 256
  if (!p.pair && p.BN == 256 && force_split <= 1 && force_persistent >= 0 && g_gemm_force_persistent >= 0) {
    const long pad192 = (M + 191) / 192 * 192L, pad256 = (M + 255) / 256 * 256L;
    if (pad192 * 115 <= pad256 * 100 && n_tiles * (pad192 / 192) > sms) p.BN = 192;
  }
  if (force_bn == 32 || force_bn == 64 || force_bn == 128 || force_bn == 192 || force_bn == 256) p.BN = force_bn;
  if (force_pair > 0) p.pair = (p.BN == 128 || p.BN == 256) && N % (2 * TILE_W) == 0;
  p.stages = force_stages > 0 ? force_stages : p.pair ? pair_stages : (p.BN == 128 ? 3 : 4);
  p.num_kb = (K + TILE_K - 1) / TILE_K;
  p.m_tiles = (M + p.BN - 1) / p.BN;
  const long tiles = (long)p.m_tiles * n_tiles;
  // every split adds a slab the consumer has to read: with few activation rows
  // one wave of CTAs is enough, with 128-row tiles two CTAs per SM pay off
  // (two CTAs per SM also for 64-row tiles when there are two or more of them per weight tile)
  const bool two_per_sm = p.BN == 128 || (p.BN == 64 && p.m_tiles > 1);
  int S = two_per_sm ? (int)(2L * sms / tiles) : (int)((sms + tiles - 1) / tiles);  // all CTAs resident at once
  const int max_s = p.num_kb / 4 > 1 ? p.num_kb / 4 : 1;
  if (S > max_s) S = max_s;
  if (S < 1) S = 1;
  if (p.pair && force_pair == 0) S = 1;
  if (force_split > 0) S = force_split < p.num_kb ? force_split : p.num_kb;
  // more tiles than SMs, no split, one-CTA 256-row tiles: the persistent kernel (epilogue under the next main loop)
  if (force_persistent == 0) force_persistent = g_gemm_force_persistent;
  p.persistent = (force_persistent >= 0) && !p.pair && (p.BN == 256 || p.BN == 192) && S == 1 &&
                 (force_persistent > 0 || tiles > sms || p.BN == 192);
  p.upc = (p.num_kb + S - 1) / S;                 // k-blocks per split
  p.S_max = (p.num_kb + p.upc - 1) / p.upc;       // no empty split
  p.ctas = (int)tiles * p.S_max;
  p.total_units = (int)tiles * p.num_kb;
  return p;
}

cudaError_t launch_gemm_bf16(const Launch& L, const void* A, const void* W, float* part, int M, int N, int K,
                             const GemmPlan& plan, const char** err, void* act_out, int m_ffn) {
  static const char* e_shape = "bf16 GEMM needs K % 8 == 0 and 16-byte aligned operands";
  static const char* e_map = "cuTensorMapEncodeTiled failed or is unavailable";
  if (M <= 0 || N <= 0) return cudaSuccess;
  if (K <= 0 || (K & 7) || ((uintptr_t)A & 15) || ((uintptr_t)W & 15)) {
    if (err) *err = e_shape;
    return cudaErrorInvalidValue;
  }
  if (!act_out && m_ffn < 0 && (plan.S_max != 1 || ((uintptr_t)part & 15))) {
    if (err) *err = "the estimate epilogue needs an unsplit plan";
    return cudaErrorInvalidValue;
  }
  if (act_out && (plan.S_max != 1 || N != 2 * m_ffn || (m_ffn & 63) || ((uintptr_t)act_out & 7))) {
    if (err) *err = "the SwiGLU epilogue needs an unsplit plan and d_ffn % 64 == 0";
    return cudaErrorInvalidValue;
  }
  CUtensorMap tmW, tmA;
  if (!get_tensor_map_2d(W, (uint64_t)N, (uint64_t)K, TILE_W, &tmW) ||
      !get_tensor_map_2d(A, (uint64_t)M, (uint64_t)K, (uint32_t)(plan.pair ? plan.BN / 2 : plan.BN), &tmA)) {
    if (err) *err = e_map;
    return cudaErrorInvalidValue;
  }
  const int num_kb = (K + TILE_K - 1) / TILE_K;
  if (plan.pair) {
    if (N % (2 * TILE_W)) {
      if (err) *err = "CTA pairs need N % 256 == 0";
      return cudaErrorInvalidValue;
    }
    return plan.BN == 128 ? launch_pair<128>(L, tmW, tmA, part, M, N, num_kb, plan, act_out, m_ffn)
                          : launch_pair<256>(L, tmW, tmA, part, M, N, num_kb, plan, act_out, m_ffn);
  }
  if (plan.persistent)
    return plan.BN == 192 ? launch_persistent<192>(L, tmW, tmA, part, M, N, num_kb, plan, act_out, m_ffn)
                          : launch_persistent<256>(L, tmW, tmA, part, M, N, num_kb, plan, act_out, m_ffn);
  if (plan.BN == 192) {
    if (err) *err = "192-row tiles exist in the persistent kernel only";
    return cudaErrorInvalidValue;
  }
  switch (plan.BN) {
    case 32: return launch_one<32>(L, tmW, tmA, part, M, N, num_kb, plan, act_out, m_ffn);
    case 64: return launch_one<64>(L, tmW, tmA, part, M, N, num_kb, plan, act_out, m_ffn);
    case 128: return launch_one<128>(L, tmW, tmA, part, M, N, num_kb, plan, act_out, m_ffn);
    default: return launch_one<256>(L, tmW, tmA, part, M, N, num_kb, plan, act_out, m_ffn);
  }
}

}  // namespace dllm

namespace dllm {
cudaError_t set_debug_skip_act_load(int enable) {
  const int v = enable != 0;
  return cudaMemcpyToSymbol(g_debug_skip_act_load, &v, sizeof v);
}
}  // namespace dllm

extern "C" dllm_status dllm_debug_gemm_plan(int persistent) {
  if (persistent < -1 || persistent > 1) {
    dllm::set_last_error("dllm_debug_gemm_plan: -1, 0 or 1");
    return DLLM_INVALID_ARG;
  }
  dllm::g_gemm_force_persistent = persistent;
  return DLLM_OK;
}

DLLM_TIMELINE_HOOKS(gemm_tcgen05)
DLLM_WAIT_LIMIT_HOOK(gemm_tcgen05)
