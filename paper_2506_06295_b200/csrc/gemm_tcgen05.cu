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
//   * the kernel is persistent: work is cut into units (output tile, k-block)
//     in tile-major order and CTA i (one per SM) owns a contiguous run of
//     them, so all SMs stream the same number of weight bytes whatever N/128
//     is; a CTA writes each run of k-blocks of one tile ("segment") to its own
//     slab and the consumer kernel adds the slabs of a tile in k order (no
//     atomics, bit-reproducible); two TMEM accumulators let the epilogue warps
//     drain one segment while the next is being multiplied;
//   * weight tiles are requested before griddepcontrol.wait, so with
//     programmatic dependent launch the ring (up to ~200 KB per SM) fills
//     while the kernel that produces the activations is still running;
//   * rows of A beyond M and k beyond K are zero-filled by TMA.
//
// Every wait on an mbarrier is bounded (2 s of %globaltimer); on expiry the
// CTA records a code in the status word, skips its epilogue, lets copies in
// flight land, frees its TMEM and returns.
#include <mutex>
#include <unordered_map>

#include "internal.h"
#include "tma.cuh"
#include "umma.cuh"

namespace dllm {

namespace {

constexpr int TILE_W = 128;  // weight rows per CTA (UMMA M)
constexpr int TILE_K = 64;   // k per stage: 64 bf16 = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr uint32_t W_STAGE_BYTES = TILE_W * TILE_K * 2;

constexpr int MAX_STAGES = 12;
constexpr int GEMM_THREADS = 192;  // warp 0: TMA producer, warp 1: MMA issuer, warps 2-5: epilogue

// WM = weight sub-tiles of 128 rows per tile: one activation tile in shared
// memory feeds WM MMAs, so the activation rows cross the L2 -> SM fabric once
// per 128 * WM weight rows.
template <int BN, int WM>
struct SmemLayout {
  static constexpr uint32_t W_BYTES = WM * W_STAGE_BYTES;
  static constexpr uint32_t A_STAGE_BYTES = BN * TILE_K * 2;
  static constexpr uint32_t STAGE_BYTES = W_BYTES + A_STAGE_BYTES;
  static constexpr uint32_t total(int stages) { return (uint32_t)stages * STAGE_BYTES + 1024; }  // + slack to align the base to 1024
};

// One contiguous run of k-blocks of one output tile inside a CTA's unit range.
struct Segment {
  int tile, kb0, nkb;
};
__device__ __forceinline__ Segment segment_at(int u, int u1, int num_kb) {
  Segment sg;
  sg.tile = u / num_kb;
  sg.kb0 = u - sg.tile * num_kb;
  sg.nkb = min(num_kb - sg.kb0, u1 - u);
  return sg;
}

// Work = units (output tile, k-block), tile-major; CTA i owns units
// [i*upc, (i+1)*upc).  A CTA therefore computes a sequence of segments (runs of
// k-blocks of one tile); the segment of CTA i for a tile goes to slab
// i - first_cta(tile) of that tile, so a consumer that adds the slabs of a tile
// in index order adds the k ranges in ascending order, whatever ran first.
template <int BN, int WM>
__global__ void __launch_bounds__(GEMM_THREADS) gemm_bf16_tcgen05_kernel(
    const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmA, float* __restrict__ part, int M,
    int N, int num_kb, int m_tiles, int total_units, int upc, size_t split_stride, int STAGES, int w_tiled,
    int* __restrict__ status) {
  using SL = SmemLayout<BN, WM>;
  constexpr int TW = TILE_W * WM;                            // weight rows per tile
  constexpr int ACC_BUFS = (2 * WM * BN <= 512) ? 2 : 1;     // accumulator sets in TMEM
  constexpr uint32_t ACC_COLS = WM * BN;
  constexpr uint32_t TMEM_COLS = ACC_BUFS * ACC_COLS < 32 ? 32 : ACC_BUFS * ACC_COLS;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t empty_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t acc_full[2];
  __shared__ __align__(8) uint64_t acc_empty[2];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int u0 = blockIdx.x * upc;
  const int u1 = min(total_units, u0 + upc);
  const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;
  volatile int* abortp = &abort_flag;
  int pre = 0;  // stages whose weight tile was requested before the dependency wait
  // weight tile (nt, kb): a box of the row-major [N, K] matrix, or one contiguous
  // 16 KB block of the tiled layout [N/128][K/64][128][64]
  auto load_w = [&](uint32_t dst, uint32_t bar, int nt, int kb) {
#pragma unroll
    for (int w = 0; w < WM; ++w) {
      if (w_tiled)
        tma_load_2d(dst + w * W_STAGE_BYTES, &tmW, bar, 0, ((nt * WM + w) * num_kb + kb) * TILE_W);
      else
        tma_load_2d(dst + w * W_STAGE_BYTES, &tmW, bar, kb * TILE_K, nt * TW + w * TILE_W);
    }
  };

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    for (int b = 0; b < ACC_BUFS; ++b) {
      mbar_init(smem_u32(&acc_full[b]), 1);
      mbar_init(smem_u32(&acc_empty[b]), 4);  // one arrival per epilogue warp
    }
    mbar_fence_init();
    // Weights are written by no kernel: start streaming them before the grid
    // this launch depends on has finished.  The activation tile of the same
    // stage is requested after pdl_wait(); the stage's barrier completes when
    // both have landed.
    prefetch_tensormap(&tmW);
    prefetch_tensormap(&tmA);
    pre = min(STAGES, u1 - u0);
    for (int i = 0; i < pre; ++i) {
      const Segment sg = segment_at(u0 + i, u1, num_kb);
      const uint32_t fb = smem_u32(&full_bar[i]);
      mbar_expect_tx(fb, SL::STAGE_BYTES);
      load_w(tiles + i * SL::STAGE_BYTES, fb, sg.tile / m_tiles, sg.kb0);
    }
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_d = tmem_base_slot;
  pdl_wait();     // activation rows and the slab buffer belong to the preceding kernels
  pdl_trigger();  // (after this CTA holds its TMEM: a dependent CTA can only queue behind it)

  if (warp == 0 && lane == 0) {
    // ---------------- TMA producer ----------------
    int s = 0;
    uint32_t ph = 0;
    int u = u0;
    for (int i = 0; u < u1; ++i, ++u) {
      const int tile = u / num_kb, kb = u - tile * num_kb;
      const uint32_t fb = smem_u32(&full_bar[s]);
      const uint32_t dstW = tiles + s * SL::STAGE_BYTES;
      if (i >= pre) {
        if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, abortp)) {
          if (status) atomicCAS(status, ST_OK, ST_TIMEOUT_TMA);
          break;
        }
        mbar_expect_tx(fb, SL::STAGE_BYTES);
        load_w(dstW, fb, tile / m_tiles, kb);
      }
      tma_load_2d(dstW + SL::W_BYTES, &tmA, fb, kb * TILE_K, (tile % m_tiles) * BN);
      if (++s == STAGES) {
        s = 0;
        ph ^= 1u;
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ---------------- MMA issuer ----------------
    constexpr uint32_t idesc = make_idesc(TILE_W, BN);
    int s = 0;
    uint32_t ph = 0;
    bool ok = true;
    int seg = 0;
    for (int u = u0; u < u1 && ok; ++seg) {
      const Segment sg = segment_at(u, u1, num_kb);
      const int buf = seg % ACC_BUFS;
      // the epilogue has drained the accumulator this segment reuses
      if (!mbar_wait(smem_u32(&acc_empty[buf]), (((uint32_t)(seg / ACC_BUFS)) & 1u) ^ 1u, abortp)) {
        if (status) atomicCAS(status, ST_OK, ST_TIMEOUT_MMA);
        ok = false;
        break;
      }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t d_addr = tmem_d + (uint32_t)buf * ACC_COLS;
      for (int i = 0; i < sg.nkb; ++i) {
        if (!mbar_wait(smem_u32(&full_bar[s]), ph, abortp)) {
          if (status) atomicCAS(status, ST_OK, ST_TIMEOUT_MMA);
          ok = false;
          break;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t sW = tiles + s * SL::STAGE_BYTES;
        const uint64_t dA = make_smem_desc(sW + SL::W_BYTES);
#pragma unroll
        for (int k = 0; k < TILE_K / UMMA_K; ++k) {
#pragma unroll
          for (int w = 0; w < WM; ++w) {
            // advance 32 bytes (16 bf16) along K inside the swizzle row: +2 in 16-byte units
            const uint64_t dW = make_smem_desc(sW + w * W_STAGE_BYTES);
            umma_bf16(d_addr + (uint32_t)(w * BN), dW + (uint64_t)(2 * k), dA + (uint64_t)(2 * k), idesc,
                      (i > 0 || k > 0) ? 1u : 0u);
          }
        }
        umma_commit(smem_u32(&empty_bar[s]));  // stage reusable once these MMAs have read it
        if (++s == STAGES) {
          s = 0;
          ph ^= 1u;
        }
      }
      if (ok) umma_commit(smem_u32(&acc_full[buf]));
      u += sg.nkb;
    }
  } else if (warp >= 2) {
    // ---------------- epilogue: TMEM -> registers -> slab (warps 2..5) ----------------
    const int q = warp & 3;  // the TMEM lane quarter this warp may read
    int seg = 0;
    for (int u = u0; u < u1; ++seg) {
      const Segment sg = segment_at(u, u1, num_kb);
      const int buf = seg % ACC_BUFS;
      const bool have = mbar_wait(smem_u32(&acc_full[buf]), ((uint32_t)(seg / ACC_BUFS)) & 1u, abortp);
      if (!__all_sync(0xffffffffu, have)) {  // the whole warp must agree before the warp-collective loads
        if (lane == 0 && status) atomicCAS(status, ST_OK, ST_TIMEOUT_EPI);
        break;
      }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int nt = sg.tile / m_tiles, mt = sg.tile - nt * m_tiles;
      const int m0 = mt * BN;
      const int slab = (int)blockIdx.x - (sg.tile * num_kb) / upc;
#pragma unroll 1
      for (int w = 0; w < WM; ++w) {
        const int n = nt * TW + w * TILE_W + q * 32 + lane;
        float* out = part + (size_t)slab * split_stride + n;
        const uint32_t t_addr = tmem_d + ((uint32_t)(q * 32) << 16) + (uint32_t)buf * ACC_COLS + (uint32_t)(w * BN);
#pragma unroll 1
        for (int c = 0; c < BN; c += 16) {
          if (m0 + c >= M) break;
          uint32_t r[16];
          tmem_ld16(t_addr + (uint32_t)c, r);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
          if (n < N) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int m = m0 + c + j;
              if (m < M) out[(size_t)m * N] = __uint_as_float(r[j]);
            }
          }
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&acc_empty[buf]));
      u += sg.nkb;
    }
  }
  if (*abortp) drain_delay();  // gave up: let copies in flight land before shared memory is released
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(TMEM_COLS) : "memory");
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
  bool operator==(const MapKey& o) const {
    return base == o.base && batch == o.batch && rows == o.rows && cols == o.cols && box_rows == o.box_rows;
  }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    size_t h = std::hash<const void*>()(k.base);
    h ^= std::hash<uint64_t>()(k.rows * 1315423911ull + k.cols + k.batch * 2654435761ull) + 0x9e3779b97f4a7c15ull +
         (h << 6) + (h >> 2);
    return h ^ (k.box_rows * 2654435761u);
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
constexpr int max_stages(int bn, int wm) {
  const int fit = (227 * 1024 - 1024 - 512) / (int)(wm * W_STAGE_BYTES + bn * TILE_K * 2);
  return fit < MAX_STAGES ? fit : MAX_STAGES;
}

template <int BN, int WM>
cudaError_t launch_one(const Launch& L, const CUtensorMap& tmW, const CUtensorMap& tmA, float* part, int M, int N,
                       const GemmPlan& plan) {
  using SL = SmemLayout<BN, WM>;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(gemm_bf16_tcgen05_kernel<BN, WM>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)SL::total(max_stages(BN, WM)));
    if (e != cudaSuccess) return e;
    configured = true;
  }
  const int stages = plan.stages < 2 ? 2 : plan.stages > max_stages(BN, WM) ? max_stages(BN, WM) : plan.stages;
  cudaError_t e = launch_k(L, gemm_bf16_tcgen05_kernel<BN, WM>, dim3(plan.ctas), dim3(GEMM_THREADS), SL::total(stages), tmW,
                           tmA, part, M, N, plan.num_kb, plan.m_tiles, plan.total_units, plan.upc, (size_t)M * N, stages,
                           plan.w_tiled, L.d_status);
  L.count();
  return e != cudaSuccess ? e : cudaGetLastError();
}

int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
      n = v;
    else
      return 148;  // no device visible (host-only size queries): a B200's count
  }
  return n;
}

}  // namespace

bool get_tensor_map_2d(const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows, CUtensorMap* out) {
  return get_map(MapKey{base, 0, rows, cols, box_rows}, out);
}
bool get_tensor_map_3d(const void* base, uint64_t batch, uint64_t rows, uint64_t cols, uint32_t box_rows,
                       CUtensorMap* out) {
  return get_map(MapKey{base, batch, rows, cols, box_rows}, out);
}

Partials make_partials(const float* p, int M, int N, const GemmPlan& plan) {
  Partials out{p, (size_t)M * N, plan.S_max, N};
  if (plan.S_max > 1) {
    out.upc = plan.upc;
    out.num_kb = plan.num_kb;
    out.m_tiles = plan.m_tiles;
    out.BN = plan.BN;
    out.TW = plan.WM * TILE_W;
  } else {
    out.S = 1;
  }
  return out;
}

GemmPlan plan_gemm_bf16(int M, int N, int K, int force_ctas, int force_stages, int force_bn, bool whole_tiles,
                        int force_wm) {
  GemmPlan p;
  p.BN = M <= 32 ? 32 : M <= 64 ? 64 : M <= 128 ? 128 : 256;
  if (force_bn == 32 || force_bn == 64 || force_bn == 128 || force_bn == 256) p.BN = force_bn;
  p.num_kb = (K + TILE_K - 1) / TILE_K;
  const int wm_max = p.BN <= 64 ? 4 : p.BN == 128 ? 2 : 1;
  p.WM = (force_wm == 1 || force_wm == 2 || force_wm == 4) ? (force_wm <= wm_max ? force_wm : wm_max) : 1;
  p.m_tiles = (M + p.BN - 1) / p.BN;
  const int tw = p.WM * TILE_W;
  const long tiles = (long)p.m_tiles * ((N + tw - 1) / tw);
  const long total = tiles * p.num_kb;
  const int sms = sm_count();
  long upc;
  if (force_ctas > 0) {
    upc = (total + force_ctas - 1) / force_ctas;
  } else if (!whole_tiles && p.BN == 256 && tiles < 8L * sms) {
    // one CTA per SM anyway (the ring and both accumulators fill it): deal the
    // (tile, k-block) units evenly, whatever the tile count
    upc = (total + sms - 1) / sms;
    if (upc < 4) upc = 4;
  } else if (whole_tiles || tiles >= sms) {
    // enough tiles: whole tiles, one slab, no reduction; the tiles are dealt
    // evenly to at most two CTAs per SM
    const long per = (tiles + 2 * sms - 1) / (2 * sms);
    upc = per * p.num_kb;
  } else {
    // few tiles: split every tile's k range S ways so that about one CTA per
    // SM streams weights; S slabs per tile, added in order by the consumer
    long S = (sms + tiles - 1) / tiles;
    const long max_s = p.num_kb / 4 > 1 ? p.num_kb / 4 : 1;
    if (S > max_s) S = max_s;
    upc = (p.num_kb + S - 1) / S;
  }
  if (upc > total) upc = total;
  p.total_units = (int)total;
  p.upc = (int)upc;
  p.ctas = (int)((total + upc - 1) / upc);
  p.S_max = (upc % p.num_kb == 0) ? 1 : (p.num_kb - 1) / (int)upc + 2;
  // ring depth: two CTAs fit one SM when the split plan launches more CTAs than SMs
  const int deep = max_stages(p.BN, p.WM);
  p.stages = force_stages > 0 ? force_stages : (p.ctas > sms && deep > 4 ? 4 : deep);
  return p;
}

cudaError_t launch_gemm_bf16(const Launch& L, const void* A, const void* W, float* part, int M, int N, int K,
                             const GemmPlan& plan, const char** err) {
  static const char* e_shape = "bf16 GEMM needs K % 8 == 0 and 16-byte aligned operands";
  static const char* e_map = "cuTensorMapEncodeTiled failed or is unavailable";
  if (M <= 0 || N <= 0) return cudaSuccess;
  if (K <= 0 || (K & 7) || ((uintptr_t)A & 15) || ((uintptr_t)W & 15)) {
    if (err) *err = e_shape;
    return cudaErrorInvalidValue;
  }
  CUtensorMap tmW, tmA;
  const uint64_t n_tiles = (uint64_t)(N + TILE_W - 1) / TILE_W;
  const bool okW = plan.w_tiled ? get_tensor_map_2d(W, n_tiles * plan.num_kb * TILE_W, TILE_K, TILE_W, &tmW)
                                : get_tensor_map_2d(W, (uint64_t)N, (uint64_t)K, TILE_W, &tmW);
  if (!okW ||
      !get_tensor_map_2d(A, (uint64_t)M, (uint64_t)K, (uint32_t)plan.BN, &tmA)) {
    if (err) *err = e_map;
    return cudaErrorInvalidValue;
  }
  switch (plan.BN * 8 + plan.WM) {
    case 32 * 8 + 1: return launch_one<32, 1>(L, tmW, tmA, part, M, N, plan);
    case 32 * 8 + 2: return launch_one<32, 2>(L, tmW, tmA, part, M, N, plan);
    case 32 * 8 + 4: return launch_one<32, 4>(L, tmW, tmA, part, M, N, plan);
    case 64 * 8 + 1: return launch_one<64, 1>(L, tmW, tmA, part, M, N, plan);
    case 64 * 8 + 2: return launch_one<64, 2>(L, tmW, tmA, part, M, N, plan);
    case 64 * 8 + 4: return launch_one<64, 4>(L, tmW, tmA, part, M, N, plan);
    case 128 * 8 + 1: return launch_one<128, 1>(L, tmW, tmA, part, M, N, plan);
    case 128 * 8 + 2: return launch_one<128, 2>(L, tmW, tmA, part, M, N, plan);
    case 256 * 8 + 1: return launch_one<256, 1>(L, tmW, tmA, part, M, N, plan);
    default: break;
  }
  if (err) *err = "unsupported (activation tile, weight sub-tiles) combination";
  return cudaErrorInvalidValue;
}

}  // namespace dllm
