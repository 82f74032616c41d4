// Host-side launcher interfaces shared by the translation units of the library.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <atomic>

#include "common.cuh"

namespace dllm {

// One-time set-up per DEVICE of a process (cudaFuncSetAttribute and the like are per device): run(fn) calls
// fn() the first time it is reached with a given device current and again after a failure.  Devices beyond
// the 64 tracked ones are set up at every call.
struct DeviceOnce {
  std::atomic<uint64_t> done{0};
  template <class F>
  cudaError_t run(F&& fn) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const bool tracked = dev >= 0 && dev < 64;
    if (tracked && ((done.load(std::memory_order_acquire) >> dev) & 1ull)) return cudaSuccess;
    e = fn();
    if (e == cudaSuccess && tracked) done.fetch_or(1ull << dev, std::memory_order_release);
    return e;
  }
};
// Multiprocessors of the current device (148 on a B200; that value too when no device is visible, for the
// host-only size queries).
int sm_count();

struct Launch {
  cudaStream_t stream;
  int* d_status;        // device status word (may be null for kernel-level hooks)
  uint64_t* counter;    // host launch counter (may be null)
  bool pdl = false;     // launch with programmatic stream serialization (see launch_k)
  inline void count(int k = 1) const {
    if (counter) *counter += (uint64_t)k;
  }
};

// Launches `kernel`.  With L.pdl the launch carries the programmatic stream
// serialization attribute: the grid may become resident while its predecessor
// in the stream is still running, and everything it does before pdl_wait()
// (set-up, prefetch of weights, which no kernel writes) overlaps the
// predecessor's tail.  Every kernel of the library calls pdl_wait() before it
// touches memory another kernel writes or reads.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(const Launch& L, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                            Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = L.stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = L.pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
// The same for a kernel whose CTAs form clusters of `cluster` (grid dimensions are multiples of it).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_k_cluster(const Launch& L, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                    dim3 cluster, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = L.stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cluster.x;
  attr[0].val.clusterDim.y = cluster.y;
  attr[0].val.clusterDim.z = cluster.z;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = L.pdl ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Partial sums of one GEMM: slabs of [M, N] fp32, slab stride in floats.  With
// upc == 0 every element has S slabs; otherwise the tile that holds (row, col)
// has as many slabs as CTAs of the persistent GEMM touched it (see
// gemm_tcgen05.cu): units of a tile are [tile*num_kb, (tile+1)*num_kb) and CTA
// i owns units [i*upc, (i+1)*upc).
struct Partials {
  const float* p;
  size_t split_stride;
  int S;
  int N;  // row length
  int upc = 0, num_kb = 0, m_tiles = 1, BN = 256, TW = 128;
  __host__ __device__ inline int count(int row, int col) const {
    if (upc == 0) return S;
    const int tile = (col / TW) * m_tiles + row / BN;
    return ((tile + 1) * num_kb - 1) / upc - (tile * num_kb) / upc + 1;
  }
};

// ---------------- api.cu ----------------
// Message that dllm_last_error() returns on this thread.
void set_last_error(const char* msg);
// Device address, on the current device, of the status word the kernel-level entry points hand to their
// kernels (read and cleared by dllm_kernel_status); nullptr if it cannot be resolved.
int* kernel_status_word();

// ---------------- elementwise.cu ----------------
// out[c] = rmsnorm(x[c]) * gain for carried rows c0 <= c < c1 (out has the model dtype).
void launch_rmsnorm(const Launch& L, int dtype, const float* x, const float* gain, void* out, int d, float eps,
                    int c0, int c1);
// V-verify (Eq. 6) fused with the whole-V overwrite: for every response row
// sums the partials, rounds to the cache dtype, takes the cosine against the
// cached row, overwrites the cached row, writes sim[row].
// Lists of a response refresh without prompt refresh, where every response row is active in carried order:
// V-verify writes sel[c] = row within the sequence, act[c] = c, inv[c] = c for its row c.
struct IdentityLists {
  int32_t *sel = nullptr, *act = nullptr, *inv = nullptr;
};
void launch_vverify(const Launch& L, int dtype, Partials part, void* Vc_layer, float* sim, Geo g, int dkv,
                    int metric = 0, int write_v = 1, const IdentityLists* lists = nullptr);
// The same test on K (ablation of Sec. 4.3): slab sum of the K projection of all
// response rows, RoPE, score against the cached (post-RoPE) K, whole-K overwrite.
void launch_kverify(const Launch& L, int dtype, Partials part, void* Kc_layer, float* sim, const float* rope_tab, Geo g,
                    int Hkv, int hd, int metric);
// Bottom-k selection per sequence + active-row list.  mode 0: all R rows,
// 1: bottom-k by (round(sim*2^20), index), 2: forced list.
// inv (may be null): for every carried row its position in the active list, or -1.
cudaError_t launch_select(const Launch& L, const float* sim, const int32_t* forced, int mode, int ksel, int32_t* sel,
                          int sel_stride, int32_t* act, int32_t* inv, Geo g, int refresh_prompt);
// Selection, active list, inverse list and the gather of the active rows of u
// into ua in one launch (R <= 1024; sel rows have stride R).
void launch_select_gather(const Launch& L, int dtype, const float* sim, const int32_t* forced, int mode, int ksel,
                          int32_t* sel, int32_t* act, int32_t* inv, const void* u, void* ua, Geo g,
                          int refresh_prompt);
// x[c] = E[token(c)], u[c] = rmsnorm(x[c]) * gain for carried rows c0 <= c < c1.
void launch_embed_norm(const Launch& L, int dtype, const void* E, const int32_t* tokens, float* x, const float* gain,
                       void* u, Geo g, int c0, int c1, float eps);
// End of a layer for carried rows c0 <= c < c1: FFNOut rows of the active set
// (slabs in `part`, row = inv[c]) -> cache; x <- (x + AttnOut) + FFNOut from the
// caches; u = rmsnorm(x) * gain.  inv == nullptr: no active row.
void launch_tail(const Launch& L, int dtype, Partials part, const int32_t* inv, float* x, OutRows Ac_layer,
                 OutRows Fc_layer, const float* gain, void* u, Geo g, int c0, int c1, float eps);
void launch_gather_rows(const Launch& L, int dtype, const void* src, const int32_t* act, void* dst, int rows, int d);
// RoPE on Q and K of the active rows; Q -> qbuf [Ma, dq]; K -> K cache rows.
void launch_qk_rope(const Launch& L, int dtype, Partials part, const int32_t* act, const float* rope_tab, void* qbuf,
                    void* Kc_layer, Geo g, int Ma, int H, int Hkv, int hd);
// rows of `part` -> cache rows (model dtype).  act == nullptr: rows are the
// carried ids c_base + i; otherwise act[i].
void launch_scatter_rows(const Launch& L, int dtype, Partials part, const int32_t* act, int c_base, void* cache_layer,
                         Geo g, int rows, int width);
// AttnOut rows -> cache; h = x + AttnOut; hn = rmsnorm(h) * gain2 (model dtype).
void launch_oproj_epilogue(const Launch& L, int dtype, Partials part, const int32_t* act, const float* x,
                           const float* gain2, OutRows Ac_layer, void* hn, Geo g, int Ma, float eps);
// act[i][j] = silu(gate) * up from partials [Ma, 2m] (gate columns first).
// interleaved: the columns of `part` are blocks of 64 gate columns followed by the 64 up columns of the same
// FFN columns (the layout of the stacked weight when d_ffn % 64 == 0 in bf16); else all gate, then all up.
void launch_silu_mul(const Launch& L, int dtype, Partials part, void* out, int Ma, int m, int interleaved = 0);
// (x0, conf) per response row from fp32 logits; the mask id never wins.
void launch_argmax_conf(const Launch& L, const float* logits, int rows, int vocab, int mask_id, int32_t* x0,
                        float* conf, int R = 0, int blk_start = 0, int blk_len = 0);
// x0 / conf from the per-tile records of the LM head's estimate epilogue; row mapping as launch_argmax_conf
void launch_estimate_merge(const Launch& L, const float* records, int rows, int n_tiles, int32_t* x0, float* conf,
                           int R = 0, int blk_start = 0, int blk_len = 0);
// dst[b * len + i] = src[b * R + start + i], rows of d elements (d * element size a multiple of 16 bytes)
void launch_gather_block_rows(const Launch& L, int dtype, const void* src, void* dst, int B, int R, int start, int len,
                              int d);
void launch_remask(const Launch& L, int32_t* tokens, const int32_t* x0, const float* conf, Geo g, int mask_id,
                   int block_start, int block_len, int n_transfer);
void launch_reduce_partials(const Launch& L, Partials part, float* C, int M);
// cache <-> float32 conversion for the inspection hooks
void launch_convert_to_f32(const Launch& L, int dtype, const void* src, float* dst, size_t n);
void launch_convert_from_f32(const Launch& L, int dtype, const float* src, void* dst, size_t n);
void launch_mask_column(const Launch& L, float* logits, int rows, int vocab, int mask_id);
void launch_vverify_rows(const Launch& L, int dtype, const void* vnew, void* vcache, float* sim, int rows, int width);

// ---------------- gemm_simt.cu ----------------
// C[M,N] fp32 = A[M,K] * W[N,K]^T on the plain ALUs (fp32 mode; reference path for tests).
void launch_gemm_simt(const Launch& L, int dtype, const void* A, const void* W, float* C, int M, int N, int K);

// ---------------- gemm_tcgen05.cu ----------------
struct GemmPlan {
  int BN;           // activation tile rows (UMMA N)
  int stages;       // depth of the TMA ring
  int num_kb;       // k-blocks of 64
  int m_tiles;      // activation tiles
  int total_units;  // tiles * num_kb
  int upc;          // k-blocks per split
  int ctas;         // grid size
  int S_max;        // split-K factor: slabs per output element
  int pair = 0;     // 1: CTA pairs (cta_group::2) share the activation tile of BN rows
  int persistent = 0;  // 1: one CTA per SM walks through the tiles, epilogue under the next tile's main loop
};
// 0 = auto.  force_pair: 0 auto, 1 CTA pairs (BN 128 or 256, N a multiple of 256), -1 never.
// force_persistent: 0 auto, 1 the persistent kernel (unsplit plans with 256-row tiles only), -1 never.
GemmPlan plan_gemm_bf16(int M, int N, int K, int force_split = 0, int force_stages = 0, int force_bn = 0,
                        int force_pair = 0, int force_persistent = 0);
Partials make_partials(const float* p, int M, int N, const GemmPlan& plan);
// Returns cudaSuccess or the failing error.  part must hold S*M*N floats.
// act_out != nullptr (unsplit plan, W = gate / up rows interleaved in blocks of 64, N = 2 * m_ffn): instead of
// fp32 slabs the epilogue writes silu(gate) * up as bf16 [M, m_ffn].
// act_out == nullptr and m_ffn = -1 - mask_id (unsplit plan): instead of logits the epilogue writes, at `part`,
// one {max, sum exp, argmax, -} record per row and weight tile, [M][ceil(N / 128)] float4 (see launch_estimate_merge).
cudaError_t launch_gemm_bf16(const Launch& L, const void* A, const void* W, float* part, int M, int N, int K,
                             const GemmPlan& plan, const char** err, void* act_out = nullptr, int m_ffn = 0);

// Test hooks of the bounded device-side waits (see dllm_debug_* in the C ABI): the wait limit of each
// translation unit that waits on mbarriers (0 = the 2 s default), and the dropped activation load.
cudaError_t set_wait_limit_gemm_tcgen05(unsigned long long ns);
cudaError_t set_wait_limit_attention(unsigned long long ns);
cudaError_t set_wait_limit_attention_umma(unsigned long long ns);
cudaError_t set_debug_skip_act_load(int enable);

// ---------------- attention.cu ----------------
struct AttnPlan {
  int S;               // key-range splits
  int keys_per_split;  // multiple of the key tile
  size_t scratch_floats;
  int few_rg = 0;      // 64-row kernel family: 0 = the 64-row kernel, 1 / 2 = the few-rows kernel with 16 / 32 rows per CTA
  int row_tiles = 2;   // tcgen05 kernel: 128-row tiles per CTA (2, or 1 when two-tile CTAs would be too few)
};
AttnPlan plan_attention(int B, int a_seq, int n, int H, int Hkv);
// Plan of the 128-row tcgen05 kernel (attention_umma.cu) with at most scratch_floats floats for split partials.
AttnPlan plan_attention_umma(int B, int a_seq, int n, int H, int Hkv, size_t scratch_floats);
// Which of the two tensor-core kernels a bf16 shape runs on (more than 64 (query, head-of-group) rows per KV
// head: tcgen05), with the plan it takes given that much scratch.  launch_attention, the scratch-size query
// and the entry point with built-in scratch all decide through this one function.
struct AttnChoice {
  bool umma = false;
  AttnPlan plan{1, 0, 0, 0, 2};
};
AttnChoice choose_attention(int B, int a_seq, int n, int H, int Hkv, size_t scratch_floats);
extern int g_attn_force_splits;   // tuning override of both plans' split count (0 = automatic)
extern int g_attn_umma_min_rows;  // rows per KV head from which the tcgen05 kernel is taken
extern int g_attn_few_rows;       // 0: never the few-rows kernel
extern int g_attn_umma_row_tiles; // tcgen05 kernel: 0 = the plan chooses one or two 128-row tiles per CTA, 1 / 2 forced
// bf16 with head_dim 64 / 128 runs on the tensor cores (scratch holds the
// partials of split key ranges; without it one split is used); everything else
// on the plain-ALU kernel.  k_static / v_static: the first so many keys of every sequence hold K / V rows that
// no launch since the one BEFORE the launch preceding this attention has written (0 when unknown): the 64-row
// kernel requests tiles made of such rows ahead of its dependency wait.
cudaError_t launch_attention(const Launch& L, int dtype, const void* q, const void* Kc, const void* Vc, void* o, int B,
                             int a_seq, int n, int H, int Hkv, int hd, float* scratch, size_t scratch_floats,
                             bool force_simt, int k_static = 0, int v_static = 0);

// The same attention with 128-row tiles on tcgen05 (attention_umma.cu), for
// many active rows per KV head.  *S_out: key-range splits used (> 1: the caller
// merges the partials in `scratch` with the combine kernel).
cudaError_t launch_attention_umma(const Launch& L, const void* q, const void* Kc, const void* Vc, void* o, int B,
                                  int a_seq, int n, int H, int Hkv, int hd, float* scratch, size_t scratch_floats,
                                  int* S_out);

}  // namespace dllm
