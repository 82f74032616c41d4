/*
 * dllm.h -- C ABI of the B200 (sm_100a) library for one denoising step of a
 * bidirectional masked-diffusion transformer under adaptive feature caching.
 *
 * Vocabulary follows the paper: prompt c of length P, response y^(k) of length
 * R (n = P + R rows per sequence), denoising steps k = K..1, Prompt Cache C_p
 * and Response Cache C_r holding K, V, AttnOut, FFNOut per layer (Sec. 3.2),
 * refresh intervals K_p and K_r, adaptive update ratio rho (Sec. 3.2), V-verify
 * (Eq. 6), transition S with low-confidence remasking (Eq. 5, Sec. A.11).
 *
 * Conventions
 *   - Every call returns a dllm_status; nothing throws, aborts or traps.
 *     dllm_last_error(handle) returns a readable message for the last failure
 *     recorded on that live model or session handle; with NULL (or a pointer
 *     that is no live handle) it returns the last failure of any call on the
 *     calling thread, which is how failures of *_create calls, size queries
 *     and the kernel-level entry points are read.  The string stays valid
 *     until the same thread calls dllm_last_error again.
 *   - The caller owns all device memory: the weight blob, the cache blob and
 *     the workspace blob are device pointers the caller allocated (256-byte
 *     aligned) with at least the byte counts the size queries return, and must
 *     keep alive until the handle using them is destroyed.  The library frees
 *     only its own host-side handles (and the CUDA graphs it instantiates).
 *   - "h_" arguments are HOST pointers, "d_" arguments are DEVICE pointers.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Step
 *     and remask calls only enqueue work on it; they do not synchronise.
 *     Inspection calls (dllm_get_*, dllm_set_*) synchronise the stream they are
 *     given before copying.
 *   - All matrices are row-major.  Linear maps are stored [out, in] and applied
 *     as y = x W^T.  Storage type of weights and caches is the model's dtype;
 *     accumulation, softmax, norms, cosine and the residual stream are fp32.
 *   - Invalid arguments return DLLM_INVALID_ARG and have no side effect.
 */
#ifndef DLLM_H_
#define DLLM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  DLLM_OK = 0,
  DLLM_INVALID_ARG = 1,
  DLLM_BAD_STATE = 2,      /* e.g. a cached step before any full step */
  DLLM_UNSUPPORTED = 3,    /* shape outside what the kernels handle */
  DLLM_OUT_OF_MEMORY = 4,  /* host allocation failed */
  DLLM_CUDA_ERROR = 5,
  DLLM_TIMEOUT = 6         /* a bounded device-side wait gave up */
} dllm_status;

enum { DLLM_FP32 = 0, DLLM_BF16 = 1 };

/* Architecture of the mask predictor p_theta (Sec. 3.1): pre-norm transformer
 * with RMSNorm, rotary embedding (rotate-half pairing, absolute position in
 * [prompt; response]), bidirectional softmax attention with n_heads query heads
 * sharing n_kv_heads key/value heads, and a SwiGLU FFN of width d_ffn (three
 * matmuls, Sec. A.7).  No biases; embedding and LM head are separate. */
typedef struct {
  int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab, mask_id;
  float rms_eps, rope_theta;
  int32_t dtype; /* DLLM_FP32 or DLLM_BF16 */
} dllm_config;

/* How floor(rho * R) is rounded.  The paper writes floor (Sec. 3.2.2). */
typedef enum { DLLM_K_FLOOR = 0, DLLM_K_CEIL = 1 } dllm_kround;

enum { DLLM_CACHE_K = 0, DLLM_CACHE_V = 1, DLLM_CACHE_ATTN = 2, DLLM_CACHE_FFN = 3 };

/* Session flags.  DLLM_SESSION_COMPACT_CACHE: the AttnOut and FFNOut caches keep the
 * response rows only ([B, R, d_model] per layer instead of [B, n, d_model]).
 * Between prompt refreshes no step reads the prompt's AttnOut / FFNOut (the
 * prompt's residual stream is not carried then) and a prompt refresh recomputes
 * them before it uses them, so every output of every step is bit-identical to
 * the four-tensor layout; the cache shrinks by 2 * P * d_model elements per
 * layer and sequence (the memory overhead for long sequences that Sec. A.10
 * item (1) names; Sec. A.9 counts the four full tensors). */
enum { DLLM_SESSION_DEFAULT = 0, DLLM_SESSION_COMPACT_CACHE = 1 };

typedef struct dllm_model dllm_model;
typedef struct dllm_session dllm_session;

const char* dllm_last_error(const void* handle);

/* ---- sizes --------------------------------------------------------------- */
/* Bytes of the packed weight blob for this architecture. */
size_t dllm_weights_bytes(const dllm_config* cfg);
/* Bytes of the feature caches for B sequences of P + R rows: per layer
 * K, V [B, n, n_kv_heads*head_dim] and AttnOut, FFNOut [B, n, d_model] in the
 * model dtype -- exactly the four tensors per layer of Sec. A.9. */
size_t dllm_cache_bytes(const dllm_config* cfg, int B, int P, int R);
/* Bytes of scratch the step needs (residual stream, staging buffers, GEMM
 * partial sums, logits, selection state).  The GEMM part follows the launch
 * plans of the device that is current when the query is made: ask with the
 * session's device current. */
size_t dllm_workspace_bytes(const dllm_config* cfg, int B, int P, int R);
/* The same two sizes for a session created with `flags` (DLLM_SESSION_*; 0 for
 * an unknown flag).  With DLLM_SESSION_COMPACT_CACHE the cache holds, per layer,
 * K, V [B, n, Hkv*hd] and AttnOut, FFNOut [B, R, d_model]: Sec. A.9's count
 * minus 2 * P * d_model elements per layer and sequence. */
size_t dllm_cache_bytes_ex(const dllm_config* cfg, int B, int P, int R, int flags);
size_t dllm_workspace_bytes_ex(const dllm_config* cfg, int B, int P, int R, int flags);
/* Byte offset and element count of one named tensor inside the weight blob, so
 * a caller may fill the blob on the device.  Names: "embed", "lm_head" [vocab,
 * d_model]; "norm_f" [d_model]; "layers.<l>.{norm1,norm2}" [d_model];
 * "layers.<l>.wq" [H*hd, d]; ".wk", ".wv" [Hkv*hd, d]; ".wo" [d, H*hd];
 * ".wg", ".wu" [d_ffn, d]; ".wd" [d, d_ffn].  Norm gains are always fp32;
 * everything else has the model dtype. */
dllm_status dllm_tensor_offset(const dllm_config* cfg, const char* name, size_t* offset_bytes,
                               size_t* n_elements);
/* Row blocking of a tensor inside the blob.  *block_rows == 0: its n_elements
 * are contiguous from its offset.  Otherwise its rows are stored in blocks of
 * *block_rows consecutive rows, block b starting *block_stride_bytes * b after
 * the tensor's offset.  Only ".wg" and ".wu" of a bf16 model with
 * d_ffn % 64 == 0 are blocked (64 rows of W_gate, then the same 64 rows of
 * W_up, and so on), so that the projection that forms both halves of the
 * SwiGLU FFN (Sec. A.7 counts it as 2 of the 3 d x d_ffn products) can apply
 * silu(gate) * up to its own output tile.  dllm_model_set_tensor() places the
 * rows itself; only a caller that writes the blob directly needs this. */
dllm_status dllm_tensor_blocks(const dllm_config* cfg, const char* name, size_t* block_rows,
                               size_t* block_stride_bytes);

/* ---- model p_theta --------------------------------------------------------- */
/* Binds a model handle to a caller-owned device blob of dllm_weights_bytes(). */
dllm_status dllm_model_create(const dllm_config* cfg, void* d_weights, dllm_model** out);
/* Uploads one tensor from HOST float32 values (converted to the model dtype
 * with round-to-nearest-even).  n_elements must match the tensor. */
dllm_status dllm_model_set_tensor(dllm_model* m, const char* name, const float* h_src, size_t n_elements);
dllm_status dllm_model_destroy(dllm_model* m);

/* ---- session: tokens (c, y^(k)) and caches C_p, C_r ------------------------ */
/* d_cache: dllm_cache_bytes(); d_workspace: dllm_workspace_bytes().  Both are
 * zeroed asynchronously on `stream`. */
dllm_status dllm_session_create(dllm_model* m, int B, int P, int R, void* d_cache, void* d_workspace,
                                void* stream, dllm_session** out);
/* The same with session flags; d_cache / d_workspace sized by the _ex queries
 * with the same flags. */
dllm_status dllm_session_create_ex(dllm_model* m, int B, int P, int R, int flags, void* d_cache,
                                   void* d_workspace, void* stream, dllm_session** out);
dllm_status dllm_session_destroy(dllm_session* s);
/* tokens <- [prompt ; MASK x R] for every sequence (Eq. 2); caches become
 * invalid until the next full step.  h_prompt: int32 [B, P], ids in [0, vocab). */
dllm_status dllm_session_set_prompt(dllm_session* s, const int32_t* h_prompt, void* stream);

/* ---- the denoising step ---------------------------------------------------- */
/* Initialisation / full refresh (k = K, Sec. 3.2): all features of all n rows
 * are computed and written to C_p and C_r; leaves (x0, conf) for the response. */
dllm_status dllm_step_full(dllm_session* s, void* stream);
/* One step under the caching rule (Sec. 3.2 items (1)-(3), Sec. 3.2.2):
 *   refresh_prompt   != 0: prompt rows are recomputed and C_p rewritten;
 *   refresh_response != 0: all response rows are recomputed against the cached
 *                          prompt K/V and C_r rewritten;
 *   otherwise adaptive partial update: V is projected for all R response rows,
 *   s_j = cos(V_new[j], V_cached[j]) (Eq. 6), the k_sel = floor(rho*R) rows with
 *   the lowest s_j are selected per sequence and per layer (ties: lower
 *   round(s*2^20) first, then lower index), the whole response V cache is
 *   overwritten, and Q/K/attention/O-proj/FFN run only for the selected rows
 *   over the full cached K/V; their K, AttnOut, FFNOut rows are scattered back.
 *   rho in [0,1]; k_sel = 0 leaves all caches untouched.
 * Returns DLLM_BAD_STATE before the first full step. */
dllm_status dllm_step_cached(dllm_session* s, int refresh_prompt, int refresh_response, float rho,
                             dllm_kround kround, void* stream);
/* dllm_step_cached with one update ratio PER LAYER (the cross-layer allocation of
 * Sec. A.4, Table 11: e.g. 0.375 -> 0.125 front-heavy): h_rho host float
 * [n_layers], n_layers must equal the model's.  Layer l recomputes
 * floor(rho_l * R) rows; a layer with 0 rows is fully cached. */
dllm_status dllm_step_cached_layers(dllm_session* s, int refresh_prompt, int refresh_response, const float* h_rho,
                                    int n_layers, dllm_kround kround, void* stream);
/* Applies the schedule at step k of K (counting down): refresh everything at
 * k = K, the prompt when k mod Kp == 0, the response when k mod Kr == 0. */
dllm_status dllm_step_scheduled(dllm_session* s, int k, int K, int Kp, int Kr, float rho,
                                dllm_kround kround, void* stream);
/* The same step with the prediction (Eqs. 3-4: logits, greedy estimate, confidence)
 * restricted to response positions [block_start, block_start + block_len) of
 * every sequence: the only positions the transition of a semi-autoregressive
 * step reads (Eq. 5 over the current block).  The layers, the caches and the
 * hidden states are exactly those of dllm_step_scheduled; x0 / conf of the
 * block are bit-identical to it, those of other positions keep the values of
 * an earlier step (dllm_get_logits recomputes all rows from the hidden states
 * and is unaffected).  The LM head then streams its weights for block_len rows
 * instead of R and the estimate reads block_len rows of logits. */
dllm_status dllm_step_scheduled_block(dllm_session* s, int k, int K, int Kp, int Kr, float rho, dllm_kround kround,
                                      int block_start, int block_len, void* stream);
/* enable != 0: dllm_generate uses dllm_step_scheduled_block with the block each
 * step works on (the generated tokens are the same).  Default off. */
dllm_status dllm_session_predict_block_only(dllm_session* s, int enable);
/* Transition S with low-confidence remasking (Eq. 5): among the still masked
 * response positions in [block_start, block_start + block_len) the
 * min(n_transfer, #masked) positions with the highest confidence (ties: lowest
 * position) receive their greedy estimate x0; all others stay as they are.
 * Uses the (x0, conf) of the last step. */
dllm_status dllm_remask_low_confidence(dllm_session* s, int block_start, int block_len, int n_transfer,
                                       void* stream);
/* K steps k = K..1 of dllm_step_scheduled, each followed by the transition on
 * the block that step works on (blocks of block_len, K / (R / block_len) steps
 * per block, block_len / steps_per_block tokens per step).  R must be a
 * multiple of block_len and K a multiple of R / block_len. */
dllm_status dllm_generate(dllm_session* s, int K, int Kp, int Kr, float rho, dllm_kround kround,
                          int block_len, void* stream);
/* Waits for the stream and returns DLLM_TIMEOUT / DLLM_CUDA_ERROR if a kernel
 * recorded a problem in the session's device status word. */
dllm_status dllm_sync(dllm_session* s, void* stream);

/* ---- inspection and test hooks (host buffers owned by the caller) ---------- */
dllm_status dllm_get_tokens(dllm_session* s, int32_t* h_out /* [B, P+R] */, void* stream);
dllm_status dllm_set_response_tokens(dllm_session* s, const int32_t* h_tok /* [B, R] */, void* stream);
dllm_status dllm_get_hidden(dllm_session* s, float* h_out /* [B, R, d_model] residual before final norm */,
                            void* stream);
dllm_status dllm_get_pred(dllm_session* s, int32_t* h_x0 /* [B, R] */, float* h_conf /* [B, R] */, void* stream);
/* Recomputes and returns the logits of the last step's hidden state (mask id
 * column set to -inf).  Slow path for small vocabularies. */
dllm_status dllm_get_logits(dllm_session* s, float* h_out /* [B, R, vocab] */, void* stream);
/* Selection of the last step at one layer: h_idx int32 [B, k_sel] ascending
 * response-relative indices (k_sel = R on a response refresh), h_sim float
 * [B, R] (Eq. 6 values; only meaningful after an adaptive step).  Either
 * pointer may be NULL.  *k_sel_out receives k_sel. */
dllm_status dllm_get_selected(dllm_session* s, int layer, int32_t* h_idx, float* h_sim, int* k_sel_out,
                              void* stream);
/* One cache tensor of one layer as float32 [B, n, width] (width = Hkv*hd for K
 * and V, d_model for AttnOut and FFNOut).  In a DLLM_SESSION_COMPACT_CACHE
 * session AttnOut and FFNOut are [B, R, d_model]: the response rows only. */
dllm_status dllm_get_cache(dllm_session* s, int layer, int which, float* h_out, void* stream);
dllm_status dllm_set_cache(dllm_session* s, int layer, int which, const float* h_in, void* stream);
/* Replaces the V-verify choice of `layer` on adaptive steps by the given
 * response-relative indices (int32 [B, count], count must equal k_sel of the
 * steps that follow); count = -1 clears.  V-verify still runs and V is still
 * overwritten.  Lets a test tell a legal tie flip from an arithmetic fault. */
dllm_status dllm_force_selection(dllm_session* s, int layer, const int32_t* h_idx, int count);
/* The paper's ablations of the adaptive step (Sec. 4.3 selection strategies,
 * Sec. A.6 metric, Sec. A.5 V update).  Defaults: V-verify, cosine, whole-V
 * overwrite.
 *   strategy DLLM_SELECT_K_VERIFY: the test of Eq. 6 on the post-RoPE K; K of all
 *     response rows is projected and overwritten, V only at the selected rows.
 *   strategy DLLM_SELECT_RANDOM: no projection over all rows; the k_sel lowest of
 *     the scores given with dllm_set_scores are taken (same tie rule), V only at
 *     the selected rows.
 *   metric DLLM_METRIC_L2: score = -||new - cached||_2 instead of the cosine.
 *   v_selected_only != 0 (V-verify): only the selected tokens' V is written.
 * Response-refresh and full steps are unaffected. */
typedef enum { DLLM_SELECT_V_VERIFY = 0, DLLM_SELECT_K_VERIFY = 1, DLLM_SELECT_RANDOM = 2 } dllm_select_strategy;
typedef enum { DLLM_METRIC_COSINE = 0, DLLM_METRIC_L2 = 1 } dllm_metric;
dllm_status dllm_session_set_selection(dllm_session* s, int strategy, int metric, int v_selected_only);
/* Scores of one layer for DLLM_SELECT_RANDOM: host float [B, R]; they stay in
 * place until set again (any other strategy overwrites them with its own). */
dllm_status dllm_set_scores(dllm_session* s, int layer, const float* h_scores, void* stream);
/* Number of kernel launches the library has enqueued for this session. */
uint64_t dllm_launch_count(const dllm_session* s);
/* 1: replay each step kind from a CUDA graph captured on first use (default);
 * 0: launch kernels one by one. */
dllm_status dllm_session_use_graphs(dllm_session* s, int enable);

/* 1 (default): the kernels of a step are launched with programmatic stream
 * serialization, so each kernel's set-up (and the weight prefetch of the
 * projections) overlaps the tail of the kernel before it; 0: plain launches. */
dllm_status dllm_session_use_pdl(dllm_session* s, int enable);

/* Per-kernel timing.  While enabled, every kernel launch of a step is bracketed
 * by a pair of CUDA events on the caller's stream and no launch overlaps its
 * predecessor (no programmatic dependent launch).  With CUDA graphs on, the
 * event records are nodes of the step's graph, so no host latency falls between
 * a pair and its kernel; every step then ends with a stream synchronisation
 * that reads the pairs back.  _profile_read synchronises the device and
 * returns, for one class of launches, the summed event time, the number of
 * launches, and their algorithmic bytes and FLOPs: what the operation must
 * move and compute (a projection: W and A once in, one result out; attention:
 * K, V, Q in, O out; a row-wise kernel: its rows in and out), not the split-K
 * slabs or other scratch traffic.  DLLM_PROF_GEMM and DLLM_PROF_ATTENTION are
 * sums over their sub-classes.  Enabling or disabling discards earlier records. */
enum {
  DLLM_PROF_GEMM = 0,       /* all projections: the six classes GEMM_V .. GEMM_HEAD */
  DLLM_PROF_ATTENTION = 1,  /* both attention kernels, each with the merge of its key-range splits */
  DLLM_PROF_GEMM_V = 2,     /* V (K in the K-verify ablation) of all response rows; V of prompt / selected rows */
  DLLM_PROF_GEMM_QK = 3,    /* Q and K of the active rows */
  DLLM_PROF_GEMM_O = 4,
  DLLM_PROF_GEMM_GU = 5,    /* gate and up, with SwiGLU in the epilogue when unsplit */
  DLLM_PROF_GEMM_D = 6,
  DLLM_PROF_GEMM_HEAD = 7,  /* LM head with the estimate epilogue */
  DLLM_PROF_ATTN_MMA = 8,   /* up to 64 rows per KV head (mma.sync) */
  DLLM_PROF_ATTN_UMMA = 9,  /* more rows (tcgen05) */
  DLLM_PROF_VVERIFY = 10,   /* Eq. 6 + V overwrite */
  DLLM_PROF_SELECT = 11,    /* bottom-k selection + gather of the active rows */
  DLLM_PROF_ROPE = 12,      /* RoPE + K scatter */
  DLLM_PROF_OEPI = 13,      /* AttnOut scatter + residual + RMSNorm-2 */
  DLLM_PROF_SILU = 14,      /* SwiGLU after a split gate / up projection */
  DLLM_PROF_TAIL = 15,      /* FFNOut scatter + residual assembly + next RMSNorm */
  DLLM_PROF_EMBED = 16,     /* embedding + first RMSNorm */
  DLLM_PROF_ESTIMATE = 17,  /* merge of the estimate records (or argmax over logits) */
  DLLM_PROF_SCATTER = 18,   /* V rows of prompt / selected rows into the cache */
  DLLM_PROF_COUNT = 19
};
dllm_status dllm_session_profile(dllm_session* s, int enable);
dllm_status dllm_session_profile_read(dllm_session* s, int cls, double* total_ms, uint64_t* launches,
                                      double* algorithmic_bytes, double* flops);
/* Test hook: 1 runs the bf16 GEMMs and attention of the step on the plain-ALU
 * kernels instead of the tensor-core kernels (to localise a fault); default 0. */
dllm_status dllm_session_use_simt_gemm(dllm_session* s, int enable);

/* ---- kernel-level entry points (parity tests and micro-benchmarks) --------- */
/* The kernel-level calls below have no session, so the bounded waits of their
 * kernels (the same TMA / tcgen05 pipelines the step uses) report into one
 * status word inside the library image, per GPU (nothing is allocated for it).
 * dllm_kernel_status synchronises `stream`, reads the word of the current
 * device and clears it: DLLM_OK, or DLLM_TIMEOUT when a wait of any
 * kernel-level call since the last read gave up (its output is then
 * unspecified), as dllm_sync does for a session. */
dllm_status dllm_kernel_status(void* stream);
/* Test hooks for the DLLM_TIMEOUT path; they fault nothing and hang nothing.
 * dllm_debug_set_wait_limit_ns: the time after which a device-side wait of the
 * TMA / tcgen05 pipelines gives up (0 restores the default of 2 s), on the
 * current device, for every kernel launched afterwards.
 * dllm_debug_skip_one_load(1): from now on the first CTA of every launch of
 * the one-CTA bf16 GEMM kernel leaves out one activation-tile copy, so one of
 * its pipeline stages never completes, its waits run into the limit, the CTA
 * records the status code, skips its epilogue, frees its tensor memory and
 * returns normally; (0) switches that off.  Both calls synchronise the device. */
dllm_status dllm_debug_set_wait_limit_ns(uint64_t ns);
/* Tuning / test hook: kernel choice of the bf16 projections whose plan has no
 * split and 256-row activation tiles, for every later call in this process:
 * 0 automatic (the persistent kernel when there are more tiles than SMs), 1
 * always the persistent kernel, -1 always the one-tile-per-CTA kernel.  The two
 * kernels give bit-identical results. */
dllm_status dllm_debug_gemm_plan(int persistent);
/* Tuning hook: overrides, for every later call in this process, the number of
 * key-range splits the tensor-core attention kernels take (0 = automatic); if
 * tcgen05_min_rows > 0, the number of (query, head-of-group) rows per KV head
 * from which the 128-row tcgen05 kernel is taken instead of the 64-row mma.sync
 * kernel; and whether shapes with at most 32 rows per KV head and at least 1024
 * keys take the few-rows kernel (warps share the rows and split the key tiles;
 * 1, the default) or stay on the 64-row kernel (0); and whether a CTA of the
 * tcgen05 kernel takes one or two 128-row tiles (tcgen05_row_tiles 1 or 2;
 * 0 = the plan's choice).  Results stay within the attention tolerance; the
 * merge order changes with the plan. */
dllm_status dllm_debug_attention_plan(int splits, int tcgen05_min_rows, int few_rows_kernel, int tcgen05_row_tiles);
dllm_status dllm_debug_skip_one_load(int enable);
/* C[M,N] (fp32, row-major, DEVICE) = A[M,K] * W[N,K]^T with bf16 operands on
 * the tensor cores (tcgen05 + TMA).  d_partials is scratch of
 * dllm_gemm_bf16_scratch_bytes(M,N,K); partial sums over k ranges are reduced
 * in a fixed order.  K must be a multiple of 8 (16-byte rows). */
size_t dllm_gemm_bf16_scratch_bytes(int M, int N, int K);
dllm_status dllm_gemm_bf16(const void* d_A, const void* d_W, float* d_C, int M, int N, int K,
                           void* d_partials, void* stream);
/* The same product with an explicit launch plan, for tuning: act_tile = rows of
 * A per CTA (32, 64, 128 or 256; 192 with splits = 1 only: the persistent kernel),
 * splits = split-K factor, stages = depth of the TMA ring (clamped to what fits
 * shared memory); 0 picks the default of each.
 * d_partials (device, partials_bytes >= dllm_gemm_bf16_planned_scratch_bytes)
 * holds the split-K slabs; with splits > 1 and d_C NULL the slabs are left
 * unreduced there (what the step's fused consumers read). */
size_t dllm_gemm_bf16_planned_scratch_bytes(int M, int N, int K, int act_tile, int splits);
dllm_status dllm_gemm_bf16_planned(const void* d_A, const void* d_W, float* d_C, int M, int N, int K, int act_tile,
                                   int splits, int stages, void* d_partials, size_t partials_bytes, void* stream);
/* The same product computed by PAIRS of CTAs (tcgen05 cta_group::2): two CTAs
 * of a cluster share one activation tile of act_tile (128 or 256) rows, each
 * staging half of it, so the tile crosses the L2 -> SM fabric once per 256
 * weight rows.  N must be a multiple of 256.  splits / stages / scratch as for
 * dllm_gemm_bf16_planned; the result is bit-identical to the one-CTA kernel
 * with the same act_tile and splits. */
size_t dllm_gemm_bf16_pair_scratch_bytes(int M, int N, int K, int act_tile, int splits);
dllm_status dllm_gemm_bf16_pair(const void* d_A, const void* d_W, float* d_C, int M, int N, int K, int act_tile,
                                int splits, int stages, void* d_partials, size_t partials_bytes, void* stream);
/* Gate and up projection of the SwiGLU FFN with the activation applied in the
 * GEMM's epilogue (Sec. A.7's FFN: two of its three d x d_ffn products):
 * out[M, d_ffn] (bf16, DEVICE) = silu(A Wg^T) * (A Wu^T), A [M, K] bf16,
 * d_Wgu [2 * d_ffn, K] bf16 holding 64 rows of Wg, the same 64 rows of Wu, the
 * next 64 of Wg and so on (the blocked layout of dllm_tensor_blocks).  No
 * split-K, no scratch; products accumulate in fp32 and the result is rounded to
 * bf16 once.  d_ffn must be a multiple of 64, K of 8.  act_tile / stages as in
 * dllm_gemm_bf16_planned. */
dllm_status dllm_ffn_gate_up_bf16(const void* d_A, const void* d_Wgu, void* d_out, int M, int d_ffn, int K,
                                  int act_tile, int stages, void* stream);
/* The same product on the plain fp32 ALUs (operands fp32 or bf16): the GEMM of
 * the fp32 mode. */
dllm_status dllm_gemm_simt(const void* d_A, const void* d_W, float* d_C, int M, int N, int K, int dtype,
                           void* stream);
/* Non-causal attention of `a` query rows per sequence over n cached keys
 * (Sec. A.7, the 4 r n d term).  d_q [B*a, H*hd], d_k / d_v [B, n, Hkv*hd], d_o
 * [B*a, H*hd]; dtype as above.  bf16 with head_dim 64 or 128 runs on the tensor
 * cores -- up to 64 (query, head-of-group) rows per KV head on a 64-row
 * mma.sync kernel, more on a 128-row tcgen05 kernel -- and, when few rows are
 * active, splits the key range over CTAs; the partial results of the splits go
 * to d_scratch (device).  dllm_attention_scratch_bytes() is what the plan of
 * the kernel that shape runs on would like; with less the 64-row kernel does
 * not split and the 128-row kernel splits as far as the buffer allows. */
size_t dllm_attention_scratch_bytes(int B, int a, int n, int H, int Hkv, int hd, int dtype);
dllm_status dllm_attention(const void* d_q, const void* d_k, const void* d_v, void* d_o, int B, int a, int n,
                           int H, int Hkv, int hd, int dtype, void* d_scratch, size_t scratch_bytes, void* stream);
/* (No counterpart in the paper: an engineering variant of dllm_attention.)
 * The same bf16 tensor-core attention for callers that cannot create device
 * allocations where they call it -- a thread that only holds raw pointers
 * handed over by another component, a process with a fixed memory plan, or
 * a point where cudaMalloc's implicit device synchronisation is not acceptable.
 * The caller passes inputs and the output as for dllm_attention (bf16,
 * head_dim 64 or 128); the scratch for split key ranges is an 8 MiB array
 * inside the library image, which every GPU that loads the library holds until
 * the process exits.  The call allocates no device memory.
 *   - The first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress) with that device current; make that first call
 *     before any stream capture.
 *   - It runs exactly what dllm_attention runs when given
 *     dllm_attention_scratch_bytes() of scratch.  Shapes for which that is
 *     more than the 8 MiB return DLLM_UNSUPPORTED with a message; use
 *     dllm_attention with your own scratch for those.
 *   - All calls share the one array and it keeps the previous call's contents
 *     (nothing needs clearing: every value read is written first by the same
 *     call).  Two calls that overlap on the GPU -- different streams, or the
 *     same shape replayed concurrently -- race on it; serialise them. */
dllm_status dllm_attention_noalloc(const void* d_q, const void* d_k, const void* d_v, void* d_o, int B, int a,
                                   int n, int H, int Hkv, int hd, void* stream);
/* V-verify + selection alone (Eq. 6 and the bottom-k rule): d_vnew, d_vcache
 * [B, R, width] in `dtype`; writes d_sim float [B, R] and d_idx int32 [B, k]
 * ascending; overwrites d_vcache with d_vnew. */
dllm_status dllm_vverify_select(const void* d_vnew, void* d_vcache, float* d_sim, int32_t* d_idx, int B, int R,
                                int width, int k, int dtype, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* DLLM_H_ */
