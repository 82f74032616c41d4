// Host side of the C ABI: handles, blob layouts, argument checks, the step
// procedure (which kernels run for which active-row set), CUDA-graph replay and
// the inspection hooks.  No step of the method is computed here: the host only
// enqueues kernels.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <map>
#include <mutex>
#include <new>
#include <string>
#include <unordered_map>
#include <vector>

#include "../../include/dllm.h"
#include "internal.h"
#include "tma.cuh"

using namespace dllm;

namespace {

thread_local std::string g_err;  // last failure on this thread (what dllm_last_error(NULL) returns)

// Live handles and where each keeps its last message, so that dllm_last_error(handle) can tell a model from a
// session (and both from a stale pointer) without trusting the caller.
std::mutex g_handles_mu;
std::unordered_map<const void*, const std::string*> g_handles;
void register_handle(const void* h, const std::string* slot) {
  std::lock_guard<std::mutex> lock(g_handles_mu);
  g_handles[h] = slot;
}
void unregister_handle(const void* h) {
  std::lock_guard<std::mutex> lock(g_handles_mu);
  g_handles.erase(h);
}

size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

struct LayerOff {
  size_t norm1, wqkv, wo, norm2, wgu, wd;
};
struct WeightLayout {
  size_t embed, lm_head, norm_f, total;
  std::vector<LayerOff> layers;
};

size_t esize(const dllm_config& c) { return c.dtype == DLLM_BF16 ? 2 : 4; }

WeightLayout make_layout(const dllm_config& c) {
  WeightLayout w;
  const size_t es = esize(c), d = c.d_model, dq = (size_t)c.n_heads * c.head_dim,
               dkv = (size_t)c.n_kv_heads * c.head_dim, m = c.d_ffn, V = c.vocab;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes);
    return o;
  };
  w.embed = take(V * d * es);
  w.lm_head = take(V * d * es);
  w.norm_f = take(d * 4);
  w.layers.resize(c.n_layers);
  for (auto& l : w.layers) {
    l.norm1 = take(d * 4);
    l.wqkv = take((dq + 2 * dkv) * d * es);  // rows: W_q, then W_k, then W_v
    l.wo = take(d * dq * es);
    l.norm2 = take(d * 4);
    l.wgu = take(2 * m * d * es);            // rows: W_gate, then W_up (or blocks of 64 and 64: gu_interleaved)
    l.wd = take(d * m * es);
  }
  w.total = off;
  return w;
}

const char* check_config(const dllm_config* c) {
  if (!c) return "config is NULL";
  if (c->n_layers <= 0 || c->d_model <= 0 || c->n_heads <= 0 || c->n_kv_heads <= 0 || c->head_dim <= 0 ||
      c->d_ffn <= 0 || c->vocab <= 1)
    return "non-positive dimension";
  if (c->dtype != DLLM_FP32 && c->dtype != DLLM_BF16) return "dtype must be DLLM_FP32 or DLLM_BF16";
  if (c->n_heads % c->n_kv_heads) return "n_heads must be a multiple of n_kv_heads";
  if (c->mask_id < 0 || c->mask_id >= c->vocab) return "mask_id outside the vocabulary";
  if (!(c->rms_eps >= 0.f) || !(c->rope_theta > 0.f)) return "rms_eps / rope_theta out of range";
  return nullptr;
}
const char* check_supported(const dllm_config* c) {
  if (c->d_model % 8 || c->d_ffn % 8 || c->vocab % 8) return "d_model, d_ffn and vocab must be multiples of 8";
  if (c->head_dim % 32 || c->head_dim > 128) return "head_dim must be 32, 64, 96 or 128";
  return nullptr;
}

// bf16 models whose d_ffn is a multiple of 64 store W_gate and W_up row-interleaved in blocks of 64: gate row r
// is stacked row (r / 64) * 128 + r % 64 and up row r is 64 rows further, so that one 128-row GEMM tile holds
// both halves of 64 FFN columns and its epilogue can form silu(gate) * up (Sec. A.7's FFN, one pass less).
bool gu_interleaved(const dllm_config& c) { return c.dtype == DLLM_BF16 && c.d_ffn % 64 == 0; }

struct TensorRef {
  size_t off, n;
  bool f32;
  size_t block_rows = 0;    // 0: contiguous; else the rows come in blocks of this many ...
  size_t block_stride = 0;  // ... whose starts are this many bytes apart
};

bool find_tensor(const dllm_config& c, const WeightLayout& w, const char* name, TensorRef* out) {
  const size_t es = esize(c), d = c.d_model, dq = (size_t)c.n_heads * c.head_dim,
               dkv = (size_t)c.n_kv_heads * c.head_dim, m = c.d_ffn, V = c.vocab;
  if (!strcmp(name, "embed")) return *out = {w.embed, V * d, false}, true;
  if (!strcmp(name, "lm_head")) return *out = {w.lm_head, V * d, false}, true;
  if (!strcmp(name, "norm_f")) return *out = {w.norm_f, d, true}, true;
  int l = -1, pos = 0;
  if (sscanf(name, "layers.%d.%n", &l, &pos) < 1 || pos == 0 || l < 0 || l >= c.n_layers) return false;
  const char* t = name + pos;
  const LayerOff& L = w.layers[l];
  if (!strcmp(t, "norm1")) return *out = {L.norm1, d, true}, true;
  if (!strcmp(t, "norm2")) return *out = {L.norm2, d, true}, true;
  if (!strcmp(t, "wq")) return *out = {L.wqkv, dq * d, false}, true;
  if (!strcmp(t, "wk")) return *out = {L.wqkv + dq * d * es, dkv * d, false}, true;
  if (!strcmp(t, "wv")) return *out = {L.wqkv + (dq + dkv) * d * es, dkv * d, false}, true;
  if (!strcmp(t, "wo")) return *out = {L.wo, d * dq, false}, true;
  if (!strcmp(t, "wg") || !strcmp(t, "wu")) {
    const bool up = t[1] == 'u';
    if (gu_interleaved(c)) return *out = {L.wgu + (up ? 64 * d * es : 0), m * d, false, 64, 128 * d * es}, true;
    return *out = {L.wgu + (up ? m * d * es : 0), m * d, false}, true;
  }
  if (!strcmp(t, "wd")) return *out = {L.wd, d * m, false}, true;
  return false;
}

uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu)) return (uint16_t)((u >> 16) | 0x40);  // NaN
  u += 0x7FFFu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}

// workspace carve-up
struct Workspace {
  size_t status, tokens, x, u, ua, qbuf, obuf, hn, ffn, x0, conf, sim, sel, forced, act, inv, rope, pouts, attn,
      part, total;
  size_t part_floats, attn_floats;
};

Workspace make_workspace(const dllm_config& c, int B, int P, int R, int flags) {
  Workspace w;
  const size_t es = esize(c), d = c.d_model, dq = (size_t)c.n_heads * c.head_dim,
               dkv = (size_t)c.n_kv_heads * c.head_dim, m = c.d_ffn, V = c.vocab;
  const size_t n = (size_t)P + R, rows = (size_t)B * n, BR = (size_t)B * R, T = c.n_layers;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes);
    return o;
  };
  w.status = take(256);
  w.tokens = take(rows * 4);
  w.x = take(rows * d * 4);
  w.u = take(rows * d * es);
  w.ua = take(rows * d * es);
  w.qbuf = take(rows * dq * es);
  w.obuf = take(rows * dq * es);
  w.hn = take(rows * d * es);
  w.ffn = take(rows * m * es);
  w.x0 = take(BR * 4);
  w.conf = take(BR * 4);
  w.sim = take(T * BR * 4);
  w.sel = take(T * BR * 4);
  w.forced = take(T * BR * 4);
  w.act = take(rows * 4);
  w.inv = take(rows * 4);
  w.rope = take(n * c.head_dim * 4);
  // compact caches: AttnOut and FFNOut of the prompt rows live here for the length of one layer of a
  // prompt-refresh step ([B, P, d] each, carried order)
  w.pouts = take((flags & DLLM_SESSION_COMPACT_CACHE) ? 2 * (size_t)B * P * d * es : 0);
  // partial outputs of split key ranges: the 64-row kernel splits only while fewer CTAs than SMs exist, so
  // splits * (row, head) pairs < 2 * SMs * 64 (the few-rows kernel: 32 rows); the tcgen05 kernel, whose CTAs
  // hold up to 256 rows, lowers its split count to what this holds
  w.attn_floats = (size_t)2 * sm_count() * 256 * (128 + 2);
  w.attn = take(w.attn_floats * 4);
  // the GEMM slab buffer: the largest S * M * N over every projection a step of this session can launch (V and
  // the LM head over the B * R response rows, V over the prompt rows, and Q/K, O, gate/up, down and V over any
  // number of active rows), and the fp32 staging of the inspection hooks (a cache tensor, the logits)
  size_t mn = std::max(BR * V, rows * std::max(d, dkv));
  if (c.dtype == DLLM_BF16) {
    auto slabs = [&](size_t M, size_t N, size_t K) {
      if (M == 0) return;
      const GemmPlan p = plan_gemm_bf16((int)M, (int)N, (int)K);
      mn = std::max(mn, (size_t)p.S_max * M * N);
    };
    slabs(BR, dkv, d);
    slabs(BR, V, d);
    slabs((size_t)B * P, dkv, d);
    for (size_t Ma = 1; Ma <= rows; ++Ma) {
      slabs(Ma, dq + dkv, d);
      slabs(Ma, dkv, d);
      slabs(Ma, d, dq);
      slabs(Ma, 2 * m, d);
      slabs(Ma, d, m);
    }
  } else {
    mn = std::max(mn, rows * std::max(std::max(dq + dkv, d), 2 * m));
  }
  w.part_floats = mn + 4096;
  w.part = take(w.part_floats * 4);
  w.total = off;
  return w;
}

}  // namespace

struct dllm_model {
  dllm_config cfg;
  WeightLayout lay;
  uint8_t* d_w;
  std::string err;
};

struct StepKey {
  int rp, rr, ksel;
  uint64_t forced_sig;
  int variant = 0;
  uint64_t ksel_sig = 0;  // per-layer row counts (cross-layer allocation of rho)
  int head_start = 0, head_len = 0;  // prediction restricted to one block of the response (0 rows: all of it)
  int prof = 0;                      // graph with event-record nodes around the GEMM and attention launches
  bool operator<(const StepKey& o) const {
    if (prof != o.prof) return prof < o.prof;
    if (head_start != o.head_start) return head_start < o.head_start;
    if (head_len != o.head_len) return head_len < o.head_len;
    if (variant != o.variant) return variant < o.variant;
    if (ksel_sig != o.ksel_sig) return ksel_sig < o.ksel_sig;
    if (rp != o.rp) return rp < o.rp;
    if (rr != o.rr) return rr < o.rr;
    if (ksel != o.ksel) return ksel < o.ksel;
    return forced_sig < o.forced_sig;
  }
};

struct dllm_session {
  dllm_model* m;
  int B, P, R, n;
  uint8_t* d_cache;
  uint8_t* d_ws;
  Workspace ws;
  bool compact = false;    // AttnOut / FFNOut caches hold the response rows only
  bool valid = false;      // caches hold a full step
  bool have_pred = false;
  std::vector<int> last_ksel;  // per layer
  std::vector<int> forced_count;  // per layer, -1 = none
  uint64_t launches = 0;
  bool use_graphs = true;
  bool simt_gemm = false;
  bool use_pdl = true;
  int sel_strategy = DLLM_SELECT_V_VERIFY, sel_metric = DLLM_METRIC_COSINE, v_selected_only = 0;  // ablation variants
  bool block_head = false;     // dllm_generate predicts only the block each step works on
  struct GraphEntry {
    cudaGraphExec_t exec;
    uint64_t kernels;
    size_t rec0 = 0, rec1 = 0;  // profiling graphs: their event pairs are graph_prof[rec0 .. rec1)
  };
  std::map<StepKey, GraphEntry> graphs;
  std::string err;
  // profiling: event pairs around GEMM (class 0) and attention (class 1) launches.  Launched kernel by kernel the
  // pairs are recorded by the host; inside a captured step they become event-record nodes of the graph (no host
  // latency between a pair and its kernel), are re-recorded at every replay and read back after it.
  struct ProfRec {
    int cls;
    cudaEvent_t a, b;
    double bytes, flops;
  };
  struct ProfSum {
    double ms = 0, bytes = 0, flops = 0;
    uint64_t launches = 0;
  };
  bool profiling = false;
  std::vector<ProfRec> prof;        // recorded by the host, one pair per launch
  std::vector<ProfRec> graph_prof;  // owned by profiling graphs
  ProfSum prof_sum[DLLM_PROF_COUNT];  // read back from graph replays
  std::vector<cudaEvent_t> event_pool;
  cudaEvent_t take_event() {
    if (!event_pool.empty()) {
      cudaEvent_t e = event_pool.back();
      event_pool.pop_back();
      return e;
    }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
  }
  // inside a stream capture the record becomes an event-record node of the graph (a plain cudaEventRecord would
  // only express a dependency of the capture)
  static void record(cudaEvent_t e, cudaStream_t st) {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cs) == cudaSuccess && cs == cudaStreamCaptureStatusActive)
      cudaEventRecordWithFlags(e, st, cudaEventRecordExternal);
    else
      cudaEventRecord(e, st);
  }
  void prof_begin(int cls, double bytes, double flops, cudaStream_t st) {
    if (!profiling) return;
    ProfRec r{cls, take_event(), take_event(), bytes, flops};
    record(r.a, st);
    prof.push_back(r);
  }
  void prof_end(cudaStream_t st) {
    if (!profiling) return;
    record(prof.back().b, st);
  }

  void drop_graphs() {
    for (auto& kv : graphs) cudaGraphExecDestroy(kv.second.exec);
    graphs.clear();
    for (auto& r : graph_prof) {
      event_pool.push_back(r.a);
      event_pool.push_back(r.b);
    }
    graph_prof.clear();
  }

  size_t es() const { return esize(m->cfg); }
  size_t dkv() const { return (size_t)m->cfg.n_kv_heads * m->cfg.head_dim; }
  size_t dq() const { return (size_t)m->cfg.n_heads * m->cfg.head_dim; }
  size_t out_rows() const { return (size_t)B * (compact ? R : n); }  // rows of an AttnOut / FFNOut tensor
  size_t layer_bytes() const {
    return ((size_t)B * n * 2 * dkv() + out_rows() * 2 * (size_t)m->cfg.d_model) * es();
  }
  uint8_t* cache(int layer, int which) const {
    size_t off = (size_t)layer * layer_bytes();
    const size_t kv = (size_t)B * n * dkv() * es(), ad = out_rows() * (size_t)m->cfg.d_model * es();
    if (which >= 1) off += kv;
    if (which >= 2) off += kv;
    if (which >= 3) off += ad;
    return d_cache + off;
  }
  // AttnOut (which = DLLM_CACHE_ATTN) or FFNOut rows of a layer as the row-wise kernels address them
  OutRows outs(int layer, int which) const {
    uint8_t* prompt = d_ws + ws.pouts + (which == DLLM_CACHE_FFN ? (size_t)B * P * m->cfg.d_model * es() : 0);
    return OutRows{cache(layer, which), compact ? prompt : nullptr, compact ? 1 : 0};
  }
  template <typename T>
  T* wsp(size_t off) const {
    return reinterpret_cast<T*>(d_ws + off);
  }
  Geo geo() const { return Geo{B, P, R, n, m->cfg.d_model}; }
};

namespace {

dllm_status fail(std::string* slot, dllm_status st, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  g_err = buf;
  if (slot) *slot = buf;
  return st;
}

#define CU_TRY(slot, expr)                                                                          \
  do {                                                                                              \
    cudaError_t e_ = (expr);                                                                        \
    if (e_ != cudaSuccess) return fail(slot, DLLM_CUDA_ERROR, "%s: %s", #expr, cudaGetErrorString(e_)); \
  } while (0)

// Host -> device copy ordered on the caller's stream and complete on return.
// (A plain cudaMemcpy from pageable memory may return before its DMA has
// finished and is ordered only against the legacy stream, so kernels enqueued
// on a non-blocking stream afterwards could read stale data.)
cudaError_t h2d(void* dst, const void* src, size_t bytes, cudaStream_t st) {
  cudaError_t e = cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return e;
  return cudaStreamSynchronize(st);
}

int k_selected(float rho, int R, dllm_kround kr) {
  const double v = (double)rho * (double)R;
  long k = kr == DLLM_K_CEIL ? (long)ceil(v - 1e-6) : (long)floor(v + 1e-6);
  if (k < 0) k = 0;
  if (k > R) k = R;
  return (int)k;
}

// Event pair of one launch while the session is profiling (class, algorithmic bytes and FLOPs of the launch).
struct ProfScope {
  dllm_session* s;
  cudaStream_t st;
  ProfScope(dllm_session* s_, int cls, double bytes, double flops, cudaStream_t st_) : s(s_), st(st_) {
    s->prof_begin(cls, bytes, flops, st);
  }
  ~ProfScope() { s->prof_end(st); }
  ProfScope(const ProfScope&) = delete;
  ProfScope& operator=(const ProfScope&) = delete;
};

// One GEMM of the step: out = A[M,K] * W[N,K]^T as split-K partial slabs.
dllm_status run_gemm(dllm_session* s, const Launch& L, int cls, const void* A, const void* W, int M, int N, int K,
                     Partials* out, void* swiglu_out = nullptr, bool* fused = nullptr, int estimate_mask_id = -1) {
  float* part = s->wsp<float>(s->ws.part);
  if (fused) *fused = false;
  *out = Partials{part, (size_t)M * N, 1, N};
  if (M <= 0) return DLLM_OK;
  const double es = (double)s->es();
  const bool tensor = !(s->m->cfg.dtype == DLLM_FP32 || s->simt_gemm);
  const GemmPlan plan = tensor ? plan_gemm_bf16(M, N, K) : GemmPlan{};
  // an unsplit gate / up projection of an interleaved weight finishes SwiGLU in its own epilogue, and an unsplit
  // LM head writes per-tile estimate records instead of logits
  const bool estimate = tensor && !swiglu_out && estimate_mask_id >= 0 && plan.S_max == 1;
  const bool fuse = estimate || (tensor && swiglu_out && plan.S_max == 1 && gu_interleaved(s->m->cfg));
  // algorithmic traffic of one projection: the weight matrix and the activation rows once in, one result out
  // (fp32, or what the fused epilogue writes; split-K slabs are overhead, not counted)
  const double out_bytes = estimate ? (double)M * ((N + 127) / 128) * 16.0 : fuse ? (double)M * (N / 2) * 2.0 : (double)M * N * 4.0;
  s->prof_begin(cls, ((double)N * K + (double)M * K) * es + out_bytes, 2.0 * M * N * K, L.stream);
  struct End {
    dllm_session* s;
    cudaStream_t st;
    ~End() { s->prof_end(st); }
  } end_guard{s, L.stream};
  if (!tensor) {
    launch_gemm_simt(L, s->m->cfg.dtype, A, W, part, M, N, K);
    return DLLM_OK;
  }
  if ((size_t)plan.S_max * M * N > s->ws.part_floats)
    return fail(&s->err, DLLM_UNSUPPORTED, "GEMM %dx%dx%d with %d slabs exceeds the workspace", M, N, K, plan.S_max);
  const char* why = nullptr;
  cudaError_t e = launch_gemm_bf16(L, A, W, part, M, N, K, plan, &why, fuse && !estimate ? swiglu_out : nullptr,
                                   estimate ? -1 - estimate_mask_id : fuse ? N / 2 : 0);
  if (e != cudaSuccess)
    return fail(&s->err, DLLM_CUDA_ERROR, "bf16 GEMM %dx%dx%d: %s", M, N, K, why ? why : cudaGetErrorString(e));
  if (fused) *fused = fuse;
  *out = make_partials(part, M, N, plan);
  return DLLM_OK;
}

// Enqueue one denoising step.  Active rows per sequence: the prompt rows on a
// prompt refresh plus either all R response rows (response refresh) or the
// ksel rows V-verify picks.
dllm_status enqueue_step(dllm_session* s, int rp, int rr, const std::vector<int>& ksels, cudaStream_t stream,
                         int head_start = 0, int head_len = 0) {
  const dllm_config& c = s->m->cfg;
  const WeightLayout& wl = s->m->lay;
  const Geo g = s->geo();
  const int dt = c.dtype, d = c.d_model, H = c.n_heads, Hkv = c.n_kv_heads, hd = c.head_dim, m = c.d_ffn;
  const int dq = H * hd, dkv = Hkv * hd, BR = s->B * s->R, BP = s->B * s->P;
  const size_t es = s->es();
  Launch L{stream, s->wsp<int>(s->ws.status), &s->launches, s->use_pdl && !s->profiling};
  uint8_t* W = s->m->d_w;
  const int c0 = 0, c1 = BR + (rp ? BP : 0);
  float* x = s->wsp<float>(s->ws.x);
  uint8_t* u = s->wsp<uint8_t>(s->ws.u);
  int32_t* act = s->wsp<int32_t>(s->ws.act);
  dllm_status st;
  Partials part{nullptr, 0, 1, 0};

  int32_t* inv = s->wsp<int32_t>(s->ws.inv);
  {
    ProfScope ps(s, DLLM_PROF_EMBED, (double)(c1 - c0) * d * (4.0 + 2.0 * es), 4.0 * (c1 - c0) * d, stream);
    launch_embed_norm(L, dt, W + wl.embed, s->wsp<int32_t>(s->ws.tokens), x,
                      reinterpret_cast<const float*>(W + wl.layers[0].norm1), u, g, c0, c1, c.rms_eps);
  }
  for (int l = 0; l < c.n_layers; ++l) {
    const LayerOff& lo = wl.layers[l];
    uint8_t* Wq = W + lo.wqkv;
    uint8_t* Wv = Wq + (size_t)(dq + dkv) * d * es;
    float* sim = s->wsp<float>(s->ws.sim) + (size_t)l * BR;
    int32_t* sel = s->wsp<int32_t>(s->ws.sel) + (size_t)l * BR;
    const int32_t* forced = s->wsp<int32_t>(s->ws.forced) + (size_t)l * BR;

    const int ksel = ksels[l];  // rows of the response this layer recomputes
    const int a_seq = (rp ? s->P : 0) + ksel;
    const int Ma = s->B * a_seq;
    const bool adaptive = !rr && ksel > 0;
    const int mode = rr ? 0 : (s->forced_count[l] >= 0 ? 2 : 1);
    // A response refresh alone takes every response row in carried order: u itself is the operand of the
    // projections and V-verify writes the (identity) lists, so no selection or gather launch is needed.
    const bool identity = rr && !rp && Ma > 0;
    if (rr || (adaptive && s->sel_strategy == DLLM_SELECT_V_VERIFY)) {
      // V for ALL response rows (the 2 r d^2 term of Sec. A.7), V-verify, V overwrite
      if ((st = run_gemm(s, L, DLLM_PROF_GEMM_V, u, Wv, BR, dkv, d, &part)) != DLLM_OK) return st;
      const IdentityLists id{sel, act, inv};
      {  // the projection's fp32 result in, the cached row in, the row out
        ProfScope ps(s, DLLM_PROF_VVERIFY, (double)BR * dkv * (4.0 + 2.0 * es), 6.0 * BR * dkv, stream);
        launch_vverify(L, dt, part, s->cache(l, DLLM_CACHE_V), sim, g, dkv, rr ? 0 : s->sel_metric,
                       rr || !s->v_selected_only, identity ? &id : nullptr);
      }
    } else if (adaptive && s->sel_strategy == DLLM_SELECT_K_VERIFY) {
      // ablation: the same test on K; K of ALL response rows is projected, rotated and overwritten
      if ((st = run_gemm(s, L, DLLM_PROF_GEMM_V, u, Wq + (size_t)dq * d * es, BR, dkv, d, &part)) != DLLM_OK) return st;
      ProfScope ps(s, DLLM_PROF_VVERIFY, (double)BR * dkv * (4.0 + 2.0 * es), 10.0 * BR * dkv, stream);
      launch_kverify(L, dt, part, s->cache(l, DLLM_CACHE_K), sim, s->wsp<float>(s->ws.rope), g, Hkv, hd,
                     s->sel_metric);
    }  // random selection: the scores were set by dllm_set_scores
    // V of the active rows is still missing when the verify pass did not write it
    const bool v_for_active = adaptive && (s->sel_strategy != DLLM_SELECT_V_VERIFY || s->v_selected_only);
    if (rp) {
      if ((st = run_gemm(s, L, DLLM_PROF_GEMM_V, u + (size_t)BR * d * es, Wv, BP, dkv, d, &part)) != DLLM_OK) return st;
      ProfScope ps(s, DLLM_PROF_SCATTER, (double)BP * dkv * (4.0 + es), 0.0, stream);
      launch_scatter_rows(L, dt, part, nullptr, BR, s->cache(l, DLLM_CACHE_V), g, BP, dkv);
    }
    if (Ma > 0) {
      const uint8_t* ua = s->wsp<uint8_t>(s->ws.ua);
      if (identity) {
        ua = u;
      } else if (s->R <= 1024 && (long)Ma * s->R <= 64L * 1024) {
        // few active rows: every CTA of the gather repeats the selection rather than wait for a launch
        ProfScope ps(s, DLLM_PROF_SELECT, (double)Ma * d * 2.0 * es + (double)BR * 4.0, 0.0, stream);
        launch_select_gather(L, dt, sim, forced, mode, ksel, sel, act, inv, u, s->wsp<uint8_t>(s->ws.ua), g, rp);
      } else {
        ProfScope ps(s, DLLM_PROF_SELECT, (double)Ma * d * 2.0 * es + (double)BR * 4.0, 0.0, stream);
        cudaError_t se = launch_select(L, sim, forced, mode, ksel, sel, s->R, act, inv, g, rp);
        if (se != cudaSuccess) return fail(&s->err, DLLM_CUDA_ERROR, "selection: %s", cudaGetErrorString(se));
        launch_gather_rows(L, dt, u, act, s->wsp<uint8_t>(s->ws.ua), Ma, d);
      }
      if (v_for_active) {
        if ((st = run_gemm(s, L, DLLM_PROF_GEMM_V, ua, Wv, Ma, dkv, d, &part)) != DLLM_OK) return st;
        ProfScope ps(s, DLLM_PROF_SCATTER, (double)Ma * dkv * (4.0 + es), 0.0, stream);
        launch_scatter_rows(L, dt, part, act, 0, s->cache(l, DLLM_CACHE_V), g, Ma, dkv);
      }
      // Q and K of the active rows in one GEMM over the stacked [W_q; W_k]
      if ((st = run_gemm(s, L, DLLM_PROF_GEMM_QK, ua, Wq, Ma, dq + dkv, d, &part)) != DLLM_OK) return st;
      {
        ProfScope ps(s, DLLM_PROF_ROPE, (double)Ma * (dq + dkv) * (4.0 + es), 6.0 * Ma * (dq + dkv), stream);
        launch_qk_rope(L, dt, part, act, s->wsp<float>(s->ws.rope), s->wsp<uint8_t>(s->ws.qbuf),
                       s->cache(l, DLLM_CACHE_K), g, Ma, H, Hkv, hd);
      }
      // algorithmic traffic: K and V of every sequence once, Q in, O out (the merge of split key ranges runs
      // inside the same pair).  Class by the kernel the shape takes: 64-row mma.sync or 128-row tcgen05.
      const bool attn_tc = dt == DLLM_BF16 && !s->simt_gemm && (hd == 64 || hd == 128);
      s->prof_begin(attn_tc && a_seq * (H / Hkv) > 64 ? DLLM_PROF_ATTN_UMMA : DLLM_PROF_ATTN_MMA,
                    (2.0 * s->B * s->n * dkv + 2.0 * Ma * dq) * (double)es, 4.0 * Ma * (double)s->n * dq, stream);
      cudaError_t e = launch_attention(L, dt, s->wsp<uint8_t>(s->ws.qbuf), s->cache(l, DLLM_CACHE_K),
                                       s->cache(l, DLLM_CACHE_V), s->wsp<uint8_t>(s->ws.obuf), s->B, a_seq, s->n, H,
                                       Hkv, hd, s->wsp<float>(s->ws.attn), s->ws.attn_floats, s->simt_gemm,
                                       // the launch before attention is RoPE + K scatter (after the Q / K projection):
                                       // every V row of the layer and, unless the prompt is refreshed, the prompt's K
                                       // rows were written at least two launches earlier
                                       rp ? 0 : s->P, s->n);
      s->prof_end(stream);
      if (e != cudaSuccess) return fail(&s->err, DLLM_CUDA_ERROR, "attention: %s", cudaGetErrorString(e));
      if ((st = run_gemm(s, L, DLLM_PROF_GEMM_O, s->wsp<uint8_t>(s->ws.obuf), W + lo.wo, Ma, d, dq, &part)) != DLLM_OK)
        return st;
      {  // projection result and x in, AttnOut row and the normalised row out
        ProfScope ps(s, DLLM_PROF_OEPI, (double)Ma * d * (8.0 + 2.0 * es), 6.0 * Ma * d, stream);
        launch_oproj_epilogue(L, dt, part, act, x, reinterpret_cast<const float*>(W + lo.norm2),
                              s->outs(l, DLLM_CACHE_ATTN), s->wsp<uint8_t>(s->ws.hn), g, Ma, c.rms_eps);
      }
      bool fused = false;
      if ((st = run_gemm(s, L, DLLM_PROF_GEMM_GU, s->wsp<uint8_t>(s->ws.hn), W + lo.wgu, Ma, 2 * m, d, &part,
                         s->wsp<uint8_t>(s->ws.ffn), &fused)) != DLLM_OK)
        return st;
      if (!fused) {
        ProfScope ps(s, DLLM_PROF_SILU, (double)Ma * m * (8.0 + es), 8.0 * Ma * m, stream);
        launch_silu_mul(L, dt, part, s->wsp<uint8_t>(s->ws.ffn), Ma, m, gu_interleaved(c));
      }
      if ((st = run_gemm(s, L, DLLM_PROF_GEMM_D, s->wsp<uint8_t>(s->ws.ffn), W + lo.wd, Ma, d, m, &part)) != DLLM_OK)
        return st;
    }
    // FFNOut rows -> cache, residual assembly for all carried rows, next norm
    const float* gain_next = reinterpret_cast<const float*>(l + 1 < c.n_layers ? W + wl.layers[l + 1].norm1 : W + wl.norm_f);
    {  // x in and out, AttnOut and FFNOut rows in, the normalised row out; the FFN result of the active rows in and out
      ProfScope ps(s, DLLM_PROF_TAIL, (double)(c1 - c0) * d * (8.0 + 3.0 * es) + (double)Ma * d * (4.0 + es),
                   6.0 * (c1 - c0) * d, stream);
      launch_tail(L, dt, part, Ma > 0 ? inv : nullptr, x, s->outs(l, DLLM_CACHE_ATTN), s->outs(l, DLLM_CACHE_FFN),
                  gain_next, u, g, c0, c1, c.rms_eps);
    }
  }
  // prediction at the response rows (Eqs. 3-4); u holds the final norm.  With head_len > 0 only the rows of
  // one block are predicted: the transition of a semi-autoregressive step reads no others (Eq. 5).
  const uint8_t* head_in = u;
  int head_rows = BR;
  if (head_len > 0) {
    head_rows = s->B * head_len;
    if (s->B == 1) {
      head_in = u + (size_t)head_start * d * es;
    } else {
      launch_gather_block_rows(L, dt, u, s->wsp<uint8_t>(s->ws.ua), s->B, s->R, head_start, head_len, d);
      head_in = s->wsp<uint8_t>(s->ws.ua);
    }
  }
  bool est = false;
  if ((st = run_gemm(s, L, DLLM_PROF_GEMM_HEAD, head_in, W + wl.lm_head, head_rows, c.vocab, d, &part, nullptr, &est,
                     c.mask_id)) != DLLM_OK)
    return st;
  if (part.S != 1) return fail(&s->err, DLLM_UNSUPPORTED, "LM head GEMM must not be split");
  {
    ProfScope ps(s, DLLM_PROF_ESTIMATE,
                 est ? (double)head_rows * ((c.vocab + 127) / 128) * 16.0 : (double)head_rows * c.vocab * 4.0,
                 est ? 0.0 : 4.0 * head_rows * c.vocab, stream);
    if (est)  // the projection left one (max, sum exp, argmax) record per row and weight tile instead of logits
      launch_estimate_merge(L, part.p, head_rows, (c.vocab + 127) / 128, s->wsp<int32_t>(s->ws.x0),
                            s->wsp<float>(s->ws.conf), s->R, head_start, head_len);
    else
      launch_argmax_conf(L, part.p, head_rows, c.vocab, c.mask_id, s->wsp<int32_t>(s->ws.x0),
                         s->wsp<float>(s->ws.conf), s->R, head_start, head_len);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(&s->err, DLLM_CUDA_ERROR, "step launch: %s", cudaGetErrorString(e));
  return DLLM_OK;
}

uint64_t forced_signature(const dllm_session* s) {
  uint64_t h = 1469598103934665603ull;
  for (int fc : s->forced_count) h = (h ^ (uint64_t)(fc >= 0)) * 1099511628211ull;
  return h;
}

dllm_status run_step(dllm_session* s, int rp, int rr, const float* rhos, int n_rho, dllm_kround kr, void* stream_v,
                     int head_start = 0, int head_len = 0) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  const int T = s->m->cfg.n_layers;
  if (!rhos || (n_rho != 1 && n_rho != T)) return fail(&s->err, DLLM_INVALID_ARG, "one rho, or one per layer");
  for (int i = 0; i < n_rho; ++i)
    if (!(rhos[i] >= 0.f && rhos[i] <= 1.f)) return fail(&s->err, DLLM_INVALID_ARG, "rho must lie in [0, 1]");
  if (kr != DLLM_K_FLOOR && kr != DLLM_K_CEIL) return fail(&s->err, DLLM_INVALID_ARG, "bad kround");
  rp = rp != 0;
  rr = rr != 0;
  if (!s->valid && !(rp && rr)) return fail(&s->err, DLLM_BAD_STATE, "cached step before any full step");
  std::vector<int> ksels(T);
  bool uniform = true;
  uint64_t sig = 1469598103934665603ull;
  for (int l = 0; l < T; ++l) {
    ksels[l] = rr ? s->R : k_selected(rhos[n_rho == 1 ? 0 : l], s->R, kr);
    uniform = uniform && ksels[l] == ksels[0];
    sig = (sig ^ (uint64_t)ksels[l]) * 1099511628211ull;
  }
  if (!rr)
    for (int l = 0; l < T; ++l)
      if (s->forced_count[l] >= 0 && s->forced_count[l] != ksels[l])
        return fail(&s->err, DLLM_INVALID_ARG, "forced selection of layer %d has %d rows, step selects %d", l,
                    s->forced_count[l], ksels[l]);
  cudaStream_t stream = (cudaStream_t)stream_v;
  dllm_status st = DLLM_OK;
  const bool graph_ok = s->use_graphs && stream != nullptr && stream != cudaStreamLegacy;
  if (head_len < 0 || head_start < 0 || head_start + head_len > s->R)
    return fail(&s->err, DLLM_INVALID_ARG, "block [%d, %d) outside the response", head_start, head_start + head_len);
  if (head_len == s->R) head_start = head_len = 0;  // the whole response: the ordinary step
  if (!graph_ok) {
    st = enqueue_step(s, rp, rr, ksels, stream, head_start, head_len);
  } else {
    StepKey key{rp, rr, ksels[0], forced_signature(s), s->sel_strategy * 4 + s->sel_metric * 2 + s->v_selected_only,
                uniform ? 0 : sig, head_start, head_len, s->profiling ? 1 : 0};
    auto it = s->graphs.find(key);
    if (it == s->graphs.end()) {
      cudaGraph_t graph = nullptr;
      CU_TRY(&s->err, cudaStreamBeginCapture(stream, cudaStreamCaptureModeThreadLocal));
      const uint64_t before = s->launches;
      const size_t host_recs = s->prof.size();
      st = enqueue_step(s, rp, rr, ksels, stream, head_start, head_len);
      cudaError_t e = cudaStreamEndCapture(stream, &graph);
      // event pairs recorded during the capture belong to the graph
      const size_t rec0 = s->graph_prof.size();
      s->graph_prof.insert(s->graph_prof.end(), s->prof.begin() + host_recs, s->prof.end());
      s->prof.resize(host_recs);
      if (st != DLLM_OK) {
        if (graph) cudaGraphDestroy(graph);
        return st;
      }
      if (e != cudaSuccess) return fail(&s->err, DLLM_CUDA_ERROR, "graph capture: %s", cudaGetErrorString(e));
      cudaGraphExec_t exec = nullptr;
      e = cudaGraphInstantiate(&exec, graph, 0);
      cudaGraphDestroy(graph);
      if (e != cudaSuccess) return fail(&s->err, DLLM_CUDA_ERROR, "graph instantiate: %s", cudaGetErrorString(e));
      const uint64_t kernels = s->launches - before;
      s->launches = before;  // counted at every replay instead
      it = s->graphs.emplace(key, dllm_session::GraphEntry{exec, kernels, rec0, s->graph_prof.size()}).first;
    }
    CU_TRY(&s->err, cudaGraphLaunch(it->second.exec, stream));
    s->launches += it->second.kernels;
    if (s->profiling && it->second.rec1 > it->second.rec0) {
      CU_TRY(&s->err, cudaStreamSynchronize(stream));
      for (size_t i = it->second.rec0; i < it->second.rec1; ++i) {
        const dllm_session::ProfRec& r = s->graph_prof[i];
        float t = 0.f;
        CU_TRY(&s->err, cudaEventElapsedTime(&t, r.a, r.b));
        dllm_session::ProfSum& acc = s->prof_sum[r.cls];
        acc.ms += t;
        acc.bytes += r.bytes;
        acc.flops += r.flops;
        ++acc.launches;
      }
    }
  }
  if (st != DLLM_OK) return st;
  s->valid = true;
  s->have_pred = true;
  s->last_ksel = ksels;
  return DLLM_OK;
}

}  // namespace

namespace dllm {
void set_last_error(const char* msg) { g_err = msg ? msg : ""; }

// Status word of the kernel-level entry points (they have no session whose workspace could hold one): a
// file-scope device variable, one per GPU that loads the library, addressed through cudaGetSymbolAddress
// once per device -- nothing is allocated.
static __device__ int g_kernel_status = 0;
int* kernel_status_word() {
  static std::mutex mu;
  static int* per_device[64] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (!per_device[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_kernel_status) != cudaSuccess) return nullptr;
    per_device[dev] = static_cast<int*>(p);
  }
  return per_device[dev];
}
}  // namespace dllm

// =============================================================================
// extern "C" entry points
// =============================================================================
extern "C" {

const char* dllm_last_error(const void* handle) {
  if (handle) {
    std::lock_guard<std::mutex> lock(g_handles_mu);
    auto it = g_handles.find(handle);
    if (it != g_handles.end()) {
      // copied to a per-thread buffer: the handle's own string may change under another thread's call
      thread_local std::string copy;
      copy = *it->second;
      return copy.c_str();
    }
  }
  return g_err.c_str();  // NULL or unknown handle: the last failing call on this thread
}

size_t dllm_weights_bytes(const dllm_config* cfg) {
  if (check_config(cfg)) return 0;
  return make_layout(*cfg).total;
}

size_t dllm_cache_bytes_ex(const dllm_config* cfg, int B, int P, int R, int flags) {
  if (check_config(cfg) || B <= 0 || P <= 0 || R <= 0 || (flags & ~DLLM_SESSION_COMPACT_CACHE)) return 0;
  const size_t dkv = (size_t)cfg->n_kv_heads * cfg->head_dim, n = (size_t)P + R;
  const size_t out_rows = (flags & DLLM_SESSION_COMPACT_CACHE) ? (size_t)R : n;
  return (size_t)cfg->n_layers * B * (n * 2 * dkv + out_rows * 2 * (size_t)cfg->d_model) * esize(*cfg);
}
size_t dllm_cache_bytes(const dllm_config* cfg, int B, int P, int R) { return dllm_cache_bytes_ex(cfg, B, P, R, 0); }

size_t dllm_workspace_bytes_ex(const dllm_config* cfg, int B, int P, int R, int flags) {
  if (check_config(cfg) || B <= 0 || P <= 0 || R <= 0 || (flags & ~DLLM_SESSION_COMPACT_CACHE)) return 0;
  return make_workspace(*cfg, B, P, R, flags).total;
}
size_t dllm_workspace_bytes(const dllm_config* cfg, int B, int P, int R) {
  return dllm_workspace_bytes_ex(cfg, B, P, R, 0);
}

dllm_status dllm_tensor_offset(const dllm_config* cfg, const char* name, size_t* offset_bytes, size_t* n_elements) {
  const char* why = check_config(cfg);
  if (why) return fail(nullptr, DLLM_INVALID_ARG, "%s", why);
  if (!name) return fail(nullptr, DLLM_INVALID_ARG, "name is NULL");
  TensorRef t;
  if (!find_tensor(*cfg, make_layout(*cfg), name, &t)) return fail(nullptr, DLLM_INVALID_ARG, "unknown tensor '%s'", name);
  if (offset_bytes) *offset_bytes = t.off;
  if (n_elements) *n_elements = t.n;
  return DLLM_OK;
}

dllm_status dllm_tensor_blocks(const dllm_config* cfg, const char* name, size_t* block_rows, size_t* block_stride_bytes) {
  const char* why = check_config(cfg);
  if (why) return fail(nullptr, DLLM_INVALID_ARG, "%s", why);
  if (!name) return fail(nullptr, DLLM_INVALID_ARG, "name is NULL");
  TensorRef t;
  if (!find_tensor(*cfg, make_layout(*cfg), name, &t)) return fail(nullptr, DLLM_INVALID_ARG, "unknown tensor '%s'", name);
  if (block_rows) *block_rows = t.block_rows;
  if (block_stride_bytes) *block_stride_bytes = t.block_stride;
  return DLLM_OK;
}

dllm_status dllm_model_create(const dllm_config* cfg, void* d_weights, dllm_model** out) {
  if (!out) return fail(nullptr, DLLM_INVALID_ARG, "out is NULL");
  *out = nullptr;
  const char* why = check_config(cfg);
  if (why) return fail(nullptr, DLLM_INVALID_ARG, "%s", why);
  if ((why = check_supported(cfg))) return fail(nullptr, DLLM_UNSUPPORTED, "%s", why);
  if (!d_weights || ((uintptr_t)d_weights & 255)) return fail(nullptr, DLLM_INVALID_ARG, "d_weights must be a 256-byte aligned device pointer");
  dllm_model* m = new (std::nothrow) dllm_model();
  if (!m) return fail(nullptr, DLLM_OUT_OF_MEMORY, "host allocation failed");
  m->cfg = *cfg;
  m->lay = make_layout(*cfg);
  m->d_w = static_cast<uint8_t*>(d_weights);
  register_handle(m, &m->err);
  *out = m;
  return DLLM_OK;
}

dllm_status dllm_model_set_tensor(dllm_model* m, const char* name, const float* h_src, size_t n_elements) {
  if (!m) return fail(nullptr, DLLM_INVALID_ARG, "model is NULL");
  if (!name || !h_src) return fail(&m->err, DLLM_INVALID_ARG, "NULL argument");
  TensorRef t;
  if (!find_tensor(m->cfg, m->lay, name, &t)) return fail(&m->err, DLLM_INVALID_ARG, "unknown tensor '%s'", name);
  if (t.n != n_elements)
    return fail(&m->err, DLLM_INVALID_ARG, "tensor '%s' has %zu elements, got %zu", name, t.n, n_elements);
  if (t.f32 || m->cfg.dtype == DLLM_FP32) {
    CU_TRY(&m->err, cudaMemcpy(m->d_w + t.off, h_src, t.n * 4, cudaMemcpyHostToDevice));
    CU_TRY(&m->err, cudaDeviceSynchronize());  // DMA from pageable memory has landed on return
    return DLLM_OK;
  }
  std::vector<uint16_t> tmp;
  try {
    tmp.resize(t.n);
  } catch (...) {
    return fail(&m->err, DLLM_OUT_OF_MEMORY, "host allocation failed");
  }
  for (size_t i = 0; i < t.n; ++i) tmp[i] = f32_to_bf16_rne(h_src[i]);
  if (t.block_rows) {
    const size_t block_bytes = t.block_rows * (size_t)m->cfg.d_model * 2;
    CU_TRY(&m->err, cudaMemcpy2D(m->d_w + t.off, t.block_stride, tmp.data(), block_bytes, block_bytes,
                                 t.n * 2 / block_bytes, cudaMemcpyHostToDevice));
  } else {
    CU_TRY(&m->err, cudaMemcpy(m->d_w + t.off, tmp.data(), t.n * 2, cudaMemcpyHostToDevice));
  }
  CU_TRY(&m->err, cudaDeviceSynchronize());
  return DLLM_OK;
}

dllm_status dllm_model_destroy(dllm_model* m) {
  if (m) unregister_handle(m);
  delete m;
  return DLLM_OK;
}

dllm_status dllm_session_create(dllm_model* m, int B, int P, int R, void* d_cache, void* d_workspace, void* stream,
                                dllm_session** out) {
  return dllm_session_create_ex(m, B, P, R, 0, d_cache, d_workspace, stream, out);
}

dllm_status dllm_session_create_ex(dllm_model* m, int B, int P, int R, int flags, void* d_cache, void* d_workspace,
                                   void* stream, dllm_session** out) {
  if (!out) return fail(nullptr, DLLM_INVALID_ARG, "out is NULL");
  *out = nullptr;
  if (!m) return fail(nullptr, DLLM_INVALID_ARG, "model is NULL");
  if (flags & ~DLLM_SESSION_COMPACT_CACHE) return fail(&m->err, DLLM_INVALID_ARG, "unknown session flag");
  if (B <= 0 || P <= 0 || R <= 0) return fail(&m->err, DLLM_INVALID_ARG, "B, P and R must be positive");
  if (R > 8192) return fail(&m->err, DLLM_UNSUPPORTED, "R > 8192 is not supported by the selection kernel");
  if (!d_cache || !d_workspace || ((uintptr_t)d_cache & 255) || ((uintptr_t)d_workspace & 255))
    return fail(&m->err, DLLM_INVALID_ARG, "d_cache and d_workspace must be 256-byte aligned device pointers");
  dllm_session* s = new (std::nothrow) dllm_session();
  if (!s) return fail(&m->err, DLLM_OUT_OF_MEMORY, "host allocation failed");
  s->m = m;
  s->B = B;
  s->P = P;
  s->R = R;
  s->n = P + R;
  s->d_cache = static_cast<uint8_t*>(d_cache);
  s->d_ws = static_cast<uint8_t*>(d_workspace);
  s->compact = (flags & DLLM_SESSION_COMPACT_CACHE) != 0;
  s->ws = make_workspace(m->cfg, B, P, R, flags);
  s->forced_count.assign(m->cfg.n_layers, -1);
  cudaStream_t st = (cudaStream_t)stream;
  // rotary table: [pos][cos(hd/2) | sin(hd/2)], angle = pos * theta^(-2i/hd), evaluated in double
  const int hd = m->cfg.head_dim, half = hd / 2;
  std::vector<float> tab((size_t)s->n * hd);
  for (int pos = 0; pos < s->n; ++pos)
    for (int i = 0; i < half; ++i) {
      const double ang = (double)pos * pow((double)m->cfg.rope_theta, -2.0 * i / hd);
      tab[(size_t)pos * hd + i] = (float)cos(ang);
      tab[(size_t)pos * hd + half + i] = (float)sin(ang);
    }
  cudaError_t e = cudaMemsetAsync(d_cache, 0, dllm_cache_bytes_ex(&m->cfg, B, P, R, flags), st);
  // everything but the (large) GEMM slab is cleared; the slab is always written before it is read
  if (e == cudaSuccess) e = cudaMemsetAsync(d_workspace, 0, s->ws.part, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e == cudaSuccess) e = h2d(s->d_ws + s->ws.rope, tab.data(), tab.size() * 4, st);
  if (e != cudaSuccess) {
    delete s;
    return fail(&m->err, DLLM_CUDA_ERROR, "session setup: %s", cudaGetErrorString(e));
  }
  register_handle(s, &s->err);
  *out = s;
  return DLLM_OK;
}

dllm_status dllm_session_destroy(dllm_session* s) {
  if (!s) return DLLM_OK;
  unregister_handle(s);
  for (auto& kv : s->graphs) cudaGraphExecDestroy(kv.second.exec);
  for (auto& r : s->prof) {
    cudaEventDestroy(r.a);
    cudaEventDestroy(r.b);
  }
  for (auto e : s->event_pool) cudaEventDestroy(e);
  delete s;
  return DLLM_OK;
}

dllm_status dllm_session_set_prompt(dllm_session* s, const int32_t* h_prompt, void* stream) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  if (!h_prompt) return fail(&s->err, DLLM_INVALID_ARG, "h_prompt is NULL");
  const int V = s->m->cfg.vocab;
  std::vector<int32_t> tok((size_t)s->B * s->n);
  for (int b = 0; b < s->B; ++b) {
    for (int i = 0; i < s->P; ++i) {
      const int32_t t = h_prompt[(size_t)b * s->P + i];
      if (t < 0 || t >= V) return fail(&s->err, DLLM_INVALID_ARG, "prompt id %d outside [0, %d)", t, V);
      tok[(size_t)b * s->n + i] = t;
    }
    for (int j = 0; j < s->R; ++j) tok[(size_t)b * s->n + s->P + j] = s->m->cfg.mask_id;
  }
  cudaStream_t st = (cudaStream_t)stream;
  CU_TRY(&s->err, cudaStreamSynchronize(st));
  CU_TRY(&s->err, h2d(s->d_ws + s->ws.tokens, tok.data(), tok.size() * 4, st));
  s->valid = false;
  s->have_pred = false;
  return DLLM_OK;
}

dllm_status dllm_step_full(dllm_session* s, void* stream) {
  const float rho = 0.f;
  return run_step(s, 1, 1, &rho, 1, DLLM_K_FLOOR, stream);
}

dllm_status dllm_step_cached(dllm_session* s, int refresh_prompt, int refresh_response, float rho, dllm_kround kround,
                             void* stream) {
  return run_step(s, refresh_prompt, refresh_response, &rho, 1, kround, stream);
}

dllm_status dllm_step_cached_layers(dllm_session* s, int refresh_prompt, int refresh_response, const float* h_rho,
                                    int n_layers, dllm_kround kround, void* stream) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  if (n_layers != s->m->cfg.n_layers) return fail(&s->err, DLLM_INVALID_ARG, "one rho per layer expected");
  return run_step(s, refresh_prompt, refresh_response, h_rho, n_layers, kround, stream);
}

dllm_status dllm_step_scheduled(dllm_session* s, int k, int K, int Kp, int Kr, float rho, dllm_kround kround,
                                void* stream) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  if (K <= 0 || k <= 0 || k > K || Kp <= 0 || Kr <= 0)
    return fail(&s->err, DLLM_INVALID_ARG, "need 1 <= k <= K and positive K_p, K_r");
  const int rp = (k == K) || (k % Kp == 0), rr = (k == K) || (k % Kr == 0);
  return run_step(s, rp, rr, &rho, 1, kround, stream);
}

dllm_status dllm_step_scheduled_block(dllm_session* s, int k, int K, int Kp, int Kr, float rho, dllm_kround kround,
                                      int block_start, int block_len, void* stream) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  if (K <= 0 || k <= 0 || k > K || Kp <= 0 || Kr <= 0)
    return fail(&s->err, DLLM_INVALID_ARG, "need 1 <= k <= K and positive K_p, K_r");
  if (block_len <= 0) return fail(&s->err, DLLM_INVALID_ARG, "block_len must be positive");
  const int rp = (k == K) || (k % Kp == 0), rr = (k == K) || (k % Kr == 0);
  return run_step(s, rp, rr, &rho, 1, kround, stream, block_start, block_len);
}

dllm_status dllm_session_predict_block_only(dllm_session* s, int enable) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  s->block_head = enable != 0;
  return DLLM_OK;
}

dllm_status dllm_remask_low_confidence(dllm_session* s, int block_start, int block_len, int n_transfer, void* stream) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  if (block_start < 0 || block_len <= 0 || block_start + block_len > s->R || n_transfer < 0)
    return fail(&s->err, DLLM_INVALID_ARG, "block [%d, %d) outside the response or n_transfer < 0", block_start,
                block_start + block_len);
  if (block_len > 4096) return fail(&s->err, DLLM_UNSUPPORTED, "block_len > 4096");
  if (!s->have_pred) return fail(&s->err, DLLM_BAD_STATE, "no prediction yet: run a step first");
  Launch L{(cudaStream_t)stream, s->wsp<int>(s->ws.status), &s->launches};
  launch_remask(L, s->wsp<int32_t>(s->ws.tokens), s->wsp<int32_t>(s->ws.x0), s->wsp<float>(s->ws.conf), s->geo(),
                s->m->cfg.mask_id, block_start, block_len, n_transfer);
  CU_TRY(&s->err, cudaGetLastError());
  return DLLM_OK;
}

dllm_status dllm_generate(dllm_session* s, int K, int Kp, int Kr, float rho, dllm_kround kround, int block_len,
                          void* stream) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  if (K <= 0 || Kp <= 0 || Kr <= 0 || block_len <= 0 || s->R % block_len)
    return fail(&s->err, DLLM_INVALID_ARG, "need positive K, K_p, K_r and block_len dividing R");
  const int blocks = s->R / block_len;
  if (K % blocks) return fail(&s->err, DLLM_INVALID_ARG, "K must be a multiple of the number of blocks");
  const int spb = K / blocks;
  for (int k = K; k >= 1; --k) {
    const int t = K - k, blk = std::min(t / spb, blocks - 1), i = t - blk * spb;
    dllm_status st = s->block_head
                         ? dllm_step_scheduled_block(s, k, K, Kp, Kr, rho, kround, blk * block_len, block_len, stream)
                         : dllm_step_scheduled(s, k, K, Kp, Kr, rho, kround, stream);
    if (st != DLLM_OK) return st;
    const int n_transfer = block_len / spb + (i < block_len % spb ? 1 : 0);
    st = dllm_remask_low_confidence(s, blk * block_len, block_len, n_transfer, stream);
    if (st != DLLM_OK) return st;
  }
  return DLLM_OK;
}

// Reads and clears a device status word after the stream has drained.
static dllm_status read_status_word(std::string* slot, int* d_word, cudaStream_t stream) {
  CU_TRY(slot, cudaStreamSynchronize(stream));
  int code = 0;
  CU_TRY(slot, cudaMemcpy(&code, d_word, 4, cudaMemcpyDeviceToHost));
  if (code == 0) return DLLM_OK;
  cudaMemsetAsync(d_word, 0, 4, stream);
  cudaStreamSynchronize(stream);
  if (code >= 100 && code < 200) return fail(slot, DLLM_TIMEOUT, "a device-side wait gave up (code %d)", code);
  return fail(slot, DLLM_CUDA_ERROR, "device status %d", code);
}

dllm_status dllm_sync(dllm_session* s, void* stream) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  const dllm_status st = read_status_word(&s->err, s->wsp<int>(s->ws.status), (cudaStream_t)stream);
  // host-recorded event pairs of a profiled run have completed: fold them into the sums and reuse the events
  for (auto& r : s->prof) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, r.a, r.b) == cudaSuccess) {
      dllm_session::ProfSum& acc = s->prof_sum[r.cls];
      acc.ms += t;
      acc.bytes += r.bytes;
      acc.flops += r.flops;
      ++acc.launches;
    }
    s->event_pool.push_back(r.a);
    s->event_pool.push_back(r.b);
  }
  s->prof.clear();
  return st;
}

dllm_status dllm_kernel_status(void* stream) {
  int* w = kernel_status_word();
  if (!w) return fail(nullptr, DLLM_CUDA_ERROR, "no status word on this device");
  return read_status_word(nullptr, w, (cudaStream_t)stream);
}

dllm_status dllm_debug_set_wait_limit_ns(uint64_t ns) {
  CU_TRY(nullptr, cudaDeviceSynchronize());
  CU_TRY(nullptr, set_wait_limit_gemm_tcgen05(ns));
  CU_TRY(nullptr, set_wait_limit_attention(ns));
  CU_TRY(nullptr, set_wait_limit_attention_umma(ns));
  CU_TRY(nullptr, cudaDeviceSynchronize());
  return DLLM_OK;
}

dllm_status dllm_debug_skip_one_load(int enable) {
  CU_TRY(nullptr, cudaDeviceSynchronize());
  CU_TRY(nullptr, set_debug_skip_act_load(enable));
  CU_TRY(nullptr, cudaDeviceSynchronize());
  return DLLM_OK;
}

dllm_status dllm_get_tokens(dllm_session* s, int32_t* h_out, void* stream) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  if (!h_out) return fail(&s->err, DLLM_INVALID_ARG, "h_out is NULL");
  CU_TRY(&s->err, cudaStreamSynchronize((cudaStream_t)stream));
  CU_TRY(&s->err, cudaMemcpy(h_out, s->d_ws + s->ws.tokens, (size_t)s->B * s->n * 4, cudaMemcpyDeviceToHost));
  return DLLM_OK;
}

dllm_status dllm_set_response_tokens(dllm_session* s, const int32_t* h_tok, void* stream) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  if (!h_tok) return fail(&s->err, DLLM_INVALID_ARG, "h_tok is NULL");
  for (size_t i = 0; i < (size_t)s->B * s->R; ++i)
    if (h_tok[i] < 0 || h_tok[i] >= s->m->cfg.vocab) return fail(&s->err, DLLM_INVALID_ARG, "token id out of range");
  CU_TRY(&s->err, cudaStreamSynchronize((cudaStream_t)stream));
  CU_TRY(&s->err, cudaMemcpy2DAsync(s->d_ws + s->ws.tokens + (size_t)s->P * 4, (size_t)s->n * 4, h_tok,
                                    (size_t)s->R * 4, (size_t)s->R * 4, s->B, cudaMemcpyHostToDevice,
                                    (cudaStream_t)stream));
  CU_TRY(&s->err, cudaStreamSynchronize((cudaStream_t)stream));
  return DLLM_OK;
}

dllm_status dllm_get_hidden(dllm_session* s, float* h_out, void* stream) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  if (!h_out) return fail(&s->err, DLLM_INVALID_ARG, "h_out is NULL");
  if (!s->have_pred) return fail(&s->err, DLLM_BAD_STATE, "no step has run");
  CU_TRY(&s->err, cudaStreamSynchronize((cudaStream_t)stream));
  // response rows come first in the residual stream
  CU_TRY(&s->err, cudaMemcpy(h_out, s->d_ws + s->ws.x, (size_t)s->B * s->R * s->m->cfg.d_model * 4,
                             cudaMemcpyDeviceToHost));
  return DLLM_OK;
}

dllm_status dllm_get_pred(dllm_session* s, int32_t* h_x0, float* h_conf, void* stream) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  if (!s->have_pred) return fail(&s->err, DLLM_BAD_STATE, "no step has run");
  CU_TRY(&s->err, cudaStreamSynchronize((cudaStream_t)stream));
  const size_t BR = (size_t)s->B * s->R;
  if (h_x0) CU_TRY(&s->err, cudaMemcpy(h_x0, s->d_ws + s->ws.x0, BR * 4, cudaMemcpyDeviceToHost));
  if (h_conf) CU_TRY(&s->err, cudaMemcpy(h_conf, s->d_ws + s->ws.conf, BR * 4, cudaMemcpyDeviceToHost));
  return DLLM_OK;
}

dllm_status dllm_get_logits(dllm_session* s, float* h_out, void* stream) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  if (!h_out) return fail(&s->err, DLLM_INVALID_ARG, "h_out is NULL");
  if (!s->have_pred) return fail(&s->err, DLLM_BAD_STATE, "no step has run");
  const dllm_config& c = s->m->cfg;
  cudaStream_t st = (cudaStream_t)stream;
  Launch L{st, s->wsp<int>(s->ws.status), &s->launches};
  const int BR = s->B * s->R;
  launch_rmsnorm(L, c.dtype, s->wsp<float>(s->ws.x), reinterpret_cast<const float*>(s->m->d_w + s->m->lay.norm_f),
                 s->wsp<uint8_t>(s->ws.u), c.d_model, c.rms_eps, 0, BR);
  Partials part{nullptr, 0, 1, 0};
  dllm_status r = run_gemm(s, L, DLLM_PROF_GEMM_HEAD, s->wsp<uint8_t>(s->ws.u), s->m->d_w + s->m->lay.lm_head, BR,
                           c.vocab, c.d_model, &part);
  if (r != DLLM_OK) return r;
  launch_mask_column(L, s->wsp<float>(s->ws.part), BR, c.vocab, c.mask_id);
  CU_TRY(&s->err, cudaStreamSynchronize(st));
  CU_TRY(&s->err, cudaMemcpy(h_out, s->d_ws + s->ws.part, (size_t)BR * c.vocab * 4, cudaMemcpyDeviceToHost));
  return DLLM_OK;
}

dllm_status dllm_get_selected(dllm_session* s, int layer, int32_t* h_idx, float* h_sim, int* k_sel_out, void* stream) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  if (layer < 0 || layer >= s->m->cfg.n_layers) return fail(&s->err, DLLM_INVALID_ARG, "layer out of range");
  if (!s->have_pred) return fail(&s->err, DLLM_BAD_STATE, "no step has run");
  CU_TRY(&s->err, cudaStreamSynchronize((cudaStream_t)stream));
  const size_t BR = (size_t)s->B * s->R;
  const int k_l = layer < (int)s->last_ksel.size() ? s->last_ksel[layer] : 0;
  if (k_sel_out) *k_sel_out = k_l;
  if (h_idx && k_l > 0)
    CU_TRY(&s->err, cudaMemcpy2D(h_idx, (size_t)k_l * 4, s->d_ws + s->ws.sel + (size_t)layer * BR * 4,
                                 (size_t)s->R * 4, (size_t)k_l * 4, s->B, cudaMemcpyDeviceToHost));
  if (h_sim)
    CU_TRY(&s->err, cudaMemcpy(h_sim, s->d_ws + s->ws.sim + (size_t)layer * BR * 4, BR * 4, cudaMemcpyDeviceToHost));
  return DLLM_OK;
}

static dllm_status cache_args(dllm_session* s, int layer, int which, const void* p, size_t* n_elems) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  if (!p) return fail(&s->err, DLLM_INVALID_ARG, "host buffer is NULL");
  if (layer < 0 || layer >= s->m->cfg.n_layers) return fail(&s->err, DLLM_INVALID_ARG, "layer out of range");
  if (which < DLLM_CACHE_K || which > DLLM_CACHE_FFN) return fail(&s->err, DLLM_INVALID_ARG, "bad cache id");
  *n_elems = which <= DLLM_CACHE_V ? (size_t)s->B * s->n * s->dkv() : s->out_rows() * (size_t)s->m->cfg.d_model;
  return DLLM_OK;
}

dllm_status dllm_get_cache(dllm_session* s, int layer, int which, float* h_out, void* stream) {
  size_t n;
  dllm_status r = cache_args(s, layer, which, h_out, &n);
  if (r != DLLM_OK) return r;
  cudaStream_t st = (cudaStream_t)stream;
  Launch L{st, nullptr, &s->launches};
  launch_convert_to_f32(L, s->m->cfg.dtype, s->cache(layer, which), s->wsp<float>(s->ws.part), n);
  CU_TRY(&s->err, cudaStreamSynchronize(st));
  CU_TRY(&s->err, cudaMemcpy(h_out, s->d_ws + s->ws.part, n * 4, cudaMemcpyDeviceToHost));
  return DLLM_OK;
}

dllm_status dllm_set_cache(dllm_session* s, int layer, int which, const float* h_in, void* stream) {
  size_t n;
  dllm_status r = cache_args(s, layer, which, h_in, &n);
  if (r != DLLM_OK) return r;
  cudaStream_t st = (cudaStream_t)stream;
  CU_TRY(&s->err, cudaStreamSynchronize(st));
  CU_TRY(&s->err, h2d(s->d_ws + s->ws.part, h_in, n * 4, st));
  Launch L{st, nullptr, &s->launches};
  launch_convert_from_f32(L, s->m->cfg.dtype, s->wsp<float>(s->ws.part), s->cache(layer, which), n);
  CU_TRY(&s->err, cudaStreamSynchronize(st));
  return DLLM_OK;
}

dllm_status dllm_force_selection(dllm_session* s, int layer, const int32_t* h_idx, int count) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  if (layer < 0 || layer >= s->m->cfg.n_layers) return fail(&s->err, DLLM_INVALID_ARG, "layer out of range");
  if (count < 0) {
    s->forced_count[layer] = -1;
    return DLLM_OK;
  }
  if (count > s->R || (count > 0 && !h_idx)) return fail(&s->err, DLLM_INVALID_ARG, "bad forced selection");
  std::vector<int32_t> buf((size_t)s->B * s->R, 0);
  for (int b = 0; b < s->B; ++b) {
    std::vector<int32_t> row(h_idx + (size_t)b * count, h_idx + (size_t)(b + 1) * count);
    std::sort(row.begin(), row.end());
    for (int r = 0; r < count; ++r) {
      if (row[r] < 0 || row[r] >= s->R || (r && row[r] == row[r - 1]))
        return fail(&s->err, DLLM_INVALID_ARG, "forced indices must be distinct and inside [0, R)");
      buf[(size_t)b * s->R + r] = row[r];
    }
  }
  CU_TRY(&s->err, cudaDeviceSynchronize());
  CU_TRY(&s->err, cudaMemcpy(s->d_ws + s->ws.forced + (size_t)layer * s->B * s->R * 4, buf.data(), buf.size() * 4,
                             cudaMemcpyHostToDevice));
  CU_TRY(&s->err, cudaDeviceSynchronize());  // the copy's DMA has landed before any stream may read it
  s->forced_count[layer] = count;
  return DLLM_OK;
}

uint64_t dllm_launch_count(const dllm_session* s) { return s ? s->launches : 0; }

dllm_status dllm_session_use_graphs(dllm_session* s, int enable) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  s->use_graphs = enable != 0;
  return DLLM_OK;
}

dllm_status dllm_session_use_pdl(dllm_session* s, int enable) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  if ((enable != 0) != s->use_pdl) {
    s->drop_graphs();
  }
  s->use_pdl = enable != 0;
  return DLLM_OK;
}

dllm_status dllm_session_set_selection(dllm_session* s, int strategy, int metric, int v_selected_only) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  if (strategy < DLLM_SELECT_V_VERIFY || strategy > DLLM_SELECT_RANDOM || (metric != DLLM_METRIC_COSINE && metric != DLLM_METRIC_L2))
    return fail(&s->err, DLLM_INVALID_ARG, "unknown selection strategy or metric");
  s->sel_strategy = strategy;
  s->sel_metric = metric;
  s->v_selected_only = v_selected_only != 0;
  return DLLM_OK;
}

dllm_status dllm_set_scores(dllm_session* s, int layer, const float* h_scores, void* stream) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  if (!h_scores) return fail(&s->err, DLLM_INVALID_ARG, "h_scores is NULL");
  if (layer < 0 || layer >= s->m->cfg.n_layers) return fail(&s->err, DLLM_INVALID_ARG, "layer out of range");
  const size_t BR = (size_t)s->B * s->R;
  cudaStream_t st = (cudaStream_t)stream;
  CU_TRY(&s->err, cudaStreamSynchronize(st));
  CU_TRY(&s->err, h2d(s->d_ws + s->ws.sim + (size_t)layer * BR * 4, h_scores, BR * 4, st));
  return DLLM_OK;
}

dllm_status dllm_session_use_simt_gemm(dllm_session* s, int enable) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  if ((enable != 0) != s->simt_gemm) {
    s->drop_graphs();
  }
  s->simt_gemm = enable != 0;
  return DLLM_OK;
}

dllm_status dllm_session_profile(dllm_session* s, int enable) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  CU_TRY(&s->err, cudaDeviceSynchronize());
  for (auto& r : s->prof) {
    s->event_pool.push_back(r.a);
    s->event_pool.push_back(r.b);
  }
  s->prof.clear();
  for (auto& ps : s->prof_sum) ps = dllm_session::ProfSum{};
  s->profiling = enable != 0;
  return DLLM_OK;
}

dllm_status dllm_session_profile_read(dllm_session* s, int cls, double* total_ms, uint64_t* launches,
                                      double* algorithmic_bytes, double* flops) {
  if (!s) return fail(nullptr, DLLM_INVALID_ARG, "session is NULL");
  if (cls < 0 || cls >= DLLM_PROF_COUNT) return fail(&s->err, DLLM_INVALID_ARG, "unknown profile class");
  CU_TRY(&s->err, cudaDeviceSynchronize());
  // the two aggregates: every projection, every attention launch
  auto in_class = [cls](int c) {
    if (cls == DLLM_PROF_GEMM) return c >= DLLM_PROF_GEMM_V && c <= DLLM_PROF_GEMM_HEAD;
    if (cls == DLLM_PROF_ATTENTION) return c == DLLM_PROF_ATTN_MMA || c == DLLM_PROF_ATTN_UMMA;
    return c == cls;
  };
  double ms = 0, by = 0, fl = 0;
  uint64_t cnt = 0;
  for (int c = 0; c < DLLM_PROF_COUNT; ++c)
    if (in_class(c)) {
      ms += s->prof_sum[c].ms;
      by += s->prof_sum[c].bytes;
      fl += s->prof_sum[c].flops;
      cnt += s->prof_sum[c].launches;
    }
  for (auto& r : s->prof) {
    if (!in_class(r.cls)) continue;
    float t = 0.f;
    CU_TRY(&s->err, cudaEventElapsedTime(&t, r.a, r.b));
    ms += t;
    by += r.bytes;
    fl += r.flops;
    ++cnt;
  }
  if (total_ms) *total_ms = ms;
  if (launches) *launches = cnt;
  if (algorithmic_bytes) *algorithmic_bytes = by;
  if (flops) *flops = fl;
  return DLLM_OK;
}

// ---- kernel-level entry points ------------------------------------------------
size_t dllm_gemm_bf16_scratch_bytes(int M, int N, int K) {
  if (M <= 0 || N <= 0 || K <= 0) return 0;
  const GemmPlan p = plan_gemm_bf16(M, N, K);
  return p.S_max > 1 ? (size_t)p.S_max * M * N * 4 : 0;
}

dllm_status dllm_gemm_bf16(const void* d_A, const void* d_W, float* d_C, int M, int N, int K, void* d_partials,
                           void* stream) {
  if (!d_A || !d_W || !d_C || M <= 0 || N <= 0 || K <= 0) return fail(nullptr, DLLM_INVALID_ARG, "bad GEMM arguments");
  if (K % 8) return fail(nullptr, DLLM_INVALID_ARG, "K must be a multiple of 8");
  const GemmPlan p = plan_gemm_bf16(M, N, K);
  if (p.S_max > 1 && !d_partials) return fail(nullptr, DLLM_INVALID_ARG, "this shape needs slab scratch");
  Launch L{(cudaStream_t)stream, kernel_status_word(), nullptr};
  float* part = p.S_max > 1 ? static_cast<float*>(d_partials) : d_C;
  const char* why = nullptr;
  cudaError_t e = launch_gemm_bf16(L, d_A, d_W, part, M, N, K, p, &why);
  if (e != cudaSuccess) return fail(nullptr, DLLM_CUDA_ERROR, "bf16 GEMM: %s", why ? why : cudaGetErrorString(e));
  if (p.S_max > 1) launch_reduce_partials(L, make_partials(part, M, N, p), d_C, M);
  CU_TRY(nullptr, cudaGetLastError());
  return DLLM_OK;
}

size_t dllm_gemm_bf16_planned_scratch_bytes(int M, int N, int K, int act_tile, int splits) {
  if (M <= 0 || N <= 0 || K <= 0 || act_tile < 0 || splits < 0) return 0;
  const GemmPlan p = plan_gemm_bf16(M, N, K, splits, 0, act_tile);
  return p.S_max > 1 ? (size_t)p.S_max * M * N * 4 : 0;
}

dllm_status dllm_gemm_bf16_planned(const void* d_A, const void* d_W, float* d_C, int M, int N, int K, int act_tile,
                                   int splits, int stages, void* d_partials, size_t partials_bytes, void* stream) {
  if (!d_A || !d_W || M <= 0 || N <= 0 || K <= 0) return fail(nullptr, DLLM_INVALID_ARG, "bad GEMM arguments");
  if (K % 8) return fail(nullptr, DLLM_INVALID_ARG, "K must be a multiple of 8");
  if (act_tile < 0 || splits < 0 || stages < 0) return fail(nullptr, DLLM_INVALID_ARG, "negative plan parameter");
  if (act_tile && act_tile != 32 && act_tile != 64 && act_tile != 128 && act_tile != 192 && act_tile != 256)
    return fail(nullptr, DLLM_INVALID_ARG, "act_tile must be 0, 32, 64, 128, 192 or 256");
  if (act_tile == 192 && splits != 1)
    return fail(nullptr, DLLM_INVALID_ARG, "192-row tiles exist in the unsplit persistent kernel only: splits must be 1");
  const GemmPlan p = plan_gemm_bf16(M, N, K, splits, stages, act_tile);
  if (p.S_max > 1 && (!d_partials || partials_bytes < (size_t)p.S_max * M * N * 4))
    return fail(nullptr, DLLM_INVALID_ARG, "this plan needs %zu bytes of slab scratch", (size_t)p.S_max * M * N * 4);
  Launch L{(cudaStream_t)stream, kernel_status_word(), nullptr};
  if (!d_C && (p.S_max == 1 || !d_partials)) return fail(nullptr, DLLM_INVALID_ARG, "d_C is NULL");
  float* part = p.S_max > 1 ? static_cast<float*>(d_partials) : d_C;
  const char* why = nullptr;
  cudaError_t e = launch_gemm_bf16(L, d_A, d_W, part, M, N, K, p, &why);
  if (e != cudaSuccess) return fail(nullptr, DLLM_CUDA_ERROR, "bf16 GEMM: %s", why ? why : cudaGetErrorString(e));
  if (p.S_max > 1 && d_C) launch_reduce_partials(L, make_partials(part, M, N, p), d_C, M);
  CU_TRY(nullptr, cudaGetLastError());
  return DLLM_OK;
}

dllm_status dllm_ffn_gate_up_bf16(const void* d_A, const void* d_Wgu, void* d_out, int M, int d_ffn, int K,
                                  int act_tile, int stages, void* stream) {
  if (!d_A || !d_Wgu || !d_out || M <= 0 || d_ffn <= 0 || K <= 0)
    return fail(nullptr, DLLM_INVALID_ARG, "bad gate / up arguments");
  if (K % 8 || d_ffn % 64) return fail(nullptr, DLLM_INVALID_ARG, "K must be a multiple of 8 and d_ffn of 64");
  if (act_tile < 0 || stages < 0 ||
      (act_tile && act_tile != 32 && act_tile != 64 && act_tile != 128 && act_tile != 192 && act_tile != 256))
    return fail(nullptr, DLLM_INVALID_ARG, "act_tile must be 0, 32, 64, 128, 192 or 256");
  const GemmPlan p = plan_gemm_bf16(M, 2 * d_ffn, K, 1, stages, act_tile);
  Launch L{(cudaStream_t)stream, kernel_status_word(), nullptr};
  const char* why = nullptr;
  cudaError_t e = launch_gemm_bf16(L, d_A, d_Wgu, nullptr, M, 2 * d_ffn, K, p, &why, d_out, d_ffn);
  if (e != cudaSuccess) return fail(nullptr, DLLM_CUDA_ERROR, "gate / up GEMM: %s", why ? why : cudaGetErrorString(e));
  CU_TRY(nullptr, cudaGetLastError());
  return DLLM_OK;
}

size_t dllm_gemm_bf16_pair_scratch_bytes(int M, int N, int K, int act_tile, int splits) {
  if (M <= 0 || N <= 0 || K <= 0 || splits < 0 || (act_tile != 128 && act_tile != 256)) return 0;
  const GemmPlan p = plan_gemm_bf16(M, N, K, splits, 0, act_tile, 1);
  return p.S_max > 1 ? (size_t)p.S_max * M * N * 4 : 0;
}

dllm_status dllm_gemm_bf16_pair(const void* d_A, const void* d_W, float* d_C, int M, int N, int K, int act_tile,
                                int splits, int stages, void* d_partials, size_t partials_bytes, void* stream) {
  if (!d_A || !d_W || !d_C || M <= 0 || N <= 0 || K <= 0) return fail(nullptr, DLLM_INVALID_ARG, "bad GEMM arguments");
  if (K % 8 || N % 256) return fail(nullptr, DLLM_INVALID_ARG, "K must be a multiple of 8 and N of 256");
  if (splits < 0 || stages < 0 || (act_tile != 128 && act_tile != 256))
    return fail(nullptr, DLLM_INVALID_ARG, "act_tile must be 128 or 256");
  const GemmPlan p = plan_gemm_bf16(M, N, K, splits, stages, act_tile, 1);
  if (p.S_max > 1 && (!d_partials || partials_bytes < (size_t)p.S_max * M * N * 4))
    return fail(nullptr, DLLM_INVALID_ARG, "this plan needs %zu bytes of slab scratch", (size_t)p.S_max * M * N * 4);
  Launch L{(cudaStream_t)stream, kernel_status_word(), nullptr};
  float* part = p.S_max > 1 ? static_cast<float*>(d_partials) : d_C;
  const char* why = nullptr;
  cudaError_t e = launch_gemm_bf16(L, d_A, d_W, part, M, N, K, p, &why);
  if (e != cudaSuccess) return fail(nullptr, DLLM_CUDA_ERROR, "bf16 GEMM: %s", why ? why : cudaGetErrorString(e));
  if (p.S_max > 1) launch_reduce_partials(L, make_partials(part, M, N, p), d_C, M);
  CU_TRY(nullptr, cudaGetLastError());
  return DLLM_OK;
}

dllm_status dllm_gemm_simt(const void* d_A, const void* d_W, float* d_C, int M, int N, int K, int dtype,
                           void* stream) {
  if (!d_A || !d_W || !d_C || M <= 0 || N <= 0 || K <= 0) return fail(nullptr, DLLM_INVALID_ARG, "bad GEMM arguments");
  if (dtype != DLLM_FP32 && dtype != DLLM_BF16) return fail(nullptr, DLLM_INVALID_ARG, "bad dtype");
  Launch L{(cudaStream_t)stream, kernel_status_word(), nullptr};
  launch_gemm_simt(L, dtype, d_A, d_W, d_C, M, N, K);
  CU_TRY(nullptr, cudaGetLastError());
  return DLLM_OK;
}

size_t dllm_attention_scratch_bytes(int B, int a, int n, int H, int Hkv, int hd, int dtype) {
  if (B <= 0 || a <= 0 || n <= 0 || H <= 0 || Hkv <= 0 || H % Hkv || dtype != DLLM_BF16 || (hd != 64 && hd != 128))
    return 0;
  return choose_attention(B, a, n, H, Hkv, SIZE_MAX).plan.scratch_floats * 4;
}

dllm_status dllm_attention(const void* d_q, const void* d_k, const void* d_v, void* d_o, int B, int a, int n, int H,
                           int Hkv, int hd, int dtype, void* d_scratch, size_t scratch_bytes, void* stream) {
  if (!d_q || !d_k || !d_v || !d_o || B <= 0 || a <= 0 || n <= 0 || H <= 0 || Hkv <= 0 || H % Hkv)
    return fail(nullptr, DLLM_INVALID_ARG, "bad attention arguments");
  if (dtype != DLLM_FP32 && dtype != DLLM_BF16) return fail(nullptr, DLLM_INVALID_ARG, "bad dtype");
  if (hd % 32 || hd > 128) return fail(nullptr, DLLM_UNSUPPORTED, "head_dim must be 32, 64, 96 or 128");
  Launch L{(cudaStream_t)stream, kernel_status_word(), nullptr};
  cudaError_t e = launch_attention(L, dtype, d_q, d_k, d_v, d_o, B, a, n, H, Hkv, hd, static_cast<float*>(d_scratch),
                                   scratch_bytes / 4, false);
  if (e != cudaSuccess) return fail(nullptr, DLLM_CUDA_ERROR, "attention: %s", cudaGetErrorString(e));
  return DLLM_OK;
}

dllm_status dllm_vverify_select(const void* d_vnew, void* d_vcache, float* d_sim, int32_t* d_idx, int B, int R,
                                int width, int k, int dtype, void* stream) {
  if (!d_vnew || !d_vcache || !d_sim || B <= 0 || R <= 0 || width <= 0 || k < 0 || k > R || (k > 0 && !d_idx))
    return fail(nullptr, DLLM_INVALID_ARG, "bad V-verify arguments");
  if (dtype != DLLM_FP32 && dtype != DLLM_BF16) return fail(nullptr, DLLM_INVALID_ARG, "bad dtype");
  if (width % 8 || R > 8192) return fail(nullptr, DLLM_UNSUPPORTED, "width must be a multiple of 8 and R <= 8192");
  Launch L{(cudaStream_t)stream, kernel_status_word(), nullptr};
  launch_vverify_rows(L, dtype, d_vnew, d_vcache, d_sim, B * R, width);
  if (k > 0) CU_TRY(nullptr, launch_select(L, d_sim, nullptr, 1, k, d_idx, k, nullptr, nullptr, Geo{B, 0, R, R, width}, 0));
  CU_TRY(nullptr, cudaGetLastError());
  return DLLM_OK;
}

}  // extern "C"
