// Persistent layer kernel: every layer of one cached denoising step (response
// refresh or adaptive partial update, Sec. 3.2) in ONE cooperative launch of
// one CTA per SM.
//
// Why: at batch 1 a cached step is bound by streaming ~15 GB of weights, but a
// layer is a chain of five small projections separated by row-wise work on a
// few hundred rows.  Launched kernel by kernel, every link of the chain pays a
// launch, a pipeline fill and a drain, and HBM idles in between.  Here the
// weight stream never stops: in every CTA one thread walks the static list of
// (layer, projection, tile, k-block) units of its SM and keeps a ring of
// shared-memory stages full with TMA loads of weight tiles, independent of how
// far the dependent work has come.  The activation tile of a stage is loaded
// by a second thread once the phase that produces it has finished on all SMs.
//
// Roles inside a CTA (256 threads):
//   warp 0, lane 0   weight producer (TMA, runs ahead across phases and layers)
//   warp 2, lane 0   activation producer (TMA, gated by the grid phase counter)
//   warp 1, lane 0   tcgen05.mma issuer; accumulators in TMEM, two sets
//   warps 4..7       workers: drain accumulators to fp32 slabs, then run the
//                    row-wise phases (V-verify of Eq. 6, bottom-k selection,
//                    gather, RoPE + K scatter, attention, output epilogues,
//                    SwiGLU gate, residual + next RMSNorm)
// Phases are separated by a grid barrier (one counter per phase in global
// memory, one arrival per CTA); only the workers and the activation producer
// wait on it.  Partial sums of a tile whose k range is shared by several CTAs
// go to slabs that the consuming phase adds in k order (bit-reproducible).
//
// Every wait is bounded (2 s): on expiry the CTA records a code in the status
// word, raises the abort flag that all its loops poll, and returns after its
// copies in flight have landed; other CTAs stop at their next barrier wait.
#include "attention_core.cuh"
#include "internal.h"
#include "tma.cuh"
#include "umma.cuh"

namespace dllm {

namespace {

constexpr int MK_THREADS = 256;
constexpr int MK_WORKERS = 128;                 // warps 4..7
constexpr int MK_STAGES = 4;
constexpr uint32_t MK_W_BYTES = 128 * 64 * 2;   // weight tile: 128 rows x 64 k
constexpr uint32_t MK_A_BYTES = 128 * 64 * 2;   // activation tile: up to 128 rows x 64 k
constexpr uint32_t MK_STAGE_BYTES = MK_W_BYTES + MK_A_BYTES;
constexpr uint32_t MK_RING_BYTES = MK_STAGES * MK_STAGE_BYTES;
constexpr uint32_t MK_TMEM_COLS = 256;          // two accumulators of up to 128 columns
constexpr int MK_MAX_R = 1024;                  // selection keys live in shared memory

using bf16 = __nv_bfloat16;

// ---- phase numbering (identical in every role) -------------------------------
// phase 0: embedding + first RMSNorm.  Then per layer, in order:
//   V, vverify, select, QK, rope, attention, [combine], O, o-epilogue, GU, silu, D, tail
struct Phases {
  int npl, hc;
  __device__ Phases(int has_comb) : npl(12 + has_comb), hc(has_comb) {}
  __device__ int base(int l) const { return 1 + l * npl; }
  // the phase whose completion makes the activation operand of projection g of layer l ready
  __device__ int a_ready(int l, int g) const {
    const int b = base(l);
    switch (g) {
      case MK_V: return b - 1;        // previous layer's tail (or phase 0)
      case MK_QK: return b + 2;       // select + gather
      case MK_O: return b + 5 + hc;   // attention or its combine
      case MK_GU: return b + 7 + hc;  // o-epilogue
      default: return b + 9 + hc;     // silu
    }
  }
};

struct Ctx {
  int tid;              // worker thread id 0..127 (workers only)
  int cta, G;
  volatile int* abortp;
  const MkParams* p;
};

__device__ __forceinline__ void wk_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Sum over the 128 workers; every worker gets the result.  red: >= 4 floats.
__device__ __forceinline__ float wk_sum(float v, float* red, int tid) {
  v = warp_sum(v);
  wk_sync();
  if ((tid & 31) == 0) red[tid >> 5] = v;
  wk_sync();
  return red[0] + red[1] + red[2] + red[3];
}

// ---- grid barrier ---------------------------------------------------------------
// arrive: all workers of the CTA have finished their writes of the phase.
__device__ __forceinline__ void grid_arrive(const Ctx& c, int phase) {
  asm volatile("fence.proxy.async;" ::: "memory");  // later TMA reads of what was written with plain stores
  __threadfence();
  wk_sync();
  if (c.tid == 0) atomicAdd(c.p->bar + phase, 1u);
}
// Spin (one thread) until `phase` has completed on every CTA.  false: gave up.
__device__ __forceinline__ bool phase_spin(const MkParams& p, int phase, int G, volatile int* abortp) {
  const unsigned target = (unsigned)G;  // every phase has a counter of its own: one arrival per CTA
  const volatile unsigned* bar = p.bar + phase;
  if (*bar >= target) return true;
  const uint64_t t0 = gtime();
  uint32_t it = 0;
  while (*bar < target) {
    if ((++it & 255u) == 0u) {
      if (*abortp) return false;
      if (*reinterpret_cast<const volatile int*>(p.status) != ST_OK || gtime() - t0 > WAIT_LIMIT_NS) {
        atomicCAS(p.status, ST_OK, ST_TIMEOUT_GRID);
        *abortp = 1;
        return false;
      }
    }
  }
  return true;
}
// wait (workers): returns false on abort, uniformly for all 128 workers.
__device__ __forceinline__ bool grid_wait(const Ctx& c, int phase) {
  bool ok = true;
  if (c.tid == 0) {
    ok = phase_spin(*c.p, phase, c.G, c.abortp);
    __threadfence();
  }
  return at_sync_and(ok);
}

// ---- projection roles -----------------------------------------------------------------
struct Seg {
  int tile, kb0, nkb;
};
__device__ __forceinline__ Seg seg_at(int u, int u1, int num_kb) {
  Seg s;
  s.tile = u / num_kb;
  s.kb0 = u - s.tile * num_kb;
  s.nkb = min(num_kb - s.kb0, u1 - u);
  return s;
}

__device__ void weight_producer(const MkParams& p, int cta, uint32_t ring, uint64_t* full_bar, uint64_t* empty_bar,
                                volatile int* abortp) {
  int s = 0;
  uint32_t ph = 0;
  for (int l = 0; l < p.T; ++l) {
    for (int g = 0; g < 5; ++g) {
      const MkGemm& G = p.g[g];
      const CUtensorMap* tm = p.maps_fixed + (l * 5 + g);
      if (G.total <= 0) continue;
      const int u0 = cta * G.upc, u1 = min(G.total, u0 + G.upc);
      const uint32_t bytes = MK_W_BYTES + (uint32_t)G.BN * 128u;
      for (int u = u0; u < u1; ++u) {
        const int tile = u / G.num_kb, kb = u - tile * G.num_kb;
        if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, abortp)) {
          atomicCAS(p.status, ST_OK, ST_TIMEOUT_TMA);
          return;
        }
        const uint32_t fb = smem_u32(&full_bar[s]);
        mbar_expect_tx(fb, bytes);
        tma_load_2d(ring + s * MK_STAGE_BYTES, tm, fb, kb * 64, (tile / G.m_tiles) * 128);
        if (++s == MK_STAGES) {
          s = 0;
          ph ^= 1u;
        }
      }
    }
  }
}

__device__ void activation_producer(const MkParams& p, int cta, int G_ctas, uint32_t ring, uint64_t* full_bar,
                                    uint64_t* empty_bar, volatile int* abortp) {
  const Phases P(p.has_comb);
  int s = 0;
  uint32_t ph = 0;
  for (int l = 0; l < p.T; ++l) {
    for (int g = 0; g < 5; ++g) {
      const MkGemm& G = p.g[g];
      if (G.total <= 0) continue;
      const int u0 = cta * G.upc, u1 = min(G.total, u0 + G.upc);
      if (u0 >= u1) continue;
      if (!phase_spin(p, P.a_ready(l, g), G_ctas, abortp)) return;
      __threadfence();
      asm volatile("fence.proxy.async;" ::: "memory");
      const CUtensorMap* tm = &p.amap[g];
      for (int u = u0; u < u1; ++u) {
        const int tile = u / G.num_kb, kb = u - tile * G.num_kb;
        // the stage is free (its previous contents were multiplied); the weight
        // producer arms the same barrier with the byte count of both tiles
        if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, abortp)) {
          atomicCAS(p.status, ST_OK, ST_TIMEOUT_TMA);
          return;
        }
        tma_load_2d(ring + s * MK_STAGE_BYTES + MK_W_BYTES, tm, smem_u32(&full_bar[s]), kb * 64,
                    (tile % G.m_tiles) * G.BN);
        if (++s == MK_STAGES) {
          s = 0;
          ph ^= 1u;
        }
      }
    }
  }
}

__device__ void mma_issuer(const MkParams& p, int cta, uint32_t ring, uint32_t tmem_d, uint64_t* full_bar,
                           uint64_t* empty_bar, uint64_t* acc_full, uint64_t* acc_empty, volatile int* abortp) {
  int s = 0;
  uint32_t ph = 0;
  uint32_t seg = 0;
  for (int l = 0; l < p.T; ++l) {
    for (int g = 0; g < 5; ++g) {
      const MkGemm& G = p.g[g];
      if (G.total <= 0) continue;
      const int u0 = cta * G.upc, u1 = min(G.total, u0 + G.upc);
      const uint32_t idesc = make_idesc(128, G.BN);
      for (int u = u0; u < u1; ++seg) {
        const Seg sg = seg_at(u, u1, G.num_kb);
        const uint32_t buf = seg & 1u;
        if (!mbar_wait(smem_u32(&acc_empty[buf]), ((seg >> 1) & 1u) ^ 1u, abortp)) {
          atomicCAS(p.status, ST_OK, ST_TIMEOUT_MMA);
          return;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t d_addr = tmem_d + buf * 128u;
        for (int i = 0; i < sg.nkb; ++i) {
          if (!mbar_wait(smem_u32(&full_bar[s]), ph, abortp)) {
            atomicCAS(p.status, ST_OK, ST_TIMEOUT_MMA);
            return;
          }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t sW = ring + s * MK_STAGE_BYTES;
          const uint64_t dW = make_smem_desc(sW);
          const uint64_t dA = make_smem_desc(sW + MK_W_BYTES);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_bf16(d_addr, dW + (uint64_t)(2 * k), dA + (uint64_t)(2 * k), idesc, (i > 0 || k > 0) ? 1u : 0u);
          umma_commit(smem_u32(&empty_bar[s]));
          if (++s == MK_STAGES) {
            s = 0;
            ph ^= 1u;
          }
        }
        umma_commit(smem_u32(&acc_full[buf]));
        u += sg.nkb;
      }
    }
  }
}

// Workers: drain this CTA's segments of projection g into the slab buffer.
// seg: running segment counter of the CTA (selects the accumulator set).
__device__ bool drain_projection(const Ctx& c, const MkGemm& G, uint32_t tmem_d, uint64_t* acc_full,
                                 uint64_t* acc_empty, uint32_t& seg) {
  const MkParams& p = *c.p;
  if (G.total <= 0) return true;
  const int u0 = c.cta * G.upc, u1 = min(G.total, u0 + G.upc);
  const int warp = c.tid >> 5, lane = c.tid & 31;  // worker warp w reads TMEM lanes 32w..32w+31 (warps 4..7 -> w%4)
  const size_t stride = (size_t)G.M * G.N;
  for (int u = u0; u < u1; ++seg) {
    const Seg sg = seg_at(u, u1, G.num_kb);
    const uint32_t buf = seg & 1u;
    const bool have = mbar_wait(smem_u32(&acc_full[buf]), (seg >> 1) & 1u, c.abortp);
    if (!at_sync_and(have)) {
      if (c.tid == 0) atomicCAS(p.status, ST_OK, ST_TIMEOUT_EPI);
      return false;
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const int nt = sg.tile / G.m_tiles, mt = sg.tile - nt * G.m_tiles;
    const int m0 = mt * G.BN;
    const int n = nt * 128 + warp * 32 + lane;
    const int slab = c.cta - (sg.tile * G.num_kb) / G.upc;
    float* out = p.part + (size_t)slab * stride + n;
    const uint32_t t_addr = tmem_d + ((uint32_t)(warp * 32) << 16) + buf * 128u;
#pragma unroll 1
    for (int col = 0; col < G.BN; col += 16) {
      if (m0 + col >= G.M) break;
      uint32_t r[16];
      tmem_ld16(t_addr + (uint32_t)col, r);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      if (n < G.N) {
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int m = m0 + col + j;
          if (m < G.M) out[(size_t)m * G.N] = __uint_as_float(r[j]);
        }
      }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&acc_empty[buf]));
    u += sg.nkb;
  }
  return true;
}

__device__ __forceinline__ Partials mk_partials(const MkParams& p, const MkGemm& G) {
  Partials out{p.part, (size_t)G.M * G.N, 1, G.N};
  if (G.upc % G.num_kb != 0) {
    out.upc = G.upc;
    out.num_kb = G.num_kb;
    out.m_tiles = G.m_tiles;
    out.BN = G.BN;
    out.TW = 128;
  }
  return out;
}

// ---- row-wise phases (workers) ------------------------------------------------------
__device__ __forceinline__ void row_pos(const MkParams& p, int c, int& b, int& pos) {  // carried response row -> (sequence, position)
  b = c / p.R;
  pos = p.P + (c - b * p.R);
}
__device__ __forceinline__ uint8_t* layer_cache(const MkParams& p, int l, size_t which_off) {
  return p.cache + (size_t)l * p.cache_layer_bytes + which_off;
}
__device__ __forceinline__ const uint8_t* layer_w(const MkParams& p, int l, size_t off) {
  return p.W + (size_t)l * p.layer_stride + off;
}

// u[row] = rmsnorm(x[row]) * gain, x[row] given by fill(i, v[8]) which also stores it.
template <typename Fill>
__device__ __forceinline__ void fill_and_norm(const Ctx& c, int row, const float* gain, float* red, Fill fill) {
  const MkParams& p = *c.p;
  const int d = p.d;
  float* xr = p.x + (size_t)row * d;
  float ss = 0.f;
  for (int i = c.tid * 8; i < d; i += MK_WORKERS * 8) {
    float v[8];
    fill(i, v);
    Vec8<float>::store(xr + i, v);
#pragma unroll
    for (int j = 0; j < 8; ++j) ss += v[j] * v[j];
  }
  ss = wk_sum(ss, red, c.tid);
  const float r = rsqrtf(ss / (float)d + p.eps);
  bf16* orow = static_cast<bf16*>(p.u) + (size_t)row * d;
  for (int i = c.tid * 8; i < d; i += MK_WORKERS * 8) {
    float v[8], gv[8];
    Vec8<float>::load(xr + i, v);  // this thread's own stores
    Vec8<float>::load(gain + i, gv);
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = v[j] * r * gv[j];
    Vec8<bf16>::store(orow + i, v);
  }
}

// phase 0: x = E[token], u = rmsnorm(x) * norm1 of layer 0, response rows.
__device__ void phase_embed(const Ctx& c, float* red) {
  const MkParams& p = *c.p;
  const bf16* E = reinterpret_cast<const bf16*>(p.W + p.o_embed);
  const float* gain = reinterpret_cast<const float*>(layer_w(p, 0, p.o_norm1));
  for (int row = c.cta; row < p.BR; row += c.G) {
    int b, pos;
    row_pos(p, row, b, pos);
    const int tok = p.tokens[(size_t)b * p.n + pos];
    const bf16* src = E + (size_t)tok * p.d;
    fill_and_norm(c, row, gain, red, [&](int i, float (&v)[8]) { Vec8<bf16>::load(src + i, v); });
  }
}

// V-verify (Eq. 6) with the whole-V overwrite (Sec. A.5), one response row at a time.
__device__ void phase_vverify(const Ctx& c, int l, float* red) {
  const MkParams& p = *c.p;
  const Partials part = mk_partials(p, p.g[MK_V]);
  const int dkv = p.dkv;
  bf16* Vc = reinterpret_cast<bf16*>(layer_cache(p, l, p.c_v));
  float* sim = p.sim + (size_t)l * p.BR;
  for (int row = c.cta; row < p.BR; row += c.G) {
    int b, pos;
    row_pos(p, row, b, pos);
    bf16* vrow = Vc + ((size_t)b * p.n + pos) * dkv;
    float dot = 0.f, na = 0.f, nb = 0.f;
    for (int i = c.tid * 8; i < dkv; i += MK_WORKERS * 8) {
      float vn[8], vo[8];
      sum_partials8(part.p, part.split_stride, part.count(row, i), (size_t)row * part.N + i, vn);
      Vec8<bf16>::load(vrow + i, vo);
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        vn[t] = Vec8<bf16>::round(vn[t]);  // compare what the cache will hold
        dot += vn[t] * vo[t];
        na += vn[t] * vn[t];
        nb += vo[t] * vo[t];
      }
      Vec8<bf16>::store(vrow + i, vn);
    }
    dot = warp_sum(dot);
    na = warp_sum(na);
    nb = warp_sum(nb);
    wk_sync();
    if ((c.tid & 31) == 0) {
      red[(c.tid >> 5) * 3 + 0] = dot;
      red[(c.tid >> 5) * 3 + 1] = na;
      red[(c.tid >> 5) * 3 + 2] = nb;
    }
    wk_sync();
    if (c.tid == 0) {
      const float D = red[0] + red[3] + red[6] + red[9], A = red[1] + red[4] + red[7] + red[10],
                  Bn = red[2] + red[5] + red[8] + red[11];
      sim[row] = D / fmaxf(sqrtf(A * Bn), 1e-8f);
    }
  }
}

// Bottom-k selection (Sec. 3.2.2) for the sequences this CTA needs, the active
// row list, its inverse, and the gather of the selected rows of u into ua.
// scratch: >= R * 17 bytes of shared memory.
__device__ void phase_select(const Ctx& c, int l, uint8_t* scratch) {
  const MkParams& p = *c.p;
  const int R = p.R, ksel = p.ksel, a_seq = p.a_seq;
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(scratch);
  int32_t* sel_s = reinterpret_cast<int32_t*>(scratch + (size_t)R * 8);
  int32_t* inv_s = sel_s + R;
  const int mode = p.rr ? 0 : (((p.forced_mask >> l) & 1ull) ? 2 : 1);
  const float* sim = p.sim + (size_t)l * p.BR;
  int32_t* sel = p.sel + (size_t)l * p.BR;
  const int32_t* forced = p.forced + (size_t)l * p.BR;
  for (int b = 0; b < p.B; ++b) {
    const bool owner = (b % c.G) == c.cta;
    // rows of the active list that fall to this CTA and belong to sequence b
    const int r_lo = b * a_seq, r_hi = r_lo + a_seq;
    int first = c.cta + ((r_lo > c.cta) ? ((r_lo - c.cta + c.G - 1) / c.G) * c.G : 0);
    const bool has_rows = !p.rr && first < r_hi;
    if (!owner && !has_rows) continue;
    wk_sync();
    for (int j = c.tid; j < R; j += MK_WORKERS) inv_s[j] = -1;
    if (mode == 0) {
      for (int j = c.tid; j < R; j += MK_WORKERS) sel_s[j] = j;
    } else if (mode == 2) {
      for (int r = c.tid; r < ksel; r += MK_WORKERS) sel_s[r] = forced[(size_t)b * R + r];
    } else {
      for (int j = c.tid; j < R; j += MK_WORKERS) {
        const float s = __ldcg(sim + (size_t)b * R + j);
        // key = round(s * 2^20), offset into 1 .. 2^32 - 1 (scores beyond +-2047 saturate); NaN sorts first
        const float qf = fminf(fmaxf(rintf(s * 1048576.0f), -2147483520.0f), 2147483520.0f);
        const long long q = (s == s) ? (long long)qf + (1ll << 31) : 0ll;
        keys[j] = ((unsigned long long)q << 32) | (unsigned)j;
      }
      wk_sync();
      // keys are unique, so the rank of a key is its position in sorted order;
      // the selected rows in ascending index order: row j gets slot #selected before j
      unsigned char* flag = reinterpret_cast<unsigned char*>(inv_s + R);
      for (int j = c.tid; j < R; j += MK_WORKERS) {
        const unsigned long long kj = keys[j];
        int rank = 0;
        for (int i = 0; i < R; ++i) rank += (keys[i] < kj);
        flag[j] = (rank < ksel);
      }
      wk_sync();
      for (int j = c.tid; j < R; j += MK_WORKERS) {
        if (!flag[j]) continue;
        int r = 0;
        for (int i = 0; i < j; ++i) r += flag[i];
        sel_s[r] = j;
      }
    }
    wk_sync();
    for (int r = c.tid; r < a_seq; r += MK_WORKERS) inv_s[sel_s[r]] = r;
    wk_sync();
    if (owner) {
      for (int r = c.tid; r < a_seq; r += MK_WORKERS) {
        sel[(size_t)b * R + r] = sel_s[r];
        p.act[(size_t)b * a_seq + r] = b * R + sel_s[r];
      }
      for (int j = c.tid; j < R; j += MK_WORKERS) p.inv[(size_t)b * R + j] = inv_s[j] >= 0 ? b * a_seq + inv_s[j] : -1;
    }
    if (has_rows) {
      const int nvec = p.d * 2 / 16;
      for (int r = first; r < r_hi; r += c.G) {
        const int crow = b * R + sel_s[r - r_lo];
        const uint4* s4 = reinterpret_cast<const uint4*>(static_cast<const bf16*>(p.u) + (size_t)crow * p.d);
        uint4* o4 = reinterpret_cast<uint4*>(static_cast<bf16*>(p.ua) + (size_t)r * p.d);
        for (int i = c.tid; i < nvec; i += MK_WORKERS) o4[i] = __ldcg(s4 + i);
      }
    }
  }
}

// RoPE on Q and K of the active rows; Q -> qbuf, K -> K cache rows (post-RoPE).
__device__ void phase_rope(const Ctx& c, int l) {
  const MkParams& p = *c.p;
  const Partials part = mk_partials(p, p.g[MK_QK]);
  const int hd = p.hd, half = hd >> 1, H = p.H, q4 = half >> 2;
  bf16* Kc = reinterpret_cast<bf16*>(layer_cache(p, l, 0));
  bf16* qbuf = static_cast<bf16*>(p.qbuf);
  const int groups = (H + p.Hkv) * q4;
  for (int r = c.cta; r < p.Ma; r += c.G) {
    const int crow = p.rr ? r : __ldcg(p.act + r);
    int b, pos;
    row_pos(p, crow, b, pos);
    const float* tab = p.rope + (size_t)pos * hd;  // [cos(half) | sin(half)]
    const float* prow = part.p + (size_t)r * part.N;
    for (int gidx = c.tid; gidx < groups; gidx += MK_WORKERS) {
      const int head = gidx / q4, i0 = (gidx - head * q4) * 4;
      const bool is_q = head < H;
      const int col0 = is_q ? head * hd : p.dq + (head - H) * hd;
      bf16* dst = is_q ? qbuf + (size_t)r * p.dq + head * hd : Kc + ((size_t)b * p.n + pos) * p.dkv + (head - H) * hd;
      float lo[4] = {0.f, 0.f, 0.f, 0.f}, hi[4] = {0.f, 0.f, 0.f, 0.f};
      const int n_lo = part.count(r, col0 + i0), n_hi = part.count(r, col0 + i0 + half);
      for (int s = 0; s < n_lo; ++s) {
        const float4 t = __ldcg(reinterpret_cast<const float4*>(prow + (size_t)s * part.split_stride + col0 + i0));
        lo[0] += t.x; lo[1] += t.y; lo[2] += t.z; lo[3] += t.w;
      }
      for (int s = 0; s < n_hi; ++s) {
        const float4 t = __ldcg(reinterpret_cast<const float4*>(prow + (size_t)s * part.split_stride + col0 + i0 + half));
        hi[0] += t.x; hi[1] += t.y; hi[2] += t.z; hi[3] += t.w;
      }
      const float4 cs = *reinterpret_cast<const float4*>(tab + i0);
      const float4 sn = *reinterpret_cast<const float4*>(tab + half + i0);
      const float cc[4] = {cs.x, cs.y, cs.z, cs.w}, ss[4] = {sn.x, sn.y, sn.z, sn.w};
      float o_lo[4], o_hi[4];
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        o_lo[t] = lo[t] * cc[t] - hi[t] * ss[t];
        o_hi[t] = hi[t] * cc[t] + lo[t] * ss[t];
      }
      *reinterpret_cast<uint2*>(dst + i0) = make_uint2(pack_bf16(o_lo[0], o_lo[1]), pack_bf16(o_lo[2], o_lo[3]));
      *reinterpret_cast<uint2*>(dst + i0 + half) = make_uint2(pack_bf16(o_hi[0], o_hi[1]), pack_bf16(o_hi[2], o_hi[3]));
    }
  }
}

template <int HD>
__device__ bool phase_attention(const Ctx& c, int l, uint8_t* at_gen, uint32_t at_sh, uint64_t* at_bar,
                                uint32_t& kv_iter) {
  const MkParams& p = *c.p;
  const int G = p.H / p.Hkv;
  const int x_tiles = (p.a_seq * G + AT_ROWS - 1) / AT_ROWS;
  const int items = x_tiles * p.Hkv * p.B * p.attn_S;
  const CUtensorMap* tmK = p.maps_fixed + p.T * 5 + 2 * l;
  const size_t total = (size_t)p.B * p.a_seq * p.H;
  float* o_part = p.attn_scratch;
  float* ml_part = p.attn_scratch + (size_t)p.attn_S * total * HD;
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)HD);
  for (int it = c.cta; it < items; it += c.G) {
    const int bx = it % x_tiles, by = (it / x_tiles) % p.Hkv, bz = it / (x_tiles * p.Hkv);
    if (!attn_tile<HD>(c.tid, at_gen, at_sh, at_bar, kv_iter, c.abortp, tmK, tmK + 1,
                       static_cast<const bf16*>(p.qbuf), static_cast<bf16*>(p.obuf), o_part, ml_part, p.a_seq, p.n,
                       p.H, p.Hkv, p.attn_S, p.attn_kps, scale_log2, p.B, bx, by, bz)) {
      if (c.tid == 0) atomicCAS(p.status, ST_OK, ST_TIMEOUT_TMA);
      return false;
    }
  }
  return true;
}

// Merges the key-range splits: out = sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s; one warp per (row, head).
__device__ void phase_combine(const Ctx& c) {
  const MkParams& p = *c.p;
  const int S = p.attn_S, hd = p.hd;
  const size_t total = (size_t)p.B * p.a_seq * p.H;
  const float* o_part = p.attn_scratch;
  const float* ml_part = p.attn_scratch + (size_t)S * total * hd;
  bf16* o = static_cast<bf16*>(p.obuf);
  const int warp = c.tid >> 5, lane = c.tid & 31;
  for (size_t rh = (size_t)c.cta * 4 + warp; rh < total; rh += (size_t)c.G * 4) {
    float M = -INFINITY;
    for (int s = 0; s < S; ++s) M = fmaxf(M, __ldcg(ml_part + ((size_t)s * total + rh) * 2));
    float L = 0.f;
    for (int s = 0; s < S; ++s) {
      const float* ml = ml_part + ((size_t)s * total + rh) * 2;
      L += exp2f(__ldcg(ml) - M) * __ldcg(ml + 1);
    }
    const float inv = 1.f / L;
    for (int dd = lane; dd < hd; dd += 32) {
      float acc = 0.f;
      for (int s = 0; s < S; ++s)
        acc += exp2f(__ldcg(ml_part + ((size_t)s * total + rh) * 2) - M) * __ldcg(o_part + ((size_t)s * total + rh) * hd + dd);
      o[rh * hd + dd] = __float2bfloat16_rn(acc * inv);
    }
  }
}

// AttnOut rows -> cache (rounded to bf16); h = x + AttnOut; hn = rmsnorm(h) * norm2.
__device__ void phase_oepi(const Ctx& c, int l, float* hrow, float* red) {
  const MkParams& p = *c.p;
  const Partials part = mk_partials(p, p.g[MK_O]);
  const int d = p.d;
  bf16* Ac = reinterpret_cast<bf16*>(layer_cache(p, l, p.c_a));
  const float* gain2 = reinterpret_cast<const float*>(layer_w(p, l, p.o_norm2));
  for (int r = c.cta; r < p.Ma; r += c.G) {
    const int crow = p.rr ? r : __ldcg(p.act + r);
    int b, pos;
    row_pos(p, crow, b, pos);
    bf16* arow = Ac + ((size_t)b * p.n + pos) * d;
    const float* xr = p.x + (size_t)crow * d;
    float ss = 0.f;
    wk_sync();  // hrow of the previous row has been read
    for (int i = c.tid * 8; i < d; i += MK_WORKERS * 8) {
      float a[8], xv[8];
      sum_partials8(part.p, part.split_stride, part.count(r, i), (size_t)r * part.N + i, a);
      Vec8<float>::load_cg(xr + i, xv);
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        a[t] = Vec8<bf16>::round(a[t]);
        xv[t] += a[t];
        ss += xv[t] * xv[t];
      }
      Vec8<bf16>::store(arow + i, a);
      Vec8<float>::store(hrow + i, xv);
    }
    ss = wk_sum(ss, red, c.tid);
    const float rs = rsqrtf(ss / (float)d + p.eps);
    bf16* out = static_cast<bf16*>(p.hn) + (size_t)r * d;
    for (int i = c.tid * 8; i < d; i += MK_WORKERS * 8) {
      float v[8], gv[8];
      Vec8<float>::load(hrow + i, v);
      Vec8<float>::load(gain2 + i, gv);
#pragma unroll
      for (int t = 0; t < 8; ++t) v[t] = v[t] * rs * gv[t];
      Vec8<bf16>::store(out + i, v);
    }
  }
}

// act = silu(gate) * up from the slabs of the stacked [W_gate; W_up] projection.
__device__ void phase_silu(const Ctx& c) {
  const MkParams& p = *c.p;
  const Partials part = mk_partials(p, p.g[MK_GU]);
  const int m = p.m, mv = m >> 3;
  const size_t total = (size_t)p.Ma * mv;
  bf16* out = static_cast<bf16*>(p.ffn);
  for (size_t idx = (size_t)c.cta * MK_WORKERS + c.tid; idx < total; idx += (size_t)c.G * MK_WORKERS) {
    const int r = (int)(idx / mv), j = (int)(idx - (size_t)r * mv) * 8;
    float gt[8], up[8];
    const int cg = p.gu_interleaved ? (j >> 6) * 128 + (j & 63) : j, cu = p.gu_interleaved ? cg + 64 : m + j;
    sum_partials8(part.p, part.split_stride, part.count(r, cg), (size_t)r * part.N + cg, gt);
    sum_partials8(part.p, part.split_stride, part.count(r, cu), (size_t)r * part.N + cu, up);
#pragma unroll
    for (int t = 0; t < 8; ++t) gt[t] = gt[t] / (1.f + expf(-gt[t])) * up[t];
    Vec8<bf16>::store(out + (size_t)r * m + j, gt);
  }
}

// FFNOut rows of the active set -> cache; x <- (x + AttnOut) + FFNOut from the
// caches for every response row (Sec. 3.2 item (3)); u = rmsnorm(x) * gain of
// the next layer's first norm (the final norm after the last layer).
__device__ void phase_tail(const Ctx& c, int l, float* red) {
  const MkParams& p = *c.p;
  const Partials part = mk_partials(p, p.g[MK_D]);
  const int d = p.d;
  const bf16* Ac = reinterpret_cast<const bf16*>(layer_cache(p, l, p.c_a));
  bf16* Fc = reinterpret_cast<bf16*>(layer_cache(p, l, p.c_f));
  const float* gain = (l + 1 < p.T) ? reinterpret_cast<const float*>(layer_w(p, l + 1, p.o_norm1))
                                    : reinterpret_cast<const float*>(p.W + p.o_norm_f);
  for (int row = c.cta; row < p.BR; row += c.G) {
    int b, pos;
    row_pos(p, row, b, pos);
    const size_t crow = ((size_t)b * p.n + pos) * d;
    const int r = p.rr ? row : __ldcg(p.inv + row);
    const float* xr = p.x + (size_t)row * d;
    fill_and_norm(c, row, gain, red, [&](int i, float (&v)[8]) {
      float a[8], f[8];
      if (r >= 0) {
        sum_partials8(part.p, part.split_stride, part.count(r, i), (size_t)r * part.N + i, f);
        Vec8<bf16>::store(Fc + crow + i, f);
#pragma unroll
        for (int t = 0; t < 8; ++t) f[t] = Vec8<bf16>::round(f[t]);
      } else {
        Vec8<bf16>::load_cg(Fc + crow + i, f);
      }
      Vec8<float>::load_cg(xr + i, v);
      Vec8<bf16>::load_cg(Ac + crow + i, a);
#pragma unroll
      for (int t = 0; t < 8; ++t) v[t] = (v[t] + a[t]) + f[t];
    });
  }
}

// ---- the kernel -------------------------------------------------------------------------
template <int HD>
__device__ void worker_main(const Ctx& c, uint32_t tmem_d, uint64_t* acc_full, uint64_t* acc_empty, uint8_t* at_gen,
                            uint32_t at_sh, uint64_t* at_bar, float* red) {
  const MkParams& p = *c.p;
  const Phases P(p.has_comb);
  uint32_t seg = 0, kv_iter = 0;
  float* hrow = reinterpret_cast<float*>(at_gen);
  phase_embed(c, red);
  grid_arrive(c, 0);
  for (int l = 0; l < p.T; ++l) {
    const int b = P.base(l);
    if (!drain_projection(c, p.g[MK_V], tmem_d, acc_full, acc_empty, seg)) return;
    grid_arrive(c, b + 0);
    if (!grid_wait(c, b + 0)) return;
    phase_vverify(c, l, red);
    grid_arrive(c, b + 1);
    if (!grid_wait(c, b + 1)) return;
    phase_select(c, l, at_gen);
    grid_arrive(c, b + 2);
    if (!drain_projection(c, p.g[MK_QK], tmem_d, acc_full, acc_empty, seg)) return;
    grid_arrive(c, b + 3);
    if (!grid_wait(c, b + 3)) return;
    phase_rope(c, l);
    grid_arrive(c, b + 4);
    if (!grid_wait(c, b + 4)) return;
    if (c.tid == 0) asm volatile("fence.proxy.async;" ::: "memory");
    if (!phase_attention<HD>(c, l, at_gen, at_sh, at_bar, kv_iter)) return;
    grid_arrive(c, b + 5);
    if (p.has_comb) {
      if (!grid_wait(c, b + 5)) return;
      phase_combine(c);
      grid_arrive(c, b + 6);
    }
    if (!drain_projection(c, p.g[MK_O], tmem_d, acc_full, acc_empty, seg)) return;
    grid_arrive(c, b + 6 + P.hc);
    if (!grid_wait(c, b + 6 + P.hc)) return;
    phase_oepi(c, l, hrow, red);
    grid_arrive(c, b + 7 + P.hc);
    if (!drain_projection(c, p.g[MK_GU], tmem_d, acc_full, acc_empty, seg)) return;
    grid_arrive(c, b + 8 + P.hc);
    if (!grid_wait(c, b + 8 + P.hc)) return;
    phase_silu(c);
    grid_arrive(c, b + 9 + P.hc);
    if (!drain_projection(c, p.g[MK_D], tmem_d, acc_full, acc_empty, seg)) return;
    grid_arrive(c, b + 10 + P.hc);
    if (!grid_wait(c, b + 10 + P.hc)) return;
    phase_tail(c, l, red);
    grid_arrive(c, b + 11 + P.hc);
  }
}

template <int HD>
__global__ void __launch_bounds__(MK_THREADS, 1) layer_megakernel(const __grid_constant__ MkParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[MK_STAGES];
  __shared__ __align__(8) uint64_t empty_bar[MK_STAGES];
  __shared__ __align__(8) uint64_t acc_full[2];
  __shared__ __align__(8) uint64_t acc_empty[2];
  __shared__ __align__(8) uint64_t at_bar[2];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  __shared__ float red[16];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* ring_gen = smem_raw + (ring - smem_u32(smem_raw));
  uint8_t* at_gen = ring_gen + MK_RING_BYTES;
  const uint32_t at_sh = ring + MK_RING_BYTES;
  volatile int* abortp = &abort_flag;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < MK_STAGES; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&acc_full[b]), 1);
      mbar_init(smem_u32(&acc_empty[b]), 4);  // one arrival per worker warp
      mbar_init(smem_u32(&at_bar[b]), 1);
    }
    mbar_fence_init();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"(MK_TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_d = tmem_base_slot;
  pdl_wait();  // tokens, caches and the previous step's state belong to earlier kernels
  pdl_trigger();

  const int cta = (int)blockIdx.x, G = (int)gridDim.x;
  if (warp == 0) {
    if (lane == 0) weight_producer(p, cta, ring, full_bar, empty_bar, abortp);
  } else if (warp == 1) {
    if (lane == 0) mma_issuer(p, cta, ring, tmem_d, full_bar, empty_bar, acc_full, acc_empty, abortp);
  } else if (warp == 2) {
    if (lane == 0) activation_producer(p, cta, G, ring, full_bar, empty_bar, abortp);
  } else if (warp >= 4) {
    Ctx c{(int)threadIdx.x - 128, cta, G, abortp, &p};
    worker_main<HD>(c, tmem_d, acc_full, acc_empty, at_gen, at_sh, at_bar, red);
  }
  __syncwarp();
  if (*abortp) drain_delay();  // gave up: let copies in flight land before shared memory is released
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(MK_TMEM_COLS) : "memory");
  }
}

template <int HD>
constexpr size_t mk_smem_bytes() {
  return MK_RING_BYTES + (size_t)AttnSmem<HD>::BYTES + 1024;
}

}  // namespace

// ---- host side ---------------------------------------------------------------------------------
int mk_act_tile(int M) { return M <= 32 ? 32 : M <= 64 ? 64 : 128; }

bool mk_supported(int dtype, int B, int P, int R, int d, int H, int Hkv, int hd, int m, int T, int rp, int ksel) {
  (void)P;
  if (dtype != 1 || rp || ksel <= 0) return false;
  if (hd != 64 && hd != 128) return false;
  if (R > MK_MAX_R || T > 64 || B < 1) return false;
  if ((d & 7) || (m & 7) || ((Hkv * hd) & 7) || (H % Hkv)) return false;
  // the o-epilogue keeps one row of h (d floats) and the selection keeps 17 R
  // bytes in the attention phase's shared memory
  const size_t at = hd == 64 ? (size_t)AttnSmem<64>::BYTES : (size_t)AttnSmem<128>::BYTES;
  if ((size_t)d * 4 > at || (size_t)R * 17 > at) return false;
  return true;
}

static int mk_grid() {
  static int n = 0;
  if (n == 0) {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
      n = v;
    else
      return 148;
  }
  return n;
}

void mk_plan(MkParams& p) {
  const int G = mk_grid();
  auto set = [&](MkGemm& g, int M, int N, int K) {
    g.M = M;
    g.N = N;
    g.K = K;
    g.BN = mk_act_tile(M);
    g.m_tiles = (M + g.BN - 1) / g.BN;
    g.num_kb = (K + 63) / 64;
    g.total = M > 0 ? g.m_tiles * ((N + 127) / 128) * g.num_kb : 0;
    g.upc = g.total > 0 ? (g.total + G - 1) / G : 1;
  };
  set(p.g[MK_V], p.BR, p.dkv, p.d);
  set(p.g[MK_QK], p.Ma, p.dq + p.dkv, p.d);
  set(p.g[MK_O], p.Ma, p.d, p.dq);
  set(p.g[MK_GU], p.Ma, 2 * p.m, p.d);
  set(p.g[MK_D], p.Ma, p.d, p.m);
  const AttnPlan ap = plan_attention(p.B, p.a_seq, p.n, p.H, p.Hkv);
  p.attn_S = ap.S;
  p.attn_kps = ap.keys_per_split;
  p.has_comb = ap.S > 1 ? 1 : 0;
}

size_t mk_part_floats(const MkParams& p) {
  size_t need = 0;
  for (int i = 0; i < 5; ++i) {
    const MkGemm& g = p.g[i];
    if (g.total <= 0) continue;
    const size_t slabs = (g.upc % g.num_kb == 0) ? 1 : (size_t)(g.num_kb - 1) / g.upc + 2;
    const size_t f = slabs * (size_t)g.M * g.N;
    if (f > need) need = f;
  }
  return need;
}

cudaError_t launch_layer_megakernel(const Launch& L, const MkParams& p) {
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(layer_megakernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)mk_smem_bytes<64>());
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(layer_megakernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               (int)mk_smem_bytes<128>());
    if (e != cudaSuccess) return e;
    configured = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(mk_grid());
  cfg.blockDim = dim3(MK_THREADS);
  cfg.dynamicSmemBytes = p.hd == 64 ? mk_smem_bytes<64>() : mk_smem_bytes<128>();
  cfg.stream = L.stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;  // all CTAs resident: they wait on one another
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = p.hd == 64 ? cudaLaunchKernelEx(&cfg, layer_megakernel<64>, p)
                             : cudaLaunchKernelEx(&cfg, layer_megakernel<128>, p);
  L.count();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace dllm

DLLM_TIMELINE_HOOKS(megakernel)
