// Non-causal attention of the active query rows over ALL n cached keys of their
// sequence (Sec. A.7: the recomputed rows attend to the full sequence), with
// grouped KV heads (query head h reads KV head h / (H/Hkv)).
//
// attn_simt_kernel: fp32 arithmetic on the plain ALUs for any storage type.
// One CTA = 16 query rows of one sequence x one query head; keys and values
// are staged 32 rows at a time in shared memory; each warp owns 4 queries,
// lane = key for the scores, lane = output column for P*V; online softmax.
#include "internal.h"

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

}  // namespace

cudaError_t launch_attention(const Launch& L, int dtype, const void* q, const void* Kc, const void* Vc, void* o, int B,
                             int a_seq, int n, int H, int Hkv, int hd) {
  if (B <= 0 || a_seq <= 0) return cudaSuccess;
  if (hd > HD_MAX || (hd & 31) || H % Hkv) return cudaErrorInvalidValue;
  const float scale = 1.0f / sqrtf((float)hd);
  dim3 grid((a_seq + TQ - 1) / TQ, H, B);
  if (dtype == 0)
    attn_simt_kernel<float><<<grid, 128, 0, L.stream>>>((const float*)q, (const float*)Kc, (const float*)Vc,
                                                        (float*)o, a_seq, n, H, Hkv, hd, scale);
  else
    attn_simt_kernel<__nv_bfloat16><<<grid, 128, 0, L.stream>>>((const __nv_bfloat16*)q, (const __nv_bfloat16*)Kc,
                                                                (const __nv_bfloat16*)Vc, (__nv_bfloat16*)o, a_seq, n,
                                                                H, Hkv, hd, scale);
  L.count();
  return cudaGetLastError();
}

}  // namespace dllm
