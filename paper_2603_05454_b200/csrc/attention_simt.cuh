// CUDA-core flash-style attention: suffix queries over [contiguous prefix cache | this pass's staged rows].
// Non-causal: every query row sees every key (the bidirectional lookahead of Sec. 3.2).  fp32 arithmetic with
// an online softmax; used for fp32 models and as the switchable reference of the tensor-core kernel.
#pragma once
#include "common.cuh"

namespace lsp {

constexpr int AS_BQ = 16;   // queries per block (4 per warp)
constexpr int AS_BK = 32;   // keys per tile (one per lane)

// grid = (ceil(max_rows_per_seq / 16), n_heads, batch), block = 128.
// q: [M, n_heads*DH]; cache_k/v: this layer's planes [batch_max][max_len][n_kv*DH]; stage_k/v: this layer's
// staged planes [M][n_kv*DH]; out: [M, n_heads*DH].
template <typename T, int DH>
__global__ void __launch_bounds__(128) k_attn_simt(const T* __restrict__ q, const T* __restrict__ cache_k,
                                                   const T* __restrict__ cache_v, const T* __restrict__ stage_k,
                                                   const T* __restrict__ stage_v, T* __restrict__ out, StepDesc sd,
                                                   int n_heads, int n_kv_heads, size_t cache_seq_elems,
                                                   float scale, int inplace) {
  __shared__ float Qs[AS_BQ][DH];
  __shared__ float Ks[AS_BK][DH + 1];
  __shared__ float Vs[AS_BK][DH];
  pdl_begin();
  const int b = blockIdx.z, h = blockIdx.y;
  const int r0 = sd.row_off[b];
  const int Qn = sd.row_off[b + 1] - r0;
  const int q0 = blockIdx.x * AS_BQ;
  if (q0 >= Qn) return;
  const int S = sd.F[b] + Qn;
  const int F = inplace ? S : sd.F[b];      // in-place layout: this pass's K/V rows already sit behind the prefix in the cache
  const int kvh = h / (n_heads / n_kv_heads);
  const int ldq = n_heads * DH, ldkv = n_kv_heads * DH;
  const int t = threadIdx.x, lane = t & 31, w = t >> 5;
  for (int i = t; i < AS_BQ * DH; i += 128) {
    const int qi = i / DH, d = i % DH;
    Qs[qi][d] = (q0 + qi < Qn) ? to_f(q[(size_t)(r0 + q0 + qi) * ldq + h * DH + d]) : 0.f;
  }
  constexpr int NC = DH / 32;
  float acc[4][NC];
  float m_run[4], l_run[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    m_run[i] = -INFINITY;
    l_run[i] = 0.f;
#pragma unroll
    for (int c = 0; c < NC; ++c) acc[i][c] = 0.f;
  }
  const T* ck = cache_k + (size_t)b * cache_seq_elems + kvh * DH;
  const T* cv = cache_v + (size_t)b * cache_seq_elems + kvh * DH;
  const T* sk = stage_k + (size_t)r0 * ldkv + kvh * DH;
  const T* sv = stage_v + (size_t)r0 * ldkv + kvh * DH;
  for (int s0 = 0; s0 < S; s0 += AS_BK) {
    __syncthreads();
    {
      const int key = t >> 2, part = (t & 3) * (DH / 4);
      const int s = s0 + key;
      const T* kp = nullptr;
      const T* vp = nullptr;
      if (s < F) { kp = ck + (size_t)s * ldkv; vp = cv + (size_t)s * ldkv; }
      else if (s < S) { kp = sk + (size_t)(s - F) * ldkv; vp = sv + (size_t)(s - F) * ldkv; }
#pragma unroll 4
      for (int d = 0; d < DH / 4; ++d) {
        Ks[key][part + d] = kp ? to_f(kp[part + d]) : 0.f;
        Vs[key][part + d] = vp ? to_f(vp[part + d]) : 0.f;
      }
    }
    __syncthreads();
    const bool kvalid = (s0 + lane) < S;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int qi = w * 4 + i;
      float dot = 0.f;
#pragma unroll 8
      for (int d = 0; d < DH; ++d) dot = fmaf(Qs[qi][d], Ks[lane][d], dot);
      const float sc = kvalid ? dot * scale : -INFINITY;
      const float m_new = fmaxf(m_run[i], warp_max(sc));
      const float p = kvalid ? __expf(sc - m_new) : 0.f;
      const float corr = __expf(m_run[i] - m_new);
      l_run[i] = l_run[i] * corr + warp_sum(p);
      m_run[i] = m_new;
#pragma unroll
      for (int c = 0; c < NC; ++c) acc[i][c] *= corr;
      for (int k = 0; k < AS_BK; ++k) {
        const float pk = __shfl_sync(0xffffffffu, p, k);
#pragma unroll
        for (int c = 0; c < NC; ++c) acc[i][c] = fmaf(pk, Vs[k][lane + 32 * c], acc[i][c]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int qq = q0 + w * 4 + i;
    if (qq >= Qn) continue;
    const float inv = 1.f / l_run[i];
#pragma unroll
    for (int c = 0; c < NC; ++c)
      out[(size_t)(r0 + qq) * ldq + h * DH + lane + 32 * c] = from_f<T>(acc[i][c] * inv);
  }
}

}  // namespace lsp
