// CUDA-core GEMM (fp32 accumulate) with the shared epilogues.  It is the compute path of fp32 models and
// the reference implementation the tcgen05 kernels can be switched against; it is not tuned.
#pragma once
#include "epilogues.cuh"

namespace lsp {

__device__ __forceinline__ void load4(const float* p, float (&v)[4]) {
  const float4 t = *reinterpret_cast<const float4*>(p);
  v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
__device__ __forceinline__ void load4(const bf16* p, float (&v)[4]) {
  const uint2 t = *reinterpret_cast<const uint2*>(p);
  const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&t.x);
  const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&t.y);
  v[0] = __low2float(a); v[1] = __high2float(a); v[2] = __low2float(b); v[3] = __high2float(b);
}

constexpr int SG_BM = 64, SG_BN = 64, SG_BK = 16;

// grid = (ceil(NP / 64), ceil(M / 64)), block = 256.  A: [M, K]; W0/W1: [*, K] row-major.
template <typename T, typename Epi>
__global__ void __launch_bounds__(256) k_gemm_simt(const T* __restrict__ A, const T* __restrict__ W0,
                                                   const T* __restrict__ W1, int M, int NP, int K, Epi epi) {
  __shared__ float As[SG_BK][SG_BM + 4];
  __shared__ float B0s[SG_BK][SG_BN + 4];
  __shared__ float B1s[Epi::kDual ? SG_BK : 1][SG_BN + 4];
  pdl_begin();
  const int t = threadIdx.x;
  const int m0 = blockIdx.y * SG_BM, j0 = blockIdx.x * SG_BN;
  const int lrow = t >> 2, lk = (t & 3) * 4;
  const int am = m0 + lrow;
  const int bj = j0 + lrow;
  const T* ap = (am < M) ? A + (size_t)am * K + lk : nullptr;
  const T* b0p = (bj < NP) ? W0 + (size_t)epi.row0(bj) * K + lk : nullptr;
  const T* b1p = (Epi::kDual && bj < NP) ? W1 + (size_t)epi.row1(bj) * K + lk : nullptr;
  const int ty = t >> 4, tx = t & 15;
  float acc0[4][4] = {}, acc1[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += SG_BK) {
    float v[4] = {0.f, 0.f, 0.f, 0.f};
    if (ap) load4(ap + k0, v);
#pragma unroll
    for (int i = 0; i < 4; ++i) As[lk + i][lrow] = v[i];
    float w[4] = {0.f, 0.f, 0.f, 0.f};
    if (b0p) load4(b0p + k0, w);
#pragma unroll
    for (int i = 0; i < 4; ++i) B0s[lk + i][lrow] = w[i];
    if (Epi::kDual) {
      float u[4] = {0.f, 0.f, 0.f, 0.f};
      if (b1p) load4(b1p + k0, u);
#pragma unroll
      for (int i = 0; i < 4; ++i) B1s[lk + i][lrow] = u[i];
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < SG_BK; ++kk) {
      float a[4], b0[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[kk][ty * 4 + i]; b0[i] = B0s[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc0[i][j] = fmaf(a[i], b0[j], acc0[i][j]);
      if (Epi::kDual) {
        float b1[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) b1[i] = B1s[kk][tx * 4 + i];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc1[i][j] = fmaf(a[i], b1[j], acc1[i][j]);
      }
    }
    __syncthreads();
  }
  if constexpr (Epi::kReduce) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int m = m0 + ty * 4 + i;
      Top2 r = top2_empty();
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int col = j0 + tx * 4 + j;
        if (epi.valid(col)) top2_push(r, acc0[i][j], col);
      }
#pragma unroll
      for (int o = 1; o < 16; o <<= 1) r = top2_merge(r, top2_shfl_xor(r, o));
      if (tx == 0 && m < M) epi.part[(size_t)m * epi.n_tiles + blockIdx.x] = r;
    }
  } else {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int m = m0 + ty * 4 + i;
      if (m >= M) continue;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int col = j0 + tx * 4 + j;
        if (col < NP) epi.elem(m, col, acc0[i][j], acc1[i][j]);
      }
    }
  }
}

}  // namespace lsp
