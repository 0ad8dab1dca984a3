// GEMM epilogues shared by the CUDA-core and the tcgen05 GEMM kernels.
//
// A GEMM here computes, for activation row m and "pair index" j, two fp32 accumulators
//   a0 = sum_k A[m,k] * W0[row0(j), k]        a1 = sum_k A[m,k] * W1[row1(j), k]
// and hands them to the epilogue.  Plain epilogues ignore a1 (kDual = false).  Pairing exists so that the
// two values an element-wise fusion needs sit in the same thread:
//   * SwiGLU: W0 = gate, W1 = up, same row j                     -> silu(a0) * a1
//   * rotary: W0 = W1 = fused QKV weight, rows (n, n + head_dim/2) -> the rotate-half pair
#pragma once
#include "common.cuh"

namespace lsp {

// out[m, j] = a0
template <typename T>
struct EpiStore {
  static constexpr bool kDual = false;
  static constexpr bool kReduce = false;
  T* out;
  int ld;
  __device__ __forceinline__ int row0(int j) const { return j; }
  __device__ __forceinline__ int row1(int j) const { return j; }
  __device__ __forceinline__ void elem(int m, int j, float a0, float) const {
    out[(size_t)m * ld + j] = from_f<T>(a0);
  }
};

// x[m, j] = round(x[m, j] + a0)   (residual-stream update)
template <typename T>
struct EpiResidual {
  static constexpr bool kDual = false;
  static constexpr bool kReduce = false;
  T* x;
  int ld;
  __device__ __forceinline__ int row0(int j) const { return j; }
  __device__ __forceinline__ int row1(int j) const { return j; }
  __device__ __forceinline__ void elem(int m, int j, float a0, float) const {
    T* p = x + (size_t)m * ld + j;
    *p = from_f<T>(to_f(*p) + a0);
  }
};

// out[m, j] = silu(gate) * up, fp32 then rounded
template <typename T>
struct EpiSwiGLU {
  static constexpr bool kDual = true;
  static constexpr bool kReduce = false;
  T* out;
  int ld;
  __device__ __forceinline__ int row0(int j) const { return j; }
  __device__ __forceinline__ int row1(int j) const { return j; }
  __device__ __forceinline__ void elem(int m, int j, float g, float u) const {
    out[(size_t)m * ld + j] = from_f<T>(g / (1.f + __expf(-g)) * u);
  }
};

// Fused QKV projection: pair index j = head * (dh/2) + i over all (n_heads + 2 n_kv_heads) heads.
// Query and key heads are rotated by the row's absolute position (fp32, on the accumulators), value heads
// pass through.  Q goes to q_out[m, head*dh + .], K and V to the staging planes in cache row layout.
template <typename T>
struct EpiQKVRope {
  static constexpr bool kDual = true;
  static constexpr bool kReduce = false;
  T* q_out;         // [M, n_heads * dh]
  T* k_stage;       // [M, n_kv_heads * dh]
  T* v_stage;       // [M, n_kv_heads * dh]
  const float2* cs; // [max_len, dh/2] (cos, sin)
  const int* row_pos;
  int n_heads, n_kv_heads, half; // half = dh / 2
  __device__ __forceinline__ int row0(int j) const { return (j / half) * 2 * half + (j % half); }
  __device__ __forceinline__ int row1(int j) const { return row0(j) + half; }
  __device__ __forceinline__ void elem(int m, int j, float a0, float a1) const {
    const int h = j / half, i = j % half;
    const int dh = 2 * half;
    if (h < n_heads + n_kv_heads) {
      const float2 c = cs[(size_t)row_pos[m] * half + i];
      const float r0 = a0 * c.x - a1 * c.y;
      const float r1 = a1 * c.x + a0 * c.y;
      T* dst = (h < n_heads) ? q_out + (size_t)m * n_heads * dh + h * dh
                             : k_stage + (size_t)m * n_kv_heads * dh + (h - n_heads) * dh;
      dst[i] = from_f<T>(r0);
      dst[i + half] = from_f<T>(r1);
    } else {
      T* dst = v_stage + (size_t)m * n_kv_heads * dh + (h - n_heads - n_kv_heads) * dh;
      dst[i] = from_f<T>(a0);
      dst[i + half] = from_f<T>(a1);
    }
  }
};

// LM head: no store of logits.  The kernel reduces each row of its vocab tile to a Top2 partial
// (Eq. 1's two largest logits, the argmax id, and the softmax denominator) and writes it to
// part[m * n_tiles + tile].  Columns >= vocab and the excluded id are skipped.
struct EpiHead {
  static constexpr bool kDual = false;
  static constexpr bool kReduce = true;
  Top2* part;
  int n_tiles;
  int vocab;
  int exclude_id; // -1 = none
  __device__ __forceinline__ int row0(int j) const { return j; }
  __device__ __forceinline__ int row1(int j) const { return j; }
  __device__ __forceinline__ bool valid(int j) const { return j < vocab && j != exclude_id; }
};

}  // namespace lsp
