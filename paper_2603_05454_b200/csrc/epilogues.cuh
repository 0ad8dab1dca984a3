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
  // K/V destination row of packed row m: m itself (staging planes), or, with seq_stride > 0, the row's own cache slot
  // row_seq[m] * seq_stride + row_pos[m] (k_stage / v_stage then point at the cache planes: the in-place layout)
  const int* row_seq = nullptr;
  int seq_stride = 0;
  __device__ __forceinline__ size_t kv_row(int m) const {
    return seq_stride > 0 ? (size_t)row_seq[m] * seq_stride + row_pos[m] : (size_t)m;
  }
  __device__ __forceinline__ int row0(int j) const { return (j / half) * 2 * half + (j % half); }
  __device__ __forceinline__ int row1(int j) const { return row0(j) + half; }
  __device__ __forceinline__ void elem(int m, int j, float a0, float a1) const {
    const int h = j / half, i = j % half;
    const int dh = 2 * half;
    if (h >= n_heads && seq_stride > 0 && row_seq[m] < 0) return;      // in-place layout: a row of no sequence has no cache slot
    if (h < n_heads + n_kv_heads) {
      const float2 c = cs[(size_t)row_pos[m] * half + i];
      const float r0 = a0 * c.x - a1 * c.y;
      const float r1 = a1 * c.x + a0 * c.y;
      T* dst = (h < n_heads) ? q_out + (size_t)m * n_heads * dh + h * dh
                             : k_stage + kv_row(m) * n_kv_heads * dh + (h - n_heads) * dh;
      dst[i] = from_f<T>(r0);
      dst[i + half] = from_f<T>(r1);
    } else {
      T* dst = v_stage + kv_row(m) * n_kv_heads * dh + (h - n_heads - n_kv_heads) * dh;
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

// Sixteen consecutive logits z[0..15] of columns col0.. pushed into the running reduction without data-dependent
// branches: the top-2 state by compare-and-select per element (strict ">" keeps the lowest id on ties, as top2_push),
// the sum rescaled once per chunk to the new maximum and the sixteen exponentials independent of one another.
// Equivalent to sixteen top2_push calls up to the rounding of the sum.
__device__ __forceinline__ void top2_push16(Top2& t, const float* z, int col0, const EpiHead& e) {
  float v[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = e.valid(col0 + i) ? z[i] : -INFINITY;
  float cm = v[0];
#pragma unroll
  for (int i = 1; i < 16; ++i) cm = fmaxf(cm, v[i]);
  if (cm == -INFINITY) return;                       // nothing valid in this chunk (uniform per thread, rare)
  const float m_new = fmaxf(t.m1, cm);
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < 16; ++i) sum += __expf(v[i] - m_new);          // exp(-inf) = 0 for the masked columns
  t.s = t.s * __expf(t.m1 - m_new) + sum;            // t.m1 = -inf on the first chunk: exp(-inf) = 0, t.s = 0
  float m1 = t.m1, m2 = t.m2;
  int i1 = t.i1;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const bool gt = v[i] > m1;
    m2 = gt ? m1 : fmaxf(m2, v[i]);
    i1 = gt ? col0 + i : i1;
    m1 = gt ? v[i] : m1;
  }
  t.m1 = m1;
  t.m2 = m2;
  t.i1 = i1;
}

}  // namespace lsp
