// Tensor-core flash-style attention for bf16: suffix queries over [contiguous prefix cache | this pass's staged
// rows], non-causal (every query sees every key: the bidirectional lookahead of Sec. 3.2), MHA and GQA.
//
// One CTA (4 warps) owns 64 "rows" of one (sequence, KV head): a row is a (query position, query head of the
// group) pair, so with grouped-query attention the heads that share a KV head also share each K/V tile.
// K/V tiles of 64 keys are streamed once, contiguously (the cache is position-major per sequence, so a tile is
// one contiguous run of 128-bit loads per row), through a two-deep cp.async pipeline into padded shared memory;
// QK^T and PV run on mma.sync m16n8k16 (bf16 in, fp32 accumulate) with an fp32 online softmax.
// This step is bound by streaming K/V from HBM whenever rows * group <= ~200 (the decode regime).
#pragma once
#include "common.cuh"

namespace lsp {

constexpr int AM_BM = 64;
constexpr int AM_BN = 64;

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int bytes = valid ? 16 : 0;   // 0 source bytes = zero fill
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

template <int DH>
constexpr int attn_mma_smem_bytes() { return (AM_BM + 4 * AM_BN) * (DH + 8) * 2; }

// grid = (ceil(max_rows_per_seq * group / 64), n_kv_heads, batch), block = 128, dynamic smem = attn_mma_smem_bytes.
template <int DH>
__global__ void __launch_bounds__(128) k_attn_mma(const bf16* __restrict__ q, const bf16* __restrict__ cache_k,
                                                  const bf16* __restrict__ cache_v, const bf16* __restrict__ stage_k,
                                                  const bf16* __restrict__ stage_v, bf16* __restrict__ out, StepDesc sd,
                                                  int n_heads, int n_kv_heads, size_t cache_seq_elems,
                                                  float scale_log2, int inplace) {
  constexpr int LD = DH + 8;            // padded row (elements): 16-byte shift per row, conflict-free ldmatrix
  constexpr int CPR = DH / 8;           // 16-byte chunks per row
  extern __shared__ __align__(16) uint8_t attn_smem[];
  pdl_begin();
  bf16* Qs = reinterpret_cast<bf16*>(attn_smem);
  bf16* Ks = Qs + AM_BM * LD;           // [2][AM_BN][LD]
  bf16* Vs = Ks + 2 * AM_BN * LD;       // [2][AM_BN][LD]
  const int b = blockIdx.z, kvh = blockIdx.y;
  const int G = n_heads / n_kv_heads;
  const int r0 = sd.row_off[b];
  const int Qn = sd.row_off[b + 1] - r0;
  const int rows_total = Qn * G;
  const int row_base = blockIdx.x * AM_BM;
  if (row_base >= rows_total) return;
  const int S = sd.F[b] + Qn;
  const int F = inplace ? S : sd.F[b];      // in-place layout: this pass's K/V rows already sit behind the prefix in the cache
  const int ldq = n_heads * DH, ldkv = n_kv_heads * DH;
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  const bf16* ck = cache_k + (size_t)b * cache_seq_elems + kvh * DH;
  const bf16* cv = cache_v + (size_t)b * cache_seq_elems + kvh * DH;
  const bf16* sk = stage_k + (size_t)r0 * ldkv + kvh * DH;
  const bf16* sv = stage_v + (size_t)r0 * ldkv + kvh * DH;

  // ---- Q tile -> smem
  for (int i = tid; i < AM_BM * CPR; i += 128) {
    const int r = i / CPR, ch = i % CPR;
    const int row = row_base + r;
    const bool valid = row < rows_total;
    const int qi = valid ? row / G : 0, hg = valid ? row % G : 0;
    const bf16* src = q + (size_t)(r0 + qi) * ldq + (kvh * G + hg) * DH + ch * 8;
    cp_async16(smem_u32(Qs + r * LD + ch * 8), src, valid);
  }
  auto load_kv = [&](int tile, int buf) {
    const int s0 = tile * AM_BN;
    bf16* kd = Ks + buf * AM_BN * LD;
    bf16* vd = Vs + buf * AM_BN * LD;
    for (int i = tid; i < AM_BN * CPR; i += 128) {
      const int r = i / CPR, ch = i % CPR;
      const int s = s0 + r;
      const bool valid = s < S;
      const bf16* kp = ck;
      const bf16* vp = cv;
      if (valid) {
        if (s < F) { kp = ck + (size_t)s * ldkv; vp = cv + (size_t)s * ldkv; }
        else { kp = sk + (size_t)(s - F) * ldkv; vp = sv + (size_t)(s - F) * ldkv; }
      }
      cp_async16(smem_u32(kd + r * LD + ch * 8), kp + ch * 8, valid);
      cp_async16(smem_u32(vd + r * LD + ch * 8), vp + ch * 8, valid);
    }
  };
  const int n_tiles = (S + AM_BN - 1) / AM_BN;
  load_kv(0, 0);
  cp_async_commit();

  float o[DH / 8][4];
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  uint32_t qf[DH / 16][4];
  const int g = lane >> 2, t = lane & 3;

  for (int tile = 0; tile < n_tiles; ++tile) {
    const int buf = tile & 1;
    if (tile + 1 < n_tiles) {
      load_kv(tile + 1, buf ^ 1);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    if (tile == 0) {
      // Q fragments (A operand): rows w*16 .. +15
#pragma unroll
      for (int kk = 0; kk < DH / 16; ++kk) {
        const int row = w * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        const int col = kk * 16 + (lane >> 4) * 8;
        ldsm_x4(smem_u32(Qs + row * LD + col), qf[kk][0], qf[kk][1], qf[kk][2], qf[kk][3]);
      }
    }
    const bf16* kt = Ks + buf * AM_BN * LD;
    const bf16* vt = Vs + buf * AM_BN * LD;
    // ---- S = Q K^T for this key tile: 16 rows x 64 keys per warp
    float sacc[AM_BN / 8][4];
#pragma unroll
    for (int j = 0; j < AM_BN / 8; ++j) { sacc[j][0] = sacc[j][1] = sacc[j][2] = sacc[j][3] = 0.f; }
#pragma unroll
    for (int kk = 0; kk < DH / 16; kk += 2) {
#pragma unroll
      for (int j = 0; j < AM_BN / 8; ++j) {
        uint32_t b0, b1, b2, b3;
        const int row = j * 8 + (lane & 7);
        const int col = kk * 16 + (lane >> 3) * 8;
        ldsm_x4(smem_u32(kt + row * LD + col), b0, b1, b2, b3);
        mma_bf16(sacc[j], qf[kk][0], qf[kk][1], qf[kk][2], qf[kk][3], b0, b1);
        mma_bf16(sacc[j], qf[kk + 1][0], qf[kk + 1][1], qf[kk + 1][2], qf[kk + 1][3], b2, b3);
      }
    }
    // ---- online softmax (rows g and g+8 of this warp's 16)
    const int s0 = tile * AM_BN;
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int j = 0; j < AM_BN / 8; ++j) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int key = s0 + j * 8 + 2 * t + (e & 1);
        const float v = (key < S) ? sacc[j][e] * scale_log2 : -INFINITY;
        sacc[j][e] = v;
        mx[e >> 1] = fmaxf(mx[e >> 1], v);
      }
    }
    float corr[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
      mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
      const float m_new = fmaxf(m_run[h], mx[h]);       // finite: every tile has at least one valid key
      corr[h] = exp2f(m_run[h] - m_new);
      m_run[h] = m_new;
    }
    float ls[2] = {0.f, 0.f};
#pragma unroll
    for (int j = 0; j < AM_BN / 8; ++j) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float p = exp2f(sacc[j][e] - m_run[e >> 1]);
        sacc[j][e] = p;
        ls[e >> 1] += p;
      }
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      ls[h] += __shfl_xor_sync(0xffffffffu, ls[h], 1);
      ls[h] += __shfl_xor_sync(0xffffffffu, ls[h], 2);
      l_run[h] = l_run[h] * corr[h] + ls[h];
    }
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) {
      o[i][0] *= corr[0]; o[i][1] *= corr[0];
      o[i][2] *= corr[1]; o[i][3] *= corr[1];
    }
    // ---- O += P V
#pragma unroll
    for (int kk = 0; kk < AM_BN / 16; ++kk) {
      const uint32_t a0 = pack_bf16(sacc[2 * kk][0], sacc[2 * kk][1]);
      const uint32_t a1 = pack_bf16(sacc[2 * kk][2], sacc[2 * kk][3]);
      const uint32_t a2 = pack_bf16(sacc[2 * kk + 1][0], sacc[2 * kk + 1][1]);
      const uint32_t a3 = pack_bf16(sacc[2 * kk + 1][2], sacc[2 * kk + 1][3]);
#pragma unroll
      for (int nt = 0; nt < DH / 8; nt += 2) {
        uint32_t b0, b1, b2, b3;
        const int row = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        const int col = nt * 8 + (lane >> 4) * 8;
        ldsm_x4_t(smem_u32(vt + row * LD + col), b0, b1, b2, b3);
        mma_bf16(o[nt], a0, a1, a2, a3, b0, b1);
        mma_bf16(o[nt + 1], a0, a1, a2, a3, b2, b3);
      }
    }
    __syncthreads();   // the buffer is refilled two iterations from now
  }
  // ---- normalise and store
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int row = row_base + w * 16 + g + 8 * h;
    if (row >= rows_total) continue;
    const int qi = row / G, hg = row % G;
    bf16* dst = out + (size_t)(r0 + qi) * ldq + (kvh * G + hg) * DH;
    const float inv = 1.f / l_run[h];
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) {
      const uint32_t v = pack_bf16(o[i][2 * h] * inv, o[i][2 * h + 1] * inv);
      *reinterpret_cast<uint32_t*>(dst + i * 8 + 2 * t) = v;
    }
  }
}

}  // namespace lsp
