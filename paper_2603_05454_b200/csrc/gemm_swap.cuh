// bf16 GEMM with the operands swapped, for passes of 129..256 activation rows.
//
//   acc[c, m] = sum_k Wt[c, k] * A[m, k]        the transpose of the product k_gemm_stream computes
//
// tcgen05.mma produces 128 accumulator rows per instruction whatever the problem needs, so with the activations as
// the M-side operand 138 rows cost the tensor pipe as much as 256 (two row tiles), and in this row range the tensor
// pipe is what bounds a layer GEMM.  Here the 128-row side is a block of 128 weight rows and the activation rows are
// the N side, which the instruction takes in steps of 16: the tensor time follows the real row count.
//
// One CTA owns a tile of NACC blocks of 128 weight rows (NACC accumulators of `nr` columns each in tensor memory,
// nr = rows rounded up to 16) and one K slice; the K slices of a tile form a thread block cluster of 1, 2 or 4 CTAs.
// The shared-memory stage is the one k_gemm_stream uses (activation box, then the weight tile as two box groups, so
// that accumulator 0 and accumulator 1 hold the pair a fused epilogue needs: gate / up, rotate-half partners; for a
// plain epilogue with NACC = 2 they are simply columns j and j + 128).
// Epilogue: thread (warp quarter, lane) owns weight row n of each accumulator and walks the activation rows 16 at a
// time, so the fused epilogues run element-wise (epiT16 below); a warp stores 32 consecutive output features of one
// row at a time.
// Split K: rank r of the cluster finishes the r-th share of the 16-row chunks; it publishes the other chunks of its
// partial accumulators in its own shared memory (the pipeline stages are idle by then), and after a cluster barrier
// adds, for its chunks, the other ranks' pieces (in rank order, so the result does not depend on timing) to what it
// kept in tensor memory.
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = TMEM allocator + MMA issuer, warps 2..5 = epilogue.
// Every wait is bounded; on expiry the kernel records (code, site) in the status word, drains and returns.
#pragma once
#include "gemm_stream.cuh"

namespace lsp {

constexpr int SW_THREADS = 192;
constexpr int SW_MAX_STAGES = 8;

struct SwapArgs {
  int M;          // activation rows
  int n_pairs;    // dual: pair indices; plain: output columns
  int kc;         // K chunks of 64 elements per CTA (its K slice)
  int nr;         // activation rows rounded up to 16: the MMA's N and the activation box's rows
  int box_rows;   // weight rows per TMA box (a divisor of 64 NACC)
  int stages;
  int cluster;    // CTAs per tile (K slices): 1, 2 or 4
  unsigned* status;
};

__device__ __forceinline__ float ld_cluster_f32(uint32_t addr) {
  float v;
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
  return v;
}

__device__ __forceinline__ float4 ld_cluster_v4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
}

// Transposed epilogues: one thread holds output feature j (a pair index for the paired epilogues) of the `cnt` (<= 16)
// consecutive activation rows m0 .. m0 + cnt - 1.  Everything a row needs from memory is fetched for all rows first
// (the stores of one row could alias the loads of the next as far as the compiler can tell, which would put one memory
// round trip per row on the critical path); a warp writes 32 consecutive features of one row at a time.
__device__ __forceinline__ void epiT16(const EpiStore<bf16>& e, int m0, int cnt, int j, const float* a0, const float*) {
#pragma unroll
  for (int i = 0; i < 16; ++i)
    if (i < cnt) e.out[(size_t)(m0 + i) * e.ld + j] = __float2bfloat16_rn(a0[i]);
}
__device__ __forceinline__ void epiT16(const EpiResidual<bf16>& e, int m0, int cnt, int j, const float* a0, const float*) {
  float old[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) old[i] = i < cnt ? __bfloat162float(e.x[(size_t)(m0 + i) * e.ld + j]) : 0.f;
#pragma unroll
  for (int i = 0; i < 16; ++i)
    if (i < cnt) e.x[(size_t)(m0 + i) * e.ld + j] = __float2bfloat16_rn(old[i] + a0[i]);
}
__device__ __forceinline__ void epiT16(const EpiSwiGLU<bf16>& e, int m0, int cnt, int j, const float* g, const float* u) {
#pragma unroll
  for (int i = 0; i < 16; ++i)
    if (i < cnt) e.out[(size_t)(m0 + i) * e.ld + j] = __float2bfloat16_rn(__fdividef(g[i], 1.f + __expf(-g[i])) * u[i]);
}
__device__ __forceinline__ void epiT16(const EpiQKVRope<bf16>& e, int m0, int cnt, int j, const float* a0, const float* a1) {
  const int h = j / e.half, ii = j % e.half, dh = 2 * e.half;
  const bool rot = h < e.n_heads + e.n_kv_heads;
  float2 cs[16];
  size_t dst[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    cs[i] = make_float2(1.f, 0.f);
    dst[i] = ~(size_t)0;
    if (i < cnt) {
      const int m = m0 + i;
      if (rot) cs[i] = __ldg(e.cs + (size_t)__ldg(e.row_pos + m) * e.half + ii);
      if (h < e.n_heads) dst[i] = (size_t)m * e.n_heads * dh + (size_t)h * dh + ii;
      else if (e.seq_stride > 0 && __ldg(e.row_seq + m) < 0) dst[i] = ~(size_t)0;      // in-place layout: a row of no sequence
      else dst[i] = e.kv_row(m) * e.n_kv_heads * dh + (size_t)(h - e.n_heads - (rot ? 0 : e.n_kv_heads)) * dh + ii;
    }
  }
  bf16* base = h < e.n_heads ? e.q_out : (rot ? e.k_stage : e.v_stage);
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    if (i < cnt && dst[i] != ~(size_t)0) {
      base[dst[i]] = __float2bfloat16_rn(a0[i] * cs[i].x - a1[i] * cs[i].y);
      base[dst[i] + e.half] = __float2bfloat16_rn(a1[i] * cs[i].x + a0[i] * cs[i].y);
    }
  }
}

template <int NACC, typename Epi>
__global__ void __launch_bounds__(SW_THREADS, 1)
k_gemm_swap(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b0,
            const __grid_constant__ CUtensorMap map_b1, SwapArgs args, Epi epi) {
  extern __shared__ uint8_t smem_raw[];
  pdl_release();
  static_assert(NACC == 1 || NACC == 2, "one or two blocks of 128 weight rows per tile");
  static_assert(!Epi::kReduce, "the reducing head epilogue keeps the row-major kernel");
  static_assert(!Epi::kDual || NACC == 2, "paired epilogues need both accumulators");
  constexpr int BN = 128 * NACC;                 // weight rows per tile
  constexpr int HALF = BN / 2;                   // weight rows per box group
  constexpr int B_BYTES = BN * 128;              // one 64-element K chunk of the weight tile
  const int NR = args.nr;
  const int A_BYTES = NR * 128;
  const int STAGE_BYTES = A_BYTES + B_BYTES;
  const uint32_t TMEM_COLS = NACC * NR <= 32 ? 32u : (NACC * NR <= 64 ? 64u : (NACC * NR <= 128 ? 128u : (NACC * NR <= 256 ? 256u : 512u)));
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int S = args.stages;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)S * STAGE_BYTES);
  // bars[0..S) full, [S..2S) empty, [2S] accumulators complete
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * S + 1);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  volatile uint32_t* epi_fail = tmem_slot + 2;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (S + s); };
  const uint32_t acc_bar = bar_base + 8u * (2 * S);

  const int C = args.cluster;
  const int rank = C > 1 ? (int)cluster_ctarank() : 0;
  const int tile = blockIdx.x / C;
  const int kc = args.kc;
  const int k_first = rank * kc;                 // first 64-element K chunk of this CTA's slice

  auto load_weights = [&](int c, int s) {
    const uint32_t sb = smem_u32(smem + (size_t)s * STAGE_BYTES) + A_BYTES;
    const int k0 = (k_first + c) * UM_BK;
    for (int b = 0; b < HALF; b += args.box_rows) {
      int row_b0, row_b1;
      if (Epi::kDual) { row_b0 = epi.row0(tile * HALF + b); row_b1 = epi.row1(tile * HALF + b); }
      else { row_b0 = tile * BN + b; row_b1 = tile * BN + HALF + b; }
      tma_load_2d(sb + b * 128, &map_b0, k0, row_b0, full_bar(s));
      tma_load_2d(sb + HALF * 128 + b * 128, &map_b1, k0, row_b1, full_bar(s));
    }
  };
  const int n_pre = kc < S ? kc : S;
  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    mbar_init(acc_bar, 1);
    *abort_flag = 0;
    *epi_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    // weights are never written by any kernel: the first stages' weight tiles are requested while the preceding kernel
    // (launched with programmatic serialisation) is still running; this thread is also the producer below
    for (int c = 0; c < n_pre; ++c) {
      mbar_expect_tx(full_bar(c), STAGE_BYTES);
      load_weights(c, c);
    }
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int issued = 0, s = 0;
      uint32_t ph = 0;
      for (int c = 0; c < kc; ++c) {
        if (c >= n_pre) {
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) {
            if (!*abort_flag) { *abort_flag = 1; atomicExch(args.status, 1u); args.status[1] = 31u; }
            break;
          }
          mbar_expect_tx(full_bar(s), STAGE_BYTES);
          load_weights(c, s);
        }
        tma_load_2d(smem_u32(smem + (size_t)s * STAGE_BYTES), &map_a, (k_first + c) * UM_BK, 0, full_bar(s));
        ++issued;
        if (++s == S) { s = 0; ph ^= 1u; }
      }
      // do not leave while copies may still be landing in this CTA's shared memory
      for (int c = issued > S ? issued - S : 0; c < issued; ++c) {
        volatile uint32_t no_abort = 0;
        mbar_wait(full_bar(c % S), (uint32_t)(c / S) & 1u, &no_abort);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      const uint32_t idesc = make_idesc(NR);
      bool ok = true;
      int s = 0;
      uint32_t ph = 0;
      for (int c = 0; c < kc; ++c) {
        if (!mbar_wait(full_bar(s), ph, abort_flag)) {
          if (!*abort_flag) { *abort_flag = 1; atomicExch(args.status, 1u); args.status[1] = 32u; }
          ok = false;
          break;
        }
        tc_fence_after();
        const uint32_t sa = smem_u32(smem + (size_t)s * STAGE_BYTES);
        const uint64_t dact = make_smem_desc(sa);                     // N-side operand: the activation rows
        const uint64_t dw = make_smem_desc(sa + A_BYTES);             // M-side operand: 128 weight rows per accumulator
#pragma unroll
        for (int k = 0; k < 4; ++k) {
#pragma unroll
          for (int a = 0; a < NACC; ++a)
            tc_mma_f16(tmem_base + (uint32_t)(a * NR), dw + (uint64_t)(a * 1024 + 2 * k), dact + (uint64_t)(2 * k), idesc,
                       (c | k) != 0 ? 1u : 0u);
        }
        tc_commit(empty_bar(s));
        if (++s == S) { s = 0; ph ^= 1u; }
      }
      if (ok) tc_commit(acc_bar);
    }
  }
  // ---------------- epilogue (warps 2..5) ----------------
  const int q = warp & 3;
  const int n = q * 32 + lane;                                  // weight row within an accumulator = TMEM lane
  const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16);
  const int NCH = NR / 16;                                      // chunks of 16 activation rows
  const int lo = NCH * rank / C, hi = NCH * (rank + 1) / C;     // this rank's chunks
  auto compact = [&](int ch, int p) {                           // index of chunk ch in rank p's published piece
    const int plo = NCH * p / C, phi = NCH * (p + 1) / C;
    return ch < plo ? ch : ch - (phi - plo);
  };
  bool ok = true;
  if (warp >= 2) {
    ok = mbar_wait(acc_bar, 0u, abort_flag);
    if (!ok) *epi_fail = 1;
    asm volatile("bar.sync 1, 128;" ::: "memory");               // the four epilogue warps agree on the outcome
    ok = (*epi_fail == 0);
    if (!ok) {
      if (lane == 0 && !*abort_flag) { *abort_flag = 1; atomicExch(args.status, 1u); args.status[1] = 33u; }
    } else if (C > 1) {
      // publish the chunks other ranks finish: [compact chunk][accumulator][group of 4 rows][128 lanes] float4
      tc_fence_after();
      float4* pub = reinterpret_cast<float4*>(smem);
#pragma unroll 1
      for (int ch = 0; ch < NCH; ++ch) {
        if (ch >= lo && ch < hi) continue;
        const int cc = compact(ch, rank);
#pragma unroll
        for (int a = 0; a < NACC; ++a) {
          float v[16];
          tc_ld16(t_row + (uint32_t)(a * NR + ch * 16), v);
#pragma unroll
          for (int g = 0; g < 4; ++g)
            pub[((cc * NACC + a) * 4 + g) * 128 + n] = make_float4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
        }
      }
    }
  }
  if (C > 1) cluster_sync();          // every thread of every CTA of the cluster reaches both barriers
  if (warp >= 2 && ok) {
    tc_fence_after();
    const int j = tile * (Epi::kDual ? HALF : BN) + n;          // pair index (dual) or output column of accumulator 0
    const uint32_t pub_base = smem_u32(smem);
#pragma unroll 1
    for (int ch = lo; ch < hi; ++ch) {
      float a0[16], a1[16];
      tc_ld16(t_row + (uint32_t)(ch * 16), a0);
      if (NACC == 2) tc_ld16(t_row + (uint32_t)(NR + ch * 16), a1);
      for (int p = 0; p < C; ++p) {
        if (p == rank) continue;
        const uint32_t peer = cluster_map(pub_base, (unsigned)p);
        const int cc = compact(ch, p);
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          const float4 t0 = ld_cluster_v4(peer + (uint32_t)((((cc * NACC + 0) * 4 + g) * 128 + n) * 16));
          a0[4 * g] += t0.x; a0[4 * g + 1] += t0.y; a0[4 * g + 2] += t0.z; a0[4 * g + 3] += t0.w;
          if (NACC == 2) {
            const float4 t1 = ld_cluster_v4(peer + (uint32_t)((((cc * NACC + 1) * 4 + g) * 128 + n) * 16));
            a1[4 * g] += t1.x; a1[4 * g + 1] += t1.y; a1[4 * g + 2] += t1.z; a1[4 * g + 3] += t1.w;
          }
        }
      }
      const int m0 = ch * 16, cnt = min(16, args.M - m0);
      if (cnt > 0) {
        if (Epi::kDual) {
          if (j < args.n_pairs) epiT16(epi, m0, cnt, j, a0, a1);
        } else {
          if (j < args.n_pairs) epiT16(epi, m0, cnt, j, a0, a0);
          if (NACC == 2 && j + 128 < args.n_pairs) epiT16(epi, m0, cnt, j + 128, a1, a1);
        }
      }
    }
  }
  if (C > 1) cluster_sync();          // nobody leaves while a peer may still read its shared memory
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// ---- host side ------------------------------------------------------------------------------------------------
// Launches the swapped kernel, or returns 1 when this problem is not one it takes (the caller then uses k_gemm_stream).
template <int NACC, typename Epi>
int swap_launch(UmmaState& st, cudaStream_t stream, const bf16* A, const bf16* W0, const bf16* W1, int M, int NP, int K,
                int n_rows_w, const Epi& epi, unsigned* status, int box_rows) {
  constexpr int BN = 128 * NACC;
  const int per_tile = Epi::kDual ? BN / 2 : BN;
  const int n_tiles = (NP + per_tile - 1) / per_tile;
  const int nr = (M + 15) / 16 * 16;
  if (nr > 256 || NACC * nr > 512 || n_tiles > st.n_sm || K % UM_BK) return 1;
  const int kc_all = K / UM_BK;
  // K slices per tile: as many CTAs as fit in one wave of resident clusters
  int C = 1;
  for (int c = 4; c >= 2; c >>= 1)
    if (n_tiles * c <= st.n_sm && n_tiles <= st.max_clusters[c] && kc_all % c == 0 && kc_all / c >= 4) { C = c; break; }
  // Where it pays (measured on the LLaDA, Dream and a third model's layer shapes at 130..256 rows against
  // k_gemm_stream): with at least 96 CTAs pulling operands, and up to 224 rows -- up to 256 when the K slices are four
  // (the row-major kernel then runs two row tiles on four-CTA clusters, its slowest configuration).  Fewer CTAs make
  // the launch intake-bound, and there the row-major kernel's narrower tiles win.
  if (!st.swap_force && (n_tiles * C < 96 || (nr > 224 && C != 4))) return 1;
  const int stage = nr * 128 + BN * 128;
  const int aux = 1024 + 8 * (2 * SW_MAX_STAGES + 1) + 16;
  // half an SM's shared memory when four stages still fit: the following kernel's CTA can then be resident beside this
  // one and request its first weight tiles early
  int budget = st.max_smem;
  const int half = (st.sm_smem / 2 - 1024) & ~1023;
  if (st.stream_half_sm && half < budget && (half - aux) / stage >= 4) budget = half;
  int stages = (budget - aux) / stage;
  if (stages > SW_MAX_STAGES) stages = SW_MAX_STAGES;
  const int kc = kc_all / C;
  if (stages > kc) stages = kc;
  if (stages < 2) return 1;
  // the published pieces of the split must fit in the stage area
  const size_t pub = C > 1 ? (size_t)(nr / 16 - (nr / 16) / C) * NACC * 16 * 128 * 4 : 0;
  if (pub > (size_t)stages * stage) return 1;
  const size_t smem = (size_t)stages * stage + aux;
  static bool attr_set = false;   // per instantiation
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(k_gemm_swap<NACC, Epi>, cudaFuncAttributeMaxDynamicSharedMemorySize, st.max_smem);
    if (e != cudaSuccess) { st.err = cudaGetErrorString(e); return -3; }
    attr_set = true;
  }
  if (st.cache.size() > 4096) st.cache.clear();
  if (box_rows <= 0 || box_rows > BN / 2 || (BN / 2) % box_rows || box_rows % 8) box_rows = BN / 2;
  const CUtensorMap* ma = umma_map(st, A, M, K, nr);
  const CUtensorMap* mb0 = umma_map(st, W0, n_rows_w, K, box_rows);
  const CUtensorMap* mb1 = umma_map(st, W1, n_rows_w, K, box_rows);
  if (!ma || !mb0 || !mb1) return -4;
  SwapArgs args{M, NP, kc, nr, box_rows, stages, C, status};
  cudaError_t e = launch_k(st.pdl, k_gemm_swap<NACC, Epi>, dim3(n_tiles * C), dim3(SW_THREADS), smem, stream, C, *ma, *mb0, *mb1,
                           args, epi);
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) { st.err = cudaGetErrorString(e); return -5; }
  return 0;
}

}  // namespace lsp
