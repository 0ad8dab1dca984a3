// Suffix-over-prefix attention on the 5th-generation tensor cores (tcgen05 + TMEM), head_dim 128, bf16.
//
// Same contract as attention_mma.cuh: the query rows of this pass attend, without any mask, over the contiguous prefix
// cache [0, F) followed by this pass's staged rows (Sec. 3.2: bidirectional lookahead over the frozen prefix and the
// active suffix).  One CTA owns 128 "rows" of one (sequence, KV head): a row is a (query position, query head of
// the group) pair, so grouped-query heads share every K/V tile.
//
//   per key tile of 128 keys:   S = Q K^T          tcgen05.mma, A = Q (smem), B = K tile (smem, K-major), D in TMEM
//                               P = exp2(S - m)    128 threads, one row each: tcgen05.ld, online max / sum, bf16 P to smem
//                               O += P V           tcgen05.mma, A = P (smem), B = V tile read MN-major (keys are rows)
//
// K and V tiles come straight from the cache / staging planes by TMA (two 64-column boxes each, 128-byte swizzle)
// through a two-stage ring; S is double-buffered in TMEM so that the next tile's QK^T overlaps this tile's softmax.
// A 128 x 128 score tile costs the softmax threads about 3.5 times what its two MMAs cost the tensor pipe, so two
// softmax groups of 128 threads work on alternate key tiles, each with its own running maximum, row sum, P tile and
// accumulator (O_0 and O_1 in TMEM, 512 columns with the two S buffers); their partial results are combined per row at
// the end exactly like the partials of a key split across a cluster.
// The running maximum is only raised when it grows by more than 8 (log2 units): the accumulator rescale (a TMEM
// read-modify-write) then happens on the first tiles only, and exp2(S - m) stays below 2^8, which bf16 P and the
// fp32 row sum hold without loss; the final O / l is the same quantity.
// Warps 0..3 and 4..7 = softmax groups 0 and 1 (warp w owns TMEM lanes 32 (w mod 4) ..), group 0 also the epilogue;
// warps 8 and 11 = TMA producers of the K and the V tiles, warp 9 = TMEM allocator and issuer of the Q K^T MMAs,
// warp 10 = issuer of the P V MMAs.
// Every wait is bounded; on expiry the kernel records (code, site), drains and returns.
#pragma once
#include "gemm_stream.cuh"

namespace lsp {

constexpr int AU_BM = 128;        // rows per CTA
constexpr int AU_BN = 128;        // keys per tile
constexpr int AU_THREADS = 384;   // warps 0..3 and 4..7: the two softmax groups; 8, 11: TMA producers (K, V); 9, 10: MMA issuers
constexpr int AU_W_TMA = 8, AU_W_QK = 9, AU_W_PV = 10, AU_W_TMAV = 11;
constexpr int AU_ATOM = 128 * 128;            // bytes of one [128 rows x 64 bf16] swizzle atom
constexpr int AU_TILE = 2 * AU_ATOM;          // one 128 x 128 bf16 operand tile
constexpr int AU_SMEM = 1024 + 3 * AU_TILE /*Q, P0, P1*/ + 2 * 2 * AU_TILE /*K, V stages*/ + 256 /*barriers, flags*/ + 1024 /*(m, l)*/;

__device__ __forceinline__ void tc_st16(uint32_t taddr, const float (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
        "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])),
        "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
        "r"(__float_as_uint(v[15]))
      : "memory");
}
// Placed after tc_wait_ld(): makes every later use of v[0..15] depend on a statement that follows the wait, so that the
// compiler cannot schedule arithmetic on the loaded values ahead of it.
__device__ __forceinline__ void tc_pin16p(float* v) {
  asm volatile("" : "+f"(v[0]), "+f"(v[1]), "+f"(v[2]), "+f"(v[3]), "+f"(v[4]), "+f"(v[5]), "+f"(v[6]), "+f"(v[7]), "+f"(v[8]),
               "+f"(v[9]), "+f"(v[10]), "+f"(v[11]), "+f"(v[12]), "+f"(v[13]), "+f"(v[14]), "+f"(v[15]));
}
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float ld_cluster_f1(uint32_t addr) {
  float v;
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory descriptor of an MN-major bf16 operand tile stored as [K rows][64 MN elements] atoms with the
// 128-byte swizzle: 8-row K groups are 1024 bytes apart (stride byte offset), the next 64 MN elements are one atom
// (16 KB) further (leading byte offset).
__device__ __forceinline__ uint64_t make_smem_desc_mn(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)(AU_ATOM >> 4) << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// byte offset of 16-byte chunk c (0..15) of row r inside a K-major [128 x 128] bf16 tile made of two swizzled atoms
__device__ __forceinline__ uint32_t au_swz(int r, int c) {
  return (uint32_t)((c >> 3) * AU_ATOM + (r >> 3) * 1024 + (r & 7) * 128 + (((c & 7) ^ (r & 7)) << 4));
}

// grid = (ceil(max rows per sequence * group / 128) * cluster, n_kv_heads, batch)
__global__ void __launch_bounds__(AU_THREADS, 1)
k_attn_umma(const __grid_constant__ CUtensorMap map_ck, const __grid_constant__ CUtensorMap map_cv,
            const __grid_constant__ CUtensorMap map_sk, const __grid_constant__ CUtensorMap map_sv,
            const bf16* __restrict__ q, bf16* __restrict__ out, StepDesc sd, int n_heads, int n_kv_heads, int max_len,
            float scale_log2, int cluster, int inplace, unsigned* status) {
  constexpr int DH = 128;
  extern __shared__ uint8_t smem_raw[];
  pdl_release();
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* Qs = smem;
  uint8_t* Ps = smem + AU_TILE;                         // P of softmax group w at Ps + w * AU_TILE
  uint8_t* KVs = smem + 3 * AU_TILE;                    // stage s: K at s * 2 * AU_TILE, V right behind it
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 7 * AU_TILE);
  // bars (each + stage s = softmax group w = tile parity): 0 k_full; 2 k_empty; 4 v_full; 6 v_empty; 8 s_full; 10 s_empty;
  // 12 p_ready; 14 pv_done.  K and V stages are released separately (K by the tile's Q K^T, V by its P V), so that the
  // next tile's K is on its way while this tile's softmax runs.
  // 16 q_ready: the eight softmax warps have put the Q tile in place (only the Q K^T issuer waits for it, so the K/V
  // copies are already under way while Q is being loaded)
  constexpr int B_KF = 0, B_KE = 2, B_VF = 4, B_VE = 6, B_SF = 8, B_SE = 10, B_PR = 12, B_PD = 14, B_Q = 16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 18);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  float* ml1 = reinterpret_cast<float*>(tmem_slot + 4);       // group 1's (m, l) per row, for the merge: 2 x 128 floats
  const uint32_t bb = smem_u32(bars);
  auto bar = [&](int i) { return bb + 8u * i; };
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const int b = blockIdx.z, kvh = blockIdx.y;
  const int G = n_heads / n_kv_heads;
  if (threadIdx.x == 0) {
    for (int i = 0; i < 16; ++i) mbar_init(bar(i), (i >= B_SE && i < B_PD) ? 4 : 1);     // s_empty, p_ready: four warps arrive
    mbar_init(bar(B_Q), 8);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == AU_W_QK) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // tensor memory columns: O of group 0 at 0, O of group 1 at 128, S buffer s at 256 + 128 s
  pdl_wait();

  const int r0 = sd.row_off[b];
  const int Qn = sd.row_off[b + 1] - r0;
  const int rows_total = Qn * G;
  // With clusters (size C along x) the C CTAs of a cluster share one row tile and deal its key tiles round-robin:
  // rank r takes tiles r, r + C, ...; their partial (m, l, O) are merged through distributed shared memory at the end.
  const int C = cluster > 1 ? cluster : 1;
  const int rank = (int)(blockIdx.x % C);
  const int row_base = (int)(blockIdx.x / C) * AU_BM;
  // in-place layout: this pass's K/V rows already sit behind the prefix in the cache, so every key tile is a cache tile
  const int F = sd.F[b] + (inplace ? Qn : 0);
  const int n_c = (F + AU_BN - 1) / AU_BN, n_s = inplace ? 0 : (Qn + AU_BN - 1) / AU_BN;
  const int n_all = (row_base < rows_total) ? n_c + n_s : 0;       // a CTA past the last row does nothing
  const int n_tiles = n_all > rank ? (n_all - rank + C - 1) / C : 0;   // this CTA's tiles; t below counts them
  const int ldq = n_heads * DH;

  if (warp < 8) {
    // ---- Q tile -> swizzled shared memory (zeros for rows past the end): row r by two threads, eight chunks each
    const int r = threadIdx.x & 127, c0 = (threadIdx.x >> 7) * 8;
    const int row = row_base + r;
    const bool valid = row < rows_total;
    if (n_tiles > 0) {
      const int qi = valid ? row / G : 0, hg = valid ? row % G : 0;
      const uint4* src = reinterpret_cast<const uint4*>(q + (size_t)(r0 + qi) * ldq + (kvh * G + hg) * DH);
#pragma unroll
      for (int c = c0; c < c0 + 8; ++c) {
        const uint4 v = valid ? __ldg(src + c) : make_uint4(0u, 0u, 0u, 0u);
        *reinterpret_cast<uint4*>(Qs + au_swz(r, c)) = v;
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(bar(B_Q));
  }

  if (warp == AU_W_TMA || warp == AU_W_TMAV) {
    // ---------------- TMA producers: one thread streams the K tiles, another the V tiles ----------------
    if (lane == 0) {
      const bool is_v = warp == AU_W_TMAV;
      const int full = is_v ? B_VF : B_KF, empty = is_v ? B_VE : B_KE;
      int issued = 0;
      for (int t = 0; t < n_tiles; ++t) {
        const int s = t & 1;
        if (!mbar_wait(bar(empty + s), ((uint32_t)(t >> 1) & 1u) ^ 1u, abort_flag)) {
          if (!*abort_flag) { *abort_flag = 1; atomicExch(status, 1u); status[1] = 21u; }
          break;
        }
        mbar_expect_tx(bar(full + s), AU_TILE);
        const uint32_t dst = smem_u32(KVs + (size_t)s * 2 * AU_TILE) + (is_v ? AU_TILE : 0);
        const int gt = rank + t * C;                    // tile index in the sequence's key range
        const bool cache = gt < n_c;
        const int row = cache ? b * max_len + gt * AU_BN : r0 + (gt - n_c) * AU_BN;
        const CUtensorMap* mp = cache ? (is_v ? &map_cv : &map_ck) : (is_v ? &map_sv : &map_sk);
        tma_load_2d(dst, mp, kvh * DH, row, bar(full + s));
        tma_load_2d(dst + AU_ATOM, mp, kvh * DH + 64, row, bar(full + s));
        ++issued;
      }
      // do not leave while copies may still be landing in this CTA's shared memory
      for (int t = issued > 2 ? issued - 2 : 0; t < issued; ++t) {
        volatile uint32_t no_abort = 0;
        mbar_wait(bar(full + (t & 1)), (uint32_t)(t >> 1) & 1u, &no_abort);
      }
    }
  } else if (warp == AU_W_QK) {
    // ---------------- MMA issuer 1: S = Q K^T of every tile ----------------
    if (lane == 0) {
      constexpr uint32_t idesc_qk = make_idesc(AU_BN);
      if (n_tiles > 0 && !mbar_wait(bar(B_Q), 0u, abort_flag)) {
        if (!*abort_flag) { *abort_flag = 1; atomicExch(status, 1u); status[1] = 26u; }
      }
      for (int t = 0; t < n_tiles && !*abort_flag; ++t) {
        const int s = t & 1;
        if (!mbar_wait(bar(B_KF + s), (uint32_t)(t >> 1) & 1u, abort_flag) ||
            !mbar_wait(bar(B_SE + s), ((uint32_t)(t >> 1) & 1u) ^ 1u, abort_flag)) {
          if (!*abort_flag) { *abort_flag = 1; atomicExch(status, 1u); status[1] = 22u; }
          break;
        }
        tc_fence_after();
        const uint32_t kd = smem_u32(KVs + (size_t)s * 2 * AU_TILE);
        const uint32_t d = tmem_base + 256u + (uint32_t)(s * AU_BN);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint64_t da = make_smem_desc(smem_u32(Qs) + (k >> 2) * AU_ATOM) + (uint64_t)(2 * (k & 3));
          const uint64_t db = make_smem_desc(kd + (k >> 2) * AU_ATOM) + (uint64_t)(2 * (k & 3));
          tc_mma_f16(d, da, db, idesc_qk, k ? 1u : 0u);
        }
        tc_commit(bar(B_SF + s));     // scores ready
        tc_commit(bar(B_KE + s));     // K stage free
      }
    }
  } else if (warp == AU_W_PV) {
    // ---------------- MMA issuer 2: O_w += P_w V of every tile (w = tile parity) ----------------
    if (lane == 0) {
      constexpr uint32_t idesc_pv = make_idesc(DH) | (1u << 16);          // B operand (V) is MN-major
      for (int t = 0; t < n_tiles; ++t) {
        const int s = t & 1;                  // K/V stage, S buffer and softmax group of this tile
        const uint32_t par = (uint32_t)(t >> 1) & 1u;
        if (!mbar_wait(bar(B_VF + s), par, abort_flag) || !mbar_wait(bar(B_PR + s), par, abort_flag)) {
          if (!*abort_flag) { *abort_flag = 1; atomicExch(status, 1u); status[1] = 23u; }
          break;
        }
        tc_fence_after();
        const uint32_t vd = smem_u32(KVs + (size_t)s * 2 * AU_TILE) + AU_TILE;
        const uint32_t pa = smem_u32(Ps + (size_t)s * AU_TILE);
#pragma unroll
        for (int k = 0; k < 8; ++k) {          // 16 keys per step
          const uint64_t da = make_smem_desc(pa + (k >> 2) * AU_ATOM) + (uint64_t)(2 * (k & 3));
          const uint64_t db = make_smem_desc_mn(vd) + (uint64_t)(k * (2048 >> 4));
          tc_mma_f16(tmem_base + (uint32_t)(s * DH), da, db, idesc_pv, ((t >> 1) | k) ? 1u : 0u);
        }
        tc_commit(bar(B_VE + s));     // V stage free
        tc_commit(bar(B_PD + s));     // P_w free, O_w updated
      }
    }
  } else {
    // ---------------- softmax (two groups of four warps, one row per thread; group w takes the tiles of parity w, with
    // its own running maximum, row sum and accumulator O_w) and, for group 0, the epilogue ----------------
    const int w = warp >> 2;                           // softmax group
    const int r = threadIdx.x & 127;
    const uint32_t lane_base = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t o_col = (uint32_t)(w * DH);
    uint8_t* Pw = Ps + (size_t)w * AU_TILE;
    float m_used = -INFINITY, l = 0.f;
    bool ok = true;
    int mine = 0;                                       // tiles this group has processed
    for (int t = w; t < n_tiles; t += 2, ++mine) {
      const uint32_t par = (uint32_t)mine & 1u;
      if (!mbar_wait(bar(B_SF + w), par, abort_flag)) {
        if (lane == 0 && !*abort_flag) { *abort_flag = 1; atomicExch(status, 1u); status[1] = 24u; }
        ok = false;
        break;
      }
      tc_fence_after();
      const int gt = rank + t * C;
      const int valid_keys = (gt < n_c) ? min(AU_BN, F - gt * AU_BN) : min(AU_BN, Qn - (gt - n_c) * AU_BN);
      float sv[AU_BN];
#pragma unroll
      for (int c = 0; c < AU_BN; c += 16) tc_ld16_nowait(lane_base + 256u + (uint32_t)(w * AU_BN + c), sv + c);
      tc_wait_ld();
#pragma unroll
      for (int c = 0; c < AU_BN; c += 16) tc_pin16p(sv + c);      // no use of the scores may be scheduled ahead of the wait
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_SE + w));       // S buffer read
      // raw scores; the scale (positive) is folded into the exponent's FMA, masking only touches a ragged last tile
      if (valid_keys < AU_BN) {
#pragma unroll
        for (int i = 0; i < AU_BN; ++i)
          if (i >= valid_keys) sv[i] = -INFINITY;
        // The tile's V rows past the last key hold whatever lies behind it in the plane (cache rows the library never
        // wrote, another sequence's staged rows), and 0 x NaN = NaN would reach every output row through P V.  Thread r
        // clears key row r of the V stage (128 bytes in each of its two atoms; the swizzle only permutes within a row).
        // The stage cannot be refilled before this tile's P is published below, so the completed phase is still current.
        if (r >= valid_keys && mbar_wait(bar(B_VF + w), par, abort_flag)) {
          uint8_t* vrow = KVs + (size_t)w * 2 * AU_TILE + AU_TILE + (r >> 3) * 1024 + (r & 7) * 128;
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            *reinterpret_cast<uint4*>(vrow + 16 * c) = make_uint4(0u, 0u, 0u, 0u);
            *reinterpret_cast<uint4*>(vrow + AU_ATOM + 16 * c) = make_uint4(0u, 0u, 0u, 0u);
          }
        }
      }
      float mx = -INFINITY;
#pragma unroll
      for (int i = 0; i < AU_BN; ++i) mx = fmaxf(mx, sv[i]);
      mx *= scale_log2;
      float corr = 1.f;
      bool raise = false;
      if (mx > m_used + 8.f) {                          // also the group's first tile (m_used = -inf)
        corr = ex2_approx(m_used - mx);                 // 0 on the first tile
        m_used = mx;
        raise = mine > 0;
      }
      if (mine > 0) {
        // P_w and O_w are free once the group's previous tile's P V has completed
        if (!mbar_wait(bar(B_PD + w), (uint32_t)(mine - 1) & 1u, abort_flag)) {
          if (lane == 0 && !*abort_flag) { *abort_flag = 1; atomicExch(status, 1u); status[1] = 25u; }
          ok = false;
          break;
        }
        tc_fence_after();
        if (__any_sync(0xffffffffu, raise)) {           // rare after the first tiles: rescale the accumulator rows
#pragma unroll 1
          for (int c = 0; c < DH; c += 16) {
            float v[16];
            tc_ld16(lane_base + o_col + (uint32_t)c, v);
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] *= corr;
            tc_st16(lane_base + o_col + (uint32_t)c, v);
          }
          tc_wait_st();
        }
      }
      // exponentials, sixteen keys at a time, straight into the swizzled P tile
      float sum = 0.f;
      const float neg_m = -m_used;
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        uint32_t pk[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float p0 = ex2_approx(fmaf(sv[8 * c + 2 * j], scale_log2, neg_m));
          const float p1 = ex2_approx(fmaf(sv[8 * c + 2 * j + 1], scale_log2, neg_m));
          sum += p0 + p1;
          const __nv_bfloat162 pb = __floats2bfloat162_rn(p0, p1);
          pk[j] = *reinterpret_cast<const uint32_t*>(&pb);
        }
        *reinterpret_cast<uint4*>(Pw + au_swz(r, c)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
      }
      l = l * corr + sum;
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_PR + w));        // P_w ready
    }
    bool have = ok && mine > 0 && mbar_wait(bar(B_PD + w), (uint32_t)(mine - 1) & 1u, abort_flag);
    if (have) tc_fence_after();
    // ---- the two groups' partial results of row r: weights exp2(m_w - max) as in the merge across a cluster
    if (w == 1) {
      ml1[r] = have ? m_used : -INFINITY;
      ml1[AU_BM + r] = have ? l : 0.f;
    }
    asm volatile("bar.sync 2, 256;" ::: "memory");       // the eight softmax warps
    if (w == 0) {
      const float m1 = ml1[r], l1 = ml1[AU_BM + r];
      const bool have1 = m1 != -INFINITY;
      const float m0 = have ? m_used : -INFINITY;
      const float mm = fmaxf(m0, m1);
      const float w0 = have ? ex2_approx(m0 - mm) : 0.f, w1 = have1 ? ex2_approx(m1 - mm) : 0.f;
      const float lsum = w0 * l + w1 * l1;
      const bool any = have || have1;
      if (have1) tc_fence_after();
      if (C == 1) {
        if (any) {
          const int row = row_base + r;
          const float inv = __fdividef(1.f, lsum);
          const float f0 = w0 * inv, f1 = w1 * inv;
          const bool valid = row < rows_total;
          const int qi = valid ? row / G : 0, hg = valid ? row % G : 0;
          uint4* dst = reinterpret_cast<uint4*>(out + (size_t)(r0 + qi) * ldq + (kvh * G + hg) * DH);
#pragma unroll 1
          for (int c = 0; c < DH; c += 16) {
            float v[16], u[16];
            if (have) tc_ld16(lane_base + (uint32_t)c, v);
            if (have1) tc_ld16(lane_base + (uint32_t)(DH + c), u);
            if (valid) {
#pragma unroll
              for (int i = 0; i < 16; ++i) v[i] = (have ? v[i] * f0 : 0.f) + (have1 ? u[i] * f1 : 0.f);
              dst[c >> 3] = pack8(v);
              dst[(c >> 3) + 1] = pack8(v + 8);
            }
          }
        }
      } else {
        // publish this CTA's partial result in its own shared memory (the K/V stages are idle by now):
        // O as [16-column chunk][quarter][row][4 floats] (64 KB), then m and l per row
        float4* po = reinterpret_cast<float4*>(KVs);
        float* pm = reinterpret_cast<float*>(KVs + AU_BM * DH * 4);
#pragma unroll 1
        for (int c = 0; c < DH; c += 16) {
          float v[16], u[16];
          if (have) tc_ld16(lane_base + (uint32_t)c, v);
          if (have1) tc_ld16(lane_base + (uint32_t)(DH + c), u);
#pragma unroll
          for (int i = 0; i < 16; ++i) v[i] = (have ? v[i] * w0 : 0.f) + (have1 ? u[i] * w1 : 0.f);
#pragma unroll
          for (int i = 0; i < 4; ++i) po[((c >> 4) * 4 + i) * AU_BM + r] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
        }
        pm[r] = any ? mm : -INFINITY;
        pm[AU_BM + r] = any ? lsum : 0.f;
      }
    }
  }
  if (C > 1) {
    // Merge across the cluster: rank r finishes its share of the 16-column chunks for all 128 rows, combining the
    // ranks' partials in rank order with the weights exp2(m_p - max_p m_p).  All threads of all CTAs reach both barriers.
    cluster_sync();
    if (warp < 4 && n_all > 0) {
      const int r = threadIdx.x;
      const int row = row_base + r;
      const bool valid = row < rows_total;
      const uint32_t base_o = smem_u32(KVs), base_m = base_o + AU_BM * DH * 4;
      float wgt[8];
      float mmax = -INFINITY;
      for (int p = 0; p < C; ++p) {
        wgt[p] = ld_cluster_f1(cluster_map(base_m + 4u * r, (unsigned)p));
        mmax = fmaxf(mmax, wgt[p]);
      }
      float L = 0.f;
      for (int p = 0; p < C; ++p) {
        wgt[p] = (wgt[p] == -INFINITY) ? 0.f : ex2_approx(wgt[p] - mmax);
        L += wgt[p] * ld_cluster_f1(cluster_map(base_m + 4u * (AU_BM + r), (unsigned)p));
      }
      const float inv = __fdividef(1.f, L);
      const int qi = valid ? row / G : 0, hg = valid ? row % G : 0;
      uint4* dst = reinterpret_cast<uint4*>(out + (size_t)(r0 + qi) * ldq + (kvh * G + hg) * DH);
      const int ch_lo = (DH / 16) * rank / C, ch_hi = (DH / 16) * (rank + 1) / C;
      for (int ch = ch_lo; ch < ch_hi; ++ch) {
        float v[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = 0.f;
        for (int p = 0; p < C; ++p) {
          const uint32_t peer = cluster_map(base_o + (uint32_t)((ch * 4 * AU_BM + r) * 16), (unsigned)p);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float4 t4 = ld_cluster_f4(peer + (uint32_t)(i * AU_BM * 16));
            v[4 * i] += wgt[p] * t4.x; v[4 * i + 1] += wgt[p] * t4.y; v[4 * i + 2] += wgt[p] * t4.z; v[4 * i + 3] += wgt[p] * t4.w;
          }
        }
        if (valid) {
#pragma unroll
          for (int i = 0; i < 16; ++i) v[i] *= inv;
          dst[2 * ch] = pack8(v);
          dst[2 * ch + 1] = pack8(v + 8);
        }
      }
    }
    cluster_sync();
  }
  tc_fence_before();
  __syncthreads();
  if (warp == AU_W_QK) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// 2-D bf16 tensor map of a K or V plane [rows, kvd] with a box of 64 columns x 128 rows (one swizzle atom).
inline bool attn_umma_map(UmmaState& st, CUtensorMap* m, const void* base, size_t rows, int kvd) {
  cuuint64_t dims[2] = {(cuuint64_t)kvd, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)kvd * 2};
  cuuint32_t box[2] = {64, (cuuint32_t)AU_BN};
  cuuint32_t estr[2] = {1, 1};
  return st.encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace lsp
