// Persistent bf16 GEMM on tcgen05, built for the weight-streaming regime (at most 256 activation rows: the shrinking
// suffix of late decode steps) and also used, with whole tiles per CTA, for larger problems.
//
//   acc[m, c] = sum_k A[m, k] * Wt[c, k]        operands, descriptors and fused epilogues: gemm_umma.cuh
//
// With M <= 256 a layer GEMM is bound by reading its weights from HBM once (at the upper end the tensor cores need
// about as long), so the kernel is built around one uninterrupted stream of weight tiles per SM, each weight tile
// being used for every activation row while it is in shared memory (MT = 1 or 2 row tiles of 128, one accumulator
// each):
//   * persistent CTAs, at most one per SM; the (column tile, K chunk) units of the whole problem are dealt out in
//     equal contiguous shares (a share may start and end in the middle of a tile), in a single wave;
//   * a pipeline stage holds 128 elements of K (two 128-byte swizzle atoms per operand) when at least three such
//     stages fit, else 64: 256 contiguous bytes per weight row and stage stream at 5.3 TB/s on B200 where 128 bytes
//     per row and stage reach only 3.7 TB/s;
//   * only the activation rows that exist are loaded (a box of M rounded up to 8 rows); the MMAs still span 128
//     accumulator rows each, and the rows past the box, computed from whatever the stage holds, are never stored;
//   * accumulators are double-buffered in tensor memory when two sets fit in its 512 columns, so the epilogue of one
//     tile overlaps the loads and MMAs of the next; only the first fill and the last epilogue of a CTA are exposed;
//   * a tile that spans several CTAs is finished by the CTA that arrives last at the tile's counter: every
//     contributor writes its fp32 partial tile to scratch, and the finisher sums all of them in CTA order (the same
//     order whoever finishes, so results are deterministic) before running the fused epilogue.
// Tile width: measured per shape and row count (see umma_gemm): 128 columns for plain epilogues in the streaming
// regime (no K split needed with 96 tiles), 256 for dual epilogues and for every problem with several row groups.
// Warp roles: warp 0 = TMA producer, warp 1 = TMEM allocator + MMA issuer, warps 2..5 = epilogue, warp 6 = second MMA
// issuer (see the note on issue rate in the kernel).
// Every wait is bounded; on expiry the kernel records (code, site) in the status word, drains and returns.
#pragma once
#include "gemm_umma.cuh"

namespace lsp {

constexpr int ST_MAX_STAGES = 8;

struct StreamArgs {
  int M;            // activation rows (<= 128 MT)
  int n_pairs;      // dual: pair indices; plain: output columns
  int n_tiles;      // column tiles
  int row_groups;   // groups of 128 MT activation rows (1 when M <= 128 MT); a tile is (column tile, row group), row
                    // group fastest, so a CTA meets the same weight tile again while it is still in L2
  int whole_tiles;  // 1: shares are whole tiles (no tile is split between CTAs)
  int cluster;      // > 1: the launch uses thread block clusters of this size, one cluster per tile, CTA rank r owning the
                    // r-th K slice; the partial tiles are then reduced through distributed shared memory (see the kernel)
  int cl_rounds;    // ... in this many rounds: 1 = the whole partial tile at once, MT = one row tile (128 rows) at a time,
                    // for partial tiles larger than the pipeline's shared memory; 0 = clusters of 2 exchange halves (each
                    // CTA publishes only the half its peer finishes and keeps its own half in tensor memory)
  int kc;           // K chunks (one per stage) per tile
  int a_rows;       // activation box rows (M rounded up to a multiple of 8)
  int atoms;        // 64-element K atoms per stage (1 or 2)
  int box_rows;     // weight rows per TMA box: BN/2, or fewer when the rows of a half tile are not contiguous (rotary pairs)
  int stages;
  int half_tile1;   // two row tiles, every CTA one whole tile, at most 192 rows: the second row tile's MMAs span 64
                    // accumulator rows instead of 128 (its rows sit in the lower half of every warp's tensor-memory lanes)
  float* scratch;   // [gridDim.x][2][128 MT][BN] fp32 partial tiles
  unsigned* counters;  // one per column tile, zero between launches
  unsigned* status;
};

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// thread block cluster helpers
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ unsigned cluster_ctarank() {
  unsigned r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// address, in the cluster's shared window, of this CTA's shared address saddr as seen in CTA `rank`
__device__ __forceinline__ uint32_t cluster_map(uint32_t saddr, unsigned rank) {
  uint32_t d;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(d) : "r"(saddr), "r"(rank));
  return d;
}
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}

// first unit of CTA g when U units are dealt to G CTAs
// (units are counted in 32 bits: a 64-bit division is a subroutine call, which no path of this kernel may contain; the
// host checks that U * G fits)
__device__ __forceinline__ int st_first_unit(int U, int G, int g) { return (int)((unsigned)U * (unsigned)g / (unsigned)G); }
// CTA that owns unit u
__device__ __forceinline__ int st_owner(int U, int G, int u) { return (int)(((unsigned)(u + 1) * (unsigned)G + (unsigned)U - 1u) / (unsigned)U) - 1; }

constexpr int ST_THREADS = 224;            // warp 0 producer, warps 1 and 6 MMA issuers, warps 2..5 epilogue

template <int BN, int MT, int NI, typename Epi>
__global__ void __launch_bounds__(ST_THREADS, 1)
k_gemm_stream(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b0,
              const __grid_constant__ CUtensorMap map_b1, StreamArgs args, Epi epi) {
  extern __shared__ uint8_t smem_raw[];
  pdl_release();
  constexpr int HALF = BN / 2;
  constexpr int B_HALF_ATOM = HALF * 128;               // bytes of one half-tile atom (64 K elements)
  constexpr int B_ATOM = BN * 128;
  constexpr int ROWS = UM_BM * MT;                        // accumulator rows
  // In an isolated probe one thread issues a tcgen05.mma about every 150 cycles whatever the instruction's N, and two
  // issuing threads in different warps double that rate.  NI = 2 therefore lets two warps share the issue without sharing
  // an accumulator: with two row tiles each takes one; with one row tile they take alternate K steps into accumulators of
  // their own (ACC = 2), which the epilogue adds.  In this kernel the issue rate turned out not to be the limit (the
  // operand stream is): NI = 2 measures the same as NI = 1 at every shape, so one row tile uses NI = 1 by default.
  static_assert(NI == 1 || NI == 2, "one or two MMA issuers");
  static_assert(MT == 1 || NI == 2, "two row tiles are issued by two warps");
  constexpr int ACC = (MT == 1 && NI == 2) ? 2 : 1;       // accumulators per row tile
  constexpr int SET_COLS = MT * ACC * BN;                 // columns of one accumulator set
  constexpr int NBUF = (2 * SET_COLS <= 512) ? 2 : 1;     // accumulator sets in tensor memory
  // tensor memory is allocated in powers of two (192-wide tiles use 384 of 512 columns)
  constexpr uint32_t TMEM_COLS = (NBUF * SET_COLS <= 128) ? 128 : (NBUF * SET_COLS <= 256 ? 256 : 512);
  const int A_ATOM = args.a_rows * 128;
  const int AT = args.atoms;
  const int STAGE_BYTES = AT * (A_ATOM + B_ATOM);
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int S = args.stages;
  // the barriers sit behind the stages and the padding the MMA may read (never written) past the last stage
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)S * STAGE_BYTES + ROWS * 128);
  // bars[0..S) full, [S..2S) empty, [2S..2S+2) accumulator full, [2S+2..2S+4) accumulator empty
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * S + 4);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  volatile uint32_t* epi_flag = tmem_slot + 2;          // epilogue warps: this CTA finishes the tile
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bar_base = smem_u32(bars);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (S + s); };
  auto accf_bar = [&](int b) { return bar_base + 8u * (2 * S + b); };
  auto acce_bar = [&](int b) { return bar_base + 8u * (2 * S + 2 + b); };

  const int G = gridDim.x, g = blockIdx.x;
  const int RG = args.row_groups;
  const int T = args.n_tiles * RG;
  const int U = T * args.kc;
  // Split shares: CTA g owns the contiguous units [U g / G, U (g + 1) / G).  Whole-tile shares: CTA g owns tiles
  // g, g + G, g + 2 G, ... (units are then counted within its own tiles), so that the CTAs running at any moment work
  // on neighbouring tiles: the same few weight tiles for every row group, which keeps the working set inside L2.
  const int u0 = args.whole_tiles ? 0 : st_first_unit(U, G, g);
  const int u1 = args.whole_tiles ? ((T - g + G - 1) / G) * args.kc : st_first_unit(U, G, g + 1);
  const int n_units = (int)(u1 - u0);
  int cl_tile = 0, cl_row0 = 0;      // cluster mode: the tile this CTA contributed a K slice to

  // Position of the producer in the unit space, advanced without divisions (its loop has to keep ahead of the tensor pipe).
  struct Pos {
    int vt, c, tile, rg;
  };
  auto pos_set = [&](Pos& p, int vt, int c) {
    p.vt = vt;
    p.c = c;
    const int tlin = args.whole_tiles ? g + vt * G : vt;
    p.tile = tlin / RG;
    p.rg = tlin % RG;
  };
  auto pos_next = [&](Pos& p) {
    if (++p.c == args.kc) pos_set(p, p.vt + 1, 0);
  };
  // weight boxes of one stage: the atoms of a row group back to back (AT x 128 contiguous bytes per weight row)
  auto load_weights = [&](const Pos& p, int s) {
    const uint32_t sb = smem_u32(smem + (size_t)s * STAGE_BYTES) + AT * A_ATOM;
    const int k0 = p.c * AT * UM_BK;
    for (int b = 0; b < HALF; b += args.box_rows) {
      int row_b0, row_b1;
      if (Epi::kDual) { row_b0 = epi.row0(p.tile * HALF + b); row_b1 = epi.row1(p.tile * HALF + b); }
      else { row_b0 = p.tile * BN + b; row_b1 = p.tile * BN + HALF + b; }
      for (int j = 0; j < AT; ++j) tma_load_2d(sb + j * B_ATOM + b * 128, &map_b0, k0 + 64 * j, row_b0, full_bar(s));
      for (int j = 0; j < AT; ++j)
        tma_load_2d(sb + j * B_ATOM + B_HALF_ATOM + b * 128, &map_b1, k0 + 64 * j, row_b1, full_bar(s));
    }
  };
  auto load_acts = [&](const Pos& p, int s) {
    const uint32_t sa = smem_u32(smem + (size_t)s * STAGE_BYTES);
    const int k0 = p.c * AT * UM_BK;
    for (int j = 0; j < AT; ++j) tma_load_2d(sa + j * A_ATOM, &map_a, k0 + 64 * j, p.rg * ROWS, full_bar(s));
  };

  const int n_pre = n_units < S ? n_units : S;      // stages whose weights are requested before the predecessor is done
  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), NI);          // every issuer commits the stage
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(accf_bar(b), NI);           // ... and the accumulator set
      mbar_init(acce_bar(b), 4);
    }
    *abort_flag = 0;
    *epi_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    // The weights are never written by any kernel, so the first stages' weight tiles can be requested at once, while a
    // preceding kernel (launched with programmatic serialisation) is still running; the activations follow after
    // pdl_wait().  This thread is also the producer below.
    Pos p;
    pos_set(p, (int)(u0 / args.kc), (int)(u0 % args.kc));
    for (int it = 0; it < n_pre; ++it) {
      mbar_expect_tx(full_bar(it), STAGE_BYTES);
      load_weights(p, it);
      pos_next(p);
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
  pdl_wait();          // barriers and tensor memory are set up; from here on the kernel reads what its predecessor wrote

  if (warp == 0) {
    // ---------------- TMA producer: one uninterrupted stream over this CTA's units ----------------
    if (lane == 0) {
      int issued = 0;
      Pos p;
      pos_set(p, (int)(u0 / args.kc), (int)(u0 % args.kc));
      int s = 0;
      uint32_t ph = 0;
      for (int it = 0; it < n_units; ++it) {
        if (it < n_pre) {
          load_acts(p, s);                   // the stage is armed and its weights are on their way
        } else {
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) {
            if (!*abort_flag) { *abort_flag = 1; atomicExch(args.status, 1u); args.status[1] = 11u; }
            break;
          }
          mbar_expect_tx(full_bar(s), STAGE_BYTES);
          load_weights(p, s);
          load_acts(p, s);
        }
        ++issued;
        if (++s == S) { s = 0; ph ^= 1u; }
        pos_next(p);
      }
      // do not leave while copies may still be landing in this CTA's shared memory
      const int first = issued > S ? issued - S : 0;
      for (int it = first; it < issued; ++it) {
        volatile uint32_t no_abort = 0;
        mbar_wait(full_bar((int)(it % S)), (uint32_t)(it / S) & 1u, &no_abort);
      }
    }
  } else if (warp == 1 || warp == 6) {
    // ---------------- MMA issuers ----------------
    const int is = warp == 1 ? 0 : 1;                   // issuer index
    if (lane == 0 && is < NI) {
      const uint32_t idesc = (MT == 2 && is == 1 && args.half_tile1) ? make_idesc_m64(BN) : make_idesc(BN);
      int seg = 0;
      bool ok = true;
      int s = 0;
      uint32_t ph = 0;
      for (int u = u0; u < u1 && ok;) {
        const int vt = (int)(u / args.kc);
        const int seg_end = min(u1, (vt + 1) * args.kc);
        const int buf = seg % NBUF, use = seg / NBUF;
        // wait until the epilogue has drained this accumulator set (its previous use was segment seg - NBUF)
        if (use >= 1 && !mbar_wait(acce_bar(buf), (uint32_t)(use - 1) & 1u, abort_flag)) {
          if (!*abort_flag) { *abort_flag = 1; atomicExch(args.status, 1u); args.status[1] = 12u; }
          ok = false;
          break;
        }
        tc_fence_after();
        // this issuer's accumulator: row tile `is` (two row tiles) or K-parity accumulator `is` (one row tile)
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * SET_COLS + (NI == 2 ? is * BN : 0));
        bool first = true;
        for (; u < seg_end; ++u) {
          if (!mbar_wait(full_bar(s), ph, abort_flag)) {
            if (!*abort_flag) { *abort_flag = 1; atomicExch(args.status, 1u); args.status[1] = 13u; }
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + (size_t)s * STAGE_BYTES);
          const uint32_t sb = sa + AT * A_ATOM;
          for (int j = 0; j < AT; ++j) {
            // row tile 1 starts 128 rows = 16 KB (1024 descriptor units) further into the activation atom
            const uint64_t da = make_smem_desc(sa + j * A_ATOM) + (uint64_t)((MT == 2 && is == 1) ? 1024 : 0);
            const uint64_t db = make_smem_desc(sb + j * B_ATOM);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              if (MT == 1 && NI == 2 && (k & 1) != is) continue;       // alternate K steps
              tc_mma_f16(d_tmem, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, first ? 0u : 1u);
              first = false;
            }
          }
          tc_commit(empty_bar(s));
          if (++s == S) { s = 0; ph ^= 1u; }
        }
        if (ok) tc_commit(accf_bar(buf));
        ++seg;
      }
    }
  } else {
    // ---------------- epilogue (warps 2..5) ----------------
    const int q = warp & 3;
    const int r_in = q * 32 + lane;                       // accumulator lane this thread reads
    constexpr int CH = Epi::kDual ? HALF : BN;            // pair indices (dual) or columns (plain) per tile
    int seg = 0;
    bool ok = true;
    for (int u = u0; u < u1 && ok; ++seg) {
      const int vt = (int)(u / args.kc);
      const int tlin = args.whole_tiles ? g + vt * G : vt;
      const int tile = tlin / RG, row0 = (tlin % RG) * ROWS;      // column tile, first activation row
      const int tile_u0 = vt * args.kc;
      const int seg_end = min(u1, tile_u0 + args.kc);
      const bool whole = (u == tile_u0) && (seg_end == tile_u0 + args.kc);
      const int buf = seg % NBUF, use = seg / NBUF;
      if (!mbar_wait(accf_bar(buf), (uint32_t)use & 1u, abort_flag)) {
        if (lane == 0 && !*abort_flag) { *abort_flag = 1; atomicExch(args.status, 1u); args.status[1] = 14u; }
        ok = false;
        break;
      }
      tc_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * SET_COLS);
      const int j0 = tile * CH;
      if (whole) {
        // the accumulator is complete in tensor memory: each thread owns one row of every row tile
#pragma unroll 1
        for (int mt = 0; mt < MT; ++mt) {
          int m = row0 + mt * UM_BM + r_in;
          if (MT == 2 && mt == 1 && args.half_tile1) m = lane < 16 ? row0 + UM_BM + q * 16 + lane : 0x7fffffff;   // 64-row accumulator
          Top2 red = top2_empty();
          // one chunk of 16 columns (or pairs) at a time; the next chunk's tensor-memory loads are in flight while this
          // one is converted and stored (with K-parity accumulators the extra loads are not pipelined)
          auto consume = [&](int c, float (&a0)[16], float (&a1)[16]) {
            if constexpr (ACC == 2) {               // add the second K-parity accumulator
              float b0[16];
              tc_ld16(t_row + BN + c, b0);
#pragma unroll
              for (int i = 0; i < 16; ++i) a0[i] += b0[i];
              if (Epi::kDual) {
                tc_ld16(t_row + BN + HALF + c, b0);
#pragma unroll
                for (int i = 0; i < 16; ++i) a1[i] += b0[i];
              }
            }
            if constexpr (Epi::kReduce) {
              top2_push16(red, a0, j0 + c, epi);
            } else {
              if (m < args.M && j0 + c < args.n_pairs) epi16(epi, m, j0 + c, a0, a1);
            }
          };
          auto request = [&](int c, float (&a0)[16], float (&a1)[16]) {
            tc_ld16_nowait(t_row + mt * ACC * BN + c, a0);
            if (Epi::kDual) tc_ld16_nowait(t_row + mt * ACC * BN + HALF + c, a1);
          };
          float p0[16], p1[16], q0[16], q1[16];
          request(0, p0, p1);
#pragma unroll 1
          for (int c = 0; c < CH; c += 32) {
            tc_wait_ld();
            tc_pin16(p0);
            if (Epi::kDual) tc_pin16(p1);
            if (c + 16 < CH) request(c + 16, q0, q1);
            consume(c, p0, p1);
            if (c + 16 < CH) {                     // CH is a multiple of 16, not always of 32 (48 pairs per tile)
              tc_wait_ld();
              tc_pin16(q0);
              if (Epi::kDual) tc_pin16(q1);
              if (c + 32 < CH) request(c + 32, p0, p1);
              consume(c + 16, q0, q1);
            }
          }
          if constexpr (Epi::kReduce) {
            if (m < args.M) epi.part[(size_t)m * epi.n_tiles + tile] = red;
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(acce_bar(buf));
      } else {
        // publish this CTA's partial tile, then count its chunks in; the CTA that completes the count finishes the tile.
        // Partial tile layout: [16-column chunk][quarter][row][4 floats], so that the lanes of a warp (consecutive
        // rows) write and read consecutive 16-byte pieces.
        // With clusters the partial tile goes to this CTA's own shared memory (the pipeline stages are idle by now) and
        // is reduced after the role loops; without, to the global scratch slot of this CTA.
        if (args.cluster == 2 && args.cl_rounds == 0) {
          // Exchange between the two CTAs of a pair: each finishes half of the tile's 16-column chunks, so each
          // publishes only the half its peer will finish and keeps its own half in tensor memory (see below).
          if constexpr (ACC == 1) {
            constexpr int P = Epi::kDual ? 2 : 1;
            const int rank = (int)cluster_ctarank();
            const int p_lo = (CH / 16) * (1 - rank) / 2, p_hi = (CH / 16) * (2 - rank) / 2;     // the peer's chunks
            float4* slot = reinterpret_cast<float4*>(smem);
#pragma unroll 1
            for (int mt = 0; mt < MT; ++mt) {
              const int m = mt * UM_BM + r_in;
#pragma unroll 1
              for (int ch = p_lo; ch < p_hi; ++ch) {
#pragma unroll
                for (int p = 0; p < P; ++p) {
                  float v[16];
                  tc_ld16(t_row + mt * BN + p * HALF + ch * 16, v);
                  if (row0 + m < args.M) {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                      slot[(size_t)(((ch - p_lo) * P + p) * 4 + i) * ROWS + m] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                  }
                }
              }
            }
          }
          cl_tile = tile;
          cl_row0 = row0;
          u = seg_end;
          continue;
        }
        float4* slot_base = args.cluster > 1
                                ? reinterpret_cast<float4*>(smem)
                                : reinterpret_cast<float4*>(args.scratch + (size_t)(g * 2 + (seg == 0 ? 0 : 1)) * ROWS * BN);
        // with several cluster rounds only the first row tile is published here; the others stay in tensor memory
        const bool by_tile = args.cluster > 1 && args.cl_rounds > 1;
        const int PR = by_tile ? UM_BM : ROWS;          // rows of the published partial
#pragma unroll 1
        for (int mt = 0; mt < (by_tile ? 1 : MT); ++mt) {
          const int m = mt * UM_BM + r_in;              // row within the row group
#pragma unroll 1
          for (int c = 0; c < BN; c += 16) {
            float v[16];
            tc_ld16(t_row + mt * ACC * BN + c, v);
            if constexpr (ACC == 2) {
              float b0[16];
              tc_ld16(t_row + BN + c, b0);
#pragma unroll
              for (int i = 0; i < 16; ++i) v[i] += b0[i];
            }
            if (row0 + m < args.M) {
#pragma unroll
              for (int i = 0; i < 4; ++i)
                slot_base[(size_t)((c >> 4) * 4 + i) * PR + m] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            }
          }
        }
        // the accumulator set is free as soon as every warp has read it
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(acce_bar(buf));
        if (args.cluster > 1) {          // reduced after the cluster barrier below
          cl_tile = tile;
          cl_row0 = row0;
          u = seg_end;
          continue;
        }
        __threadfence();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (threadIdx.x == 64) {
          const unsigned add = (unsigned)(seg_end - u);
          const unsigned old = atomicAdd(args.counters + tlin, add);
          const bool last = (old + add == (unsigned)args.kc);
          if (last) args.counters[tlin] = 0;          // ready for the next launch
          *epi_flag = last ? 1u : 0u;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (*epi_flag != 0) {
          __threadfence();
          const int g_lo = st_owner(U, G, tile_u0), g_hi = st_owner(U, G, tile_u0 + args.kc - 1);
          // The tile is the sum of the contributors' partial tiles.  Work items are (row, 16-column chunk), dealt over
          // the 128 epilogue threads so that a tile with few rows still uses all of them, and every item issues the
          // loads of up to four contributors before it adds them (in CTA order: deterministic).
          constexpr int NCH = CH / 16;                 // chunks per row
          constexpr int RPP = 128 / NCH;               // rows per pass
          const int et = threadIdx.x - 64;
          // plain epilogues: consecutive lanes take consecutive rows (coalesced reads of the partials); the reducing
          // epilogue keeps a row's chunks in neighbouring lanes so that they can be merged with shuffles
          const int ch = Epi::kReduce ? et % NCH : et / RPP, c = ch * 16;
          const int rows_here = min(ROWS, args.M - row0);           // rows of this row group
          for (int mm0 = 0; mm0 < rows_here; mm0 += RPP) {
            const int mm = mm0 + (Epi::kReduce ? et / NCH : et % RPP);   // row within the row group
            const bool valid = mm < rows_here;
            float a0[16], a1[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) { a0[i] = 0.f; a1[i] = 0.f; }
            if (valid) {
              for (int gb = g_lo; gb <= g_hi; gb += 4) {
                float4 t0[4][4], t1[4][4];
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                  const int gg = gb + x;
                  if (gg <= g_hi) {
                    // contributor gg's segment of this tile is its first one iff its share starts inside the tile
                    const int slot = (st_first_unit(U, G, gg) >= tile_u0) ? 0 : 1;
                    const float4* base = reinterpret_cast<const float4*>(args.scratch + (size_t)(gg * 2 + slot) * ROWS * BN) + mm;
                    const float4* p0 = base + (size_t)(c >> 4) * 4 * ROWS;
#pragma unroll
                    for (int i = 0; i < 4; ++i) t0[x][i] = __ldcg(p0 + (size_t)i * ROWS);
                    if (Epi::kDual) {
                      const float4* p1 = base + (size_t)((HALF + c) >> 4) * 4 * ROWS;
#pragma unroll
                      for (int i = 0; i < 4; ++i) t1[x][i] = __ldcg(p1 + (size_t)i * ROWS);
                    }
                  }
                }
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                  if (gb + x <= g_hi) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                      a0[4 * i] += t0[x][i].x; a0[4 * i + 1] += t0[x][i].y; a0[4 * i + 2] += t0[x][i].z; a0[4 * i + 3] += t0[x][i].w;
                      if (Epi::kDual) {
                        a1[4 * i] += t1[x][i].x; a1[4 * i + 1] += t1[x][i].y; a1[4 * i + 2] += t1[x][i].z; a1[4 * i + 3] += t1[x][i].w;
                      }
                    }
                  }
                }
              }
            }
            if constexpr (Epi::kReduce) {
              Top2 red = top2_empty();
              if (valid) top2_push16(red, a0, j0 + c, epi);
#pragma unroll
              for (int o = 1; o < NCH; o <<= 1) red = top2_merge(red, top2_shfl_xor(red, o));
              if (valid && ch == 0) epi.part[(size_t)(row0 + mm) * epi.n_tiles + tile] = red;
            } else {
              if (valid && j0 + c < args.n_pairs) epi16(epi, row0 + mm, j0 + c, a0, a1);
            }
          }
        }
      }
      u = seg_end;
    }
  }
  if (args.cluster == 2 && args.cl_rounds == 0) {
    // Pair exchange: after the barrier each CTA adds, for its own half of the chunks, its accumulator (still in tensor
    // memory) and the peer's published piece, and runs the fused epilogue.  One row per thread, as in the plain epilogue.
    cluster_sync();
    if constexpr (!Epi::kReduce && ACC == 1) {
      if (warp >= 2 && warp <= 5 && n_units > 0) {
        constexpr int CH = Epi::kDual ? HALF : BN;
        constexpr int P = Epi::kDual ? 2 : 1;
        const int rank = (int)cluster_ctarank();
        const int o_lo = (CH / 16) * rank / 2, o_hi = (CH / 16) * (rank + 1) / 2;               // this CTA's chunks
        const int q = warp & 3, r_in = q * 32 + lane;
        const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t peer = cluster_map(smem_u32(smem), (unsigned)(rank ^ 1));
        const int j0 = cl_tile * CH;
        tc_fence_after();
#pragma unroll 1
        for (int mt = 0; mt < MT; ++mt) {
          const int m = mt * UM_BM + r_in;
          const bool live = cl_row0 + m < args.M;
#pragma unroll 1
          for (int ch = o_lo; ch < o_hi; ++ch) {
            float a0[16], a1[16];
            tc_ld16(t_row + mt * BN + ch * 16, a0);
            if (Epi::kDual) tc_ld16(t_row + mt * BN + HALF + ch * 16, a1);
            if (live) {
              float4 t0[4], t1[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) t0[i] = ld_cluster_f4(peer + (uint32_t)(((((ch - o_lo) * P) * 4 + i) * ROWS + m) * 16));
              if (Epi::kDual) {
#pragma unroll
                for (int i = 0; i < 4; ++i) t1[i] = ld_cluster_f4(peer + (uint32_t)(((((ch - o_lo) * P + 1) * 4 + i) * ROWS + m) * 16));
              }
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                a0[4 * i] += t0[i].x; a0[4 * i + 1] += t0[i].y; a0[4 * i + 2] += t0[i].z; a0[4 * i + 3] += t0[i].w;
                if (Epi::kDual) {
                  a1[4 * i] += t1[i].x; a1[4 * i + 1] += t1[i].y; a1[4 * i + 2] += t1[i].z; a1[4 * i + 3] += t1[i].w;
                }
              }
              if (j0 + ch * 16 < args.n_pairs) epi16(epi, cl_row0 + m, j0 + ch * 16, a0, a1);
            }
          }
        }
      }
    }
    cluster_sync();      // nobody leaves while its peer may still read its shared memory
  } else if (args.cluster > 1) {
    // Split-K reduction inside the cluster: every CTA's partial tile sits in its shared memory; after the barrier CTA
    // rank r sums, for its share of the 16-column chunks, the partials of all ranks in rank order (= K order, so the
    // result does not depend on timing) straight from their shared memory, and runs the fused epilogue on them.
    // Every thread of every CTA reaches both barriers (no early exits above), so they cannot hang.
    const int C = args.cluster;
    const int rounds = args.cl_rounds > 1 ? MT : 1;
    const int PR = rounds > 1 ? UM_BM : ROWS;            // rows of the partial published per round
#pragma unroll 1
    for (int rd = 0; rd < rounds; ++rd) {
      if (rd > 0 && warp >= 2 && warp <= 5 && n_units > 0) {
        // publish the next row tile (a cluster CTA has a single segment: accumulator set 0, ACC = 1 with two row tiles)
        const int q = warp & 3, r_in = q * 32 + lane;
        const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16);
        float4* slot_base = reinterpret_cast<float4*>(smem);
        tc_fence_after();
#pragma unroll 1
        for (int c = 0; c < BN; c += 16) {
          float v[16];
          tc_ld16(t_row + rd * ACC * BN + c, v);
          if (cl_row0 + rd * UM_BM + r_in < args.M) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
              slot_base[(size_t)((c >> 4) * 4 + i) * PR + r_in] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
          }
        }
      }
      cluster_sync();
      if constexpr (!Epi::kReduce) {
        if (warp >= 2 && warp <= 5 && n_units > 0) {
          constexpr int CH = Epi::kDual ? HALF : BN;
          constexpr int NCH = CH / 16;
          const unsigned rank = cluster_ctarank();
          const int ch_lo = NCH * (int)rank / C, ch_hi = NCH * ((int)rank + 1) / C;
          const int r_first = cl_row0 + rd * PR;                       // first activation row of this round
          const int rows_here = max(0, min(PR, args.M - r_first));
          const int n_items = rows_here * (ch_hi - ch_lo);
          const uint32_t base = smem_u32(smem);
          for (int idx = threadIdx.x - 64; idx < n_items; idx += 128) {
            const int mm = idx % rows_here, ch = ch_lo + idx / rows_here, c = ch * 16;
            float a0[16], a1[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) { a0[i] = 0.f; a1[i] = 0.f; }
            const uint32_t off0 = (uint32_t)(((c >> 4) * 4 * PR + mm) * 16);
            const uint32_t off1 = (uint32_t)((((HALF + c) >> 4) * 4 * PR + mm) * 16);
            // up to four ranks' pieces are requested before any is added (the loads are independent; the sum stays in
            // rank order)
            for (int pb = 0; pb < C; pb += 4) {
              float4 t0[4][4], t1[4][4];
#pragma unroll
              for (int x = 0; x < 4; ++x) {
                if (pb + x < C) {
                  const uint32_t peer = cluster_map(base, (unsigned)(pb + x));
#pragma unroll
                  for (int i = 0; i < 4; ++i) t0[x][i] = ld_cluster_f4(peer + off0 + (uint32_t)(i * PR * 16));
                  if (Epi::kDual) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) t1[x][i] = ld_cluster_f4(peer + off1 + (uint32_t)(i * PR * 16));
                  }
                }
              }
#pragma unroll
              for (int x = 0; x < 4; ++x) {
                if (pb + x < C) {
#pragma unroll
                  for (int i = 0; i < 4; ++i) {
                    a0[4 * i] += t0[x][i].x; a0[4 * i + 1] += t0[x][i].y; a0[4 * i + 2] += t0[x][i].z; a0[4 * i + 3] += t0[x][i].w;
                    if (Epi::kDual) {
                      a1[4 * i] += t1[x][i].x; a1[4 * i + 1] += t1[x][i].y; a1[4 * i + 2] += t1[x][i].z; a1[4 * i + 3] += t1[x][i].w;
                    }
                  }
                }
              }
            }
            const int j0 = cl_tile * CH;
            if (j0 + c < args.n_pairs) epi16(epi, r_first + mm, j0 + c, a0, a1);
          }
        }
      }
      cluster_sync();      // nobody overwrites its partial, or leaves, while a peer may still read its shared memory
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// ---- host side ------------------------------------------------------------------------------------------------
// Scratch the streaming kernel needs for a grid of n_ctas CTAs, tile width bn and mt row tiles.
inline size_t stream_scratch_bytes(int n_ctas, int bn, int mt) { return (size_t)n_ctas * 2 * UM_BM * mt * bn * sizeof(float); }

// Number of CTAs.  Dealing the units evenly over all SMs balances the weight stream perfectly but splits almost every
// tile between two CTAs, which costs a partial tile written and read back per split (M x BN x 4 bytes each way).
// With at most as many tiles as SMs, a grid that is a multiple of the tile count splits each tile into equal K slices
// instead (no split at all when there are more than half as many tiles as SMs).  Measured on the LLaDA layer shapes
// the second choice is as fast or faster at every row count from 2 to 128, so it is the default.
// K slices per tile when the tiles are fewer than the SMs.  With clusters on, the slices of a tile form one cluster of 2
// to 8 CTAs, and a launch never asks for more clusters than can be resident at once: the GPC layout fits 74 / 45 / 33 /
// 26 / 22 / 15 / 15 clusters of 2 ... 8 one-per-SM CTAs, so e.g. 48 clusters of 3 or 16 of 8 would run as two waves
// (measured: 40 % and 100 % slower than the next smaller split).
inline int stream_splits(const UmmaState& st, long n_tiles) {
  int splits = n_tiles <= st.n_sm ? (int)(st.n_sm / n_tiles) : 0;
  if (st.stream_cluster && splits > 1) {
    int c = splits < 8 ? splits : 8;
    while (c > 1 && n_tiles > st.max_clusters[c]) --c;
    splits = c;
  }
  return splits;
}

inline int stream_grid(const UmmaState& st, int n_tiles, int M) {
  if (st.target_ctas > 0) return st.target_ctas;
  const int splits = stream_splits(st, n_tiles);
  const int aligned = splits > 0 ? n_tiles * splits : st.n_sm;
  if (st.stream_grid_mode == 1) return st.n_sm;
  if (st.stream_grid_mode == 2) return aligned;
  return M <= st.stream_even_max_rows ? st.n_sm : aligned;
}

// Stage shape for an activation box of a_rows rows and tile width bn: two K atoms per stage when at least
// stream_min_stages2 such stages fit.
struct StreamShape { int a_rows, atoms, stages, stage_bytes, aux; };
inline StreamShape stream_shape(const UmmaState& st, int a_rows, int bn, int mt, int K) {
  StreamShape sh;
  sh.a_rows = a_rows;
  sh.aux = 1024 + UM_BM * mt * 128 + 8 * (2 * ST_MAX_STAGES + 4) + 16;
  const int atom = sh.a_rows * 128 + bn * 128;
  sh.atoms = (K % 128 == 0 && (st.max_smem - sh.aux) / (2 * atom) >= st.stream_min_stages2) ? 2 : 1;
  if (st.stream_atoms == 1 || (st.stream_atoms == 2 && K % 128 == 0)) sh.atoms = st.stream_atoms;
  sh.stage_bytes = sh.atoms * atom;
  // Half an SM's shared memory when that still gives three stages (it costs no bandwidth, measured): the next kernel's
  // CTA can then become resident beside this one and request its first weight tiles before this kernel has finished.
  int budget = st.max_smem;
  if (st.stream_half_sm) {
    const int half = (st.sm_smem / 2 - 1024) & ~1023;
    if (half < budget && (half - sh.aux) / sh.stage_bytes >= 3) budget = half;
  }
  sh.stages = (budget - sh.aux) / sh.stage_bytes;
  if (sh.stages > ST_MAX_STAGES) sh.stages = ST_MAX_STAGES;
  if (sh.stages > st.max_stages) sh.stages = st.max_stages;
  return sh;
}
// Activation box rows: all rows (rounded up to 8) when they fit one group of 128 mt rows, else a full group.
inline int stream_a_rows(int M, int mt) { return M <= UM_BM * mt ? (M + 7) / 8 * 8 : UM_BM * mt; }

// Asks the runtime how many clusters of 2 ... 8 CTAs of the streaming kernel (one CTA per SM) can be resident at once.
inline void stream_query_clusters(UmmaState& st) {
  auto kern = k_gemm_stream<128, 1, 1, EpiStore<bf16>>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, st.max_smem) != cudaSuccess) return;
  st.max_clusters[1] = st.n_sm;
  for (int c = 2; c <= 8; ++c) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * c * st.n_sm);
    cfg.blockDim = dim3(ST_THREADS);
    cfg.dynamicSmemBytes = (size_t)st.max_smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)c;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) == cudaSuccess && n > 0) st.max_clusters[c] = n;
  }
  cudaGetLastError();
}

template <int BN, int MT, int NI, typename Epi>
int stream_launch(UmmaState& st, cudaStream_t stream, const bf16* A, const bf16* W0, const bf16* W1, int M, int NP, int K,
                  int n_rows_w, const Epi& epi, unsigned* status, int box_rows) {
  const StreamShape sh = stream_shape(st, stream_a_rows(M, MT), BN, MT, K);
  if (sh.stages < 2) { st.err = "not enough shared memory for the streaming GEMM"; return -2; }
  const size_t smem = (size_t)sh.stages * sh.stage_bytes + sh.aux;
  static bool attr_set = false;   // per instantiation
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(k_gemm_stream<BN, MT, NI, Epi>, cudaFuncAttributeMaxDynamicSharedMemorySize, st.max_smem);
    if (e != cudaSuccess) { st.err = cudaGetErrorString(e); return -3; }
    attr_set = true;
  }
  if (st.cache.size() > 4096) st.cache.clear();
  if (box_rows <= 0 || box_rows > BN / 2 || (BN / 2) % box_rows || box_rows % 8) box_rows = BN / 2;
  const CUtensorMap* ma = umma_map(st, A, M, K, sh.a_rows);
  const CUtensorMap* mb0 = umma_map(st, W0, n_rows_w, K, box_rows);
  const CUtensorMap* mb1 = umma_map(st, W1, n_rows_w, K, box_rows);
  if (!ma || !mb0 || !mb1) return -4;
  const int per_tile = Epi::kDual ? BN / 2 : BN;
  const int n_tiles = (NP + per_tile - 1) / per_tile;
  const int kc = K / (sh.atoms * UM_BK);
  const int row_groups = (M + UM_BM * MT - 1) / (UM_BM * MT);
  // several row groups and at least as many tiles as SMs: whole tiles per CTA; else K slices as stream_grid says
  const long T = (long)n_tiles * row_groups;
  const int whole = (row_groups > 1 && T >= st.n_sm) ? 1 : 0;
  int grid = whole ? st.n_sm : stream_grid(st, (int)T, M);
  if (grid > T * kc) grid = (int)(T * kc);
  if ((double)T * kc * (grid + 1) >= 4.0e9) { st.err = "too many work units for the streaming GEMM"; return -9; }   // 32-bit unit arithmetic
  // K slices of one tile on the CTAs of one cluster: the reduction then stays on chip
  int cluster = 0, cl_rounds = 1;
  if (!whole && !Epi::kReduce && st.stream_cluster && grid % T == 0) {
    const int splits = (int)(grid / T);
    const size_t area = (size_t)sh.stages * sh.stage_bytes, tile_bytes = (size_t)UM_BM * BN * sizeof(float);
    if (splits >= 2 && splits <= 8 && kc >= splits && area >= tile_bytes) {
      cluster = splits;
      if (area < MT * tile_bytes) cl_rounds = MT;      // the partial tile is published one row tile at a time
      if (splits == 2 && st.stream_exchange && !(MT == 1 && NI == 2) && 2 * area >= MT * tile_bytes) cl_rounds = 0;
    }
  }
  // at most 192 rows on two row tiles, every CTA one unsplit tile: 64-row MMAs for the second row tile
  const int half_tile1 = (MT == 2 && !Epi::kReduce && st.stream_half_tile1 && row_groups == 1 && M <= UM_BM + 64 && grid == (int)T &&
                          cluster == 0) ? 1 : 0;
  StreamArgs args{M, NP, n_tiles, row_groups, whole, cluster, cl_rounds, kc, sh.a_rows, sh.atoms, box_rows, sh.stages, half_tile1,
                  st.scratch, st.counters, status};
  cudaError_t e = launch_k(st.pdl, k_gemm_stream<BN, MT, NI, Epi>, dim3(grid), dim3(ST_THREADS), smem, stream, cluster, *ma, *mb0,
                           *mb1, args, epi);
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) { st.err = cudaGetErrorString(e); return -5; }
  return 0;
}

// Row tiles per CTA the streaming kernel would use for M rows, or 0 when it cannot take the problem (a tile too wide
// for the accumulators, scratch or counters too small for a split grid, too little shared memory).
template <typename Epi>
int stream_row_tiles(const UmmaState& st, int M, int NP, int K, int bn) {
  const int per_tile = Epi::kDual ? bn / 2 : bn;
  const long n_tiles = (NP + per_tile - 1) / per_tile;
  int mt;
  if (M <= UM_BM) mt = 1;
  else if (M <= 2 * UM_BM) {
    // layer GEMMs: two row tiles per CTA (each weight tile is used for all rows while it is in shared memory); the LM
    // head has hundreds of column tiles, so two row groups of whole 128 x 256 tiles keep double-buffered accumulators
    // and run 1.5 x faster there (the second row group finds its weight tile in L2)
    mt = (Epi::kReduce || st.stream_two_tiles == 2) ? 1 : 2;
  }
  else if (st.stream_big_mt == 1 || st.stream_big_mt == 2) mt = st.stream_big_mt;
  else {
    // 256 x 256 tiles (two row tiles per CTA) need a third less operand data per flop than 128 x 256 ones, which the
    // SM's shared-memory fill rate cannot quite sustain: they measure about 1.25 x faster when both fill the SMs equally
    // well.  Otherwise the better-filled grid wins; few tiles count with the K split their cluster would get, and rows
    // that only pad the last row group count as waste.
    auto fill = [&](int m) {
      const long groups = (M + UM_BM * m - 1) / (UM_BM * m);
      const long t = n_tiles * groups;
      long ctas = t;
      if (t < st.n_sm && st.stream_cluster && !Epi::kReduce) ctas = t * stream_splits(st, t);
      const double waves = (double)((ctas + st.n_sm - 1) / st.n_sm * st.n_sm);
      return (double)ctas / waves * (double)M / (double)(groups * UM_BM * m);
    };
    mt = (2 * bn <= 512 && 1.25 * fill(2) > fill(1)) ? 2 : 1;
  }
  if (mt == 0 || mt * bn > 512) return 0;
  const int row_groups = (M + UM_BM * mt - 1) / (UM_BM * mt);
  const long T = n_tiles * row_groups;
  if (!(row_groups > 1 && T >= st.n_sm)) {         // tiles may be split between CTAs: scratch and counters
    if (st.scratch == nullptr || T > st.n_counters ||
        stream_scratch_bytes(stream_grid(st, (int)T, M), bn, mt) > st.scratch_bytes)
      return 0;
  }
  return stream_shape(st, stream_a_rows(M, mt), bn, mt, K).stages >= 2 ? mt : 0;
}

}  // namespace lsp
