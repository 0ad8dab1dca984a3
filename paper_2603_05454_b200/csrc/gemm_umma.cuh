// bf16 GEMM on the 5th-generation tensor cores (tcgen05) for sm_100a: the parts shared by every kernel that uses them.
//
//   acc[m, c] = sum_k A[m, k] * Wt[c, k]        A: [M, K] bf16 row-major, Wt: weight rows, K-major, fp32 accumulate
//
// This header holds the PTX wrappers (mbarrier with bounded waits, TMA tile loads (every CTA fetches its own tiles), tcgen05.mma /
// .commit / .ld), the shared-memory and instruction descriptors, the vectorised fused epilogues (store / residual /
// SwiGLU / rotary + K/V staging), the host state (tensor-map cache, tuning fields) and the dispatch that picks tile
// width and row tiles per CTA.  The kernel itself is the persistent k_gemm_stream of gemm_stream.cuh; the attention
// kernel (attention_umma.cuh) uses the same wrappers.
//
// The B tile is two TMA boxes of BN/2 weight rows each (possibly from two tensors), so accumulator columns
// c and c + BN/2 of one thread hold the pair an element-wise fusion needs (gate/up, rotate-half partners).
// Every wait is bounded by wall-clock time; on expiry a kernel records (code, site) in a status word, lets
// all roles drain and returns, so a protocol error can never hang the device.
#pragma once
#include <cuda.h>

#include <map>
#include <string>
#include <tuple>

#include "epilogues.cuh"

namespace lsp {

constexpr int UM_BM = 128;
constexpr int UM_BK = 64;                 // bf16 elements = one 128-byte swizzle row
constexpr int UM_MAX_STAGES = 12;
constexpr uint64_t UM_WAIT_NS = 2000000000ull;   // 2 s

// ---- PTX wrappers -----------------------------------------------------------------------------------------
__device__ __forceinline__ uint64_t globaltimer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
// Bounded wait.  Returns false after limit_ns (default UM_WAIT_NS) or when another role has raised the abort flag.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint64_t limit_ns = UM_WAIT_NS) {
  uint64_t t0 = 0;
  for (uint32_t spin = 0;; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spin & 1023u) == 1023u) {
      if (*abort_flag) return false;
      const uint64_t now = globaltimer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) return false;
    }
  }
}

// Self-test of the bounded-wait protocol: one thread waits on a barrier that nobody ever arrives at, gives up after
// limit_ns and reports it exactly as the kernels' roles do: (code 1, site 99) in the status word.  Nothing else runs,
// nothing is in flight, the context stays usable.
__global__ void k_wait_selftest(unsigned* status, unsigned long long limit_ns) {
  __shared__ uint64_t never;
  __shared__ uint32_t no_abort;
  if (threadIdx.x == 0) {
    no_abort = 0;
    mbar_init(smem_u32(&never), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (!mbar_wait(smem_u32(&never), 0u, &no_abort, (uint64_t)limit_ns)) {
      atomicExch(status, 1u);
      status[1] = 99u;
    }
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                           uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// 16 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// 16 consecutive fp32 columns of this thread's TMEM lane, without waiting: several loads can be in flight before one
// tc_wait_ld(); the destination must not be read before that wait.
__device__ __forceinline__ void tc_ld16_nowait(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// Placed after tc_wait_ld(): makes every later use of v depend on a statement that follows the wait, so that the compiler
// cannot schedule arithmetic on the loaded values ahead of it.
__device__ __forceinline__ void tc_pin16(float (&v)[16]) {
  asm volatile("" : "+f"(v[0]), "+f"(v[1]), "+f"(v[2]), "+f"(v[3]), "+f"(v[4]), "+f"(v[5]), "+f"(v[6]), "+f"(v[7]), "+f"(v[8]),
               "+f"(v[9]), "+f"(v[10]), "+f"(v[11]), "+f"(v[12]), "+f"(v[13]), "+f"(v[14]), "+f"(v[15]));
}

// Shared-memory matrix descriptor for a K-major bf16 tile stored as rows of 128 bytes with the 128-byte swizzle:
// 8-row groups are 1024 bytes apart (stride byte offset); the leading byte offset is unused for this layout.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);        // start address, 16-byte units
  d |= (uint64_t)1 << 16;                          // leading byte offset (ignored with swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset
  d |= (uint64_t)1 << 46;                          // descriptor version for this architecture
  d |= (uint64_t)2 << 61;                          // layout: 128-byte swizzle
  return d;
}
// Instruction descriptor: D = f32, A = B = bf16, both K-major, M = 128, N = BN.
// (M = 64 puts accumulator row r in tensor-memory lane 32 (r / 16) + r % 16: the lower half of every warp's lane quarter.)
__host__ __device__ constexpr uint32_t make_idesc_m64(int bn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(64 >> 4) << 24);
}
__host__ __device__ constexpr uint32_t make_idesc(int bn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(UM_BM >> 4) << 24);
}

// ---- vector helpers for the epilogues ------------------------------------------------------------------
__device__ __forceinline__ uint4 pack8(const float* v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]);
  __nv_bfloat162 b = __floats2bfloat162_rn(v[2], v[3]);
  __nv_bfloat162 c = __floats2bfloat162_rn(v[4], v[5]);
  __nv_bfloat162 d = __floats2bfloat162_rn(v[6], v[7]);
  uint4 r;
  r.x = *reinterpret_cast<uint32_t*>(&a);
  r.y = *reinterpret_cast<uint32_t*>(&b);
  r.z = *reinterpret_cast<uint32_t*>(&c);
  r.w = *reinterpret_cast<uint32_t*>(&d);
  return r;
}
__device__ __forceinline__ void unpack8(const uint4& u, float* v) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __low2float(p[i]);
    v[2 * i + 1] = __high2float(p[i]);
  }
}

// 16 consecutive pair indices j..j+15 of row m (a1 unused for plain epilogues).
__device__ __forceinline__ void epi16(const EpiStore<bf16>& e, int m, int j, const float* a0, const float*) {
  uint4* p = reinterpret_cast<uint4*>(e.out + (size_t)m * e.ld + j);
  p[0] = pack8(a0);
  p[1] = pack8(a0 + 8);
}
__device__ __forceinline__ void epi16(const EpiResidual<bf16>& e, int m, int j, const float* a0, const float*) {
  uint4* p = reinterpret_cast<uint4*>(e.x + (size_t)m * e.ld + j);
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    float x[8];
    unpack8(p[h], x);
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] += a0[8 * h + i];
    p[h] = pack8(x);
  }
}
__device__ __forceinline__ void epi16(const EpiSwiGLU<bf16>& e, int m, int j, const float* g, const float* u) {
  float r[16];
#pragma unroll
  // __fdividef (reciprocal + multiply, 2 ulp): the IEEE division's slow path is a subroutine call inside the epilogue,
  // and its mere presence cost the whole kernel 5-7 us at every row count (39.4 -> 34.4 us at 2 rows, 61.7 -> 54.6 at 256)
  for (int i = 0; i < 16; ++i) r[i] = __fdividef(g[i], 1.f + __expf(-g[i])) * u[i];
  uint4* p = reinterpret_cast<uint4*>(e.out + (size_t)m * e.ld + j);
  p[0] = pack8(r);
  p[1] = pack8(r + 8);
}
__device__ __forceinline__ void epi16(const EpiQKVRope<bf16>& e, int m, int j, const float* a0, const float* a1) {
  const int h = j / e.half, i = j % e.half;       // 16 indices stay inside one head (half is a multiple of 16)
  const int dh = 2 * e.half;
  float r0[16], r1[16];
  bf16* dst;
  if (h >= e.n_heads && e.seq_stride > 0 && e.row_seq[m] < 0) return;      // in-place layout: a row of no sequence has no cache slot
  if (h < e.n_heads + e.n_kv_heads) {
    const float4* c4 = reinterpret_cast<const float4*>(e.cs + (size_t)e.row_pos[m] * e.half + i);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const float4 c = __ldg(c4 + q);             // (cos, sin) of two consecutive frequencies
      r0[2 * q] = a0[2 * q] * c.x - a1[2 * q] * c.y;
      r1[2 * q] = a1[2 * q] * c.x + a0[2 * q] * c.y;
      r0[2 * q + 1] = a0[2 * q + 1] * c.z - a1[2 * q + 1] * c.w;
      r1[2 * q + 1] = a1[2 * q + 1] * c.z + a0[2 * q + 1] * c.w;
    }
    dst = (h < e.n_heads) ? e.q_out + (size_t)m * e.n_heads * dh + h * dh
                          : e.k_stage + e.kv_row(m) * e.n_kv_heads * dh + (h - e.n_heads) * dh;
  } else {
#pragma unroll
    for (int q = 0; q < 16; ++q) { r0[q] = a0[q]; r1[q] = a1[q]; }
    dst = e.v_stage + e.kv_row(m) * e.n_kv_heads * dh + (h - e.n_heads - e.n_kv_heads) * dh;
  }
  uint4* p0 = reinterpret_cast<uint4*>(dst + i);
  uint4* p1 = reinterpret_cast<uint4*>(dst + i + e.half);
  p0[0] = pack8(r0);
  p0[1] = pack8(r0 + 8);
  p1[0] = pack8(r1);
  p1[1] = pack8(r1 + 8);
}

// ---- host side ------------------------------------------------------------------------------------------------
typedef CUresult (*PFN_encodeTiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct UmmaState {
  PFN_encodeTiled encode = nullptr;
  std::map<std::tuple<const void*, int, int, int>, CUtensorMap> cache;
  int max_smem = 0;
  int n_sm = 148;
  float* scratch = nullptr;        // split-K partial tiles (device), scratch_bytes long
  size_t scratch_bytes = 0;
  unsigned* counters = nullptr;    // split-K arrival counters (device), n_counters entries, zero between launches
  int n_counters = 0;
  int target_ctas = 0;             // 0 = one CTA per SM
  int max_stages = UM_MAX_STAGES;
  int sm_smem = 233472;            // shared memory per SM
  int pdl = 1;                     // launch with the programmatic-serialisation attribute
  int stream_cluster = 1;          // persistent kernel: K slices of a tile on one thread block cluster, reduced through DSMEM
  int max_clusters[9] = {0, 148, 74, 45, 33, 26, 22, 15, 15};   // [c]: clusters of c one-per-SM CTAs that can be resident at once (queried at init)
  int stream_half_sm = 1;          // persistent kernel: cap shared memory at half an SM when three stages still fit
  int stream_issuers = 1;          // MMA-issuing warps with one row tile per CTA (two row tiles always use two); measured: no gain from 2
  int stream_two_tiles = 1;        // 129..256 rows: 1 = two row tiles per CTA, 2 = two row groups
  int stream_big_mt = 3;           // ... and for more rows: 1 or 2 row tiles per CTA, 3 = whichever fills the SMs better
  int stream_bn = 0;               // its tile width with one row tile (0 = automatic)
  int stream_bn2 = 0;              // ... and with two row tiles
  int stream_bn_dual = 0;          // tile width of dual epilogues: 0 = automatic, 192 or 256
  int stream_exchange = 1;         // clusters of 2 exchange half tiles instead of publishing whole partial tiles
  int stream_atoms = 0;            // K atoms per stage: 0 = two when stream_min_stages2 such stages fit, else 1 or 2 as given
  int stream_min_stages2 = 3;
  int stream_half_tile1 = 1;       // 129..192 rows on two row tiles, unsplit: 64-row MMAs for the second row tile
  int swap_min_rows = 129;         // row counts [min, max] that take the operand-swapped kernel (gemm_swap.cuh); max 0 = never
  int swap_max_rows = 256;
  int swap_force = 0;              // 1: take it whenever it can run (tests), not only where it was measured to pay
  int stream_grid_mode = 2;        // its grid: 0 = by row count, 1 = one CTA per SM (even shares), 2 = multiple of the tile count
  int stream_even_max_rows = 0;    // mode 0: even shares up to this many activation rows
  std::string err;
};

inline int umma_init(UmmaState& st) {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess || fn == nullptr || qres != cudaDriverEntryPointSuccess) {
    st.err = "cuTensorMapEncodeTiled not available";
    return -1;
  }
  st.encode = (PFN_encodeTiled)fn;
  int dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&st.max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  cudaDeviceGetAttribute(&st.n_sm, cudaDevAttrMultiProcessorCount, dev);
  cudaDeviceGetAttribute(&st.sm_smem, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev);
  return 0;
}

// 2-D bf16 tensor [rows, K] row-major, box = [64 (K), box_rows], 128-byte swizzle, zero fill out of bounds.
inline const CUtensorMap* umma_map(UmmaState& st, const void* base, int rows, int K, int box_rows) {
  auto key = std::make_tuple(base, rows, K, box_rows);
  auto it = st.cache.find(key);
  if (it != st.cache.end()) return &it->second;
  CUtensorMap m;
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {(cuuint32_t)UM_BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = st.encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    st.err = "cuTensorMapEncodeTiled failed (" + std::to_string((int)r) + ")";
    return nullptr;
  }
  return &st.cache.emplace(key, m).first->second;
}

constexpr int UM_HEAD_BN = 256;
inline int umma_head_tiles(int vocab) { return (vocab + UM_HEAD_BN - 1) / UM_HEAD_BN; }

template <typename Epi> int stream_row_tiles(const UmmaState& st, int M, int NP, int K, int bn);
template <int NACC, typename Epi>
int swap_launch(UmmaState& st, cudaStream_t stream, const bf16* A, const bf16* W0, const bf16* W1, int M, int NP, int K,
                int n_rows_w, const Epi& epi, unsigned* status, int box_rows);
template <int BN, int MT, int NI, typename Epi>
int stream_launch(UmmaState& st, cudaStream_t stream, const bf16* A, const bf16* W0, const bf16* W1, int M, int NP, int K,
                  int n_rows_w, const Epi& epi, unsigned* status, int box_rows);

// Instantiation choice for the streaming kernel: tile width 128 or 256, one or two row tiles, one or two MMA issuers
// (two row tiles always have two).
template <typename Epi>
int stream_dispatch(UmmaState& st, cudaStream_t stream, const bf16* A, const bf16* W0, const bf16* W1, int M, int NP, int K,
                    int n_rows_w, const Epi& epi, unsigned* status, int box_rows, int bn, int mt, int ni) {
#define LSP_STREAM_CASE(BN_, MT_, NI_) \
  if (bn == BN_ && mt == MT_ && ni == NI_) \
    return stream_launch<BN_, MT_, NI_, Epi>(st, stream, A, W0, W1, M, NP, K, n_rows_w, epi, status, box_rows)
  if (mt == 2) ni = 2;
  LSP_STREAM_CASE(256, 1, 1);
  LSP_STREAM_CASE(256, 1, 2);
  LSP_STREAM_CASE(256, 2, 2);
  if constexpr (Epi::kDual && !std::is_same<Epi, EpiQKVRope<bf16>>::value) {    // 96 pairs per tile: whole tiles only (see umma_gemm)
    if (bn == 192 && mt == 1) ni = 1;
    LSP_STREAM_CASE(192, 1, 1);
    LSP_STREAM_CASE(192, 2, 2);
  }
  if constexpr (!Epi::kReduce) {
    LSP_STREAM_CASE(128, 1, 1);
    LSP_STREAM_CASE(128, 1, 2);
    LSP_STREAM_CASE(128, 2, 2);
  }
#undef LSP_STREAM_CASE
  st.err = "no streaming-kernel instantiation for this tile shape";
  return -7;
}

// Tile-width choice for the persistent kernel (the K split follows from the tile count, see stream_launch).
//  * The rotary epilogue needs both partners of a pair inside one head: its half tiles are fetched head by head.
//  * A shape the kernel cannot take (none of a transformer layer's: it would need more than 4096 column tiles in a
//    launch whose tiles are split between CTAs) is an error, not a fallback.
template <typename Epi>
int umma_gemm(UmmaState& st, cudaStream_t stream, const bf16* A, const bf16* W0, const bf16* W1, int M, int NP, int K,
              int n_rows_w, const Epi& epi, unsigned* status) {
  if (K % UM_BK) { st.err = "K must be a multiple of 64"; return -6; }
  if constexpr (Epi::kReduce) {
    {
      const int smt = stream_row_tiles<Epi>(st, M, NP, K, UM_HEAD_BN);
      if (smt > 0)
        return stream_dispatch<Epi>(st, stream, A, W0, W1, M, NP, K, n_rows_w, epi, status, 0, UM_HEAD_BN, smt,
                                    st.stream_issuers);
    }
    st.err = "the tcgen05 head GEMM cannot take this shape";
    return -8;
  } else {
    const int cols = Epi::kDual ? 2 * NP : NP;
    if (M >= st.swap_min_rows && M <= st.swap_max_rows) {
      // 129..256 rows: the tensor pipe bounds the launch, and with the operands swapped its time follows the row count
      int rc;
      if constexpr (std::is_same<Epi, EpiQKVRope<bf16>>::value) rc = swap_launch<2, Epi>(st, stream, A, W0, W1, M, NP, K, n_rows_w, epi, status, epi.half);
      else if constexpr (Epi::kDual) rc = st.swap_force ? swap_launch<2, Epi>(st, stream, A, W0, W1, M, NP, K, n_rows_w, epi, status, 0) : 1;   // gate/up: one K slice only, 96 CTAs of 3 MB intake each: the 192-wide row-major tiles win (measured)
      else if (cols >= 8192) rc = swap_launch<2, Epi>(st, stream, A, W0, W1, M, NP, K, n_rows_w, epi, status, 0);
      else rc = swap_launch<1, Epi>(st, stream, A, W0, W1, M, NP, K, n_rows_w, epi, status, 0);
      if (rc <= 0) return rc;          // 1 = not a problem that kernel takes
    }
    {
      // Tile width, from measurements on the LLaDA layer shapes at 2..256 rows: dual epilogues take 256 columns (128
      // pairs); plain ones take 128, which needs no K split with 96 tiles, except that a wide GEMM with at most 32
      // rows takes 256 (its partial tiles are small, and half as many MMA instructions are issued).  The rotary
      // epilogue's half tiles are fetched head by head.
      // With 129..256 rows (two row tiles per CTA) a wide GEMM again takes 256 columns, its K halves on a cluster of 2
      // that exchanges half tiles: 256 x 256 tiles need a third less shared-memory fill than 256 x 128 ones (QKV-sized
      // GEMM 38-40 -> 35-37.5 us); a narrow GEMM (36 tiles of 128) is better off with more, smaller tiles.
      const bool wide_two_tiles = M > UM_BM && M <= 2 * UM_BM && cols >= 8192 && st.stream_exchange && st.stream_cluster;
      int sbn = Epi::kDual ? 256 : (((M <= 32 || wide_two_tiles) && cols >= 8192) ? 256 : 128), box_rows = 0;
      if constexpr (std::is_same<Epi, EpiQKVRope<bf16>>::value) {
        box_rows = epi.half;
        sbn = (M <= 32 || wide_two_tiles) ? 256 : 128;
      }
      if (M > 2 * UM_BM || (M > UM_BM && st.stream_two_tiles == 2)) sbn = 256;   // several row groups: the widest MMA
      if (M <= UM_BM && st.stream_bn > 0) sbn = st.stream_bn;
      if (M > UM_BM && M <= 2 * UM_BM && st.stream_bn2 > 0) sbn = st.stream_bn2;
      if (box_rows > sbn / 2) sbn = 2 * box_rows;
      if constexpr (Epi::kDual && !std::is_same<Epi, EpiQKVRope<bf16>>::value) {
        // 192-wide tiles (96 pairs): with 12288 pairs that is 128 tiles instead of 96, i.e. a third more SMs pulling
        // operands, and a quarter less shared-memory fill per CTA.  Only where no tile would be split between CTAs
        // (the split paths assume a power-of-two chunk count): one wave of whole tiles, or several row groups.
        // (The same idea for the rotary QKV GEMM, 96-wide tiles that straddle heads, needs 16-row TMA boxes of 2 KB,
        // and those cost far more than the fuller wave gains: +0.7 ms per LLaDA-shaped pass.  Not kept.)
        if (st.stream_bn_dual != 256 && NP % 96 == 0 && st.stream_grid_mode == 2 && st.target_ctas == 0) {
          const int mt192 = M <= UM_BM ? 1 : 2;
          const long groups = (M + UM_BM * mt192 - 1) / (UM_BM * mt192);
          const long t192 = (long)(NP / 96) * groups, t256 = (long)((NP + 127) / 128) * groups;
          const bool whole192 = (groups == 1 && t192 <= st.n_sm && 2 * t192 > st.n_sm) || (groups > 1 && t192 >= st.n_sm);
          const bool better = M <= 2 * UM_BM ? (t256 < t192 && t256 < st.n_sm) : false;
          if (whole192 && (st.stream_bn_dual == 192 || better)) sbn = 192;
        }
      }
      const int smt = stream_row_tiles<Epi>(st, M, NP, K, sbn);
      if (smt > 0 && (sbn == 128 || sbn == 256 || sbn == 192))
        return stream_dispatch<Epi>(st, stream, A, W0, W1, M, NP, K, n_rows_w, epi, status, box_rows, sbn, smt,
                                    st.stream_issuers);
    }
    st.err = "the tcgen05 GEMM cannot take this shape";
    return -8;
  }
}

}  // namespace lsp
