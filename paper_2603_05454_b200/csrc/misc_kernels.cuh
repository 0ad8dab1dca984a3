// Row assembly + embedding, RMSNorm, vocab-partial merge, the LSP scan, and commit/KV-append kernels.
#pragma once
#include "common.cuh"

namespace lsp {

// ---------------------------------------------------------------------------------------------
// Row assembly + embedding (input of Algorithm 1's forward pass): packed row r of sequence b is position
// F_b + j; the first pend_b rows carry the tokens committed by the previous step, the rest [MASK].
// One block per row.  Also fills row_seq / row_pos and the list of rows that go through the LM head.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void k_assemble_embed(StepDesc sd, int batch, const int32_t* __restrict__ tokens, int tok_stride,
                                 int mask_id, const T* __restrict__ embed, int d, T* __restrict__ X,
                                 int* __restrict__ row_seq, int* __restrict__ row_pos,
                                 int* __restrict__ head_src, int* __restrict__ head_pos, int scattered) {
  pdl_begin();
  const int r = blockIdx.x;
  // The grid may be larger than the pass (a host that sizes launches from an upper bound of the row counts): rows past
  // the last real one are zero vectors that belong to no sequence, and the spare head slots point at row 0.
  if (r >= sd.head_off[batch] && threadIdx.x == 0) head_src[r] = 0;
  if (r >= sd.row_off[batch]) {
    if (threadIdx.x == 0) { row_seq[r] = -1; row_pos[r] = 0; }
    uint4* z = reinterpret_cast<uint4*>(X + (size_t)r * d);
    for (int i = threadIdx.x; i < d * (int)sizeof(T) / 16; i += blockDim.x) z[i] = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  int b = 0;
  while (b + 1 < batch && r >= sd.row_off[b + 1]) ++b;
  const int j = r - sd.row_off[b];
  const int F = sd.F[b], pend = sd.pend[b];
  const int pos = F + j;
  // prefix topology: rows past the pending block are the masked suffix; scattered topology: every row reads the token
  // buffer (committed positions hold their token, the others the mask id) and k_compact_masked lists the masked rows
  const int tok = (scattered || j < pend) ? tokens[(size_t)b * tok_stride + pos] : mask_id;
  if (threadIdx.x == 0) {
    row_seq[r] = b;
    row_pos[r] = pos;
    if (!scattered && j >= pend) {
      head_src[sd.head_off[b] + (j - pend)] = r;
      head_pos[sd.head_off[b] + (j - pend)] = pos;
    }
  }
  const uint4* src = reinterpret_cast<const uint4*>(embed + (size_t)tok * d);
  uint4* dst = reinterpret_cast<uint4*>(X + (size_t)r * d);
  const int nv = d * (int)sizeof(T) / 16;
  for (int i = threadIdx.x; i < nv; i += blockDim.x) dst[i] = __ldg(src + i);
}

// ---------------------------------------------------------------------------------------------
// RMSNorm: out[r] = x[src[r]] / sqrt(mean(x^2) + eps) * g, fp32 arithmetic, one block per output row.
// The row is read once with 128-bit loads and kept in registers between the reduction and the scaling
// (up to RN_VPT vectors per thread; longer rows fall back to a second read).
// ---------------------------------------------------------------------------------------------
constexpr int RN_THREADS = 256;
constexpr int RN_VPT = 4;      // 16-byte vectors per thread held in registers

template <typename T> struct Vec16 { static constexpr int N = 16 / (int)sizeof(T); };

__device__ __forceinline__ void vec_to_f(const uint4& u, float (&v)[4]) {
  v[0] = __uint_as_float(u.x); v[1] = __uint_as_float(u.y); v[2] = __uint_as_float(u.z); v[3] = __uint_as_float(u.w);
}
__device__ __forceinline__ void vec_to_f(const uint4& u, float (&v)[8]) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
  for (int i = 0; i < 4; ++i) { v[2 * i] = __low2float(p[i]); v[2 * i + 1] = __high2float(p[i]); }
}
__device__ __forceinline__ uint4 f_to_vec(const float (&v)[4]) {
  return make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]));
}
__device__ __forceinline__ uint4 f_to_vec(const float (&v)[8]) {
  uint4 r;
  __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
  __nv_bfloat162 c = __floats2bfloat162_rn(v[4], v[5]), d = __floats2bfloat162_rn(v[6], v[7]);
  r.x = *reinterpret_cast<uint32_t*>(&a); r.y = *reinterpret_cast<uint32_t*>(&b);
  r.z = *reinterpret_cast<uint32_t*>(&c); r.w = *reinterpret_cast<uint32_t*>(&d);
  return r;
}

template <typename T>
__global__ void __launch_bounds__(RN_THREADS) k_rmsnorm(const T* __restrict__ x, const T* __restrict__ g, T* __restrict__ out,
                                                       const int* __restrict__ src_rows, int d, float eps) {
  constexpr int E = Vec16<T>::N;                 // elements per 16-byte vector
  __shared__ float red[RN_THREADS / 32];
  pdl_begin();
  const int r = blockIdx.x;
  const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)(src_rows ? src_rows[r] : r) * d);
  const uint4* gr = reinterpret_cast<const uint4*>(g);
  uint4* o = reinterpret_cast<uint4*>(out + (size_t)r * d);
  const int nv = d / E;                          // d is a multiple of 64
  const bool in_regs = nv <= RN_VPT * RN_THREADS;
  uint4 keep[RN_VPT];
  float ss = 0.f;
  if (in_regs) {
#pragma unroll
    for (int j = 0; j < RN_VPT; ++j) {
      const int i = threadIdx.x + j * RN_THREADS;
      keep[j] = (i < nv) ? xr[i] : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int j = 0; j < RN_VPT; ++j) {
      float v[E];
      vec_to_f(keep[j], v);
#pragma unroll
      for (int e = 0; e < E; ++e) ss += v[e] * v[e];
    }
  } else {
    for (int i = threadIdx.x; i < nv; i += RN_THREADS) {
      float v[E];
      vec_to_f(xr[i], v);
#pragma unroll
      for (int e = 0; e < E; ++e) ss += v[e] * v[e];
    }
  }
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < RN_THREADS / 32; ++w) tot += red[w];      // same order in every thread
  const float inv = rsqrtf(__fdividef(tot, (float)d) + eps);      // fast division: no IEEE slow-path subroutine in the kernel
  if (in_regs) {
#pragma unroll
    for (int j = 0; j < RN_VPT; ++j) {
      const int i = threadIdx.x + j * RN_THREADS;
      if (i < nv) {
        float v[E], gv[E];
        vec_to_f(keep[j], v);
        vec_to_f(__ldg(gr + i), gv);
#pragma unroll
        for (int e = 0; e < E; ++e) v[e] = v[e] * inv * gv[e];
        o[i] = f_to_vec(v);
      }
    }
  } else {
    for (int i = threadIdx.x; i < nv; i += RN_THREADS) {
      float v[E], gv[E];
      vec_to_f(xr[i], v);
      vec_to_f(__ldg(gr + i), gv);
#pragma unroll
      for (int e = 0; e < E; ++e) v[e] = v[e] * inv * gv[e];
      o[i] = f_to_vec(v);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Merge of the per-vocab-tile partials of one row into (yhat, p_max, delta).  One warp per row.
// ---------------------------------------------------------------------------------------------
__global__ void k_merge_partials(const Top2* __restrict__ part, int n_tiles, int rows, int32_t* __restrict__ yhat,
                                 float* __restrict__ pmax, float* __restrict__ margin) {
  pdl_begin();
  const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (r >= rows) return;
  const int lane = threadIdx.x & 31;
  Top2 t = top2_empty();
  for (int i = lane; i < n_tiles; i += 32) t = top2_merge(t, part[(size_t)r * n_tiles + i]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t = top2_merge(t, top2_shfl_xor(t, o));
  if (lane == 0) {
    yhat[r] = t.i1;
    pmax[r] = __fdividef(1.f, t.s);
    margin[r] = t.m1 - t.m2;
  }
}

// ---------------------------------------------------------------------------------------------
// LSP scan (Sec. 3.2): one warp per sequence.
//   fixed mode    : L' = longest left-aligned run with score_i >= tau             (ballot + ffs)
//   adaptive mode : prefix minimum pm; m is achievable iff pm[m] > pm[m+1]; the largest achievable
//                   m in [ceil(alpha N), floor(beta N)] is taken, tau = pm[m] (Eq. 2)
//   snap          : last delimiter j <= L' with L' - j <= W, else the run's end; L' = N commits all;
//                   L = min(N, max(L, L_min, 1))                               (Algorithm 1: snap, fallback)
// ---------------------------------------------------------------------------------------------
struct ScanParams {
  int mode;
  float tau, alpha, beta;
  int l_min, W, fixed_k;
  const uint8_t* delim;
  float flag_tol, tie_tol;
};

__device__ __forceinline__ bool is_delim(const uint8_t* bm, int id) {
  return bm != nullptr && ((bm[id >> 3] >> (id & 7)) & 1);
}

__global__ void k_lsp_scan(const float* __restrict__ score, const int32_t* __restrict__ yhat,
                           const float* __restrict__ margin, const int* __restrict__ seq_off, ScanParams p,
                           int32_t* __restrict__ o_run, int32_t* __restrict__ o_commit, uint32_t* __restrict__ o_flags,
                           float* __restrict__ o_tau) {
  pdl_begin();
  const int b = blockIdx.x;
  const int lane = threadIdx.x;
  const int base = seq_off[b];
  const int N = seq_off[b + 1] - base;
  if (N <= 0) {
    if (lane == 0) { o_run[b] = 0; o_commit[b] = 0; o_flags[b] = 0; o_tau[b] = 0.f; }
    return;
  }
  const float* sc = score + base;
  const int32_t* yh = yhat + base;
  unsigned flags = 0;
  int Lrun = 0;
  float tau = p.tau;
  if (p.mode == 2) {
    int L = min(N, max(1, p.fixed_k));
    if (lane == 0) { o_run[b] = L; o_commit[b] = L; o_flags[b] = 0; o_tau[b] = __int_as_float(0x7fc00000); }
    return;
  }
  if (p.mode == 1) {
    const int lo = max(1, (int)ceil((double)p.alpha * (double)N));
    const int hi = min(N, max(lo, (int)floor((double)p.beta * (double)N)));
    float carry = INFINITY;   // pm[m0] for the chunk start
    int best = 0;
    float best_pm = 0.f, pm_hi = 0.f;
    for (int m0 = 0; m0 < hi; m0 += 32) {
      const int m = m0 + lane + 1;                       // 1-based length this lane stands for
      float v = (m <= N) ? sc[m - 1] : INFINITY;
      // inclusive prefix min across the warp
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const float u = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v = fminf(v, u);
      }
      const float pm = fminf(v, carry);                   // pm[m]
      const bool ach = (m >= lo && m <= hi) && (m == N || sc[m] < pm);
      const unsigned bal = __ballot_sync(0xffffffffu, ach);
      if (bal) {
        const int top = 31 - __clz(bal);
        best = m0 + top + 1;
        best_pm = __shfl_sync(0xffffffffu, pm, top);
      }
      const int hl = hi - m0 - 1;                          // lane holding pm[hi], if in this chunk
      if (hl >= 0 && hl < 32) pm_hi = __shfl_sync(0xffffffffu, pm, hl);
      carry = __shfl_sync(0xffffffffu, pm, 31);
    }
    if (best > 0) { Lrun = best; tau = best_pm; }
    else { Lrun = hi; tau = pm_hi; flags |= 4u; }
  } else {
    Lrun = N;
    for (int i0 = 0; i0 < N; i0 += 32) {
      const int i = i0 + lane;
      const bool pass = (i < N) ? (sc[i] >= tau) : false;
      const unsigned fail = ~__ballot_sync(0xffffffffu, pass);
      if (fail) { Lrun = min(N, i0 + __ffs(fail) - 1); break; }
    }
  }
  int L;
  if (Lrun == N) {
    L = N;
    flags |= 8u;
  } else {
    const int lo_j = (p.W < 0) ? 1 : max(1, Lrun - p.W);
    int maxJ = 0;
    for (int hi_j = Lrun; hi_j >= lo_j && maxJ == 0; hi_j -= 32) {
      const int j = hi_j - lane;                           // lane 0 looks at the right end
      const bool d = (j >= lo_j) && is_delim(p.delim, yh[j - 1]);
      const unsigned bal = __ballot_sync(0xffffffffu, d);
      if (bal) maxJ = hi_j - (__ffs(bal) - 1);
    }
    if (maxJ > 0) {
      L = max(p.l_min, maxJ);
      if (L < Lrun) flags |= 1u;
    } else {
      L = max(p.l_min, Lrun);
    }
    if (Lrun < max(1, p.l_min)) flags |= 2u;
  }
  L = min(N, max(L, 1));
  if (p.flag_tol > 0.f || p.tie_tol > 0.f) {
    bool near = false, tie = false;
    const int lim = min(N, Lrun + 1);
    if (p.flag_tol > 0.f)
      for (int i = lane; i < lim; i += 32) near |= fabsf(sc[i] - tau) <= p.flag_tol;
    if (margin != nullptr && p.tie_tol > 0.f)
      for (int i = lane; i < L; i += 32) tie |= margin[base + i] <= p.tie_tol;
    if (__any_sync(0xffffffffu, near)) flags |= 16u;
    if (__any_sync(0xffffffffu, tie)) flags |= 32u;
  }
  if (lane == 0) { o_run[b] = Lrun; o_commit[b] = L; o_flags[b] = flags; o_tau[b] = tau; }
}

// ---------------------------------------------------------------------------------------------
// Commit (Algorithm 1: commit and AppendToCache).  grid = (chunks, n_layers * 2, batch):
//   * the pending block's K/V rows, staged by the last pass at packed rows [row_off_b, row_off_b + pend_b),
//     are copied to cache rows [F_b, F_b + pend_b): one contiguous 128-bit-vector copy per (layer, K|V, b);
//   * block (0, 0, b) also writes yhat_{1:L_b} into the token buffer at [Fp_b, Fp_b + L_b).
// The host advances F, Fp, pend, N after enqueueing this kernel (stream order makes the commit atomic).
// ---------------------------------------------------------------------------------------------
__global__ void k_commit_append(StepDesc sd, const uint4* __restrict__ stage, uint4* __restrict__ cache,
                                size_t stage_plane_v4,   // uint4 per (layer, K|V) plane of the staging buffer
                                size_t cache_plane_v4,   // uint4 per (layer, K|V) plane of the cache
                                size_t cache_seq_v4,     // uint4 per sequence inside a cache plane
                                int row_v4,              // uint4 per row (n_kv_heads * head_dim * sizeof(T) / 16)
                                const int32_t* __restrict__ yhat, int32_t* __restrict__ tokens, int tok_stride,
                                int write_tokens, int copy_rows) {
  pdl_begin();
  const int b = blockIdx.z;
  const int plane = blockIdx.y;
  const int pend = sd.pend[b];
  const size_t n = copy_rows ? (size_t)pend * row_v4 : 0;      // in-place layout: nothing to move, the append is the length bump
  const uint4* src = stage + plane * stage_plane_v4 + (size_t)sd.row_off[b] * row_v4;
  uint4* dst = cache + plane * cache_plane_v4 + b * cache_seq_v4 + (size_t)sd.F[b] * row_v4;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    dst[i] = src[i];
  if (write_tokens && blockIdx.x == 0 && plane == 0) {
    const int L = sd.Lc[b];
    const int ho = sd.head_off[b];
    int32_t* t = tokens + (size_t)b * tok_stride + sd.Fp[b];
    for (int i = threadIdx.x; i < L; i += blockDim.x) t[i] = yhat[ho + i];
  }
}

// ---------------------------------------------------------------------------------------------
// Next step's descriptor, computed on the device from this step's and the scan's block lengths (prefix topology), so
// that the host can enqueue the next pass without reading L back first:
//   F += pend;  pend = L;  N -= L;  Fp += L;  rows = pend + N (0 once N = 0);  row_off / head_off = prefix sums.
// One thread; runs after the commit kernel of the step (which still reads the current descriptor).
// ---------------------------------------------------------------------------------------------
__global__ void k_advance(StepDesc cur, int* __restrict__ nxt, int stride, const int32_t* __restrict__ L_commit, int batch) {
  pdl_begin();
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  int M = 0, Mh = 0;
  for (int b = 0; b < batch; ++b) {
    const int N = cur.N[b];
    const int L = N > 0 ? L_commit[b] : 0;
    const int pend = N > 0 ? cur.pend[b] : 0;
    const int N2 = N - L;
    nxt[0 * stride + b] = cur.F[b] + pend;
    nxt[1 * stride + b] = N2 > 0 ? L : 0;
    nxt[2 * stride + b] = N2;
    nxt[3 * stride + b] = M;
    nxt[4 * stride + b] = Mh;
    nxt[5 * stride + b] = cur.Fp[b] + L;
    M += N2 > 0 ? L + N2 : 0;
    Mh += N2;
  }
  nxt[3 * stride + batch] = M;
  nxt[4 * stride + batch] = Mh;
}

// ---------------------------------------------------------------------------------------------
// Scattered topology: lists, in ascending position, the rows of sequence b whose token is still [MASK].
// One block of 256 threads per sequence; rows [pend_b, pend_b + N_b) of the pass are its generation region.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_compact_masked(StepDesc sd, const int32_t* __restrict__ tokens, int tok_stride,
                                                        int mask_id, int* __restrict__ head_src,
                                                        int* __restrict__ head_pos) {
  __shared__ int warp_cnt[8];
  __shared__ int base;
  pdl_begin();
  const int b = blockIdx.x;
  const int pend = sd.pend[b], n = sd.N[b], F = sd.F[b], r0 = sd.row_off[b], ho = sd.head_off[b];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (threadIdx.x == 0) base = 0;
  __syncthreads();
  for (int j0 = 0; j0 < n; j0 += 256) {
    const int j = j0 + threadIdx.x;
    const int pos = F + pend + j;
    const bool m = (j < n) && tokens[(size_t)b * tok_stride + pos] == mask_id;
    const unsigned bal = __ballot_sync(0xffffffffu, m);
    if (lane == 0) warp_cnt[w] = __popc(bal);
    __syncthreads();
    int off = base;
    for (int i = 0; i < w; ++i) off += warp_cnt[i];
    if (m) {
      const int idx = off + __popc(bal & ((1u << lane) - 1u));
      head_src[ho + idx] = r0 + pend + j;
      head_pos[ho + idx] = pos;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      int t = 0;
      for (int i = 0; i < 8; ++i) t += warp_cnt[i];
      base += t;
    }
    __syncthreads();
  }
}

// ---------------------------------------------------------------------------------------------
// Token flips (Fig. 3): for every masked position of this step, compares its argmax with the one the previous step
// stored for the same absolute position (-1 = not scored before), counts the differences, and stores the new argmax.
// One block of 256 threads per sequence.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_flip_count(const int* __restrict__ head_off, const int* __restrict__ head_pos,
                                                    const int32_t* __restrict__ yhat, int32_t* __restrict__ prev,
                                                    int prev_stride, int32_t* __restrict__ o_flips,
                                                    int32_t* __restrict__ o_base) {
  __shared__ int red[2][8];
  pdl_begin();
  const int b = blockIdx.x;
  const int a = head_off[b], e = head_off[b + 1];
  int flips = 0, base = 0;
  for (int i = a + threadIdx.x; i < e; i += 256) {
    int32_t* p = prev + (size_t)b * prev_stride + head_pos[i];
    const int32_t old = *p, cur = yhat[i];
    if (old >= 0) { ++base; flips += (old != cur); }
    *p = cur;
  }
  flips = (int)warp_sum((float)flips);
  base = (int)warp_sum((float)base);
  if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = flips; red[1][threadIdx.x >> 5] = base; }
  __syncthreads();
  if (threadIdx.x == 0) {
    int f = 0, t = 0;
    for (int i = 0; i < 8; ++i) { f += red[0][i]; t += red[1][i]; }
    o_flips[b] = f;
    o_base[b] = t;
  }
}

// ---------------------------------------------------------------------------------------------
// Scattered commit: accepts the Lc_b most confident masked positions of sequence b (rank by counting: position i
// is accepted iff fewer than Lc_b positions beat it; a tie goes to the lower position) and writes their predictions
// into the token buffer at their own positions.  One block of 256 threads per sequence; scores staged in shared
// memory (dynamic, 4 bytes per masked position of the longest sequence).
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_scatter_commit(StepDesc sd, const float* __restrict__ score,
                                                        const int32_t* __restrict__ yhat, const int* __restrict__ head_pos,
                                                        int32_t* __restrict__ tokens, int tok_stride) {
  extern __shared__ float sc_s[];
  pdl_begin();
  const int b = blockIdx.x;
  const int a = sd.head_off[b], n = sd.head_off[b + 1] - a, L = sd.Lc[b];
  for (int i = threadIdx.x; i < n; i += 256) sc_s[i] = score[a + i];
  __syncthreads();
  for (int i = threadIdx.x; i < n; i += 256) {
    const float si = sc_s[i];
    int rank = 0;
    for (int j = 0; j < n; ++j) {
      const float sj = sc_s[j];
      rank += (sj > si) || (sj == si && j < i);
    }
    if (rank < L) tokens[(size_t)b * tok_stride + head_pos[a + i]] = yhat[a + i];
  }
}

__global__ void k_fill_mask(int32_t* tokens, int tok_stride, const int* __restrict__ P, const int* __restrict__ G,
                            int mask_id) {
  const int b = blockIdx.x;
  for (int i = threadIdx.x; i < G[b]; i += blockDim.x) tokens[(size_t)b * tok_stride + P[b] + i] = mask_id;
}

// Rotary table in double precision: cs[pos][i] = (cos, sin)(pos * theta^(-2i/dh)), stored fp32.
__global__ void k_rope_table(float2* __restrict__ cs, int max_len, int half, double theta) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= max_len * half) return;
  const int pos = idx / half, i = idx % half;
  const double inv = pow(theta, -(double)i / (double)half);
  double s, c;
  sincos((double)pos * inv, &s, &c);
  cs[idx] = make_float2((float)c, (float)s);
}

}  // namespace lsp
