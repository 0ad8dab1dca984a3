// Host step driver and C ABI of the LSP decode library (see include/lsp.h for the contract).
#include <cuda_runtime.h>

#include <algorithm>
#include <chrono>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <type_traits>
#include <string>
#include <vector>

#include "../../include/lsp.h"
#include "lsp_tuning.h"
#include "attention_mma.cuh"
#include "attention_simt.cuh"
#include "gemm_simt.cuh"
#include "misc_kernels.cuh"
#ifndef LSP_NO_UMMA
#include "gemm_stream.cuh"
#include "gemm_swap.cuh"
#include "attention_umma.cuh"
#endif

using namespace lsp;

namespace {
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
}  // namespace

struct lsp_ctx {
  lsp_model_cfg m{};
  lsp_sched_cfg s{};
  const void *embed = nullptr, *final_norm = nullptr, *w_head = nullptr;
  std::vector<const void*> attn_norm, w_qkv, w_o, ffn_norm, w_gate, w_up, w_down;
  char* kv_cache = nullptr;
  int max_batch = 0, max_len = 0, max_rows = 0;
  size_t esz = 0;
  cudaStream_t stream = nullptr;
  int gemm_impl = 1, attn_impl = 2, timing = 0, async_ops = 0, op_repeat = 1, op_rotate = 1, pdl = 1, attn_umma_min_rows = 0, attn_cluster = 1;
  // workspace carve (device)
  char *X = nullptr, *Nrm = nullptr, *Qb = nullptr, *Att = nullptr, *Hf = nullptr, *stage = nullptr;
  Top2* part = nullptr;
  int32_t* yhat = nullptr;
  float *pmax = nullptr, *margin = nullptr;
  int *row_seq = nullptr, *row_pos = nullptr, *head_src = nullptr, *head_pos = nullptr;
  int32_t* prev_yhat = nullptr;  // [max_batch][max_len] argmax of the previous step per absolute position (-1 = none)
  int* d_desc = nullptr;      // 2 descriptors of 7 arrays of (max_batch + 1) ints
  int* d_scan = nullptr;      // 6 arrays of max_batch (run, commit, flags, tau, flips, flip base)
  float2* rope_cs = nullptr;
  unsigned* d_status = nullptr;
  // pinned host mirrors
  int* h_desc = nullptr;
  int* h_scan = nullptr;
  unsigned* h_status = nullptr;
  // decode state (host is the authority; the device sees it through the descriptors)
  int32_t* tokens = nullptr;
  int tok_stride = 0, batch = 0, step = 0;
  std::vector<int> F, Fp, pend, N, Lprop, G;
  bool proposed = false;
  int score_rows = 0;
  int last_M = 0;
  int lagged = 0;                   // lsp_generate keeps the block lengths on the device (see lsp_set_option key 4)
  int lag_tail = 8;                 // ... until at most this many masked positions per sequence remain
  // ring of result slots for the lagged loop: scan outputs + status word (pinned), completion and timing events
  static constexpr int kRing = 4;
  int* h_ring = nullptr;            // kRing x (6 max_batch + 4) ints
  cudaEvent_t ring_done[kRing] = {}, ring_t0[kRing] = {}, ring_t1[kRing] = {};
  int kv_inplace = 0;               // K/V layout: 0 = staging planes + append copy, 1 = written in place (see lsp_set_option key 3)
  int last_attn_kernel = 0, last_attn_cluster = 1;   // what the last attention launch was (see lsp_get_counters)
  cudaEvent_t ev0 = nullptr, ev1 = nullptr;
  float timing_ms[8] = {0};
  std::vector<cudaEvent_t> seg_ev;      // per-class timing: pairs of events, created on demand
  std::vector<int> seg_cls;
  int seg_n = 0;
  double counters[18] = {0};            // see lsp_get_counters (16, 17 are filled on read)
  std::string err;
#ifndef LSP_NO_UMMA
  UmmaState umma;
  std::vector<CUtensorMap> attn_maps;    // per layer: cache K, cache V, staging K, staging V (tcgen05 attention)
#endif
};

namespace {

int fail(lsp_ctx* c, int code, const char* fmt, ...) {
  if (c) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    c->err = buf;
  }
  return code;
}

enum { CLS_MISC = 0, CLS_GEMM = 1, CLS_ATTN = 2, CLS_HEAD = 3, CLS_SCAN = 4, CLS_COMMIT = 5 };
enum { CNT_LAUNCHES = 0, CNT_GEMM_BYTES = 1, CNT_GEMM_FLOPS = 2, CNT_ATTN_BYTES = 3, CNT_APPEND_BYTES = 4,
       CNT_HEAD_BYTES = 5, CNT_HEAD_FLOPS = 6, CNT_STEPS = 7, CNT_CLS_LAUNCHES = 8 /* + class, 6 entries */,
       CNT_ATTN_FLOPS = 14, CNT_TOKENS = 15 };

// Counts n kernel launches of class cls.
void count_launch(lsp_ctx* c, int cls, int n = 1) {
  c->counters[CNT_LAUNCHES] += n;
  c->counters[CNT_CLS_LAUNCHES + cls] += n;
}

// Opens a timed segment of kernel class cls (only when per-class timing is on).
void seg_begin(lsp_ctx* c, int cls) {
  if (!c->timing) return;
  if ((size_t)(2 * c->seg_n + 2) > c->seg_ev.size()) {
    cudaEvent_t a, b;
    cudaEventCreate(&a);
    cudaEventCreate(&b);
    c->seg_ev.push_back(a);
    c->seg_ev.push_back(b);
    c->seg_cls.push_back(cls);
  }
  c->seg_cls[c->seg_n] = cls;
  cudaEventRecord(c->seg_ev[2 * c->seg_n], c->stream);
}
void seg_end(lsp_ctx* c) {
  if (!c->timing) return;
  cudaEventRecord(c->seg_ev[2 * c->seg_n + 1], c->stream);
  c->seg_n += 1;
}
// After a stream synchronisation: adds the elapsed time of every closed segment to its class.
void seg_collect(lsp_ctx* c) {
  if (!c->timing) return;
  for (int i = 0; i < c->seg_n; ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, c->seg_ev[2 * i], c->seg_ev[2 * i + 1]) == cudaSuccess) c->timing_ms[c->seg_cls[i]] += ms;
  }
  c->seg_n = 0;
}

#define CU(call)                                                                                   \
  do {                                                                                             \
    cudaError_t e_ = (call);                                                                       \
    if (e_ != cudaSuccess) return fail(c, LSP_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e_)); \
  } while (0)

// The device holds two descriptors (7 arrays of max_batch + 1 ints each); the synchronous path uses the first.
StepDesc desc_of(const lsp_ctx* c, int which = 0) {
  const int s = c->max_batch + 1;
  int* base = c->d_desc + (size_t)which * 7 * s;
  StepDesc d;
  d.F = base + 0 * s;
  d.pend = base + 1 * s;
  d.N = base + 2 * s;
  d.row_off = base + 3 * s;
  d.head_off = base + 4 * s;
  d.Fp = base + 5 * s;
  d.Lc = base + 6 * s;
  return d;
}

struct Carve {
  size_t off = 0;
  size_t take(size_t bytes) {
    const size_t o = off;
    off = align_up(off + bytes, 256);
    return o;
  }
};

struct Layout {
  size_t X, Nrm, Qb, Att, Hf, part, yhat, pmax, margin, row_seq, row_pos, head_src, head_pos, prev_yhat, desc, scan, rope, status,
      gemm_scratch, gemm_counters, stage, total;
};

constexpr size_t kGemmScratchBytes = 80u << 20;   // split-K partial tiles (the streaming GEMM needs 74 MiB at its widest)
constexpr int kGemmCounters = 4096;               // split-K arrival counters

int head_tiles_max(const lsp_model_cfg* m) { return (m->vocab + 63) / 64; }

Layout make_layout(const lsp_model_cfg* m, int max_batch, int max_len) {
  const size_t esz = m->dtype == 0 ? 4 : 2;
  const size_t R = (size_t)max_batch * max_len;
  const size_t qd = (size_t)m->n_heads * m->head_dim, kvd = (size_t)m->n_kv_heads * m->head_dim;
  Carve cv;
  Layout L;
  L.X = cv.take(R * m->d_model * esz);
  L.Nrm = cv.take(R * m->d_model * esz);
  L.Qb = cv.take(R * qd * esz);
  L.Att = cv.take(R * qd * esz);
  L.Hf = cv.take(R * m->d_ffn * esz);
  L.part = cv.take(R * head_tiles_max(m) * sizeof(Top2));
  L.yhat = cv.take(R * 4);
  L.pmax = cv.take(R * 4);
  L.margin = cv.take(R * 4);
  L.row_seq = cv.take(R * 4);
  L.row_pos = cv.take(R * 4);
  L.head_src = cv.take(R * 4);
  L.head_pos = cv.take(R * 4);
  L.prev_yhat = cv.take(R * 4);
  L.desc = cv.take(2 * 7 * (size_t)(max_batch + 1) * 4);
  L.scan = cv.take(6 * (size_t)max_batch * 4);
  L.rope = cv.take((size_t)max_len * (m->head_dim / 2) * sizeof(float2));
  L.status = cv.take(256);
  L.gemm_scratch = cv.take(kGemmScratchBytes);
  L.gemm_counters = cv.take(kGemmCounters * 4);
  L.stage = cv.take((size_t)m->n_layers * 2 * R * kvd * esz);
  L.total = cv.off;
  return L;
}

int check_model(const lsp_model_cfg* m) {
  if (!m) return LSP_ERR_ARG;
  if (m->dtype != 0 && m->dtype != 1) return LSP_ERR_ARG;
  if (m->n_layers < 1 || m->vocab < 2 || m->mask_id < 0 || m->mask_id >= m->vocab) return LSP_ERR_ARG;
  if (m->head_dim != 64 && m->head_dim != 128) return LSP_ERR_SHAPE;
  if (m->d_model % 64 || m->d_ffn % 64 || m->n_heads < 1 || m->n_kv_heads < 1 || m->n_heads % m->n_kv_heads)
    return LSP_ERR_SHAPE;
  return LSP_OK;
}

// ---- GEMM dispatch ------------------------------------------------------------------------------------
template <typename T, typename Epi>
int run_gemm(lsp_ctx* c, const T* A, const T* W0, const T* W1, int M, int NP, int K, int n_rows_w, const Epi& epi) {
  if (M <= 0) return LSP_OK;
  {
    // algorithmic work of this launch: every operand and result once
    const double cols = Epi::kDual ? 2.0 * NP : (double)NP;
    const double outb = Epi::kReduce ? 16.0 * M : (double)M * NP * sizeof(T);
    const int k_b = Epi::kReduce ? CNT_HEAD_BYTES : CNT_GEMM_BYTES, k_f = Epi::kReduce ? CNT_HEAD_FLOPS : CNT_GEMM_FLOPS;
    c->counters[k_b] += (cols * K + (double)M * K) * sizeof(T) + outb;
    c->counters[k_f] += 2.0 * M * cols * K;
    count_launch(c, Epi::kReduce ? CLS_HEAD : CLS_GEMM);
  }
  seg_begin(c, Epi::kReduce ? CLS_HEAD : CLS_GEMM);
  struct SegGuard { lsp_ctx* c; ~SegGuard() { seg_end(c); } } seg_guard{c};
#ifndef LSP_NO_UMMA
  if constexpr (std::is_same<T, bf16>::value) {
    if (c->gemm_impl == 1) {
      const int rc = umma_gemm<Epi>(c->umma, c->stream, A, W0, W1, M, NP, K, n_rows_w, epi, c->d_status);
      if (rc != 0) return fail(c, LSP_ERR_CUDA, "tcgen05 GEMM launch failed (%d): %s", rc, c->umma.err.c_str());
      return LSP_OK;
    }
  }
#endif
  dim3 grid((NP + SG_BN - 1) / SG_BN, (M + SG_BM - 1) / SG_BM);
  CU(launch_k(c->pdl, k_gemm_simt<T, Epi>, grid, dim3(256), 0, c->stream, A, W0, W1, M, NP, K, epi));
  return LSP_OK;
}

template <typename T>
int run_head(lsp_ctx* c, const T* hidden, int rows, int* n_tiles_out) {
  const lsp_model_cfg& m = c->m;
  EpiHead epi;
  epi.part = c->part;
  epi.vocab = m.vocab;
  epi.exclude_id = c->s.exclude_mask_logit ? m.mask_id : -1;
  int n_tiles = (m.vocab + SG_BN - 1) / SG_BN;
#ifndef LSP_NO_UMMA
  if (std::is_same<T, bf16>::value && c->gemm_impl == 1) n_tiles = umma_head_tiles(m.vocab);
#endif
  epi.n_tiles = n_tiles;
  *n_tiles_out = n_tiles;
  return run_gemm<T, EpiHead>(c, hidden, (const T*)c->w_head, (const T*)c->w_head, rows, m.vocab, m.d_model,
                              m.vocab, epi);
}

ScanParams scan_params(const lsp_ctx* c) {
  ScanParams p;
  p.mode = c->s.mode;
  p.tau = c->s.tau;
  p.alpha = c->s.alpha;
  p.beta = c->s.beta;
  p.l_min = c->s.l_min < 1 ? 1 : c->s.l_min;
  p.W = c->s.snap_window;
  p.fixed_k = c->s.fixed_k;
  p.delim = c->s.delim_bitmap;
  p.flag_tol = c->s.flag_tol;
  p.tie_tol = c->s.tie_tol;
  return p;
}

// merge partials -> scores, scan, copy the scan outputs to the pinned mirror (async)
int run_merge_scan(lsp_ctx* c, int rows, int n_tiles, const int* d_seq_off, int batch, bool count_flips, int* h_dst = nullptr) {
  if (rows > 0) {
    CU(launch_k(c->pdl, k_merge_partials, dim3((rows + 3) / 4), dim3(128), 0, c->stream, (const Top2*)c->part, n_tiles, rows, c->yhat,
                c->pmax, c->margin));
  }
  const float* score = c->s.score == 1 ? c->margin : c->pmax;
  int* o = c->d_scan;
  const int mb = c->max_batch;
  if (count_flips) {
    launch_k(c->pdl, k_flip_count, dim3(batch), dim3(256), 0, c->stream, d_seq_off, (const int*)c->head_pos,
             (const int32_t*)c->yhat, c->prev_yhat, c->max_len, o + 4 * mb, o + 5 * mb);
    CU(cudaGetLastError());
  }
  launch_k(c->pdl, k_lsp_scan, dim3(batch), dim3(32), 0, c->stream, score, c->yhat, c->margin, d_seq_off, scan_params(c), o, o + mb,
                                          (uint32_t*)(o + 2 * mb), (float*)(o + 3 * mb));
  CU(cudaGetLastError());
  if (h_dst) {        // a slot of the lagged loop's ring: scan outputs, then the status word
    CU(cudaMemcpyAsync(h_dst, c->d_scan, 6 * (size_t)mb * 4, cudaMemcpyDeviceToHost, c->stream));
    CU(cudaMemcpyAsync(h_dst + 6 * mb, c->d_status, 16, cudaMemcpyDeviceToHost, c->stream));
    return LSP_OK;
  }
  CU(cudaMemcpyAsync(c->h_scan, c->d_scan, 6 * (size_t)mb * 4, cudaMemcpyDeviceToHost, c->stream));
  CU(cudaMemcpyAsync(c->h_status, c->d_status, 16, cudaMemcpyDeviceToHost, c->stream));
  return LSP_OK;
}

int check_status(lsp_ctx* c) {
  if (c->h_status[0] != 0) {
    const unsigned code = c->h_status[0], where = c->h_status[1];
    cudaMemsetAsync(c->d_status, 0, 16, c->stream);
#ifndef LSP_NO_UMMA
    if (c->umma.counters) cudaMemsetAsync(c->umma.counters, 0, (size_t)c->umma.n_counters * 4, c->stream);
#endif
    cudaStreamSynchronize(c->stream);
    return fail(c, LSP_ERR_DEVICE_TIMEOUT, "device-side bounded wait expired (code %u, site %u)", code, where);
  }
  return LSP_OK;
}

// Suffix-over-prefix attention of layer l (Sec. 3.2: every query row of the pass sees the cached prefix [0, F_b) and all
// of the pass's own rows).  Reads the uploaded descriptor (F, row_off), Q from q, K/V from the cache and the staging
// planes of layer l; writes out.  max_q: most query rows of one sequence; max_keys: most keys of one sequence.
template <typename T>
int run_attention(lsp_ctx* c, int l, const T* Qb, T* Att, const StepDesc& sd, int B, int maxQ, int max_keys, int inplace) {
  const lsp_model_cfg& m = c->m;
  const int dh = m.head_dim, kvd = m.n_kv_heads * dh;
  const size_t plane = (size_t)c->max_rows * kvd;
  const size_t cplane = (size_t)c->max_batch * c->max_len * kvd;
  const T* stK = (const T*)c->stage + (size_t)(2 * l) * plane;
  const T* stV = stK + plane;
  const T* cK = (const T*)c->kv_cache + (size_t)(2 * l) * cplane;
  const T* cV = cK + cplane;
  const float scale = 1.0f / sqrtf((float)dh);
  count_launch(c, CLS_ATTN);
  seg_begin(c, CLS_ATTN);
  bool done = false;
  c->last_attn_kernel = 0;
  c->last_attn_cluster = 1;
#ifndef LSP_NO_UMMA
  if constexpr (std::is_same<T, bf16>::value) {
    // the tcgen05 kernel (128-row tiles; with few CTAs the keys of a row tile are split over a cluster); a row-count
    // threshold can send small passes to the 64-row mma.sync kernel instead
    if (c->attn_impl == 2 && dh == 128 && !c->attn_maps.empty() && maxQ * (m.n_heads / m.n_kv_heads) >= c->attn_umma_min_rows) {
      const int G = m.n_heads / m.n_kv_heads;
      const int row_tiles = (maxQ * G + AU_BM - 1) / AU_BM;
      // few CTAs: split every row tile's keys over a cluster of 2, 4 or 8 CTAs (merged through DSMEM)
      int cl = 1;
      if (c->attn_cluster) {
        const int key_tiles = (max_keys + AU_BN - 1) / AU_BN;
        const int ctas = row_tiles * m.n_kv_heads * B;
        // ... as long as that many clusters can be resident at once (this kernel, too, runs one CTA per SM)
        while (cl < 8 && 2 * cl * ctas <= c->umma.n_sm && 2 * cl <= key_tiles && ctas <= c->umma.max_clusters[2 * cl]) cl *= 2;
      }
      dim3 g3(row_tiles * cl, m.n_kv_heads, B);
      const float sl2 = scale * 1.4426950408889634f;
      const CUtensorMap* mp = &c->attn_maps[4 * l];
      launch_k(c->pdl, k_attn_umma, g3, dim3(AU_THREADS), (size_t)AU_SMEM, c->stream, cl, mp[0], mp[1], mp[2], mp[3],
               (const bf16*)Qb, Att, sd, m.n_heads, m.n_kv_heads, c->max_len, sl2, cl, inplace, c->d_status);
      c->last_attn_kernel = 2;
      c->last_attn_cluster = cl;
      done = true;
    }
  }
#endif
  if constexpr (std::is_same<T, bf16>::value) {
    if (!done && c->attn_impl >= 1) {
      const int G = m.n_heads / m.n_kv_heads;
      dim3 g2((maxQ * G + AM_BM - 1) / AM_BM, m.n_kv_heads, B);
      const float sl2 = scale * 1.4426950408889634f;
      if (dh == 128)
        launch_k(c->pdl, k_attn_mma<128>, dim3(g2), dim3(128), attn_mma_smem_bytes<128>(), c->stream, Qb, cK, cV, stK, stV, Att, sd, m.n_heads, m.n_kv_heads, (size_t)c->max_len * kvd, sl2, inplace);
      else
        launch_k(c->pdl, k_attn_mma<64>, dim3(g2), dim3(128), attn_mma_smem_bytes<64>(), c->stream, Qb, cK, cV, stK, stV, Att, sd, m.n_heads, m.n_kv_heads, (size_t)c->max_len * kvd, sl2, inplace);
      c->last_attn_kernel = 1;
      done = true;
    }
  }
  dim3 grid((maxQ + AS_BQ - 1) / AS_BQ, m.n_heads, B);
  if (done) {
  } else if (dh == 128)
    launch_k(c->pdl, k_attn_simt<T, 128>, dim3(grid), dim3(128), 0, c->stream, Qb, cK, cV, stK, stV, Att, sd, m.n_heads, m.n_kv_heads,
                                                     (size_t)c->max_len * kvd, scale, inplace);
  else
    launch_k(c->pdl, k_attn_simt<T, 64>, dim3(grid), dim3(128), 0, c->stream, Qb, cK, cV, stK, stV, Att, sd, m.n_heads, m.n_kv_heads,
                                                    (size_t)c->max_len * kvd, scale, inplace);
  seg_end(c);
  CU(cudaGetLastError());
  return LSP_OK;
}

// Launch shape of one denoiser pass.  The row counts may be upper bounds of what the device-side descriptor says (the
// lagged loop sizes a pass before it has read the previous block lengths): rows past the real ones are inert.
struct PassDims {
  int M = 0, Mh = 0;            // packed rows of the pass; rows that go through the LM head
  int maxQ = 0, max_keys = 0;   // most rows / most keys of one sequence
  double attn_bytes = 0, attn_flops = 0;      // algorithmic attention work per layer (accounting only)
};

// Enqueues one pass (Algorithm 1: forward pass, scores, scan) that reads descriptor sd on the device.
template <typename T>
int enqueue_pass(lsp_ctx* c, const StepDesc& sd, int B, const PassDims& pd, int* h_dst) {
  const lsp_model_cfg& m = c->m;
  const bool scattered = c->s.topology == 1;
  const int M = pd.M, Mh = pd.Mh;
  const int d = m.d_model, dh = m.head_dim, qd = m.n_heads * dh, kvd = m.n_kv_heads * dh;
  T* X = (T*)c->X;
  T* Nrm = (T*)c->Nrm;
  T* Qb = (T*)c->Qb;
  T* Att = (T*)c->Att;
  T* Hf = (T*)c->Hf;
  seg_begin(c, CLS_MISC);
  launch_k(c->pdl, k_assemble_embed<T>, dim3(M), dim3(128), 0, c->stream, sd, B, c->tokens, c->tok_stride, m.mask_id, (const T*)c->embed, d, X,
                                               c->row_seq, c->row_pos, c->head_src, c->head_pos, scattered ? 1 : 0);
  CU(cudaGetLastError());
  if (scattered) {
    launch_k(c->pdl, k_compact_masked, dim3(B), dim3(256), 0, c->stream, sd, (const int32_t*)c->tokens, c->tok_stride, m.mask_id,
             c->head_src, c->head_pos);
    CU(cudaGetLastError());
    count_launch(c, CLS_MISC);
  }
  seg_end(c);
  count_launch(c, CLS_MISC);
  const size_t plane = (size_t)c->max_rows * kvd;           // elements per staged (layer, K|V) plane
  const size_t cplane = (size_t)c->max_batch * c->max_len * kvd;
  for (int l = 0; l < m.n_layers; ++l) {
    // this pass's K/V: the staging planes, or (in-place layout) each row's own slot in the cache planes
    T* stK = c->kv_inplace ? (T*)c->kv_cache + (size_t)(2 * l) * cplane : (T*)c->stage + (size_t)(2 * l) * plane;
    T* stV = stK + (c->kv_inplace ? cplane : plane);
    seg_begin(c, CLS_MISC);
    launch_k(c->pdl, k_rmsnorm<T>, dim3(M), dim3(256), 0, c->stream, X, (const T*)c->attn_norm[l], Nrm, nullptr, d, m.rms_eps);
    seg_end(c);
    count_launch(c, CLS_MISC);
    CU(cudaGetLastError());
    {
      EpiQKVRope<T> e{Qb, stK, stV, c->rope_cs, c->row_pos, m.n_heads, m.n_kv_heads, dh / 2, c->row_seq,
                      c->kv_inplace ? c->max_len : 0};
      const int rc = run_gemm<T>(c, Nrm, (const T*)c->w_qkv[l], (const T*)c->w_qkv[l], M, (qd + 2 * kvd) / 2, d,
                                 qd + 2 * kvd, e);
      if (rc) return rc;
    }
    {
      c->counters[CNT_ATTN_BYTES] += pd.attn_bytes;
      c->counters[CNT_ATTN_FLOPS] += pd.attn_flops;
      const int rc = run_attention<T>(c, l, Qb, Att, sd, B, pd.maxQ, pd.max_keys, c->kv_inplace);
      if (rc) return rc;
    }
    {
      EpiResidual<T> e{X, d};
      const int rc = run_gemm<T>(c, Att, (const T*)c->w_o[l], (const T*)c->w_o[l], M, d, qd, d, e);
      if (rc) return rc;
    }
    seg_begin(c, CLS_MISC);
    launch_k(c->pdl, k_rmsnorm<T>, dim3(M), dim3(256), 0, c->stream, X, (const T*)c->ffn_norm[l], Nrm, nullptr, d, m.rms_eps);
    seg_end(c);
    count_launch(c, CLS_MISC);
    CU(cudaGetLastError());
    {
      EpiSwiGLU<T> e{Hf, m.d_ffn};
      const int rc = run_gemm<T>(c, Nrm, (const T*)c->w_gate[l], (const T*)c->w_up[l], M, m.d_ffn, d, m.d_ffn, e);
      if (rc) return rc;
    }
    {
      EpiResidual<T> e{X, d};
      const int rc = run_gemm<T>(c, Hf, (const T*)c->w_down[l], (const T*)c->w_down[l], M, d, m.d_ffn, d, e);
      if (rc) return rc;
    }
  }
  // masked rows only: final norm (gathered), fused head, merge, scan
  seg_begin(c, CLS_MISC);
  launch_k(c->pdl, k_rmsnorm<T>, dim3(Mh), dim3(256), 0, c->stream, X, (const T*)c->final_norm, Nrm, c->head_src, d, m.rms_eps);
  seg_end(c);
  count_launch(c, CLS_MISC);
  CU(cudaGetLastError());
  int n_tiles = 0;
  int rc = run_head<T>(c, Nrm, Mh, &n_tiles);
  if (rc) return rc;
  seg_begin(c, CLS_SCAN);
  rc = run_merge_scan(c, Mh, n_tiles, sd.head_off, B, true, h_dst);
  seg_end(c);
  count_launch(c, CLS_SCAN, 2);
  c->counters[CNT_STEPS] += 1;
  return rc;
}

// Fills the pinned descriptor mirror from the host's state (arrays 0..5) and returns the pass's exact launch shape.
PassDims host_descriptor(lsp_ctx* c) {
  const lsp_model_cfg& m = c->m;
  const int B = c->batch, s = c->max_batch + 1;
  const bool scattered = c->s.topology == 1;
  const double qd = (double)m.n_heads * m.head_dim, kvd = (double)m.n_kv_heads * m.head_dim;
  int* h = c->h_desc;
  PassDims pd;
  for (int b = 0; b < B; ++b) {
    const int pend = c->N[b] > 0 ? c->pend[b] : 0;
    // rows past the pending block: the masked suffix (prefix topology) or the whole generation region (scattered)
    const int tail = c->N[b] > 0 ? (scattered ? c->G[b] : c->N[b]) : 0;
    const int rows = pend + tail;
    h[0 * s + b] = c->F[b];
    h[1 * s + b] = pend;
    h[2 * s + b] = tail;
    h[3 * s + b] = pd.M;
    h[4 * s + b] = pd.Mh;
    h[5 * s + b] = c->Fp[b];
    pd.M += rows;
    pd.Mh += c->N[b];
    pd.maxQ = std::max(pd.maxQ, rows);
    if (rows > 0) {
      pd.max_keys = std::max(pd.max_keys, c->F[b] + rows);
      // algorithmic attention traffic: every key/value row of the sequence once per layer, plus Q and O
      pd.attn_bytes += (2.0 * (c->F[b] + rows) * kvd + 2.0 * rows * qd) * c->esz;
      pd.attn_flops += 4.0 * rows * (c->F[b] + rows) * qd;
    }
  }
  h[3 * s + B] = pd.M;
  h[4 * s + B] = pd.Mh;
  return pd;
}

template <typename T>
int step_impl(lsp_ctx* c, lsp_step_rec* rec) {
  const int B = c->batch, s = c->max_batch + 1;
  const bool scattered = c->s.topology == 1;
  const PassDims pd = host_descriptor(c);
  const int M = pd.M, Mh = pd.Mh;
  if (M == 0) return fail(c, LSP_ERR_STATE, "lsp_denoise_step: every sequence is already fully committed");
  const auto host_t0 = std::chrono::steady_clock::now();
  CU(cudaEventRecord(c->ev0, c->stream));
  // the step owns the first six arrays; the seventh (commit lengths) belongs to lsp_commit, whose upload from the same
  // pinned mirror may still be in flight
  CU(cudaMemcpyAsync(c->d_desc, c->h_desc, 6 * (size_t)s * 4, cudaMemcpyHostToDevice, c->stream));
  int rc = enqueue_pass<T>(c, desc_of(c), B, pd, nullptr);
  if (rc) return rc;
  CU(cudaEventRecord(c->ev1, c->stream));
  // host time spent queueing the pass (everything between the two event records)
  c->timing_ms[7] += std::chrono::duration<float, std::milli>(std::chrono::steady_clock::now() - host_t0).count();
  CU(cudaStreamSynchronize(c->stream));
  seg_collect(c);
  rc = check_status(c);
  if (rc) return rc;
  float ms = 0.f;
  CU(cudaEventElapsedTime(&ms, c->ev0, c->ev1));
  const int mb = c->max_batch;
  for (int b = 0; b < B; ++b) {
    c->Lprop[b] = c->N[b] > 0 ? c->h_scan[mb + b] : 0;
    if (rec) {
      rec[b].step = c->step;
      rec[b].n_before = c->N[b];
      rec[b].rows = c->N[b] > 0 ? c->pend[b] + (scattered ? c->G[b] : c->N[b]) : 0;
      rec[b].flips = c->N[b] > 0 ? c->h_scan[4 * mb + b] : 0;
      rec[b].flip_base = c->N[b] > 0 ? c->h_scan[5 * mb + b] : 0;
      rec[b].l_run = c->h_scan[b];
      rec[b].l_commit = c->h_scan[mb + b];
      rec[b].flags = (unsigned)c->h_scan[2 * mb + b];
      memcpy(&rec[b].tau_used, &c->h_scan[3 * mb + b], 4);
      rec[b].ms = ms;
    }
  }
  c->timing_ms[6] += ms;
  c->proposed = true;
  c->score_rows = Mh;
  c->last_M = M;
  return LSP_OK;
}

static int scan_outputs(lsp_ctx* c, int batch, int32_t* l_run, int32_t* l_commit, uint32_t* flags, float* tau_used) {
  CU(cudaStreamSynchronize(c->stream));
  int rc = check_status(c);
  if (rc) return rc;
  const int mb = c->max_batch;
  for (int b = 0; b < batch; ++b) {
    if (l_run) l_run[b] = c->h_scan[b];
    if (l_commit) l_commit[b] = c->h_scan[mb + b];
    if (flags) flags[b] = (uint32_t)c->h_scan[2 * mb + b];
    if (tau_used) memcpy(&tau_used[b], &c->h_scan[3 * mb + b], 4);
  }
  return LSP_OK;
}

static int upload_offsets(lsp_ctx* c, const int32_t* seq_offsets, int batch, int* rows_out) {
  if (!seq_offsets || batch < 1 || batch > c->max_batch) return fail(c, LSP_ERR_ARG, "bad seq_offsets / batch");
  if (seq_offsets[0] != 0) return fail(c, LSP_ERR_ARG, "seq_offsets[0] must be 0");
  for (int b = 0; b < batch; ++b)
    if (seq_offsets[b + 1] < seq_offsets[b]) return fail(c, LSP_ERR_ARG, "seq_offsets must ascend");
  const int rows = seq_offsets[batch];
  if (rows > c->max_rows) return fail(c, LSP_ERR_ARG, "rows %d exceed max_batch*max_len %d", rows, c->max_rows);
  const int s = c->max_batch + 1;
  int* h = c->h_desc + 4 * s;
  for (int b = 0; b <= batch; ++b) h[b] = seq_offsets[b];
  CU(cudaMemcpyAsync(c->d_desc + 4 * s, h, (size_t)(batch + 1) * 4, cudaMemcpyHostToDevice, c->stream));
  *rows_out = rows;
  return LSP_OK;
}

template <typename T>
static int op_linear_impl(lsp_ctx* c, int op, const void* A, const void* W, const void* W2, void* out, int M, int N,
                          int K) {
  if (op == 0) {
    EpiStore<T> e{(T*)out, N};
    return run_gemm<T>(c, (const T*)A, (const T*)W, (const T*)W, M, N, K, N, e);
  } else if (op == 1) {
    EpiResidual<T> e{(T*)out, N};
    return run_gemm<T>(c, (const T*)A, (const T*)W, (const T*)W, M, N, K, N, e);
  } else {
    EpiSwiGLU<T> e{(T*)out, N};
    return run_gemm<T>(c, (const T*)A, (const T*)W, (const T*)W2, M, N, K, N, e);
  }
}

}  // namespace

extern "C" {

size_t lsp_workspace_bytes(const lsp_model_cfg* model, int max_batch, int max_len) {
  if (check_model(model) != LSP_OK || max_batch < 1 || max_len < 2) return 0;
  return make_layout(model, max_batch, max_len).total;
}

size_t lsp_kv_cache_bytes(const lsp_model_cfg* model, int max_batch, int max_len) {
  if (check_model(model) != LSP_OK || max_batch < 1 || max_len < 2) return 0;
  const size_t esz = model->dtype == 0 ? 4 : 2;
  return (size_t)model->n_layers * 2 * max_batch * max_len * model->n_kv_heads * model->head_dim * esz;
}

int lsp_init(lsp_ctx** out, const lsp_model_cfg* model, const lsp_sched_cfg* sched, const lsp_weights* w,
             void* kv_cache, void* workspace, size_t workspace_bytes, int max_batch, int max_len, void* cuda_stream) {
  if (!out) return LSP_ERR_ARG;
  *out = nullptr;
  if (!model || !sched || !w || !kv_cache || !workspace || max_batch < 1 || max_len < 2) return LSP_ERR_ARG;
  int rc = check_model(model);
  if (rc) return rc;
  if (!w->embed || !w->final_norm || !w->w_head || !w->attn_norm || !w->w_qkv || !w->w_o || !w->ffn_norm ||
      !w->w_gate || !w->w_up || !w->w_down)
    return LSP_ERR_ARG;
  const Layout L = make_layout(model, max_batch, max_len);
  if (workspace_bytes < L.total) return LSP_ERR_WORKSPACE;
  if (((uintptr_t)workspace & 255) || ((uintptr_t)kv_cache & 255)) return LSP_ERR_ARG;
  lsp_ctx* c = new lsp_ctx();
  c->m = *model;
  c->s = *sched;
  c->embed = w->embed;
  c->final_norm = w->final_norm;
  c->w_head = w->w_head;
  for (int l = 0; l < model->n_layers; ++l) {
    c->attn_norm.push_back(w->attn_norm[l]);
    c->w_qkv.push_back(w->w_qkv[l]);
    c->w_o.push_back(w->w_o[l]);
    c->ffn_norm.push_back(w->ffn_norm[l]);
    c->w_gate.push_back(w->w_gate[l]);
    c->w_up.push_back(w->w_up[l]);
    c->w_down.push_back(w->w_down[l]);
  }
  c->kv_cache = (char*)kv_cache;
  c->max_batch = max_batch;
  c->max_len = max_len;
  c->max_rows = max_batch * max_len;
  c->esz = model->dtype == 0 ? 4 : 2;
  c->stream = (cudaStream_t)cuda_stream;
  char* ws = (char*)workspace;
  c->X = ws + L.X;
  c->Nrm = ws + L.Nrm;
  c->Qb = ws + L.Qb;
  c->Att = ws + L.Att;
  c->Hf = ws + L.Hf;
  c->part = (Top2*)(ws + L.part);
  c->yhat = (int32_t*)(ws + L.yhat);
  c->pmax = (float*)(ws + L.pmax);
  c->margin = (float*)(ws + L.margin);
  c->row_seq = (int*)(ws + L.row_seq);
  c->row_pos = (int*)(ws + L.row_pos);
  c->head_src = (int*)(ws + L.head_src);
  c->head_pos = (int*)(ws + L.head_pos);
  c->prev_yhat = (int32_t*)(ws + L.prev_yhat);
  c->d_desc = (int*)(ws + L.desc);
  c->d_scan = (int*)(ws + L.scan);
  c->rope_cs = (float2*)(ws + L.rope);
  c->d_status = (unsigned*)(ws + L.status);
  c->stage = ws + L.stage;
  cudaError_t e = cudaHostAlloc((void**)&c->h_desc, 7 * (size_t)(max_batch + 1) * 4, cudaHostAllocDefault);
  if (e == cudaSuccess) e = cudaHostAlloc((void**)&c->h_scan, 6 * (size_t)max_batch * 4, cudaHostAllocDefault);
  if (e == cudaSuccess) e = cudaHostAlloc((void**)&c->h_status, 16, cudaHostAllocDefault);
  if (e == cudaSuccess) e = cudaHostAlloc((void**)&c->h_ring, (size_t)lsp_ctx::kRing * (6 * max_batch + 4) * 4, cudaHostAllocDefault);
  for (int i = 0; i < lsp_ctx::kRing && e == cudaSuccess; ++i) {
    e = cudaEventCreateWithFlags(&c->ring_done[i], cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreate(&c->ring_t0[i]);
    if (e == cudaSuccess) e = cudaEventCreate(&c->ring_t1[i]);
  }
  if (e == cudaSuccess) e = cudaEventCreate(&c->ev0);
  if (e == cudaSuccess) e = cudaEventCreate(&c->ev1);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->d_status, 0, 256, c->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(ws + L.gemm_counters, 0, kGemmCounters * 4, c->stream);
  if (e == cudaSuccess) {
    const int n = max_len * (model->head_dim / 2);
    k_rope_table<<<(n + 255) / 256, 256, 0, c->stream>>>(c->rope_cs, max_len, model->head_dim / 2,
                                                       (double)model->rope_theta);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
  if (e != cudaSuccess) {
    lsp_destroy(c);
    return LSP_ERR_CUDA;
  }
  c->h_status[0] = 0;
#ifndef LSP_NO_UMMA
  if (model->dtype == 1) {
    c->umma.scratch = (float*)(ws + L.gemm_scratch);
    c->umma.scratch_bytes = kGemmScratchBytes;
    c->umma.counters = (unsigned*)(ws + L.gemm_counters);
    c->umma.n_counters = kGemmCounters;
    cudaFuncSetAttribute(k_attn_mma<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_mma_smem_bytes<128>());
    cudaFuncSetAttribute(k_attn_mma<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_mma_smem_bytes<64>());
    const int urc = umma_init(c->umma);
    if (urc != 0) {
      lsp_destroy(c);
      return LSP_ERR_CUDA;
    }
    stream_query_clusters(c->umma);
    if (model->head_dim == 128) {
      // tensor maps of the K / V planes for the tcgen05 attention kernel
      const int kvd = model->n_kv_heads * model->head_dim;
      const size_t plane = (size_t)max_batch * max_len * kvd * 2;      // bytes of one (layer, K|V) plane, cache and staging alike
      c->attn_maps.resize((size_t)4 * model->n_layers);
      bool ok = cudaFuncSetAttribute(k_attn_umma, cudaFuncAttributeMaxDynamicSharedMemorySize, AU_SMEM) == cudaSuccess;
      for (int l = 0; l < model->n_layers && ok; ++l) {
        const char* ck = c->kv_cache + (size_t)(2 * l) * plane;
        const char* sk = c->stage + (size_t)(2 * l) * plane;
        ok = attn_umma_map(c->umma, &c->attn_maps[4 * l + 0], ck, (size_t)max_batch * max_len, kvd) &&
             attn_umma_map(c->umma, &c->attn_maps[4 * l + 1], ck + plane, (size_t)max_batch * max_len, kvd) &&
             attn_umma_map(c->umma, &c->attn_maps[4 * l + 2], sk, (size_t)max_batch * max_len, kvd) &&
             attn_umma_map(c->umma, &c->attn_maps[4 * l + 3], sk + plane, (size_t)max_batch * max_len, kvd);
      }
      if (!ok) c->attn_maps.clear();      // the mma.sync kernel takes over
    }
  }
#endif
  *out = c;
  return LSP_OK;
}

int lsp_set_sched(lsp_ctx* c, const lsp_sched_cfg* sched) {
  if (!c || !sched) return LSP_ERR_ARG;
  if (sched->mode < 0 || sched->mode > 2 || sched->score < 0 || sched->score > 1 || sched->topology < 0 ||
      sched->topology > 1)
    return fail(c, LSP_ERR_ARG, "lsp_set_sched: bad mode/score/topology");
  if (sched->topology != c->s.topology && c->tokens && c->step > 0) {
    bool active = false;
    for (int b = 0; b < c->batch; ++b) active |= c->N[b] > 0;
    if (active) return fail(c, LSP_ERR_STATE, "lsp_set_sched: the topology cannot change in the middle of a decode");
  }
  c->s = *sched;
  return LSP_OK;
}

int lsp_set_option(lsp_ctx* c, int key, int value) {
  if (!c) return LSP_ERR_ARG;
  if (key == 0) c->gemm_impl = value;
  else if (key == 1) c->attn_impl = value;
  else if (key == 2) c->timing = value;
  else if (key == 3) {
    if (c->tokens && c->step > 0) {
      bool active = false;
      for (int b = 0; b < c->batch; ++b) active |= c->N[b] > 0;
      if (active && (value != 0) != (c->kv_inplace != 0))
        return fail(c, LSP_ERR_STATE, "lsp_set_option: the K/V layout cannot change in the middle of a decode");
    }
    c->kv_inplace = value ? 1 : 0;
  }
  else if (key == 4) c->lagged = value ? 1 : 0;
  else return fail(c, LSP_ERR_ARG, "lsp_set_option: unknown key %d", key);
  return LSP_OK;
}

int lsp_debug_set(lsp_ctx* c, int key, int value) {
  if (!c) return LSP_ERR_ARG;
  if (key == 28) c->attn_umma_min_rows = value;
  else if (key == 31) c->lag_tail = value < 1 ? 1 : value;
  else if (key == 36) c->umma.swap_min_rows = value;
  else if (key == 37) c->umma.swap_max_rows = value;
  else if (key == 38) c->umma.swap_force = value ? 1 : 0;
  else if (key == 39) c->umma.stream_half_tile1 = value ? 1 : 0;
  else if (key == 30) c->attn_cluster = value ? 1 : 0;
  else if (key == 3) c->async_ops = value;
  else if (key == 4) c->op_repeat = value < 1 ? 1 : value;
  else if (key == 5) c->op_rotate = value < 1 ? 1 : value;
#ifndef LSP_NO_UMMA
  else if (key == 10) c->umma.target_ctas = value;
  else if (key == 11) c->umma.max_stages = value < 1 ? 1 : (value > UM_MAX_STAGES ? UM_MAX_STAGES : value);
  else if (key == 25) { c->pdl = value ? 1 : 0; c->umma.pdl = c->pdl; }
  else if (key == 17) c->umma.stream_grid_mode = value;
  else if (key == 18) c->umma.stream_even_max_rows = value;
  else if (key == 19) c->umma.stream_two_tiles = value == 2 ? 2 : 1;
  else if (key == 27) c->umma.stream_half_sm = value ? 1 : 0;
  else if (key == 29) c->umma.stream_cluster = value ? 1 : 0;
  else if (key == 32) c->umma.stream_bn_dual = (value == 192 || value == 256) ? value : 0;
  else if (key == 33) c->umma.stream_exchange = value ? 1 : 0;
  else if (key == 26) c->umma.stream_issuers = value == 1 ? 1 : 2;
  else if (key == 24) c->umma.stream_big_mt = (value == 1 || value == 2) ? value : 3;
  else if (key == 20) c->umma.stream_bn2 = (value == 256 || value == 128) ? value : 0;
  else if (key == 23) c->umma.stream_bn = (value == 256 || value == 128) ? value : 0;
  else if (key == 21) c->umma.stream_atoms = value;
  else if (key == 22) c->umma.stream_min_stages2 = value < 2 ? 2 : value;
#endif
  else return fail(c, LSP_ERR_ARG, "lsp_debug_set: unknown key %d", key);
  return LSP_OK;
}

int lsp_begin(lsp_ctx* c, int32_t* tokens, int token_stride, const int32_t* prompt_len, const int32_t* gen_len,
              int batch) {
  if (!c || !tokens || !prompt_len || !gen_len) return LSP_ERR_ARG;
  if (batch < 1 || batch > c->max_batch) return fail(c, LSP_ERR_ARG, "lsp_begin: batch %d not in [1, %d]", batch, c->max_batch);
  for (int b = 0; b < batch; ++b)
    if (prompt_len[b] < 1 || gen_len[b] < 1 || prompt_len[b] + gen_len[b] > c->max_len ||
        prompt_len[b] + gen_len[b] > token_stride)
      return fail(c, LSP_ERR_ARG, "lsp_begin: sequence %d has prompt %d + gen %d outside [2, min(max_len %d, stride %d)]",
                  b, prompt_len[b], gen_len[b], c->max_len, token_stride);
  c->tokens = tokens;
  c->tok_stride = token_stride;
  c->batch = batch;
  c->step = 0;
  c->F.assign(batch, 0);
  c->Fp.assign(prompt_len, prompt_len + batch);
  c->pend.assign(prompt_len, prompt_len + batch);   // the prompt is step 0's pending block (CacheInit)
  c->N.assign(gen_len, gen_len + batch);
  c->G.assign(gen_len, gen_len + batch);
  c->Lprop.assign(batch, 0);
  CU(cudaMemsetAsync(c->prev_yhat, 0xFF, (size_t)c->max_rows * 4, c->stream));      // -1: no previous prediction
  c->proposed = false;
  // mask fill: reuse the descriptor's F/pend slots to pass P and G
  const int s = c->max_batch + 1;
  for (int b = 0; b < batch; ++b) { c->h_desc[b] = prompt_len[b]; c->h_desc[s + b] = gen_len[b]; }
  CU(cudaMemcpyAsync(c->d_desc, c->h_desc, 2 * (size_t)s * 4, cudaMemcpyHostToDevice, c->stream));
  k_fill_mask<<<batch, 256, 0, c->stream>>>(tokens, token_stride, c->d_desc, c->d_desc + s, c->m.mask_id);
  CU(cudaGetLastError());
  CU(cudaStreamSynchronize(c->stream));
  return LSP_OK;
}

int lsp_denoise_step(lsp_ctx* c, lsp_step_rec* rec) {
  if (!c) return LSP_ERR_ARG;
  if (!c->tokens) return fail(c, LSP_ERR_STATE, "lsp_denoise_step before lsp_begin");
  return c->m.dtype == 0 ? step_impl<float>(c, rec) : step_impl<bf16>(c, rec);
}

}  // extern "C"

namespace {

// Enqueues the commit kernel(s) of a step that read descriptor sd (whose Lc array holds the block lengths).
// max_pend: the longest pending block (an upper bound is enough: it only sizes the copy's grid).
int enqueue_commit(lsp_ctx* c, const StepDesc& sd, int B, int max_pend, int max_n) {
  const lsp_model_cfg& m = c->m;
  const size_t kvd = (size_t)m.n_kv_heads * m.head_dim;
  const int row_v4 = (int)(kvd * c->esz / 16);
  const size_t stage_plane_v4 = (size_t)c->max_rows * row_v4;
  const size_t cache_seq_v4 = (size_t)c->max_len * row_v4;
  const size_t cache_plane_v4 = (size_t)c->max_batch * cache_seq_v4;
  size_t n_v4 = (size_t)max_pend * row_v4;
  int chunks = (int)((n_v4 + 256 * 8 - 1) / (256 * 8));
  if (chunks < 1) chunks = 1;
  if (chunks > 64) chunks = 64;
  dim3 grid(chunks, m.n_layers * 2, B);
  seg_begin(c, CLS_COMMIT);
  const bool scattered = c->s.topology == 1;
  const bool copy = !c->kv_inplace;          // in-place layout: the pending block's K/V are already where they belong
  if (!copy) grid = dim3(1, 1, B);
  if ((!scattered || max_pend > 0) && (copy || !scattered)) {
    launch_k(c->pdl, k_commit_append, dim3(grid), dim3(256), 0, c->stream, sd, (const uint4*)c->stage, (uint4*)c->kv_cache,
                                                 stage_plane_v4, cache_plane_v4, cache_seq_v4, row_v4, c->yhat,
                                                 c->tokens, c->tok_stride, scattered ? 0 : 1, copy ? 1 : 0);
    count_launch(c, CLS_COMMIT);
  }
  if (scattered) {
    // accept the L most confident masked positions wherever they are
    const float* score = c->s.score == 1 ? c->margin : c->pmax;
    launch_k(c->pdl, k_scatter_commit, dim3(B), dim3(256), (size_t)max_n * sizeof(float), c->stream, sd, score,
             (const int32_t*)c->yhat, (const int*)c->head_pos, c->tokens, c->tok_stride);
    count_launch(c, CLS_COMMIT);
  }
  seg_end(c);
  CU(cudaGetLastError());
  return LSP_OK;
}

// Algorithm 1's loop with the block lengths kept on the device (prefix topology).  Pass j+1 is enqueued before L_j has
// been read back: the scan's L goes straight into the commit kernel, k_advance derives the next descriptor from it on
// the device, and the host only needs the row counts to size the launches -- and those it knows one step late, because
// a sequence's rows at step j+1 (pending block + masked suffix) are exactly its masked suffix at step j, N_j, which
// follows from L_{j-1}.  The LM-head row count is an upper bound (N_j - 1); rows beyond the real ones are inert.
// Near the end (at most lag_tail masked positions per sequence left) every step is read before the next one is sized,
// so that no empty pass is launched after the last commit; a sequence that runs to its end earlier costs one empty pass.
template <typename T>
int generate_lagged(lsp_ctx* c, lsp_step_rec* recs, int max_recs, int* n_steps) {
  const lsp_model_cfg& m = c->m;
  const int B = c->batch, s = c->max_batch + 1, mb = c->max_batch, R = lsp_ctx::kRing;
  const int slot_ints = 6 * mb + 4;
  const double qd = (double)m.n_heads * m.head_dim, kvd = (double)m.n_kv_heads * m.head_dim;
  std::vector<int> total(B);                       // prompt + generation length: F + rows of any pass of the sequence
  for (int b = 0; b < B; ++b) total[b] = c->Fp[b] + c->N[b];
  // host state = state before step `read` (results of steps < read have been applied)
  int launched = 0, read = 0, used = 0, steps_done = 0;
  int last_L = 1;                                  // longest block of the last step read (sizes the next append's grid)
  auto apply_results = [&](int j) -> int {         // waits for step j, folds its block lengths into the host state
    const int slot = j % R;
    CU(cudaEventSynchronize(c->ring_done[slot]));
    const int* r = c->h_ring + (size_t)slot * slot_ints;
    if (r[6 * mb] != 0) {
      memcpy(c->h_status, r + 6 * mb, 16);
      return check_status(c);
    }
    float ms = 0.f;
    cudaEventElapsedTime(&ms, c->ring_t0[slot], c->ring_t1[slot]);
    c->timing_ms[6] += ms;
    bool any = false;
    for (int b = 0; b < B; ++b) any |= c->N[b] > 0;
    for (int b = 0; b < B; ++b) {
      const int L = c->N[b] > 0 ? r[mb + b] : 0;
      if (any && recs && used < max_recs) {
        lsp_step_rec& o = recs[used++];
        o.step = c->step;
        o.n_before = c->N[b];
        o.rows = c->N[b] > 0 ? c->pend[b] + c->N[b] : 0;
        o.l_run = r[b];
        o.l_commit = r[mb + b];
        o.flags = (unsigned)r[2 * mb + b];
        memcpy(&o.tau_used, &r[3 * mb + b], 4);
        o.ms = ms;
        o.flips = c->N[b] > 0 ? r[4 * mb + b] : 0;
        o.flip_base = c->N[b] > 0 ? r[5 * mb + b] : 0;
      }
      if (c->N[b] == 0) continue;
      if (L < 1 || L > c->N[b]) return fail(c, LSP_ERR_STATE, "lagged loop: step %d proposed L[%d] = %d outside [1, %d]", j, b, L, c->N[b]);
      if (!c->kv_inplace) c->counters[CNT_APPEND_BYTES] += 2.0 * c->pend[b] * kvd * c->esz * 2.0 * m.n_layers;
      c->counters[CNT_TOKENS] += L;
      c->F[b] += c->pend[b];
      c->Fp[b] += L;
      c->pend[b] = L;
      c->N[b] -= L;
    }
    if (any) {
      c->step += 1;
      ++steps_done;
      last_L = 1;
      for (int b = 0; b < B; ++b) last_L = std::max(last_L, c->pend[b]);
    }
    return LSP_OK;
  };
  int rc = LSP_OK;
  for (;;) {
    // before sizing step `launched`, the host must know N of step launched - 1, i.e. have read step launched - 2
    while (read < launched - 1) { rc = apply_results(read); if (rc) return rc; ++read; }
    int remaining = 0, most = 0;
    for (int b = 0; b < B; ++b) { remaining += c->N[b]; most = std::max(most, c->N[b]); }
    // host state is now that before step launched - 1 (or before step 0).  Near the end, or when that step may have
    // finished every sequence, read it too.
    if (launched > read && (most <= c->lag_tail || remaining == 0)) { rc = apply_results(read); if (rc) return rc; ++read; }
    remaining = 0;
    for (int b = 0; b < B; ++b) remaining += c->N[b];
    if (remaining == 0) break;
    const bool exact = (read == launched);           // the host state is that of the step about to be launched
    PassDims pd;
    if (exact) {
      pd = host_descriptor(c);
      // the device descriptor of this step: the first one is uploaded; later ones were derived on the device (k_advance)
      // from the same block lengths and are equal to the host's
      if (launched == 0) CU(cudaMemcpyAsync(c->d_desc, c->h_desc, 6 * (size_t)s * 4, cudaMemcpyHostToDevice, c->stream));
    } else {
      // host state is that before step launched - 1: this step's rows of sequence b are N there (if it goes on at all)
      for (int b = 0; b < B; ++b) {
        const int rows = c->N[b] >= 2 ? c->N[b] : 0;
        pd.M += rows;
        pd.Mh += rows > 0 ? rows - 1 : 0;
        pd.maxQ = std::max(pd.maxQ, rows);
        if (rows > 0) {
          pd.max_keys = std::max(pd.max_keys, total[b]);
          pd.attn_bytes += (2.0 * total[b] * kvd + 2.0 * rows * qd) * c->esz;
          pd.attn_flops += 4.0 * rows * (double)total[b] * qd;
        }
      }
      if (pd.M == 0) {            // every unfinished sequence has one masked position left: the step in flight ends them
        rc = apply_results(read); if (rc) return rc; ++read;
        continue;
      }
    }
    const int par = launched & 1, slot = launched % R;
    const StepDesc sd = desc_of(c, par);
    CU(cudaEventRecord(c->ring_t0[slot], c->stream));
    rc = enqueue_pass<T>(c, sd, B, pd, c->h_ring + (size_t)slot * slot_ints);
    if (rc) return rc;
    CU(cudaEventRecord(c->ring_t1[slot], c->stream));
    CU(cudaEventRecord(c->ring_done[slot], c->stream));
    // commit with the scan's own block lengths, then the next step's descriptor
    StepDesc sc = sd;
    sc.Lc = c->d_scan + mb;
    int max_pend = 0;
    if (exact) { for (int b = 0; b < B; ++b) if (c->N[b] > 0) max_pend = std::max(max_pend, c->pend[b]); }
    else max_pend = std::min(pd.maxQ, std::max(8, 2 * last_L));
    rc = enqueue_commit(c, sc, B, max_pend, 0);
    if (rc) return rc;
    launch_k(c->pdl, k_advance, dim3(1), dim3(32), 0, c->stream, sd, c->d_desc + (size_t)(par ^ 1) * 7 * s, s,
             (const int32_t*)(c->d_scan + mb), B);
    CU(cudaGetLastError());
    count_launch(c, CLS_COMMIT);
    c->last_M = pd.M;
    c->score_rows = pd.Mh;
    ++launched;
  }
  while (read < launched) { rc = apply_results(read); if (rc) return rc; ++read; }
  CU(cudaStreamSynchronize(c->stream));
  c->proposed = false;
  if (n_steps) *n_steps = steps_done;
  return LSP_OK;
}

}  // namespace

extern "C" {

int lsp_commit(lsp_ctx* c, const int32_t* L_override) {
  if (!c) return LSP_ERR_ARG;
  if (!c->proposed) return fail(c, LSP_ERR_STATE, "lsp_commit without a preceding lsp_denoise_step");
  const int B = c->batch, s = c->max_batch + 1;
  std::vector<int> L(B, 0);
  int max_pend = 0;
  for (int b = 0; b < B; ++b) {
    if (c->N[b] == 0) continue;
    L[b] = L_override ? L_override[b] : c->Lprop[b];
    if (L[b] < 1 || L[b] > c->N[b])
      return fail(c, LSP_ERR_STATE, "lsp_commit: L[%d] = %d outside [1, %d]", b, L[b], c->N[b]);
    if (c->pend[b] > max_pend) max_pend = c->pend[b];
  }
  int* hl = c->h_desc + 6 * s;
  for (int b = 0; b < B; ++b) hl[b] = L[b];
  CU(cudaMemcpyAsync(c->d_desc + 6 * s, hl, (size_t)B * 4, cudaMemcpyHostToDevice, c->stream));
  const lsp_model_cfg& m = c->m;
  const size_t kvd = (size_t)m.n_kv_heads * m.head_dim;
  const bool scattered = c->s.topology == 1;
  int max_n = 0;
  for (int b = 0; b < B; ++b) if (c->N[b] > max_n) max_n = c->N[b];
  const int rc = enqueue_commit(c, desc_of(c), B, max_pend, max_n);
  if (rc) return rc;
  for (int b = 0; b < B; ++b)
    if (c->N[b] > 0 && !c->kv_inplace) c->counters[CNT_APPEND_BYTES] += 2.0 * c->pend[b] * kvd * c->esz * 2.0 * m.n_layers;
  for (int b = 0; b < B; ++b) {
    if (c->N[b] == 0) continue;
    c->F[b] += c->pend[b];
    c->counters[CNT_TOKENS] += L[b];
    c->Fp[b] += L[b];
    c->pend[b] = scattered ? 0 : L[b];       // scattered: nothing becomes pending, the region is recomputed every pass
    c->N[b] -= L[b];
  }
  c->proposed = false;
  c->step += 1;
  return LSP_OK;
}

int lsp_generate(lsp_ctx* c, lsp_step_rec* recs, int max_recs, int* n_steps) {
  if (!c) return LSP_ERR_ARG;
  if (!c->tokens) return fail(c, LSP_ERR_STATE, "lsp_generate before lsp_begin");
  if (c->lagged && c->s.topology == 0 && !c->timing && !c->proposed)
    return c->m.dtype == 0 ? generate_lagged<float>(c, recs, max_recs, n_steps) : generate_lagged<bf16>(c, recs, max_recs, n_steps);
  int steps = 0, used = 0;
  std::vector<lsp_step_rec> tmp(c->batch);
  for (;;) {
    bool any = false;
    for (int b = 0; b < c->batch; ++b) any |= c->N[b] > 0;
    if (!any) break;
    int rc = lsp_denoise_step(c, tmp.data());
    if (rc) return rc;
    for (int b = 0; b < c->batch && recs && used < max_recs; ++b) recs[used++] = tmp[b];
    rc = lsp_commit(c, nullptr);
    if (rc) return rc;
    ++steps;
  }
  CU(cudaStreamSynchronize(c->stream));
  if (n_steps) *n_steps = steps;
  return LSP_OK;
}

int lsp_generate_host(lsp_ctx* c, int32_t* tokens, int token_stride, const int32_t* tokens_in, int32_t* tokens_out,
                      const int32_t* prompt_len, const int32_t* gen_len, int batch, lsp_step_rec* recs, int max_recs,
                      int* n_steps) {
  if (!c || !tokens || !tokens_in || !tokens_out || !prompt_len || !gen_len) return LSP_ERR_ARG;
  if (batch < 1 || batch > c->max_batch || token_stride < 2)
    return fail(c, LSP_ERR_ARG, "lsp_generate_host: batch %d not in [1, %d] or bad stride", batch, c->max_batch);
  const size_t bytes = (size_t)batch * token_stride * sizeof(int32_t);
  CU(cudaMemcpyAsync(tokens, tokens_in, bytes, cudaMemcpyHostToDevice, c->stream));
  int rc = lsp_begin(c, tokens, token_stride, prompt_len, gen_len, batch);
  if (rc) return rc;
  rc = lsp_generate(c, recs, max_recs, n_steps);
  if (rc) return rc;
  CU(cudaMemcpyAsync(tokens_out, tokens, bytes, cudaMemcpyDeviceToHost, c->stream));
  CU(cudaStreamSynchronize(c->stream));
  return LSP_OK;
}

int lsp_active(lsp_ctx* c, int32_t* n_active, int* n_unfinished) {
  if (!c) return LSP_ERR_ARG;
  int u = 0;
  for (int b = 0; b < c->batch; ++b) {
    if (n_active) n_active[b] = c->N[b];
    u += c->N[b] > 0;
  }
  if (n_unfinished) *n_unfinished = u;
  return LSP_OK;
}

int lsp_score_rows(lsp_ctx* c) { return c ? c->score_rows : LSP_ERR_ARG; }

int lsp_get_scores(lsp_ctx* c, int32_t* yhat, float* pmax, float* margin) {
  if (!c) return LSP_ERR_ARG;
  const size_t n = (size_t)c->score_rows * 4;
  if (n == 0) return LSP_OK;
  if (yhat) CU(cudaMemcpyAsync(yhat, c->yhat, n, cudaMemcpyDeviceToHost, c->stream));
  if (pmax) CU(cudaMemcpyAsync(pmax, c->pmax, n, cudaMemcpyDeviceToHost, c->stream));
  if (margin) CU(cudaMemcpyAsync(margin, c->margin, n, cudaMemcpyDeviceToHost, c->stream));
  CU(cudaStreamSynchronize(c->stream));
  return LSP_OK;
}

int lsp_head_scan(lsp_ctx* c, const void* hidden, const int32_t* seq_offsets, int batch, int32_t* l_run,
                  int32_t* l_commit, uint32_t* flags, float* tau_used) {
  if (!c || !hidden) return LSP_ERR_ARG;
  int rows = 0;
  int rc = upload_offsets(c, seq_offsets, batch, &rows);
  if (rc) return rc;
  c->proposed = false;
  int n_tiles = 0;
  rc = c->m.dtype == 0 ? run_head<float>(c, (const float*)hidden, rows, &n_tiles)
                       : run_head<bf16>(c, (const bf16*)hidden, rows, &n_tiles);
  if (rc) return rc;
  seg_begin(c, CLS_SCAN);
  rc = run_merge_scan(c, rows, n_tiles, c->d_desc + 4 * (c->max_batch + 1), batch, false);
  seg_end(c);
  count_launch(c, CLS_SCAN, 2);
  c->counters[CNT_STEPS] += 1;
  if (rc) return rc;
  c->score_rows = rows;
  return scan_outputs(c, batch, l_run, l_commit, flags, tau_used);
}

int lsp_scan(lsp_ctx* c, const float* score, const int32_t* yhat, const float* margin, const int32_t* seq_offsets,
             int batch, int32_t* l_run, int32_t* l_commit, uint32_t* flags, float* tau_used) {
  if (!c || !score || !yhat) return LSP_ERR_ARG;
  int rows = 0;
  int rc = upload_offsets(c, seq_offsets, batch, &rows);
  if (rc) return rc;
  c->proposed = false;
  int* o = c->d_scan;
  const int mb = c->max_batch;
  launch_k(c->pdl, k_lsp_scan, dim3(batch), dim3(32), 0, c->stream, score, yhat, margin, c->d_desc + 4 * (c->max_batch + 1), scan_params(c), o,
                                          o + mb, (uint32_t*)(o + 2 * mb), (float*)(o + 3 * mb));
  CU(cudaGetLastError());
  CU(cudaMemcpyAsync(c->h_scan, c->d_scan, 4 * (size_t)mb * 4, cudaMemcpyDeviceToHost, c->stream));
  CU(cudaMemcpyAsync(c->h_status, c->d_status, 16, cudaMemcpyDeviceToHost, c->stream));
  return scan_outputs(c, batch, l_run, l_commit, flags, tau_used);
}

int lsp_op_linear(lsp_ctx* c, int op, const void* A, const void* W, const void* W2, void* out, int M, int N, int K) {
  if (!c || !A || !W || !out || M < 0 || N < 1 || K < 1) return LSP_ERR_ARG;
  if (op < 0 || op > 2 || (op == 2 && !W2)) return fail(c, LSP_ERR_ARG, "lsp_op_linear: bad op");
  if (K % 64 || N % 16) return fail(c, LSP_ERR_SHAPE, "lsp_op_linear: K must be a multiple of 64 and N of 16");
  int rc = 0;
  for (int r = 0; r < c->op_repeat && rc == 0; ++r) {
    const size_t off = (size_t)(r % c->op_rotate) * N * K * c->esz;
    const void* w = (const char*)W + off;
    const void* w2 = W2 ? (const char*)W2 + off : nullptr;
    rc = c->m.dtype == 0 ? op_linear_impl<float>(c, op, A, w, w2, out, M, N, K)
                         : op_linear_impl<bf16>(c, op, A, w, w2, out, M, N, K);
  }
  if (rc) return rc;
  if (c->async_ops) return LSP_OK;
  CU(cudaMemcpyAsync(c->h_status, c->d_status, 16, cudaMemcpyDeviceToHost, c->stream));
  CU(cudaStreamSynchronize(c->stream));
  return check_status(c);
}

int lsp_op_attention(lsp_ctx* c, int layer, const void* q, const void* k_new, const void* v_new, void* out,
                     const int32_t* cache_len, const int32_t* rows, int batch) {
  if (!c || !q || !k_new || !v_new || !out || !cache_len || !rows) return LSP_ERR_ARG;
  if (layer < 0 || layer >= c->m.n_layers || batch < 1 || batch > c->max_batch)
    return fail(c, LSP_ERR_ARG, "lsp_op_attention: layer %d or batch %d out of range", layer, batch);
  const int s = c->max_batch + 1;
  int* h = c->h_desc;
  int M = 0, maxQ = 0, max_keys = 0;
  for (int b = 0; b < batch; ++b) {
    if (cache_len[b] < 0 || rows[b] < 0 || cache_len[b] + rows[b] > c->max_len)
      return fail(c, LSP_ERR_ARG, "lsp_op_attention: sequence %d has %d cached + %d new positions, more than max_len %d", b,
                  cache_len[b], rows[b], c->max_len);
    h[0 * s + b] = cache_len[b];
    h[3 * s + b] = M;
    M += rows[b];
    maxQ = std::max(maxQ, rows[b]);
    if (rows[b] > 0) max_keys = std::max(max_keys, cache_len[b] + rows[b]);
  }
  h[3 * s + batch] = M;
  c->proposed = false;                 // the descriptor of a pending lsp_denoise_step is overwritten
  if (M == 0) return LSP_OK;
  CU(cudaMemcpyAsync(c->d_desc, h, (size_t)s * 4, cudaMemcpyHostToDevice, c->stream));
  CU(cudaMemcpyAsync(c->d_desc + 3 * s, h + 3 * s, (size_t)s * 4, cudaMemcpyHostToDevice, c->stream));
  const size_t kvd = (size_t)c->m.n_kv_heads * c->m.head_dim;
  const size_t plane = (size_t)c->max_rows * kvd * c->esz;
  char* stK = c->stage + (size_t)(2 * layer) * plane;
  CU(cudaMemcpyAsync(stK, k_new, (size_t)M * kvd * c->esz, cudaMemcpyDeviceToDevice, c->stream));
  CU(cudaMemcpyAsync(stK + plane, v_new, (size_t)M * kvd * c->esz, cudaMemcpyDeviceToDevice, c->stream));
  const int rc = c->m.dtype == 0 ? run_attention<float>(c, layer, (const float*)q, (float*)out, desc_of(c), batch, maxQ, max_keys, 0)
                                 : run_attention<bf16>(c, layer, (const bf16*)q, (bf16*)out, desc_of(c), batch, maxQ, max_keys, 0);
  if (rc) return rc;
  CU(cudaMemcpyAsync(c->h_status, c->d_status, 16, cudaMemcpyDeviceToHost, c->stream));
  CU(cudaStreamSynchronize(c->stream));
  return check_status(c);
}

int lsp_debug_wait_selftest(lsp_ctx* c, int limit_us) {
  if (!c) return LSP_ERR_ARG;
#ifndef LSP_NO_UMMA
  if (limit_us < 1 || limit_us > 1000000) return fail(c, LSP_ERR_ARG, "lsp_debug_wait_selftest: limit outside [1 us, 1 s]");
  k_wait_selftest<<<1, 32, 0, c->stream>>>(c->d_status, (unsigned long long)limit_us * 1000ull);
  CU(cudaGetLastError());
  CU(cudaMemcpyAsync(c->h_status, c->d_status, 16, cudaMemcpyDeviceToHost, c->stream));
  CU(cudaStreamSynchronize(c->stream));
  return check_status(c);
#else
  return fail(c, LSP_ERR_SHAPE, "built without the tcgen05 kernels");
#endif
}

int lsp_last_timing(lsp_ctx* c, float* ms) {
  if (!c || !ms) return LSP_ERR_ARG;
  CU(cudaStreamSynchronize(c->stream));
  seg_collect(c);
  memcpy(ms, c->timing_ms, sizeof c->timing_ms);
  return LSP_OK;
}

int lsp_get_counters(lsp_ctx* c, double* out) {
  if (!c || !out) return LSP_ERR_ARG;
  c->counters[16] = c->last_attn_kernel;
  c->counters[17] = c->last_attn_cluster;
  memcpy(out, c->counters, sizeof c->counters);
  return LSP_OK;
}

int lsp_reset_counters(lsp_ctx* c) {
  if (!c) return LSP_ERR_ARG;
  cudaStreamSynchronize(c->stream);
  seg_collect(c);
  memset(c->counters, 0, sizeof c->counters);
  memset(c->timing_ms, 0, sizeof c->timing_ms);
  return LSP_OK;
}

// ---- lsp_linear_static: the streaming GEMM with its scratch in a static device array ----------------------------
namespace {

constexpr int kStaticMaxCtas = 64;        // CTAs the static variant launches at most
constexpr int kStaticBN = 128;            // its tile width
constexpr int kStaticMaxTiles = 4096;     // tile counters
constexpr size_t kStaticPartialBytes = (size_t)kStaticMaxCtas * 2 * UM_BM * kStaticBN * sizeof(float);   // 8 MiB
constexpr size_t kStaticScratchBytes = kStaticPartialBytes + (size_t)kStaticMaxTiles * sizeof(unsigned) + 256;

// Partial tiles, then the tile counters, then the status word.  One copy per GPU that loads the library, held until
// the process exits.  In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kStaticMaxDevices = 64;
struct StaticDev {
  std::once_flag once;
  cudaError_t setup_rc = cudaErrorUnknown;
  unsigned char* scratch = nullptr;      // device address of g_static_scratch on this device
  PFN_encodeTiled encode = nullptr;
  int max_smem = 0, n_sm = 0;
};
StaticDev g_static_dev[kStaticMaxDevices];

void static_msg(char* err, size_t err_len, const char* fmt, ...) {
  if (!err || err_len == 0) return;
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(err, err_len, fmt, ap);
  va_end(ap);
}

bool static_map(PFN_encodeTiled encode, CUtensorMap* m, const void* base, int rows, int K, int box_rows) {
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {(cuuint32_t)UM_BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

int lsp_linear_static(const void* A, const void* W, void* out, int M, int N, int K, void* cuda_stream, char* err,
                      size_t err_len) {
  if (err && err_len) err[0] = 0;
  if (!A || !W || !out) { static_msg(err, err_len, "lsp_linear_static: NULL pointer"); return LSP_ERR_ARG; }
  if (M < 1 || M > UM_BM || N < 16 || N % 16 || K < 64 || K % 64 || (N + kStaticBN - 1) / kStaticBN > kStaticMaxTiles) {
    static_msg(err, err_len,
               "lsp_linear_static: M = %d, N = %d, K = %d outside the static scratch's limits (1 <= M <= %d, N a multiple "
               "of 16 up to %d, K a multiple of 64)", M, N, K, UM_BM, kStaticMaxTiles * kStaticBN);
    return LSP_ERR_SHAPE;
  }
  if (((uintptr_t)A | (uintptr_t)W | (uintptr_t)out) & 15) {
    static_msg(err, err_len, "lsp_linear_static: pointers must be 16-byte aligned");
    return LSP_ERR_ARG;
  }
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kStaticMaxDevices) {
    static_msg(err, err_len, "lsp_linear_static: no usable current device (%s)", cudaGetErrorString(e));
    return LSP_ERR_CUDA;
  }
  StaticDev& sd = g_static_dev[dev];
  // First call on this device (with that device current): resolve the device address of the static array.
  std::call_once(sd.once, [&sd, dev]() {
    void* p = nullptr;
    cudaError_t rc = cudaGetSymbolAddress(&p, g_static_scratch);
    if (rc == cudaSuccess) {
      sd.scratch = (unsigned char*)p;
      void* fn = nullptr;
      cudaDriverEntryPointQueryResult q;
      rc = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
      if (rc == cudaSuccess && (fn == nullptr || q != cudaDriverEntryPointSuccess)) rc = cudaErrorNotSupported;
      sd.encode = (PFN_encodeTiled)fn;
    }
    if (rc == cudaSuccess) rc = cudaDeviceGetAttribute(&sd.max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (rc == cudaSuccess) rc = cudaDeviceGetAttribute(&sd.n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (rc == cudaSuccess)
      rc = cudaFuncSetAttribute(k_gemm_stream<kStaticBN, 1, 2, EpiStore<bf16>>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                sd.max_smem);
    sd.setup_rc = rc;
  });
  if (sd.setup_rc != cudaSuccess) {
    static_msg(err, err_len, "lsp_linear_static: set-up on device %d failed (%s)", dev, cudaGetErrorString(sd.setup_rc));
    return LSP_ERR_CUDA;
  }
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  // stage shape: as many two-atom stages as fit, else one-atom stages
  const int a_rows = (M + 7) / 8 * 8;
  const int aux = 1024 + UM_BM * 128 + 8 * (2 * ST_MAX_STAGES + 4) + 16;
  const int atom = a_rows * 128 + kStaticBN * 128;
  const int atoms = (K % 128 == 0 && (sd.max_smem - aux) / (2 * atom) >= 3) ? 2 : 1;
  int stages = (sd.max_smem - aux) / (atoms * atom);
  if (stages > ST_MAX_STAGES) stages = ST_MAX_STAGES;
  const size_t smem = (size_t)stages * atoms * atom + aux;
  CUtensorMap ma, mb;
  if (stages < 2 || !static_map(sd.encode, &ma, A, M, K, a_rows) || !static_map(sd.encode, &mb, W, N, K, kStaticBN / 2)) {
    static_msg(err, err_len, "lsp_linear_static: could not describe the operands to the copy engine");
    return LSP_ERR_CUDA;
  }
  const int n_tiles = (N + kStaticBN - 1) / kStaticBN;
  const int kc = K / (atoms * UM_BK);
  const long U = (long)n_tiles * kc;
  const int max_ctas = sd.n_sm < kStaticMaxCtas ? sd.n_sm : kStaticMaxCtas;
  int grid = n_tiles <= max_ctas ? n_tiles * (max_ctas / n_tiles) : max_ctas;
  if (grid > U) grid = (int)U;
  float* partials = (float*)sd.scratch;
  unsigned* counters = (unsigned*)(sd.scratch + kStaticPartialBytes);
  unsigned* status = counters + kStaticMaxTiles;
  // the array keeps whatever the last call left: the counters (and the status word) must start at zero
  e = cudaMemsetAsync(counters, 0, (size_t)kStaticMaxTiles * sizeof(unsigned) + 16, stream);
  if (e != cudaSuccess) {
    static_msg(err, err_len, "lsp_linear_static: clearing the counters failed (%s)", cudaGetErrorString(e));
    return LSP_ERR_CUDA;
  }
  StreamArgs args{M, N, n_tiles, 1, 0, 0, 1, kc, a_rows, atoms, kStaticBN / 2, stages, 0, partials, counters, status};
  EpiStore<bf16> epi{(bf16*)out, N};
  k_gemm_stream<kStaticBN, 1, 2, EpiStore<bf16>><<<grid, ST_THREADS, smem, stream>>>(ma, mb, mb, args, epi);
  e = cudaGetLastError();
  if (e != cudaSuccess) {
    static_msg(err, err_len, "lsp_linear_static: launch failed (%s)", cudaGetErrorString(e));
    return LSP_ERR_CUDA;
  }
  return LSP_OK;
}

const char* lsp_last_error(const lsp_ctx* c) { return c ? c->err.c_str() : "null context"; }

int lsp_destroy(lsp_ctx* c) {
  if (!c) return LSP_ERR_ARG;
  if (c->h_desc) cudaFreeHost(c->h_desc);
  if (c->h_scan) cudaFreeHost(c->h_scan);
  if (c->h_status) cudaFreeHost(c->h_status);
  if (c->h_ring) cudaFreeHost(c->h_ring);
  for (int i = 0; i < lsp_ctx::kRing; ++i) {
    if (c->ring_done[i]) cudaEventDestroy(c->ring_done[i]);
    if (c->ring_t0[i]) cudaEventDestroy(c->ring_t0[i]);
    if (c->ring_t1[i]) cudaEventDestroy(c->ring_t1[i]);
  }
  if (c->ev0) cudaEventDestroy(c->ev0);
  if (c->ev1) cudaEventDestroy(c->ev1);
  for (cudaEvent_t e : c->seg_ev) cudaEventDestroy(e);
  delete c;
  return LSP_OK;
}

}  // extern "C"
