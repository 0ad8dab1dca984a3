/*
 * lsp.h -- C ABI of the B200 (sm_100a) Longest-Stable-Prefix decode library.
 *
 * The library runs the per-step hot path of the LSP scheduler for diffusion language models:
 * one bidirectional denoiser pass over [pending block | masked suffix] with the committed prefix
 * served from a contiguous KV cache (Algorithm 1, the forward pass), the fused LM-head + confidence
 * reduction (Eq. 1 and the softmax max-probability), the longest-stable-run scan with
 * adaptive threshold (Eq. 2), delimiter snap and fallback (Sec. 3.2), and the atomic commit with
 * the contiguous KV append (Algorithm 1, commit and AppendToCache).
 *
 * Conventions
 *  - Every function returns 0 on success or a negative LSP_ERR_* code; lsp_last_error() gives text.
 *  - "device" pointers are CUDA global memory of the current device; "host" pointers are ordinary
 *    host memory.  The library never allocates device memory: weights, KV cache, workspace, token
 *    buffer and the stream belong to the caller and are borrowed until lsp_destroy().
 *  - Work is enqueued on the stream given to lsp_init().  A call that returns host-visible results
 *    synchronises that stream (only); the others return as soon as the work is enqueued.
 *  - Element type T is float (dtype 0) or bfloat16 (dtype 1).  bf16 GEMMs run on tcgen05 tensor
 *    cores with fp32 accumulation; fp32 models run on CUDA cores.
 *  - All linear weights are row-major [out_features, in_features] (K-major operands).
 */
#ifndef LSP_H_
#define LSP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LSP_OK 0
#define LSP_ERR_ARG (-1)            /* NULL pointer, negative size, bad enum value */
#define LSP_ERR_SHAPE (-2)          /* model shape not supported (see lsp_init) */
#define LSP_ERR_WORKSPACE (-3)      /* workspace smaller than lsp_workspace_bytes() */
#define LSP_ERR_STATE (-4)          /* call out of order, L out of range, decode already finished */
#define LSP_ERR_CUDA (-5)           /* a CUDA runtime/driver call failed */
#define LSP_ERR_DEVICE_TIMEOUT (-6) /* a bounded device-side wait expired; results of the step are invalid */

/* flags in lsp_step_rec.flags */
#define LSP_FLAG_SNAPPED 1u
#define LSP_FLAG_FALLBACK 2u
#define LSP_FLAG_RANGE_UNACHIEVABLE 4u
#define LSP_FLAG_RUN_TO_END 8u
#define LSP_FLAG_NEAR_THRESHOLD 16u
#define LSP_FLAG_NEAR_TIE 32u

typedef struct lsp_ctx lsp_ctx;

/* Transformer shape (the paper treats p_theta as a black box; the shape is the benchmark's):
 * pre-norm blocks, RMSNorm, rotary positions with rotate-half pairing (i, i + head_dim/2),
 * non-causal attention (n_heads query heads, n_kv_heads key/value heads), SwiGLU FFN, no biases,
 * untied head.  Requirements: head_dim in {64, 128}; d_model, d_ffn, n_heads*head_dim multiples
 * of 64; n_heads % n_kv_heads == 0. */
typedef struct {
  int n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
  float rms_eps, rope_theta;
  int dtype;   /* 0 = fp32, 1 = bf16 */
  int mask_id; /* id of the [MASK] token */
} lsp_model_cfg;

/* Scheduler policy (Sec. 3.2; Algorithm 1 inputs). */
typedef struct {
  int score;       /* 0 = softmax max-probability, 1 = logit margin delta_i (Eq. 1) */
  int mode;        /* 0 = fixed threshold tau, 1 = adaptive tau with L' in [alpha N, beta N] (Eq. 2),
                      2 = commit exactly fixed_k tokens per step (ablation policy, no snapping) */
  float tau, alpha, beta;
  int l_min;       /* L_min >= 1 */
  int snap_window; /* W >= 0; negative = unbounded look-back */
  int fixed_k;
  const uint8_t* delim_bitmap; /* device, (vocab+7)/8 bytes, bit (v & 7) of byte v >> 3; NULL = empty set D */
  int exclude_mask_logit;      /* 1: the mask_id column takes no part in argmax / margin / probability */
  float flag_tol;              /* NEAR_THRESHOLD flag: |score_i - tau| <= flag_tol for some i <= L'+1; 0 disables */
  float tie_tol;               /* NEAR_TIE flag: delta_i <= tie_tol for some committed i; 0 disables */
  int topology;                /* 0 = prefix: commit the left-aligned block yhat_{1:L} (the LSP scheduler);
                                  1 = scattered acceptance, the baseline the paper compares with (Sec. 4): every pass
                                  covers the whole generation region and the L most confident masked positions are
                                  accepted wherever they are (ties: lower position).  L comes from the same policy:
                                  mode 2 gives top-k with k = fixed_k, modes 0/1 give the "Scattered-Margin" ablation
                                  (LSP's block sizing, scattered topology).  Only the prompt's K/V are cached. */
} lsp_sched_cfg;

/* Device pointers to the weights, all element type T.  Per-layer arrays are HOST arrays of
 * n_layers device pointers.  w_qkv rows: n_heads*head_dim query rows, then n_kv_heads*head_dim key
 * rows, then n_kv_heads*head_dim value rows. */
typedef struct {
  const void* embed;       /* [vocab, d_model] */
  const void* final_norm;  /* [d_model] */
  const void* w_head;      /* [vocab, d_model] */
  const void* const* attn_norm; /* [d_model] */
  const void* const* w_qkv;     /* [(n_heads + 2 n_kv_heads) head_dim, d_model] */
  const void* const* w_o;       /* [d_model, n_heads head_dim] */
  const void* const* ffn_norm;  /* [d_model] */
  const void* const* w_gate;    /* [d_ffn, d_model] */
  const void* const* w_up;      /* [d_ffn, d_model] */
  const void* const* w_down;    /* [d_model, d_ffn] */
} lsp_weights;

/* One record per sequence and step. */
typedef struct {
  int step;      /* step index k */
  int n_before;  /* N_k, active positions before the commit */
  int rows;      /* query rows this sequence contributed to the pass (pending block + N_k) */
  int l_run;     /* L' */
  int l_commit;  /* L */
  float tau_used;
  unsigned flags;
  float ms;      /* device time of the whole step (same value for every sequence of the batch) */
  int flips;     /* masked positions whose argmax differs from the previous step's (the paper's token flips, Fig. 3) */
  int flip_base; /* masked positions that were also scored by the previous step (denominator of the flip rate) */
} lsp_step_rec;

/* Bytes of workspace lsp_init() needs for up to max_batch sequences of up to max_len positions
 * (prompt + generation).  Includes the staging buffer that holds one pass's K/V for all layers. */
size_t lsp_workspace_bytes(const lsp_model_cfg* model, int max_batch, int max_len);

/* Bytes of the contiguous prefix KV cache: [n_layers][2][max_batch][max_len][n_kv_heads*head_dim] T. */
size_t lsp_kv_cache_bytes(const lsp_model_cfg* model, int max_batch, int max_len);

/* Creates a context.  kv_cache and workspace are device buffers of at least the sizes above, 256-byte
 * aligned; neither needs initialising (no result ever depends on memory the library has not written);
 * cuda_stream is a cudaStream_t (NULL = default stream).  The call builds the rotary table on the
 * device; it does not allocate device memory. */
int lsp_init(lsp_ctx** out, const lsp_model_cfg* model, const lsp_sched_cfg* sched, const lsp_weights* weights,
             void* kv_cache, void* workspace, size_t workspace_bytes, int max_batch, int max_len,
             void* cuda_stream);

/* Replaces the scheduler policy (allowed between steps). */
int lsp_set_sched(lsp_ctx* ctx, const lsp_sched_cfg* sched);

/* Implementation switches: key 0 = GEMM implementation for bf16 models (0 = CUDA-core reference kernels, 1 = tcgen05,
 * default 1); key 1 = attention implementation for bf16 models (0 = CUDA-core, 1 = mma.sync tensor cores, 2 = default:
 * tcgen05 tensor cores for head_dim 128, else as 1); key 2 = per-class CUDA-event timing (0 off, 1 on; see
 * lsp_last_timing); key 3 = K/V layout of a pass: 0 (default, the contract) = the pass writes its keys / values to
 * staging planes and lsp_commit appends the pending block's rows to the cache as one contiguous copy per layer
 * (Algorithm 1, AppendToCache); 1 = in place: the pass writes every row's K/V at that row's absolute position in the
 * cache buffer, behind the committed prefix, so the append is only the length bump (rows [F, F + rows) of a sequence
 * then hold provisional values between steps; rows [0, F) are final and never rewritten in either layout).  The layout
 * cannot change in the middle of a decode (LSP_ERR_STATE); key 4 = where lsp_generate keeps the block lengths: 0
 * (default) = it reads L back after every pass before it enqueues the next; 1 = device-resident: the scan's L feeds the
 * commit kernel directly, the next pass's descriptor is derived from it on the device, and the host enqueues pass k+1
 * while pass k runs, reading L one step late (it sizes launches from row counts it knows a step late, upper bounds for
 * the LM-head rows; rows beyond the real ones are inert).  The decode is the same: identical tokens, boundaries and
 * records on fp32 models; on bf16 models up to the last bits of a score (the LM-head launch has more rows, which can
 * move a tile boundary of its reduction), i.e. up to decisions within rounding distance of a threshold or tie.  Prefix
 * topology only, and only while per-class timing is off (otherwise the synchronous loop runs).  Any other key:
 * LSP_ERR_ARG. */
int lsp_set_option(lsp_ctx* ctx, int key, int value);

/* Algorithm 1, state initialisation: X_F <- prompt, X_A <- masks, K <- empty.  tokens: device int32
 * [batch, token_stride], caller-owned, prompt ids already at [0, prompt_len[b]); the library writes
 * mask_id over [prompt_len[b], prompt_len[b]+gen_len[b]) and later the committed ids.  prompt_len,
 * gen_len: host [batch].  prompt_len[b] >= 1, gen_len[b] >= 1, sum <= max_len, <= token_stride. */
int lsp_begin(lsp_ctx* ctx, int32_t* tokens, int token_stride, const int32_t* prompt_len,
              const int32_t* gen_len, int batch);

/* Algorithm 1, forward pass through fallback, for every unfinished sequence: the pass, the scores, the scan; proposes L
 * and changes no committed state.  rec: host [batch] or NULL.  Synchronises the stream. */
int lsp_denoise_step(lsp_ctx* ctx, lsp_step_rec* rec);

/* (Scattered topology: writes the L most confident predictions at their own positions instead, and appends only the
 * prompt's K/V after the first pass.)
 * Algorithm 1, commit and AppendToCache: writes yhat_{1:L} into the token buffer, appends the pending block's K/V
 * (computed by the last pass) to the cache as one contiguous copy per layer, and makes the new
 * block pending.  L_override: host [batch] (entries of finished sequences ignored) or NULL to use the
 * proposed lengths.  Needs a preceding lsp_denoise_step; 1 <= L <= N_b else LSP_ERR_STATE and nothing
 * changes.  Asynchronous. */
int lsp_commit(lsp_ctx* ctx, const int32_t* L_override);

/* Algorithm 1, the whole loop: step + commit until every sequence is fully committed.  recs: host
 * [max_recs] records in (step, sequence) order, or NULL; n_steps: number of denoiser passes. */
int lsp_generate(lsp_ctx* ctx, lsp_step_rec* recs, int max_recs, int* n_steps);

/* Algorithm 1 from host memory: copies tokens_in (host int32 [batch, token_stride], prompt ids at
 * [0, prompt_len[b]) of every row; pinned or pageable) into the caller's device buffer tokens (device int32
 * [batch, token_stride], scratch the caller owns), runs lsp_begin + lsp_generate, and copies the finished
 * buffer (prompt followed by the committed ids) to tokens_out (host, same shape; may equal tokens_in).
 * Both copies run on the context's stream; the call returns after the result has arrived.  Errors as
 * lsp_begin / lsp_generate; on error tokens_out is not written. */
int lsp_generate_host(lsp_ctx* ctx, int32_t* tokens, int token_stride, const int32_t* tokens_in,
                      int32_t* tokens_out, const int32_t* prompt_len, const int32_t* gen_len, int batch,
                      lsp_step_rec* recs, int max_recs, int* n_steps);

/* Number of still-active positions per sequence (host [batch]); returns the count of unfinished sequences
 * through *n_unfinished. */
int lsp_active(lsp_ctx* ctx, int32_t* n_active, int* n_unfinished);

/* Per-position outputs of the last step / last lsp_head_scan, copied to host arrays of
 * lsp_score_rows() entries (sequence-major, active positions in order).  Any pointer may be NULL. */
int lsp_score_rows(lsp_ctx* ctx);
int lsp_get_scores(lsp_ctx* ctx, int32_t* yhat, float* pmax, float* margin);

/* The fused LM-head + confidence reduction and the scan alone (Eq. 1, Eq. 2, snapping), on hidden
 * states the caller provides: hidden device [rows, d_model] T (used as given: no normalisation),
 * seq_offsets host [batch+1] ascending with seq_offsets[batch] = rows <= max_batch*max_len.
 * Outputs host [batch] each (may be NULL).  Full-vocabulary logits are never written to memory.
 * Synchronises the stream. */
int lsp_head_scan(lsp_ctx* ctx, const void* hidden, const int32_t* seq_offsets, int batch, int32_t* l_run,
                  int32_t* l_commit, uint32_t* flags, float* tau_used);

/* The scan alone on caller-provided device arrays score[rows] (fp32), yhat[rows]; margin may be NULL.
 * Same outputs as lsp_head_scan. */
int lsp_scan(lsp_ctx* ctx, const float* score, const int32_t* yhat, const float* margin,
             const int32_t* seq_offsets, int batch, int32_t* l_run, int32_t* l_commit, uint32_t* flags,
             float* tau_used);

/* Kernel-level entry points used for parity checks at full shapes (device pointers, element type T
 * of the context).  op: 0 = out[M,N] = A W^T; 1 = out[M,N] += A W^T (residual update);
 * 2 = out[M,N] = silu(A W^T) * (A W2^T) (SwiGLU product, Sec. "transformer shape").  W, W2: [N, K]. */
int lsp_op_linear(lsp_ctx* ctx, int op, const void* A, const void* W, const void* W2, void* out, int M,
                  int N, int K);

/* The suffix-over-prefix attention of one layer alone (Sec. 3.2, "bidirectional lookahead" over the frozen prefix and
 * the active suffix; the attention inside Algorithm 1's forward pass), for parity checks at full head shapes:
 *   out[r, h, :] = softmax_j(q[r, h, :] . k_j / sqrt(head_dim)) v_j    over j in cache[0, cache_len[b]) then the pass's
 * own rows of sequence b, no mask; query head h reads KV head h / (n_heads / n_kv_heads).
 *   q, out        device [rows_total, n_heads * head_dim] T, sequences packed back to back (rows_total = sum rows[b])
 *   k_new, v_new  device [rows_total, n_kv_heads * head_dim] T: this pass's keys / values (already rotated); they are
 *                 copied into the context's staging planes of `layer`
 *   cache_len, rows   host [batch]; the cached keys / values are read from the caller's kv_cache, layer `layer`,
 *                 sequence slot b, positions [0, cache_len[b]) (layout: lsp_kv_cache_bytes)
 * Takes the same kernel choice as lsp_denoise_step would for these sizes (lsp_get_counters 16, 17 tell which).
 * Must not be called between lsp_denoise_step and lsp_commit (it overwrites the step's descriptor: the pending
 * proposal is dropped).  Synchronises the stream; returns LSP_ERR_DEVICE_TIMEOUT like a step. */
int lsp_op_attention(lsp_ctx* ctx, int layer, const void* q, const void* k_new, const void* v_new, void* out,
                     const int32_t* cache_len, const int32_t* rows, int batch);

/* Device time (ms) accumulated since lsp_reset_counters() by kernel class, host float[8]:
 * 0 embed+norms, 1 layer GEMMs, 2 attention, 3 fused LM head, 4 merge+scan, 5 commit/append, 6 whole steps
 * (always filled), 7 host time spent queueing those steps' launches (always filled).  Classes 0-5 are only filled while option key 2 (per-class CUDA-event timing)
 * is 1.  Synchronises the stream. */
int lsp_last_timing(lsp_ctx* ctx, float* ms);

/* Host-side accounting since lsp_reset_counters(), host double[18]: 0 kernel launches, 1 layer-GEMM algorithmic
 * bytes (every operand and result once), 2 layer-GEMM flops, 3 attention bytes (every K/V row once per layer
 * plus Q and O), 4 KV-append bytes (read + write), 5 LM-head bytes, 6 LM-head flops, 7 denoiser passes,
 * 8..13 kernel launches by class (same classes as lsp_last_timing 0..5), 14 attention flops
 * (4 * queries * keys * n_heads * head_dim per layer), 15 committed tokens; not counters but the last attention
 * launch: 16 its kernel (0 CUDA cores, 1 mma.sync, 2 tcgen05), 17 the thread block cluster size its key tiles were
 * split over (1 = no split). */
int lsp_get_counters(lsp_ctx* ctx, double* out);
int lsp_reset_counters(lsp_ctx* ctx);

/* (No counterpart in the paper: a convenience for callers that cannot allocate.)
 * out[M, N] = A[M, K] W[N, K]^T in bfloat16 with fp32 accumulation, without a context and without any allocation:
 * the split-K partial tiles and tile counters that lsp_op_linear keeps in the caller's workspace live here in a
 * static array inside the library's device image (8 MiB + 16 KiB; every GPU that loads the library holds it until
 * the process exits).  It is meant for code that runs where cudaMalloc is off limits, such as a plug-in called inside
 * another framework's memory pool or from a real-time loop, and therefore cannot create the workspace lsp_init() needs.
 *   A, W, out  device pointers, 16-byte aligned, row-major, bfloat16; out is written completely.
 *   limits     1 <= M <= 128; N a multiple of 16, at most 524288; K a multiple of 64.  Anything else returns
 *              LSP_ERR_SHAPE (NULL or misaligned pointers: LSP_ERR_ARG) and writes a message into err.
 *   cuda_stream  a cudaStream_t (NULL = default stream); the call only enqueues work and returns.  It never reads
 *              anything back, so a device-side bounded wait that expires inside the kernel (2 s; a protocol fault,
 *              not a data-dependent event) is NOT reported by this entry point: `out` is then left partly written
 *              and the call has long since returned LSP_OK.  A caller that must know runs the same product once
 *              through lsp_op_linear, which synchronises and returns LSP_ERR_DEVICE_TIMEOUT.
 *   err, err_len  optional host buffer that receives a message when the call fails.
 * The first call on a device looks up the array's device address and sets a kernel attribute, once, with that
 * device current; make that first call outside any stream capture.  Every call uses the same array: it clears the
 * counters itself (so a call that was aborted leaves nothing behind), but two calls whose kernels overlap on the GPU,
 * from different streams or threads, race on it and give wrong results; calls on one stream are safe.  The call
 * itself performs no cudaMalloc/cudaFree and uses no allocating library routine. */
int lsp_linear_static(const void* A, const void* W, void* out, int M, int N, int K, void* cuda_stream, char* err,
                      size_t err_len);

const char* lsp_last_error(const lsp_ctx* ctx);
int lsp_destroy(lsp_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* LSP_H_ */
