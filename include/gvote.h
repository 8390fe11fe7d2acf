/*
 * gvote.h — C ABI of the GVote per-request KV-cache compression pass for NVIDIA B200 (sm_100a).
 *
 * The pass is Algorithm 1 of "Adaptive KV-Cache Compression without Manually Setting Budget"
 * (GVote), run once per layer at the end of prefill, per request and per KV head
 * (Section 3.2): fit a diagonal Gaussian to the hidden states (Step 2), draw S synthetic
 * hidden states (Step 3), project them through W_q and rotate them with the RoPE cos/sin
 * averaged over n_f future positions (Step 3), score them against all cached keys, let each
 * synthetic query pick its keys (top-k with k = |C0|, where C0 is the top-p set of the
 * current query, Step 1), OR the picks into one keep-mask per KV head (Step 4) and prune K
 * and V to that set (the pruning step of Algorithm 1).
 *
 * Conventions, valid for every entry point unless it says otherwise
 *  - Every pointer named below is a DEVICE pointer unless its comment says "host".
 *  - The caller owns every buffer.  The library allocates nothing, frees nothing and keeps
 *    no pointer after a call returns (gvote_compress_host is the one exception, see there).
 *  - Work is enqueued on the given CUDA stream (passed as void* = cudaStream_t); calls return
 *    without synchronising.
 *  - Return value: GVOTE_OK (0) or a negative GVOTE_ERR_* code.  On an error detected on the
 *    host nothing has been enqueued.  A bounded device-side wait that ran out is reported
 *    through the status word at the start of the workspace: read it with gvote_poll_status.
 *  - Pointers must be 16-byte aligned; d_h must be a multiple of 8, d_k a multiple of 8.
 *  - A ragged batch packs its requests along the token axis; cu_seqlens [batch+1] int32
 *    (device) holds the prefix sums of the request lengths N_r (request r owns tokens
 *    cu_seqlens[r] .. cu_seqlens[r+1]-1).  `total_tokens` = cu_seqlens[batch] and `max_N` =
 *    the longest request are passed from the host so that no call has to read the device.
 *    A request may be empty (N_r = 0): nothing is read or written for it, its budgets and |C0| are 0.
 *    A non-empty request needs N_r - n_s >= 2 rows for the fit.
 *  - bf16 tensors: W_q [n_q_heads*d_k, d_h], one row per output feature (the paper's W_q
 *    stored transposed, as linear layers keep it), row stride wq_ld elements;
 *    K and V [n_kv_heads, total_tokens, d_k] with element strides (head_stride, tok_stride),
 *    inner dimension contiguous; keys are stored as the model stores them (already rotated).
 *  - Positions: request r's keys sit at positions 0..N_r-1, its current query at N_r-1 and the
 *    n_f future positions are N_r .. N_r+n_f-1.
 *  - Keep-mask: uint32 words, bit (n mod 32) of word (n div 32) is key n of the request; each
 *    request's bit row starts on a word boundary at word gvote_mask_word_offset(cu_seqlens[r], r)
 *    of its head's row; a head's row has gvote_mask_row_words(total_tokens, batch) words;
 *    padding bits are zero.
 */
#ifndef GVOTE_H_
#define GVOTE_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define GVOTE_API __attribute__((visibility("default")))
#else
#define GVOTE_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

enum {
  GVOTE_OK = 0,
  GVOTE_ERR_INVALID_ARG = -1,
  GVOTE_ERR_UNALIGNED = -2,
  GVOTE_ERR_WORKSPACE_TOO_SMALL = -3,
  GVOTE_ERR_UNSUPPORTED_SHAPE = -4,
  GVOTE_ERR_CUDA = -5,
  GVOTE_ERR_TIMEOUT = -6
};

enum { GVOTE_SEL_TOPK_C0 = 0, GVOTE_SEL_TOPP = 1 };
enum { GVOTE_DTYPE_F32 = 0, GVOTE_DTYPE_BF16 = 1 };

/* Hyper-parameters and model shape (Algorithm 1, "Require" line, plus what it uses implicitly). */
typedef struct {
  int32_t d_h;          /* hidden size */
  int32_t n_q_heads;    /* query heads */
  int32_t n_kv_heads;   /* KV heads; n_q_heads must be a multiple */
  int32_t d_k;          /* head dimension */
  double  rope_theta;   /* RoPE base; rotate-half pairing (j, j+d_k/2), w_j = theta^(-2j/d_k) */
  int32_t S;            /* synthetic queries per request (Section 3.5: S >= 8 advised) */
  float   p_nuc;        /* nucleus mass threshold in (0,1] (Section 3.5: 0.95 advised) */
  int32_t n_f;          /* future positions whose cos/sin are averaged (Step 3) */
  int32_t n_s;          /* leading sink tokens the fit ignores (Step 2) */
  int32_t sel_mode;     /* GVOTE_SEL_TOPK_C0: the TopK step of Algorithm 1.  GVOTE_SEL_TOPP: the top-p rule
                           of Section 3.1 applied to every synthetic query instead. */
  int32_t include_c0;   /* non-zero: the current query's set C0 joins the union (Algorithm 1 unions
                           the synthetic sets only; default 0) */
  uint64_t seed;        /* Philox key */
  uint32_t layer_id;    /* Philox counter word: gives every layer its own stream */
  int32_t h_dtype;      /* GVOTE_DTYPE_F32 or GVOTE_DTYPE_BF16: element type of h and h_last */
} gvote_params;

/* Words per head in the keep-mask, and the word where request r's bits start. */
static inline int64_t gvote_mask_row_words(int64_t total_tokens, int32_t batch) {
  return (total_tokens >> 5) + batch;
}
static inline int64_t gvote_mask_word_offset(int64_t cu_seqlens_r, int32_t r) {
  return (cu_seqlens_r >> 5) + r;
}

/* Bytes of scratch every entry point below accepts as `ws` for a batch of this size.  The
 * first 256 bytes hold the status word; a workspace must be zero-filled once after
 * allocation (the library keeps it consistent afterwards).  Returns 0 on invalid params.
 * The size depends on p->sel_mode.  GVOTE_SEL_TOPK_C0 (Algorithm 1) keeps no logits matrix: per synthetic
 * query a few thousand sampled 16-bit keys and a short candidate list, per current query one fp32 row
 * (Section 4.4 names the S x N matrix as what runs out of memory beyond 128K context).  GVOTE_SEL_TOPP
 * needs every row's softmax mass and keeps the fp32 logits of all (S+1) x n_q_heads rows:
 * 4 (S+1) n_q_heads total_tokens bytes more.  A call that asks for the softmax rows (dbg_probs) needs the
 * GVOTE_SEL_TOPP size whatever its mode, as do shapes the fused kernels do not take (d_k other than 64
 * or 128, more than 16 query heads per KV head): gvote_workspace_bytes accounts for that. */
GVOTE_API size_t gvote_workspace_bytes(const gvote_params* p, int32_t batch, int64_t total_tokens, int64_t max_N);

/* Where gvote_select and the whole-pass entry points (gvote_compress, gvote_compress_moments, gvote_recompress) leave the
 * rotated queries of Algorithm 1 that their vote used - Q0 (exact position) and the S synthetic queries
 * (averaged cos/sin) of every query head: byte offset into `ws` of a bf16 array
 * [batch][n_kv_heads][G (S+1)][d_k], G = n_q_heads / n_kv_heads, the layout gvote_project writes (per KV
 * head the G*S synthetic rows, query head by query head, then the G current-query rows).  They stay valid
 * until the next call that uses the workspace; gvote_overlap and a caller's own checks can read them there.
 * Returns 0 on invalid params (offset 0 is the status block, never the queries). */
GVOTE_API size_t gvote_workspace_queries(const gvote_params* p, int32_t batch, int64_t total_tokens, int64_t max_N);

/* Step 2 of Section 3.2 (the Gaussian fit of Algorithm 1).  mu[r][c], var[r][c] = mean and unbiased variance over rows
 * cu_seqlens[r]+n_s .. cu_seqlens[r+1]-1 of h [total_tokens, d_h] (row stride h_row_stride
 * elements).  Every request needs N_r - n_s >= 2 (the result is NaN otherwise; the host cannot
 * check device-resident lengths, it checks max_N only).  mu, var: [batch, d_h] float. */
GVOTE_API int32_t gvote_fit(const gvote_params* p, const void* h, int64_t h_row_stride,
                  const int32_t* cu_seqlens, int32_t batch, int64_t total_tokens, int64_t max_N,
                  float* mu, float* var, void* ws, size_t ws_bytes, void* stream);

/* Step 2 while the prompt streams by (the Gaussian needs only running moments, not the hidden states:
 * an engine can feed each prefill chunk's layer-norm output and drop it, which takes the fit's read of
 * all hidden states out of the compression pass).
 * state: [batch, 3, d_h] double, zero-filled before the first block; per request and channel it
 * holds the number of rows seen, their mean and their sum of squared deviations.
 * gvote_fit_update folds one block of rows into the state: h_block [total_rows, d_h] holds the new rows
 * of every request, request r owning rows cu_block[r] .. cu_block[r+1]-1 (a request may have none).
 * Every row given is counted: leaving out the n_s sink tokens is the caller's doing here (p->n_s is not
 * used).  Blocks are merged with the pairwise update of Chan, Golub and LeVeque in fp64.
 * gvote_fit_finish turns the state into mu and the unbiased variance (NaN below two rows), the inputs
 * of gvote_sample and gvote_compress_moments. */
GVOTE_API int32_t gvote_fit_update(const gvote_params* p, const void* h_block, int64_t h_row_stride,
                         const int32_t* cu_block, int32_t batch, int64_t total_rows, int64_t max_rows,
                         double* state, void* ws, size_t ws_bytes, void* stream);
GVOTE_API int32_t gvote_fit_finish(const gvote_params* p, const double* state, int32_t batch,
                         float* mu, float* var, void* stream);

/* Fit without any allocation (the paper has no counterpart: this entry point exists for the
 * integration, not for the method).  Same result as gvote_fit, but the per-chunk partial moments
 * live in a fixed 1 MiB array inside the library's device image (GVOTE_FIT_STATIC_MAX_ENTRIES
 * pairs of floats, present on every GPU that loads the library until the process exits), so the
 * caller passes inputs and outputs only and the call obtains no memory, from CUDA or from
 * anyone else.  Use it where asking for device memory is not possible: inside an allocator or
 * memory-pool callback, in a serving loop whose pool is frozen after warm-up, on a thread that
 * may not wait on the allocator's lock.
 *  - Limit: batch * d_h <= GVOTE_FIT_STATIC_MAX_ENTRIES, else GVOTE_ERR_UNSUPPORTED_SHAPE and
 *    nothing is enqueued.  Long inputs are fine: fewer, longer row chunks are used instead.
 *  - The first call on each device looks up the array's device address (with that device
 *    current).  Make that first call before starting any stream capture.
 *  - All calls on a device share the one array.  It needs no clearing (every entry a call reads
 *    it has written itself), but two calls whose kernels may overlap on the GPU (different
 *    streams, no dependency) race on it: serialise them.
 *  - There is no status word here: a bounded device-side wait that ran out shows as NaN in mu.
 * Arguments as in gvote_fit, minus the workspace and total_tokens. */
#define GVOTE_FIT_STATIC_MAX_ENTRIES 131072
GVOTE_API int32_t gvote_fit_static(const gvote_params* p, const void* h, int64_t h_row_stride,
                         const int32_t* cu_seqlens, int32_t batch, int64_t max_N,
                         float* mu, float* var, void* stream);

/* Step 3 of Section 3.2 (the sampling step of Algorithm 1).  H_tilde[r][s][c] = mu[r][c] + sqrt(var[r][c]) * z, z a standard
 * normal drawn by Box-Muller from Philox4x32-10 with key = (seed low, seed high) and counter
 * = (c div 4, s, layer_id, r); word pairs (0,1) and (2,3) of a block give channels 4b..4b+3;
 * u = ((x >> 9) + 0.5) * 2^-23.  H_tilde: [batch, S, d_h] float.  raw_u32_or_null, when given,
 * receives the Philox words [batch, S, d_h] (bit-exact by definition). */
GVOTE_API int32_t gvote_sample(const gvote_params* p, const float* mu, const float* var, int32_t batch,
                     float* H_tilde, uint32_t* raw_u32_or_null, void* stream);

/* Algorithm 1: the current query Q0, AverageCosSin and the synthetic queries.  X = [h_last[r]; H_tilde[r]] is rounded to bf16, multiplied
 * by W_q (fp32 accumulation), b_q added when given ([n_q_heads*d_k] float), then rotated: row 0
 * exactly at position N_r-1, rows 1..S with the mean cos/sin of positions N_r..N_r+n_f-1.
 * Q: [batch, n_kv_heads, G*(S+1), d_k] bf16 with G = n_q_heads / n_kv_heads; the rows of a KV head
 * are ordered for the score contraction: first the S synthetic rows of each of its G query heads
 * (row gl*S + s), then the G current-query rows (row G*S + gl).  h_last: [batch, d_h] of p->h_dtype. */
GVOTE_API int32_t gvote_project(const gvote_params* p, const float* H_tilde, const void* h_last,
                      const void* W_q, int64_t wq_ld, const float* b_q_or_null,
                      const int32_t* cu_seqlens, int32_t batch,
                      void* Q, void* ws, size_t ws_bytes, void* stream);

/* Algorithm 1, the current-query steps (A0, C0, B_step) and the vote (logits, TopK, union), given the rotated queries (layout as written by gvote_project).
 * Per query head g: logits of its
 * S+1 rows against the N_r keys of KV head g div G, scaled by 1/sqrt(d_k); row 0 -> softmax ->
 * top-p -> b_step[r][g] = |C0|; rows 1..S -> top-k(b_step) on logits (or top-p on their softmax
 * in GVOTE_SEL_TOPP); mask[h] = OR over the rows of the head's group; budget[r][h] = popcount.
 * Ties at a selection boundary go to the lower key index.  mask: [n_kv_heads, row_words] is
 * overwritten.  dbg_probs_or_null: [sum_r n_q_heads*(S+1)*N_r] float, request-major, receives the
 * softmax rows (small cases only). */
GVOTE_API int32_t gvote_vote(const gvote_params* p, const void* Q,
                   const void* K, int64_t k_tok_stride, int64_t k_head_stride,
                   const int32_t* cu_seqlens, int32_t batch, int64_t total_tokens, int64_t max_N,
                   uint32_t* mask, int32_t* budget, int32_t* b_step,
                   float* dbg_probs_or_null, void* ws, size_t ws_bytes, void* stream);

/* gvote_project followed by gvote_vote (Algorithm 1 without the fit, the sampling and the pruning); Q lives in ws. */
GVOTE_API int32_t gvote_select(const gvote_params* p, const float* H_tilde, const void* h_last,
                     const void* W_q, int64_t wq_ld, const float* b_q_or_null,
                     const void* K, int64_t k_tok_stride, int64_t k_head_stride,
                     const int32_t* cu_seqlens, int32_t batch, int64_t total_tokens, int64_t max_N,
                     uint32_t* mask, int32_t* budget, int32_t* b_step,
                     float* dbg_probs_or_null, void* ws, size_t ws_bytes, void* stream);

/* Algorithm 1, the pruning step.  In place: for every request r and KV head h the kept rows of K and V
 * move, in ascending key order, to rows cu_seqlens[r] .. cu_seqlens[r]+budget[r][h]-1 of the
 * head's slab; rows behind them are left as they are.  budget [batch, n_kv_heads] is written
 * (popcount of the mask).  Rows are d_k bf16 values, moved in 16-byte pieces. */
GVOTE_API int32_t gvote_compact(const gvote_params* p, void* K, void* V, int64_t tok_stride, int64_t head_stride,
                      const uint32_t* mask, const int32_t* cu_seqlens, int32_t batch,
                      int64_t total_tokens, int64_t max_N, int32_t* budget,
                      void* ws, size_t ws_bytes, void* stream);

/* Section 3.3's yardstick applied to a keep-mask: overlap[r][g] = the share of the current query's
 * attention (softmax weights of Eq. 1 over all N_r keys) of query head g that falls on the keys its
 * KV head keeps; 1 means nothing the query looks at was pruned.  Q as written by gvote_project (the
 * current-query rows are used), K the UNPRUNED keys, mask as written by gvote_vote.  overlap:
 * [batch, n_q_heads] float.  A diagnostic: fp32 logits, not on the compression path. */
GVOTE_API int32_t gvote_overlap(const gvote_params* p, const void* Q,
                      const void* K, int64_t k_tok_stride, int64_t k_head_stride,
                      const uint32_t* mask, const int32_t* cu_seqlens, int32_t batch,
                      int64_t total_tokens, int64_t max_N, float* overlap,
                      void* ws, size_t ws_bytes, void* stream);

/* Section 3.4: the pruned cache in the layout a variable-length attention kernel consumes, written
 * out of place from the UNPRUNED K and V and the keep-mask (use it instead of gvote_compact when
 * the engine wants one dense buffer rather than per-head slabs).  "Sequence" s = r * n_kv_heads + h
 * (request r, KV head h) owns rows cu_seqlens_k[s] .. cu_seqlens_k[s+1]-1 of K_packed and V_packed
 * ([capacity_rows, d_k] bf16, dense), kept rows in ascending key order; cu_seqlens_k
 * [batch*n_kv_heads + 1] int32 and budget [batch, n_kv_heads] are written.  The buffers need
 * cu_seqlens_k[last] rows, at most n_kv_heads * total_tokens; if capacity_rows is smaller than what the
 * mask keeps, the rows that do not fit are not written and the workspace status word reads
 * GVOTE_ERR_WORKSPACE_TOO_SMALL (gvote_poll_status).  K and V are not modified. */
GVOTE_API int32_t gvote_pack(const gvote_params* p, const void* K, const void* V, int64_t tok_stride, int64_t head_stride,
                   const uint32_t* mask, const int32_t* cu_seqlens, int32_t batch,
                   int64_t total_tokens, int64_t max_N, void* K_packed, void* V_packed, int64_t capacity_rows,
                   int32_t* cu_seqlens_k, int32_t* budget, void* ws, size_t ws_bytes, void* stream);

/* Algorithm 1, whole: fit, sample, project, vote, compact for one layer.  The current query's
 * hidden state is the last row of each request in h unless h_last_or_null is given.
 * Outputs: mask, budget, b_step as in gvote_vote; K and V compacted in place. */
GVOTE_API int32_t gvote_compress(const gvote_params* p, const void* h, int64_t h_row_stride, const void* h_last_or_null,
                       const void* W_q, int64_t wq_ld, const float* b_q_or_null,
                       void* K, void* V, int64_t tok_stride, int64_t head_stride,
                       const int32_t* cu_seqlens, int32_t batch, int64_t total_tokens, int64_t max_N,
                       uint32_t* mask, int32_t* budget, int32_t* b_step,
                       void* ws, size_t ws_bytes, void* stream);

/* Algorithm 1 from the sampling step on, for a caller that already has the Gaussian (gvote_fit_finish): sample,
 * project, vote, compact.  mu, var [batch, d_h] float; h_last [batch, d_h] of p->h_dtype is the current
 * query's hidden state.  Other arguments and outputs as in gvote_compress. */
GVOTE_API int32_t gvote_compress_moments(const gvote_params* p, const float* mu, const float* var, const void* h_last,
                               const void* W_q, int64_t wq_ld, const float* b_q_or_null,
                               void* K, void* V, int64_t tok_stride, int64_t head_stride,
                               const int32_t* cu_seqlens, int32_t batch, int64_t total_tokens, int64_t max_N,
                               uint32_t* mask, int32_t* budget, int32_t* b_step,
                               void* ws, size_t ws_bytes, void* stream);

/* The pass applied again to a cache it has pruned before and that has grown since (an extension: in
 * Section 3.4 the pass runs once, after prefill).  The heads of such a cache differ in length, and a slot
 * no longer is a position, so the N of Algorithm 1 splits in two:
 *  - kv_len [batch, n_kv_heads] int32 (device): rows KV head h of request r holds (kept earlier plus
 *    appended since), at the front of its slab cu_seqlens[r] .. ; rows beyond are ignored.  Every query
 *    head votes over the rows of its own KV head only (current-query steps and vote); kv_len may be 0 (budget 0).
 *  - seq_len [batch] int32 (device): tokens the request has seen.  The current query is rotated at
 *    position seq_len - 1, the synthetic queries with the mean over positions seq_len .. seq_len+n_f-1
 *    (the current query and AverageCosSin); keys stay rotated where they were written.
 *  - cu_seqlens / total_tokens / max_N describe the slabs (capacity), as in gvote_compress.
 *  - token_pos_or_null [n_kv_heads, total_tokens] int32 (device, in/out): the original position of every
 *    slot; its kept entries move to the front of the slab with the rows (entries beyond the new budget
 *    are left as they were).
 * mu, var: the caller's running fit (gvote_fit_update / gvote_fit_finish over all tokens seen).
 * Outputs as in gvote_compress: mask over slots, budget = new rows per head, b_step, K and V compacted
 * in place. */
GVOTE_API int32_t gvote_recompress(const gvote_params* p, const float* mu, const float* var, const void* h_last,
                         const void* W_q, int64_t wq_ld, const float* b_q_or_null,
                         void* K, void* V, int64_t tok_stride, int64_t head_stride,
                         const int32_t* cu_seqlens, const int32_t* kv_len, const int32_t* seq_len,
                         int32_t* token_pos_or_null, int32_t batch, int64_t total_tokens, int64_t max_N,
                         uint32_t* mask, int32_t* budget, int32_t* b_step,
                         void* ws, size_t ws_bytes, void* stream);

/* The same pass for a caller whose tensors live in HOST memory (pinned memory gives full copy
 * speed): all pointers are host pointers, K and V are dense ([n_kv_heads, total_tokens, d_k]),
 * h is dense [total_tokens, d_h].  The call copies the inputs to device buffers it keeps in a
 * grow-only per-device arena (released by gvote_host_arena_release), runs gvote_compress on an
 * internal stream, copies mask, budget, b_step and the compacted K and V back, and returns after
 * everything has completed.  This is the only entry point that allocates or synchronises. */
GVOTE_API int32_t gvote_compress_host(const gvote_params* p, const void* h, const void* W_q, const float* b_q_or_null,
                            void* K, void* V, const int32_t* cu_seqlens_host, int32_t batch,
                            uint32_t* mask, int32_t* budget, int32_t* b_step);
GVOTE_API void gvote_host_arena_release(void);

/* Reads the status word of a workspace (synchronises the stream): GVOTE_OK, GVOTE_ERR_TIMEOUT (a bounded
 * device-side wait ran out) or GVOTE_ERR_WORKSPACE_TOO_SMALL (gvote_pack: capacity_rows too small).  The word
 * is only ever set by kernels and STAYS set: every later poll of that workspace reports it again until the
 * caller clears it, with gvote_clear_status (enqueued on the stream) or by zero-filling the first 256 bytes.
 * gvote_compress_host clears the status of its own arena at the start of every call. */
GVOTE_API int32_t gvote_poll_status(void* ws, void* stream);
GVOTE_API int32_t gvote_clear_status(void* ws, void* stream);

/* Diagnostic of the default selection mode (Algorithm 1's TopK step): how many (request, KV head) pairs
 * had to be selected again by the exact route because a row's sampled bracket missed its k-th logit or a
 * candidate list overflowed, since the workspace's status block was last cleared (synchronises the
 * stream).  The result is the same either way; the exact route only costs time.  Negative: an error code. */
GVOTE_API int64_t gvote_exact_heads(void* ws, void* stream);

/* Per-kernel timing for benchmarks.  While enabled, every kernel launch of the library is
 * bracketed by two CUDA events on its stream.  Enabling (or disabling) drops earlier records.
 * gvote_profile_report synchronises the device and writes one text line per kernel,
 * "name launches total_ms", into buf (host, NUL-terminated, truncated to cap); it returns the
 * bytes needed.  Not thread safe against concurrent launches from other threads. */
GVOTE_API void gvote_profile_enable(int32_t on);
GVOTE_API size_t gvote_profile_report(char* buf, size_t cap);

/* Number of kernel launches the library has enqueued in this process (all entry points). */
GVOTE_API int64_t gvote_launch_count(void);

GVOTE_API const char* gvote_status_string(int32_t status);
/* Text of the last CUDA error seen by the calling thread's last failing call ("" if none). */
GVOTE_API const char* gvote_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* GVOTE_H_ */
