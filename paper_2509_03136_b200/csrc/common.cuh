// Shared host/device helpers of the GVote library: error plumbing, the workspace map and a
// few device utilities.  Nothing here is specific to one step of Algorithm 1.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/gvote.h"

namespace gvote {

// ---------------------------------------------------------------------------------- errors
void set_cuda_error(cudaError_t e, const char* where);
void count_launch(int n = 1);

// Brackets one kernel launch with CUDA events on its stream when per-kernel timing is switched on
// (gvote_profile_enable); otherwise it does nothing.
struct LaunchScope {
  LaunchScope(const char* name, cudaStream_t st);
  ~LaunchScope();
  int slot;
  cudaStream_t st;
};

#define GVOTE_CUDA_CHECK(expr)                                   \
  do {                                                           \
    cudaError_t e__ = (expr);                                    \
    if (e__ != cudaSuccess) {                                    \
      ::gvote::set_cuda_error(e__, #expr);                       \
      return GVOTE_ERR_CUDA;                                     \
    }                                                            \
  } while (0)

#define GVOTE_LAUNCH_CHECK(name)                                 \
  do {                                                           \
    ::gvote::count_launch();                                     \
    cudaError_t e__ = cudaGetLastError();                        \
    if (e__ != cudaSuccess) {                                    \
      ::gvote::set_cuda_error(e__, name);                        \
      return GVOTE_ERR_CUDA;                                     \
    }                                                            \
  } while (0)

// One kernel launch on a stream (typed: the arguments are converted to the kernel's parameter types).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_on(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                             Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int32_t validate_params(const gvote_params* p);

// ---------------------------------------------------------------------------------- workspace
// Status block (first 256 bytes): word 0 = sticky error status, word 1 = where it was raised.
constexpr size_t kStatusBytes = 256;
constexpr int kCompactTile = 128;   // tokens per compaction tile
constexpr int kFitStripCols = 256;  // channels per fit CTA (64 column threads x 4 channels)
constexpr int kOverlapKeys = 1024;  // keys per CTA of the attention-overlap diagnostic

struct WorkspaceMap {
  size_t status;        // int32[64]
  size_t fit_partial;   // float2 [batch][fit_chunks][d_h]
  size_t mu, var;       // float [batch][d_h]
  size_t h_tilde;       // float [batch][S][d_h]
  size_t x_bf16;        // bf16 [batch][S+1][d_h]
  size_t q_f32;         // float [proj_splits][batch*(S+1)][Hq*d_k]
  size_t q_bf16;        // bf16 [batch][Hq][S+1][d_k]
  size_t rope;          // float [batch][4][d_k/2]  (cos0, sin0, cbar, sbar)
  // --- the vote.  full_rows: fp32 logits of every row, [Hq*(S+1) * total_tokens] request-major (the
  // per-sample top-p mode, the softmax dump, shapes the tensor-core kernels do not take); otherwise only
  // the current-query rows, [Hq * total_tokens], and the state of the fused top-k (vote_geom.cuh)
  bool full_rows;
  size_t logits;
  size_t tmask;         // uint32 [Hkv][row_words]   (cleared, like head_bad and the keep mask, by the vote's first kernel)
  size_t head_bad;      // uint32 [batch][Hkv]
  size_t rowmax;        // uint32 [batch][Hq][<= 148]  maxima of the current-query rows met by the first pass's CTAs
  size_t sample;        // uint16 [Hkv][sample_slots][row_chunks][128][128]
  size_t bracket;       // RowBracket [batch*Hq*S]
  size_t segstat;       // uint2 [batch*Hq*S][cand_segs]
  size_t cand;          // uint2 [Hq*S][cand_strip]
  int64_t cand_strip;
  int cand_segs;
  int64_t sample_slots;
  size_t remap_tmp;     // int32 [Hkv][total_tokens]  scratch of the slot -> position map's gather
  size_t ov_partial;    // float4 [batch][Hq][ceil(max_N / kOverlapKeys)]  partial sums of gvote_overlap
  size_t prefix;        // int32 [Hkv][row_words]  exclusive popcount prefix per mask word
  size_t flags;         // int32 [2*Hkv*n_tiles] compaction "tile loaded" flags + [2*Hkv][32] ticket counters
  size_t total;
  int fit_chunks;       // row chunks per request in the fit
  int proj_splits;      // split-K factor of the projection
  int64_t n_tiles;      // compaction tiles over the packed token axis (upper bound)
  int64_t row_words;    // mask words per head
};

// Row tiling of the tensor-core score kernel: the G*S synthetic rows of a head group are split into
// `row_chunks` chunks of RC = 128 rows (the current-query rows travel with chunk 0).
struct ScoreGeometry { int RC; int row_chunks; };
ScoreGeometry score_geometry(const gvote_params* p);
bool sweep_umma_supported(const gvote_params* p);
// Whether the vote of these parameters keeps fp32 logits of every row (see WorkspaceMap::full_rows).
bool vote_needs_full_rows(const gvote_params* p);
WorkspaceMap workspace_map(const gvote_params* p, int32_t batch, int64_t total_tokens, int64_t max_N,
                           bool full_rows);
inline WorkspaceMap workspace_map(const gvote_params* p, int32_t batch, int64_t total_tokens, int64_t max_N) {
  return workspace_map(p, batch, total_tokens, max_N, vote_needs_full_rows(p));
}

// ---------------------------------------------------------------------------------- stage launchers
// (each enqueues kernels on `st`; pointers are device pointers; see gvote.h for the layouts)
int32_t launch_fit(const gvote_params* p, const void* h, int64_t ld, const int32_t* cu, int32_t batch,
                   int64_t rows_bound, int fit_chunks, float2* partial, int32_t* status, float* mu, float* var,
                   cudaStream_t st);
int32_t launch_fit_partial(const gvote_params* p, const void* h, int64_t ld, const int32_t* cu, int32_t batch,
                           int64_t rows_bound, int fit_chunks, float2* partial, int32_t* status, cudaStream_t st);
int32_t launch_fit_state_update(const gvote_params* p, const void* h, int64_t ld, const int32_t* cu, int32_t batch,
                                int64_t rows_bound, int fit_chunks, float2* partial, int32_t* status, double* state,
                                cudaStream_t st);
// Row chunks per request for the fit (see fit.cu).
int fit_chunk_count(const gvote_params* p, int32_t batch, int64_t max_N);
int32_t launch_fit_state_finish(const gvote_params* p, const double* state, int32_t batch, float* mu, float* var,
                                cudaStream_t st);
int32_t launch_sample(const gvote_params* p, const float* mu, const float* var, int32_t batch,
                      float* H_tilde, uint32_t* raw, cudaStream_t st);
// Fused middle of the whole pass: merges the fit partials (mu, var), draws the S samples and writes
// the bf16 projection input X = [h_last; H~] and the RoPE tables, in one launch.
int32_t launch_prep(const gvote_params* p, const float2* partial, int fit_chunks, const void* h_last,
                    int64_t h_last_ld, const int32_t* h_last_rows_from_cu, const int32_t* cu, int32_t batch,
                    float* mu, float* var, __nv_bfloat16* X, float* rope_table, cudaStream_t st);
// Projection of a staged X (bf16 [batch*(S+1), d_h]) with ready RoPE tables: GEMM + finish.
int32_t launch_project_staged(const gvote_params* p, const __nv_bfloat16* X, const float* rope_table, const void* W_q,
                              int64_t wq_ld, const float* b_q, int32_t batch, const WorkspaceMap& m, char* ws,
                              __nv_bfloat16* Q, cudaStream_t st);
int project_umma_splits(const gvote_params* p, int rows_total);
int32_t launch_project(const gvote_params* p, const float* H_tilde, const void* h_last, int64_t h_last_ld,
                       const int32_t* h_last_rows_from_cu,  // when non-null: row index = cu[r+1]-1 of h_last
                       const void* W_q, int64_t wq_ld, const float* b_q, const int32_t* cu, int32_t batch,
                       const WorkspaceMap& m, char* ws, __nv_bfloat16* Q, cudaStream_t st,
                       const int32_t* seq_len = nullptr);  // [batch] tokens seen (positions), or the slab lengths
// Moves the kept entries of a per-head slot -> position map to the front of each slab, like the rows.
int32_t launch_remap(const gvote_params* p, int32_t* token_pos, const uint32_t* mask, const int32_t* cu, int32_t batch,
                     int64_t total_tokens, int64_t max_N, const int32_t* budget, const WorkspaceMap& m, char* ws,
                     cudaStream_t st);
int32_t launch_vote(const gvote_params* p, const __nv_bfloat16* Q, const __nv_bfloat16* K, int64_t k_tok,
                    int64_t k_head, const int32_t* cu, int32_t batch, int64_t total_tokens, int64_t max_N,
                    uint32_t* mask, int32_t* budget, int32_t* b_step, float* dbg_probs,
                    char* ws, size_t ws_bytes, cudaStream_t st,
                    const int32_t* kv_len = nullptr,    // [batch][n_kv_heads] rows that count, or all
                    bool* merge_deferred = nullptr);    // given: the vote may leave the union of the settled heads in
                                                        // the workspace's tentative mask for launch_compact's scan
                                                        // to merge (*merge_deferred says whether it did)
// merge_tentative: see launch_vote; the mask is then written, too.
int32_t launch_compact(const gvote_params* p, __nv_bfloat16* K, __nv_bfloat16* V, int64_t tok, int64_t head,
                       const uint32_t* mask, const int32_t* cu, int32_t batch, int64_t total_tokens,
                       int64_t max_N, int32_t* budget, const WorkspaceMap& m, char* ws, cudaStream_t st,
                       bool merge_tentative = false);

int32_t launch_pack(const gvote_params* p, const __nv_bfloat16* K, const __nv_bfloat16* V, int64_t tok, int64_t head,
                    const uint32_t* mask, const int32_t* cu, int32_t batch, int64_t total_tokens, int64_t max_N,
                    __nv_bfloat16* K_packed, __nv_bfloat16* V_packed, int64_t capacity_rows, int32_t* cu_seqlens_k,
                    int32_t* budget, const WorkspaceMap& m, char* ws, cudaStream_t st);

int32_t launch_overlap(const gvote_params* p, const __nv_bfloat16* Q, const __nv_bfloat16* K, int64_t k_tok,
                       int64_t k_head, const uint32_t* mask, const int32_t* cu, int32_t batch, int64_t max_N,
                       float* overlap, const WorkspaceMap& m, char* ws, cudaStream_t st);

// ---------------------------------------------------------------------------------- device helpers
#ifdef __CUDACC__

// Monotone map from float to uint32: a > b  <=>  key(a) > key(b)  (no NaNs expected).
__device__ __forceinline__ uint32_t ordered_key(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ int warp_sum_i(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Request lookup shared by the ragged kernels: word offset of request r in a mask row and
// tile offset in the compaction tile list (both over-allocate by one unit per request).
__device__ __forceinline__ int64_t mask_word_offset(int cu_r, int r) { return (int64_t)(cu_r >> 5) + r; }
__device__ __forceinline__ int64_t tile_offset(int cu_r, int r) { return (int64_t)(cu_r >> 7) + r; }


// Rows of chunk `c` of a request whose fitted rows are [first, last): [a, b).
// Keys of KV head kh of request r that take part in the vote: all N rows of the request's slab, or
// (a cache that was pruned before: heads differ in length) the head's own count kv_len[r][kh].
__device__ __forceinline__ int valid_keys(const int32_t* __restrict__ kv_len, int r, int n_kv_heads, int kh, int N) {
  if (!kv_len) return N;
  const int v = kv_len[r * n_kv_heads + kh];
  return v < 0 ? 0 : (v < N ? v : N);
}

__device__ __forceinline__ void fit_chunk_rows(int first, int last, int chunks, int c, int& a, int& b) {
  const int n = max(last - first, 0);
  const int per = (n + chunks - 1) / chunks;
  a = min(first + c * per, last);
  b = min(a + per, last);
}

// Merging the per-chunk (mean, M2) pairs of one channel (the pairwise update of Chan, Golub and
// LeVeque, written against a common reference value so that one pass and no division per chunk
// suffice): with ref = mean of chunk 0, A = sum n_c (mean_c - ref), B = sum n_c (mean_c - ref)^2,
// C = sum M2_c, the merged mean is ref + A/n and the merged M2 is C + B - A^2/n.  `lane` of
// `lanes` takes every lanes-th chunk; the caller adds the lanes' (n, A, B + C) and finishes.
struct FitMoments { double n, a, bc; };
__device__ __forceinline__ FitMoments fit_merge_lane(const float2* __restrict__ partial, int r, int chunks, int d_h,
                                                     int col, int first, int last, int lane, int lanes, double ref) {
  FitMoments m{0.0, 0.0, 0.0};
  for (int c = lane; c < chunks; c += lanes) {
    int a, b;
    fit_chunk_rows(first, last, chunks, c, a, b);
    if (b <= a) continue;
    const float2 pc = partial[((int64_t)(r * chunks + c)) * d_h + col];
    const double nc = (double)(b - a), d = (double)pc.x - ref;
    m.n += nc;
    m.a = fma(nc, d, m.a);
    m.bc += fma(nc * d, d, (double)pc.y);
  }
  return m;
}
__device__ __forceinline__ void fit_merge_finish(const FitMoments& m, double ref, float& mu, float& var) {
  const double mean = ref + m.a / m.n;
  const double m2 = m.bc - m.a * m.a / m.n;
  mu = (float)mean;
  var = (float)(fmax(m2, 0.0) / (m.n - 1.0));      // NaN/inf when fewer than 2 rows
}

#endif  // __CUDACC__

}  // namespace gvote
