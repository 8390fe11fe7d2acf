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

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int32_t validate_params(const gvote_params* p);

// ---------------------------------------------------------------------------------- workspace
// Status block (first 256 bytes): word 0 = sticky error status, word 1 = where it was raised.
constexpr size_t kStatusBytes = 256;
constexpr int kCompactTile = 128;   // tokens per compaction tile
constexpr int kFitStripCols = 256;  // channels per fit CTA (64 threads x float4)

struct WorkspaceMap {
  size_t status;        // int32[64]
  size_t fit_partial;   // float2 [batch][fit_chunks][d_h]
  size_t mu, var;       // float [batch][d_h]
  size_t h_tilde;       // float [batch][S][d_h]
  size_t x_bf16;        // bf16 [batch][S+1][d_h]
  size_t q_f32;         // float [proj_splits][batch*(S+1)][Hq*d_k]
  size_t q_bf16;        // bf16 [batch][Hq][S+1][d_k]
  size_t rope;          // float [batch][4][d_k/2]  (cos0, sin0, cbar, sbar)
  size_t logits;        // float [Hq*(S+1) * total_tokens], request-major
  size_t keys16;        // uint16 [Hq*S * (padded tokens)]: 16-bit logit keys of the synthetic rows
  size_t prefix;        // int32 [Hkv][row_words]  exclusive popcount prefix per mask word
  size_t flags;         // int32 [2*Hkv*n_tiles + 4]  compaction "tile loaded" flags + ticket
  size_t total;
  int fit_chunks;       // row chunks per request in the fit
  int proj_splits;      // split-K factor of the projection
  int64_t n_tiles;      // compaction tiles over the packed token axis (upper bound)
  int64_t row_words;    // mask words per head
};

// Row tiling of the tensor-core score kernel: the (S+1)*G rows of a head group are split into
// `row_chunks` chunks of RC rows (RC a multiple of 16, at most 240).
struct ScoreGeometry { int RC; int row_chunks; };
ScoreGeometry score_geometry(const gvote_params* p);
size_t keys16_elems(const gvote_params* p, int32_t batch, int64_t total_tokens);
WorkspaceMap workspace_map(const gvote_params* p, int32_t batch, int64_t total_tokens, int64_t max_N);

// ---------------------------------------------------------------------------------- stage launchers
// (each enqueues kernels on `st`; pointers are device pointers; see gvote.h for the layouts)
int32_t launch_fit(const gvote_params* p, const void* h, int64_t ld, const int32_t* cu, int32_t batch,
                   int fit_chunks, float2* partial, float* mu, float* var, cudaStream_t st);
int32_t launch_sample(const gvote_params* p, const float* mu, const float* var, int32_t batch,
                      float* H_tilde, uint32_t* raw, cudaStream_t st);
int32_t launch_project(const gvote_params* p, const float* H_tilde, const void* h_last, int64_t h_last_ld,
                       const int32_t* h_last_rows_from_cu,  // when non-null: row index = cu[r+1]-1 of h_last
                       const void* W_q, int64_t wq_ld, const float* b_q, const int32_t* cu, int32_t batch,
                       const WorkspaceMap& m, char* ws, __nv_bfloat16* Q, cudaStream_t st);
int32_t launch_vote(const gvote_params* p, const __nv_bfloat16* Q, const __nv_bfloat16* K, int64_t k_tok,
                    int64_t k_head, const int32_t* cu, int32_t batch, int64_t total_tokens, int64_t max_N,
                    uint32_t* mask, int32_t* budget, int32_t* b_step, float* dbg_probs,
                    const WorkspaceMap& m, char* ws, cudaStream_t st);
int32_t launch_compact(const gvote_params* p, __nv_bfloat16* K, __nv_bfloat16* V, int64_t tok, int64_t head,
                       const uint32_t* mask, const int32_t* cu, int32_t batch, int64_t total_tokens,
                       int64_t max_N, int32_t* budget, const WorkspaceMap& m, char* ws, cudaStream_t st);

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

#endif  // __CUDACC__

}  // namespace gvote
