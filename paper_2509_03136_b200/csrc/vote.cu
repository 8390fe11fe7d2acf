// Algorithm 1, the current-query steps and the vote: attention logits of the current query and of the S synthetic
// queries against all cached keys, the current query's top-p set size |C0| (the step budget),
// each synthetic query's selection (top-k with k = |C0|, or top-p in the alternative mode), and
// the union of the selections as one keep bit-mask per KV head.
//
// Selection never sorts.  A row's threshold is found by a most-significant-digit radix search
// over an order-preserving 32-bit image of the fp32 logit: three histogram passes (11, 11 and 10
// bits) in shared memory narrow the threshold to one exact value; counts are integers and
// softmax mass is accumulated in 2^-40 fixed point, so the search is order independent and two
// runs give the same bits.  Ties at the threshold go to the lower key index.  The union is a
// warp ballot per 32 keys OR-ed into the mask word.
#include "common.cuh"
#include "select_common.cuh"
#include "vote_geom.cuh"

namespace gvote {
namespace {

using namespace sel;

constexpr int kSelThreads = 256;

// ---------------------------------------------------------------------------------- logits (SIMT)
// logits[row][n] = (Q[row] . K[n]) / sqrt(d_k) for the rows of one KV head's group.
// CTA: 64 keys x all group rows; thread: 2 keys x 8 rows.
constexpr int kScoreKeys = 64;
constexpr int kScoreRowChunk = 64;

__global__ void __launch_bounds__(256)
score_simt_kernel(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K, int64_t k_tok,
                  int64_t k_head, const int32_t* __restrict__ cu, int Hq, int G, int S1, int d_k, float scale,
                  float* __restrict__ logits) {
  extern __shared__ __align__(16) uint32_t smem_u32[];
  const int r = blockIdx.z, kh = blockIdx.y;
  const int start = cu[r], N = cu[r + 1] - start;
  const int n0 = blockIdx.x * kScoreKeys;
  if (n0 >= N) return;
  const int half = d_k / 2;               // bf16 pairs per row
  const int kpitch = half + 1;            // odd pitch: conflict-free across keys
  uint32_t* Ks = smem_u32;                              // [64][kpitch]
  uint32_t* Qs = smem_u32 + kScoreKeys * kpitch;        // [64][half]
  const int tid = threadIdx.x, lane = tid & 31, rg = tid >> 5;   // 8 row groups of 8 rows

  const __nv_bfloat16* Kbase = K + (int64_t)kh * k_head + (int64_t)(start + n0) * k_tok;
  for (int idx = tid; idx < kScoreKeys * half; idx += blockDim.x) {
    const int key = idx / half, d2 = idx % half;
    uint32_t v = 0;
    if (n0 + key < N) v = *reinterpret_cast<const uint32_t*>(Kbase + (int64_t)key * k_tok + 2 * d2);
    Ks[key * kpitch + d2] = v;
  }
  const int R = G * S1;
  const __nv_bfloat16* Qbase = Q + ((int64_t)r * (Hq / G) + kh) * R * d_k;   // the group's rows: synthetic first, then real
  float* Lbase = logits + (int64_t)Hq * S1 * start + (int64_t)kh * G * S1 * N;

  for (int c0 = 0; c0 < R; c0 += kScoreRowChunk) {
    __syncthreads();
    for (int idx = tid; idx < kScoreRowChunk * half; idx += blockDim.x) {
      const int row = idx / half, d2 = idx % half;
      uint32_t v = 0;
      if (c0 + row < R) v = *reinterpret_cast<const uint32_t*>(Qbase + (int64_t)(c0 + row) * d_k + 2 * d2);
      Qs[row * half + d2] = v;
    }
    __syncthreads();
    float acc0[8], acc1[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) { acc0[j] = 0.f; acc1[j] = 0.f; }
    for (int d2 = 0; d2 < half; ++d2) {
      const float2 ka = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&Ks[lane * kpitch + d2]));
      const float2 kb = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&Ks[(lane + 32) * kpitch + d2]));
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float2 q = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&Qs[(rg * 8 + j) * half + d2]));
        acc0[j] = fmaf(q.x, ka.x, acc0[j]); acc0[j] = fmaf(q.y, ka.y, acc0[j]);
        acc1[j] = fmaf(q.x, kb.x, acc1[j]); acc1[j] = fmaf(q.y, kb.y, acc1[j]);
      }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int grow = c0 + rg * 8 + j;
      if (grow < R) {
        // group row -> (query head, sample): the logits buffer keeps row 0 of a head for the real query
        const int S = S1 - 1;
        const int row = (grow < G * S) ? (grow / S) * S1 + grow % S + 1 : (grow - G * S) * S1;
        if (n0 + lane < N) Lbase[(int64_t)row * N + n0 + lane] = acc0[j] * scale;
        if (n0 + lane + 32 < N) Lbase[(int64_t)row * N + n0 + lane + 32] = acc1[j] * scale;
      }
    }
  }
}

// ---------------------------------------------------------------------------------- top-p rows
// One CTA per row.  rows_per_head = 1: only the current query's row of every head (row 0);
// rows_per_head = S+1: every row (top-p mode).  Row 0 always publishes b_step = |C0|.
constexpr int kToppThreads = 1024;
__global__ void __launch_bounds__(kToppThreads)
topp_rows_kernel(const float* __restrict__ logits, const int32_t* __restrict__ cu, int Hq, int G, int S1,
                 int rows_per_head, float p_nuc, int include_c0, int64_t row_words, uint32_t* __restrict__ mask,
                 int32_t* __restrict__ b_step, int row_elems, const int32_t* __restrict__ kv_len) {
  extern __shared__ __align__(16) float row_sm[];
  __shared__ SelShared sh;
  const int r = blockIdx.z, g = blockIdx.y, row = blockIdx.x;   // row < rows_per_head
  const int start = cu[r], Ncap = cu[r + 1] - start;       // Ncap: rows of the slab (layout); N: rows that count
  const int N = valid_keys(kv_len, r, Hq / G, g / G, Ncap);
  if (N <= 0) { if (row == 0 && threadIdx.x == 0) b_step[r * Hq + g] = 0; return; }
  const float* Lg = logits + (int64_t)Hq * S1 * start + ((int64_t)g * S1 + row) * Ncap;
  const int tid = threadIdx.x, nthr = blockDim.x;

  // the row is staged in shared memory when it fits (eight loads in flight per thread), so the
  // passes below do not wait on global memory; the running maximum is taken on the way in
  const bool fits = N <= row_elems;
  const StoredRow L{fits ? row_sm : Lg};
  float mx = -INFINITY;
  for (int base = 0; base < N; base += nthr * 8) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int n = base + u * nthr + tid;
      v[u] = (n < N) ? Lg[n] : -INFINITY;
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int n = base + u * nthr + tid;
      if (fits && n < N) row_sm[n] = v[u];
      mx = fmaxf(mx, v[u]);
    }
  }
  mx = block_max(mx, sh.redf);      // (its barriers also publish the staged row)
  unsigned long long z = 0;
  for (int n = tid; n < N; n += nthr) z += mass_fix(L(n), mx);
  z = block_sum_u64(z, sh.red64);
  // smallest integer mass that is >= p * Z
  unsigned long long need = (unsigned long long)ceil((double)p_nuc * (double)z);
  if (need > z) need = z;
  if (need == 0) need = 1;

  uint32_t t, above_cnt, eq_cnt;
  unsigned long long above_mass;
  radix_threshold<true>(L, N, mx, need, sh, t, above_cnt, above_mass, eq_cnt);
  // every key equal to t has the same logit, hence the same mass e_t: take the fewest that reach p
  float lt;
  {
    const uint32_t u = (t & 0x80000000u) ? (t & 0x7fffffffu) : ~t;
    lt = __uint_as_float(u);
  }
  const unsigned long long e_t = mass_fix(lt, mx);
  uint32_t ties = eq_cnt;
  if (e_t > 0) {
    const unsigned long long lack = need - above_mass;             // > 0 by construction
    const unsigned long long j = (lack + e_t - 1) / e_t;
    ties = (uint32_t)(j < (unsigned long long)eq_cnt ? j : eq_cnt);
  }
  if (ties == 0) ties = 1;
  if (row == 0 && tid == 0) b_step[r * Hq + g] = (int32_t)(above_cnt + ties);
  const bool emit = (row == 0) ? (include_c0 != 0) : true;
  if (emit) {
    uint32_t* mrow = mask + (int64_t)(g / G) * row_words + mask_word_offset(start, r);
    emit_row(L, N, t, ties, eq_cnt, mrow, sh);
  }
}

// ---------------------------------------------------------------------------------- top-k rows
// One CTA per synthetic row: the b_step[g] largest logits, ties to the lower index.
__global__ void __launch_bounds__(kSelThreads)
topk_rows_kernel(const float* __restrict__ logits, const int32_t* __restrict__ cu, int Hq, int G, int S1,
                 const int32_t* __restrict__ b_step, int64_t row_words, uint32_t* __restrict__ mask,
                 const int32_t* __restrict__ kv_len) {
  __shared__ SelShared sh;
  const int r = blockIdx.z, g = blockIdx.y, row = blockIdx.x + 1;
  const int start = cu[r], Ncap = cu[r + 1] - start;       // Ncap: rows of the slab (layout); N: rows that count
  const int N = valid_keys(kv_len, r, Hq / G, g / G, Ncap);
  if (N <= 0) return;
  int k = b_step[r * Hq + g];
  if (k <= 0) return;
  if (k > N) k = N;
  const StoredRow L{logits + (int64_t)Hq * S1 * start + ((int64_t)g * S1 + row) * Ncap};
  uint32_t t, above_cnt, eq_cnt;
  unsigned long long above_mass;
  radix_threshold<false>(L, N, 0.f, (unsigned long long)k, sh, t, above_cnt, above_mass, eq_cnt);
  const uint32_t ties = (uint32_t)k - above_cnt;
  uint32_t* mrow = mask + (int64_t)(g / G) * row_words + mask_word_offset(start, r);
  emit_row(L, N, t, ties, eq_cnt, mrow, sh);
}

// ---------------------------------------------------------------------------------- softmax dump
__global__ void __launch_bounds__(kSelThreads)
softmax_dump_kernel(const float* __restrict__ logits, const int32_t* __restrict__ cu, int Hq, int S1,
                    float* __restrict__ probs) {
  __shared__ float red[kSelThreads / 32];
  __shared__ double redd[kSelThreads / 32];
  const int r = blockIdx.z, g = blockIdx.y, row = blockIdx.x;
  const int start = cu[r], N = cu[r + 1] - start;
  const int64_t off = (int64_t)Hq * S1 * start + ((int64_t)g * S1 + row) * N;
  const float* L = logits + off;
  const int tid = threadIdx.x;
  float mx = -INFINITY;
  for (int n = tid; n < N; n += kSelThreads) mx = fmaxf(mx, L[n]);
  mx = block_max(mx, red);
  double z = 0.0;
  for (int n = tid; n < N; n += kSelThreads) z += (double)expf(L[n] - mx);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
  if ((tid & 31) == 0) redd[tid >> 5] = z;
  __syncthreads();
  double zt = 0.0;
  for (int i = 0; i < kSelThreads / 32; ++i) zt += redd[i];
  const float inv = (float)(1.0 / zt);
  for (int n = tid; n < N; n += kSelThreads) probs[off + n] = expf(L[n] - mx) * inv;
}

// ---------------------------------------------------------------------------------- budgets
__global__ void __launch_bounds__(256)
budget_kernel(const uint32_t* __restrict__ mask, const int32_t* __restrict__ cu, int Hkv, int64_t row_words,
              int32_t* __restrict__ budget) {
  __shared__ uint32_t red[8];
  const int r = blockIdx.y, h = blockIdx.x;
  const int start = cu[r], N = cu[r + 1] - start;
  const int words = (N + 31) >> 5;
  const uint32_t* m = mask + (int64_t)h * row_words + mask_word_offset(start, r);
  uint32_t c = 0;
  for (int w = threadIdx.x; w < words; w += blockDim.x) c += __popc(m[w]);
  c = block_sum_u32(c, red);
  if (threadIdx.x == 0) budget[r * Hkv + h] = (int32_t)c;
}

}  // namespace

bool score_umma_supported(const gvote_params* p);
int32_t launch_score_umma(const gvote_params* p, const __nv_bfloat16* Q, const __nv_bfloat16* K, int64_t k_tok,
                          int64_t k_head, const int32_t* cu, int32_t batch, int64_t total_tokens, int64_t max_N,
                          float* logits, int32_t* status, const int32_t* kv_len, cudaStream_t st);
int32_t launch_score_sample(const gvote_params* p, const __nv_bfloat16* Q, const __nv_bfloat16* K, int64_t k_tok,
                            int64_t k_head, const int32_t* cu, int32_t batch, int64_t total_tokens, int64_t max_N,
                            float* real_logits, uint32_t* rowmax_part, int* n_part, const VoteState& vs, uint32_t* mask,
                            int64_t row_words, int32_t* status, const int32_t* kv_len, cudaStream_t st);
int32_t launch_score_sweep(const gvote_params* p, const __nv_bfloat16* Q, const __nv_bfloat16* K, int64_t k_tok,
                           int64_t k_head, const int32_t* cu, int32_t batch, int64_t total_tokens, int64_t max_N,
                           const VoteState& vs, int64_t row_words, int32_t* status, const int32_t* kv_len,
                           cudaStream_t st);
int32_t launch_bracket(const gvote_params* p, const int32_t* cu, int32_t batch, int64_t max_N, const int32_t* b_step,
                       const VoteState& vs, const int32_t* kv_len, cudaStream_t st);
int32_t launch_resolve(const gvote_params* p, const int32_t* cu, int32_t batch, int64_t max_N, const int32_t* b_step,
                       const VoteState& vs, int64_t row_words, const int32_t* kv_len, cudaStream_t st);
int32_t launch_commit(const gvote_params* p, const __nv_bfloat16* Q, const __nv_bfloat16* K, int64_t k_tok, int64_t k_head,
                      const int32_t* cu, int32_t batch, const int32_t* b_step, const VoteState& vs, int64_t row_words,
                      uint32_t* mask, const int32_t* kv_len, bool copy_good, cudaStream_t st);
int32_t launch_real_topp(const gvote_params* p, const float* logits, const int32_t* cu, int32_t batch, int64_t max_N,
                         const uint32_t* rowmax_part, int n_part, int64_t row_words, uint32_t* mask, int32_t* b_step,
                         const int32_t* kv_len, cudaStream_t st);

namespace {

int32_t launch_budget(const gvote_params* p, const uint32_t* mask, const int32_t* cu, int32_t batch, int64_t row_words,
                      int32_t* budget, cudaStream_t st) {
  dim3 gb(p->n_kv_heads, batch);
  {
    LaunchScope scope_("budget_kernel", st);
    budget_kernel<<<gb, 256, 0, st>>>(mask, cu, p->n_kv_heads, row_words, budget);
  }
  GVOTE_LAUNCH_CHECK("budget_kernel");
  return GVOTE_OK;
}

// The default route: current-query top-p and the fused top-k of the synthetic queries on the tensor
// cores; nothing of size S x N is written anywhere.  GVOTE_ERR_UNSUPPORTED_SHAPE (before anything has been
// enqueued) when no tensor map describes the operands.
int32_t vote_fused(const gvote_params* p, const __nv_bfloat16* Q, const __nv_bfloat16* K, int64_t k_tok, int64_t k_head,
                   const int32_t* cu, int32_t batch, int64_t total_tokens, int64_t max_N, uint32_t* mask,
                   int32_t* b_step, const WorkspaceMap& m, char* ws, cudaStream_t st, const int32_t* kv_len,
                   bool defer_merge) {
  VoteState vs;
  vs.sample = reinterpret_cast<uint16_t*>(ws + m.sample);
  vs.bracket = reinterpret_cast<RowBracket*>(ws + m.bracket);
  vs.segstat = reinterpret_cast<uint2*>(ws + m.segstat);
  vs.cand = reinterpret_cast<uint2*>(ws + m.cand);
  vs.tmask = reinterpret_cast<uint32_t*>(ws + m.tmask);
  vs.head_bad = reinterpret_cast<uint32_t*>(ws + m.head_bad);
  vs.status = reinterpret_cast<int32_t*>(ws + m.status);
  vs.lay = cand_layout(m.cand_segs, batch, total_tokens, max_N);
  vs.sample_slots = m.sample_slots;
  float* real_logits = reinterpret_cast<float*>(ws + m.logits);
  uint32_t* rowmax = reinterpret_cast<uint32_t*>(ws + m.rowmax);
  int32_t* status = reinterpret_cast<int32_t*>(ws + m.status);
  // (the first kernel also clears the keep mask, the tentative mask and the per-head flags)
  int n_part = 1;
  const int32_t rc = launch_score_sample(p, Q, K, k_tok, k_head, cu, batch, total_tokens, max_N, real_logits, rowmax, &n_part,
                                         vs, mask, m.row_words, status, kv_len, st);
  if (rc != GVOTE_OK) return rc;
#define GVOTE_STEP(expr) do { const int32_t rc__ = (expr); if (rc__ != GVOTE_OK) return rc__; } while (0)
  GVOTE_STEP(launch_real_topp(p, real_logits, cu, batch, max_N, rowmax, n_part, m.row_words, mask, b_step, kv_len, st));
  GVOTE_STEP(launch_bracket(p, cu, batch, max_N, b_step, vs, kv_len, st));
  GVOTE_STEP(launch_score_sweep(p, Q, K, k_tok, k_head, cu, batch, total_tokens, max_N, vs, m.row_words, status, kv_len,
                                st));
  GVOTE_STEP(launch_resolve(p, cu, batch, max_N, b_step, vs, m.row_words, kv_len, st));
  GVOTE_STEP(launch_commit(p, Q, K, k_tok, k_head, cu, batch, b_step, vs, m.row_words, mask, kv_len, !defer_merge, st));
#undef GVOTE_STEP
  return GVOTE_OK;
}

}  // namespace

int32_t launch_vote(const gvote_params* p, const __nv_bfloat16* Q, const __nv_bfloat16* K, int64_t k_tok,
                    int64_t k_head, const int32_t* cu, int32_t batch, int64_t total_tokens, int64_t max_N,
                    uint32_t* mask, int32_t* budget, int32_t* b_step, float* dbg_probs, char* ws, size_t ws_bytes,
                    cudaStream_t st, const int32_t* kv_len, bool* merge_deferred) {
  const int Hq = p->n_q_heads, Hkv = p->n_kv_heads, G = Hq / Hkv, S1 = p->S + 1, d_k = p->d_k;
  const bool defer = merge_deferred != nullptr;
  if (merge_deferred) *merge_deferred = false;
  const float scale = (float)(1.0 / sqrt((double)d_k));

  if (!vote_needs_full_rows(p) && dbg_probs == nullptr && max_N > 0) {
    const WorkspaceMap m = workspace_map(p, batch, total_tokens, max_N, false);
    const int32_t rc = vote_fused(p, Q, K, k_tok, k_head, cu, batch, total_tokens, max_N, mask, b_step, m, ws, st, kv_len,
                                  defer);
    if (rc == GVOTE_OK) {
      if (merge_deferred) *merge_deferred = true;
      // (a caller that defers the merge takes its budgets from the scan that does it)
      return (budget && !defer) ? launch_budget(p, mask, cu, batch, m.row_words, budget, st) : GVOTE_OK;
    }
    if (rc != GVOTE_ERR_UNSUPPORTED_SHAPE) return rc;
    // operands no tensor map describes: the route below, if the workspace has room for its fp32 rows
  }

  // fp32 logits of every row: the per-sample top-p mode, the softmax dump, shapes the tensor-core kernels
  // do not take.  On the tensor cores when possible, else SIMT.
  const WorkspaceMap m = workspace_map(p, batch, total_tokens, max_N, true);
  if (ws_bytes < m.total) return vote_needs_full_rows(p) || dbg_probs ? GVOTE_ERR_WORKSPACE_TOO_SMALL : GVOTE_ERR_UNSUPPORTED_SHAPE;
  float* logits = reinterpret_cast<float*>(ws + m.logits);
  int32_t* status = reinterpret_cast<int32_t*>(ws + m.status);
  GVOTE_CUDA_CHECK(cudaMemsetAsync(mask, 0, (size_t)Hkv * m.row_words * sizeof(uint32_t), st));
  bool tensor_path = false;
  if (score_umma_supported(p) && max_N > 0) {
    const int32_t rc = launch_score_umma(p, Q, K, k_tok, k_head, cu, batch, total_tokens, max_N, logits, status, kv_len, st);
    if (rc == GVOTE_OK) tensor_path = true;
    else if (rc != GVOTE_ERR_UNSUPPORTED_SHAPE) return rc;
  }
  if (!tensor_path) {
    const int half = d_k / 2;
    const size_t smem = ((size_t)kScoreKeys * (half + 1) + (size_t)kScoreRowChunk * half) * sizeof(uint32_t);
    if (smem > 48 * 1024) {
      GVOTE_CUDA_CHECK(cudaFuncSetAttribute(score_simt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    }
    dim3 grid((unsigned)ceil_div(max_N > 0 ? max_N : 1, kScoreKeys), Hkv, batch);
    {
      LaunchScope scope_("score_simt_kernel", st);
      score_simt_kernel<<<grid, 256, smem, st>>>(Q, K, k_tok, k_head, cu, Hq, G, S1, d_k, scale, logits);
    }
    GVOTE_LAUNCH_CHECK("score_simt_kernel");
  }
  if (dbg_probs) {
    dim3 grid(S1, Hq, batch);
    {
      LaunchScope scope_("softmax_dump_kernel", st);
      softmax_dump_kernel<<<grid, kSelThreads, 0, st>>>(logits, cu, Hq, S1, dbg_probs);
    }
    GVOTE_LAUNCH_CHECK("softmax_dump_kernel");
  }
  // top-p rows up to 48K keys are staged in shared memory (192 KB)
  int topp_row_elems = (int)max_N;
  if (topp_row_elems > 48 * 1024) topp_row_elems = 0;
  const size_t topp_smem = (size_t)topp_row_elems * sizeof(float);
  if (topp_smem > 16 * 1024)
    GVOTE_CUDA_CHECK(cudaFuncSetAttribute(topp_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)topp_smem));
  const bool topk = p->sel_mode == GVOTE_SEL_TOPK_C0;
  dim3 g1(topk ? 1 : S1, Hq, batch);
  {
    LaunchScope scope_("topp_rows_kernel", st);
    topp_rows_kernel<<<g1, kToppThreads, topp_smem, st>>>(logits, cu, Hq, G, S1, topk ? 1 : S1, p->p_nuc, p->include_c0,
                                                          m.row_words, mask, b_step, topp_row_elems, kv_len);
  }
  GVOTE_LAUNCH_CHECK("topp_rows_kernel");
  if (topk) {
    dim3 g2(p->S, Hq, batch);
    {
      LaunchScope scope_("topk_rows_kernel", st);
      topk_rows_kernel<<<g2, kSelThreads, 0, st>>>(logits, cu, Hq, G, S1, b_step, m.row_words, mask, kv_len);
    }
    GVOTE_LAUNCH_CHECK("topk_rows_kernel");
  }
  return budget ? launch_budget(p, mask, cu, batch, m.row_words, budget, st) : GVOTE_OK;
}

}  // namespace gvote
