// C-ABI entry points of the GVote library (declared in include/gvote.h): argument checks, the
// workspace map, the per-stage wrappers, the whole-pass call and its host-memory variant.
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <string>
#include <vector>

#include "common.cuh"
#include "vote_geom.cuh"

namespace gvote {

static thread_local char g_cuda_err[512] = "";
static std::atomic<long long> g_launches{0};

void set_cuda_error(cudaError_t e, const char* where) {
  snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s (%s)", where, cudaGetErrorName(e), cudaGetErrorString(e));
}
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// ---------------------------------------------------------------------------------- per-kernel timing
namespace {
struct ProfRec { const char* name; cudaEvent_t a, b; };
std::mutex g_prof_mu;
std::atomic<bool> g_prof_on{false};
std::vector<ProfRec> g_prof_recs;
std::vector<cudaEvent_t> g_prof_pool;

cudaEvent_t prof_event() {
  if (!g_prof_pool.empty()) { cudaEvent_t e = g_prof_pool.back(); g_prof_pool.pop_back(); return e; }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}
}  // namespace

LaunchScope::LaunchScope(const char* name, cudaStream_t stream) : slot(-1), st(stream) {
  if (!g_prof_on.load(std::memory_order_relaxed)) return;
  std::lock_guard<std::mutex> lk(g_prof_mu);
  ProfRec r{name, prof_event(), prof_event()};
  if (!r.a || !r.b) return;
  cudaEventRecord(r.a, st);
  slot = (int)g_prof_recs.size();
  g_prof_recs.push_back(r);
}
LaunchScope::~LaunchScope() {
  if (slot < 0) return;
  std::lock_guard<std::mutex> lk(g_prof_mu);
  cudaEventRecord(g_prof_recs[slot].b, st);
}

int32_t validate_params(const gvote_params* p) {
  if (!p) return GVOTE_ERR_INVALID_ARG;
  if (p->d_h <= 0 || p->n_q_heads <= 0 || p->n_kv_heads <= 0 || p->d_k <= 0) return GVOTE_ERR_INVALID_ARG;
  if (p->n_q_heads % p->n_kv_heads != 0) return GVOTE_ERR_INVALID_ARG;
  if (p->S < 1 || p->n_f < 1 || p->n_s < 0) return GVOTE_ERR_INVALID_ARG;
  if (!(p->p_nuc > 0.f) || !(p->p_nuc <= 1.f)) return GVOTE_ERR_INVALID_ARG;
  if (!(p->rope_theta > 1.0)) return GVOTE_ERR_INVALID_ARG;
  if (p->sel_mode != GVOTE_SEL_TOPK_C0 && p->sel_mode != GVOTE_SEL_TOPP) return GVOTE_ERR_INVALID_ARG;
  if (p->h_dtype != GVOTE_DTYPE_F32 && p->h_dtype != GVOTE_DTYPE_BF16) return GVOTE_ERR_INVALID_ARG;
  if (p->d_h % 8 != 0 || p->d_k % 8 != 0) return GVOTE_ERR_UNSUPPORTED_SHAPE;
  if (p->d_k > 512 || p->S > 4096) return GVOTE_ERR_UNSUPPORTED_SHAPE;
  return GVOTE_OK;
}

static int32_t validate_batch(int32_t batch, int64_t total_tokens, int64_t max_N) {
  if (batch < 1 || total_tokens < 0 || max_N < 0 || max_N > total_tokens) return GVOTE_ERR_INVALID_ARG;
  if (total_tokens > (int64_t)1 << 30) return GVOTE_ERR_UNSUPPORTED_SHAPE;
  return GVOTE_OK;
}

bool vote_needs_full_rows(const gvote_params* p) {
  return p->sel_mode != GVOTE_SEL_TOPK_C0 || !sweep_umma_supported(p);
}

WorkspaceMap workspace_map(const gvote_params* p, int32_t batch, int64_t total_tokens, int64_t max_N,
                           bool full_rows) {
  WorkspaceMap m;
  memset(&m, 0, sizeof(m));
  const int64_t S1 = p->S + 1, F = (int64_t)p->n_q_heads * p->d_k;
  const int64_t chunks = fit_chunk_count(p, batch, max_N);
  m.fit_chunks = (int)chunks;
  m.proj_splits = project_umma_splits(p, batch * (p->S + 1));
  m.n_tiles = (total_tokens >> 7) + batch;
  m.row_words = gvote_mask_row_words(total_tokens, batch);
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  m.status = take(kStatusBytes);
  m.fit_partial = take((size_t)batch * chunks * p->d_h * sizeof(float2));
  m.mu = take((size_t)batch * p->d_h * sizeof(float));
  m.var = take((size_t)batch * p->d_h * sizeof(float));
  m.h_tilde = take((size_t)batch * p->S * p->d_h * sizeof(float));
  m.x_bf16 = take((size_t)batch * S1 * p->d_h * sizeof(__nv_bfloat16));
  m.q_f32 = take((size_t)m.proj_splits * batch * S1 * F * sizeof(float));
  m.q_bf16 = take((size_t)batch * S1 * F * sizeof(__nv_bfloat16));
  m.rope = take((size_t)batch * 4 * (p->d_k / 2) * sizeof(float));
  m.full_rows = full_rows;
  m.logits = take((size_t)p->n_q_heads * (full_rows ? S1 : 1) * (size_t)total_tokens * sizeof(float));
  if (!full_rows) {
    const size_t rows = (size_t)batch * p->n_q_heads * p->S;
    m.cand_segs = 4 * sweep_geometry(p, batch, max_N).X;
    m.cand_strip = cand_layout(m.cand_segs, batch, total_tokens, max_N).strip;
    m.sample_slots = sample_slots_total(batch, total_tokens, max_N);
    m.tmask = take((size_t)p->n_kv_heads * m.row_words * sizeof(uint32_t));
    m.head_bad = take((size_t)batch * p->n_kv_heads * sizeof(uint32_t));
    m.rowmax = take((size_t)batch * p->n_q_heads * 148 * sizeof(uint32_t));
    m.sample = take((size_t)p->n_kv_heads * m.sample_slots * score_geometry(p).row_chunks * kVoteRowChunk *
                    kVoteTileKeys * sizeof(uint16_t));
    m.bracket = take(rows * sizeof(RowBracket));
    m.segstat = take(rows * (size_t)m.cand_segs * sizeof(uint2));
    m.cand = take((size_t)p->n_q_heads * p->S * (size_t)m.cand_strip * sizeof(uint2));
  }
  m.remap_tmp = take((size_t)p->n_kv_heads * (size_t)total_tokens * sizeof(int32_t));
  m.ov_partial = take((size_t)batch * p->n_q_heads * (size_t)ceil_div(max_N > 0 ? max_N : 1, kOverlapKeys) * 16);
  m.prefix = take((size_t)p->n_kv_heads * m.row_words * sizeof(int32_t));
  m.flags = take(((size_t)2 * p->n_kv_heads * m.n_tiles + (size_t)2 * p->n_kv_heads * 32) * sizeof(int32_t));
  m.total = off;
  return m;
}

}  // namespace gvote

using namespace gvote;

#define REQUIRE_PTR(x) do { if (!(x)) return GVOTE_ERR_INVALID_ARG; if (!aligned16(x)) return GVOTE_ERR_UNALIGNED; } while (0)
#define OPTIONAL_PTR(x) do { if ((x) && !aligned16(x)) return GVOTE_ERR_UNALIGNED; } while (0)
#define PROPAGATE(expr) do { int32_t s__ = (expr); if (s__ != GVOTE_OK) return s__; } while (0)

extern "C" {

size_t gvote_workspace_bytes(const gvote_params* p, int32_t batch, int64_t total_tokens, int64_t max_N) {
  if (validate_params(p) != GVOTE_OK || validate_batch(batch, total_tokens, max_N) != GVOTE_OK) return 0;
  return workspace_map(p, batch, total_tokens, max_N).total;
}

size_t gvote_workspace_queries(const gvote_params* p, int32_t batch, int64_t total_tokens, int64_t max_N) {
  if (validate_params(p) != GVOTE_OK || validate_batch(batch, total_tokens, max_N) != GVOTE_OK) return 0;
  return workspace_map(p, batch, total_tokens, max_N).q_bf16;
}

int32_t gvote_fit(const gvote_params* p, const void* h, int64_t h_row_stride, const int32_t* cu_seqlens,
                  int32_t batch, int64_t total_tokens, int64_t max_N, float* mu, float* var, void* ws,
                  size_t ws_bytes, void* stream) {
  PROPAGATE(validate_params(p));
  PROPAGATE(validate_batch(batch, total_tokens, max_N));
  REQUIRE_PTR(h); REQUIRE_PTR(cu_seqlens); REQUIRE_PTR(mu); REQUIRE_PTR(var); REQUIRE_PTR(ws);
  if (h_row_stride < p->d_h || h_row_stride % 8 != 0) return GVOTE_ERR_UNALIGNED;
  if (max_N - p->n_s < 2) return GVOTE_ERR_INVALID_ARG;
  const WorkspaceMap m = workspace_map(p, batch, total_tokens, max_N);
  if (ws_bytes < m.total) return GVOTE_ERR_WORKSPACE_TOO_SMALL;
  return launch_fit(p, h, h_row_stride, cu_seqlens, batch, total_tokens, m.fit_chunks,
                    reinterpret_cast<float2*>((char*)ws + m.fit_partial), reinterpret_cast<int32_t*>((char*)ws + m.status),
                    mu, var, (cudaStream_t)stream);
}

int32_t gvote_sample(const gvote_params* p, const float* mu, const float* var, int32_t batch, float* H_tilde,
                     uint32_t* raw_u32_or_null, void* stream) {
  PROPAGATE(validate_params(p));
  if (batch < 1) return GVOTE_ERR_INVALID_ARG;
  REQUIRE_PTR(mu); REQUIRE_PTR(var); REQUIRE_PTR(H_tilde); OPTIONAL_PTR(raw_u32_or_null);
  return launch_sample(p, mu, var, batch, H_tilde, raw_u32_or_null, (cudaStream_t)stream);
}

int32_t gvote_project(const gvote_params* p, const float* H_tilde, const void* h_last, const void* W_q,
                      int64_t wq_ld, const float* b_q_or_null, const int32_t* cu_seqlens, int32_t batch, void* Q,
                      void* ws, size_t ws_bytes, void* stream) {
  PROPAGATE(validate_params(p));
  if (batch < 1) return GVOTE_ERR_INVALID_ARG;
  REQUIRE_PTR(H_tilde); REQUIRE_PTR(h_last); REQUIRE_PTR(W_q); OPTIONAL_PTR(b_q_or_null);
  REQUIRE_PTR(cu_seqlens); REQUIRE_PTR(Q); REQUIRE_PTR(ws);
  if (wq_ld < p->d_h || wq_ld % 8 != 0) return GVOTE_ERR_UNALIGNED;
  // the projection's scratch does not depend on the token counts
  const WorkspaceMap m = workspace_map(p, batch, 0, 0);
  if (ws_bytes < m.logits) return GVOTE_ERR_WORKSPACE_TOO_SMALL;      // the areas up to the vote's
  return launch_project(p, H_tilde, h_last, p->d_h, nullptr, W_q, wq_ld, b_q_or_null, cu_seqlens, batch, m,
                        (char*)ws, (__nv_bfloat16*)Q, (cudaStream_t)stream);
}

int32_t gvote_vote(const gvote_params* p, const void* Q, const void* K, int64_t k_tok_stride, int64_t k_head_stride,
                   const int32_t* cu_seqlens, int32_t batch, int64_t total_tokens, int64_t max_N, uint32_t* mask,
                   int32_t* budget, int32_t* b_step, float* dbg_probs_or_null, void* ws, size_t ws_bytes,
                   void* stream) {
  PROPAGATE(validate_params(p));
  PROPAGATE(validate_batch(batch, total_tokens, max_N));
  REQUIRE_PTR(Q); REQUIRE_PTR(K); REQUIRE_PTR(cu_seqlens); REQUIRE_PTR(mask); REQUIRE_PTR(budget);
  REQUIRE_PTR(b_step); OPTIONAL_PTR(dbg_probs_or_null); REQUIRE_PTR(ws);
  if (k_tok_stride < p->d_k || k_tok_stride % 8 != 0 || k_head_stride % 8 != 0) return GVOTE_ERR_UNALIGNED;
  // the softmax dump needs the fp32 logits of every row: the workspace of the per-sample top-p mode
  const WorkspaceMap m = workspace_map(p, batch, total_tokens, max_N, vote_needs_full_rows(p) || dbg_probs_or_null);
  if (ws_bytes < m.total) return GVOTE_ERR_WORKSPACE_TOO_SMALL;
  return launch_vote(p, (const __nv_bfloat16*)Q, (const __nv_bfloat16*)K, k_tok_stride, k_head_stride, cu_seqlens,
                     batch, total_tokens, max_N, mask, budget, b_step, dbg_probs_or_null, (char*)ws, ws_bytes,
                     (cudaStream_t)stream);
}

int32_t gvote_select(const gvote_params* p, const float* H_tilde, const void* h_last, const void* W_q, int64_t wq_ld,
                     const float* b_q_or_null, const void* K, int64_t k_tok_stride, int64_t k_head_stride,
                     const int32_t* cu_seqlens, int32_t batch, int64_t total_tokens, int64_t max_N, uint32_t* mask,
                     int32_t* budget, int32_t* b_step, float* dbg_probs_or_null, void* ws, size_t ws_bytes,
                     void* stream) {
  PROPAGATE(validate_params(p));
  PROPAGATE(validate_batch(batch, total_tokens, max_N));
  REQUIRE_PTR(H_tilde); REQUIRE_PTR(h_last); REQUIRE_PTR(W_q); OPTIONAL_PTR(b_q_or_null); REQUIRE_PTR(K);
  REQUIRE_PTR(cu_seqlens); REQUIRE_PTR(mask); REQUIRE_PTR(budget); REQUIRE_PTR(b_step);
  OPTIONAL_PTR(dbg_probs_or_null); REQUIRE_PTR(ws);
  if (wq_ld < p->d_h || wq_ld % 8 != 0) return GVOTE_ERR_UNALIGNED;
  if (k_tok_stride < p->d_k || k_tok_stride % 8 != 0 || k_head_stride % 8 != 0) return GVOTE_ERR_UNALIGNED;
  const WorkspaceMap m = workspace_map(p, batch, total_tokens, max_N, vote_needs_full_rows(p) || dbg_probs_or_null);
  if (ws_bytes < m.total) return GVOTE_ERR_WORKSPACE_TOO_SMALL;
  __nv_bfloat16* Q = reinterpret_cast<__nv_bfloat16*>((char*)ws + m.q_bf16);
  PROPAGATE(launch_project(p, H_tilde, h_last, p->d_h, nullptr, W_q, wq_ld, b_q_or_null, cu_seqlens, batch, m,
                           (char*)ws, Q, (cudaStream_t)stream));
  return launch_vote(p, Q, (const __nv_bfloat16*)K, k_tok_stride, k_head_stride, cu_seqlens, batch, total_tokens,
                     max_N, mask, budget, b_step, dbg_probs_or_null, (char*)ws, ws_bytes, (cudaStream_t)stream);
}

int32_t gvote_compact(const gvote_params* p, void* K, void* V, int64_t tok_stride, int64_t head_stride,
                      const uint32_t* mask, const int32_t* cu_seqlens, int32_t batch, int64_t total_tokens,
                      int64_t max_N, int32_t* budget, void* ws, size_t ws_bytes, void* stream) {
  PROPAGATE(validate_params(p));
  PROPAGATE(validate_batch(batch, total_tokens, max_N));
  REQUIRE_PTR(K); REQUIRE_PTR(V); REQUIRE_PTR(mask); REQUIRE_PTR(cu_seqlens); REQUIRE_PTR(budget); REQUIRE_PTR(ws);
  if (tok_stride < p->d_k || tok_stride % 8 != 0 || head_stride % 8 != 0) return GVOTE_ERR_UNALIGNED;
  const WorkspaceMap m = workspace_map(p, batch, total_tokens, max_N);
  if (ws_bytes < m.total) return GVOTE_ERR_WORKSPACE_TOO_SMALL;
  return launch_compact(p, (__nv_bfloat16*)K, (__nv_bfloat16*)V, tok_stride, head_stride, mask, cu_seqlens, batch,
                        total_tokens, max_N, budget, m, (char*)ws, (cudaStream_t)stream);
}

int32_t gvote_fit_update(const gvote_params* p, const void* h_block, int64_t h_row_stride,
                         const int32_t* cu_block, int32_t batch, int64_t total_rows, int64_t max_rows, double* state,
                         void* ws, size_t ws_bytes, void* stream) {
  PROPAGATE(validate_params(p));
  PROPAGATE(validate_batch(batch, total_rows, max_rows));
  REQUIRE_PTR(h_block); REQUIRE_PTR(cu_block); REQUIRE_PTR(state); REQUIRE_PTR(ws);
  if (h_row_stride < p->d_h || h_row_stride % 8 != 0) return GVOTE_ERR_UNALIGNED;
  const WorkspaceMap m = workspace_map(p, batch, total_rows, max_rows);
  if (ws_bytes < m.total) return GVOTE_ERR_WORKSPACE_TOO_SMALL;
  return launch_fit_state_update(p, h_block, h_row_stride, cu_block, batch, total_rows, m.fit_chunks,
                                 reinterpret_cast<float2*>((char*)ws + m.fit_partial),
                                 reinterpret_cast<int32_t*>((char*)ws + m.status), state, (cudaStream_t)stream);
}

int32_t gvote_fit_finish(const gvote_params* p, const double* state, int32_t batch, float* mu, float* var,
                         void* stream) {
  PROPAGATE(validate_params(p));
  if (batch < 1) return GVOTE_ERR_INVALID_ARG;
  REQUIRE_PTR(state); REQUIRE_PTR(mu); REQUIRE_PTR(var);
  return launch_fit_state_finish(p, state, batch, mu, var, (cudaStream_t)stream);
}

namespace {
// The pass from the sampling step of Algorithm 1 on, from fitted moments; kv_len / seq_len / token_pos are the extras of the
// re-application (all null for a cache that has not been pruned before).
int32_t compress_from_moments(const gvote_params* p, const float* mu, const float* var, const void* h_last,
                              const void* W_q, int64_t wq_ld, const float* b_q_or_null, void* K, void* V,
                              int64_t tok_stride, int64_t head_stride, const int32_t* cu_seqlens,
                              const int32_t* kv_len, const int32_t* seq_len, int32_t* token_pos, int32_t batch,
                              int64_t total_tokens, int64_t max_N, uint32_t* mask, int32_t* budget, int32_t* b_step,
                              void* ws, size_t ws_bytes, void* stream) {
  PROPAGATE(validate_params(p));
  PROPAGATE(validate_batch(batch, total_tokens, max_N));
  REQUIRE_PTR(mu); REQUIRE_PTR(var); REQUIRE_PTR(h_last); REQUIRE_PTR(W_q); OPTIONAL_PTR(b_q_or_null); REQUIRE_PTR(K);
  REQUIRE_PTR(V); REQUIRE_PTR(cu_seqlens); REQUIRE_PTR(mask); REQUIRE_PTR(budget); REQUIRE_PTR(b_step);
  REQUIRE_PTR(ws);
  if (wq_ld < p->d_h || wq_ld % 8 != 0) return GVOTE_ERR_UNALIGNED;
  if (tok_stride < p->d_k || tok_stride % 8 != 0 || head_stride % 8 != 0) return GVOTE_ERR_UNALIGNED;
  const WorkspaceMap m = workspace_map(p, batch, total_tokens, max_N);
  if (ws_bytes < m.total) return GVOTE_ERR_WORKSPACE_TOO_SMALL;
  char* w = (char*)ws;
  cudaStream_t st = (cudaStream_t)stream;
  float* Ht = reinterpret_cast<float*>(w + m.h_tilde);
  __nv_bfloat16* Q = reinterpret_cast<__nv_bfloat16*>(w + m.q_bf16);
  PROPAGATE(launch_sample(p, mu, var, batch, Ht, nullptr, st));
  PROPAGATE(launch_project(p, Ht, h_last, p->d_h, nullptr, W_q, wq_ld, b_q_or_null, cu_seqlens, batch, m, w, Q, st,
                           seq_len));
  bool merge_deferred = false;   // whether the settled heads' union still waits in the tentative mask
  PROPAGATE(launch_vote(p, Q, (const __nv_bfloat16*)K, tok_stride, head_stride, cu_seqlens, batch, total_tokens,
                        max_N, mask, nullptr, b_step, nullptr, w, ws_bytes, st, kv_len, &merge_deferred));
  PROPAGATE(launch_compact(p, (__nv_bfloat16*)K, (__nv_bfloat16*)V, tok_stride, head_stride, mask, cu_seqlens, batch,
                           total_tokens, max_N, budget, m, w, st, merge_deferred));
  if (token_pos) PROPAGATE(launch_remap(p, token_pos, mask, cu_seqlens, batch, total_tokens, max_N, budget, m, w, st));
  return GVOTE_OK;
}
}  // namespace

int32_t gvote_compress_moments(const gvote_params* p, const float* mu, const float* var, const void* h_last,
                               const void* W_q, int64_t wq_ld, const float* b_q_or_null, void* K, void* V,
                               int64_t tok_stride, int64_t head_stride, const int32_t* cu_seqlens, int32_t batch,
                               int64_t total_tokens, int64_t max_N, uint32_t* mask, int32_t* budget, int32_t* b_step,
                               void* ws, size_t ws_bytes, void* stream) {
  return compress_from_moments(p, mu, var, h_last, W_q, wq_ld, b_q_or_null, K, V, tok_stride, head_stride, cu_seqlens,
                               nullptr, nullptr, nullptr, batch, total_tokens, max_N, mask, budget, b_step, ws,
                               ws_bytes, stream);
}

int32_t gvote_recompress(const gvote_params* p, const float* mu, const float* var, const void* h_last,
                         const void* W_q, int64_t wq_ld, const float* b_q_or_null, void* K, void* V,
                         int64_t tok_stride, int64_t head_stride, const int32_t* cu_seqlens, const int32_t* kv_len,
                         const int32_t* seq_len, int32_t* token_pos_or_null, int32_t batch, int64_t total_tokens,
                         int64_t max_N, uint32_t* mask, int32_t* budget, int32_t* b_step, void* ws, size_t ws_bytes,
                         void* stream) {
  REQUIRE_PTR(kv_len); REQUIRE_PTR(seq_len); OPTIONAL_PTR(token_pos_or_null);
  return compress_from_moments(p, mu, var, h_last, W_q, wq_ld, b_q_or_null, K, V, tok_stride, head_stride, cu_seqlens,
                               kv_len, seq_len, token_pos_or_null, batch, total_tokens, max_N, mask, budget, b_step, ws,
                               ws_bytes, stream);
}

int32_t gvote_overlap(const gvote_params* p, const void* Q, const void* K, int64_t k_tok_stride, int64_t k_head_stride,
                      const uint32_t* mask, const int32_t* cu_seqlens, int32_t batch, int64_t total_tokens,
                      int64_t max_N, float* overlap, void* ws, size_t ws_bytes, void* stream) {
  PROPAGATE(validate_params(p));
  PROPAGATE(validate_batch(batch, total_tokens, max_N));
  REQUIRE_PTR(Q); REQUIRE_PTR(K); REQUIRE_PTR(mask); REQUIRE_PTR(cu_seqlens); REQUIRE_PTR(overlap); REQUIRE_PTR(ws);
  if (k_tok_stride < p->d_k || k_tok_stride % 8 != 0 || k_head_stride % 8 != 0) return GVOTE_ERR_UNALIGNED;
  const WorkspaceMap m = workspace_map(p, batch, total_tokens, max_N);
  if (ws_bytes < m.total) return GVOTE_ERR_WORKSPACE_TOO_SMALL;
  return launch_overlap(p, (const __nv_bfloat16*)Q, (const __nv_bfloat16*)K, k_tok_stride, k_head_stride, mask,
                        cu_seqlens, batch, max_N, overlap, m, (char*)ws, (cudaStream_t)stream);
}

int32_t gvote_pack(const gvote_params* p, const void* K, const void* V, int64_t tok_stride, int64_t head_stride,
                   const uint32_t* mask, const int32_t* cu_seqlens, int32_t batch, int64_t total_tokens, int64_t max_N,
                   void* K_packed, void* V_packed, int64_t capacity_rows, int32_t* cu_seqlens_k, int32_t* budget,
                   void* ws, size_t ws_bytes, void* stream) {
  PROPAGATE(validate_params(p));
  PROPAGATE(validate_batch(batch, total_tokens, max_N));
  REQUIRE_PTR(K); REQUIRE_PTR(V); REQUIRE_PTR(mask); REQUIRE_PTR(cu_seqlens); REQUIRE_PTR(K_packed);
  REQUIRE_PTR(V_packed); REQUIRE_PTR(cu_seqlens_k); REQUIRE_PTR(budget); REQUIRE_PTR(ws);
  if (tok_stride < p->d_k || tok_stride % 8 != 0 || head_stride % 8 != 0) return GVOTE_ERR_UNALIGNED;
  if (capacity_rows < 0) return GVOTE_ERR_INVALID_ARG;
  const WorkspaceMap m = workspace_map(p, batch, total_tokens, max_N);
  if (ws_bytes < m.total) return GVOTE_ERR_WORKSPACE_TOO_SMALL;
  return launch_pack(p, (const __nv_bfloat16*)K, (const __nv_bfloat16*)V, tok_stride, head_stride, mask, cu_seqlens,
                     batch, total_tokens, max_N, (__nv_bfloat16*)K_packed, (__nv_bfloat16*)V_packed, capacity_rows,
                     cu_seqlens_k, budget, m, (char*)ws, (cudaStream_t)stream);
}

int32_t gvote_compress(const gvote_params* p, const void* h, int64_t h_row_stride, const void* h_last_or_null,
                       const void* W_q, int64_t wq_ld, const float* b_q_or_null, void* K, void* V,
                       int64_t tok_stride, int64_t head_stride, const int32_t* cu_seqlens, int32_t batch,
                       int64_t total_tokens, int64_t max_N, uint32_t* mask, int32_t* budget, int32_t* b_step,
                       void* ws, size_t ws_bytes, void* stream) {
  PROPAGATE(validate_params(p));
  PROPAGATE(validate_batch(batch, total_tokens, max_N));
  REQUIRE_PTR(h); OPTIONAL_PTR(h_last_or_null); REQUIRE_PTR(W_q); OPTIONAL_PTR(b_q_or_null); REQUIRE_PTR(K);
  REQUIRE_PTR(V); REQUIRE_PTR(cu_seqlens); REQUIRE_PTR(mask); REQUIRE_PTR(budget); REQUIRE_PTR(b_step);
  REQUIRE_PTR(ws);
  if (h_row_stride < p->d_h || h_row_stride % 8 != 0) return GVOTE_ERR_UNALIGNED;
  if (wq_ld < p->d_h || wq_ld % 8 != 0) return GVOTE_ERR_UNALIGNED;
  if (tok_stride < p->d_k || tok_stride % 8 != 0 || head_stride % 8 != 0) return GVOTE_ERR_UNALIGNED;
  if (max_N - p->n_s < 2) return GVOTE_ERR_INVALID_ARG;
  const WorkspaceMap m = workspace_map(p, batch, total_tokens, max_N);
  if (ws_bytes < m.total) return GVOTE_ERR_WORKSPACE_TOO_SMALL;
  char* w = (char*)ws;
  cudaStream_t st = (cudaStream_t)stream;
  float* mu = reinterpret_cast<float*>(w + m.mu);
  float* var = reinterpret_cast<float*>(w + m.var);
  __nv_bfloat16* Q = reinterpret_cast<__nv_bfloat16*>(w + m.q_bf16);
  PROPAGATE(launch_fit_partial(p, h, h_row_stride, cu_seqlens, batch, total_tokens, m.fit_chunks,
                               reinterpret_cast<float2*>(w + m.fit_partial), reinterpret_cast<int32_t*>(w + m.status), st));
  __nv_bfloat16* X = reinterpret_cast<__nv_bfloat16*>(w + m.x_bf16);
  float* rope = reinterpret_cast<float*>(w + m.rope);
  if (h_last_or_null)
    PROPAGATE(launch_prep(p, reinterpret_cast<const float2*>(w + m.fit_partial), m.fit_chunks, h_last_or_null, p->d_h,
                          nullptr, cu_seqlens, batch, mu, var, X, rope, st));
  else
    PROPAGATE(launch_prep(p, reinterpret_cast<const float2*>(w + m.fit_partial), m.fit_chunks, h, h_row_stride,
                          cu_seqlens, cu_seqlens, batch, mu, var, X, rope, st));
  PROPAGATE(launch_project_staged(p, X, rope, W_q, wq_ld, b_q_or_null, batch, m, w, Q, st));
  bool merge_deferred = false;   // whether the settled heads' union still waits in the tentative mask
  PROPAGATE(launch_vote(p, Q, (const __nv_bfloat16*)K, tok_stride, head_stride, cu_seqlens, batch, total_tokens,
                        max_N, mask, nullptr, b_step, nullptr, w, ws_bytes, st, nullptr, &merge_deferred));
  return launch_compact(p, (__nv_bfloat16*)K, (__nv_bfloat16*)V, tok_stride, head_stride, mask, cu_seqlens, batch,
                        total_tokens, max_N, budget, m, w, st, merge_deferred);   // (budgets come from its scan)
}

// ------------------------------------------------------------------------------------ host variant
namespace {
struct HostArena {
  std::mutex mu;
  int device = -1;
  char* base = nullptr;
  size_t cap = 0;
  cudaStream_t stream = nullptr;
};
HostArena g_arena;
}  // namespace

void gvote_host_arena_release(void) {
  std::lock_guard<std::mutex> lk(g_arena.mu);
  if (g_arena.base) cudaFree(g_arena.base);
  if (g_arena.stream) cudaStreamDestroy(g_arena.stream);
  g_arena.base = nullptr; g_arena.cap = 0; g_arena.stream = nullptr; g_arena.device = -1;
}

int32_t gvote_compress_host(const gvote_params* p, const void* h, const void* W_q, const float* b_q_or_null,
                            void* K, void* V, const int32_t* cu_seqlens_host, int32_t batch, uint32_t* mask,
                            int32_t* budget, int32_t* b_step) {
  PROPAGATE(validate_params(p));
  if (batch < 1 || !h || !W_q || !K || !V || !cu_seqlens_host || !mask || !budget || !b_step)
    return GVOTE_ERR_INVALID_ARG;
  int64_t total = cu_seqlens_host[batch], max_N = 0;
  for (int r = 0; r < batch; ++r) {
    const int64_t n = (int64_t)cu_seqlens_host[r + 1] - cu_seqlens_host[r];
    if (n - p->n_s < 2) return GVOTE_ERR_INVALID_ARG;
    if (n > max_N) max_N = n;
  }
  PROPAGATE(validate_batch(batch, total, max_N));
  const WorkspaceMap m = workspace_map(p, batch, total, max_N);
  const size_t esz = p->h_dtype == GVOTE_DTYPE_F32 ? 4 : 2;
  const size_t F = (size_t)p->n_q_heads * p->d_k;
  const size_t b_h = (size_t)total * p->d_h * esz, b_w = F * p->d_h * 2, b_b = b_q_or_null ? F * 4 : 0;
  const size_t b_kv = (size_t)p->n_kv_heads * total * p->d_k * 2, b_cu = (size_t)(batch + 1) * 4;
  const size_t b_mask = (size_t)p->n_kv_heads * m.row_words * 4, b_bud = (size_t)batch * p->n_kv_heads * 4;
  const size_t b_bs = (size_t)batch * p->n_q_heads * 4;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const size_t o_ws = take(m.total), o_h = take(b_h), o_w = take(b_w), o_b = take(b_b ? b_b : 16), o_k = take(b_kv),
               o_v = take(b_kv), o_cu = take(b_cu), o_mask = take(b_mask), o_bud = take(b_bud), o_bs = take(b_bs);

  std::lock_guard<std::mutex> lk(g_arena.mu);
  int dev = 0;
  GVOTE_CUDA_CHECK(cudaGetDevice(&dev));
  if (g_arena.device != dev || g_arena.cap < off) {
    if (g_arena.base) { GVOTE_CUDA_CHECK(cudaFree(g_arena.base)); g_arena.base = nullptr; g_arena.cap = 0; }
    if (g_arena.stream && g_arena.device != dev) { cudaStreamDestroy(g_arena.stream); g_arena.stream = nullptr; }
    GVOTE_CUDA_CHECK(cudaMalloc((void**)&g_arena.base, off));
    g_arena.cap = off;
    g_arena.device = dev;
    if (!g_arena.stream) GVOTE_CUDA_CHECK(cudaStreamCreateWithFlags(&g_arena.stream, cudaStreamNonBlocking));
    GVOTE_CUDA_CHECK(cudaMemsetAsync(g_arena.base + o_ws, 0, kStatusBytes, g_arena.stream));
  }
  char* d = g_arena.base;
  cudaStream_t st = g_arena.stream;
  // a status left by an earlier call on this arena must not be reported again
  GVOTE_CUDA_CHECK(cudaMemsetAsync(d + o_ws, 0, kStatusBytes, st));
  GVOTE_CUDA_CHECK(cudaMemcpyAsync(d + o_cu, cu_seqlens_host, b_cu, cudaMemcpyHostToDevice, st));
  GVOTE_CUDA_CHECK(cudaMemcpyAsync(d + o_h, h, b_h, cudaMemcpyHostToDevice, st));
  GVOTE_CUDA_CHECK(cudaMemcpyAsync(d + o_w, W_q, b_w, cudaMemcpyHostToDevice, st));
  if (b_b) GVOTE_CUDA_CHECK(cudaMemcpyAsync(d + o_b, b_q_or_null, b_b, cudaMemcpyHostToDevice, st));
  GVOTE_CUDA_CHECK(cudaMemcpyAsync(d + o_k, K, b_kv, cudaMemcpyHostToDevice, st));
  GVOTE_CUDA_CHECK(cudaMemcpyAsync(d + o_v, V, b_kv, cudaMemcpyHostToDevice, st));
  PROPAGATE(gvote_compress(p, d + o_h, p->d_h, nullptr, d + o_w, p->d_h, b_b ? (const float*)(d + o_b) : nullptr,
                           d + o_k, d + o_v, p->d_k, (int64_t)total * p->d_k, (const int32_t*)(d + o_cu), batch,
                           total, max_N, (uint32_t*)(d + o_mask), (int32_t*)(d + o_bud), (int32_t*)(d + o_bs),
                           d + o_ws, m.total, st));
  GVOTE_CUDA_CHECK(cudaMemcpyAsync(mask, d + o_mask, b_mask, cudaMemcpyDeviceToHost, st));
  GVOTE_CUDA_CHECK(cudaMemcpyAsync(budget, d + o_bud, b_bud, cudaMemcpyDeviceToHost, st));
  GVOTE_CUDA_CHECK(cudaMemcpyAsync(b_step, d + o_bs, b_bs, cudaMemcpyDeviceToHost, st));
  GVOTE_CUDA_CHECK(cudaMemcpyAsync(K, d + o_k, b_kv, cudaMemcpyDeviceToHost, st));
  GVOTE_CUDA_CHECK(cudaMemcpyAsync(V, d + o_v, b_kv, cudaMemcpyDeviceToHost, st));
  GVOTE_CUDA_CHECK(cudaStreamSynchronize(st));
  int32_t status[2] = {0, 0};
  GVOTE_CUDA_CHECK(cudaMemcpy(status, d + o_ws, sizeof(status), cudaMemcpyDeviceToHost));
  return status[0];
}

int32_t gvote_poll_status(void* ws, void* stream) {
  if (!ws) return GVOTE_ERR_INVALID_ARG;
  GVOTE_CUDA_CHECK(cudaStreamSynchronize((cudaStream_t)stream));
  int32_t status = 0;
  GVOTE_CUDA_CHECK(cudaMemcpy(&status, ws, sizeof(status), cudaMemcpyDeviceToHost));
  return status;
}

int32_t gvote_clear_status(void* ws, void* stream) {
  if (!ws) return GVOTE_ERR_INVALID_ARG;
  GVOTE_CUDA_CHECK(cudaMemsetAsync(ws, 0, kStatusBytes, (cudaStream_t)stream));
  return GVOTE_OK;
}

int64_t gvote_exact_heads(void* ws, void* stream) {
  if (!ws) return GVOTE_ERR_INVALID_ARG;
  GVOTE_CUDA_CHECK(cudaStreamSynchronize((cudaStream_t)stream));
  int32_t words[4] = {0, 0, 0, 0};
  GVOTE_CUDA_CHECK(cudaMemcpy(words, ws, sizeof(words), cudaMemcpyDeviceToHost));
  return words[2];
}

void gvote_profile_enable(int32_t on) {
  std::lock_guard<std::mutex> lk(g_prof_mu);
  for (auto& r : g_prof_recs) { g_prof_pool.push_back(r.a); g_prof_pool.push_back(r.b); }
  g_prof_recs.clear();
  g_prof_on.store(on != 0);
}

size_t gvote_profile_report(char* buf, size_t cap) {
  cudaDeviceSynchronize();
  std::lock_guard<std::mutex> lk(g_prof_mu);
  std::map<std::string, std::pair<long long, double>> agg;
  std::vector<std::string> order;
  for (auto& r : g_prof_recs) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, r.a, r.b) != cudaSuccess) continue;
    auto it = agg.find(r.name);
    if (it == agg.end()) { order.push_back(r.name); it = agg.emplace(r.name, std::make_pair(0LL, 0.0)).first; }
    it->second.first += 1;
    it->second.second += ms;
  }
  std::string out;
  char line[256];
  for (auto& n : order) {
    snprintf(line, sizeof(line), "%s %lld %.6f\n", n.c_str(), agg[n].first, agg[n].second);
    out += line;
  }
  if (buf && cap > 0) {
    const size_t n = out.size() < cap - 1 ? out.size() : cap - 1;
    memcpy(buf, out.data(), n);
    buf[n] = 0;
  }
  return out.size() + 1;
}

int64_t gvote_launch_count(void) { return (int64_t)g_launches.load(std::memory_order_relaxed); }

const char* gvote_status_string(int32_t s) {
  switch (s) {
    case GVOTE_OK: return "ok";
    case GVOTE_ERR_INVALID_ARG: return "invalid argument";
    case GVOTE_ERR_UNALIGNED: return "pointer or stride not 16-byte aligned";
    case GVOTE_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case GVOTE_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case GVOTE_ERR_CUDA: return "CUDA error (see gvote_last_cuda_error)";
    case GVOTE_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    default: return "unknown status";
  }
}

const char* gvote_last_cuda_error(void) { return g_cuda_err; }

}  // extern "C"
