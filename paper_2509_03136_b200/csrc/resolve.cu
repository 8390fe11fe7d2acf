// Algorithm 1, the TopK step of the synthetic queries around the tensor-core sweep (sweep_umma.cu):
//
//   bracket_kernel   before the sweep: two order statistics of a row's sampled half-precision keys that
//                    enclose its k-th largest logit (k = B_step of the row's query head), as fp32 bounds
//                    [lo, hi]; also clears the row's counters.
//   resolve_kernel   after the sweep: a row whose bracket held (#above <= k <= #above + #listed, list not
//                    overflowed) takes the k - #above largest of its listed candidates by (fp32 logit
//                    descending, key index ascending) and ORs them into the tentative mask; a row whose
//                    bracket missed marks its KV head.
//   commit_kernel    the union becomes final: a KV head whose rows all settled copies its tentative mask
//                    into the keep mask; a marked head discards it and every row of the head is selected
//                    again by the exact route (fp32 logits recomputed from Q and K, radix search over the
//                    row, no sample involved), so a missed bracket costs time, never correctness.
//
// Order statistics are found by bisection on an order-preserving integer image of the values: one
// count over the thread's elements and one block-wide sum per bit, no sorting, no atomics, the same
// bits on every run.
#include <cuda_fp16.h>

#include "select_common.cuh"
#include "vote_geom.cuh"

namespace gvote {
namespace {

using namespace sel;

constexpr int kRowThreads = 256;

// Half bits <-> 16-bit code whose unsigned order is the numeric order.
__device__ __forceinline__ uint32_t raw_of_code(uint32_t c) { return (c & 0x8000u) ? (c & 0x7fffu) : (~c & 0xffffu); }
__device__ __forceinline__ float float_of_code(uint32_t c) {
  return __half2float(__ushort_as_half((unsigned short)raw_of_code(c)));
}

// Sum of one value per thread over the CTA.  `red` holds two rows of one slot per warp, used alternately,
// so that consecutive sums need one barrier each.
struct BlockSum {
  uint32_t* red;    // [2][kRowThreads / 32]
  int flip;
  __device__ __forceinline__ uint32_t operator()(uint32_t v) {
    v = (uint32_t)warp_sum_i((int)v);
    uint32_t* row = red + flip * (kRowThreads / 32);
    flip ^= 1;
    if ((threadIdx.x & 31) == 0) row[threadIdx.x >> 5] = v;
    __syncthreads();
    uint32_t s = 0;
#pragma unroll
    for (int w = 0; w < kRowThreads / 32; ++w) s += row[w];
    return s;
  }
  __device__ __forceinline__ void sum2(uint32_t a, uint32_t b, uint32_t& sa, uint32_t& sb) {
    a = (uint32_t)warp_sum_i((int)a);
    b = (uint32_t)warp_sum_i((int)b);
    uint32_t* row = red + flip * (kRowThreads / 32);
    flip ^= 1;
    if ((threadIdx.x & 31) == 0) row[threadIdx.x >> 5] = (a << 16) | b;      // both counts are below 2^16
    __syncthreads();
    sa = 0;
    sb = 0;
#pragma unroll
    for (int w = 0; w < kRowThreads / 32; ++w) { sa += row[w] >> 16; sb += row[w] & 0xffffu; }
  }
};

// ------------------------------------------------------------------------------------ bracket
constexpr int kBrVecs = 8;      // 16-byte vectors of sampled keys per thread: 256 * 8 * 8 = 16384 keys at most

__device__ __forceinline__ uint32_t count_ge(const uint4 (&v)[kBrVecs], uint32_t raw) {
  const uint32_t p = raw | (raw << 16);
  const __half2 th = *reinterpret_cast<const __half2*>(&p);
  uint32_t c = 0;
#pragma unroll
  for (int u = 0; u < kBrVecs; ++u) {
    const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
    for (int j = 0; j < 4; ++j) c += __popc(__hge2_mask(*reinterpret_cast<const __half2*>(&w[j]), th));
  }
  return c >> 4;
}

__global__ void __launch_bounds__(kRowThreads)
bracket_kernel(const uint16_t* __restrict__ sample, int64_t sample_slots, const int32_t* __restrict__ cu, int Hq,
               int G, int S, int row_chunks, const int32_t* __restrict__ b_step, RowBracket* __restrict__ bracket,
               uint32_t* __restrict__ above, uint32_t* __restrict__ ncand, const int32_t* __restrict__ kv_len) {
  __shared__ uint32_t red[2 * (kRowThreads / 32)];
  const int r = blockIdx.z, g = blockIdx.y, s = blockIdx.x;
  const int rowid = (r * Hq + g) * S + s;
  const int start = cu[r];
  const int kh = g / G;
  const int N = valid_keys(kv_len, r, Hq / G, kh, cu[r + 1] - start);
  const int tid = threadIdx.x;
  if (tid == 0) { above[rowid] = 0; ncand[rowid] = 0; }
  const int k = N > 0 ? b_step[r * Hq + g] : 0;
  if (N <= 0 || k <= 0) {                                  // nothing to select
    if (tid == 0) bracket[rowid] = RowBracket{INFINITY, INFINITY};
    return;
  }
  if (k >= N) {                                            // every key is selected: all of them lie "above"
    if (tid == 0) bracket[rowid] = RowBracket{-INFINITY, -INFINITY};
    return;
  }
  const SampleGeom geo = sample_geom(N);
  const int grow = (g % G) * S + s;
  const int chunk = grow / kVoteRowChunk, crow = grow % kVoteRowChunk;
  const int64_t slot_stride = (int64_t)row_chunks * kVoteRowChunk * kVoteTileKeys;
  const uint16_t* base = sample + ((((int64_t)kh * sample_slots + sample_slot_offset(start, r)) * row_chunks + chunk) *
                                   kVoteRowChunk + crow) * kVoteTileKeys;
  uint4 v[kBrVecs];
  const int n_vecs = geo.ns * 16;
#pragma unroll
  for (int u = 0; u < kBrVecs; ++u) {
    const int i = u * kRowThreads + tid;
    v[u] = make_uint4(0xfc00fc00u, 0xfc00fc00u, 0xfc00fc00u, 0xfc00fc00u);     // -inf: never counted
    if (i < n_vecs) v[u] = *reinterpret_cast<const uint4*>(base + (int64_t)(i >> 4) * slot_stride + (i & 15) * 8);
  }
  // ranks (1-based, among the m sampled keys) whose keys become the bounds
  const int m = sample_keys(geo, N);
  uint32_t rank_hi, rank_lo;                               // rank_hi <= rank_lo; 0 = no bound on that side
  if (geo.whole) {
    rank_hi = rank_lo = (uint32_t)k;                       // the sample is the row: its k-th key is the threshold
  } else {
    // 4.5 standard deviations of the sampling error of a rank, either side of the expected one
    const float frac = (float)k / (float)N;
    const float rk = frac * (float)m;
    const float dlt = 4.5f * sqrtf(rk * (1.0f - frac)) + 6.0f;
    const int r_lo = (int)ceilf(rk + dlt), r_hi = (int)floorf(rk - dlt);
    rank_lo = r_lo > m ? 0u : (uint32_t)r_lo;
    rank_hi = r_hi >= 1 ? (uint32_t)r_hi : 0u;
  }
  // both order statistics at once, bit by bit from the top: largest code c with #(key >= c) >= rank
  BlockSum sum{red, 0};
  uint32_t code_hi = 0, code_lo = 0;
  for (int bit = 15; bit >= 0; --bit) {
    const uint32_t t_hi = code_hi | (1u << bit), t_lo = code_lo | (1u << bit);
    uint32_t c_hi, c_lo;
    sum.sum2(rank_hi ? count_ge(v, raw_of_code(t_hi)) : 0u, rank_lo ? count_ge(v, raw_of_code(t_lo)) : 0u, c_hi, c_lo);
    if (rank_hi && c_hi >= rank_hi) code_hi = t_hi;
    if (rank_lo && c_lo >= rank_lo) code_lo = t_lo;
  }
  if (tid == 0) {
    // two codes of slack either side: the sweep compares fp32 logits, the sample held their roundings
    RowBracket b;
    b.lo = (rank_lo && code_lo >= 0x0402u) ? float_of_code(code_lo - 2u) : -INFINITY;
    b.hi = (rank_hi && code_hi + 2u <= 0xfbffu) ? float_of_code(code_hi + 2u) : INFINITY;
    bracket[rowid] = b;
  }
}

// ------------------------------------------------------------------------------------ resolve
// Candidate keys as order-preserving integers, in shared memory when the list fits there, else read
// from the list in global memory.
struct CandKeys {
  const uint32_t* p;
  int stride;
  __device__ __forceinline__ uint32_t operator[](int i) const { return p[(int64_t)i * stride]; }
};

__global__ void __launch_bounds__(kRowThreads)
resolve_kernel(const int32_t* __restrict__ cu, int Hq, int G, int S, const int32_t* __restrict__ b_step,
               const VoteState vs, int smem_keys, int64_t row_words, const int32_t* __restrict__ kv_len) {
  extern __shared__ __align__(16) uint32_t keys_sm[];
  __shared__ uint32_t red[2 * (kRowThreads / 32)];
  __shared__ uint32_t s_min, s_max;
  const int r = blockIdx.z, g = blockIdx.y, s = blockIdx.x;
  const int rowid = (r * Hq + g) * S + s;
  const int start = cu[r], Ncap = cu[r + 1] - start;
  const int kh = g / G, Hkv = Hq / G;
  const int N = valid_keys(kv_len, r, Hkv, kh, Ncap);
  if (N <= 0) return;
  const int k = min(b_step[r * Hq + g], N);
  if (k <= 0) return;
  const int tid = threadIdx.x;
  const uint32_t A = vs.above[rowid], C = vs.ncand[rowid];
  if (A > (uint32_t)k || C > (uint32_t)vs.lay.cap(Ncap) || A + C < (uint32_t)k) {   // the bracket missed or the list overflowed
    if (tid == 0) atomicExch(&vs.head_bad[r * Hkv + kh], 1u);
    return;
  }
  const uint32_t need = (uint32_t)k - A;
  if (need == 0) return;
  uint2* list = vs.list(g, s, S, start, r);
  uint32_t* mrow = vs.tmask + (int64_t)kh * row_words + mask_word_offset(start, r);
  if (need == C) {                                         // every listed key is taken
    for (int i = tid; i < (int)C; i += kRowThreads) {
      const uint32_t n = list[i].y;
      atomicOr(&mrow[n >> 5], 1u << (n & 31));
    }
    return;
  }
  // order-preserving images of the listed logits
  CandKeys keys;
  if ((int)C <= smem_keys) {
    for (int i = tid; i < (int)C; i += kRowThreads) keys_sm[i] = ordered_key(__uint_as_float(list[i].x));
    keys.p = keys_sm;
    keys.stride = 1;
  } else {
    for (int i = tid; i < (int)C; i += kRowThreads) list[i].x = ordered_key(__uint_as_float(list[i].x));
    keys.p = reinterpret_cast<const uint32_t*>(list);
    keys.stride = 2;
  }
  if (tid == 0) { s_min = 0xffffffffu; s_max = 0u; }
  __syncthreads();
  {
    uint32_t mn = 0xffffffffu, mx = 0u;
    for (int i = tid; i < (int)C; i += kRowThreads) { const uint32_t x = keys[i]; mn = min(mn, x); mx = max(mx, x); }
    mn = __reduce_min_sync(0xffffffffu, mn);
    mx = __reduce_max_sync(0xffffffffu, mx);
    if ((tid & 31) == 0) { atomicMin(&s_min, mn); atomicMax(&s_max, mx); }
  }
  __syncthreads();
  // the need-th largest key: the bits above the first one in which the extremes differ are common to all
  BlockSum sum{red, 0};
  const uint32_t diff = s_min ^ s_max;
  uint32_t T = s_max;
  if (diff) {
    const int top = 31 - __clz(diff);
    T = top == 31 ? 0u : (s_max & ~((2u << top) - 1u));
    for (int bit = top; bit >= 0; --bit) {
      const uint32_t trial = T | (1u << bit);
      uint32_t c = 0;
      for (int i = tid; i < (int)C; i += kRowThreads) c += keys[i] >= trial ? 1u : 0u;
      if (sum(c) >= need) T = trial;
    }
  }
  uint32_t gt = 0, eq = 0;
  for (int i = tid; i < (int)C; i += kRowThreads) { const uint32_t x = keys[i]; gt += x > T ? 1u : 0u; eq += x == T ? 1u : 0u; }
  gt = sum(gt);
  eq = sum(eq);
  const uint32_t ties = need - gt;                         // 1 <= ties <= eq
  // equal logits go to the lower key index: the ties-th smallest index among them bounds the ones taken
  uint32_t idx_max = 0xffffffffu;
  if (ties < eq) {
    uint32_t vlim = 0;                                     // largest v with #(equal, index < v) < ties
    for (int bit = 31 - __clz(max(N - 1, 1)); bit >= 0; --bit) {
      const uint32_t trial = vlim | (1u << bit);
      uint32_t c = 0;
      for (int i = tid; i < (int)C; i += kRowThreads) c += (keys[i] == T && list[i].y < trial) ? 1u : 0u;
      if (sum(c) < ties) vlim = trial;
    }
    idx_max = vlim;
  }
  for (int i = tid; i < (int)C; i += kRowThreads) {
    const uint32_t x = keys[i], n = list[i].y;
    if (x > T || (x == T && n <= idx_max)) atomicOr(&mrow[n >> 5], 1u << (n & 31));
  }
}

// ------------------------------------------------------------------------------------ commit
// The exact fp32 logits of one row, computed where they are needed.
struct ExactRow {
  DotCtx dot;
  __device__ __forceinline__ float operator()(int n) const { return dot(n); }
};

__global__ void __launch_bounds__(kRowThreads)
commit_kernel(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K, int64_t k_tok, int64_t k_head,
              const int32_t* __restrict__ cu, int Hq, int G, int S, int d_k, float scale,
              const int32_t* __restrict__ b_step, const uint32_t* __restrict__ tmask, int64_t row_words,
              uint32_t* __restrict__ mask, const uint32_t* __restrict__ head_bad, const int32_t* __restrict__ kv_len) {
  __shared__ SelShared sh;
  __shared__ __align__(16) __nv_bfloat16 qf[512];
  const int r = blockIdx.z, g = blockIdx.y, s = blockIdx.x;
  const int start = cu[r], Ncap = cu[r + 1] - start;
  const int kh = g / G, Hkv = Hq / G;
  const int tid = threadIdx.x;
  const int64_t woff = (int64_t)kh * row_words + mask_word_offset(start, r);
  if (!head_bad[r * Hkv + kh]) {
    // the G * S rows of the head share the copy of its words
    const int words = (Ncap + 31) >> 5;
    const int idx = (g % G) * S + s;
    for (int w = idx * kRowThreads + tid; w < words; w += G * S * kRowThreads) {
      const uint32_t v = tmask[woff + w];
      if (v) mask[woff + w] |= v;
    }
    return;
  }
  // a bracket of this head missed: this row again, exactly
  const int N = valid_keys(kv_len, r, Hkv, kh, Ncap);
  if (N <= 0) return;
  const int k = min(b_step[r * Hq + g], N);
  if (k <= 0) return;
  const int grow = (g % G) * S + s;
  const __nv_bfloat16* qrow = Q + (((int64_t)r * Hkv + kh) * (G * (S + 1)) + grow) * d_k;
  for (int i = tid; i < d_k; i += kRowThreads) qf[i] = qrow[i];
  __syncthreads();
  ExactRow row{DotCtx{qf, K + (int64_t)kh * k_head + (int64_t)start * k_tok, k_tok, d_k, scale}};
  uint32_t t, above_cnt, eq_cnt;
  unsigned long long above_mass;
  radix_threshold<false>(row, N, 0.f, (unsigned long long)k, sh, t, above_cnt, above_mass, eq_cnt);
  emit_row(row, N, t, (uint32_t)k - above_cnt, eq_cnt, mask + woff, sh);
}

}  // namespace

// The three launchers: before the sweep, after it, and the commit.
int32_t launch_bracket(const gvote_params* p, const int32_t* cu, int32_t batch, const int32_t* b_step, const VoteState& vs,
                       const int32_t* kv_len, cudaStream_t st) {
  const int Hq = p->n_q_heads, G = Hq / p->n_kv_heads;
  dim3 grid(p->S, Hq, batch);
  {
    LaunchScope scope_("bracket_kernel", st);
    bracket_kernel<<<grid, kRowThreads, 0, st>>>(vs.sample, vs.sample_slots, cu, Hq, G, p->S, score_geometry(p).row_chunks,
                                                 b_step, vs.bracket, vs.above, vs.ncand, kv_len);
  }
  GVOTE_LAUNCH_CHECK("bracket_kernel");
  return GVOTE_OK;
}

int32_t launch_resolve(const gvote_params* p, const int32_t* cu, int32_t batch, int64_t max_N, const int32_t* b_step,
                       const VoteState& vs, int64_t row_words, const int32_t* kv_len, cudaStream_t st) {
  const int Hq = p->n_q_heads, G = Hq / p->n_kv_heads;
  dim3 grid(p->S, Hq, batch);
  // the keys of a list live in shared memory when it leaves room for six CTAs per SM
  const int64_t longest = vs.lay.uniform_cap > 0 ? vs.lay.uniform_cap : vs.lay.cap((int)max_N);
  const int smem_keys = (int)(longest <= 8192 ? longest : 8192);
  const size_t smem = (size_t)smem_keys * sizeof(uint32_t);
  if (smem > 48 * 1024)
    GVOTE_CUDA_CHECK(cudaFuncSetAttribute(resolve_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  {
    LaunchScope scope_("resolve_kernel", st);
    resolve_kernel<<<grid, kRowThreads, smem, st>>>(cu, Hq, G, p->S, b_step, vs, smem_keys, row_words, kv_len);
  }
  GVOTE_LAUNCH_CHECK("resolve_kernel");
  return GVOTE_OK;
}

int32_t launch_commit(const gvote_params* p, const __nv_bfloat16* Q, const __nv_bfloat16* K, int64_t k_tok, int64_t k_head,
                      const int32_t* cu, int32_t batch, const int32_t* b_step, const VoteState& vs, int64_t row_words,
                      uint32_t* mask, const int32_t* kv_len, cudaStream_t st) {
  const int Hq = p->n_q_heads, G = Hq / p->n_kv_heads;
  dim3 grid(p->S, Hq, batch);
  const float scale = (float)(1.0 / sqrt((double)p->d_k));
  {
    LaunchScope scope_("commit_kernel", st);
    commit_kernel<<<grid, kRowThreads, 0, st>>>(Q, K, k_tok, k_head, cu, Hq, G, p->S, p->d_k, scale, b_step, vs.tmask,
                                                row_words, mask, vs.head_bad, kv_len);
  }
  GVOTE_LAUNCH_CHECK("commit_kernel");
  return GVOTE_OK;
}

}  // namespace gvote
