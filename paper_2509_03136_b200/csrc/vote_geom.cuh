// Geometry shared by the kernels of the fused vote (Algorithm 1: logits, TopK, union without the S x N
// logits ever reaching memory): which key tiles of a row form its sample, where a row's sampled keys,
// its bracket, its counters and its candidate list live, and the exact fp32 logit of one key.
//
// A row is one synthetic query of one query head: global row id = (r * n_q_heads + g) * S + s.
// Inside its KV head's group it is row gl * S + s (gl = g mod G) of the G * S synthetic rows, i.e. row
// `crow` of 128-row chunk `chunk`.
#pragma once

#include "common.cuh"

namespace gvote {

constexpr int kVoteTileKeys = 128;   // keys per tile of the score contraction
constexpr int kVoteRowChunk = 128;   // synthetic rows per accumulator (MMA M)

// The sample of a row of N keys, in whole key tiles.  Rows of at most 32 tiles are sampled completely
// (the bracket then is the threshold itself); longer rows take `ns` of their full tiles, one from each
// stretch of `stride` tiles, at an offset that changes from stretch to stretch so that a periodic
// pattern in the keys cannot line up with the sample.
struct SampleGeom {
  int n_tiles, ns, stride;
  bool whole;
};
__host__ __device__ __forceinline__ SampleGeom sample_geom(int N) {
  SampleGeom g;
  g.n_tiles = (N + kVoteTileKeys - 1) / kVoteTileKeys;
  if (g.n_tiles <= 32) {
    g.ns = g.n_tiles;
    g.stride = 1;
    g.whole = true;
  } else {
    int want = g.n_tiles >> 3;
    want = want < 32 ? 32 : (want > 128 ? 128 : want);
    const int n_full = N / kVoteTileKeys;          // >= 32 here
    g.ns = want;
    g.stride = n_full / want;                      // >= 1
    g.whole = false;
  }
  return g;
}
__host__ __device__ __forceinline__ int sample_tile(const SampleGeom& g, int j) {
  if (g.stride == 1) return j;
  const uint32_t hsh = ((uint32_t)j * 2654435761u) >> 15;
  return j * g.stride + (int)(hsh % (uint32_t)g.stride);
}
// Position of tile t in the sample, or -1.
__host__ __device__ __forceinline__ int sample_slot_of_tile(const SampleGeom& g, int t) {
  const int j = t / g.stride;
  return (j < g.ns && sample_tile(g, j) == t) ? j : -1;
}
// Keys in the sample (a completely sampled row counts its N keys; the pad of its last tile reads as -inf).
__host__ __device__ __forceinline__ int sample_keys(const SampleGeom& g, int N) {
  return g.whole ? N : g.ns * kVoteTileKeys;
}
// First sample-tile slot of request r in the sample buffer, and the slots a batch needs: a request of
// N keys takes at most 32 + N / 1024 + 1 slots (closed forms: no kernel has to add up the requests before
// its own).  A single request takes exactly its own.
__host__ __device__ __forceinline__ int64_t sample_slot_offset(int cu_r, int r) { return (int64_t)34 * r + (cu_r >> 10); }
inline int64_t sample_slots_total(int32_t batch, int64_t total_tokens, int64_t max_N) {
  if (batch == 1) return sample_geom((int)max_N).ns > 0 ? sample_geom((int)max_N).ns : 1;
  return (int64_t)34 * batch + (total_tokens >> 10) + 1;
}

// Keys a row's bracket is expected to hold at most.  It spans 2 * (4.5 sqrt(m f (1 - f)) + 6) of the m
// sampled keys' ranks, at most 4.5 sqrt(m) + 12, i.e. that many times N / m keys of the row.  A completely
// sampled row lists only the keys that share the threshold's 16-bit value or its neighbours'.
inline double candidates_expected(int64_t N) {
  if (N <= 0) return 64.0;
  const SampleGeom g = sample_geom((int)N);
  if (g.whole) return 64.0;
  const double m = (double)g.ns * kVoteTileKeys;
  return (4.5 * sqrt(m) + 12.0) * ((double)N / m);
}

// Where the candidate lists live.  The sweep's read-out threads never share a list: thread (CTA x, column
// quarter c) of a row owns segment x * 4 + c of the row's list, `segs` = 4 X segments in all, and appends
// to it without atomics.  A CTA's tiles x, x + X, ... are spread evenly over the row, so a segment holds an
// even share mu of the row's candidates up to counting noise: capacity mu + 4.5 sqrt(mu) + 8 for a single
// request; in a batch, the line 20 + 29 N / (256 segs) above that, whose running sum over the requests
// has a closed form (no kernel has to add up the requests before its own).  Row (g, s) owns a strip of
// `strip` entries; request r's segments start at entry offset(r) of the strip.
struct CandLayout {
  int segs;
  int uniform_seg_cap;   // > 0: one request, this capacity per segment
  int64_t strip;
  __host__ __device__ __forceinline__ int seg_cap(int N) const {
    return uniform_seg_cap > 0 ? uniform_seg_cap : 20 + (int)(((29 * (int64_t)N) >> 8) / segs);
  }
  __host__ __device__ __forceinline__ int64_t offset(int cu_r, int r) const {
    return uniform_seg_cap > 0 ? 0 : (int64_t)segs * 20 * r + ((29 * (int64_t)cu_r) >> 8);
  }
};
inline CandLayout cand_layout(int segs, int32_t batch, int64_t total_tokens, int64_t max_N) {
  CandLayout c;
  c.segs = segs;
  if (batch == 1) {
    const double mu = candidates_expected(max_N) / segs;
    c.uniform_seg_cap = (((int)ceil(mu + 4.5 * sqrt(mu) + 8.0)) + 3) & ~3;
    c.strip = (int64_t)segs * c.uniform_seg_cap;
  } else {
    c.uniform_seg_cap = 0;
    c.strip = (int64_t)segs * 20 * batch + ((29 * total_tokens) >> 8) + 1;
  }
  return c;
}

struct RowBracket { float lo, hi; };    // keys above hi are taken, keys in [lo, hi] are listed

// Where the fused vote keeps its state in the workspace.
struct VoteState {
  uint16_t* sample;        // fp16 keys [n_kv_heads][sample slots][row_chunks][128 rows][128 keys]
  RowBracket* bracket;     // [rows]
  uint2* segstat;          // [rows][segs] (keys above the bracket, keys inside it) met by each segment's writer
  uint2* cand;             // [n_q_heads * S][strip] (fp32 logit bits, key index), see CandLayout
  CandLayout lay;
  uint32_t* tmask;         // [n_kv_heads][row_words] the union while it is tentative
  uint32_t* head_bad;      // [batch][n_kv_heads] a bracket of the head missed: redo the head exactly
  int32_t* status;         // the workspace's status block; word 2 counts the heads redone exactly
  int64_t sample_slots;
  // the first segment of the list of row (g, s) of request r
  __host__ __device__ __forceinline__ uint2* list(int g, int s, int S, int cu_r, int r) const {
    return cand + (int64_t)(g * S + s) * lay.strip + lay.offset(cu_r, r);
  }
};

// Launch geometry of the second pass (sweep_umma.cu); the segment count of the lists follows from it.
struct SweepGeom { int cg, stages, groups, X, stg; };
SweepGeom sweep_geometry(const gvote_params* p, int32_t batch, int64_t max_N);

#ifdef __CUDACC__
// Exact fp32 logit of key n for one query row (fixed summation order).
struct DotCtx {
  const __nv_bfloat16* qf;      // the row's query, d_k values (shared memory)
  const __nv_bfloat16* krows;   // K + head offset + request start
  int64_t k_tok;
  int d_k;
  float scale;
  __device__ __forceinline__ void add8(float& acc, const uint4& v, int c) const {
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 f = __bfloat1622float2(h[j]);
      const float2 q = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(qf + c * 8 + 2 * j));
      acc = fmaf(q.x, f.x, acc);
      acc = fmaf(q.y, f.y, acc);
    }
  }
  __device__ __forceinline__ float operator()(int n) const {
    const uint4* kp = reinterpret_cast<const uint4*>(krows + (int64_t)n * k_tok);
    float acc = 0.f;
    const int nc = d_k / 8;
    int c = 0;
    for (; c + 4 <= nc; c += 4) {                     // four loads in flight, summed in index order
      const uint4 v0 = __ldg(kp + c), v1 = __ldg(kp + c + 1), v2 = __ldg(kp + c + 2), v3 = __ldg(kp + c + 3);
      add8(acc, v0, c); add8(acc, v1, c + 1); add8(acc, v2, c + 2); add8(acc, v3, c + 3);
    }
    for (; c < nc; ++c) add8(acc, __ldg(kp + c), c);
    return acc * scale;
  }
};
#endif

}  // namespace gvote
