// Algorithm 1, the TopK step of the synthetic queries around the tensor-core sweep (sweep_umma.cu):
//
//   bracket_kernel   before the sweep: two order statistics of a row's sampled half-precision keys that
//                    enclose its k-th largest logit (k = B_step of the row's query head), as fp32 bounds
//                    [lo, hi].
//   resolve_kernel   after the sweep: a row whose bracket held (#above <= k <= #above + #listed, list not
//                    overflowed) takes the k - #above largest of its listed candidates by (fp32 logit
//                    descending, key index ascending) and ORs them into the tentative mask; a row whose
//                    bracket missed marks its KV head.
//   commit_kernel    the union becomes final: a KV head whose rows all settled copies its tentative mask
//                    into the keep mask; a marked head discards it and every row of the head is selected
//                    again by the exact route (fp32 logits recomputed from Q and K, radix search over the
//                    row, no sample involved), so a missed bracket costs time, never correctness.
//
// Order statistics are found by radix searches over order-preserving integer images of the values
// (histograms of integer counts: no sorting, and the same bits on every run).
#include <cuda_fp16.h>

#include "select_common.cuh"
#include "vote_geom.cuh"

namespace gvote {
namespace {

using namespace sel;

// Half bits <-> 16-bit code whose unsigned order is the numeric order.
__device__ __forceinline__ uint32_t raw_of_code(uint32_t c) { return (c & 0x8000u) ? (c & 0x7fffu) : (~c & 0xffffu); }
__device__ __forceinline__ float float_of_code(uint32_t c) {
  return __half2float(__ushort_as_half((unsigned short)raw_of_code(c)));
}

// Largest bin b of hist[0..256) whose suffix count reaches `need` (need >= 1, total >= need), found by
// one warp: every lane returns the bin and the count in the bins above it.
__device__ __forceinline__ void warp_find_bin256(const uint32_t* hist, uint32_t need, int lane, int& bin,
                                                 uint32_t& above) {
  uint32_t c = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) c += hist[lane * 8 + i];
  uint32_t cs = c;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_down_sync(0xffffffffu, cs, o);
    if (lane + o < 32) cs += t;
  }
  const uint32_t excl = cs - c;                          // count in the lanes above this one
  const bool own = excl < need && excl + c >= need;
  uint32_t a = excl;
  int b = lane * 8 + 7;
  if (own) {
    for (; b > lane * 8; --b) {
      if (a + hist[b] >= need) break;
      a += hist[b];
    }
  }
  const uint32_t who = __ballot_sync(0xffffffffu, own);
  const int src = who ? __ffs(who) - 1 : 0;
  bin = who ? __shfl_sync(0xffffffffu, b, src) : 0;
  above = who ? __shfl_sync(0xffffffffu, a, src) : 0u;
}

// ------------------------------------------------------------------------------------ bracket
// Two order statistics of a row's sampled keys (at most 16384 half-precision values, held in registers)
// by a two-level radix search over their 16-bit order-preserving codes, both ranks at a time.
// Level 1 bins the high byte.  Every sampled key takes part and a few bins take most of them, so plain
// shared-memory atomics would queue on those addresses: counting goes into one 16-bit counter per (bin,
// lane) instead, two bins to a word, word (bin / 2) * 32 + lane - the lanes of a warp never meet, and a
// counter takes at most (4 warps) x (128 keys per thread) increments.  Bins are those of the raw half bits
// (no recoding per key); the fold over the lanes puts them in code order.  Level 2 bins the low byte of
// the keys whose high byte is the one found, for the two ranks side by side.  Integer counts only: the
// same bits on every run.
constexpr int kBrThreads = 128;
// (NV: 16-byte vectors of sampled keys a thread holds: 4 for samples of up to 4096 keys - fewer registers,
// twice the CTAs per SM - and 16 for the largest, 128 * 16 * 8 = 16384 keys)

// High byte of a key's code from the high byte hb of its half bits.
__device__ __forceinline__ uint32_t ord_hi(uint32_t hb) { return hb >= 0x80u ? 0xffu - hb : 0x80u + hb; }

struct BracketShared {
  uint32_t lanes[128 * 32];     // level 1: 16-bit counters per (raw high byte, lane)
  uint32_t bins[256];           // level 1 folded, in code order
  uint32_t low[512];            // level 2: [0, 256) for the lower rank's bin, [256, 512) for the upper one's
  int bin[2];
  uint32_t above[2];
};

template <int NV>
__global__ void __launch_bounds__(kBrThreads)
bracket_kernel(const uint16_t* __restrict__ sample, int64_t sample_slots, const int32_t* __restrict__ cu, int Hq,
               int G, int S, int row_chunks, const int32_t* __restrict__ b_step, RowBracket* __restrict__ bracket,
               const int32_t* __restrict__ kv_len) {
  __shared__ BracketShared sh;
  const int r = blockIdx.z, g = blockIdx.y, s = blockIdx.x;
  const int rowid = (r * Hq + g) * S + s;
  const int start = cu[r];
  const int kh = g / G;
  const int N = valid_keys(kv_len, r, Hq / G, kh, cu[r + 1] - start);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
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
  uint4 v[NV];
  const int n_vecs = geo.ns * 16;
  const int have = (n_vecs + kBrThreads - 1) / kBrThreads;   // the same for every thread of the CTA
#pragma unroll
  for (int u = 0; u < NV; ++u) {
    const int i = u * kBrThreads + tid;
    v[u] = make_uint4(0xfc00fc00u, 0xfc00fc00u, 0xfc00fc00u, 0xfc00fc00u);     // -inf: below every rank asked for
    if (u < have && i < n_vecs) v[u] = *reinterpret_cast<const uint4*>(base + (int64_t)(i >> 4) * slot_stride + (i & 15) * 8);
  }
  const bool small = have <= 2;                            // the same for every thread of the CTA
  if (small) { for (int i = tid; i < 256; i += kBrThreads) sh.bins[i] = 0; }
  else { for (int i = tid; i < 128 * 32; i += kBrThreads) sh.lanes[i] = 0; }     // (while the loads are in flight)
  for (int i = tid; i < 512; i += kBrThreads) sh.low[i] = 0;
  // ranks (1-based, among the sampled keys; the pad counts as -inf keys) whose keys become the bounds
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
  __syncthreads();
  // ---- level 1
  if (small) {
    // a sample of at most 2048 keys: plain atomics on the 256 bins queue little, and nothing has to be folded
    for (int u = 0; u < 2; ++u) {
      if (u >= have) break;
      const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        uint32_t h0 = w[j] & 0xffffu, h1 = w[j] >> 16;
        if (h0 == 0x8000u) h0 = 0u;
        if (h1 == 0x8000u) h1 = 0u;
        atomicAdd(&sh.bins[ord_hi(h0 >> 8)], 1u);
        atomicAdd(&sh.bins[ord_hi(h1 >> 8)], 1u);
      }
    }
  } else {
#pragma unroll
  for (int u = 0; u < NV; ++u) {
    if (u >= have) break;
    const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t h0 = w[j] & 0xffffu, h1 = w[j] >> 16;
      if (h0 == 0x8000u) h0 = 0u;                          // -0 counts as +0
      if (h1 == 0x8000u) h1 = 0u;
      atomicAdd(&sh.lanes[(h0 >> 9) * 32 + lane], 1u << ((h0 >> 4) & 16u));
      atomicAdd(&sh.lanes[(h1 >> 9) * 32 + lane], 1u << ((h1 >> 4) & 16u));
    }
  }
  }
  __syncthreads();
  if (!small) {
    // thread t sums word row t (raw high bytes 2t, 2t+1) over the lanes, starting at its own lane: no conflicts
    uint32_t acc = 0;
    const uint32_t* wrow = &sh.lanes[tid * 32];
#pragma unroll 8
    for (int l = 0; l < 32; ++l) acc += wrow[(l + lane) & 31];
    sh.bins[ord_hi(2u * tid)] = acc & 0xffffu;
    sh.bins[ord_hi(2u * tid + 1u)] = acc >> 16;
  }
  __syncthreads();
  if (warp < 2) {                                          // warp 0: the lower bound's rank, warp 1: the upper one's
    const uint32_t rank = warp == 0 ? rank_lo : rank_hi;
    int bin = 0;
    uint32_t up = 0;
    if (rank) warp_find_bin256(sh.bins, rank, lane, bin, up);
    if (lane == 0) { sh.bin[warp] = bin; sh.above[warp] = up; }
  }
  __syncthreads();
  // ---- level 2
  const uint32_t bin_lo = (uint32_t)sh.bin[0], bin_hi = rank_hi ? (uint32_t)sh.bin[1] : bin_lo;
  const uint32_t up_lo = sh.above[0], up_hi = sh.above[1];
  const bool two = bin_hi != bin_lo;
  {
    // codes below 0x8000 are negative numbers: their raw bits run the other way
    const uint32_t raw_lo = bin_lo < 0x80u ? 0xffu - bin_lo : bin_lo - 0x80u, flip_lo = bin_lo < 0x80u ? 0xffu : 0u;
    const uint32_t raw_hi = bin_hi < 0x80u ? 0xffu - bin_hi : bin_hi - 0x80u, flip_hi = bin_hi < 0x80u ? 0xffu : 0u;
#pragma unroll
    for (int u = 0; u < NV; ++u) {
      if (u >= have) break;
      const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
#pragma unroll
        for (int e2 = 0; e2 < 2; ++e2) {
          uint32_t h = e2 ? (w[j] >> 16) : (w[j] & 0xffffu);
          if (h == 0x8000u) h = 0u;
          if ((h >> 8) == raw_lo) atomicAdd(&sh.low[(h & 255u) ^ flip_lo], 1u);
          else if (two && (h >> 8) == raw_hi) atomicAdd(&sh.low[256u + ((h & 255u) ^ flip_hi)], 1u);
        }
      }
    }
  }
  __syncthreads();
  if (warp < 2) {
    const uint32_t rank = warp == 0 ? rank_lo : rank_hi;
    const uint32_t up = warp == 0 ? up_lo : up_hi;
    int bin = 0;
    uint32_t dummy = 0;
    if (rank) warp_find_bin256(warp == 1 && two ? sh.low + 256 : sh.low, rank - up, lane, bin, dummy);
    if (lane == 0) sh.bin[warp] = bin;
  }
  __syncthreads();
  if (tid == 0) {
    const uint32_t code_lo = (bin_lo << 8) | (uint32_t)sh.bin[0], code_hi = (bin_hi << 8) | (uint32_t)sh.bin[1];
    // two codes of slack either side: the sweep compares fp32 logits, the sample held their roundings
    RowBracket b;
    b.lo = (rank_lo && code_lo >= 0x0402u) ? float_of_code(code_lo - 2u) : -INFINITY;
    b.hi = (rank_hi && code_hi + 2u <= 0xfbffu) ? float_of_code(code_hi + 2u) : INFINITY;
    bracket[rowid] = b;
  }
}

// ------------------------------------------------------------------------------------ resolve
constexpr int kRowThreads = 256;

struct ResolveShared {
  uint32_t hist[256];
  uint32_t red[2][kRowThreads / 32];
  uint32_t seg_off[kRowThreads / 32];   // scan scratch  (sized for the larger of the two CTA sizes)
  uint32_t total_above, total_cand, overflow;
  uint32_t kmin, kmax;
  int bin;
  uint32_t above;
};

// After the sweep: the row's k - #above largest listed candidates, by (fp32 logit descending, key index
// ascending), into the tentative mask.  The candidates of a row sit in `segs` segments (one per writer of
// the sweep); their order-preserving 32-bit images are gathered into shared memory and the threshold is
// found by a most-significant-digit radix search over them (256 bins per pass, starting at the first bit
// in which the images differ); integer counts only, so two runs give the same bits.
// NT threads per CTA: 256 for long rows, 64 where a row lists at most a couple of thousand candidates (a
// batch of short requests has many rows and little work in each: what counts there is CTAs per SM).
template <int NT>
__global__ void __launch_bounds__(NT)
resolve_kernel(const int32_t* __restrict__ cu, int Hq, int G, int S, const int32_t* __restrict__ b_step,
               const VoteState vs, int smem_keys, int64_t row_words, const int32_t* __restrict__ kv_len) {
  extern __shared__ __align__(16) uint32_t dyn[];         // [seg offsets: segs + 1][keys: smem_keys]
  __shared__ ResolveShared sh;
  const int r = blockIdx.z, g = blockIdx.y, s = blockIdx.x;
  const int rowid = (r * Hq + g) * S + s;
  const int start = cu[r], Ncap = cu[r + 1] - start;
  const int kh = g / G, Hkv = Hq / G;
  const int N = valid_keys(kv_len, r, Hkv, kh, Ncap);
  if (N <= 0) return;
  const int k = min(b_step[r * Hq + g], N);
  if (k <= 0) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int segs = vs.lay.segs, seg_cap = vs.lay.seg_cap(Ncap);
  uint32_t* seg_off = dyn;                                 // exclusive prefix of the segments' counts
  uint32_t* keys = dyn + segs + 1;
  if (tid == 0) { sh.total_above = 0; sh.overflow = 0; sh.kmin = 0xffffffffu; sh.kmax = 0u; }
  __syncthreads();
  // what the sweep's writers met: totals, overflow of any segment, and where each segment's keys go
  {
    const uint2* st = vs.segstat + (int64_t)rowid * segs;
    uint32_t run = 0;                                      // candidates in the segments before this round
    for (int base = 0; base < segs; base += NT) {
      const int i = base + tid;
      const uint2 v = i < segs ? st[i] : make_uint2(0u, 0u);
      if (v.y > (uint32_t)seg_cap) sh.overflow = 1u;
      const uint32_t a = __reduce_add_sync(0xffffffffu, v.x);
      if (lane == 0 && a) atomicAdd(&sh.total_above, a);
      uint32_t inc = v.y;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
      }
      if (lane == 31) sh.seg_off[warp] = inc;
      __syncthreads();
      uint32_t before = run, all = 0;
#pragma unroll
      for (int w = 0; w < NT / 32; ++w) { if (w < warp) before += sh.seg_off[w]; all += sh.seg_off[w]; }
      if (i < segs) seg_off[i] = before + inc - v.y;
      run += all;
      __syncthreads();
    }
    if (tid == 0) { seg_off[segs] = run; sh.total_cand = run; }
    __syncthreads();
  }
  const uint32_t A = sh.total_above, C = sh.total_cand;
  if (sh.overflow || A > (uint32_t)k || A + C < (uint32_t)k || ((uint32_t)k > A && C > (uint32_t)smem_keys)) {
    // the bracket missed or a list overflowed: the head goes the exact way (counted once per head)
    if (tid == 0 && atomicExch(&vs.head_bad[r * Hkv + kh], 1u) == 0u) atomicAdd(&vs.status[2], 1);
    return;
  }
  const uint32_t need = (uint32_t)k - A;
  if (need == 0) return;
  const uint2* list = vs.list(g, s, S, start, r);
  uint32_t* mrow = vs.tmask + (int64_t)kh * row_words + mask_word_offset(start, r);
  // one warp per segment, a lane per entry
  if (need == C) {                                         // every listed key is taken
    for (int sg = warp; sg < segs; sg += NT / 32) {
      const uint32_t cnt = seg_off[sg + 1] - seg_off[sg];
      for (uint32_t i = lane; i < cnt; i += 32) {
        const uint32_t n = list[(int64_t)sg * seg_cap + i].y;
        atomicOr(&mrow[n >> 5], 1u << (n & 31));
      }
    }
    return;
  }
  // Entry e of the row's candidates in list order: segment sg holds entries seg_off[sg] .. seg_off[sg+1]-1.
  // A thread finds the segment of its entry by bisection over the offsets, so that the loads of all its
  // entries are independent and in flight together.
  auto entry_of = [&](uint32_t e) -> const uint2* {
    int a = 0, b = segs;                                   // seg_off[a] <= e < seg_off[b]
    while (b - a > 1) {
      const int mid = (a + b) >> 1;
      if (seg_off[mid] <= e) a = mid; else b = mid;
    }
    return list + (int64_t)a * seg_cap + (e - seg_off[a]);
  };
  // gather the order-preserving images of the listed logits; the key indices of the first kHold rounds stay
  // in registers for the emission below (a row of the usual length is all of them: no second trip to the lists)
  constexpr int kHold = 3;
  uint32_t held[kHold][4];
  auto gather_round = [&](uint32_t base, uint32_t* hy, uint32_t& mn, uint32_t& mx) {
    uint2 ent[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint32_t e = base + u * NT + tid;
      ent[u] = e < C ? *entry_of(e) : make_uint2(0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint32_t e = base + u * NT + tid;
      if (hy) hy[u] = ent[u].y;
      if (e < C) {
        const uint32_t kx = ordered_key(__uint_as_float(ent[u].x));
        keys[e] = kx;
        mn = min(mn, kx);
        mx = max(mx, kx);
      }
    }
  };
  {
    uint32_t mn = 0xffffffffu, mx = 0u;
#pragma unroll
    for (int b = 0; b < kHold; ++b)
      if ((uint32_t)(b * 4 * NT) < C) gather_round((uint32_t)(b * 4 * NT), held[b], mn, mx);
    for (uint32_t base = kHold * 4 * NT; base < C; base += 4 * NT) gather_round(base, nullptr, mn, mx);
    mn = __reduce_min_sync(0xffffffffu, mn);
    mx = __reduce_max_sync(0xffffffffu, mx);
    if (lane == 0) { atomicMin(&sh.kmin, mn); atomicMax(&sh.kmax, mx); }
  }
  __syncthreads();
  // radix search for the need-th largest image, from the first bit in which the extremes differ
  uint32_t prefix = 0, known = 0, acc = 0;                 // acc: keys above the prefix found so far
  uint32_t eq = 0;
  bool whole_bin = false;                                  // every key of the last bin found is taken
  {
    const uint32_t diff = sh.kmin ^ sh.kmax;
    int top = diff ? 31 - __clz(diff) : -1;
    if (top < 31) { known = top < 0 ? 0xffffffffu : ~((2u << top) - 1u); prefix = sh.kmax & known; }
    if (top < 0) { eq = C; }
    while (top >= 0) {
      const int lo_bit = top >= 7 ? top - 7 : 0;
      const uint32_t digit_mask = (top - lo_bit == 31) ? 0xffffffffu : (((2u << (top - lo_bit)) - 1u));
      for (int i = tid; i < 256; i += NT) sh.hist[i] = 0;
      __syncthreads();
      for (uint32_t i = tid; i < C; i += NT) {
        const uint32_t x = keys[i];
        if ((x & known) == prefix) atomicAdd(&sh.hist[(x >> lo_bit) & digit_mask], 1u);
      }
      __syncthreads();
      if (warp == 0) {
        int bin;
        uint32_t up;
        warp_find_bin256(sh.hist, need - acc, lane, bin, up);
        if (lane == 0) { sh.bin = bin; sh.above = up; }
      }
      __syncthreads();
      const uint32_t bin = (uint32_t)sh.bin;
      acc += sh.above;
      eq = sh.hist[bin];
      prefix |= bin << lo_bit;
      known |= digit_mask << lo_bit;
      __syncthreads();
      if (eq == need - acc) { whole_bin = true; break; }   // the bin is taken whole: no finer digit needed
      top = lo_bit - 1;
    }
  }
  // keys above the bin found are taken; of the bin's keys either all (whole_bin, or all equal images needed)
  // or, when its keys are equal images and more than needed, the `ties` lowest key indices
  const uint32_t ties = need - acc;                        // 1 <= ties <= eq
  uint32_t idx_max = 0xffffffffu;
  if (!whole_bin && ties < eq) {
    // largest v with #(equal image, index < v) < ties, bit by bit: the ties-th lowest index among them
    uint32_t vlim = 0;
    for (int bit = 31 - __clz(max(N - 1, 1)); bit >= 0; --bit) {
      const uint32_t trial = vlim | (1u << bit);
      uint32_t c = 0;
      for (int sg = warp; sg < segs; sg += NT / 32) {
        const uint32_t o = seg_off[sg], cnt = seg_off[sg + 1] - o;
        for (uint32_t i = lane; i < cnt; i += 32)
          c += (keys[o + i] == prefix && list[(int64_t)sg * seg_cap + i].y < trial) ? 1u : 0u;
      }
      c = __reduce_add_sync(0xffffffffu, c);
      uint32_t* row = sh.red[bit & 1];
      if (lane == 0) row[warp] = c;
      __syncthreads();
      uint32_t tot = 0;
#pragma unroll
      for (int w = 0; w < NT / 32; ++w) tot += row[w];
      if (tot < ties) vlim = trial;
    }
    idx_max = vlim;
  }
  const bool all_of_bin = whole_bin || ties >= eq;
  auto emit_round = [&](uint32_t base, const uint32_t* hy) {
    uint32_t n[4];
    bool want[4], tie[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint32_t e = base + u * NT + tid;
      const uint32_t x = e < C ? keys[e] : 0u;
      const bool in_bin = e < C && (x & known) == prefix;
      want[u] = e < C && (x > (prefix | ~known) || (in_bin && all_of_bin));
      tie[u] = in_bin && !all_of_bin;
      n[u] = hy ? hy[u] : ((want[u] || tie[u]) ? entry_of(e)->y : 0u);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (want[u] || (tie[u] && n[u] <= idx_max)) atomicOr(&mrow[n[u] >> 5], 1u << (n[u] & 31));
  };
#pragma unroll
  for (int b = 0; b < kHold; ++b)
    if ((uint32_t)(b * 4 * NT) < C) emit_round((uint32_t)(b * 4 * NT), held[b]);
  for (uint32_t base = kHold * 4 * NT; base < C; base += 4 * NT) emit_round(base, nullptr);
}

// ------------------------------------------------------------------------------------ commit
// The exact fp32 logits of one row, computed where they are needed.
struct ExactRow {
  DotCtx dot;
  __device__ __forceinline__ float operator()(int n) const { return dot(n); }
};

// Grid: (row s, query head of the group, z).  CTA z walks the (request, KV head) pairs z, z + gridDim.z, ...:
// a large batch would otherwise launch a CTA per row of every head only to find the head settled.  copy_good:
// the tentative mask of a settled head is OR-ed into the keep mask here (the head's G * S CTAs a slice each);
// when the pruning step follows, its mask scan does that on its way over the words and the CTAs of settled
// heads have nothing to do.
__global__ void __launch_bounds__(kRowThreads)
commit_kernel(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K, int64_t k_tok, int64_t k_head,
              const int32_t* __restrict__ cu, int Hq, int G, int S, int d_k, float scale,
              const int32_t* __restrict__ b_step, const uint32_t* __restrict__ tmask, int64_t row_words,
              uint32_t* __restrict__ mask, const uint32_t* __restrict__ head_bad, const int32_t* __restrict__ kv_len,
              int n_pairs, int copy_good) {
  __shared__ SelShared sh;
  __shared__ __align__(16) __nv_bfloat16 qf[512];
  const int s = blockIdx.x, gl = blockIdx.y;
  const int Hkv = Hq / G;
  const int tid = threadIdx.x;
  const int step = (int)gridDim.z;
  for (int base = (int)blockIdx.z; base < n_pairs; base += 32 * step) {
    // which of the next (up to) 32 pairs of this CTA's walk need work: the flags are fetched together
    uint32_t todo = 0;
#pragma unroll 8
    for (int i = 0; i < 32; ++i) {
      const int pair = base + i * step;
      if (pair < n_pairs && (copy_good || head_bad[pair])) todo |= 1u << i;
    }
    while (todo) {
      const int i = __ffs(todo) - 1;
      todo &= todo - 1;
      const int pair = base + i * step;
      const int r = pair / Hkv, kh = pair % Hkv, g = kh * G + gl;
      const int start = cu[r], Ncap = cu[r + 1] - start;
      const int64_t woff = (int64_t)kh * row_words + mask_word_offset(start, r);
      if (!head_bad[pair]) {
        // (copy_good) the G * S rows of the head share the copy of its words
        const int words = (Ncap + 31) >> 5;
        const int idx = gl * S + s;
        for (int w = idx * kRowThreads + tid; w < words; w += G * S * kRowThreads) {
          const uint32_t v = tmask[woff + w];
          if (v) mask[woff + w] |= v;
        }
        continue;
      }
      // a bracket of this head missed: this row again, exactly
      const int N = valid_keys(kv_len, r, Hkv, kh, Ncap);
      const int k = N > 0 ? min(b_step[r * Hq + g], N) : 0;
      if (k <= 0) continue;
      const int grow = gl * S + s;
      const __nv_bfloat16* qrow = Q + (((int64_t)r * Hkv + kh) * (G * (S + 1)) + grow) * d_k;
      __syncthreads();                                     // the row before this one is through with qf and sh
      for (int c = tid; c < d_k; c += kRowThreads) qf[c] = qrow[c];
      __syncthreads();
      ExactRow row{DotCtx{qf, K + (int64_t)kh * k_head + (int64_t)start * k_tok, k_tok, d_k, scale}};
      uint32_t t, above_cnt, eq_cnt;
      unsigned long long above_mass;
      radix_threshold<false>(row, N, 0.f, (unsigned long long)k, sh, t, above_cnt, above_mass, eq_cnt);
      emit_row(row, N, t, (uint32_t)k - above_cnt, eq_cnt, mask + woff, sh);
    }
  }
}

}  // namespace

// The three launchers: before the sweep, after it, and the commit.
int32_t launch_bracket(const gvote_params* p, const int32_t* cu, int32_t batch, int64_t max_N, const int32_t* b_step,
                       const VoteState& vs, const int32_t* kv_len, cudaStream_t st) {
  const int Hq = p->n_q_heads, G = Hq / p->n_kv_heads;
  dim3 grid(p->S, Hq, batch);
  {
    LaunchScope scope_("bracket_kernel", st);
    if (sample_geom((int)max_N).ns * 16 <= 4 * kBrThreads)
      launch_on(bracket_kernel<4>, grid, dim3(kBrThreads), 0, st, vs.sample, vs.sample_slots, cu, Hq, G, p->S,
                 score_geometry(p).row_chunks, b_step, vs.bracket, kv_len);
    else
      launch_on(bracket_kernel<16>, grid, dim3(kBrThreads), 0, st, vs.sample, vs.sample_slots, cu, Hq, G, p->S,
                 score_geometry(p).row_chunks, b_step, vs.bracket, kv_len);
  }
  GVOTE_LAUNCH_CHECK("bracket_kernel");
  return GVOTE_OK;
}

int32_t launch_resolve(const gvote_params* p, const int32_t* cu, int32_t batch, int64_t max_N, const int32_t* b_step,
                       const VoteState& vs, int64_t row_words, const int32_t* kv_len, cudaStream_t st) {
  const int Hq = p->n_q_heads, G = Hq / p->n_kv_heads;
  dim3 grid(p->S, Hq, batch);
  // shared memory: the segments' offsets and the images of the listed keys.  Room for twice the keys a
  // row is expected to list at most, within 160 KB; a row that lists more goes the exact way.
  (void)max_N;
  int64_t cap_all = (int64_t)vs.lay.segs * (vs.lay.uniform_seg_cap > 0 ? vs.lay.uniform_seg_cap : vs.lay.seg_cap((int)max_N));
  if (cap_all > 40000) cap_all = 40000;
  const int smem_keys = (int)cap_all;
  const size_t smem = ((size_t)vs.lay.segs + 1 + (size_t)smem_keys) * sizeof(uint32_t);
  if (smem > 48 * 1024)
    GVOTE_CUDA_CHECK(cudaFuncSetAttribute(resolve_kernel<kRowThreads>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  {
    LaunchScope scope_("resolve_kernel", st);
    if (smem_keys <= 4096)
      launch_on(resolve_kernel<64>, grid, dim3(64), smem, st, cu, Hq, G, p->S, b_step, vs, smem_keys, row_words, kv_len);
    else
      launch_on(resolve_kernel<kRowThreads>, grid, dim3(kRowThreads), smem, st, cu, Hq, G, p->S, b_step, vs, smem_keys, row_words, kv_len);
  }
  GVOTE_LAUNCH_CHECK("resolve_kernel");
  return GVOTE_OK;
}

int32_t launch_commit(const gvote_params* p, const __nv_bfloat16* Q, const __nv_bfloat16* K, int64_t k_tok, int64_t k_head,
                      const int32_t* cu, int32_t batch, const int32_t* b_step, const VoteState& vs, int64_t row_words,
                      uint32_t* mask, const int32_t* kv_len, bool copy_good, cudaStream_t st) {
  const int Hq = p->n_q_heads, G = Hq / p->n_kv_heads;
  // about two thousand CTAs at most: each walks its share of the (request, KV head) pairs
  const int64_t pairs = (int64_t)batch * p->n_kv_heads;
  int64_t z = 2048 / ((int64_t)p->S * G);
  z = z < 1 ? 1 : (z > pairs ? pairs : z);
  dim3 grid(p->S, G, (unsigned)z);
  const float scale = (float)(1.0 / sqrt((double)p->d_k));
  {
    LaunchScope scope_("commit_kernel", st);
    launch_on(commit_kernel, grid, dim3(kRowThreads), 0, st, Q, K, k_tok, k_head, cu, Hq, G, p->S, p->d_k, scale, b_step, vs.tmask,
              row_words, mask, vs.head_bad, kv_len, (int)pairs, copy_good ? 1 : 0);
  }
  GVOTE_LAUNCH_CHECK("commit_kernel");
  return GVOTE_OK;
}

}  // namespace gvote
