// Algorithm 1, the TopK step for the synthetic queries: the k = |C0| largest logits of a row, found on the
// 16-bit keys the tensor-core score kernel leaves behind (each logit rounded to half precision), and
// OR-ed into the head's keep mask (the union step).
//
// One small CTA per synthetic row, many resident per SM.  Keys are compared as half-precision numbers,
// two per instruction; for counting they are mapped to an order-preserving 16-bit code.
//   1. A fixed sample of 4096 keys (128 evenly spaced runs of 32) brackets the k-th largest key between two of
//      the sample's order statistics, a few standard deviations of the sampling error either side of
//      the expected rank.  (Rows of at most 4096 keys are sampled completely, which settles the
//      threshold at once.)
//   2. One sweep over the row marks, in a shared-memory bit row, every key above the bracket, counts
//      them, and lists the keys inside the bracket (every thread in a list of its own).  If the bracket holds (#above <= k <= #above +
//      #listed, and the list fits), the k - #above largest listed keys are found inside the list with
//      a two-level histogram and marked too; the bit row is then OR-ed into the mask.
//   3. Keys that share the 16-bit threshold value T round to the same half-precision number, so their
//      order is settled exactly: their logits are recomputed in fp32 from Q and K and ranked by (value
//      descending, index ascending); the first k - #above-T of them are selected.
//   4. If the bracket misses or the list overflows (rare), nothing has been written yet and the row
//      takes the slower exact route: window sweeps that count the keys above a window of codes and
//      histogram the keys inside it in 2048 bins (a window wider than 2048 codes is narrowed to the
//      bin that holds T and swept again), then an emission sweep.
// Sweeps test eight keys with four compare instructions and skip vectors with nothing of interest.
#include <cuda_fp16.h>

#include "common.cuh"

namespace gvote {
namespace {

constexpr int kThreads = 128;
constexpr int kWin = 2048;              // codes per histogram window
constexpr int kTieCap = 256;
constexpr int kOvfCap = 384;            // bracket keys that did not fit their thread's list
constexpr int kSampleRound = kThreads * 4;   // sample vectors per round (four per thread): at least one round
constexpr int kTileKeys = 128;
constexpr int kLoads = 4;               // 16-byte loads in flight per thread
constexpr uint32_t kPadKey = 0xfc00u;   // -inf: what positions past the end of a row read as
constexpr uint32_t kMinCode = 0x0400u;  // code of the most negative finite half: no key lies below it

// Half bits -> code whose unsigned order is the numeric order (-0 and +0 share a code), and back.
__device__ __forceinline__ uint32_t code_of(uint32_t h) {
  if (h == 0x8000u) h = 0u;
  return (h & 0x8000u) ? (~h & 0xffffu) : (h | 0x8000u);
}
__device__ __forceinline__ uint32_t raw_of(uint32_t c) { return (c & 0x8000u) ? (c & 0x7fffu) : (~c & 0xffffu); }
__device__ __forceinline__ __half2 pair_of(uint32_t raw) {
  const uint32_t p = raw | (raw << 16);
  return *reinterpret_cast<const __half2*>(&p);
}
__device__ __forceinline__ __half2 as_h2(uint32_t w) { return *reinterpret_cast<const __half2*>(&w); }
// No key has code 0x7fff (it is -0's slot), and as a bound it would turn into -0, which compares
// equal to +0: bounds step over it.
__device__ __forceinline__ uint32_t fix_lo(uint32_t c) { return c == 0x7fffu ? 0x8000u : c; }
__device__ __forceinline__ uint32_t fix_hi(uint32_t c) { return c == 0x7fffu ? 0x7ffeu : c; }

struct Sel16Shared {
  uint32_t hist[kWin];
  __nv_bfloat16 qf[512];
  int tie_idx[kTieCap];
  float tie_val[kTieCap];
  uint32_t red[kThreads / 32];
  uint32_t red2[kThreads / 32];
  int bin;
  uint32_t above;
  uint32_t inside;
  int bin2;              // second search of a pair (sample_ranks)
  uint32_t above2;
  uint32_t ntie;
  uint32_t novf;
  uint32_t ovf_n[kOvfCap];
  uint16_t ovf_key[kOvfCap];
};

__device__ __forceinline__ uint32_t block_sum(Sel16Shared& sh, uint32_t v) {
  v = (uint32_t)warp_sum_i((int)v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) sh.red[threadIdx.x >> 5] = v;
  __syncthreads();
  uint32_t s = 0;
#pragma unroll
  for (int w = 0; w < kThreads / 32; ++w) s += sh.red[w];
  return s;
}

// Two sums over the CTA behind one pair of barriers.
__device__ __forceinline__ void block_sum2(Sel16Shared& sh, uint32_t v0, uint32_t v1, uint32_t& s0, uint32_t& s1) {
  v0 = (uint32_t)warp_sum_i((int)v0);
  v1 = (uint32_t)warp_sum_i((int)v1);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) { sh.red[threadIdx.x >> 5] = v0; sh.red2[threadIdx.x >> 5] = v1; }
  __syncthreads();
  s0 = 0;
  s1 = 0;
#pragma unroll
  for (int w = 0; w < kThreads / 32; ++w) { s0 += sh.red[w]; s1 += sh.red2[w]; }
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

// The same for the whole CTA on 256 bins in shared memory: publishes sh.bin and sh.above.
__device__ void find_bin256(Sel16Shared& sh, const uint32_t* hist, uint32_t need) {
  if (threadIdx.x < 32) {
    int bin;
    uint32_t above;
    warp_find_bin256(hist, need, threadIdx.x, bin, above);
    if (threadIdx.x == 0) { sh.bin = bin; sh.above = above; }
  }
  __syncthreads();
}

// The sample: vector i of `n_vecs` (at most four per thread).  A row of at most n_vecs vectors is
// sampled completely (stride 0).  Otherwise the sample is kThreads runs of four consecutive vectors
// (64 bytes, one DRAM access each; scattering single 16-byte vectors instead costs four times the
// accesses for the same number of keys), run j taken from the middle of the j-th of kThreads equal
// stretches of the row.  Four neighbouring lanes share a run, so a warp's load instruction asks for
// eight 64-byte pieces instead of thirty-two 16-byte ones.
struct Sample {
  int n_vecs, stride;
  __device__ __forceinline__ int vec(int i) const {
    if (stride == 0) return i;
    const int t = i % kThreads, u = i / kThreads;
    const int run = (t >> 2) + (kThreads / 4) * u;
    return run * stride + ((stride >> 1) & ~3) + (t & 3);
  }
};

// Exact fp32 logit of key n for this row's query (fixed summation order).
struct DotCtx {
  const __nv_bfloat16* qf;
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

// Where a row's keys live: eight consecutive keys form one 16-byte vector; vector v8 of the row sits in
// tile v8 / 16, at chunk position (v8 % 16) ^ swz of the row's 16 chunks there (the score kernel stores
// its tiles XOR-swizzled by the row number, swz = row % 16).  Positions >= N read as -inf.
struct RowView {
  const uint16_t* grow;         // first tile of the row in global memory
  int64_t tile_stride;          // elements between consecutive tiles of the same row
  int N, nv8;
  uint32_t swz;
  __device__ __forceinline__ uint4 load(int v8) const {
    if (v8 >= nv8) return make_uint4(0xfc00fc00u, 0xfc00fc00u, 0xfc00fc00u, 0xfc00fc00u);
    uint4 v = *reinterpret_cast<const uint4*>(grow + (int64_t)(v8 >> 4) * tile_stride + (((uint32_t)v8 & 15u) ^ swz) * 8);
    if (v8 * 8 + 8 > N) {
      uint16_t* e = reinterpret_cast<uint16_t*>(&v);
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (v8 * 8 + j >= N) e[j] = (uint16_t)kPadKey;
    }
    return v;
  }
  __device__ __forceinline__ uint32_t key_at(int n) const {
    return grow[(int64_t)(n >> 7) * tile_stride + (((((uint32_t)n & 127u) >> 3) ^ swz) << 3) + (n & 7)];
  }
};

// The sampled vectors of this thread (those past the sample read as -inf and are not counted).
struct SampleRegs {
  uint4 v[4];
  int have;
};
__device__ __forceinline__ SampleRegs sample_load(const RowView& rv, const Sample& sm) {
  SampleRegs sr;
  sr.have = 0;
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const int i = u * kThreads + (int)threadIdx.x;
    sr.v[u] = rv.load(i < sm.n_vecs ? sm.vec(i) : rv.nv8);
    if (i < sm.n_vecs) sr.have = u + 1;
  }
  return sr;
}

// High byte of a key's code from the high byte hb of its half bits, and back.
__device__ __forceinline__ uint32_t ord_hi(uint32_t hb) { return hb >= 0x80u ? 0xffu - hb : 0x80u + hb; }

// Clears the counters sample_ranks starts from.  Called between issuing the sample's loads and
// ranking it, so that the clearing and its barrier pass while the loads are in flight.
__device__ __forceinline__ void sample_begin(Sel16Shared& sh) {
  for (int b = threadIdx.x; b < kWin; b += kThreads) sh.hist[b] = 0;
  __syncthreads();
}

// The sample's rank_a-th and rank_b-th largest codes (1 <= rank_a <= rank_b <= sampled keys; rank_a = 0
// asks for the second one only).  For the second one also the number of sampled codes above it and
// equal to it.  Every thread of the CTA calls it, after sample_begin.
//
// Two levels of 256 bins, both ranks at a time (warp 0 searches for rank_b, warp 1 for rank_a).
// Level 1 bins the code's high byte.  Every sampled key takes part and a few bins take most of
// them, so plain shared-memory atomics would serialise on those addresses: counting goes into one
// 8-bit counter per (bin, lane) instead, four bins to a word, word index (bin / 4) * 32 + lane: the
// lanes of a warp never meet, and a counter takes at most (warps) * (sample keys per thread) = 4 * 32
// increments, well below 256.  Bins are those of the raw half bits here (no per-key recoding); the
// fold puts them in code order, into the tie list's space (not in use yet).  Level 2 bins the low
// byte of the keys whose high byte is the one found, for the two ranks side by side.
__device__ void sample_ranks(const SampleRegs& sr, uint32_t rank_a, uint32_t rank_b, Sel16Shared& sh,
                             uint32_t& code_a, uint32_t& code_b, uint32_t& above_b, uint32_t& equal_b) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t* bins = reinterpret_cast<uint32_t*>(sh.tie_val);
  static_assert(kTieCap >= 256, "the folded bins borrow the tie list");
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    if (u >= sr.have) break;
    const uint32_t w[4] = {sr.v[u].x, sr.v[u].y, sr.v[u].z, sr.v[u].w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t h0 = w[j] & 0xffffu, h1 = w[j] >> 16;
      if (h0 == 0x8000u) h0 = 0u;                        // -0 counts as +0
      if (h1 == 0x8000u) h1 = 0u;
      atomicAdd(&sh.hist[(h0 >> 10) * 32 + lane], 1u << ((h0 >> 5) & 24u));
      atomicAdd(&sh.hist[(h1 >> 10) * 32 + lane], 1u << ((h1 >> 5) & 24u));
    }
  }
  __syncthreads();
  // fold the lanes: thread t < 64 sums word row t (raw bins 4t .. 4t+3), two bins per accumulator
  if (tid < 64) {
    uint32_t even = 0, odd = 0;
    const uint32_t* wrow = &sh.hist[tid * 32];
#pragma unroll 8
    for (int l = 0; l < 32; ++l) {
      const uint32_t w = wrow[(l + lane) & 31];           // rotated: conflict free
      even += w & 0x00ff00ffu;
      odd += (w >> 8) & 0x00ff00ffu;
    }
    const uint32_t hb = 4u * tid;
    bins[ord_hi(hb)] = even & 0xffffu;
    bins[ord_hi(hb + 1)] = odd & 0xffffu;
    bins[ord_hi(hb + 2)] = even >> 16;
    bins[ord_hi(hb + 3)] = odd >> 16;
  }
  __syncthreads();
  if (warp == 0) {
    int bin;
    uint32_t up;
    warp_find_bin256(bins, rank_b, lane, bin, up);
    if (lane == 0) { sh.bin = bin; sh.above = up; }
  } else if (warp == 1 && rank_a) {
    int bin;
    uint32_t up;
    warp_find_bin256(bins, rank_a, lane, bin, up);
    if (lane == 0) { sh.bin2 = bin; sh.above2 = up; }
  }
  for (int b = tid; b < 512; b += kThreads) sh.hist[b] = 0;      // level 2: [0, 256) for rank_b, [256, 512) for rank_a
  __syncthreads();
  const uint32_t bin_b = (uint32_t)sh.bin, up_b = sh.above;
  const uint32_t bin_a = rank_a ? (uint32_t)sh.bin2 : bin_b, up_a = rank_a ? sh.above2 : 0u;
  const bool two = rank_a && bin_a != bin_b;
  {
    // codes below 0x8000 are negative numbers: their raw bits run the other way
    const uint32_t raw_b = bin_b < 0x80u ? 0xffu - bin_b : bin_b - 0x80u, flip_b = bin_b < 0x80u ? 0xffu : 0u;
    const uint32_t raw_a = bin_a < 0x80u ? 0xffu - bin_a : bin_a - 0x80u, flip_a = bin_a < 0x80u ? 0xffu : 0u;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (u >= sr.have) break;
      const uint32_t w[4] = {sr.v[u].x, sr.v[u].y, sr.v[u].z, sr.v[u].w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          uint32_t h = e ? (w[j] >> 16) : (w[j] & 0xffffu);
          if (h == 0x8000u) h = 0u;
          if ((h >> 8) == raw_b) atomicAdd(&sh.hist[(h & 255u) ^ flip_b], 1u);
          else if (two && (h >> 8) == raw_a) atomicAdd(&sh.hist[256u + ((h & 255u) ^ flip_a)], 1u);
        }
      }
    }
  }
  __syncthreads();
  if (warp == 0) {
    int bin;
    uint32_t up;
    warp_find_bin256(sh.hist, rank_b - up_b, lane, bin, up);
    if (lane == 0) { sh.bin = bin; sh.above = up; sh.inside = sh.hist[bin]; }
  } else if (warp == 1 && rank_a) {
    int bin;
    uint32_t up;
    warp_find_bin256(two ? sh.hist + 256 : sh.hist, rank_a - up_a, lane, bin, up);
    if (lane == 0) sh.bin2 = bin;
  }
  __syncthreads();
  code_b = (bin_b << 8) | (uint32_t)sh.bin;
  above_b = up_b + sh.above;
  equal_b = sh.inside;
  code_a = rank_a ? ((bin_a << 8) | (uint32_t)sh.bin2) : 0xffffu;
}

// One sweep: A = number of keys with code > hi; hist[(c - lo) >> shift] = number of keys with code c
// in [lo, hi] ((hi - lo) >> shift < kWin).  Neither bound is 0x7fff.
__device__ uint32_t window_pass(const RowView& rv, uint32_t lo, uint32_t hi, int shift, Sel16Shared& sh) {
  for (int b = threadIdx.x; b < kWin; b += kThreads) sh.hist[b] = 0;
  __syncthreads();
  const __half2 tlo = pair_of(raw_of(lo)), thi = pair_of(raw_of(hi));
  uint32_t a16 = 0;   // 16 per key above the window
  for (int base = 0; base < rv.nv8; base += kThreads * kLoads) {
    uint4 buf[kLoads];
#pragma unroll
    for (int u = 0; u < kLoads; ++u) buf[u] = rv.load(base + u * kThreads + (int)threadIdx.x);
#pragma unroll
    for (int u = 0; u < kLoads; ++u) {
      const uint32_t w[4] = {buf[u].x, buf[u].y, buf[u].z, buf[u].w};
      uint32_t ge[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) ge[j] = __hge2_mask(as_h2(w[j]), tlo);
      if ((ge[0] | ge[1] | ge[2] | ge[3]) == 0u) continue;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t gt = __hgt2_mask(as_h2(w[j]), thi);
        a16 += __popc(gt);
        const uint32_t in = ge[j] & ~gt;
        if (in & 0xffffu) {
          const uint32_t b = (code_of(w[j] & 0xffffu) - lo) >> shift;
          if (b < (uint32_t)kWin) atomicAdd(&sh.hist[b], 1u);
        }
        if (in >> 16) {
          const uint32_t b = (code_of(w[j] >> 16) - lo) >> shift;
          if (b < (uint32_t)kWin) atomicAdd(&sh.hist[b], 1u);
        }
      }
    }
  }
  return block_sum(sh, a16 >> 4);    // (its barriers also publish the histogram)
}

// Largest window bin whose suffix count reaches `need`; publishes sh.bin, sh.above (count in the
// bins above it) and sh.inside (count in the whole window).  If the window holds fewer than `need`
// keys, sh.bin = -1.  Thread t owns the 16 bins below kWin - 16 t.
__device__ void window_find(Sel16Shared& sh, uint32_t need) {
  constexpr int kPer = kWin / kThreads;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int top = kWin - 1 - tid * kPer;
  uint32_t own = 0;
#pragma unroll
  for (int i = 0; i < kPer; ++i) own += sh.hist[top - i];
  uint32_t inc = own;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();
  if (lane == 31) sh.red[warp] = inc;
  if (tid == 0) { sh.bin = -1; sh.above = 0; }
  __syncthreads();
  uint32_t before = 0, total = 0;
#pragma unroll
  for (int w = 0; w < kThreads / 32; ++w) {
    if (w < warp) before += sh.red[w];
    total += sh.red[w];
  }
  const uint32_t excl = before + inc - own;
  if (excl < need && excl + own >= need) {
    uint32_t a = excl;
    int b = top;
    for (; b > top - kPer + 1; --b) {
      if (a + sh.hist[b] >= need) break;
      a += sh.hist[b];
    }
    sh.bin = b;
    sh.above = a;
  }
  if (tid == 0) sh.inside = total;
  __syncthreads();
}

// SWEEP_LOADS: 16-byte loads a thread keeps in flight in the one-sweep route.  Rows short enough for
// seven or eight CTAs per SM hide the latency by occupancy (4); long rows, whose bit row and lists
// leave room for two or three CTAs only, need it per thread (8, 16).
template <int SWEEP_LOADS>
__global__ void __launch_bounds__(kThreads, SWEEP_LOADS <= 4 ? 8 : (SWEEP_LOADS <= 8 ? 4 : 2))
topk16_rows_kernel(const uint16_t* __restrict__ keys16, const __nv_bfloat16* __restrict__ Q,
                   const __nv_bfloat16* __restrict__ K, int64_t k_tok, int64_t k_head,
                   const int32_t* __restrict__ cu, int Hq, int G, int S, int d_k, int RC, int row_chunks,
                   int64_t n_tiles_total, float scale, const int32_t* __restrict__ b_step, int64_t row_words,
                   uint32_t* __restrict__ mask, int bitrow_bytes, int cand_per_thread,
                   const int32_t* __restrict__ kv_len) {
  extern __shared__ __align__(16) uint8_t dyn_smem[];   // [bit row | candidate lists]
  __shared__ Sel16Shared sh;
  const int r = blockIdx.z, g = blockIdx.y, s = blockIdx.x;
  const int start = cu[r];
  const int N = valid_keys(kv_len, r, Hq / G, g / G, cu[r + 1] - start);
  if (N <= 0) return;
  const int k = b_step[r * Hq + g];
  if (k <= 0) return;
  const int tid = threadIdx.x, lane = tid & 31;
  const int kh = g / G;
  const int grow_idx = (g % G) * S + s;                  // row within the head group (synthetic rows come first)
  const int chunk = grow_idx / RC, crow = grow_idx % RC;
  RowView rv;
  rv.N = N;
  rv.nv8 = (N + 7) >> 3;
  rv.tile_stride = (int64_t)row_chunks * RC * kTileKeys;
  rv.swz = (uint32_t)crow & 15u;
  rv.grow = keys16 + ((((int64_t)kh * n_tiles_total + tile_offset(start, r)) * row_chunks + chunk) * RC + crow) * kTileKeys;
  uint32_t* mrow = mask + (int64_t)kh * row_words + mask_word_offset(start, r);
  const int words = (N + 31) >> 5;

  if (k >= N) {                                          // every key is selected
    for (int w = tid; w < words; w += kThreads) {
      const uint32_t v = (w == words - 1 && (N & 31)) ? ((1u << (N & 31)) - 1u) : 0xffffffffu;
      atomicOr(&mrow[w], v);
    }
    return;
  }
  {
    const __nv_bfloat16* qrow = Q + (((int64_t)r * (Hq / G) + kh) * (G * (S + 1)) + grow_idx) * d_k;
    for (int i = tid; i < d_k; i += kThreads) sh.qf[i] = qrow[i];
    if (tid == 0) { sh.ntie = 0; sh.novf = 0; }
  }

  // ---------------------------------------------------------------- 1. sample
  uint32_t T = 0, above = 0, eq = 0;
  bool found = false;
  uint32_t lo, hi = 0xffffu;
  if (rv.nv8 <= kSampleRound) {
    // the whole row is the sample: its k-th largest code is the threshold
    const Sample sm{rv.nv8, 0};
    const SampleRegs sr = sample_load(rv, sm);
    sample_begin(sh);
    uint32_t unused;
    sample_ranks(sr, 0u, (uint32_t)k, sh, unused, T, above, eq);
    found = true;
    lo = T;
  } else {
    // 128 evenly spaced runs of 32 keys (4096 keys); bracket the k-th largest key between two order statistics
    // of the sample, 4.5 standard deviations of the (hypergeometric) sampling error either side
    Sample sm;
    sm.n_vecs = kSampleRound;
    sm.stride = rv.nv8 / kThreads;                      // >= 4 here
    const float m_s = (float)(sm.n_vecs * 8);
    const float frac = (float)k / (float)N;
    const float rk = frac * m_s;
    const float dlt = 4.5f * sqrtf(rk * (1.0f - frac)) + 6.0f;
    int r_lo = (int)ceilf(rk + dlt);
    if (r_lo > sm.n_vecs * 8) r_lo = sm.n_vecs * 8;
    const int r_hi = (int)floorf(rk - dlt);
    uint32_t a_s, e_s;
    const SampleRegs sr = sample_load(rv, sm);
    sample_begin(sh);
    sample_ranks(sr, r_hi >= 1 ? (uint32_t)r_hi : 0u, (uint32_t)r_lo, sh, hi, lo, a_s, e_s);
    if (lo < kMinCode) lo = kMinCode;
    if (hi < lo) hi = lo;
    lo = fix_lo(lo);
    hi = fix_hi(hi);
  }

  // ---------------------------------------------------------------- 2. one sweep with a bit row and lists
  // Every thread lists the bracket keys it meets in a slice of its own, entry = key << 16 | vector
  // number within the thread << 3 | position in the vector, stored slot-major (conflict free, no
  // atomics, no warp scans).
  if (!found && words * 4 <= bitrow_bytes) {
    uint32_t* bitrow = reinterpret_cast<uint32_t*>(dyn_smem);
    uint32_t* cand = reinterpret_cast<uint32_t*>(dyn_smem + bitrow_bytes);      // [cand_per_thread][kThreads]
    const __half2 tlo = pair_of(raw_of(lo)), thi = pair_of(raw_of(hi));
    uint8_t* bitbytes = reinterpret_cast<uint8_t*>(bitrow);     // byte v8 of the bit row = the 8 keys of vector v8
    uint32_t above_cnt = 0;   // keys above the bracket this thread has met
    int cnt = 0;              // bracket keys this thread has met
    // one vector: mark the keys above the bracket, list the keys inside it
    auto take = [&](const uint4& v, int v8) {
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
      uint32_t ge[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) ge[j] = __hge2_mask(as_h2(w[j]), tlo);
      uint32_t bits = 0;
      if ((ge[0] | ge[1] | ge[2] | ge[3]) != 0u) {
        // bit 2j of the low half and bit 2j+1 of the high half of word j mark its two keys
        uint32_t gacc = 0, cacc = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t pick = (1u << (2 * j)) | (1u << (17 + 2 * j));
          const uint32_t gt = __hgt2_mask(as_h2(w[j]), thi);
          gacc |= gt & pick;
          cacc |= (ge[j] & ~gt) & pick;
        }
        bits = (gacc | (gacc >> 16)) & 0xffu;
        above_cnt += __popc(bits);
        uint32_t cbits = (cacc | (cacc >> 16)) & 0xffu;
        const uint32_t tag = (uint32_t)(v8 / kThreads) << 3;
        while (cbits) {
          const int j = __ffs(cbits) - 1;
          cbits &= cbits - 1;
          const uint32_t ww = (j < 4) ? ((j < 2) ? w[0] : w[1]) : ((j < 6) ? w[2] : w[3]);
          const uint32_t key = (j & 1) ? (ww >> 16) : (ww & 0xffffu);
          if (cnt < cand_per_thread) {
            cand[cnt * kThreads + tid] = (key << 16) | tag | (uint32_t)j;
            ++cnt;
          } else {                                     // the rare key beyond the slice: shared spill list
            const uint32_t slot = atomicAdd(&sh.novf, 1u);
            if (slot < (uint32_t)kOvfCap) { sh.ovf_n[slot] = (uint32_t)(v8 * 8 + j); sh.ovf_key[slot] = (uint16_t)key; }
          }
        }
      }
      return bits;
    };
    // Vector v8 = base + u * kThreads + tid sits in tile (base / 16) + 8 u + tid / 16 at the thread's own
    // chunk position (tid % 16) ^ swz: whole batches need no index arithmetic and no bounds checks.
    const int full_end = ((N >> 3) / (kThreads * SWEEP_LOADS)) * (kThreads * SWEEP_LOADS);   // vectors in whole batches of whole vectors
    const uint16_t* tp = rv.grow + (int64_t)(tid >> 4) * rv.tile_stride + ((((uint32_t)tid & 15u) ^ rv.swz) << 3);
    const int64_t u_step = (int64_t)(kThreads / 16) * rv.tile_stride;
    int base = 0;
    for (; base < full_end; base += kThreads * SWEEP_LOADS, tp += SWEEP_LOADS * u_step) {
      uint4 buf[SWEEP_LOADS];
#pragma unroll
      for (int u = 0; u < SWEEP_LOADS; ++u) buf[u] = *reinterpret_cast<const uint4*>(tp + u * u_step);
#pragma unroll
      for (int u = 0; u < SWEEP_LOADS; ++u) {
        const int v8 = base + u * kThreads + tid;
        bitbytes[v8] = (uint8_t)take(buf[u], v8);
      }
    }
    for (; base < rv.nv8; base += kThreads * SWEEP_LOADS) {          // the ragged end: padded loads
      uint4 buf[SWEEP_LOADS];
#pragma unroll
      for (int u = 0; u < SWEEP_LOADS; ++u) buf[u] = rv.load(base + u * kThreads + tid);
#pragma unroll
      for (int u = 0; u < SWEEP_LOADS; ++u) {
        const int v8 = base + u * kThreads + tid;
        const uint32_t bits = take(buf[u], v8);
        if (v8 < words * 4) bitbytes[v8] = (uint8_t)bits;
      }
    }
    // the two histograms of the listed keys (high byte in [0, 256), low byte in [256, 512)) start from
    // zero; the barriers of the sums also publish them, the bit row and the spill list
    for (int b = tid; b < 512; b += kThreads) sh.hist[b] = 0;
    uint32_t A, C;
    block_sum2(sh, above_cnt, (uint32_t)cnt, A, C);
    const uint32_t novf = sh.novf;
    C += novf;
    bool settled = novf <= (uint32_t)kOvfCap && A <= (uint32_t)k && A + C >= (uint32_t)k;
    if (settled && A < (uint32_t)k) {
      // the k - A largest of the listed keys: two-level histogram over the lists
      const uint32_t need = (uint32_t)k - A;
      for (int i = 0; i < cnt; ++i) atomicAdd(&sh.hist[code_of(cand[i * kThreads + tid] >> 16) >> 8], 1u);
      for (int i = tid; i < (int)novf; i += kThreads) atomicAdd(&sh.hist[code_of(sh.ovf_key[i]) >> 8], 1u);
      __syncthreads();
      find_bin256(sh, sh.hist, need);
      const uint32_t b_top = (uint32_t)sh.bin;
      uint32_t up = sh.above;
      for (int i = 0; i < cnt; ++i) {
        const uint32_t c = code_of(cand[i * kThreads + tid] >> 16);
        if ((c >> 8) == b_top) atomicAdd(&sh.hist[256u + (c & 255u)], 1u);
      }
      for (int i = tid; i < (int)novf; i += kThreads) {
        const uint32_t c = code_of(sh.ovf_key[i]);
        if ((c >> 8) == b_top) atomicAdd(&sh.hist[256u + (c & 255u)], 1u);
      }
      __syncthreads();
      find_bin256(sh, sh.hist + 256, need - up);
      T = (b_top << 8) | (uint32_t)sh.bin;
      up += sh.above;
      eq = sh.hist[256 + sh.bin];
      const uint32_t ties = need - up;              // 1 <= ties <= eq
      if (ties < eq && eq > (uint32_t)kTieCap) {
        settled = false;                            // too many equal 16-bit keys for the list: exact route
      } else {
        for (int i = 0; i < cnt; ++i) {
          const uint32_t e = cand[i * kThreads + tid];
          const uint32_t c = code_of(e >> 16);
          const uint32_t n = ((((e >> 3) & 0x1fffu) * kThreads + (uint32_t)tid) << 3) | (e & 7u);
          if (c > T || (c == T && ties >= eq)) atomicOr(&bitrow[n >> 5], 1u << (n & 31));
          else if (c == T) sh.tie_idx[atomicAdd(&sh.ntie, 1u)] = (int)n;
        }
        for (int i = tid; i < (int)novf; i += kThreads) {
          const uint32_t c = code_of(sh.ovf_key[i]), n = sh.ovf_n[i];
          if (c > T || (c == T && ties >= eq)) atomicOr(&bitrow[n >> 5], 1u << (n & 31));
          else if (c == T) sh.tie_idx[atomicAdd(&sh.ntie, 1u)] = (int)n;
        }
        __syncthreads();
        if (ties < eq) {
          DotCtx dot{sh.qf, K + (int64_t)kh * k_head + (int64_t)start * k_tok, k_tok, d_k, scale};
          for (int i = tid; i < (int)eq; i += kThreads) sh.tie_val[i] = dot(sh.tie_idx[i]);
          __syncthreads();
          for (int i = tid; i < (int)eq; i += kThreads) {
            const float v = sh.tie_val[i];
            const int n = sh.tie_idx[i];
            uint32_t rank = 0;
            for (int u = 0; u < (int)eq; ++u) {
              const float vu = sh.tie_val[u];
              rank += (vu > v || (vu == v && sh.tie_idx[u] < n)) ? 1u : 0u;
            }
            if (rank < ties) atomicOr(&bitrow[n >> 5], 1u << (n & 31));
          }
        }
      }
    }
    __syncthreads();
    if (settled) {
      for (int w = tid; w < words; w += kThreads) {
        const uint32_t v = bitrow[w];
        if (v) atomicOr(&mrow[w], v);
      }
      return;
    }
    if (tid == 0) sh.ntie = 0;
    __syncthreads();
  }

  // ---------------------------------------------------------------- 4. exact route: window sweeps
  // A window is [lo, hi] in code space, histogrammed in 2048 bins of 2^shift codes.  A window wider
  // than 2048 codes is narrowed to the bin that holds the threshold and swept again; a bracket that
  // turns out wrong (rare) is replaced by everything above or below it.
  if (!found) {
    for (int iter = 0; iter < 12; ++iter) {
      int shift = 0;
      while (((hi - lo) >> shift) >= (uint32_t)kWin) ++shift;
      const uint32_t A = window_pass(rv, lo, hi, shift, sh);
      if (A >= (uint32_t)k) {                             // the threshold lies above the window
        lo = fix_lo(hi + 1u);
        hi = 0xffffu;
        continue;
      }
      window_find(sh, (uint32_t)k - A);
      const int bin = sh.bin;
      if (bin < 0) {                                      // the threshold lies below the window
        if (lo <= kMinCode) break;                        // cannot happen: k < N keys lie at or above kMinCode
        hi = fix_hi(lo - 1u);
        lo = kMinCode;
        __syncthreads();
        continue;
      }
      if (shift == 0) {
        T = lo + (uint32_t)bin;
        above = A + sh.above;
        eq = sh.hist[bin];
        found = true;
        break;
      }
      const uint32_t nlo = lo + ((uint32_t)bin << shift);
      const uint32_t nhi = min(nlo + (1u << shift) - 1u, hi);
      lo = fix_lo(nlo);
      hi = fix_hi(nhi);
      __syncthreads();
    }
    __syncthreads();
    if (!found) return;
  }
  const uint32_t ties = (uint32_t)k - above;              // 1 <= ties <= eq
  const bool all_ties = ties >= eq;

  // ---------------------------------------------------------------- emission sweep
  {
    const __half2 tt = pair_of(raw_of(T));
    for (int base = 0; base < rv.nv8; base += kThreads * kLoads) {
      uint4 buf[kLoads];
#pragma unroll
      for (int u = 0; u < kLoads; ++u) buf[u] = rv.load(base + u * kThreads + tid);
#pragma unroll
      for (int u = 0; u < kLoads; ++u) {
        const int v8 = base + u * kThreads + tid;
        const uint32_t w[4] = {buf[u].x, buf[u].y, buf[u].z, buf[u].w};
        uint32_t ge[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) ge[j] = __hge2_mask(as_h2(w[j]), tt);
        if (!__any_sync(0xffffffffu, (ge[0] | ge[1] | ge[2] | ge[3]) != 0u)) continue;   // warp-uniform skip
        // bit 2j of the low half and bit 2j+1 of the high half of word j mark its two keys
        uint32_t gacc = 0, eacc = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t pick = (1u << (2 * j)) | (1u << (17 + 2 * j));
          const uint32_t gt = __hgt2_mask(as_h2(w[j]), tt);
          gacc |= gt & pick;
          eacc |= (ge[j] & ~gt) & pick;
        }
        uint32_t bits = (gacc | (gacc >> 16)) & 0xffu;
        uint32_t eqbits = (eacc | (eacc >> 16)) & 0xffu;
        if (all_ties) bits |= eqbits;
        else {
          while (eqbits) {
            const int j = __ffs(eqbits) - 1;
            eqbits &= eqbits - 1;
            const uint32_t slot = atomicAdd(&sh.ntie, 1u);
            if (slot < (uint32_t)kTieCap) sh.tie_idx[slot] = v8 * 8 + j;
          }
        }
        uint32_t word = bits << (8 * (lane & 3));
        word |= __shfl_xor_sync(0xffffffffu, word, 1);
        word |= __shfl_xor_sync(0xffffffffu, word, 2);
        if ((lane & 3) == 0 && word) atomicOr(&mrow[v8 >> 2], word);
      }
    }
  }
  if (all_ties) return;
  __syncthreads();

  DotCtx dot{sh.qf, K + (int64_t)kh * k_head + (int64_t)start * k_tok, k_tok, d_k, scale};
  if (eq <= (uint32_t)kTieCap) {
    // rank the candidates by (exact logit descending, index ascending) and keep the first `ties`
    for (int i = tid; i < (int)eq; i += kThreads) sh.tie_val[i] = dot(sh.tie_idx[i]);
    __syncthreads();
    for (int i = tid; i < (int)eq; i += kThreads) {
      const float v = sh.tie_val[i];
      const int n = sh.tie_idx[i];
      uint32_t rank = 0;
      for (int u = 0; u < (int)eq; ++u) {
        const float vu = sh.tie_val[u];
        rank += (vu > v || (vu == v && sh.tie_idx[u] < n)) ? 1u : 0u;
      }
      if (rank < ties) atomicOr(&mrow[n >> 5], 1u << (n & 31));
    }
    return;
  }

  // More candidates than the list holds (many equal logits): radix search over the recomputed
  // 32-bit images of the candidates, four 8-bit passes, then an emission in index order.
  uint32_t prefix = 0, known = 0, acc = 0, eq2 = 0;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int b = tid; b < 256; b += kThreads) sh.hist[b] = 0;
    __syncthreads();
    for (int n = tid; n < N; n += kThreads) {
      if (code_of(rv.key_at(n)) == T) {
        const uint32_t key = ordered_key(dot(n));
        if ((key & known) == prefix) atomicAdd(&sh.hist[(key >> shift) & 255u], 1u);
      }
    }
    __syncthreads();
    find_bin256(sh, sh.hist, ties - acc);
    acc += sh.above;
    prefix |= (uint32_t)sh.bin << shift;
    known |= 255u << shift;
    if (pass == 3) eq2 = sh.hist[sh.bin];
    __syncthreads();
  }
  const uint32_t ties2 = ties - acc;
  uint32_t taken = 0;
  const int warp = tid >> 5;
  for (int base = 0; base < N; base += kThreads) {
    const int n = base + tid;
    const bool member = n < N && code_of(rv.key_at(n)) == T;
    const uint32_t key = member ? ordered_key(dot(n)) : 0u;
    bool sel = member && key > prefix;
    const bool tie = member && key == prefix;
    if (ties2 >= eq2) {
      sel |= tie;
    } else {
      const uint32_t tb = __ballot_sync(0xffffffffu, tie);
      __syncthreads();
      if (lane == 0) sh.red[warp] = __popc(tb);
      __syncthreads();
      uint32_t before = taken, total = 0;
      for (int w = 0; w < kThreads / 32; ++w) {
        if (w < warp) before += sh.red[w];
        total += sh.red[w];
      }
      sel |= tie && (before + __popc(tb & ((1u << lane) - 1u))) < ties2;
      taken += total;
    }
    const uint32_t bal = __ballot_sync(0xffffffffu, sel);
    if (lane == 0 && bal) atomicOr(&mrow[n >> 5], bal);
  }
}

}  // namespace

int32_t launch_topk16(const gvote_params* p, const uint16_t* keys16, const __nv_bfloat16* Q, const __nv_bfloat16* K,
                      int64_t k_tok, int64_t k_head, const int32_t* cu, int32_t batch, int64_t total_tokens,
                      int64_t max_N, const int32_t* b_step, int64_t row_words, uint32_t* mask, const int32_t* kv_len,
                      cudaStream_t st) {
  const int Hq = p->n_q_heads, G = Hq / p->n_kv_heads;
  const ScoreGeometry geo = score_geometry(p);
  dim3 grid(p->S, Hq, batch);
  const float scale = (float)(1.0 / sqrt((double)p->d_k));
  // The one-sweep route needs a bit row of max_N bits and a list slice per thread sized for the widest
  // bracket (k = N/2: 4.5 standard deviations of the 4096-key sample's rank, 32, plus 6, either side,
  // times the keys per sampled key), spread over the threads, plus 1.7 standard deviations of that
  // share; what a thread meets beyond its slice goes to a small shared spill list.  Rows too long for 32 KB of bits go
  // straight to the exact route.
  int bitrow_bytes = 0, cand_per_thread = 0;
  if (max_N > (int64_t)kSampleRound * 8 && max_N <= 256 * 1024) {
    bitrow_bytes = (int)align_up((size_t)ceil_div(max_N, 32) * 4, 16);
    const double share = 2.0 * (4.5 * 32.0 + 6.0) * ((double)max_N / (kSampleRound * 8)) / kThreads;
    cand_per_thread = (int)ceil(share + 1.7 * sqrt(share));
  }
  const size_t smem = (size_t)bitrow_bytes + (size_t)cand_per_thread * kThreads * sizeof(uint32_t);
  // CTAs an SM holds: dynamic + static shared memory + 1 KB reserved per CTA, of 228 KB
  const int per_sm = (int)((228 * 1024) / (smem + sizeof(Sel16Shared) + 1024));
  auto kern = per_sm >= 5 ? topk16_rows_kernel<4> : (per_sm >= 3 ? topk16_rows_kernel<8> : topk16_rows_kernel<16>);
  GVOTE_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  {
    LaunchScope scope_("topk16_rows_kernel", st);
    kern<<<grid, kThreads, smem, st>>>(keys16, Q, K, k_tok, k_head, cu, Hq, G, p->S, p->d_k, geo.RC, geo.row_chunks,
                                       (total_tokens >> 7) + batch, scale, b_step, row_words, mask, bitrow_bytes,
                                       cand_per_thread, kv_len);
  }
  GVOTE_LAUNCH_CHECK("topk16_rows_kernel");
  return GVOTE_OK;
}

}  // namespace gvote
