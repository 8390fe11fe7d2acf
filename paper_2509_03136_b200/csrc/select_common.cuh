// Block-wide building blocks of the selection kernels: reductions, the digit search over a shared-
// memory histogram, the three-digit radix search for a row's threshold (by count for top-k, by
// softmax mass for top-p) and the emission of a row's selection into the keep mask.
#pragma once

#include "common.cuh"

namespace gvote {
namespace sel {

constexpr float kFixScale = 1099511627776.0f;   // 2^40

// ---------------------------------------------------------------------------------- block helpers
struct SelShared {
  uint32_t cnt[2048];
  unsigned long long mass[2048];
  unsigned long long red64[32];
  uint32_t red32[32];
  float redf[32];
  // results of a digit search
  int bin;
  uint32_t cnt_above;
  unsigned long long mass_above;
  int tie_base;
};

__device__ __forceinline__ float block_max(float v, float* red) {
  v = warp_max(v);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float m = red[0];
  for (int i = 1; i < (int)blockDim.x / 32; ++i) m = fmaxf(m, red[i]);
  __syncthreads();
  return m;
}
__device__ __forceinline__ unsigned long long block_sum_u64(unsigned long long v, unsigned long long* red) {
  v = warp_sum_u64(v);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  unsigned long long s = 0;
  for (int i = 0; i < (int)blockDim.x / 32; ++i) s += red[i];
  __syncthreads();
  return s;
}
__device__ __forceinline__ uint32_t block_sum_u32(uint32_t v, uint32_t* red) {
  v = (uint32_t)warp_sum_i((int)v);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  uint32_t s = 0;
  for (int i = 0; i < (int)blockDim.x / 32; ++i) s += red[i];
  __syncthreads();
  return s;
}

// exp(l - max) in 2^-40 fixed point (l <= max, so the value is in [0, 2^40]).
__device__ __forceinline__ unsigned long long mass_fix(float l, float mx) {
  return __float2ull_rn(expf(l - mx) * kFixScale);
}

// Adds m to a 64-bit sum in shared memory with 32-bit atomics (the low word, then the carry and the high
// word when there is one - a mass has 41 bits, so mostly there is not): the sum is exact whatever the order
// of arrival, and a 32-bit shared-memory atomic does not loop.
__device__ __forceinline__ void add_mass(unsigned long long* sum, unsigned long long m) {
  uint32_t* w = reinterpret_cast<uint32_t*>(sum);
  const uint32_t lo = (uint32_t)m;
  const uint32_t old = atomicAdd(&w[0], lo);
  const uint32_t hi = (uint32_t)(m >> 32) + ((old + lo < old) ? 1u : 0u);
  if (hi) atomicAdd(&w[1], hi);
}

// Find the highest bin b of hist[0..nbins) whose suffix sum (bins >= b) reaches `need`;
// publish b and the sum of the bins above it.  MASS selects which histogram decides; the count
// of elements above is always published too.  Requires total >= need (else bin 0 is returned).
template <bool MASS>
__device__ void find_bin(SelShared& sh, int nbins, unsigned long long need) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per = nbins / (int)blockDim.x;
  unsigned long long w = 0;
  uint32_t c = 0;
  for (int i = 0; i < per; ++i) {
    const int b = tid * per + i;
    c += sh.cnt[b];
    w += MASS ? sh.mass[b] : (unsigned long long)sh.cnt[b];
  }
  // suffix sums over threads (exclusive): warp shuffle scan from the top lane down
  unsigned long long ws = w;
  uint32_t cs = c;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long tw = __shfl_down_sync(0xffffffffu, ws, o);
    const uint32_t tc = __shfl_down_sync(0xffffffffu, cs, o);
    if (lane + o < 32) { ws += tw; cs += tc; }
  }
  if (lane == 0) { sh.red64[warp] = ws; sh.red32[warp] = cs; }
  if (tid == 0) { sh.bin = 0; sh.cnt_above = 0; sh.mass_above = 0; }
  __syncthreads();
  unsigned long long hi_w = 0;
  uint32_t hi_c = 0;
  for (int i = warp + 1; i < (int)blockDim.x / 32; ++i) { hi_w += sh.red64[i]; hi_c += sh.red32[i]; }
  const unsigned long long excl_w = ws - w + hi_w;   // weight in bins of higher threads
  const uint32_t excl_c = cs - c + hi_c;
  if (excl_w < need && excl_w + w >= need) {
    unsigned long long aw = excl_w;
    uint32_t ac = excl_c;
    int b = tid * per + per - 1;
    for (; b > tid * per; --b) {
      const unsigned long long bw = MASS ? sh.mass[b] : (unsigned long long)sh.cnt[b];
      if (aw + bw >= need) break;
      aw += bw;
      ac += sh.cnt[b];
    }
    sh.bin = b;
    sh.cnt_above = ac;
    sh.mass_above = aw;
  }
  __syncthreads();
}

// Radix search for the threshold key of one row.
//   MASS = false: largest t with #(key >= t) >= need            (top-k, need = k)
//   MASS = true : largest t with mass(key >= t) >= need          (top-p, need = p * Z in fixed point)
// Only the elements `keep` accepts take part.
// Outputs (same in every thread): t, number of keys above t, their mass (MASS only: mass above
// in fixed point), number of keys equal to t.
struct KeepAll { __device__ __forceinline__ bool operator()(float) const { return true; } };
// A row of logits: anything that returns the logit of key n (stored values, or values computed on demand).
struct StoredRow {
  const float* p;
  __device__ __forceinline__ float operator()(int n) const { return p[n]; }
};

template <bool MASS, typename Row, typename Filter = KeepAll>
__device__ void radix_threshold(const Row& row, int N, float mx, unsigned long long need,
                                SelShared& sh, uint32_t& t_out, uint32_t& above_cnt,
                                unsigned long long& above_mass, uint32_t& eq_cnt, Filter keep = Filter()) {
  const int tid = threadIdx.x;
  uint32_t prefix = 0;          // digits fixed so far, left aligned
  uint32_t cnt_acc = 0;
  unsigned long long mass_acc = 0;
  const int shifts[3] = {21, 10, 0};
  const int bits[3] = {11, 11, 10};
  uint32_t known_mask = 0;
  for (int pass = 0; pass < 3; ++pass) {
    const int nb = 1 << bits[pass];
    for (int b = tid; b < nb; b += blockDim.x) { sh.cnt[b] = 0; if (MASS) sh.mass[b] = 0; }
    __syncthreads();
    for (int n = tid; n < N; n += blockDim.x) {
      const float l = row(n);
      const uint32_t key = ordered_key(l);
      if ((key & known_mask) == prefix && keep(l)) {
        const int b = (key >> shifts[pass]) & (nb - 1);
        atomicAdd(&sh.cnt[b], 1u);
        if (MASS) add_mass(&sh.mass[b], mass_fix(l, mx));
      }
    }
    __syncthreads();
    const unsigned long long remaining = need - (MASS ? mass_acc : (unsigned long long)cnt_acc);
    find_bin<MASS>(sh, nb, remaining);
    const int b = sh.bin;
    cnt_acc += sh.cnt_above;
    mass_acc += sh.mass_above;
    if (pass == 2) eq_cnt = sh.cnt[b];
    prefix |= ((uint32_t)b) << shifts[pass];
    known_mask |= ((uint32_t)(nb - 1)) << shifts[pass];
    __syncthreads();
  }
  t_out = prefix;
  above_cnt = cnt_acc;
  above_mass = mass_acc;
}

// OR the row's selection into the mask: keys above t, plus the first `ties` keys equal to t.
template <typename Row>
__device__ inline void emit_row(const Row& row, int N, uint32_t t, uint32_t ties, uint32_t eq_cnt,
                                uint32_t* __restrict__ mask_row, SelShared& sh) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool all_ties = ties >= eq_cnt;
  uint32_t taken = 0;   // ties taken so far (ordered path only)
  for (int base = 0; base < N; base += blockDim.x) {
    const int n = base + tid;
    uint32_t key = 0;
    bool valid = n < N;
    if (valid) key = ordered_key(row(n));
    bool sel = valid && key > t;
    const bool tie = valid && key == t;
    if (all_ties) {
      sel |= tie;
    } else if (ties > 0) {
      // ordered: rank of this tie among all ties of the row, by index
      const uint32_t tb = __ballot_sync(0xffffffffu, tie);
      if (lane == 0) sh.red32[warp] = __popc(tb);
      __syncthreads();
      uint32_t before = taken;
      for (int w = 0; w < warp; ++w) before += sh.red32[w];
      uint32_t total = 0;
      for (int w = 0; w < (int)blockDim.x / 32; ++w) total += sh.red32[w];
      const uint32_t rank = before + __popc(tb & ((1u << lane) - 1u));
      sel |= tie && rank < ties;
      taken += total;
      __syncthreads();
    }
    const uint32_t bal = __ballot_sync(0xffffffffu, sel);
    if (lane == 0 && bal) atomicOr(&mask_row[n >> 5], bal);
  }
}

}  // namespace sel
}  // namespace gvote
