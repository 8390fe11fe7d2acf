// Algorithm 1 lines 1-3 for the current query of every head: softmax of its logits over all cached
// keys, the smallest set C0 of keys whose weights reach the mass p, and its size B_step = |C0|.
//
// There are only n_q_heads such rows per request but each is N long, so the work is split along
// the row instead of giving a row to one CTA:
//   real_hist_kernel   (many CTAs per row) bins every key by its distance below the row maximum
//                      (512 bins of 1/16 logit, the maximum comes from the score kernel's read-out)
//                      and accumulates per bin a count and the softmax numerators exp(l - max) in
//                      2^-40 fixed point - integers, so the sums do not depend on the order of
//                      arrival and two runs give the same bits;
//   real_resolve_kernel (one CTA per row) sums the bins into Z, walks them from the top until the
//                      mass reaches p * Z, and settles the boundary inside the crossing bin exactly:
//                      its keys are collected, ranked by (weight descending, index ascending) and
//                      the shortest prefix that supplies the missing mass is taken.  A crossing bin
//                      with more keys than the list holds (many near-equal logits) goes through the
//                      generic radix search instead.
// Keys more than 32 logits below the maximum share the last bin; their numerators round to zero in
// the fixed-point format and can never be needed to reach p.
#include "select_common.cuh"

namespace gvote {
namespace {

using namespace sel;

constexpr int kBins = 512;
constexpr float kBinsPerLogit = 16.0f;
constexpr int kHistThreads = 256;
constexpr int kHistKeysPerCta = 4096;
constexpr int kResolveThreads = 1024;
constexpr int kListCap = 4096;      // keys of the crossing bin held in shared memory
constexpr int kRankCap = 256;       // keys ranked pairwise (quadratic work: keep it small)
constexpr int kSubBins = 256;

__device__ __forceinline__ float key_to_float(uint32_t key) {
  return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}
// Bin of a key `l` below the row maximum.  Keys at least `cut` logits below the maximum share the
// last bin: with cut = ln(N / (1 - p)) each of them weighs less than (1 - p) / N of the maximum's
// weight, all of them together less than (1 - p) Z, so none can belong to the top-p set.
__device__ __forceinline__ int bin_of(float l, float mx, float cut) {
  const float d = mx - l;                                   // l <= mx, so d >= 0
  if (d >= cut) return kBins - 1;
  const int b = (int)(d * kBinsPerLogit);
  return b > kBins - 2 ? kBins - 2 : b;
}
__host__ __device__ __forceinline__ float tail_cut(int N, float p_nuc) {
  const float lim = (float)(kBins - 1) / kBinsPerLogit;
  if (!(p_nuc < 1.0f)) return lim;
  const float c = logf((float)N / (1.0f - p_nuc));
  return c < lim ? c : lim;
}

__global__ void __launch_bounds__(kHistThreads)
real_hist_kernel(const float* __restrict__ logits, const int32_t* __restrict__ cu, int Hq, int S1, float p_nuc,
                 const uint32_t* __restrict__ rowmax, uint32_t* __restrict__ hist_cnt,
                 unsigned long long* __restrict__ hist_mass) {
  __shared__ uint32_t s_cnt[kBins];
  __shared__ unsigned long long s_mass[kBins];
  __shared__ unsigned long long s_red[kHistThreads / 32];
  __shared__ uint32_t s_redc[kHistThreads / 32];
  const int r = blockIdx.z, g = blockIdx.y;
  const int start = cu[r], N = cu[r + 1] - start;
  const int n0 = blockIdx.x * kHistKeysPerCta;
  if (n0 >= N) return;
  const int n1 = min(n0 + kHistKeysPerCta, N);
  const float* L = logits + (int64_t)Hq * S1 * start + ((int64_t)g * S1) * N;
  const float mx = key_to_float(rowmax[r * Hq + g]);
  const float cut = tail_cut(N, p_nuc);
  for (int b = threadIdx.x; b < kBins; b += kHistThreads) { s_cnt[b] = 0; s_mass[b] = 0; }
  __syncthreads();
  // the tail bin is summed in registers: it usually holds most keys and needs no histogram
  uint32_t tail_c = 0;
  unsigned long long tail_m = 0;
  for (int base = n0; base < n1; base += kHistThreads * 4) {
    float v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int n = base + u * kHistThreads + threadIdx.x;
      v[u] = n < n1 ? L[n] : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int n = base + u * kHistThreads + threadIdx.x;
      if (n < n1) {
        const int b = bin_of(v[u], mx, cut);
        const unsigned long long m = mass_fix(v[u], mx);
        if (b == kBins - 1) {
          tail_c += 1u;
          tail_m += m;
        } else {
          atomicAdd(&s_cnt[b], 1u);
          if (m) atomicAdd(&s_mass[b], m);
        }
      }
    }
  }
  tail_c = (uint32_t)warp_sum_i((int)tail_c);
  tail_m = warp_sum_u64(tail_m);
  if ((threadIdx.x & 31) == 0) { s_redc[threadIdx.x >> 5] = tail_c; s_red[threadIdx.x >> 5] = tail_m; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < kHistThreads / 32; ++w) { tail_c += s_redc[w]; tail_m += s_red[w]; }
    s_cnt[kBins - 1] = tail_c;
    s_mass[kBins - 1] = tail_m;
  }
  __syncthreads();
  const int64_t ho = ((int64_t)r * Hq + g) * kBins;
  for (int b = threadIdx.x; b < kBins; b += kHistThreads) {
    const uint32_t c = s_cnt[b];
    if (c) {
      atomicAdd(&hist_cnt[ho + b], c);
      const unsigned long long m = s_mass[b];
      if (m) atomicAdd(&hist_mass[ho + b], m);
    }
  }
}

struct ResolveShared {
  float val[kListCap];
  int idx[kListCap];
  unsigned long long smass[kRankCap];   // masses in rank order
  int rank[kRankCap];
  uint32_t sub_cnt[kSubBins];
  unsigned long long sub_mass[kSubBins];
  unsigned long long wmass[kResolveThreads / 32];
  uint32_t wcnt[kResolveThreads / 32];
  int crossing_bin;
  uint32_t above_cnt;
  unsigned long long above_mass;
  uint32_t n_list, n_list2;
  int pick;
  float v_t;
};

struct InBin {
  float mx, cut;
  int bin;
  __device__ __forceinline__ bool operator()(float l) const { return bin_of(l, mx, cut) == bin; }
};

// Inclusive scan over the block of one (count, mass) pair per thread; returns the exclusive
// prefix of this thread and the block totals.
__device__ __forceinline__ void block_scan_pair(uint32_t c, unsigned long long m, ResolveShared& rs, uint32_t& c_excl,
                                                unsigned long long& m_excl, unsigned long long& m_total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t c_inc = c;
  unsigned long long m_inc = m;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t tc = __shfl_up_sync(0xffffffffu, c_inc, o);
    const unsigned long long tm = __shfl_up_sync(0xffffffffu, m_inc, o);
    if (lane >= o) { c_inc += tc; m_inc += tm; }
  }
  __syncthreads();                       // earlier readers of wcnt / wmass are done
  if (lane == 31) { rs.wcnt[warp] = c_inc; rs.wmass[warp] = m_inc; }
  __syncthreads();
  uint32_t c_before = 0;
  unsigned long long m_before = 0;
  m_total = 0;
  for (int w = 0; w < kResolveThreads / 32; ++w) {
    if (w < warp) { c_before += rs.wcnt[w]; m_before += rs.wmass[w]; }
    m_total += rs.wmass[w];
  }
  c_excl = c_before + c_inc - c;
  m_excl = m_before + m_inc - m;
}

__global__ void __launch_bounds__(kResolveThreads)
real_resolve_kernel(const float* __restrict__ logits, const int32_t* __restrict__ cu, int Hq, int G, int S1,
                    const uint32_t* __restrict__ rowmax, const uint32_t* __restrict__ hist_cnt,
                    const unsigned long long* __restrict__ hist_mass, float p_nuc, int include_c0,
                    int64_t row_words, uint32_t* __restrict__ mask, int32_t* __restrict__ b_step) {
  extern __shared__ __align__(16) uint8_t dyn[];
  ResolveShared& rs = *reinterpret_cast<ResolveShared*>(dyn);
  __shared__ SelShared sh;
  const int r = blockIdx.y, g = blockIdx.x;
  const int start = cu[r], N = cu[r + 1] - start;
  const int tid = threadIdx.x;
  if (N <= 0) { if (tid == 0) b_step[r * Hq + g] = 0; return; }
  const float* L = logits + (int64_t)Hq * S1 * start + ((int64_t)g * S1) * N;
  const float mx = key_to_float(rowmax[r * Hq + g]);
  const float cut = tail_cut(N, p_nuc);
  const int64_t ho = ((int64_t)r * Hq + g) * kBins;

  // ---- which bin crosses p * Z: thread t < kBins owns bin t
  const uint32_t c_own = tid < kBins ? hist_cnt[ho + tid] : 0u;
  const unsigned long long m_own = tid < kBins ? hist_mass[ho + tid] : 0ull;
  if (tid == 0) { rs.crossing_bin = kBins - 1; rs.n_list = 0; rs.n_list2 = 0; rs.pick = 0; rs.above_cnt = 0; rs.above_mass = 0; }
  uint32_t c_excl;
  unsigned long long m_excl, z;
  block_scan_pair(c_own, m_own, rs, c_excl, m_excl, z);
  // smallest integer mass that is >= p * Z (at least one unit, at most Z)
  unsigned long long need = (unsigned long long)ceil((double)p_nuc * (double)z);
  if (need > z) need = z;
  if (need == 0) need = 1;
  if (m_excl < need && m_excl + m_own >= need) {      // exactly one bin crosses
    rs.crossing_bin = tid;
    rs.above_cnt = c_excl;
    rs.above_mass = m_excl;
  }
  __syncthreads();
  const int bstar = rs.crossing_bin;
  const uint32_t above_bins = rs.above_cnt;                 // keys in the bins above the crossing bin
  const unsigned long long lack_bins = need - rs.above_mass;   // mass the crossing bin must supply, > 0
  uint32_t above_cnt = above_bins;
  unsigned long long lack = lack_bins;
  const uint32_t in_bin = hist_cnt[ho + bstar];

  uint32_t t_key = 0, ties = 0, eq_cnt = 0;
  bool settled = false;
  if (in_bin <= (uint32_t)kListCap) {
    // ---- collect the crossing bin's keys (all of a thread's loads are issued before any is used)
    constexpr int kLoads = 16;
    for (int base = 0; base < N; base += kResolveThreads * kLoads) {
      float v[kLoads];
#pragma unroll
      for (int u = 0; u < kLoads; ++u) {
        const int n = base + u * kResolveThreads + tid;
        v[u] = n < N ? L[n] : 0.f;
      }
#pragma unroll
      for (int u = 0; u < kLoads; ++u) {
        const int n = base + u * kResolveThreads + tid;
        const bool hit = n < N && bin_of(v[u], mx, cut) == bstar;
        const uint32_t hits = __ballot_sync(0xffffffffu, hit);    // one counter update per warp
        if (hits) {
          uint32_t base_slot = 0;
          if ((tid & 31) == 0) base_slot = atomicAdd(&rs.n_list, (uint32_t)__popc(hits));
          base_slot = __shfl_sync(0xffffffffu, base_slot, 0);
          const uint32_t slot = base_slot + __popc(hits & ((1u << (tid & 31)) - 1u));
          if (hit && slot < (uint32_t)kListCap) { rs.val[slot] = v[u]; rs.idx[slot] = n; }
        }
      }
    }
    __syncthreads();
    int m = (int)min(rs.n_list, (uint32_t)kListCap);
    if (m > kRankCap) {
      // ---- second level: 256 sub-bins across the crossing bin's 1/16-logit span, over the list
      const float top = mx - (float)bstar / kBinsPerLogit;              // upper edge of the bin (never the tail bin here)
      for (int b = tid; b < kSubBins; b += kResolveThreads) { rs.sub_cnt[b] = 0; rs.sub_mass[b] = 0; }
      __syncthreads();
      auto sub_of = [&](float l) {
        const float d = (top - l) * (kBinsPerLogit * (float)kSubBins);
        return d <= 0.f ? 0 : (d >= (float)(kSubBins - 1) ? kSubBins - 1 : (int)d);
      };
      for (int i = tid; i < m; i += kResolveThreads) {
        const int b = sub_of(rs.val[i]);
        atomicAdd(&rs.sub_cnt[b], 1u);
        const unsigned long long w = mass_fix(rs.val[i], mx);
        if (w) atomicAdd(&rs.sub_mass[b], w);
      }
      __syncthreads();
      const uint32_t sc = tid < kSubBins ? rs.sub_cnt[tid] : 0u;
      const unsigned long long smw = tid < kSubBins ? rs.sub_mass[tid] : 0ull;
      uint32_t sc_excl;
      unsigned long long sm_excl, sm_tot;
      if (tid == 0) { rs.crossing_bin = kSubBins - 1; rs.above_cnt = 0; rs.above_mass = 0; }
      block_scan_pair(sc, smw, rs, sc_excl, sm_excl, sm_tot);
      if (tid < kSubBins && sm_excl < lack && sm_excl + smw >= lack) {
        rs.crossing_bin = tid;
        rs.above_cnt = sc_excl;
        rs.above_mass = sm_excl;
      }
      __syncthreads();
      const int sstar = rs.crossing_bin;
      above_cnt += rs.above_cnt;
      lack -= rs.above_mass;
      const uint32_t in_sub = rs.sub_cnt[sstar];
      if (in_sub <= (uint32_t)kRankCap) {
        // keep only the crossing sub-bin's keys: every thread reads its candidates into registers,
        // then, after a barrier, all of them are written back to the front of the list
        float cv[kListCap / kResolveThreads];
        int ci[kListCap / kResolveThreads];
        int nc = 0;
        for (int i = tid; i < m; i += kResolveThreads)
          if (sub_of(rs.val[i]) == sstar) { cv[nc] = rs.val[i]; ci[nc] = rs.idx[i]; ++nc; }
        __syncthreads();
        for (int j = 0; j < nc; ++j) {
          const uint32_t slot = atomicAdd(&rs.n_list2, 1u);
          rs.val[slot] = cv[j];
          rs.idx[slot] = ci[j];
        }
        __syncthreads();
        m = (int)rs.n_list2;
      } else {
        m = -1;                                           // still too many: radix search below
      }
    }
    if (m >= 0) {
      // ---- rank by (value descending, index ascending); ranks are distinct, so this is a permutation
      for (int i = tid; i < m; i += kResolveThreads) {
        const float v = rs.val[i];
        const int n = rs.idx[i];
        int rank = 0;
        for (int u = 0; u < m; ++u) {
          const float vu = rs.val[u];
          rank += (vu > v || (vu == v && rs.idx[u] < n)) ? 1 : 0;
        }
        rs.rank[i] = rank;
        rs.smass[rank] = mass_fix(v, mx);
      }
      __syncthreads();
      // shortest prefix of the ranked masses that supplies `lack` (kRankCap <= kResolveThreads)
      {
        const unsigned long long own = tid < m ? rs.smass[tid] : 0ull;
        uint32_t dummy;
        unsigned long long excl, tot;
        block_scan_pair(0u, own, rs, dummy, excl, tot);
        if (tid < m && excl < lack && excl + own >= lack) rs.pick = tid + 1;
        __syncthreads();
      }
      int pick = rs.pick;                                 // keys of the list that join C0
      if (pick < 1) pick = m > 0 ? m : 1;                 // cannot happen when the histograms are consistent
      if (tid == 0) b_step[r * Hq + g] = (int32_t)(above_cnt + (uint32_t)pick);
      if (!include_c0) return;
      // threshold key and tie bookkeeping for the emission below: the last key taken has rank pick-1
      for (int i = tid; i < m; i += kResolveThreads)
        if (rs.rank[i] == pick - 1) rs.v_t = rs.val[i];
      __syncthreads();
      const float v_t = rs.v_t;
      uint32_t eq = 0, gt = 0;
      for (int i = tid; i < m; i += kResolveThreads) {
        eq += rs.val[i] == v_t ? 1u : 0u;
        gt += rs.val[i] > v_t ? 1u : 0u;
      }
      eq_cnt = block_sum_u32(eq, sh.red32);
      const uint32_t gt_cnt = block_sum_u32(gt, sh.red32);
      t_key = ordered_key(v_t);
      ties = (uint32_t)pick - gt_cnt;
      settled = true;
    }
  }
  if (!settled) {
    // many near-equal logits around the boundary: radix search restricted to the crossing bin
    above_cnt = above_bins;
    lack = lack_bins;
    uint32_t a_cnt;
    unsigned long long a_mass;
    InBin keep{mx, cut, bstar};
    radix_threshold<true>(L, N, mx, lack, sh, t_key, a_cnt, a_mass, eq_cnt, keep);
    const unsigned long long e_t = mass_fix(key_to_float(t_key), mx);
    ties = eq_cnt;
    if (e_t > 0) {
      const unsigned long long still = lack - a_mass;
      const unsigned long long j = (still + e_t - 1) / e_t;
      ties = (uint32_t)(j < (unsigned long long)eq_cnt ? j : eq_cnt);
    }
    if (ties == 0) ties = 1;
    if (tid == 0) b_step[r * Hq + g] = (int32_t)(above_cnt + a_cnt + ties);
    if (!include_c0) return;
  }
  uint32_t* mrow = mask + (int64_t)(g / G) * row_words + mask_word_offset(start, r);
  emit_row(L, N, t_key, ties, eq_cnt, mrow, sh);
}

}  // namespace

size_t real_topp_scratch_bytes(const gvote_params* p, int32_t batch) {
  const size_t rows = (size_t)batch * p->n_q_heads;
  return align_up(rows * sizeof(uint32_t), 256) + rows * kBins * (sizeof(unsigned long long) + sizeof(uint32_t));
}

// rowmax / histograms live in `scratch` (real_topp_scratch_bytes), zeroed by the caller before the
// score kernel runs (its read-out fills rowmax with atomicMax).
uint32_t* real_topp_rowmax(char* scratch) { return reinterpret_cast<uint32_t*>(scratch); }

int32_t launch_real_topp(const gvote_params* p, const float* logits, const int32_t* cu, int32_t batch, int64_t max_N,
                         char* scratch, int64_t row_words, uint32_t* mask, int32_t* b_step, cudaStream_t st) {
  const int Hq = p->n_q_heads, G = Hq / p->n_kv_heads, S1 = p->S + 1;
  const size_t rows = (size_t)batch * Hq;
  uint32_t* rowmax = reinterpret_cast<uint32_t*>(scratch);
  unsigned long long* hist_mass = reinterpret_cast<unsigned long long*>(scratch + align_up(rows * sizeof(uint32_t), 256));
  uint32_t* hist_cnt = reinterpret_cast<uint32_t*>(hist_mass + rows * kBins);
  dim3 gh((unsigned)ceil_div(max_N > 0 ? max_N : 1, kHistKeysPerCta), (unsigned)Hq, (unsigned)batch);
  {
    LaunchScope scope_("real_hist_kernel", st);
    real_hist_kernel<<<gh, kHistThreads, 0, st>>>(logits, cu, Hq, S1, p->p_nuc, rowmax, hist_cnt, hist_mass);
  }
  GVOTE_LAUNCH_CHECK("real_hist_kernel");
  static_assert(kBins <= kResolveThreads && kSubBins <= kResolveThreads && kRankCap <= kResolveThreads,
                "one bin / ranked key per thread");
  GVOTE_CUDA_CHECK(cudaFuncSetAttribute(real_resolve_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)sizeof(ResolveShared)));
  dim3 gr((unsigned)Hq, (unsigned)batch);
  {
    LaunchScope scope_("real_resolve_kernel", st);
    real_resolve_kernel<<<gr, kResolveThreads, sizeof(ResolveShared), st>>>(logits, cu, Hq, G, S1, rowmax, hist_cnt,
                                                                            hist_mass, p->p_nuc, p->include_c0,
                                                                            row_words, mask, b_step);
  }
  GVOTE_LAUNCH_CHECK("real_resolve_kernel");
  return GVOTE_OK;
}

}  // namespace gvote
