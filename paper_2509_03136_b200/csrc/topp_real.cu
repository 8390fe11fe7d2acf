// Algorithm 1, the current-query steps (A0, C0, B_step), for every head: softmax of its logits over all cached
// keys, the smallest set C0 of keys whose weights reach the mass p, and its size B_step = |C0|.
//
// There are only n_q_heads such rows per request but each is N long, so a row is shared by a thread-
// block cluster of up to eight CTAs (eight for a single request, fewer when a batch brings many rows), an
// equal part of the row each, in ONE launch:
//   1. every CTA bins its keys by their distance below the row maximum (512 bins of 1/16 logit; the
//      maximum comes from the score kernel's read-out) and accumulates per bin a count and the softmax
//      numerators exp(l - max) in 2^-40 fixed point - integers, so the sums do not depend on the order
//      of arrival and two runs give the same bits;
//   2. the cluster's first CTA adds the histograms (it reads its peers' shared memory), sums the
//      bins into Z and walks them from the top until the mass reaches p * Z;
//   3. every CTA sends the keys of that crossing bin from its part of the row into a list in the first
//      CTA's shared memory;
//   4. the first CTA settles the boundary exactly: if the keys are many it refines over 256 sub-bins,
//      then ranks the few left by (weight descending, index ascending) and takes the shortest prefix
//      that supplies the missing mass.  A crossing bin with more keys than the list holds (many near-
//      equal logits) goes through the generic radix search over the row instead.
// Keys at least ln(N / (1 - p)) below the maximum share the last bin: none of them can belong to the
// set (see bin_of), so they are summed in registers and never histogrammed one by one.
// The steps are separated by cluster barriers (hardware barriers: no spinning on memory).
#include <cooperative_groups.h>

#include "select_common.cuh"

namespace gvote {
namespace {

namespace cg = cooperative_groups;
using namespace sel;

constexpr int kBins = 512;
constexpr float kBinsPerLogit = 16.0f;
constexpr int kThreads = 256;
constexpr int kListCap = 4096;      // keys of the crossing bin held in shared memory
constexpr int kRankCap = 256;       // keys ranked pairwise (quadratic work: keep it small; one per thread)
constexpr int kSubBins = 256;       // one per thread
constexpr int kLoads = 8;

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
__device__ __forceinline__ float tail_cut(int N, float p_nuc) {
  const float lim = (float)(kBins - 1) / kBinsPerLogit;
  if (!(p_nuc < 1.0f)) return lim;
  const float c = logf((float)N / (1.0f - p_nuc));
  return c < lim ? c : lim;
}

struct ClusterShared {
  uint32_t cnt[kBins];
  unsigned long long mass[kBins];
  // the first CTA's working set (the peers write the list)
  float val[kListCap];
  int idx[kListCap];
  unsigned long long smass[kRankCap];   // masses in rank order
  int rank[kRankCap];
  uint32_t sub_cnt[kSubBins];
  unsigned long long sub_mass[kSubBins];
  unsigned long long wmass[kThreads / 32];
  uint32_t wcnt[kThreads / 32];
  unsigned long long red64[kThreads / 32];
  uint32_t red32[kThreads / 32];
  int crossing_bin;                     // broadcast to the peers after step 2
  uint32_t in_bin;
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

// Exclusive prefix over the block of one (count, mass) pair per thread, and the block totals.
__device__ __forceinline__ void block_scan_pair(uint32_t c, unsigned long long m, ClusterShared& cs, uint32_t& c_excl,
                                                unsigned long long& m_excl, uint32_t& c_total,
                                                unsigned long long& m_total) {
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
  if (lane == 31) { cs.wcnt[warp] = c_inc; cs.wmass[warp] = m_inc; }
  __syncthreads();
  uint32_t c_before = 0;
  unsigned long long m_before = 0;
  c_total = 0;
  m_total = 0;
#pragma unroll
  for (int w = 0; w < kThreads / 32; ++w) {
    if (w < warp) { c_before += cs.wcnt[w]; m_before += cs.wmass[w]; }
    c_total += cs.wcnt[w];
    m_total += cs.wmass[w];
  }
  c_excl = c_before + c_inc - c;
  m_excl = m_before + m_inc - m;
}

template <int kClusterCtas>     // CTAs that share a row: 8, 4, 2 or 1
__global__ void __cluster_dims__(kClusterCtas, 1, 1) __launch_bounds__(kThreads)
real_topp_kernel(const float* __restrict__ logits, const int32_t* __restrict__ cu, int Hq, int G,
                 const uint32_t* __restrict__ rowmax_part, int n_part, float p_nuc, int include_c0, int64_t row_words,
                 uint32_t* __restrict__ mask, int32_t* __restrict__ b_step, const int32_t* __restrict__ kv_len) {
  extern __shared__ __align__(16) uint8_t dyn[];
  ClusterShared& cs = *reinterpret_cast<ClusterShared*>(dyn);
  // The generic radix search and the emission (rare routes of the first CTA) work in the space of the
  // candidate list, which is dead by the time they run.
  static_assert(sizeof(SelShared) <= sizeof(float) * kListCap + sizeof(int) * kListCap, "list area too small");
  SelShared& sh = *reinterpret_cast<SelShared*>(cs.val);
  cg::cluster_group cluster = cg::this_cluster();
  const int crank = (int)cluster.block_rank();
  ClusterShared& lead = *cluster.map_shared_rank(&cs, 0);
  const int r = blockIdx.z, g = blockIdx.y;
  const int start = cu[r], Ncap = cu[r + 1] - start;       // Ncap: rows of the slab (layout); N: rows that count
  const int N = valid_keys(kv_len, r, Hq / G, g / G, Ncap);
  const int tid = threadIdx.x, lane = tid & 31;
  if (N <= 0) {                          // uniform over the cluster: nobody reaches a cluster barrier
    if (crank == 0 && tid == 0) b_step[r * Hq + g] = 0;
    return;
  }
  const float* L = logits + (int64_t)Hq * start + (int64_t)g * Ncap;       // [n_q_heads][N] per request
  uint32_t mx_key = 0;                                       // the row maximum: the largest of the first pass's CTAs'
  for (int i = 0; i < n_part; ++i) mx_key = max(mx_key, rowmax_part[(int64_t)(r * Hq + g) * n_part + i]);
  const float mx = key_to_float(mx_key);
  const float cut = tail_cut(N, p_nuc);
  const int per = (N + kClusterCtas - 1) / kClusterCtas;
  const int n0 = min(crank * per, N), n1 = min(n0 + per, N);

  // ---- 1. this CTA's histogram
  for (int b = tid; b < kBins; b += kThreads) { cs.cnt[b] = 0; cs.mass[b] = 0; }
  if (tid == 0) {
    cs.n_list = 0; cs.n_list2 = 0; cs.pick = 0; cs.crossing_bin = kBins - 1; cs.in_bin = 0xffffffffu; cs.above_cnt = 0;
    cs.above_mass = 0;
  }
  __syncthreads();
  {
    uint32_t tail_c = 0;
    unsigned long long tail_m = 0;
    for (int base = n0; base < n1; base += kThreads * kLoads) {
      float v[kLoads];
#pragma unroll
      for (int u = 0; u < kLoads; ++u) {
        const int n = base + u * kThreads + tid;
        v[u] = n < n1 ? L[n] : 0.f;
      }
#pragma unroll
      for (int u = 0; u < kLoads; ++u) {
        const int n = base + u * kThreads + tid;
        if (n < n1) {
          const int b = bin_of(v[u], mx, cut);
          const unsigned long long m = mass_fix(v[u], mx);
          if (b == kBins - 1) {
            tail_c += 1u;
            tail_m += m;
          } else {
            atomicAdd(&cs.cnt[b], 1u);
            if (m) add_mass(&cs.mass[b], m);
          }
        }
      }
    }
    tail_c = (uint32_t)warp_sum_i((int)tail_c);
    tail_m = warp_sum_u64(tail_m);
    if (lane == 0) { cs.red32[tid >> 5] = tail_c; cs.red64[tid >> 5] = tail_m; }
    __syncthreads();
    if (tid == 0) {
      for (int w = 1; w < kThreads / 32; ++w) { tail_c += cs.red32[w]; tail_m += cs.red64[w]; }
      cs.cnt[kBins - 1] = tail_c;
      cs.mass[kBins - 1] = tail_m;
    }
  }
  cluster.sync();

  // ---- 2. the first CTA adds the histograms and finds the bin where the mass crosses p * Z
  unsigned long long need = 0;
  if (crank == 0) {
    uint32_t c_own[2];
    unsigned long long m_own[2];
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const int b = 2 * tid + q;         // thread t owns bins 2t, 2t+1
      uint32_t c = cs.cnt[b];
      unsigned long long m = cs.mass[b];
      for (int k = 1; k < kClusterCtas; ++k) {
        const ClusterShared* peer = cluster.map_shared_rank(&cs, k);
        c += peer->cnt[b];
        m += peer->mass[b];
      }
      c_own[q] = c;
      m_own[q] = m;
    }
    __syncthreads();
    cs.cnt[2 * tid] = c_own[0]; cs.cnt[2 * tid + 1] = c_own[1];
    cs.mass[2 * tid] = m_own[0]; cs.mass[2 * tid + 1] = m_own[1];
    uint32_t c_excl, c_tot;
    unsigned long long m_excl, z;
    block_scan_pair(c_own[0] + c_own[1], m_own[0] + m_own[1], cs, c_excl, m_excl, c_tot, z);
    // smallest integer mass that is >= p * Z (at least one unit, at most Z)
    need = (unsigned long long)ceil((double)p_nuc * (double)z);
    if (need > z) need = z;
    if (need == 0) need = 1;
    if (m_excl < need && m_excl + m_own[0] + m_own[1] >= need) {      // exactly one thread's pair crosses
      if (m_excl + m_own[0] >= need) {
        cs.crossing_bin = 2 * tid; cs.above_cnt = c_excl; cs.above_mass = m_excl; cs.in_bin = c_own[0];
      } else {
        cs.crossing_bin = 2 * tid + 1; cs.above_cnt = c_excl + c_own[0]; cs.above_mass = m_excl + m_own[0];
        cs.in_bin = c_own[1];
      }
    }
    __syncthreads();
  }
  cluster.sync();

  // ---- 3. every CTA sends its keys of the crossing bin to the first CTA's list
  const int bstar = lead.crossing_bin;
  const uint32_t in_bin = lead.in_bin;
  if (in_bin <= (uint32_t)kListCap) {
    for (int base = n0; base < n1; base += kThreads * kLoads) {
      float v[kLoads];
#pragma unroll
      for (int u = 0; u < kLoads; ++u) {
        const int n = base + u * kThreads + tid;
        v[u] = n < n1 ? L[n] : 0.f;
      }
#pragma unroll
      for (int u = 0; u < kLoads; ++u) {
        const int n = base + u * kThreads + tid;
        const bool hit = n < n1 && bin_of(v[u], mx, cut) == bstar;
        const uint32_t hits = __ballot_sync(0xffffffffu, hit);    // one counter update per warp
        if (hits) {
          uint32_t base_slot = 0;
          if (lane == 0) base_slot = atomicAdd(&lead.n_list, (uint32_t)__popc(hits));
          base_slot = __shfl_sync(0xffffffffu, base_slot, 0);
          const uint32_t slot = base_slot + __popc(hits & ((1u << lane) - 1u));
          if (hit && slot < (uint32_t)kListCap) { lead.val[slot] = v[u]; lead.idx[slot] = n; }
        }
      }
    }
  }
  cluster.sync();
  if (crank != 0) return;

  // ---- 4. the first CTA settles the boundary
  uint32_t above_cnt = cs.above_cnt;
  unsigned long long lack = need - cs.above_mass;          // mass the crossing bin must supply, > 0
  const uint32_t above_bins = above_cnt;
  const unsigned long long lack_bins = lack;
  uint32_t t_key = 0, ties = 0, eq_cnt = 0;
  bool settled = false;
  if (in_bin <= (uint32_t)kListCap) {
    int m = (int)min(cs.n_list, (uint32_t)kListCap);
    if (m > kRankCap) {
      // second level: 256 sub-bins across the crossing bin's 1/16-logit span, over the list
      const float top = mx - (float)bstar / kBinsPerLogit;              // upper edge of the bin
      cs.sub_cnt[tid] = 0;
      cs.sub_mass[tid] = 0;
      __syncthreads();
      auto sub_of = [&](float l) {
        const float d = (top - l) * (kBinsPerLogit * (float)kSubBins);
        return d <= 0.f ? 0 : (d >= (float)(kSubBins - 1) ? kSubBins - 1 : (int)d);
      };
      for (int i = tid; i < m; i += kThreads) {
        const int b = sub_of(cs.val[i]);
        atomicAdd(&cs.sub_cnt[b], 1u);
        const unsigned long long w = mass_fix(cs.val[i], mx);
        if (w) add_mass(&cs.sub_mass[b], w);
      }
      __syncthreads();
      const uint32_t sc = cs.sub_cnt[tid];
      const unsigned long long smw = cs.sub_mass[tid];
      uint32_t sc_excl, sc_tot;
      unsigned long long sm_excl, sm_tot;
      if (tid == 0) { cs.crossing_bin = kSubBins - 1; cs.above_cnt = 0; cs.above_mass = 0; }
      block_scan_pair(sc, smw, cs, sc_excl, sm_excl, sc_tot, sm_tot);
      if (sm_excl < lack && sm_excl + smw >= lack) {
        cs.crossing_bin = tid;
        cs.above_cnt = sc_excl;
        cs.above_mass = sm_excl;
      }
      __syncthreads();
      const int sstar = cs.crossing_bin;
      above_cnt += cs.above_cnt;
      lack -= cs.above_mass;
      const uint32_t in_sub = cs.sub_cnt[sstar];
      if (in_sub <= (uint32_t)kRankCap) {
        // keep only the crossing sub-bin's keys: every thread reads its candidates into registers,
        // then, after a barrier, all of them are written back to the front of the list
        float cv[kListCap / kThreads];
        int ci[kListCap / kThreads];
        int nc = 0;
#pragma unroll
        for (int j = 0; j < kListCap / kThreads; ++j) {
          const int i = tid + j * kThreads;
          if (i < m && sub_of(cs.val[i]) == sstar) { cv[nc] = cs.val[i]; ci[nc] = cs.idx[i]; ++nc; }
        }
        __syncthreads();
        for (int j = 0; j < nc; ++j) {
          const uint32_t slot = atomicAdd(&cs.n_list2, 1u);
          cs.val[slot] = cv[j];
          cs.idx[slot] = ci[j];
        }
        __syncthreads();
        m = (int)cs.n_list2;
      } else {
        m = -1;                                           // still too many: radix search below
      }
    }
    if (m >= 0) {
      // rank by (value descending, index ascending); ranks are distinct, so this is a permutation
      // (four list entries per step, fetched as two 16-byte loads: the loop is a chain of shared-memory
      // latencies otherwise; the list is padded with entries that rank below everything)
      if (tid < 4) { cs.val[m + tid] = -INFINITY; cs.idx[m + tid] = 0x7fffffff; }
      __syncthreads();
      if (tid < m) {
        const float v = cs.val[tid];
        const int n = cs.idx[tid];
        int r0 = 0, r1 = 0, r2 = 0, r3 = 0;
        for (int u = 0; u < m; u += 4) {
          const float4 vu = *reinterpret_cast<const float4*>(&cs.val[u]);
          const int4 nu = *reinterpret_cast<const int4*>(&cs.idx[u]);
          r0 += (vu.x > v || (vu.x == v && nu.x < n)) ? 1 : 0;
          r1 += (vu.y > v || (vu.y == v && nu.y < n)) ? 1 : 0;
          r2 += (vu.z > v || (vu.z == v && nu.z < n)) ? 1 : 0;
          r3 += (vu.w > v || (vu.w == v && nu.w < n)) ? 1 : 0;
        }
        const int rank = r0 + r1 + r2 + r3;
        cs.rank[tid] = rank;
        cs.smass[rank] = mass_fix(v, mx);
      }
      __syncthreads();
      // shortest prefix of the ranked masses that supplies `lack`
      {
        const unsigned long long own = tid < m ? cs.smass[tid] : 0ull;
        uint32_t d0, d1;
        unsigned long long excl, tot;
        block_scan_pair(0u, own, cs, d0, excl, d1, tot);
        if (tid < m && excl < lack && excl + own >= lack) cs.pick = tid + 1;
        __syncthreads();
      }
      int pick = cs.pick;                                 // keys of the list that join C0
      if (pick < 1) pick = m > 0 ? m : 1;                 // cannot happen when the histograms are consistent
      if (tid == 0) b_step[r * Hq + g] = (int32_t)(above_cnt + (uint32_t)pick);
      if (!include_c0) return;
      // threshold key and tie bookkeeping for the emission below: the last key taken has rank pick-1
      if (tid < m && cs.rank[tid] == pick - 1) cs.v_t = cs.val[tid];
      __syncthreads();
      const float v_t = cs.v_t;
      const uint32_t eq = (tid < m && cs.val[tid] == v_t) ? 1u : 0u, gt = (tid < m && cs.val[tid] > v_t) ? 1u : 0u;
      eq_cnt = block_sum_u32(eq, cs.red32);
      const uint32_t gt_cnt = block_sum_u32(gt, cs.red32);
      __syncthreads();                                    // the list is dead from here on (sh takes its place)
      t_key = ordered_key(v_t);
      ties = (uint32_t)pick - gt_cnt;
      settled = true;
    }
  }
  if (!settled) {
    // many near-equal logits around the boundary: radix search over the row, restricted to the crossing bin
    above_cnt = above_bins;
    lack = lack_bins;
    uint32_t a_cnt;
    unsigned long long a_mass;
    InBin keep{mx, cut, bstar};
    radix_threshold<true>(StoredRow{L}, N, mx, lack, sh, t_key, a_cnt, a_mass, eq_cnt, keep);
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
  emit_row(StoredRow{L}, N, t_key, ties, eq_cnt, mrow, sh);
}

}  // namespace

// `rowmax_part` [batch][n_q_heads][n_part]: the maxima (order-preserving images) the CTAs of the vote's first pass met.
int32_t launch_real_topp(const gvote_params* p, const float* logits, const int32_t* cu, int32_t batch, int64_t max_N,
                         const uint32_t* rowmax_part, int n_part, int64_t row_words, uint32_t* mask, int32_t* b_step,
                         const int32_t* kv_len, cudaStream_t st) {
  const int Hq = p->n_q_heads, G = Hq / p->n_kv_heads;
  (void)max_N;
  static_assert(kBins == 2 * kThreads && kSubBins == kThreads && kRankCap == kThreads, "bins per thread");
  // CTAs per row: eight when the rows are few (one request: n_q_heads rows, each max_N long), fewer when a
  // batch brings many rows, so that the launch stays within a few CTAs per SM - the steps of a cluster cost
  // the same whether its CTAs have 32 keys each or 4096 (16 ragged requests of 32 heads: 28 us with two CTAs
  // per row, 37 with four, 69 with eight; one request of 32768 keys: 20, 24 and 34 us with 8, 4 and 2)
  const int64_t rows = (int64_t)Hq * batch;
  const int cl = rows * 8 <= 592 ? 8 : (rows * 4 <= 592 ? 4 : 2);
  auto launch = [&](auto kernel, int n_cta) -> cudaError_t {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(ClusterShared));
    if (e != cudaSuccess) return e;
    dim3 grid((unsigned)n_cta, (unsigned)Hq, (unsigned)batch);
    LaunchScope scope_("real_topp_kernel", st);
    return launch_on(kernel, grid, dim3(kThreads), sizeof(ClusterShared), st, logits, cu, Hq, G, rowmax_part, n_part, p->p_nuc,
                     p->include_c0, row_words, mask, b_step, kv_len);
  };
  GVOTE_CUDA_CHECK(cl == 8 ? launch(real_topp_kernel<8>, 8) : (cl == 4 ? launch(real_topp_kernel<4>, 4) : launch(real_topp_kernel<2>, 2)));
  GVOTE_LAUNCH_CHECK("real_topp_kernel");
  return GVOTE_OK;
}

}  // namespace gvote
