// Algorithm 1 line 11: prune K and V to the keep-set, in place.
//
// Two kernels.  mask_scan_kernel turns each (request, KV head) bit row into an exclusive popcount
// prefix per 32-key word and the head's budget.  compact_kernel then moves the kept rows of one
// 128-token tile per CTA to their destination rows, 16 bytes per thread per step.
//
// In-place safety.  Row i moves to row prefix(i) <= i, so a tile's destination may still hold
// rows that an EARLIER tile of the same slab has not read yet.  Each CTA therefore (1) takes a
// ticket, which orders tiles so that a lower tile of a slab is always taken by a CTA that is
// already running, (2) loads its kept rows into shared memory, (3) publishes a "loaded" flag,
// (4) waits until the (at most two) earlier tiles whose rows its destination range overlaps have
// published theirs, (5) stores.  The wait is bounded: when it runs out the CTA records
// GVOTE_ERR_TIMEOUT in the workspace status word, skips its stores and returns.
#include "common.cuh"

namespace gvote {
namespace {

constexpr int kScanThreads = 256;

// One CTA per (request, head): prefix[h][word] = kept keys of the request before this word.
// Also clears the compaction flags of the request's tiles (and the ticket, once).
__global__ void __launch_bounds__(kScanThreads)
mask_scan_kernel(const uint32_t* __restrict__ mask, const int32_t* __restrict__ cu, int Hkv, int64_t row_words,
                 int32_t* __restrict__ prefix, int32_t* __restrict__ budget, int32_t* __restrict__ flags,
                 int64_t n_tiles, int32_t* __restrict__ ticket) {
  __shared__ int warp_tot[kScanThreads / 32];
  __shared__ int carry;
  const int r = blockIdx.y, h = blockIdx.x;
  const int start = cu[r], N = cu[r + 1] - start;
  const int words = (N + 31) >> 5;
  const int64_t woff = mask_word_offset(start, r);
  const uint32_t* m = mask + (int64_t)h * row_words + woff;
  int32_t* pf = prefix + (int64_t)h * row_words + woff;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) carry = 0;
  if (r == 0 && h == 0 && tid == 0) { ticket[0] = 0; }
  if (flags) {
    const int tiles = (N + kCompactTile - 1) / kCompactTile;
    const int64_t toff = tile_offset(start, r);
    for (int t = tid; t < tiles; t += kScanThreads) {
      flags[((int64_t)(2 * h) * n_tiles) + toff + t] = 0;
      flags[((int64_t)(2 * h + 1) * n_tiles) + toff + t] = 0;
    }
  }
  __syncthreads();
  for (int base = 0; base < words; base += kScanThreads) {
    const int w = base + tid;
    const int c = (w < words) ? __popc(m[w]) : 0;
    int inc = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += t;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    int before = carry;
    for (int i = 0; i < warp; ++i) before += warp_tot[i];
    if (w < words) pf[w] = before + inc - c;
    __syncthreads();
    if (tid == kScanThreads - 1) carry = before + inc;
    __syncthreads();
  }
  if (tid == 0) budget[r * Hkv + h] = carry;
}

// Find the request that owns global tile index `gt` (tile_offset is increasing in r).
__device__ __forceinline__ int find_request(const int32_t* __restrict__ cu, int batch, int64_t gt) {
  int lo = 0, hi = batch - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (tile_offset(cu[mid], mid) <= gt) lo = mid; else hi = mid - 1;
  }
  return lo;
}

constexpr int kCompactThreads = 256;
constexpr int kSpinLimit = 1 << 22;

__global__ void __launch_bounds__(kCompactThreads)
compact_kernel(__nv_bfloat16* __restrict__ Kp, __nv_bfloat16* __restrict__ Vp, int64_t tok, int64_t head,
               const uint32_t* __restrict__ mask, const int32_t* __restrict__ prefix,
               const int32_t* __restrict__ cu, const int32_t* __restrict__ budget, int batch, int Hkv, int d_k,
               int64_t row_words, int64_t n_tiles, int32_t* flags, int32_t* ticket, int32_t* status) {
  extern __shared__ __align__(16) uint4 rows_sm[];   // [kept rows][d_k*2/16]
  __shared__ int s_ticket;
  __shared__ int s_src[kCompactTile];                // source token (within request) of each kept row
  __shared__ int s_ok;
  const int tid = threadIdx.x;
  if (tid == 0) s_ticket = atomicAdd(ticket, 1);
  __syncthreads();
  const int64_t tk = s_ticket;
  // ticket order: tile-major, then (head, K|V): lower tiles of a slab always come first
  const int slabs = 2 * Hkv;
  const int64_t gt = tk / slabs;
  const int slab = (int)(tk % slabs);
  const int h = slab >> 1;
  if (gt >= n_tiles) return;
  const int r = batch == 1 ? 0 : find_request(cu, batch, gt);
  const int start = cu[r], N = cu[r + 1] - start;
  const int t = (int)(gt - tile_offset(start, r));
  const int tiles = (N + kCompactTile - 1) / kCompactTile;
  if (t >= tiles) return;   // padding slot of the tile list
  __nv_bfloat16* base = ((slab & 1) ? Vp : Kp) + (int64_t)h * head + (int64_t)start * tok;
  int32_t* my_flags = flags + (int64_t)slab * n_tiles + tile_offset(start, r);

  // the tile's four mask words and its destination offset: every load below is issued before the
  // first of them is needed
  const int64_t woff = (int64_t)h * row_words + mask_word_offset(start, r) + (int64_t)t * (kCompactTile / 32);
  const int words = min(kCompactTile / 32, ((N + 31) >> 5) - t * (kCompactTile / 32));
  const int w_mine = min(tid >> 5, words - 1), lastw = words - 1;
  const int kept_all = budget[r * Hkv + h];
  const int dst0 = prefix[woff];
  const uint32_t mw = mask[woff + w_mine];
  const int pw = prefix[woff + w_mine];
  const int p_last = prefix[woff + lastw];
  const uint32_t m_last = mask[woff + lastw];
  // a head that keeps every key moves nothing, and none of its tiles waits for another
  if (kept_all == N) return;
  if (tid < kCompactTile && (tid >> 5) < words) {
    const int b = tid & 31;
    if ((mw >> b) & 1u) s_src[(pw - dst0) + __popc(mw & ((1u << b) - 1u))] = t * kCompactTile + tid;
  }
  const int cnt = p_last - dst0 + __popc(m_last);
  __syncthreads();
  const int pieces = d_k / 8;                       // 16-byte pieces per row
  // rows whose destination equals their source need no move; they form a prefix of the tile
  // exactly when nothing was dropped before them: dst0 + i == src_i.
  // All of a thread's pieces are requested before any is waited for (asynchronous copies straight
  // into shared memory); (row, piece) advance without divisions.
  const int step_i = kCompactThreads / pieces, step_pc = kCompactThreads % pieces;
  {
    int i = tid / pieces, pc = tid % pieces;
    for (int idx = tid; idx < cnt * pieces; idx += kCompactThreads) {
      const int src = s_src[i];
      if (src != dst0 + i) {
        const uint32_t dst_s = static_cast<uint32_t>(__cvta_generic_to_shared(&rows_sm[idx]));
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_s), "l"(base + (int64_t)src * tok + pc * 8)
                     : "memory");
      }
      i += step_i;
      pc += step_pc;
      if (pc >= pieces) { pc -= pieces; ++i; }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
  }
  __syncthreads();
  if (tid == 0) {
    __threadfence();
    atomicExch(&my_flags[t], 1);                    // our source rows are safe in shared memory
    // destination rows [dst0, dst0+cnt) live in tiles ta..tb (<= t); wait for those below t
    int ok = 1;
    if (cnt > 0) {
      const int ta = dst0 / kCompactTile, tb = (dst0 + cnt - 1) / kCompactTile;
      for (int w = ta; w <= tb && w < t; ++w) {
        int spins = 0;
        while (atomicAdd(&my_flags[w], 0) == 0) {
          if (++spins > kSpinLimit) { ok = 0; break; }
          __nanosleep(64);
        }
        if (!ok) break;
      }
      if (!ok) { atomicExch(&status[0], GVOTE_ERR_TIMEOUT); atomicExch(&status[1], 1); }
      __threadfence();
    }
    s_ok = ok;
  }
  __syncthreads();
  if (!s_ok) return;
  {
    int i = tid / pieces, pc = tid % pieces;
    for (int idx = tid; idx < cnt * pieces; idx += kCompactThreads) {
      if (s_src[i] != dst0 + i)
        *reinterpret_cast<uint4*>(base + (int64_t)(dst0 + i) * tok + pc * 8) = rows_sm[idx];
      i += step_i;
      pc += step_pc;
      if (pc >= pieces) { pc -= pieces; ++i; }
    }
  }
}

}  // namespace

int32_t launch_compact(const gvote_params* p, __nv_bfloat16* K, __nv_bfloat16* V, int64_t tok, int64_t head,
                       const uint32_t* mask, const int32_t* cu, int32_t batch, int64_t total_tokens, int64_t max_N,
                       int32_t* budget, const WorkspaceMap& m, char* ws, cudaStream_t st) {
  const int Hkv = p->n_kv_heads;
  int32_t* prefix = reinterpret_cast<int32_t*>(ws + m.prefix);
  int32_t* flags = reinterpret_cast<int32_t*>(ws + m.flags);
  int32_t* ticket = flags + (size_t)2 * Hkv * m.n_tiles;
  int32_t* status = reinterpret_cast<int32_t*>(ws + m.status);
  dim3 gs(Hkv, batch);
  {
    LaunchScope scope_("mask_scan_kernel", st);
  mask_scan_kernel<<<gs, kScanThreads, 0, st>>>(mask, cu, Hkv, m.row_words, prefix, budget, flags, m.n_tiles, ticket);
  }
  GVOTE_LAUNCH_CHECK("mask_scan_kernel");
  const size_t smem = (size_t)kCompactTile * p->d_k * sizeof(__nv_bfloat16);
  if (smem > 48 * 1024)
    GVOTE_CUDA_CHECK(cudaFuncSetAttribute(compact_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  const int64_t ctas = m.n_tiles * 2 * Hkv;
  {
    LaunchScope scope_("compact_kernel", st);
  compact_kernel<<<(unsigned)ctas, kCompactThreads, smem, st>>>(K, V, tok, head, mask, prefix, cu, budget, batch, Hkv,
                                                                p->d_k, m.row_words, m.n_tiles, flags, ticket, status);
  }
  GVOTE_LAUNCH_CHECK("compact_kernel");
  return GVOTE_OK;
}

}  // namespace gvote
