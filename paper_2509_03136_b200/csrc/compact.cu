// Algorithm 1, the pruning step: prune K and V to the keep-set, in place.
//
// Two kernels.  mask_scan_kernel turns each (request, KV head) bit row into an exclusive popcount
// prefix per 32-key word and the head's budget.  compact_kernel then fills one tile of 128 DESTINATION
// rows per CTA: thread = destination row, which finds its source row from the prefix, fetches it with
// one bulk copy into shared memory; the tile is written with one bulk copy.
//
// In-place safety.  Row i moves to row prefix(i) <= i, so the rows a tile overwrites may still be
// unread sources of an EARLIER tile of the same slab (never of a later one).  Each CTA therefore
// (1) takes a ticket of its slab, which orders tiles so that a lower tile of a slab is always taken by a
// CTA that is already running, (2) loads its rows into shared memory, (3) publishes a "loaded" flag,
// (4) waits until the (at most two) earlier tiles whose sources lie in the range it overwrites have
// published theirs, (5) stores.  The wait is bounded: when it runs out the CTA records
// GVOTE_ERR_TIMEOUT in the workspace status word, skips its stores and returns.
#include "common.cuh"
#include "ptx.cuh"

namespace gvote {
namespace {

constexpr int kScanThreads = 256;
constexpr int kTicketPitch = 32;     // ints between two slabs' ticket counters (128 bytes)

// One CTA per (request, head): prefix[h][word] = kept keys of the request before this word.
// Also clears the compaction flags of the request's tiles (and the head's two ticket counters).
// When the mask comes straight from the vote of the whole pass (`tmask` given), the head's tentative mask is
// OR-ed into the keep mask in the same sweep over the words - the union becoming final - unless the head was
// marked for the exact route, whose rows have written the keep mask themselves.
__global__ void __launch_bounds__(kScanThreads)
mask_scan_kernel(uint32_t* __restrict__ mask, const uint32_t* __restrict__ tmask, const uint32_t* __restrict__ head_bad,
                 const int32_t* __restrict__ cu, int Hkv, int64_t row_words, int32_t* __restrict__ prefix,
                 int32_t* __restrict__ budget, int32_t* __restrict__ flags, int64_t n_tiles,
                 int32_t* __restrict__ ticket) {
  __shared__ int warp_tot[kScanThreads / 32];
  __shared__ int carry;
  const int r = blockIdx.y, h = blockIdx.x;
  const int start = cu[r], N = cu[r + 1] - start;
  const int words = (N + 31) >> 5;
  const int64_t woff = mask_word_offset(start, r);
  uint32_t* m = mask + (int64_t)h * row_words + woff;
  const uint32_t* merge = (tmask && !head_bad[r * Hkv + h]) ? tmask + (int64_t)h * row_words + woff : nullptr;
  int32_t* pf = prefix + (int64_t)h * row_words + woff;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) carry = 0;
  if (r == 0 && tid < 2) ticket[(2 * h + tid) * kTicketPitch] = 0;   // this head's K and V slabs
  if (flags) {
    const int tiles = (N + kCompactTile - 1) / kCompactTile;
    const int64_t toff = tile_offset(start, r);
    for (int t = tid; t < tiles; t += kScanThreads) {
      flags[((int64_t)(2 * h) * n_tiles) + toff + t] = 0;
      flags[((int64_t)(2 * h + 1) * n_tiles) + toff + t] = 0;
    }
  }
  __syncthreads();
  // four consecutive words per thread and step (1024 words = 32768 keys per step): the thread scans
  // its own four, the CTA scans the threads' totals
  for (int base = 0; base < words; base += 4 * kScanThreads) {
    const int w0 = base + 4 * tid;
    uint32_t v[4], t[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      v[j] = (w0 + j < words) ? m[w0 + j] : 0u;
      t[j] = (merge && w0 + j < words) ? merge[w0 + j] : 0u;
    }
    int c[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (t[j] & ~v[j]) { v[j] |= t[j]; m[w0 + j] = v[j]; }
      c[j] = __popc(v[j]);
    }
    const int mine = c[0] + c[1] + c[2] + c[3];
    int inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int u = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += u;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    int before = carry;
    for (int i = 0; i < warp; ++i) before += warp_tot[i];
    int run = before + inc - mine;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (w0 + j < words) pf[w0 + j] = run;
      run += c[j];
    }
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

constexpr int kCompactThreads = kCompactTile;    // one thread per row of the tile
constexpr int kSpinLimit = 1 << 22;

// Position of the (rank+1)-th kept key of a request: the last mask word whose prefix does not exceed
// `rank`, then the bit inside it.  `pf` / `m`: the request's prefix and mask words, `words` of them.
__device__ __forceinline__ int kept_position(const int32_t* __restrict__ pf, const uint32_t* __restrict__ m, int words,
                                             int rank) {
  int lo = 0, hi = words - 1;                      // pf[lo] <= rank always (pf[0] = 0)
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (pf[mid] <= rank) lo = mid; else hi = mid - 1;
  }
  const int bit = __fns(m[lo], 0, rank - pf[lo] + 1);      // the (rank - pf[lo] + 1)-th set bit of the word
  return lo * 32 + bit;
}

// One CTA per 128 DESTINATION rows of a slab (a head's K or V of one request): thread j fetches the row
// that ends up at row 128 t + j - it finds its source position from the mask's popcount prefix - with one
// bulk copy into shared-memory slot j, and the tile leaves in one bulk copy (the destination rows are
// contiguous; with strided rows, one copy per row).  Tiles whose rows all stay where they are (the prefix of
// the slab up to the first dropped key) move nothing.
__global__ void __launch_bounds__(kCompactThreads)
compact_kernel(__nv_bfloat16* __restrict__ Kp, __nv_bfloat16* __restrict__ Vp, int64_t tok, int64_t head,
               const uint32_t* __restrict__ mask, const int32_t* __restrict__ prefix,
               const int32_t* __restrict__ cu, const int32_t* __restrict__ budget, int batch, int Hkv, int d_k,
               int64_t row_words, int64_t n_tiles, int32_t* flags, int32_t* ticket, int32_t* status) {
  extern __shared__ __align__(128) uint8_t rows_sm[];   // [128 rows][d_k * 2 bytes], in destination order
  __shared__ __align__(8) uint64_t s_bar;
  __shared__ int s_ticket;
  __shared__ int s_ok;
  __shared__ int s_moves;
  const int tid = threadIdx.x;
  // A CTA belongs to one slab by its block index and takes that slab's next tile: within a slab, a lower
  // tile is always taken by a CTA that is already running.  One counter per slab (on a line of its own)
  // instead of one for all keeps the atomics from queueing on one address.
  const int slabs = 2 * Hkv;
  const int slab = (int)(blockIdx.x % slabs);
  const int h = slab >> 1;
  if (tid == 0) {
    s_ticket = atomicAdd(&ticket[slab * kTicketPitch], 1);
    s_moves = 0;
    ptx::mbar_init(&s_bar, kCompactThreads);
    ptx::fence_barrier_init();
  }
  __syncthreads();
  const int64_t gt = s_ticket;
  if (gt >= n_tiles) return;
  const int r = batch == 1 ? 0 : find_request(cu, batch, gt);
  const int start = cu[r], N = cu[r + 1] - start;
  const int t = (int)(gt - tile_offset(start, r));
  const int kept_all = budget[r * Hkv + h];
  // tiles beyond the kept rows (and the padding slots of the tile list) have nothing to do, nor has a head
  // that keeps every key; nobody waits for their flags
  if (kept_all == N || (int64_t)t * kCompactTile >= kept_all) return;
  __nv_bfloat16* base = ((slab & 1) ? Vp : Kp) + (int64_t)h * head + (int64_t)start * tok;
  int32_t* my_flags = flags + (int64_t)slab * n_tiles + tile_offset(start, r);
  const int64_t woff = (int64_t)h * row_words + mask_word_offset(start, r);
  const int words = (N + 31) >> 5;
  const int dst0 = t * kCompactTile;
  const int cnt = min(kCompactTile, kept_all - dst0);

  // thread = destination row: where does it come from?
  const uint32_t row_bytes = (uint32_t)d_k * 2u;
  const bool have = tid < cnt;
  int src = -1;
  if (have) src = kept_position(prefix + woff, mask + woff, words, dst0 + tid);
  if (have && src != dst0 + tid) s_moves = 1;              // (same value from every writer)
  __syncthreads();
  const bool tile_moves = s_moves != 0;
  uint8_t* slot = rows_sm + (size_t)tid * row_bytes;
  if (have && tile_moves) {
    ptx::mbar_arrive_expect_tx(&s_bar, row_bytes);
    ptx::bulk_load(slot, base + (int64_t)src * tok, row_bytes, &s_bar);
  } else {
    ptx::mbar_arrive(&s_bar);
  }
  bool landed = ptx::mbar_wait(&s_bar, 0);
  if (!landed) landed = ptx::mbar_wait(&s_bar, 0);          // the copies are in flight: do not leave under them
  __syncthreads();
  if (tid == 0) {
    __threadfence();
    atomicExch(&my_flags[t], 1);                    // our source rows are safe in shared memory
    // The rows [dst0, dst0 + cnt) we are about to overwrite are sources of the tiles that hold the ranks of
    // the kept keys among positions dst0 .. dst0 + 127: tiles ta .. tb (at most two, none above t).  Wait
    // for those below t to have loaded.
    int ok = 1;
    if (tile_moves) {
      const int w0 = dst0 >> 5;                                         // word of position dst0 (dst0 < N here)
      const int w1 = min(w0 + kCompactTile / 32, words) - 1;            // last word of the 128 positions
      const int r0 = prefix[woff + w0];
      const int r1 = prefix[woff + w1] + __popc(mask[woff + w1]);       // ranks [r0, r1) live at those positions
      if (r1 > r0) {
        const int ta = r0 / kCompactTile, tb = (r1 - 1) / kCompactTile;
        for (int w = ta; w <= tb && w < t; ++w) {
          int spins = 0;
          while (atomicAdd(&my_flags[w], 0) == 0) {
            if (++spins > kSpinLimit) { ok = 0; break; }
            __nanosleep(64);
          }
          if (!ok) break;
        }
      }
      if (!ok) { atomicExch(&status[0], GVOTE_ERR_TIMEOUT); atomicExch(&status[1], 1); }
      __threadfence();
    }
    s_ok = ok;
  }
  if (!landed) { atomicExch(&status[0], GVOTE_ERR_TIMEOUT); atomicExch(&status[1], 4); }
  __syncthreads();
  if (!s_ok || !landed || !tile_moves) return;
  if (tok == d_k) {                                 // dense rows: the tile leaves in one copy
    if (tid == 0) {
      ptx::fence_proxy_async();
      ptx::bulk_store(base + (int64_t)dst0 * tok, rows_sm, (uint32_t)cnt * row_bytes);
      ptx::bulk_commit();
      ptx::bulk_wait_read<0>();                     // shared memory must outlive the copy's reads
    }
  } else if (have) {
    ptx::bulk_store(base + (int64_t)(dst0 + tid) * tok, slot, row_bytes);
    ptx::bulk_commit();
    ptx::bulk_wait_read<0>();
  }
}

// ---------------------------------------------------------------------------------- slot -> position map
// A cache that has been pruned carries, per KV head, the original position of every slot.  Pruning it
// again moves the kept entries of that map to the front of the slab exactly as the rows move:
// entry n goes to prefix(n).  Done out of place (gather into scratch, copy back): the map is 4 bytes
// per slot, and this way no ordering between CTAs is needed.
__global__ void __launch_bounds__(256)
remap_gather_kernel(const int32_t* __restrict__ token_pos, int64_t slab, const uint32_t* __restrict__ mask,
                    const int32_t* __restrict__ prefix, const int32_t* __restrict__ cu, int64_t row_words,
                    int32_t* __restrict__ tmp) {
  const int r = blockIdx.z, h = blockIdx.y;
  const int start = cu[r], N = cu[r + 1] - start;
  const int n = blockIdx.x * 256 + threadIdx.x;
  if (n >= N) return;
  const int64_t woff = (int64_t)h * row_words + mask_word_offset(start, r);
  const uint32_t bits = mask[woff + (n >> 5)];
  if (!((bits >> (n & 31)) & 1u)) return;
  const int dst = prefix[woff + (n >> 5)] + __popc(bits & ((1u << (n & 31)) - 1u));
  tmp[(int64_t)h * slab + start + dst] = token_pos[(int64_t)h * slab + start + n];
}

__global__ void __launch_bounds__(256)
remap_store_kernel(int32_t* __restrict__ token_pos, int64_t slab, const int32_t* __restrict__ tmp,
                   const int32_t* __restrict__ cu, const int32_t* __restrict__ budget, int Hkv) {
  const int r = blockIdx.z, h = blockIdx.y;
  const int start = cu[r];
  const int n = blockIdx.x * 256 + threadIdx.x;
  if (n >= budget[r * Hkv + h]) return;
  token_pos[(int64_t)h * slab + start + n] = tmp[(int64_t)h * slab + start + n];
}

}  // namespace

// `tmask`, `head_bad` (or null): the tentative mask of the vote that made this mask and its per-head flags; the
// scan then merges it into `mask` (see mask_scan_kernel).  Without them `mask` is only read.
int32_t launch_mask_scan(const gvote_params* p, const uint32_t* mask, const int32_t* cu, int32_t batch,
                         int32_t* budget, const WorkspaceMap& m, char* ws, cudaStream_t st, const uint32_t* tmask,
                         const uint32_t* head_bad) {
  const int Hkv = p->n_kv_heads;
  int32_t* prefix = reinterpret_cast<int32_t*>(ws + m.prefix);
  int32_t* flags = reinterpret_cast<int32_t*>(ws + m.flags);
  int32_t* ticket = flags + (size_t)2 * Hkv * m.n_tiles;
  dim3 gs(Hkv, batch);
  {
    LaunchScope scope_("mask_scan_kernel", st);
    launch_on(mask_scan_kernel, gs, dim3(kScanThreads), 0, st, const_cast<uint32_t*>(mask), tmask, head_bad, cu, Hkv, m.row_words,
              prefix, budget, flags, m.n_tiles, ticket);
  }
  GVOTE_LAUNCH_CHECK("mask_scan_kernel");
  return GVOTE_OK;
}

int32_t launch_compact(const gvote_params* p, __nv_bfloat16* K, __nv_bfloat16* V, int64_t tok, int64_t head,
                       const uint32_t* mask, const int32_t* cu, int32_t batch, int64_t total_tokens, int64_t max_N,
                       int32_t* budget, const WorkspaceMap& m, char* ws, cudaStream_t st, bool merge_tentative) {
  const int Hkv = p->n_kv_heads;
  const int32_t* prefix = reinterpret_cast<const int32_t*>(ws + m.prefix);
  int32_t* flags = reinterpret_cast<int32_t*>(ws + m.flags);
  int32_t* ticket = flags + (size_t)2 * Hkv * m.n_tiles;
  int32_t* status = reinterpret_cast<int32_t*>(ws + m.status);
  // (merge_tentative: the vote of this pass left its union in the workspace's tentative mask, see launch_vote)
  const int32_t rc = launch_mask_scan(p, mask, cu, batch, budget, m, ws, st,
                                      merge_tentative ? reinterpret_cast<const uint32_t*>(ws + m.tmask) : nullptr,
                                      merge_tentative ? reinterpret_cast<const uint32_t*>(ws + m.head_bad) : nullptr);
  if (rc != GVOTE_OK) return rc;
  const size_t smem = (size_t)kCompactTile * p->d_k * sizeof(__nv_bfloat16);
  if (smem > 48 * 1024)
    GVOTE_CUDA_CHECK(cudaFuncSetAttribute(compact_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  const int64_t ctas = m.n_tiles * 2 * Hkv;
  {
    LaunchScope scope_("compact_kernel", st);
    launch_on(compact_kernel, dim3((unsigned)ctas), dim3(kCompactThreads), smem, st, K, V, tok, head, mask, prefix, cu, budget, batch, Hkv,
                                                                  p->d_k, m.row_words, m.n_tiles, flags, ticket, status);
  }
  GVOTE_LAUNCH_CHECK("compact_kernel");
  return GVOTE_OK;
}

// After launch_compact (which leaves the prefix in the workspace and the budgets with the caller).
int32_t launch_remap(const gvote_params* p, int32_t* token_pos, const uint32_t* mask, const int32_t* cu, int32_t batch,
                     int64_t total_tokens, int64_t max_N, const int32_t* budget, const WorkspaceMap& m, char* ws,
                     cudaStream_t st) {
  if (max_N <= 0 || total_tokens <= 0) return GVOTE_OK;
  const int Hkv = p->n_kv_heads;
  const int32_t* prefix = reinterpret_cast<const int32_t*>(ws + m.prefix);
  int32_t* tmp = reinterpret_cast<int32_t*>(ws + m.remap_tmp);
  dim3 grid((unsigned)ceil_div(max_N, 256), (unsigned)Hkv, (unsigned)batch);
  {
    LaunchScope scope_("remap_gather_kernel", st);
    remap_gather_kernel<<<grid, 256, 0, st>>>(token_pos, total_tokens, mask, prefix, cu, m.row_words, tmp);
  }
  GVOTE_LAUNCH_CHECK("remap_gather_kernel");
  {
    LaunchScope scope_("remap_store_kernel", st);
    remap_store_kernel<<<grid, 256, 0, st>>>(token_pos, total_tokens, tmp, cu, budget, Hkv);
  }
  GVOTE_LAUNCH_CHECK("remap_store_kernel");
  return GVOTE_OK;
}

}  // namespace gvote
