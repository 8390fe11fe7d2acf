// Section 3.4 of the paper: after pruning, every KV head keeps a different number of rows, and the
// decode path consumes such a cache through a variable-length attention kernel.  gvote_pack writes
// that layout directly from the unpruned cache and the keep mask: one dense [total_kept, d_k] buffer
// for K and one for V, in which "sequence" s = request * n_kv_heads + head owns rows
// cu_seqlens_k[s] .. cu_seqlens_k[s+1]-1, kept rows in ascending key order.
//
// Out of place, so there is no ordering between tiles: the mask scan of the compaction gives every
// 32-key word its number of kept predecessors, a one-CTA scan of the budgets gives cu_seqlens_k, and
// then one CTA per (128-token tile, head, K|V) fetches its kept rows with one bulk copy each into
// shared memory, in rank order, and sends them out with a single bulk copy: the tile's kept rows are
// contiguous in the packed buffer.
#include "common.cuh"
#include "ptx.cuh"

namespace gvote {

int32_t launch_mask_scan(const gvote_params* p, const uint32_t* mask, const int32_t* cu, int32_t batch,
                         int32_t* budget, const WorkspaceMap& m, char* ws, cudaStream_t st, const uint32_t* tmask = nullptr,
                         const uint32_t* head_bad = nullptr);

namespace {

constexpr int kPackThreads = kCompactTile;

// cu_k[0] = 0, cu_k[s+1] = budget[0] + .. + budget[s]  (s < n); one CTA.
__global__ void __launch_bounds__(1024)
pack_offsets_kernel(const int32_t* __restrict__ budget, int n, int32_t* __restrict__ cu_k) {
  __shared__ int warp_tot[32];
  __shared__ int carry;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) { carry = 0; cu_k[0] = 0; }
  __syncthreads();
  for (int base = 0; base < n; base += 1024) {
    const int i = base + tid;
    const int v = i < n ? budget[i] : 0;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += t;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    int before = carry;
    for (int w = 0; w < warp; ++w) before += warp_tot[w];
    if (i < n) cu_k[i + 1] = before + inc;
    __syncthreads();
    if (tid == 1023) carry = before + inc;
    __syncthreads();
  }
}

__device__ __forceinline__ int find_request_of_tile(const int32_t* __restrict__ cu, int batch, int64_t gt) {
  int lo = 0, hi = batch - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (tile_offset(cu[mid], mid) <= gt) lo = mid; else hi = mid - 1;
  }
  return lo;
}

__global__ void __launch_bounds__(kPackThreads)
pack_kernel(const __nv_bfloat16* __restrict__ Kp, const __nv_bfloat16* __restrict__ Vp, int64_t tok, int64_t head,
            const uint32_t* __restrict__ mask, const int32_t* __restrict__ prefix, const int32_t* __restrict__ cu,
            const int32_t* __restrict__ cu_k, int batch, int Hkv, int d_k, int64_t row_words, int64_t n_tiles,
            __nv_bfloat16* __restrict__ Kout, __nv_bfloat16* __restrict__ Vout, int64_t capacity_rows,
            int32_t* status) {
  extern __shared__ __align__(128) uint8_t rows_sm[];   // [kept rows][d_k * 2 bytes]
  __shared__ __align__(8) uint64_t s_bar;
  const int tid = threadIdx.x;
  const int slabs = 2 * Hkv;
  const int64_t gt = blockIdx.x / slabs;
  const int slab = (int)(blockIdx.x % slabs), h = slab >> 1;
  const int r = batch == 1 ? 0 : find_request_of_tile(cu, batch, gt);
  const int start = cu[r], N = cu[r + 1] - start;
  const int t = (int)(gt - tile_offset(start, r));
  if (t >= (N + kCompactTile - 1) / kCompactTile) return;   // padding slot of the tile list
  if (tid == 0) {
    ptx::mbar_init(&s_bar, kPackThreads);
    ptx::fence_barrier_init();
  }
  const int64_t woff = (int64_t)h * row_words + mask_word_offset(start, r) + (int64_t)t * (kCompactTile / 32);
  const int words = min(kCompactTile / 32, ((N + 31) >> 5) - t * (kCompactTile / 32));
  const int w_mine = min(tid >> 5, words - 1), lastw = words - 1;
  const int seq0 = cu_k[r * Hkv + h];
  const int dst0 = prefix[woff];
  const uint32_t mw = mask[woff + w_mine];
  const int pw = prefix[woff + w_mine];
  const int p_last = prefix[woff + lastw];
  const uint32_t m_last = mask[woff + lastw];
  const int cnt = p_last - dst0 + __popc(m_last);
  __syncthreads();
  if (cnt == 0) return;
  const int64_t out_row = (int64_t)seq0 + dst0;
  if (out_row + cnt > capacity_rows) {                      // the caller's buffers are too small
    if (tid == 0) { atomicExch(&status[0], GVOTE_ERR_WORKSPACE_TOO_SMALL); atomicExch(&status[1], 5); }
    return;
  }
  const uint32_t row_bytes = (uint32_t)d_k * 2u;
  const __nv_bfloat16* base = ((slab & 1) ? Vp : Kp) + (int64_t)h * head + (int64_t)start * tok;
  const int b = tid & 31;
  const bool kept = (tid >> 5) < words && ((mw >> b) & 1u);
  const int rank = (pw - dst0) + __popc(mw & ((1u << b) - 1u));
  if (kept) {
    ptx::mbar_arrive_expect_tx(&s_bar, row_bytes);
    ptx::bulk_load(rows_sm + (size_t)rank * row_bytes, base + (int64_t)(t * kCompactTile + tid) * tok, row_bytes, &s_bar);
  } else {
    ptx::mbar_arrive(&s_bar);
  }
  bool landed = ptx::mbar_wait(&s_bar, 0);
  if (!landed) landed = ptx::mbar_wait(&s_bar, 0);          // the copies are in flight: do not leave under them
  if (!landed) {
    atomicExch(&status[0], GVOTE_ERR_TIMEOUT);
    atomicExch(&status[1], 6);
    return;
  }
  if (tid == 0) {
    __nv_bfloat16* out = ((slab & 1) ? Vout : Kout) + out_row * d_k;
    ptx::bulk_store(out, rows_sm, (uint32_t)cnt * row_bytes);
    ptx::bulk_commit();
    ptx::bulk_wait_read<0>();                               // shared memory must outlive the copy's reads
  }
}

}  // namespace

int32_t launch_pack(const gvote_params* p, const __nv_bfloat16* K, const __nv_bfloat16* V, int64_t tok, int64_t head,
                    const uint32_t* mask, const int32_t* cu, int32_t batch, int64_t total_tokens, int64_t max_N,
                    __nv_bfloat16* K_packed, __nv_bfloat16* V_packed, int64_t capacity_rows, int32_t* cu_seqlens_k,
                    int32_t* budget, const WorkspaceMap& m, char* ws, cudaStream_t st) {
  const int Hkv = p->n_kv_heads;
  const int32_t rc = launch_mask_scan(p, mask, cu, batch, budget, m, ws, st);
  if (rc != GVOTE_OK) return rc;
  {
    LaunchScope scope_("pack_offsets_kernel", st);
    pack_offsets_kernel<<<1, 1024, 0, st>>>(budget, batch * Hkv, cu_seqlens_k);
  }
  GVOTE_LAUNCH_CHECK("pack_offsets_kernel");
  const int32_t* prefix = reinterpret_cast<const int32_t*>(ws + m.prefix);
  int32_t* status = reinterpret_cast<int32_t*>(ws + m.status);
  const size_t smem = (size_t)kCompactTile * p->d_k * sizeof(__nv_bfloat16);
  if (smem > 48 * 1024)
    GVOTE_CUDA_CHECK(cudaFuncSetAttribute(pack_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  const int64_t ctas = m.n_tiles * 2 * Hkv;
  {
    LaunchScope scope_("pack_kernel", st);
    pack_kernel<<<(unsigned)ctas, kPackThreads, smem, st>>>(K, V, tok, head, mask, prefix, cu, cu_seqlens_k, batch, Hkv,
                                                            p->d_k, m.row_words, m.n_tiles, K_packed, V_packed,
                                                            capacity_rows, status);
  }
  GVOTE_LAUNCH_CHECK("pack_kernel");
  return GVOTE_OK;
}

}  // namespace gvote
