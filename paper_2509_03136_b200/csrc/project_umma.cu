// Algorithm 1, the projections of the current query and of the synthetic queries: the matrix product out[row][f] = sum_c X[row][c] * W_q[f][c] for the
// S+1 rows of every request (current query first, then the S synthetic hidden states), on the
// fifth-generation tensor cores.
//
// The product is tiny in rows (33 at S = 32) and large in weights (33.5 MB at Llama-3-8B shape), so
// the kernel is a stream over W_q that happens to multiply: output features go on the MMA's M axis
// (128 per CTA), the rows on its N axis (padded to a multiple of 16, at most 240 per pass), and d_h
// is split across CTAs so that every SM pulls its share of W_q.  Each CTA walks its slice of d_h in
// steps of 64 columns: TMA brings a [128 x 64] tile of W_q and a [rows x 64] tile of X (both with the
// 128-byte swizzle) into a ring of shared-memory stages, one thread issues four tcgen05.mma per
// stage, the fp32 accumulator lives in tensor memory.  The CTA's partial result goes to
// part[split][row][f]; the finishing kernel adds the splits in a fixed order (so the result does not
// depend on scheduling), adds the bias, rotates and rounds.
//
// Every mbarrier wait is bounded; on expiry the CTA raises GVOTE_ERR_TIMEOUT in the workspace status
// word, stops, frees its tensor memory and returns.
#include "common.cuh"
#include "ptx.cuh"

namespace gvote {
namespace {

constexpr int kFeatTile = 128;
constexpr int kProjThreads = 192;   // warp 0: TMA, warp 1: MMA, warps 2-5: read-out

struct ProjSmemTail {
  uint64_t full[8];
  uint64_t empty[8];
  uint64_t acc_full;
  uint32_t tmem_slot;
  volatile int abort_flag;
};

__device__ __forceinline__ bool proj_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t i = 0; i < (1u << 22); ++i) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((i & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

__global__ void __launch_bounds__(kProjThreads)
project_umma_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
                    int rows_total, int F, int kchunks_total, int kchunks_per_split, int NC, int acc_cols,
                    int stages, float* __restrict__ part, int32_t* __restrict__ status) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const int m_tile = blockIdx.x, split = blockIdx.y, rchunk = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int kc0 = split * kchunks_per_split;
  const int kc1 = min(kc0 + kchunks_per_split, kchunks_total);
  const int nk = max(kc1 - kc0, 0);
  const int row0 = rchunk * NC;

  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t w_bytes = kFeatTile * 128, x_bytes = (uint32_t)NC * 128;
  const uint32_t stage_bytes = w_bytes + x_bytes;
  ProjSmemTail* tail = reinterpret_cast<ProjSmemTail*>(base + (size_t)stages * stage_bytes);

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { ptx::mbar_init(&tail->full[s], 1); ptx::mbar_init(&tail->empty[s], 1); }
    ptx::mbar_init(&tail->acc_full, 1);
    tail->abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&tmW);
    ptx::prefetch_tensormap(&tmX);
  }
  if (warp == 1) {
    ptx::tmem_alloc(&tail->tmem_slot, (uint32_t)acc_cols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = tail->tmem_slot;
  volatile int* abort_flag = &tail->abort_flag;

  if (warp == 0) {
    if (lane == 0) {
      for (int it = 0; it < nk; ++it) {
        const int s = it % stages;
        const uint32_t ph = (uint32_t)(it / stages) & 1u;
        if (!proj_wait(&tail->empty[s], ph ^ 1u, abort_flag)) break;
        ptx::mbar_arrive_expect_tx(&tail->full[s], stage_bytes);
        uint8_t* dst = base + (size_t)s * stage_bytes;
        const int col = (kc0 + it) * 64;
        ptx::tma_load_2d(dst, &tmW, &tail->full[s], col, m_tile * kFeatTile);
        ptx::tma_load_2d(dst + w_bytes, &tmX, &tail->full[s], col, row0);
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && nk > 0) {
      const uint32_t idesc = ptx::instr_desc_bf16_f32(kFeatTile, NC);
      for (int it = 0; it < nk; ++it) {
        const int s = it % stages;
        const uint32_t ph = (uint32_t)(it / stages) & 1u;
        if (!proj_wait(&tail->full[s], ph, abort_flag)) break;
        ptx::tc_fence_after_sync();
        const uint32_t w_addr = ptx::smem_u32(base + (size_t)s * stage_bytes);
        const uint32_t x_addr = w_addr + w_bytes;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const uint64_t da = ptx::smem_desc_k_sw128(w_addr + (uint32_t)k * 32u);
          const uint64_t db = ptx::smem_desc_k_sw128(x_addr + (uint32_t)k * 32u);
          ptx::umma_bf16(tmem_base, da, db, idesc, (it > 0 || k > 0) ? 1u : 0u);
        }
        ptx::umma_commit(&tail->empty[s]);
      }
      ptx::umma_commit(&tail->acc_full);
    }
  } else {
    // read-out: thread = output feature (tensor-memory lane), registers = rows
    const int q = warp & 3;
    const int f = m_tile * kFeatTile + q * 32 + lane;
    float* out = part + ((size_t)split * rows_total) * F;
    bool got = nk > 0 && proj_wait(&tail->acc_full, 0, abort_flag);
    ptx::tc_fence_after_sync();
    for (int c0 = 0; c0 < NC; c0 += 16) {
      uint32_t v[16];
      if (got) {
        ptx::tmem_ld_32x16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
        ptx::tmem_wait_ld();
      } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = 0u;      // an empty slice contributes zeros
      }
      if (f < F) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int row = row0 + c0 + i;
          if (row < rows_total) out[(size_t)row * F + f] = __uint_as_float(v[i]);
        }
      }
    }
  }

  ptx::tc_fence_before_sync();
  __syncthreads();
  if (threadIdx.x == 0 && tail->abort_flag) {
    atomicExch(&status[0], GVOTE_ERR_TIMEOUT);
    atomicExch(&status[1], 3);
  }
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, (uint32_t)acc_cols);
  }
}

}  // namespace

// Split count the tensor-core projection uses for this shape (also sizes the partial buffer).
int project_umma_splits(const gvote_params* p, int rows_total) {
  const int F = p->n_q_heads * p->d_k;
  const int m_tiles = (int)ceil_div(F, kFeatTile);
  const int kchunks = (int)ceil_div(p->d_h, 64);
  const int rchunks = (int)ceil_div(rows_total, 240);
  // at most one CTA per SM of a 148-SM part (its ring is 100 KB, so the rest of the SM stays free for
  // the kernels of other layers on other streams: fewer, longer CTAs take a little longer alone and
  // less out of an overlapped pass), every CTA with at least four 64-column steps
  int splits = (int)(148 / ((int64_t)m_tiles * rchunks));
  if (splits > kchunks / 4) splits = kchunks / 4;
  if (splits < 1) splits = 1;
  if (splits > 16) splits = 16;
  const int per = (int)ceil_div(kchunks, splits);
  return (int)ceil_div(kchunks, per);      // no empty split
}

// Returns GVOTE_ERR_UNSUPPORTED_SHAPE when the tensor maps cannot describe the operands.
int32_t launch_project_umma(const gvote_params* p, const __nv_bfloat16* X, const __nv_bfloat16* W, int64_t wq_ld,
                            int rows_total, int splits, float* part, int32_t* status, cudaStream_t st) {
  const int d_h = p->d_h, F = p->n_q_heads * p->d_k;
  const int kchunks = (int)ceil_div(d_h, 64);
  const int per = (int)ceil_div(kchunks, splits);
  const int rchunks = (int)ceil_div(rows_total, 240);
  int NC = (int)((ceil_div(rows_total, rchunks) + 15) & ~(int64_t)15);
  if (NC < 16) NC = 16;
  int acc_cols = 32;
  while (acc_cols < NC) acc_cols <<= 1;

  CUtensorMap tmW, tmX;
  {
    const uint64_t dims[2] = {(uint64_t)d_h, (uint64_t)F};
    const uint64_t strides[1] = {(uint64_t)wq_ld * 2};
    const uint32_t box[2] = {64, (uint32_t)kFeatTile};
    if (!encode_tensor_map_bf16(&tmW, W, 2, dims, strides, box)) return GVOTE_ERR_UNSUPPORTED_SHAPE;
  }
  {
    const uint64_t dims[2] = {(uint64_t)d_h, (uint64_t)rows_total};
    const uint64_t strides[1] = {(uint64_t)d_h * 2};
    const uint32_t box[2] = {64, (uint32_t)NC};
    if (!encode_tensor_map_bf16(&tmX, X, 2, dims, strides, box)) return GVOTE_ERR_UNSUPPORTED_SHAPE;
  }
  const size_t stage_bytes = (size_t)kFeatTile * 128 + (size_t)NC * 128;
  int stages = (int)((100 * 1024) / stage_bytes);
  if (stages > 8) stages = 8;
  if (stages < 3) stages = 3;
  if (stages > per) stages = per < 2 ? 2 : per;
  const size_t smem = 1024 + stages * stage_bytes + sizeof(ProjSmemTail) + 64;
  if (smem > 227 * 1024) return GVOTE_ERR_UNSUPPORTED_SHAPE;
  GVOTE_CUDA_CHECK(cudaFuncSetAttribute(project_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  dim3 grid((unsigned)ceil_div(F, kFeatTile), (unsigned)splits, (unsigned)rchunks);
  {
    LaunchScope scope_("project_umma_kernel", st);
    launch_on(project_umma_kernel, grid, dim3(kProjThreads), smem, st, tmW, tmX, rows_total, F, kchunks, per, NC, acc_cols, stages,
                                                          part, status);
  }
  GVOTE_LAUNCH_CHECK("project_umma_kernel");
  return GVOTE_OK;
}

}  // namespace gvote
