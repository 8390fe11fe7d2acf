// Algorithm 1 line 8 (and the logits of line 1) on the fifth-generation tensor cores:
// L = Q K^T / sqrt(d_k) for all (S+1)*G query rows of a KV head against that head's cached keys.
//
// Shape of the contraction.  Keys go on the MMA's M axis (128 keys per tile, read once from HBM by
// TMA with the 128-byte swizzle), query rows on its N axis (the head group's rows, padded to a
// multiple of 16, at most 240 per pass), d_k is the K axis.  Accumulators live in tensor memory,
// double buffered, so the MMA of tile t+1 overlaps the read-out of tile t.
//
// One persistent CTA walks the key tiles x, x+X, x+2X, ... of one (request, KV head, row chunk):
//   warp 0   : TMA producer - the group's query rows once, then a ring of key tiles
//   warp 1   : allocates tensor memory, issues tcgen05.mma, commits to the ring and to the read-out
//   warps 2-5: read-out - tcgen05.ld 32 rows at a time; thread = one key; scale; store
// The read-out never writes the S x N logits as fp32 in the default mode: rows of the current
// query (needed with full precision for the softmax mass) go out as fp32, rows of synthetic
// queries go out as the upper 16 bits of an order-preserving image of the logit, which is all the
// top-k search needs to bracket its threshold.
//
// Every wait on an mbarrier is bounded.  When one runs out the CTA raises a shared abort flag,
// records GVOTE_ERR_TIMEOUT in the workspace status word, leaves its loops, frees its tensor
// memory and returns.
#include "common.cuh"
#include "ptx.cuh"

namespace gvote {
namespace {

constexpr int kTileKeys = 128;
constexpr int kStages = 4;
constexpr int kUmmaThreads = 192;

struct ScoreSmemTail {
  uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t q_full;
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint32_t tmem_slot;
  volatile int abort_flag;
};

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t i = 0; i < (1u << 22); ++i) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((i & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

template <bool ALL_F32>
__global__ void __launch_bounds__(kUmmaThreads, 1)
score_umma_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ,
                  const int32_t* __restrict__ cu, int Hq, int G, int S1, int d_k, int RC, int row_chunks,
                  int acc_cols, float scale, float* __restrict__ logits, uint16_t* __restrict__ keys16,
                  int32_t* __restrict__ status) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const int r = blockIdx.z;
  const int kh = blockIdx.y / row_chunks, chunk = blockIdx.y % row_chunks;
  const int start = cu[r], N = cu[r + 1] - start;
  const int tiles = (N + kTileKeys - 1) / kTileKeys;
  const int kchunks = d_k / 64;
  const int R = G * S1;
  const int row0 = chunk * RC;                       // first group row of this CTA
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // shared memory carve-up (base is 1024-byte aligned; every operand block is a multiple of 1024)
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t q_bytes = (uint32_t)kchunks * RC * 128;
  const uint32_t stage_bytes = (uint32_t)kchunks * kTileKeys * 128;
  uint8_t* Qs = base;
  uint8_t* Ks = base + q_bytes;
  int64_t* row_meta = reinterpret_cast<int64_t*>(Ks + (size_t)kStages * stage_bytes);   // [RC]
  ScoreSmemTail* tail = reinterpret_cast<ScoreSmemTail*>(row_meta + RC);

  // per-row output offsets (relative to the request's block): bit 0 = "fp32 row"; -1 = padding row
  const int S = S1 - 1;
  const int64_t pitch16 = (N + 7) & ~7;
  for (int i = threadIdx.x; i < RC; i += blockDim.x) {
    const int row = row0 + i;
    int64_t meta = -1;
    if (row < R) {
      const int gl = row / S1, s = row % S1;
      const int g = kh * G + gl;
      if (ALL_F32 || s == 0) meta = ((((int64_t)g * S1 + s) * N) << 1) | 1;
      else meta = (((int64_t)g * S + (s - 1)) * pitch16) << 1;
    }
    row_meta[i] = meta;
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { ptx::mbar_init(&tail->full[s], 1); ptx::mbar_init(&tail->empty[s], 1); }
    ptx::mbar_init(&tail->q_full, 1);
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(&tail->tmem_full[a], 1); ptx::mbar_init(&tail->tmem_empty[a], 4); }
    tail->abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&tmK);
    ptx::prefetch_tensormap(&tmQ);
  }
  if (warp == 1) {
    ptx::tmem_alloc(&tail->tmem_slot, 2 * acc_cols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = tail->tmem_slot;
  volatile int* abort_flag = &tail->abort_flag;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && blockIdx.x < tiles) {
      const int q_row = (r * Hq + kh * G) * S1 + row0;
      ptx::mbar_arrive_expect_tx(&tail->q_full, q_bytes);
      for (int c = 0; c < kchunks; ++c) ptx::tma_load_2d(Qs + (size_t)c * RC * 128, &tmQ, &tail->q_full, c * 64, q_row);
      int it = 0;
      for (int t = blockIdx.x; t < tiles; t += gridDim.x, ++it) {
        const int s = it % kStages;
        const uint32_t ph = (uint32_t)(it / kStages) & 1u;
        if (!wait_or_abort(&tail->empty[s], ph ^ 1u, abort_flag)) break;
        ptx::mbar_arrive_expect_tx(&tail->full[s], stage_bytes);
        uint8_t* dst = Ks + (size_t)s * stage_bytes;
        for (int c = 0; c < kchunks; ++c)
          ptx::tma_load_3d(dst + (size_t)c * kTileKeys * 128, &tmK, &tail->full[s], c * 64, start + t * kTileKeys, kh);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && blockIdx.x < tiles) {
      const uint32_t idesc = ptx::instr_desc_bf16_f32(kTileKeys, RC);
      const uint32_t q_addr = ptx::smem_u32(Qs);
      bool ok = wait_or_abort(&tail->q_full, 0, abort_flag);
      int it = 0;
      for (int t = blockIdx.x; ok && t < tiles; t += gridDim.x, ++it) {
        const int s = it % kStages;
        const uint32_t ph = (uint32_t)(it / kStages) & 1u;
        const int a = it & 1;
        const uint32_t aph = (uint32_t)(it >> 1) & 1u;
        if (!wait_or_abort(&tail->tmem_empty[a], aph ^ 1u, abort_flag)) break;
        if (!wait_or_abort(&tail->full[s], ph, abort_flag)) break;
        ptx::tc_fence_after_sync();
        const uint32_t k_addr = ptx::smem_u32(Ks + (size_t)s * stage_bytes);
        const uint32_t d_tmem = tmem_base + (uint32_t)(a * acc_cols);
        const int ksteps = d_k / 16;
        for (int k = 0; k < ksteps; ++k) {
          const uint32_t koff = (uint32_t)(k >> 2), kin = (uint32_t)(k & 3) * 32u;
          const uint64_t da = ptx::smem_desc_k_sw128(k_addr + koff * (kTileKeys * 128) + kin);
          const uint64_t db = ptx::smem_desc_k_sw128(q_addr + koff * (uint32_t)(RC * 128) + kin);
          ptx::umma_bf16(d_tmem, da, db, idesc, k > 0 ? 1u : 0u);
        }
        ptx::umma_commit(&tail->empty[s]);       // the ring slot is free once these MMAs have read it
        ptx::umma_commit(&tail->tmem_full[a]);   // and the accumulator is complete
      }
    }
  } else {
    // ------------------------------------------------------------------ read-out (4 warps = 128 lanes)
    const int q = warp & 3;                      // tensor-memory lane quadrant this warp may read
    float* Lreq = logits + (int64_t)Hq * S1 * start;
    uint16_t* Kreq = keys16 + (int64_t)Hq * S * (((int64_t)(start + 7) & ~7) + 16 * (int64_t)r);
    int it = 0;
    bool ok = true;
    for (int t = blockIdx.x; ok && t < tiles; t += gridDim.x, ++it) {
      const int a = it & 1;
      const uint32_t aph = (uint32_t)(it >> 1) & 1u;
      if (!wait_or_abort(&tail->tmem_full[a], aph, abort_flag)) { ok = false; break; }
      ptx::tc_fence_after_sync();
      const int n = t * kTileKeys + q * 32 + lane;
      const bool valid = n < N;
      const uint32_t taddr = tmem_base + (uint32_t)(a * acc_cols) + ((uint32_t)(q * 32) << 16);
      for (int c0 = 0; c0 < RC; c0 += 32) {
        if (RC - c0 >= 32) {
          uint32_t v[32];
          ptx::tmem_ld_32x32(taddr + (uint32_t)c0, v);
          ptx::tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int64_t meta = row_meta[c0 + i];
            if (meta >= 0 && valid) {
              const float x = __uint_as_float(v[i]) * scale;
              if (meta & 1) Lreq[(meta >> 1) + n] = x;
              else Kreq[(meta >> 1) + n] = (uint16_t)(ordered_key(x) >> 16);
            }
          }
        } else {
          uint32_t v[16];
          ptx::tmem_ld_32x16(taddr + (uint32_t)c0, v);
          ptx::tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int64_t meta = row_meta[c0 + i];
            if (meta >= 0 && valid) {
              const float x = __uint_as_float(v[i]) * scale;
              if (meta & 1) Lreq[(meta >> 1) + n] = x;
              else Kreq[(meta >> 1) + n] = (uint16_t)(ordered_key(x) >> 16);
            }
          }
        }
      }
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&tail->tmem_empty[a]);
    }
  }

  // ------------------------------------------------------------------ teardown
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (threadIdx.x == 0 && tail->abort_flag) {
    atomicExch(&status[0], GVOTE_ERR_TIMEOUT);
    atomicExch(&status[1], 2);
  }
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, 2 * acc_cols);
  }
}

}  // namespace

// ------------------------------------------------------------------------------------ host side
bool score_umma_supported(const gvote_params* p) {
  return p->d_k % 64 == 0 && p->d_k <= 256;
}

size_t keys16_elems(const gvote_params* p, int32_t batch, int64_t total_tokens) {
  return (size_t)p->n_q_heads * p->S * (size_t)(((total_tokens + 7) & ~(int64_t)7) + 16 * (int64_t)batch);
}

// Returns GVOTE_OK, or GVOTE_ERR_UNSUPPORTED_SHAPE when the tensor maps cannot describe the
// operands (the caller then takes the SIMT path).
int32_t launch_score_umma(const gvote_params* p, const __nv_bfloat16* Q, const __nv_bfloat16* K, int64_t k_tok,
                          int64_t k_head, const int32_t* cu, int32_t batch, int64_t total_tokens, int64_t max_N,
                          bool all_f32, float* logits, uint16_t* keys16, int32_t* status, cudaStream_t st) {
  const int Hq = p->n_q_heads, Hkv = p->n_kv_heads, G = Hq / Hkv, S1 = p->S + 1, d_k = p->d_k;
  const int R = G * S1;
  const int row_chunks = (R + 239) / 240;
  int RC = (R + row_chunks - 1) / row_chunks;
  RC = (RC + 15) & ~15;
  if (RC < 16) RC = 16;
  int acc_cols = 32;
  while (acc_cols < RC) acc_cols <<= 1;

  CUtensorMap tmK, tmQ;
  {
    const uint64_t dims[3] = {(uint64_t)d_k, (uint64_t)total_tokens, (uint64_t)Hkv};
    const uint64_t strides[2] = {(uint64_t)k_tok * 2, (uint64_t)k_head * 2};
    const uint32_t box[3] = {64, (uint32_t)kTileKeys, 1};
    if (k_head <= 0 || !encode_tensor_map_bf16(&tmK, K, 3, dims, strides, box)) return GVOTE_ERR_UNSUPPORTED_SHAPE;
  }
  {
    const uint64_t dims[2] = {(uint64_t)d_k, (uint64_t)batch * Hq * S1};
    const uint64_t strides[1] = {(uint64_t)d_k * 2};
    const uint32_t box[2] = {64, (uint32_t)RC};
    if (!encode_tensor_map_bf16(&tmQ, Q, 2, dims, strides, box)) return GVOTE_ERR_UNSUPPORTED_SHAPE;
  }
  const int kchunks = d_k / 64;
  const size_t smem = 1024 + (size_t)kchunks * RC * 128 + (size_t)kStages * kchunks * kTileKeys * 128 +
                      (size_t)RC * sizeof(int64_t) + sizeof(ScoreSmemTail) + 64;
  if (smem > 227 * 1024) return GVOTE_ERR_UNSUPPORTED_SHAPE;
  const int64_t max_tiles = ceil_div(max_N, kTileKeys);
  // one CTA per SM when the batch is uniform; a ragged batch gets four times as many, shorter
  // CTAs so that the hardware scheduler can even out long and short requests
  const int64_t groups = (int64_t)Hkv * row_chunks * batch;
  int64_t X = (batch == 1 ? 148 : 592) / groups;
  if (X > max_tiles) X = max_tiles;
  if (X < 1) X = 1;
  dim3 grid((unsigned)X, (unsigned)(Hkv * row_chunks), (unsigned)batch);
  const float scale = (float)(1.0 / sqrt((double)d_k));
  auto kern = all_f32 ? score_umma_kernel<true> : score_umma_kernel<false>;
  GVOTE_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  {
    LaunchScope scope_("score_umma_kernel", st);
    kern<<<grid, kUmmaThreads, smem, st>>>(tmK, tmQ, cu, Hq, G, S1, d_k, RC, row_chunks, acc_cols, scale, logits,
                                           keys16, status);
  }
  GVOTE_LAUNCH_CHECK("score_umma_kernel");
  return GVOTE_OK;
}

}  // namespace gvote
