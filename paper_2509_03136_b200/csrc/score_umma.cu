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
//   warps 2-9: read-out - tcgen05.ld 32 rows at a time; thread = one key; two warps per lane quadrant
//
// Read-out, default mode.  The S x N logits never reach HBM as fp32.  Every logit is scaled and
// turned into a 16-bit key (its half-precision rounding: all the top-k search needs to bracket its
// threshold), staged in shared memory as a [row][128 keys] tile and
// written with one bulk copy per tile into a tile-blocked buffer keys16[head][tile][chunk][row][128].
// Only the rows of the current query (one per query head) are also written as fp32, because the
// softmax mass of line 2 needs them exactly.  In the all-fp32 mode (per-sample top-p, softmax dump)
// every row is written as fp32 instead.
//
// Every wait on an mbarrier is bounded.  When one runs out the CTA raises a shared abort flag,
// records GVOTE_ERR_TIMEOUT in the workspace status word, leaves its loops, waits for its bulk
// copies, frees its tensor memory and returns.
#include "common.cuh"
#include "ptx.cuh"

namespace gvote {
namespace {

constexpr int kTileKeys = 128;
constexpr int kStages = 3;
constexpr int kEpiWarps = 8;
constexpr int kUmmaThreads = 64 + 32 * kEpiWarps;
constexpr int kMaxChunks32 = 8;   // RC <= 256
constexpr int kMaxGroup = 64;     // query heads per KV head

struct ScoreSmemTail {
  uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t q_full;
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint32_t tmem_slot;
  volatile int abort_flag;
  volatile int epi_go;                // read-out warps continue (decided by their leader, read after a barrier)
  uint32_t real_mask[kMaxChunks32];   // per 32-row chunk: rows that belong to the current query
  uint32_t rowmax[kMaxGroup];         // running maximum (order-preserving image) of each current-query row
};

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t i = 0; i < (1u << 22); ++i) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((i & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}


// Two fp32 logits -> two 16-bit keys: their half-precision roundings (monotone; 11 significant bits,
// values beyond the half range saturate to the largest finite half).
__device__ __forceinline__ uint32_t key16x2_of(float lo, float hi) {
  uint32_t p;
  asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(p) : "f"(hi), "f"(lo));
  return p;
}

// Read-out of NR accumulator columns (query rows c0 .. c0+NR-1) held by this thread for key n.
template <bool ALL_F32, int NR>
__device__ __forceinline__ void readout_chunk(const uint32_t (&v)[NR], int c0, uint32_t real_mask,
                                              const int64_t* row_meta, uint8_t* obuf, int m, int n, bool valid,
                                              float scale, float* Lreq, int N, int S1, int g0, int real_row0,
                                              uint32_t* rowmax_s) {
  if (ALL_F32) {
#pragma unroll
    for (int i = 0; i < NR; ++i) {
      const int64_t meta = row_meta[c0 + i];
      if (meta >= 0 && valid) Lreq[meta + n] = __uint_as_float(v[i]) * scale;
    }
  } else {
    // the scaled logit is what gets rounded: 1/sqrt(d_k) keeps it well inside the half range
    uint8_t* dst = obuf + (size_t)c0 * (kTileKeys * 2) + (size_t)m * 2;
#pragma unroll
    for (int i = 0; i < NR; i += 2) {
      const uint32_t kk = key16x2_of(__uint_as_float(v[i]) * scale, __uint_as_float(v[i + 1]) * scale);
      *reinterpret_cast<uint16_t*>(dst + i * (kTileKeys * 2)) = (uint16_t)kk;
      *reinterpret_cast<uint16_t*>(dst + (i + 1) * (kTileKeys * 2)) = (uint16_t)(kk >> 16);
    }
    if (real_mask != 0) {
      // rows of the current query (they follow the synthetic rows of the group): exact fp32 logits,
      // and their running maximum for the softmax of Algorithm 1 line 1 (real_mask is warp-uniform)
#pragma unroll
      for (int i = 0; i < NR; ++i) {
        if (real_mask & (1u << i)) {
          const int gl = real_row0 + c0 + i;
          const float l = __uint_as_float(v[i]) * scale;
          if (valid) Lreq[((int64_t)(g0 + gl) * S1) * N + n] = l;
          const uint32_t wmax = __reduce_max_sync(0xffffffffu, valid ? ordered_key(l) : 0u);
          if ((threadIdx.x & 31) == 0) atomicMax(&rowmax_s[gl], wmax);
        }
      }
    }
  }
}

template <bool ALL_F32>
__global__ void __launch_bounds__(kUmmaThreads, 1)
score_umma_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ,
                  const int32_t* __restrict__ cu, int Hq, int G, int S1, int d_k, int RC, int row_chunks,
                  int acc_cols, int n_out, float scale, int64_t n_tiles_total, float* __restrict__ logits,
                  uint16_t* __restrict__ keys16, uint32_t* __restrict__ rowmax, int32_t* __restrict__ status) {
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
  const uint32_t out_bytes = (uint32_t)RC * kTileKeys * 2;
  uint8_t* Qs = base;
  uint8_t* Ks = base + q_bytes;
  uint8_t* Os = Ks + (size_t)kStages * stage_bytes;                                        // [n_out][RC][128] u16
  int64_t* row_meta = reinterpret_cast<int64_t*>(Os + (ALL_F32 ? 0 : (size_t)n_out * out_bytes));   // [RC] (all-fp32 mode)
  ScoreSmemTail* tail = reinterpret_cast<ScoreSmemTail*>(row_meta + (ALL_F32 ? RC : 0));

  if (ALL_F32) {
    // fp32 offset of every row (relative to the request's block); -1 = padding row
    for (int i = threadIdx.x; i < RC; i += blockDim.x) {
      const int row = row0 + i;
      int64_t meta = -1;
      if (row < R) {
        const int S = S1 - 1;
        const int lrow = (row < G * S) ? (kh * G + row / S) * S1 + row % S + 1 : (kh * G + row - G * S) * S1;
        meta = (int64_t)lrow * N;
      }
      row_meta[i] = meta;
    }
  }
  if (threadIdx.x < kMaxChunks32) {
    uint32_t m = 0;
    for (int i = 0; i < 32; ++i) {
      const int row = row0 + (int)threadIdx.x * 32 + i;
      if ((int)threadIdx.x * 32 + i < RC && row < R && row >= G * (S1 - 1)) m |= 1u << i;
    }
    tail->real_mask[threadIdx.x] = m;
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { ptx::mbar_init(&tail->full[s], 1); ptx::mbar_init(&tail->empty[s], 1); }
    ptx::mbar_init(&tail->q_full, 1);
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(&tail->tmem_full[a], 1); ptx::mbar_init(&tail->tmem_empty[a], kEpiWarps); }
    tail->abort_flag = 0;
    for (int i = 0; i < kMaxGroup; ++i) tail->rowmax[i] = 0;
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
      const int q_row = (r * (Hq / G) + kh) * R + row0;   // the group's rows: synthetic first, then real
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
    // ------------------------------------------------------------------ read-out (8 warps)
    const int e = warp - 2;                      // 0..7
    const int q = warp & 3;                      // tensor-memory lane quadrant this warp may read
    const int half = e >> 2;                     // which 32-row chunks this warp takes (even / odd)
    const int m = q * 32 + lane;                 // key within the tile
    const bool leader = (e == 0 && lane == 0);
    float* Lreq = logits + (int64_t)Hq * S1 * start;
    const int64_t tile_base = ((int64_t)kh * n_tiles_total + tile_offset(start, r)) * row_chunks + chunk;
    int it = 0;
    for (int t = blockIdx.x; t < tiles; t += gridDim.x, ++it) {
      const int a = it & 1;
      const uint32_t aph = (uint32_t)(it >> 1) & 1u;
      const bool got = wait_or_abort(&tail->tmem_full[a], aph, abort_flag);
      if (ALL_F32 && !got) break;               // no CTA-wide barriers in this mode: a warp may leave alone
      ptx::tc_fence_after_sync();
      const int n = t * kTileKeys + m;
      const bool valid = n < N;
      const uint32_t taddr = tmem_base + (uint32_t)(a * acc_cols) + ((uint32_t)(q * 32) << 16);
      uint8_t* obuf = Os + (size_t)(it % n_out) * out_bytes;
      if (!ALL_F32) {
        // All eight warps reach this barrier in every iteration, so the decision to stop is uniform.
        // The staging buffer about to be overwritten must have been read by its bulk copy.
        if (leader) {
          if (n_out == 2) ptx::bulk_wait_read<1>(); else ptx::bulk_wait_read<0>();
          tail->epi_go = *abort_flag ? 0 : 1;
        }
        ptx::named_barrier_sync(1, kEpiWarps * 32);
        if (!tail->epi_go) break;
      }
      for (int c0 = half * 32; c0 < RC; c0 += 64) {
        const uint32_t rm = tail->real_mask[c0 >> 5];
        if (RC - c0 >= 32) {
          uint32_t v[32];
          ptx::tmem_ld_32x32(taddr + (uint32_t)c0, v);
          ptx::tmem_wait_ld();
          readout_chunk<ALL_F32, 32>(v, c0, rm, row_meta, obuf, m, n, valid, scale, Lreq, N, S1, kh * G, row0 - G * (S1 - 1), tail->rowmax);
        } else {
          uint32_t v[16];
          ptx::tmem_ld_32x16(taddr + (uint32_t)c0, v);
          ptx::tmem_wait_ld();
          readout_chunk<ALL_F32, 16>(v, c0, rm, row_meta, obuf, m, n, valid, scale, Lreq, N, S1, kh * G, row0 - G * (S1 - 1), tail->rowmax);
        }
      }
      // accumulator drained: hand it back to the MMA warp
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&tail->tmem_empty[a]);
      if (!ALL_F32) {
        ptx::fence_proxy_async();                // staged tile visible to the bulk-copy engine
        ptx::named_barrier_sync(2, kEpiWarps * 32);
        if (leader) {
          uint16_t* gdst = keys16 + ((tile_base + (int64_t)t * row_chunks) * RC) * kTileKeys;
          ptx::bulk_store(gdst, obuf, out_bytes);
          ptx::bulk_commit();
        }
      }
    }
    if (!ALL_F32 && leader) ptx::bulk_wait_all<0>();
  }

  // ------------------------------------------------------------------ teardown
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (threadIdx.x == 0 && tail->abort_flag) {
    atomicExch(&status[0], GVOTE_ERR_TIMEOUT);
    atomicExch(&status[1], 2);
  }
  if (!ALL_F32 && rowmax != nullptr && (int)threadIdx.x < G && tail->rowmax[threadIdx.x] != 0)
    atomicMax(&rowmax[r * Hq + kh * G + (int)threadIdx.x], tail->rowmax[threadIdx.x]);
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, 2 * acc_cols);
  }
}

}  // namespace

// ------------------------------------------------------------------------------------ host side
bool score_umma_supported(const gvote_params* p) {
  return p->d_k % 64 == 0 && p->d_k <= 256 && p->n_q_heads / p->n_kv_heads <= kMaxGroup;
}

ScoreGeometry score_geometry(const gvote_params* p) {
  ScoreGeometry g;
  const int R = (p->n_q_heads / p->n_kv_heads) * (p->S + 1);
  g.row_chunks = (R + 239) / 240;
  g.RC = (((R + g.row_chunks - 1) / g.row_chunks) + 15) & ~15;
  if (g.RC < 16) g.RC = 16;
  return g;
}

size_t keys16_elems(const gvote_params* p, int32_t batch, int64_t total_tokens) {
  if (!score_umma_supported(p)) return 0;
  const ScoreGeometry g = score_geometry(p);
  const int64_t n_tiles = (total_tokens >> 7) + batch;
  return (size_t)p->n_kv_heads * n_tiles * g.row_chunks * g.RC * kTileKeys;
}

// Returns GVOTE_OK, or GVOTE_ERR_UNSUPPORTED_SHAPE when the tensor maps cannot describe the
// operands (the caller then takes the SIMT path).
int32_t launch_score_umma(const gvote_params* p, const __nv_bfloat16* Q, const __nv_bfloat16* K, int64_t k_tok,
                          int64_t k_head, const int32_t* cu, int32_t batch, int64_t total_tokens, int64_t max_N,
                          bool all_f32, float* logits, uint16_t* keys16, uint32_t* rowmax, int32_t* status,
                          cudaStream_t st) {
  const int Hq = p->n_q_heads, Hkv = p->n_kv_heads, G = Hq / Hkv, S1 = p->S + 1, d_k = p->d_k;
  const ScoreGeometry geo = score_geometry(p);
  const int RC = geo.RC, row_chunks = geo.row_chunks;
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
  const size_t fixed = 1024 + (size_t)kchunks * RC * 128 + (size_t)kStages * kchunks * kTileKeys * 128 +
                       sizeof(ScoreSmemTail) + 64;
  const size_t out_bytes = (size_t)RC * kTileKeys * 2;
  int n_out = 2;
  size_t smem = fixed + (all_f32 ? (size_t)RC * sizeof(int64_t) : n_out * out_bytes);
  if (!all_f32 && smem > 227 * 1024) { n_out = 1; smem = fixed + out_bytes; }
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
  const int64_t n_tiles_total = (total_tokens >> 7) + batch;
  auto kern = all_f32 ? score_umma_kernel<true> : score_umma_kernel<false>;
  GVOTE_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  {
    LaunchScope scope_("score_umma_kernel", st);
    kern<<<grid, kUmmaThreads, smem, st>>>(tmK, tmQ, cu, Hq, G, S1, d_k, RC, row_chunks, acc_cols, n_out, scale,
                                           n_tiles_total, logits, keys16, rowmax, status);
  }
  GVOTE_LAUNCH_CHECK("score_umma_kernel");
  return GVOTE_OK;
}

}  // namespace gvote
