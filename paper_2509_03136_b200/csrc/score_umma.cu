// The logits of Algorithm 1 for every query row, as fp32 rows in memory, on the fifth-generation tensor
// cores: L = Q K^T / sqrt(d_k) for all (S+1)*G query rows of a KV head against that head's cached keys.
// This is the route of the per-sample top-p mode (Section 3.1's rule applied to every synthetic query,
// which needs each row's softmax mass) and of the softmax dump; the default top-k mode never writes
// these rows (sweep_umma.cu).
//
// Shape of the contraction.  A KV head's G*S synthetic rows are cut into chunks of 128, and a chunk
// goes on the MMA's M axis: D1[128 rows x 128 keys] = Qs (128 x d_k) * Ktile^T per 128-key tile, so that
// in tensor memory a lane is a query row and a column is a key.  The G current-query rows ride along in
// a second, thin product with the roles swapped, D2[128 keys x 16] = Ktile * Qr^T, whose read-out thread
// is a key and writes coalesced fp32 rows.  Both products read the same K tile in shared memory (TMA,
// 128-byte swizzle, read once from HBM); both accumulators are double buffered in tensor memory so that
// the MMAs of tile t+1 overlap the read-out of tile t.
//
// One persistent CTA walks the key tiles x, x+X, x+2X, ... of one (request, KV head, row chunk):
//   warp 0   : TMA producer - the chunk's query rows once, then a ring of key tiles
//   warp 1   : allocates tensor memory, issues tcgen05.mma, commits to the ring and to the read-out
//   warps 2-9: read-out - two warps per lane quadrant, each takes 64 of the tile's 128 keys; the rows are
//              staged in shared memory (16-byte chunks XOR-swizzled by the row) and written out row by row
//
// Every wait on an mbarrier is bounded.  When one runs out the CTA raises a shared abort flag,
// records GVOTE_ERR_TIMEOUT in the workspace status word, leaves its loops, frees its tensor memory
// and returns.
#include "common.cuh"
#include "ptx.cuh"

namespace gvote {
namespace {

constexpr int kTileKeys = 128;
constexpr int kRowChunk = 128;    // synthetic rows per CTA (MMA M)
constexpr int kRealCols = 16;     // current-query rows per KV head the thin product holds (MMA N)
constexpr int kEpiWarps = 8;
constexpr int kUmmaThreads = 64 + 32 * kEpiWarps;
constexpr int kMaxStages = 3;
constexpr int kTmemCols = 512;    // 2 x 128 (D1) + 2 x 32 (D2, 16 used)
constexpr int kD2Col = 256;

struct ScoreSmemTail {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t q_full;
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint32_t tmem_slot;
  volatile int abort_flag;
  volatile int epi_go;                // read-out warps continue (decided by their leader, read after a barrier)
};

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t i = 0; i < (1u << 22); ++i) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((i & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

__device__ __forceinline__ float4 logits4(const uint32_t* v, float scale) {
  return make_float4(__uint_as_float(v[0]) * scale, __uint_as_float(v[1]) * scale, __uint_as_float(v[2]) * scale,
                     __uint_as_float(v[3]) * scale);
}

__global__ void __launch_bounds__(kUmmaThreads, 1)
score_umma_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ,
                  const __grid_constant__ CUtensorMap tmQr, const int32_t* __restrict__ cu, int Hq, int G, int S1,
                  int d_k, int row_chunks, int stages, float scale, float* __restrict__ logits,
                  int32_t* __restrict__ status, const int32_t* __restrict__ kv_len) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const int r = blockIdx.z;
  const int kh = blockIdx.y / row_chunks, chunk = blockIdx.y % row_chunks;
  const int start = cu[r], Ncap = cu[r + 1] - start;       // Ncap: rows of the slab (layout); N: rows that count
  const int N = valid_keys(kv_len, r, Hq / G, kh, Ncap);
  const int tiles = (N + kTileKeys - 1) / kTileKeys;
  const int kchunks = d_k / 64;
  const int S = S1 - 1;
  const int R = G * S1;                              // rows of the head group: G*S synthetic, then G current
  const int row0 = chunk * kRowChunk;                // first synthetic row of this CTA
  const bool with_real = chunk == 0;                 // chunk 0 also carries the current-query rows
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // shared memory carve-up (base is 1024-byte aligned; every operand block is a multiple of 1024)
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t q_bytes = (uint32_t)kchunks * kRowChunk * 128;
  const uint32_t qr_bytes = (uint32_t)kchunks * kRealCols * 128;
  const uint32_t stage_bytes = (uint32_t)kchunks * kTileKeys * 128;
  const uint32_t out_bytes = (uint32_t)kRowChunk * kTileKeys * 4;
  uint8_t* Qs = base;
  uint8_t* Qr = Qs + q_bytes;
  uint8_t* Ks = Qr + ((qr_bytes + 1023u) & ~1023u);
  uint8_t* Os = Ks + (size_t)stages * stage_bytes;
  ScoreSmemTail* tail = reinterpret_cast<ScoreSmemTail*>(Os + out_bytes);

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { ptx::mbar_init(&tail->full[s], 1); ptx::mbar_init(&tail->empty[s], 1); }
    ptx::mbar_init(&tail->q_full, 1);
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(&tail->tmem_full[a], 1); ptx::mbar_init(&tail->tmem_empty[a], kEpiWarps); }
    tail->abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&tmK);
    ptx::prefetch_tensormap(&tmQ);
    ptx::prefetch_tensormap(&tmQr);
  }
  if (warp == 1) {
    ptx::tmem_alloc(&tail->tmem_slot, kTmemCols);
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
      const int group_row = (r * (Hq / G) + kh) * R;    // the group's rows: synthetic first, then current
      ptx::mbar_arrive_expect_tx(&tail->q_full, q_bytes + (with_real ? qr_bytes : 0u));
      for (int c = 0; c < kchunks; ++c) {
        ptx::tma_load_2d(Qs + (size_t)c * kRowChunk * 128, &tmQ, &tail->q_full, c * 64, group_row + row0);
        if (with_real)
          ptx::tma_load_2d(Qr + (size_t)c * kRealCols * 128, &tmQr, &tail->q_full, c * 64, group_row + G * S);
      }
      int it = 0;
      for (int t = blockIdx.x; t < tiles; t += gridDim.x, ++it) {
        const int s = it % stages;
        const uint32_t ph = (uint32_t)(it / stages) & 1u;
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
      const uint32_t idesc1 = ptx::instr_desc_bf16_f32(kRowChunk, kTileKeys);   // rows x keys
      const uint32_t idesc2 = ptx::instr_desc_bf16_f32(kTileKeys, kRealCols);   // keys x current rows
      const uint32_t q_addr = ptx::smem_u32(Qs), qr_addr = ptx::smem_u32(Qr);
      const bool ok = wait_or_abort(&tail->q_full, 0, abort_flag);
      int it = 0;
      for (int t = blockIdx.x; ok && t < tiles; t += gridDim.x, ++it) {
        const int s = it % stages;
        const uint32_t ph = (uint32_t)(it / stages) & 1u;
        const int a = it & 1;
        const uint32_t aph = (uint32_t)(it >> 1) & 1u;
        if (!wait_or_abort(&tail->tmem_empty[a], aph ^ 1u, abort_flag)) break;
        if (!wait_or_abort(&tail->full[s], ph, abort_flag)) break;
        ptx::tc_fence_after_sync();
        const uint32_t k_addr = ptx::smem_u32(Ks + (size_t)s * stage_bytes);
        const uint32_t d1 = tmem_base + (uint32_t)(a * kRowChunk);
        const uint32_t d2 = tmem_base + (uint32_t)(kD2Col + a * 32);
        const int ksteps = d_k / 16;
        for (int k = 0; k < ksteps; ++k) {
          const uint32_t koff = (uint32_t)(k >> 2), kin = (uint32_t)(k & 3) * 32u;
          const uint64_t dq = ptx::smem_desc_k_sw128(q_addr + koff * (uint32_t)(kRowChunk * 128) + kin);
          const uint64_t dk = ptx::smem_desc_k_sw128(k_addr + koff * (uint32_t)(kTileKeys * 128) + kin);
          ptx::umma_bf16(d1, dq, dk, idesc1, k > 0 ? 1u : 0u);
        }
        if (with_real) {
          for (int k = 0; k < ksteps; ++k) {
            const uint32_t koff = (uint32_t)(k >> 2), kin = (uint32_t)(k & 3) * 32u;
            const uint64_t dk = ptx::smem_desc_k_sw128(k_addr + koff * (uint32_t)(kTileKeys * 128) + kin);
            const uint64_t dq = ptx::smem_desc_k_sw128(qr_addr + koff * (uint32_t)(kRealCols * 128) + kin);
            ptx::umma_bf16(d2, dk, dq, idesc2, k > 0 ? 1u : 0u);
          }
        }
        ptx::umma_commit(&tail->empty[s]);       // the ring slot is free once these MMAs have read it
        ptx::umma_commit(&tail->tmem_full[a]);   // and the accumulators are complete
      }
    }
  } else {
    // ------------------------------------------------------------------ read-out (8 warps)
    const int e = warp - 2;                      // 0..7
    const int q = warp & 3;                      // tensor-memory lane quadrant this warp may read
    const int half = e >> 2;                     // which 64 keys of the tile this warp takes
    const int row = q * 32 + lane;               // D1 lane = synthetic row of the chunk; D2 lane = key of the tile
    const bool leader = (e == 0 && lane == 0);
    float* Lreq = logits + (int64_t)Hq * S1 * start;
    int it = 0;
    for (int t = blockIdx.x; t < tiles; t += gridDim.x, ++it) {
      const int a = it & 1;
      const uint32_t aph = (uint32_t)(it >> 1) & 1u;
      wait_or_abort(&tail->tmem_full[a], aph, abort_flag);
      ptx::tc_fence_after_sync();
      uint8_t* obuf = Os;
      // All eight warps reach this barrier in every iteration, so the decision to stop is uniform.
      // The staging buffer about to be overwritten has been read by the row writer of the previous
      // iteration (every warp is past it here).
      if (leader) tail->epi_go = *abort_flag ? 0 : 1;
      ptx::named_barrier_sync(1, kEpiWarps * 32);
      if (!tail->epi_go) break;

      // ---- synthetic rows: thread = row, 64 consecutive keys in two loads
      const uint32_t taddr = tmem_base + (uint32_t)(a * kRowChunk) + ((uint32_t)(q * 32) << 16) + (uint32_t)(half * 64);
      uint32_t v0[32], v1[32];
      ptx::tmem_ld_32x32(taddr, v0);
      ptx::tmem_ld_32x32(taddr + 32u, v1);
      ptx::tmem_wait_ld();
      {
        // fp32 staging: 16-byte chunk c of the row (keys 4c .. 4c+3) at chunk position c ^ (row & 31)
        uint8_t* orow = obuf + (size_t)row * (kTileKeys * 4);
        const uint32_t swz = (uint32_t)row & 31u;
#pragma unroll
        for (int c = 0; c < 8; ++c)
          *reinterpret_cast<float4*>(orow + ((((uint32_t)(half * 16 + c)) ^ swz) << 4)) = logits4(&v0[4 * c], scale);
#pragma unroll
        for (int c = 0; c < 8; ++c)
          *reinterpret_cast<float4*>(orow + ((((uint32_t)(half * 16 + 8 + c)) ^ swz) << 4)) = logits4(&v1[4 * c], scale);
      }

      // ---- current-query rows (chunk 0 only): thread = key, exact fp32 logits for the softmax row A0
      if (with_real && half == 0) {
        uint32_t w[16];
        ptx::tmem_ld_32x16(tmem_base + (uint32_t)(kD2Col + a * 32) + ((uint32_t)(q * 32) << 16), w);
        ptx::tmem_wait_ld();
        const int n = t * kTileKeys + row;
        const bool valid = n < N;
#pragma unroll
        for (int i = 0; i < kRealCols; ++i) {
          if (i < G) {
            const float l = __uint_as_float(w[i]) * scale;
            if (valid) Lreq[((int64_t)(kh * G + i) * S1) * Ncap + n] = l;
          }
        }
      }

      // accumulators drained: hand them back to the MMA warp
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&tail->tmem_empty[a]);
      {
        // write the staged fp32 rows out, one row per warp and step, 128 consecutive keys per row
        ptx::named_barrier_sync(2, kEpiWarps * 32);
        for (int rr = e; rr < kRowChunk; rr += kEpiWarps) {
          const int grow = row0 + rr;
          if (grow >= G * S) break;
          float* dst = Lreq + (int64_t)((kh * G + grow / S) * S1 + grow % S + 1) * Ncap + (int64_t)t * kTileKeys;
          const uint8_t* srow = obuf + (size_t)rr * (kTileKeys * 4);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int key = j * 32 + lane;
            const uint32_t pos = ((uint32_t)(key >> 2)) ^ ((uint32_t)rr & 31u);
            const float f = *reinterpret_cast<const float*>(srow + (pos << 4) + ((key & 3) << 2));
            if (t * kTileKeys + key < N) dst[key] = f;
          }
        }
      }
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
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace

// ------------------------------------------------------------------------------------ host side
bool score_umma_supported(const gvote_params* p) {
  return p->d_k % 64 == 0 && p->d_k <= 256 && p->n_q_heads / p->n_kv_heads <= kRealCols;
}

ScoreGeometry score_geometry(const gvote_params* p) {
  ScoreGeometry g;
  const int rows = (p->n_q_heads / p->n_kv_heads) * p->S;     // synthetic rows of a head group
  g.RC = kRowChunk;
  g.row_chunks = (rows + kRowChunk - 1) / kRowChunk;
  return g;
}

// Returns GVOTE_OK, or GVOTE_ERR_UNSUPPORTED_SHAPE when the tensor maps cannot describe the
// operands (the caller then takes the SIMT path).
int32_t launch_score_umma(const gvote_params* p, const __nv_bfloat16* Q, const __nv_bfloat16* K, int64_t k_tok,
                          int64_t k_head, const int32_t* cu, int32_t batch, int64_t total_tokens, int64_t max_N,
                          float* logits, int32_t* status, const int32_t* kv_len, cudaStream_t st) {
  const int Hq = p->n_q_heads, Hkv = p->n_kv_heads, G = Hq / Hkv, S1 = p->S + 1, d_k = p->d_k;
  const ScoreGeometry geo = score_geometry(p);
  const int row_chunks = geo.row_chunks;

  CUtensorMap tmK, tmQ, tmQr;
  {
    const uint64_t dims[3] = {(uint64_t)d_k, (uint64_t)total_tokens, (uint64_t)Hkv};
    const uint64_t strides[2] = {(uint64_t)k_tok * 2, (uint64_t)k_head * 2};
    const uint32_t box[3] = {64, (uint32_t)kTileKeys, 1};
    if (k_head <= 0 || !encode_tensor_map_bf16(&tmK, K, 3, dims, strides, box)) return GVOTE_ERR_UNSUPPORTED_SHAPE;
  }
  {
    const uint64_t dims[2] = {(uint64_t)d_k, (uint64_t)batch * Hq * S1};
    const uint64_t strides[1] = {(uint64_t)d_k * 2};
    const uint32_t box[2] = {64, (uint32_t)kRowChunk};
    const uint32_t boxr[2] = {64, (uint32_t)kRealCols};
    if (!encode_tensor_map_bf16(&tmQ, Q, 2, dims, strides, box)) return GVOTE_ERR_UNSUPPORTED_SHAPE;
    if (!encode_tensor_map_bf16(&tmQr, Q, 2, dims, strides, boxr)) return GVOTE_ERR_UNSUPPORTED_SHAPE;
  }
  const int kchunks = d_k / 64;
  const size_t out_bytes = (size_t)kRowChunk * kTileKeys * 4;
  const size_t fixed = 1024 + (size_t)kchunks * kRowChunk * 128 + align_up((size_t)kchunks * kRealCols * 128, 1024) +
                       sizeof(ScoreSmemTail) + 64;
  const size_t stage_bytes = (size_t)kchunks * kTileKeys * 128;
  int stages = kMaxStages;
  auto need = [&]() { return fixed + stages * stage_bytes + out_bytes; };
  if (need() > 227 * 1024) stages = 2;
  if (need() > 227 * 1024) return GVOTE_ERR_UNSUPPORTED_SHAPE;
  const size_t smem = need();
  const int64_t max_tiles = ceil_div(max_N, kTileKeys);
  // one CTA per SM when the batch is uniform; a ragged batch gets four times as many, shorter
  // CTAs so that the hardware scheduler can even out long and short requests
  const int64_t groups = (int64_t)Hkv * row_chunks * batch;
  int64_t X = (batch == 1 ? 148 : 592) / groups;
  if (X > max_tiles) X = max_tiles;
  if (X < 1) X = 1;
  dim3 grid((unsigned)X, (unsigned)(Hkv * row_chunks), (unsigned)batch);
  const float scale = (float)(1.0 / sqrt((double)d_k));
  GVOTE_CUDA_CHECK(cudaFuncSetAttribute(score_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  {
    LaunchScope scope_("score_umma_kernel", st);
    score_umma_kernel<<<grid, kUmmaThreads, smem, st>>>(tmK, tmQ, tmQr, cu, Hq, G, S1, d_k, row_chunks, stages, scale,
                                                        logits, status, kv_len);
  }
  GVOTE_LAUNCH_CHECK("score_umma_kernel");
  return GVOTE_OK;
}

}  // namespace gvote
