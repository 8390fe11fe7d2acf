// Algorithm 1, the logits of the synthetic queries and their TopK, fused on the fifth-generation
// tensor cores so that the S x N logits matrix (the memory hazard Section 4.4 names) never exists:
// two passes over a KV head's keys, both D[128 rows x 128 keys] = Q_chunk (128 x d_k) * K_tile^T per
// 128-key tile with the accumulators in tensor memory, a lane per query row, a column per key.
//
//   score_sample_kernel  first pass.  Streams every key tile once for the G current-query rows of the
//       head (a thin second product D2[128 keys x 16] = K_tile * Qr^T on the same tile in shared
//       memory): their exact fp32 logits and running maxima, the input of the current query's top-p
//       (A0, C0, B_step).  On the tiles of the row sample (vote_geom.cuh) it also runs the full product
//       and stores the synthetic rows' logits there as half-precision keys - a few thousand keys per
//       row, from which bracket_kernel takes two order statistics [lo, hi] that enclose the row's k-th
//       largest logit.
//   score_sweep_kernel   second pass.  Every tile, every row chunk.  The read-out thread of a row holds
//       32 consecutive logits of its row in registers and compares them with the row's own bracket:
//       keys above hi are certainly among the k largest - their bits are OR-ed over the 32 rows of the
//       warp and then into the head's tentative mask (the union step), and counted per row; keys
//       inside [lo, hi] are appended, as (fp32 logit, index), to the thread's own segment of the row's
//       short candidate list.  Nothing else leaves the SM.  resolve_kernel later picks the k - #above
//       largest candidates.
//
// A CTA walks the key tiles x, x+X, ... of one (request, KV head): a tile is fetched once (TMA, 128-byte
// swizzle) and multiplied with up to four 128-row chunks of query rows.  warp 0: TMA producer; warp 1:
// tensor-memory allocation and tcgen05.mma issue; the other warps: read-out (first pass: two per lane
// quadrant, 64 keys each; second pass: four per quadrant, 32 keys each).  The first pass keeps the query
// rows in shared memory; the second keeps them in tensor memory, as the MMA's A operand.  Accumulators
// are double or triple buffered so that the MMAs of one product overlap the read-out of the one before.
//
// Every wait on an mbarrier is bounded.  When one runs out the CTA raises a shared abort flag and
// records GVOTE_ERR_TIMEOUT in the workspace status word; the remaining waits then give up at once,
// the warps run their loops to the end (all addresses stay in bounds whatever the data), bulk copies
// are drained, tensor memory is freed and the CTA returns.
#include <cuda_fp16.h>

#include "common.cuh"
#include "ptx.cuh"
#include "vote_geom.cuh"

namespace gvote {
namespace {

constexpr int kTileKeys = kVoteTileKeys;
constexpr int kRowChunk = kVoteRowChunk;
constexpr int kRealCols = 16;     // current-query rows per KV head the thin product holds (MMA N)
constexpr int kEpiWarps = 8;
constexpr int kSweepThreads = 64 + 32 * kEpiWarps;
constexpr int kMaxStages = 6;
constexpr int kTmemCols = 512;    // first pass: 2 x 128 (D1) + 8 x 32 (D2, 16 used)
constexpr int kD2Col = 256;
constexpr int kD2Bufs = 8;        // thin accumulators in flight: the MMA of a tile never waits for a read-out

struct SweepTail {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t q_full;
  uint64_t acc_full[3];
  uint64_t acc_empty[3];
  uint64_t real_full[kD2Bufs];
  uint64_t real_empty[kD2Bufs];
  uint32_t tmem_slot;
  volatile int abort_flag;
  uint32_t rowmax[kRealCols];         // running maximum (order-preserving image) of each current-query row
};

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t i = 0; i < (1u << 22); ++i) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((i & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

__device__ __forceinline__ uint32_t key16x2_of(float lo, float hi) {
  uint32_t p;
  asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(p) : "f"(hi), "f"(lo));
  return p;
}

// The key tiles a CTA walks.  Second pass: every tile x, x+X, ...  First pass: first the CTA's share of the
// row sample (slots x, x+X, ... of the sample, whatever CTA streams those tiles: every CTA gets the same
// number of full products), then, in the CTAs that stream the keys for the current-query rows, the tiles
// x, x+X, ...
struct TileWalk {
  SampleGeom g;
  int x, X, n_samp, count;
  __device__ __forceinline__ void init(int N, int x_, int X_, bool sample, bool stream) {
    g = sample_geom(N);
    x = x_; X = X_;
    n_samp = (sample && N > 0 && x < g.ns) ? (g.ns - x + X - 1) / X : 0;
    const int n_stream = (stream && N > 0 && x < g.n_tiles) ? (g.n_tiles - x + X - 1) / X : 0;
    count = n_samp + n_stream;
  }
  __device__ __forceinline__ int tile(int i) const {
    return i < n_samp ? sample_tile(g, x + i * X) : x + (i - n_samp) * X;
  }
  // position of item i in the sample, or -1 for a streamed tile
  __device__ __forceinline__ int slot(int i) const { return i < n_samp ? x + i * X : -1; }
};

struct SweepSmem {
  uint8_t* Qs;      // [chunks][kchunks][128 rows][128 bytes]
  uint8_t* Qr;      // [kchunks][16 rows][128 bytes]
  uint8_t* Ks;      // [stages][kchunks][128 keys][128 bytes]
  uint8_t* Os;      // staging of half-precision key tiles (first pass)
  SweepTail* tail;
};

__device__ __forceinline__ SweepSmem carve(uint8_t* smem_raw, int kchunks, int cg, int stages, bool with_real,
                                           uint32_t staging_bytes) {
  SweepSmem s;
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t q_bytes = (uint32_t)cg * kchunks * kRowChunk * 128;
  const uint32_t qr_bytes = with_real ? (((uint32_t)kchunks * kRealCols * 128 + 1023u) & ~1023u) : 0u;
  const uint32_t stage_bytes = (uint32_t)kchunks * kTileKeys * 128;
  s.Qs = base;
  s.Qr = s.Qs + q_bytes;
  s.Ks = s.Qr + qr_bytes;
  s.Os = s.Ks + (size_t)stages * stage_bytes;
  s.tail = reinterpret_cast<SweepTail*>(s.Os + staging_bytes);
  return s;
}

__device__ __forceinline__ void setup(SweepTail* tail, int stages, const CUtensorMap* a, const CUtensorMap* b,
                                      const CUtensorMap* c) {
  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { ptx::mbar_init(&tail->full[s], 1); ptx::mbar_init(&tail->empty[s], 1); }
    ptx::mbar_init(&tail->q_full, 1);
    for (int a2 = 0; a2 < 2; ++a2) {
      ptx::mbar_init(&tail->acc_full[a2], 1);
      ptx::mbar_init(&tail->acc_empty[a2], kEpiWarps);
    }
    for (int a2 = 0; a2 < kD2Bufs; ++a2) {
      ptx::mbar_init(&tail->real_full[a2], 1);
      ptx::mbar_init(&tail->real_empty[a2], kEpiWarps / 2);
    }
    tail->abort_flag = 0;
    for (int i = 0; i < kRealCols; ++i) tail->rowmax[i] = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(a);
    ptx::prefetch_tensormap(b);
    if (c) ptx::prefetch_tensormap(c);
  }
  if ((threadIdx.x >> 5) == 1) {
    ptx::tmem_alloc(&tail->tmem_slot, kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
}

// One 128 x 128 x d_k product into accumulator `d`: rows = the query chunk at q_addr, columns = the keys at k_addr.
__device__ __forceinline__ void issue_d1(uint32_t d, uint32_t q_addr, uint32_t k_addr, int d_k) {
  const uint32_t idesc = ptx::instr_desc_bf16_f32(kRowChunk, kTileKeys);
  const int ksteps = d_k / 16;
  for (int k = 0; k < ksteps; ++k) {
    const uint32_t koff = (uint32_t)(k >> 2), kin = (uint32_t)(k & 3) * 32u;
    const uint64_t dq = ptx::smem_desc_k_sw128(q_addr + koff * (uint32_t)(kRowChunk * 128) + kin);
    const uint64_t dk = ptx::smem_desc_k_sw128(k_addr + koff * (uint32_t)(kTileKeys * 128) + kin);
    ptx::umma_bf16(d, dq, dk, idesc, k > 0 ? 1u : 0u);
  }
}

// ------------------------------------------------------------------------------------ first pass
__global__ void __launch_bounds__(kSweepThreads, 1)
score_sample_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ,
                    const __grid_constant__ CUtensorMap tmQr, const int32_t* __restrict__ cu, int Hq, int G, int S,
                    int d_k, int row_chunks, int cg, int X0, int X1, int stages, int n_out, float scale,
                    float* __restrict__ real_logits, uint32_t* __restrict__ rowmax_part, uint16_t* __restrict__ sample,
                    int64_t sample_slots, int32_t* __restrict__ status, const int32_t* __restrict__ kv_len,
                    uint32_t* __restrict__ zero_a, uint32_t* __restrict__ zero_b, int64_t zero_words,
                    uint32_t* __restrict__ head_bad, int n_head_bad) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const int groups = (row_chunks + cg - 1) / cg;
  const int r = blockIdx.z;
  const int kh = blockIdx.y / groups, grp = blockIdx.y % groups;
  const bool do_real = grp == 0;
  const bool active = (int)blockIdx.x < (do_real ? X0 : X1);
  const int kchunks = d_k / 64;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const SweepSmem sm = carve(smem_raw, kchunks, cg, stages, true, (uint32_t)n_out * kRowChunk * kTileKeys * 2);
  SweepTail* tail = sm.tail;
  if (active) setup(tail, stages, &tmK, &tmQ, &tmQr);     // barriers, tensor memory
  // The vote starts from an empty keep mask, an empty tentative mask and no head marked: every CTA of this
  // first kernel of the vote clears its share (nothing reads them before the kernels that follow).
  {
    const int64_t n_thr = (int64_t)gridDim.x * gridDim.y * gridDim.z * blockDim.x;
    const int64_t me = (((int64_t)blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x) * blockDim.x + threadIdx.x;
    for (int64_t i = me; i < zero_words; i += n_thr) { zero_a[i] = 0u; zero_b[i] = 0u; }
    if (me < n_head_bad) head_bad[me] = 0u;
  }
  if (!active) return;
  const int start = cu[r], Ncap = cu[r + 1] - start;       // Ncap: rows of the slab (layout); N: rows that count
  const int N = valid_keys(kv_len, r, Hq / G, kh, Ncap);
  const int c_first = grp * cg, c_cnt = min(cg, row_chunks - c_first);
  TileWalk walk;
  walk.init(N, (int)blockIdx.x, do_real ? X0 : X1, true, do_real);
  const uint32_t tmem_base = tail->tmem_slot;
  volatile int* abort_flag = &tail->abort_flag;
  const uint32_t q_chunk_bytes = (uint32_t)kchunks * kRowChunk * 128;
  const uint32_t qr_bytes = (uint32_t)kchunks * kRealCols * 128;
  const uint32_t stage_bytes = (uint32_t)kchunks * kTileKeys * 128;
  const int R = G * (S + 1);                          // rows of the head group: G*S synthetic, then G current

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && walk.count > 0) {
      const int group_row = (r * (Hq / G) + kh) * R;
      ptx::mbar_arrive_expect_tx(&tail->q_full, (uint32_t)c_cnt * q_chunk_bytes + (do_real ? qr_bytes : 0u));
      for (int cc = 0; cc < c_cnt; ++cc)
        for (int c = 0; c < kchunks; ++c)
          ptx::tma_load_2d(sm.Qs + ((size_t)cc * kchunks + c) * kRowChunk * 128, &tmQ, &tail->q_full, c * 64,
                           group_row + (c_first + cc) * kRowChunk);
      if (do_real)
        for (int c = 0; c < kchunks; ++c)
          ptx::tma_load_2d(sm.Qr + (size_t)c * kRealCols * 128, &tmQr, &tail->q_full, c * 64, group_row + G * S);
      for (int it = 0; it < walk.count; ++it) {
        const int s = it % stages;
        const uint32_t ph = (uint32_t)(it / stages) & 1u;
        if (!wait_or_abort(&tail->empty[s], ph ^ 1u, abort_flag)) break;
        ptx::mbar_arrive_expect_tx(&tail->full[s], stage_bytes);
        uint8_t* dst = sm.Ks + (size_t)s * stage_bytes;
        const int t = walk.tile(it);
        for (int c = 0; c < kchunks; ++c)
          ptx::tma_load_3d(dst + (size_t)c * kTileKeys * 128, &tmK, &tail->full[s], c * 64, start + t * kTileKeys, kh);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && walk.count > 0) {
      const uint32_t idesc2 = ptx::instr_desc_bf16_f32(kTileKeys, kRealCols);   // keys x current rows
      const uint32_t q_addr = ptx::smem_u32(sm.Qs), qr_addr = ptx::smem_u32(sm.Qr);
      bool ok = wait_or_abort(&tail->q_full, 0, abort_flag);
      int n1 = 0;                                      // full products issued so far
      for (int it = 0; ok && it < walk.count; ++it) {
        const int s = it % stages;
        const uint32_t ph = (uint32_t)(it / stages) & 1u;
        if (!wait_or_abort(&tail->full[s], ph, abort_flag)) break;
        ptx::tc_fence_after_sync();
        const uint32_t k_addr = ptx::smem_u32(sm.Ks + (size_t)s * stage_bytes);
        if (it >= walk.n_samp) {
          const int is = it - walk.n_samp;                 // streamed tiles so far
          const int ar = is % kD2Bufs;
          if (!wait_or_abort(&tail->real_empty[ar], (((uint32_t)(is / kD2Bufs)) & 1u) ^ 1u, abort_flag)) break;
          ptx::tc_fence_after_sync();
          const uint32_t d2 = tmem_base + (uint32_t)(kD2Col + ar * 32);
          const int ksteps = d_k / 16;
          for (int k = 0; k < ksteps; ++k) {
            const uint32_t koff = (uint32_t)(k >> 2), kin = (uint32_t)(k & 3) * 32u;
            const uint64_t dk = ptx::smem_desc_k_sw128(k_addr + koff * (uint32_t)(kTileKeys * 128) + kin);
            const uint64_t dq = ptx::smem_desc_k_sw128(qr_addr + koff * (uint32_t)(kRealCols * 128) + kin);
            ptx::umma_bf16(d2, dk, dq, idesc2, k > 0 ? 1u : 0u);
          }
          ptx::umma_commit(&tail->real_full[ar]);
        } else {
          for (int cc = 0; ok && cc < c_cnt; ++cc, ++n1) {
            const int a = n1 & 1;
            if (!wait_or_abort(&tail->acc_empty[a], (((uint32_t)n1 >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
            ptx::tc_fence_after_sync();
            issue_d1(tmem_base + (uint32_t)(a * kRowChunk), q_addr + (uint32_t)cc * q_chunk_bytes, k_addr, d_k);
            ptx::umma_commit(&tail->acc_full[a]);
          }
        }
        ptx::umma_commit(&tail->empty[s]);       // the ring slot is free once these MMAs have read it
      }
    }
  } else {
    // ------------------------------------------------------------------ read-out (8 warps)
    const int e = warp - 2;                      // 0..7
    const int q = warp & 3;                      // tensor-memory lane quadrant this warp may read
    const int half = e >> 2;                     // which 64 keys of the tile this warp takes
    const int row = q * 32 + lane;               // D1 lane = synthetic row of the chunk; D2 lane = key of the tile
    const bool leader = (e == 0 && lane == 0);
    float* Lreq = real_logits + (int64_t)Hq * start;
    int n1 = 0;
    for (int it = 0; it < walk.count; ++it) {
      const int t = walk.tile(it);
      // ---- current-query rows: thread = key, exact fp32 logits and their running maximum
      if (it >= walk.n_samp && half == 0) {
        const int is = it - walk.n_samp;
        const int ar = is % kD2Bufs;
        const bool got = wait_or_abort(&tail->real_full[ar], ((uint32_t)(is / kD2Bufs)) & 1u, abort_flag);
        ptx::tc_fence_after_sync();
        uint32_t w[16];
        ptx::tmem_ld_32x16(tmem_base + (uint32_t)(kD2Col + ar * 32) + ((uint32_t)(q * 32) << 16), w);
        ptx::tmem_wait_ld();
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&tail->real_empty[ar]);
        const int n = t * kTileKeys + row;
        const bool valid = got && n < N;
#pragma unroll
        for (int i = 0; i < kRealCols; ++i) {
          if (i < G) {
            const float l = __uint_as_float(w[i]) * scale;
            if (valid) Lreq[(int64_t)(kh * G + i) * Ncap + n] = l;
            const uint32_t wmax = __reduce_max_sync(0xffffffffu, valid ? ordered_key(l) : 0u);
            if (lane == 0 && wmax) atomicMax(&tail->rowmax[i], wmax);
          }
        }
      }
      // ---- sampled tile: the synthetic rows' logits as half-precision keys, one staged tile per chunk
      const int js = walk.slot(it);
      if (js < 0) continue;
      const int valid_keys_in_tile = N - t * kTileKeys;          // >= 128 except on a ragged last tile
      for (int cc = 0; cc < c_cnt; ++cc, ++n1) {
        const int a = n1 & 1;
        uint8_t* obuf = sm.Os + (size_t)(n1 % n_out) * (kRowChunk * kTileKeys * 2);
        // the staging buffer about to be overwritten must have been read by its bulk copy
        if (leader) { if (n_out == 2) ptx::bulk_wait_read<1>(); else ptx::bulk_wait_read<0>(); }
        ptx::named_barrier_sync(1, kEpiWarps * 32);
        wait_or_abort(&tail->acc_full[a], ((uint32_t)n1 >> 1) & 1u, abort_flag);
        ptx::tc_fence_after_sync();
        const uint32_t taddr = tmem_base + (uint32_t)(a * kRowChunk) + ((uint32_t)(q * 32) << 16) + (uint32_t)(half * 64);
        uint32_t v0[32], v1[32];
        ptx::tmem_ld_32x32(taddr, v0);
        ptx::tmem_ld_32x32(taddr + 32u, v1);
        ptx::tmem_wait_ld();
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&tail->acc_empty[a]);
        // 16-byte piece c of the row (keys 8c .. 8c+7) sits at piece position c ^ (row & 15): the stores of
        // a warp then spread over the banks; the order inside a row's sample does not matter to its ranks
        uint8_t* orow = obuf + (size_t)row * (kTileKeys * 2);
        const uint32_t swz = (uint32_t)row & 15u;
        const int col0 = half * 64;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const uint32_t* v = c < 4 ? &v0[8 * c] : &v1[8 * (c - 4)];
          uint32_t pk[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            float l0 = __uint_as_float(v[2 * j]) * scale, l1 = __uint_as_float(v[2 * j + 1]) * scale;
            if (col0 + 8 * c + 2 * j >= valid_keys_in_tile) l0 = -INFINITY;       // pad of a ragged last tile
            if (col0 + 8 * c + 2 * j + 1 >= valid_keys_in_tile) l1 = -INFINITY;
            pk[j] = key16x2_of(l0, l1);
            if (l0 == -INFINITY) pk[j] = (pk[j] & 0xffff0000u) | 0xfc00u;         // satfinite clamps: put -inf back
            if (l1 == -INFINITY) pk[j] = (pk[j] & 0x0000ffffu) | 0xfc000000u;
          }
          *reinterpret_cast<uint4*>(orow + ((((uint32_t)(half * 8 + c)) ^ swz) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
        ptx::fence_proxy_async();                // staged tile visible to the bulk-copy engine
        ptx::named_barrier_sync(2, kEpiWarps * 32);
        if (leader) {
          const int64_t slot = sample_slot_offset(start, r) + js;
          uint16_t* gdst = sample + ((((int64_t)kh * sample_slots + slot) * row_chunks + (c_first + cc)) * kRowChunk) * kTileKeys;
          ptx::bulk_store(gdst, obuf, (uint32_t)(kRowChunk * kTileKeys * 2));
          ptx::bulk_commit();
        }
      }
    }
    if (leader) ptx::bulk_wait_all<0>();
  }

  // ------------------------------------------------------------------ teardown
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (threadIdx.x == 0 && tail->abort_flag) {
    atomicExch(&status[0], GVOTE_ERR_TIMEOUT);
    atomicExch(&status[1], 5);
  }
  // this CTA's maxima of the current-query rows (0 = it met no key): real_topp_kernel takes the largest of the X0
  if (do_real && (int)threadIdx.x < G)
    rowmax_part[(int64_t)(r * Hq + kh * G + (int)threadIdx.x) * X0 + blockIdx.x] = tail->rowmax[threadIdx.x];
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ------------------------------------------------------------------------------------ second pass
// Sixteen read-out warps: four per lane quadrant, each 32 of the tile's 128 keys, so that a thread holds 32
// consecutive logits of its row.  Four warps per scheduler hide the latencies of the chain (accumulator
// ready, tensor-memory load, compares, list writes) that two could not.
//
// The query rows are the MMA's A operand and live in TENSOR memory here, not in shared memory: each row's
// d_k bf16 values, two to a 32-bit column, written once by the read-out warps (tcgen05.st) straight from
// global memory.  With both operands in shared memory a 128 x 128 x 16 instruction has to fetch 8 KB per
// 64 clocks, all the shared-memory bandwidth there is; with A in tensor memory it fetches only the key
// tile's 4 KB, and the shared memory the rows would take goes to a deeper ring of key stages.
constexpr int kSweepEpiWarps = 16;
constexpr int kSweepBThreads = 64 + 32 * kSweepEpiWarps;

template <int CG, int STG>      // STG: logits a thread stages at a time (16, or 8 when shared memory is short)
__global__ void __launch_bounds__(kSweepBThreads, 1)
score_sweep_kernel(const __grid_constant__ CUtensorMap tmK, const __nv_bfloat16* __restrict__ Q,
                   const int32_t* __restrict__ cu, int Hq, int G, int S, int d_k, int row_chunks, int stages,
                   int nbuf, float scale, const VoteState vs, int64_t row_words, int32_t* __restrict__ status,
                   const int32_t* __restrict__ kv_len) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const int groups = (row_chunks + CG - 1) / CG;
  const int r = blockIdx.z;
  const int kh = blockIdx.y / groups, grp = blockIdx.y % groups;
  const int kchunks = d_k / 64;
  const int c_first = grp * CG, c_cnt = min(CG, row_chunks - c_first);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // [key stages | staging of the read-out: STG floats per thread | barriers]
  const SweepSmem sm = carve(smem_raw, kchunks, 0, stages, false, (uint32_t)kSweepEpiWarps * 32 * STG * 4);
  SweepTail* tail = sm.tail;
  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { ptx::mbar_init(&tail->full[s], 1); ptx::mbar_init(&tail->empty[s], 1); }
    ptx::mbar_init(&tail->q_full, kSweepEpiWarps);
    for (int a2 = 0; a2 < 3; ++a2) { ptx::mbar_init(&tail->acc_full[a2], 1); ptx::mbar_init(&tail->acc_empty[a2], kSweepEpiWarps); }
    tail->abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&tmK);
  }
  if (warp == 1) {
    ptx::tmem_alloc(&tail->tmem_slot, kTmemCols);            // nbuf x 128 accumulator columns, then the query rows
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const int start = cu[r], Ncap = cu[r + 1] - start;
  const int N = valid_keys(kv_len, r, Hq / G, kh, Ncap);
  TileWalk walk;
  walk.init(N, (int)blockIdx.x, (int)gridDim.x, false, true);
  const uint32_t tmem_base = tail->tmem_slot;
  volatile int* abort_flag = &tail->abort_flag;
  const uint32_t stage_bytes = (uint32_t)kchunks * kTileKeys * 128;
  const int R = G * (S + 1);
  const uint32_t a_cols = (uint32_t)d_k / 2;               // tensor-memory columns of one chunk's query rows
  const uint32_t a_base = (uint32_t)nbuf * kRowChunk;      // they follow the accumulators

  if (warp == 0) {
    if (lane == 0 && walk.count > 0) {
      for (int it = 0; it < walk.count; ++it) {
        const int s = it % stages;
        const uint32_t ph = (uint32_t)(it / stages) & 1u;
        if (!wait_or_abort(&tail->empty[s], ph ^ 1u, abort_flag)) break;
        ptx::mbar_arrive_expect_tx(&tail->full[s], stage_bytes);
        uint8_t* dst = sm.Ks + (size_t)s * stage_bytes;
        const int t = walk.tile(it);
        for (int c = 0; c < kchunks; ++c)
          ptx::tma_load_3d(dst + (size_t)c * kTileKeys * 128, &tmK, &tail->full[s], c * 64, start + t * kTileKeys, kh);
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && walk.count > 0) {
      const uint32_t idesc = ptx::instr_desc_bf16_f32(kRowChunk, kTileKeys);
      bool ok = wait_or_abort(&tail->q_full, 0, abort_flag);   // the query rows are in tensor memory
      ptx::tc_fence_after_sync();
      int n1 = 0;
      for (int it = 0; ok && it < walk.count; ++it) {
        const int s = it % stages;
        const uint32_t ph = (uint32_t)(it / stages) & 1u;
        if (!wait_or_abort(&tail->full[s], ph, abort_flag)) break;
        ptx::tc_fence_after_sync();
        const uint32_t k_addr = ptx::smem_u32(sm.Ks + (size_t)s * stage_bytes);
        for (int cc = 0; cc < c_cnt; ++cc, ++n1) {
          const int a = n1 % nbuf;
          if (!wait_or_abort(&tail->acc_empty[a], (((uint32_t)(n1 / nbuf)) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after_sync();
          const uint32_t d = tmem_base + (uint32_t)(a * kRowChunk), qa = tmem_base + a_base + (uint32_t)cc * a_cols;
          const int ksteps = d_k / 16;
          for (int k = 0; k < ksteps; ++k) {
            const uint32_t koff = (uint32_t)(k >> 2), kin = (uint32_t)(k & 3) * 32u;
            const uint64_t dk = ptx::smem_desc_k_sw128(k_addr + koff * (uint32_t)(kTileKeys * 128) + kin);
            ptx::umma_bf16_ts(d, qa + (uint32_t)k * 8u, dk, idesc, k > 0 ? 1u : 0u);
          }
          ptx::umma_commit(&tail->acc_full[a]);
        }
        ptx::umma_commit(&tail->empty[s]);
      }
    }
  } else {
    const int e = warp - 2;                      // 0..15
    const int q = warp & 3;                      // tensor-memory lane quadrant this warp may read
    const int cq = e >> 2;                       // which 32 keys of the tile this warp takes
    const int seg = (int)blockIdx.x * 4 + cq;    // this thread's segment of its rows' lists
    const int seg_cap = vs.lay.seg_cap(Ncap);
    // the thread's staging area: STG floats in 16-byte pieces; piece c sits at position c ^ swz, which keeps
    // the 16-byte stores of a quarter warp on different banks
    constexpr int kPieces = STG / 4;
    const float inv_scale = 1.0f / scale;
    uint8_t* stg = sm.Os + (size_t)(e * 32 + lane) * (STG * 4);
    const uint32_t stg_swz = ((uint32_t)lane >> (kPieces == 4 ? 1 : 2)) & (uint32_t)(kPieces - 1);
    // this thread's row in each chunk of the group: its bracket, its segment, its counts
    __half2 lo[CG], hi[CG];
    uint32_t abv[CG], fill[CG];
    int rowid[CG];
    uint2* segp[CG];
#pragma unroll
    for (int cc = 0; cc < CG; ++cc) {
      const int grow = (c_first + cc) * kRowChunk + q * 32 + lane;       // row within the head group
      abv[cc] = 0;
      fill[cc] = 0;
      rowid[cc] = -1;
      segp[cc] = nullptr;
      float lo_f = INFINITY, hi_f = INFINITY;              // a row that does not exist takes nothing
      if (cc < c_cnt && grow < G * S) {
        rowid[cc] = (r * Hq + kh * G + grow / S) * S + grow % S;
        segp[cc] = vs.list(kh * G + grow / S, grow % S, S, start, r) + (int64_t)seg * seg_cap;
        const RowBracket b = vs.bracket[rowid[cc]];
        lo_f = b.lo * inv_scale;
        hi_f = b.hi * inv_scale;
      }
      lo[cc] = __half2half2(__float2half_rd(lo_f));        // bounds rounded outwards
      hi[cc] = __half2half2(__float2half_ru(hi_f));
    }
    // the query rows of chunk cc go to tensor memory through the four warps with cq == cc mod 4 (one per lane
    // quadrant): a thread fetches its row from global memory, 32 columns (64 values) at a time
    if (walk.count > 0) {
#pragma unroll
      for (int cc = 0; cc < CG; ++cc) {
        if (cc >= c_cnt || (cc & 3) != cq) continue;
        const int grow = (c_first + cc) * kRowChunk + q * 32 + lane;
        const uint4* src = reinterpret_cast<const uint4*>(Q + ((int64_t)(r * (Hq / G) + kh) * R + grow) * d_k);
        for (uint32_t c0 = 0; c0 < a_cols; c0 += 32) {
          uint32_t w[32];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint4 x = grow < G * S ? __ldg(src + (c0 >> 2) + j) : make_uint4(0u, 0u, 0u, 0u);
            w[4 * j] = x.x; w[4 * j + 1] = x.y; w[4 * j + 2] = x.z; w[4 * j + 3] = x.w;
          }
          ptx::tmem_st_32x32(tmem_base + a_base + (uint32_t)cc * a_cols + c0 + ((uint32_t)(q * 32) << 16), w);
        }
      }
      ptx::tmem_wait_st();
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&tail->q_full);
    }
    uint32_t* mrow = vs.tmask + (int64_t)kh * row_words + mask_word_offset(start, r);
    int n1 = 0;
    for (int it = 0; it < walk.count; ++it) {
      const int t = walk.tile(it);
      // keys of this quarter of the tile that exist (a ragged last tile reads whatever follows the row)
      const int left = N - t * kTileKeys - cq * 32;
      const uint32_t vm = left >= 32 ? 0xffffffffu : (left > 0 ? (1u << left) - 1u : 0u);
      const int n0 = t * kTileKeys + cq * 32;
#pragma unroll
      for (int cc = 0; cc < CG; ++cc) {
        if (cc >= c_cnt) break;
        const int a = n1 % nbuf;
        wait_or_abort(&tail->acc_full[a], ((uint32_t)(n1 / nbuf)) & 1u, abort_flag);
        ++n1;
        ptx::tc_fence_after_sync();
        uint32_t v[32];
        ptx::tmem_ld_32x32(tmem_base + (uint32_t)(a * kRowChunk) + ((uint32_t)(q * 32) << 16) + (uint32_t)(cq * 32), v);
        ptx::tmem_wait_ld();
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&tail->acc_empty[a]);     // the values are in registers: free the accumulator

        // Compare as half-precision pairs, two keys per instruction, on the unscaled accumulators (the row's
        // bounds were divided by the scale and rounded outwards).  Rounding a key to half precision is monotone,
        // so every key found above the upper bound still exceeds every key that is not; keys that round onto a
        // bound are listed and settled exactly later.
        const __half2 hi2 = hi[cc], lo2 = lo[cc];
        uint32_t ab = 0, cb = 0;
#pragma unroll
        for (int g8 = 0; g8 < 4; ++g8) {                         // eight keys: bits 2j (low half) and 17 + 2j (high half)
          uint32_t gacc = 0, cacc = 0;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t pk = key16x2_of(__uint_as_float(v[8 * g8 + 2 * j]), __uint_as_float(v[8 * g8 + 2 * j + 1]));
            const __half2 h2 = *reinterpret_cast<const __half2*>(&pk);
            const uint32_t pick = (1u << (2 * j)) | (1u << (17 + 2 * j));
            gacc |= __hgt2_mask(h2, hi2) & pick;
            cacc |= __hge2_mask(h2, lo2) & pick;
          }
          ab |= ((gacc | (gacc >> 16)) & 0xffu) << (8 * g8);
          cb |= ((cacc | (cacc >> 16)) & 0xffu) << (8 * g8);
        }
        ab &= vm;
        cb &= vm & ~ab;
        // union step: the warp's 32 rows OR their bits, one atomic per mask word
        const uint32_t w = __reduce_or_sync(0xffffffffu, ab);
        if (lane == 0 && w) atomicOr(&mrow[n0 >> 5], w);
        abv[cc] += __popc(ab);
        if (cb) {
          // the listed keys: their logits go through the thread's staging area, STG at a time, so that they
          // can be fetched by position
          uint2* const sp = segp[cc];
          uint32_t f = fill[cc];
#pragma unroll
          for (int part = 0; part < 32 / STG; ++part) {
            uint32_t sub = (cb >> (STG * part)) & ((1u << STG) - 1u);
            if (sub == 0) continue;
#pragma unroll
            for (int c = 0; c < kPieces; ++c)
              *reinterpret_cast<uint4*>(stg + (((uint32_t)c ^ stg_swz) << 4)) =
                  make_uint4(v[STG * part + 4 * c], v[STG * part + 4 * c + 1], v[STG * part + 4 * c + 2], v[STG * part + 4 * c + 3]);
            while (sub) {
              const int j = __ffs(sub) - 1;
              sub &= sub - 1;
              const float acc = *reinterpret_cast<const float*>(stg + ((((uint32_t)j >> 2) ^ stg_swz) << 4) + ((j & 3) << 2));
              if (f < (uint32_t)seg_cap) sp[f] = make_uint2(__float_as_uint(acc * scale), (uint32_t)(n0 + STG * part + j));
              ++f;
            }
          }
          fill[cc] = f;
        }
      }
    }
    // what this writer met, for every row it owns (zeros too: resolve_kernel reads every segment)
#pragma unroll
    for (int cc = 0; cc < CG; ++cc)
      if (rowid[cc] >= 0) vs.segstat[(int64_t)rowid[cc] * vs.lay.segs + seg] = make_uint2(abv[cc], fill[cc]);
  }

  ptx::tc_fence_before_sync();
  __syncthreads();
  if (threadIdx.x == 0 && tail->abort_flag) {
    atomicExch(&status[0], GVOTE_ERR_TIMEOUT);
    atomicExch(&status[1], 6);
  }
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

constexpr size_t kSmemLimit = 227 * 1024;

// Largest chunk count (4, 2 or 1, at most row_chunks rounded up) whose query rows leave room for `min_stages`
// key stages next to `extra` bytes; returns the stage count through `stages`.
int pick_chunks(int row_chunks, int kchunks, size_t extra, int min_stages, int* stages) {
  const size_t q_chunk = (size_t)kchunks * kRowChunk * 128, stage = (size_t)kchunks * kTileKeys * 128;
  for (int cg = 4; cg >= 1; cg >>= 1) {
    if (cg > 1 && cg / 2 >= row_chunks) continue;
    const size_t fixed = 1024 + cg * q_chunk + extra + sizeof(SweepTail) + 64;
    if (fixed + (size_t)min_stages * stage > kSmemLimit) continue;
    int st = (int)((kSmemLimit - fixed) / stage);
    if (st > kMaxStages) st = kMaxStages;
    *stages = st;
    return cg;
  }
  return 0;
}

bool encode_maps(const gvote_params* p, const __nv_bfloat16* Q, const __nv_bfloat16* K, int64_t k_tok, int64_t k_head,
                 int32_t batch, int64_t total_tokens, CUtensorMap* tmK, CUtensorMap* tmQ, CUtensorMap* tmQr) {
  const int Hq = p->n_q_heads, Hkv = p->n_kv_heads, S1 = p->S + 1, d_k = p->d_k;
  {
    const uint64_t dims[3] = {(uint64_t)d_k, (uint64_t)total_tokens, (uint64_t)Hkv};
    const uint64_t strides[2] = {(uint64_t)k_tok * 2, (uint64_t)k_head * 2};
    const uint32_t box[3] = {64, (uint32_t)kTileKeys, 1};
    if (k_head <= 0 || !encode_tensor_map_bf16(tmK, K, 3, dims, strides, box)) return false;
  }
  const uint64_t dims[2] = {(uint64_t)d_k, (uint64_t)batch * Hq * S1};
  const uint64_t strides[1] = {(uint64_t)d_k * 2};
  const uint32_t box[2] = {64, (uint32_t)kRowChunk};
  const uint32_t boxr[2] = {64, (uint32_t)kRealCols};
  if (!encode_tensor_map_bf16(tmQ, Q, 2, dims, strides, box)) return false;
  if (tmQr && !encode_tensor_map_bf16(tmQr, Q, 2, dims, strides, boxr)) return false;
  return true;
}

}  // namespace

// Head dimensions of 64 and 128 (a key tile of 128 x d_k bf16 values, the query rows of a chunk and the
// staging areas share 227 KB of shared memory with at least two stages), at most 16 query heads per KV head.
bool sweep_umma_supported(const gvote_params* p) {
  return p->d_k % 64 == 0 && p->d_k <= 128 && p->n_q_heads / p->n_kv_heads <= kRealCols;
}

// First pass.  Returns GVOTE_ERR_UNSUPPORTED_SHAPE when the tensor maps cannot describe the operands (the
// caller then takes the SIMT path).
int32_t launch_score_sample(const gvote_params* p, const __nv_bfloat16* Q, const __nv_bfloat16* K, int64_t k_tok,
                            int64_t k_head, const int32_t* cu, int32_t batch, int64_t total_tokens, int64_t max_N,
                            float* real_logits, uint32_t* rowmax_part, int* n_part, const VoteState& vs, uint32_t* mask,
                            int64_t row_words, int32_t* status, const int32_t* kv_len, cudaStream_t st) {
  const int Hq = p->n_q_heads, Hkv = p->n_kv_heads, G = Hq / Hkv, d_k = p->d_k;
  const int row_chunks = score_geometry(p).row_chunks;
  CUtensorMap tmK, tmQ, tmQr;
  if (!encode_maps(p, Q, K, k_tok, k_head, batch, total_tokens, &tmK, &tmQ, &tmQr)) return GVOTE_ERR_UNSUPPORTED_SHAPE;
  const int kchunks = d_k / 64;
  const size_t out_bytes = (size_t)kRowChunk * kTileKeys * 2;
  const size_t qr = align_up((size_t)kchunks * kRealCols * 128, 1024);
  // one staging buffer: a CTA has few sampled tiles, and a deeper ring of key stages is worth more to the stream
  int stages = 0;
  const int n_out = 1;
  const int cg = pick_chunks(row_chunks > 2 ? 2 : row_chunks, kchunks, qr + out_bytes, 2, &stages);
  if (cg == 0) return GVOTE_ERR_UNSUPPORTED_SHAPE;
  const size_t smem = 1024 + (size_t)cg * kchunks * kRowChunk * 128 + qr + (size_t)stages * kchunks * kTileKeys * 128 +
                      n_out * out_bytes + sizeof(SweepTail) + 64;
  const int groups = (row_chunks + cg - 1) / cg;
  // CTAs per (request, KV head): one per SM when the batch is uniform; a ragged batch gets four times as
  // many, shorter CTAs so that the hardware scheduler can even out long and short requests.  The group that
  // streams every tile takes most of them, the groups that visit only the sampled tiles the rest.
  const int64_t max_tiles = ceil_div(max_N, kTileKeys);
  int64_t budget = (batch == 1 ? 148 : 592) / ((int64_t)Hkv * batch);
  if (budget < 1) budget = 1;
  int64_t X1 = groups > 1 ? budget / (6 * (groups - 1)) : 0;
  if (groups > 1 && X1 < 1) X1 = 1;
  int64_t X0 = budget - (groups - 1) * X1;
  if (X0 < 1) X0 = 1;
  if (X0 > max_tiles) X0 = max_tiles;
  dim3 grid((unsigned)(X0 > X1 ? X0 : X1), (unsigned)(Hkv * groups), (unsigned)batch);
  const float scale = (float)(1.0 / sqrt((double)d_k));
  GVOTE_CUDA_CHECK(cudaFuncSetAttribute(score_sample_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  {
    LaunchScope scope_("score_sample_kernel", st);
    launch_on(score_sample_kernel, grid, dim3(kSweepThreads), smem, st, tmK, tmQ, tmQr, cu, Hq, G, p->S, d_k, row_chunks, cg,
               (int)X0, (int)X1, stages, n_out, scale, real_logits, rowmax_part, vs.sample, vs.sample_slots, status, kv_len,
               vs.tmask, mask, (int64_t)Hkv * row_words, vs.head_bad, (int)(batch * Hkv));
  }
  *n_part = (int)X0;
  GVOTE_LAUNCH_CHECK("score_sample_kernel");
  return GVOTE_OK;
}

// Chunks per CTA, key stages and CTAs per (request, KV head, chunk group) of the second pass.
SweepGeom sweep_geometry(const gvote_params* p, int32_t batch, int64_t max_N) {
  SweepGeom g{0, 0, 1, 1, 16};
  if (!sweep_umma_supported(p)) return g;
  const int row_chunks = score_geometry(p).row_chunks;
  // chunks per CTA: their query rows share 256 columns of tensor memory, d_k / 2 columns a chunk
  int cg = 4;
  while (cg > 1 && (cg * (p->d_k / 2) > 256 || cg / 2 >= row_chunks)) cg >>= 1;
  g.cg = cg;
  const size_t stage = (size_t)(p->d_k / 64) * kTileKeys * 128;
  const size_t fixed = 1024 + (size_t)kSweepEpiWarps * 32 * 64 + sizeof(SweepTail) + 64;
  g.stages = (int)((kSmemLimit - fixed) / stage);
  if (g.stages > kMaxStages) g.stages = kMaxStages;
  if (g.stages < 2) { g.cg = 0; return g; }
  g.groups = (row_chunks + g.cg - 1) / g.cg;
  const int64_t max_tiles = ceil_div(max_N > 0 ? max_N : 1, kTileKeys);
  int64_t X = (batch == 1 ? 148 : 592) / ((int64_t)p->n_kv_heads * g.groups * batch);
  if (X > max_tiles) X = max_tiles;
  if (X < 1) X = 1;
  g.X = (int)X;
  return g;
}

// Second pass (after bracket_kernel).
int32_t launch_score_sweep(const gvote_params* p, const __nv_bfloat16* Q, const __nv_bfloat16* K, int64_t k_tok,
                           int64_t k_head, const int32_t* cu, int32_t batch, int64_t total_tokens, int64_t max_N,
                           const VoteState& vs, int64_t row_words, int32_t* status, const int32_t* kv_len,
                           cudaStream_t st) {
  const int Hq = p->n_q_heads, Hkv = p->n_kv_heads, G = Hq / Hkv, d_k = p->d_k;
  const int row_chunks = score_geometry(p).row_chunks;
  CUtensorMap tmK, tmQ;
  if (!encode_maps(p, Q, K, k_tok, k_head, batch, total_tokens, &tmK, &tmQ, nullptr)) return GVOTE_ERR_UNSUPPORTED_SHAPE;
  const int kchunks = d_k / 64;
  const SweepGeom geo = sweep_geometry(p, batch, max_N);
  if (geo.cg == 0 || vs.lay.segs != 4 * geo.X) return GVOTE_ERR_UNSUPPORTED_SHAPE;
  const size_t smem = 1024 + (size_t)geo.stages * kchunks * kTileKeys * 128 + (size_t)kSweepEpiWarps * 32 * geo.stg * 4 +
                      sizeof(SweepTail) + 64;
  dim3 grid((unsigned)geo.X, (unsigned)(Hkv * geo.groups), (unsigned)batch);
  const float scale = (float)(1.0 / sqrt((double)d_k));
  auto kern = geo.stg == 8 ? (geo.cg == 4 ? score_sweep_kernel<4, 8> : (geo.cg == 2 ? score_sweep_kernel<2, 8> : score_sweep_kernel<1, 8>))
                           : (geo.cg == 4 ? score_sweep_kernel<4, 16> : (geo.cg == 2 ? score_sweep_kernel<2, 16> : score_sweep_kernel<1, 16>));
  GVOTE_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  {
    LaunchScope scope_("score_sweep_kernel", st);
    // accumulators: three when the query rows leave room in the 512 columns of tensor memory, else two
    const int nbuf = (512 - geo.cg * (d_k / 2)) / kRowChunk >= 3 ? 3 : 2;
    launch_on(kern, grid, dim3(kSweepBThreads), smem, st, tmK, Q, cu, Hq, G, p->S, d_k, row_chunks, geo.stages, nbuf, scale, vs, row_words,
                                             status, kv_len);
  }
  GVOTE_LAUNCH_CHECK("score_sweep_kernel");
  return GVOTE_OK;
}

}  // namespace gvote
