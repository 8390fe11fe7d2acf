// Algorithm 1 line 9 for the synthetic queries: the k = |C0| largest logits of a row, found on the
// 16-bit keys the tensor-core score kernel leaves behind (the upper half of an order-preserving
// image of each fp32 logit), and OR-ed into the head's keep mask (line 10).
//
// One CTA per synthetic row.
//   A. The row is read once from the tile-blocked key buffer into shared memory; while it streams
//      in, its high bytes are counted in a histogram that keeps one counter per (bin, lane), so no
//      two lanes of a warp ever hit the same address.
//   B. The 256 bins are reduced; the bin holding the k-th largest key is found by a suffix scan.
//   C. The low bytes of the keys in that bin are counted (plain 256-bin histogram: few keys, well
//      spread), which fixes the 16-bit threshold T: keys above T are selected outright.
//   D. One pass over the row emits the mask words (8 keys per thread, 4 threads per word) and
//      collects the keys equal to T.  Those candidates share 16 leading bits, so their order is
//      settled exactly: their logits are recomputed in fp32 from Q and K and ranked by (value
//      descending, index ascending); the first k - #above of them are selected.
// Rows longer than the shared-memory budget are streamed from global memory in each pass instead.
#include "common.cuh"

namespace gvote {
namespace {

constexpr int kThreads = 256;
constexpr int kTieCap = 1024;
constexpr int kTileKeys = 128;

struct Sel16Shared {
  uint32_t hist[256];
  float qf[512];
  int tie_idx[kTieCap];
  float tie_val[kTieCap];
  uint32_t red32[kThreads / 32];
  int bin;
  uint32_t above;
  uint32_t ntie;
};

// Largest bin b of hist[0..256) whose suffix count reaches `need` (need >= 1, total >= need).
__device__ void find_bin256(Sel16Shared& sh, uint32_t need) {
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    uint32_t c = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) c += sh.hist[lane * 8 + i];
    uint32_t cs = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t t = __shfl_down_sync(0xffffffffu, cs, o);
      if (lane + o < 32) cs += t;
    }
    const uint32_t excl = cs - c;
    if (lane == 0) { sh.bin = 0; sh.above = 0; }
    __syncwarp();
    if (excl < need && excl + c >= need) {
      uint32_t a = excl;
      int b = lane * 8 + 7;
      for (; b > lane * 8; --b) {
        if (a + sh.hist[b] >= need) break;
        a += sh.hist[b];
      }
      sh.bin = b;
      sh.above = a;
    }
  }
  __syncthreads();
}

// Exact fp32 logit of key n for this row's query (fixed summation order).
struct DotCtx {
  const float* qf;
  const __nv_bfloat16* krows;   // K + head offset + request start
  int64_t k_tok;
  int d_k;
  float scale;
  __device__ __forceinline__ float operator()(int n) const {
    const uint4* kp = reinterpret_cast<const uint4*>(krows + (int64_t)n * k_tok);
    float acc = 0.f;
    for (int c = 0; c < d_k / 8; ++c) {
      const uint4 v = __ldg(kp + c);
      const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 f = __bfloat1622float2(h[j]);
        acc = fmaf(qf[c * 8 + 2 * j], f.x, acc);
        acc = fmaf(qf[c * 8 + 2 * j + 1], f.y, acc);
      }
    }
    return acc * scale;
  }
};

// Where a row's keys live: eight consecutive keys form one 16-byte vector; vector v8 of the row
// sits in tile v8 / 16 at offset (v8 % 16) * 8.  Keys at positions >= N are read as 0 (below any
// real key, whose image is never 0).
struct RowView {
  const uint16_t* smem_row;     // non-null when the row is resident in shared memory
  const uint16_t* grow;         // first tile of the row in global memory
  int64_t tile_stride;          // elements between consecutive tiles of the same row
  int N;
  __device__ __forceinline__ uint4 mask_tail(uint4 v, int v8) const {
    if (v8 * 8 + 8 > N) {
      uint16_t* e = reinterpret_cast<uint16_t*>(&v);
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (v8 * 8 + j >= N) e[j] = 0;
    }
    return v;
  }
  __device__ __forceinline__ uint4 load_global(int v8) const {
    const uint4 v = *reinterpret_cast<const uint4*>(grow + (int64_t)(v8 >> 4) * tile_stride + (v8 & 15) * 8);
    return mask_tail(v, v8);
  }
  __device__ __forceinline__ uint4 load(int v8) const {
    if (smem_row) return *reinterpret_cast<const uint4*>(smem_row + (size_t)v8 * 8);
    return load_global(v8);
  }
  __device__ __forceinline__ uint32_t key_at(int n) const {
    if (smem_row) return smem_row[n];
    return grow[(int64_t)(n >> 7) * tile_stride + (n & 127)];
  }
};

__global__ void __launch_bounds__(kThreads, 2)
topk16_rows_kernel(const uint16_t* __restrict__ keys16, const __nv_bfloat16* __restrict__ Q,
                   const __nv_bfloat16* __restrict__ K, int64_t k_tok, int64_t k_head,
                   const int32_t* __restrict__ cu, int Hq, int G, int S, int d_k, int RC, int row_chunks,
                   int64_t n_tiles_total, float scale, const int32_t* __restrict__ b_step, int64_t row_words,
                   uint32_t* __restrict__ mask, int row_elems) {
  extern __shared__ __align__(16) uint8_t dyn_smem[];
  __shared__ Sel16Shared sh;
  uint32_t* hist1 = reinterpret_cast<uint32_t*>(dyn_smem);                     // [256][32]
  uint16_t* row_sm = reinterpret_cast<uint16_t*>(dyn_smem + 256 * 32 * 4);     // [row_elems]
  const int r = blockIdx.z, g = blockIdx.y, s = blockIdx.x;
  const int start = cu[r], N = cu[r + 1] - start;
  if (N <= 0) return;
  int k = b_step[r * Hq + g];
  if (k <= 0) return;
  if (k > N) k = N;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int kh = g / G;
  const int grow_idx = (g % G) * S + s;                  // row within the head group (synthetic rows come first)
  const int chunk = grow_idx / RC, crow = grow_idx % RC;
  RowView rv;
  rv.N = N;
  rv.tile_stride = (int64_t)row_chunks * RC * kTileKeys;
  rv.grow = keys16 + ((((int64_t)kh * n_tiles_total + tile_offset(start, r)) * row_chunks + chunk) * RC + crow) * kTileKeys;
  const bool fits = N <= row_elems;
  rv.smem_row = fits ? row_sm : nullptr;
  uint32_t* mrow = mask + (int64_t)kh * row_words + mask_word_offset(start, r);
  const int nv8 = (N + 7) >> 3;

  {
    const __nv_bfloat16* qrow = Q + (((int64_t)r * (Hq / G) + kh) * (G * (S + 1)) + grow_idx) * d_k;
    for (int i = tid; i < d_k; i += kThreads) sh.qf[i] = __bfloat162float(qrow[i]);
    for (int i = tid; i < 256 * 32; i += kThreads) hist1[i] = 0;
    if (tid == 0) sh.ntie = 0;
  }
  __syncthreads();

  // A. load the row, count high bytes (one counter per bin and lane)
  // (eight 16-byte loads are put in flight before any of them is consumed)
  for (int base = 0; base < nv8; base += kThreads * 8) {
    uint4 buf[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int v8 = base + u * kThreads + tid;
      buf[u] = (v8 < nv8) ? rv.load_global(v8) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int v8 = base + u * kThreads + tid;
      if (v8 < nv8) {
        if (fits) *reinterpret_cast<uint4*>(row_sm + (size_t)v8 * 8) = buf[u];
        const uint32_t w[4] = {buf[u].x, buf[u].y, buf[u].z, buf[u].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          atomicAdd(&hist1[((w[j] >> 8) & 255u) * 32 + lane], 1u);
          atomicAdd(&hist1[(w[j] >> 24) * 32 + lane], 1u);
        }
      }
    }
  }
  __syncthreads();
  // B. reduce over lanes (rotated read: conflict free); the padding keys (0) sit in bin 0
  {
    uint32_t c = 0;
#pragma unroll 8
    for (int j = 0; j < 32; ++j) c += hist1[tid * 32 + ((j + tid) & 31)];
    if (tid == 0) c -= (uint32_t)(nv8 * 8 - N);
    sh.hist[tid] = c;
  }
  __syncthreads();
  find_bin256(sh, (uint32_t)k);
  const uint32_t b_hi = (uint32_t)sh.bin;
  uint32_t above = sh.above;
  __syncthreads();
  sh.hist[tid] = 0;
  __syncthreads();
  // C. low bytes of the keys whose high byte is b_hi
  for (int v8 = tid; v8 < nv8; v8 += kThreads) {
    const uint4 v = rv.load(v8);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (((w[j] >> 8) & 255u) == b_hi && (v8 * 8 + 2 * j) < N) atomicAdd(&sh.hist[w[j] & 255u], 1u);
      if ((w[j] >> 24) == b_hi && (v8 * 8 + 2 * j + 1) < N) atomicAdd(&sh.hist[(w[j] >> 16) & 255u], 1u);
    }
  }
  __syncthreads();
  find_bin256(sh, (uint32_t)k - above);
  const uint32_t T = (b_hi << 8) | (uint32_t)sh.bin;
  above += sh.above;
  const uint32_t eq = sh.hist[sh.bin];
  const uint32_t ties = (uint32_t)k - above;        // 1 <= ties <= eq
  __syncthreads();

  // D. emit: 8 keys per thread, 4 threads per mask word; collect the keys equal to T
  const bool all_ties = ties >= eq;
  for (int base = 0; base < nv8; base += kThreads) {
    const int v8 = base + tid;
    uint32_t bits = 0, eqbits = 0;
    if (v8 < nv8) {
      const uint4 v = rv.load(v8);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t lo = w[j] & 0xffffu, hi = w[j] >> 16;
        bits |= (lo > T ? 1u : 0u) << (2 * j);
        bits |= (hi > T ? 1u : 0u) << (2 * j + 1);
        eqbits |= (lo == T ? 1u : 0u) << (2 * j);
        eqbits |= (hi == T ? 1u : 0u) << (2 * j + 1);
      }
      if (T == 0) eqbits &= (v8 * 8 + 8 > N) ? ((1u << (N - v8 * 8)) - 1u) : 0xffu;   // padding is not a key
    }
    if (all_ties) bits |= eqbits;
    else {
      while (eqbits) {
        const int j = __ffs(eqbits) - 1;
        eqbits &= eqbits - 1;
        const uint32_t slot = atomicAdd(&sh.ntie, 1u);
        if (slot < (uint32_t)kTieCap) sh.tie_idx[slot] = v8 * 8 + j;
      }
    }
    uint32_t word = bits << (8 * (lane & 3));
    word |= __shfl_xor_sync(0xffffffffu, word, 1);
    word |= __shfl_xor_sync(0xffffffffu, word, 2);
    if ((lane & 3) == 0 && word) atomicOr(&mrow[v8 >> 2], word);
  }
  if (all_ties) return;
  __syncthreads();

  DotCtx dot{sh.qf, K + (int64_t)kh * k_head + (int64_t)start * k_tok, k_tok, d_k, scale};
  if (eq <= (uint32_t)kTieCap) {
    // rank the candidates by (exact logit descending, index ascending) and keep the first `ties`
    for (int i = tid; i < (int)eq; i += kThreads) sh.tie_val[i] = dot(sh.tie_idx[i]);
    __syncthreads();
    for (int i = tid; i < (int)eq; i += kThreads) {
      const float v = sh.tie_val[i];
      const int n = sh.tie_idx[i];
      uint32_t rank = 0;
      for (int u = 0; u < (int)eq; ++u) {
        const float vu = sh.tie_val[u];
        rank += (vu > v || (vu == v && sh.tie_idx[u] < n)) ? 1u : 0u;
      }
      if (rank < ties) atomicOr(&mrow[n >> 5], 1u << (n & 31));
    }
    return;
  }

  // More candidates than the list holds (many equal logits): radix search over the recomputed
  // 32-bit images of the candidates, four 8-bit passes, then an emission in index order.
  uint32_t prefix = 0, known = 0, acc = 0, eq2 = 0;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    sh.hist[tid] = 0;
    __syncthreads();
    for (int n = tid; n < N; n += kThreads) {
      if (rv.key_at(n) == T) {
        const uint32_t key = ordered_key(dot(n));
        if ((key & known) == prefix) atomicAdd(&sh.hist[(key >> shift) & 255u], 1u);
      }
    }
    __syncthreads();
    find_bin256(sh, ties - acc);
    acc += sh.above;
    prefix |= (uint32_t)sh.bin << shift;
    known |= 255u << shift;
    if (pass == 3) eq2 = sh.hist[sh.bin];
    __syncthreads();
  }
  const uint32_t ties2 = ties - acc;
  uint32_t taken = 0;
  for (int base = 0; base < N; base += kThreads) {
    const int n = base + tid;
    const bool member = n < N && rv.key_at(n) == T;
    const uint32_t key = member ? ordered_key(dot(n)) : 0u;
    bool sel = member && key > prefix;
    const bool tie = member && key == prefix;
    if (ties2 >= eq2) {
      sel |= tie;
    } else {
      const uint32_t tb = __ballot_sync(0xffffffffu, tie);
      if (lane == 0) sh.red32[warp] = __popc(tb);
      __syncthreads();
      uint32_t before = taken, total = 0;
      for (int w = 0; w < kThreads / 32; ++w) {
        if (w < warp) before += sh.red32[w];
        total += sh.red32[w];
      }
      sel |= tie && (before + __popc(tb & ((1u << lane) - 1u))) < ties2;
      taken += total;
      __syncthreads();
    }
    const uint32_t bal = __ballot_sync(0xffffffffu, sel);
    if (lane == 0 && bal) atomicOr(&mrow[n >> 5], bal);
  }
}

}  // namespace

int32_t launch_topk16(const gvote_params* p, const uint16_t* keys16, const __nv_bfloat16* Q, const __nv_bfloat16* K,
                      int64_t k_tok, int64_t k_head, const int32_t* cu, int32_t batch, int64_t total_tokens,
                      int64_t max_N, const int32_t* b_step, int64_t row_words, uint32_t* mask, cudaStream_t st) {
  const int Hq = p->n_q_heads, G = Hq / p->n_kv_heads;
  const ScoreGeometry geo = score_geometry(p);
  // rows up to 80K keys stay resident in shared memory next to the 32 KB histogram; longer rows
  // are streamed from global memory in each pass
  int row_elems = (int)((max_N + 127) & ~(int64_t)127);
  if (row_elems > 80 * 1024) row_elems = 0;
  const size_t smem = 256 * 32 * 4 + (size_t)row_elems * sizeof(uint16_t);
  GVOTE_CUDA_CHECK(cudaFuncSetAttribute(topk16_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  dim3 grid(p->S, Hq, batch);
  const float scale = (float)(1.0 / sqrt((double)p->d_k));
  {
    LaunchScope scope_("topk16_rows_kernel", st);
    topk16_rows_kernel<<<grid, kThreads, smem, st>>>(keys16, Q, K, k_tok, k_head, cu, Hq, G, p->S, p->d_k, geo.RC,
                                                     geo.row_chunks, (total_tokens >> 7) + batch, scale, b_step,
                                                     row_words, mask, row_elems);
  }
  GVOTE_LAUNCH_CHECK("topk16_rows_kernel");
  return GVOTE_OK;
}

}  // namespace gvote
