// Step 2 of the GVote scheme (Section 3.2; the Gaussian fit of Algorithm 1): per-channel mean and unbiased variance of the
// hidden states along the sequence axis, skipping the first n_s sink tokens of every request.
//
// The hidden-state matrix is the largest tensor the pass touches (16 KiB per token at d_h = 4096
// in fp32), so this is a pure HBM stream.  Each CTA owns a strip of 256 channels and a chunk of
// rows and pulls them through a ring of shared-memory stages: one thread asks the TMA unit for a
// [32 rows x 256 channels] box per stage (marked evict-first in L2: the data is read once), eight
// warps take the stages as they land and keep shifted first and second moments of four channels
// per thread in registers.  Few threads and registers per SM stay busy that way, which leaves room
// for the kernels of other layers that run beside the fit on other streams.  One (mean, M2) pair
// per channel and chunk goes to scratch; a second, tiny kernel merges the chunks with Chan's
// parallel-variance update in fp64.
//
// Every mbarrier wait is bounded; on expiry the CTA raises GVOTE_ERR_TIMEOUT in the status word
// (where the caller gave one), lets its copies in flight land, and writes NaN partials so that the
// failure cannot pass for a result.
#include <mutex>

#include "common.cuh"
#include "ptx.cuh"

namespace gvote {
namespace {

constexpr int kFitTx = 64;                 // column threads (x4 channels each)
constexpr int kFitTy = 4;                  // row lanes
constexpr int kFitRows = 32;               // rows per stage of fp32 hidden states (bf16: twice as many, the same 32 KB)
constexpr int kFitConsumers = kFitTx * kFitTy;
constexpr int kFitThreads = kFitConsumers + 32;    // + the producer warp
constexpr int kFitMaxStages = 8;
constexpr int kFitFlushStages = 4;         // fold the running sums into a second level every so many stages
constexpr uint32_t kFitWaitPolls = 1u << 22;

template <typename T>
__device__ __forceinline__ float4 lds4(const T* p);
template <>
__device__ __forceinline__ float4 lds4<float>(const float* p) {
  return *reinterpret_cast<const float4*>(p);
}
template <>
__device__ __forceinline__ float4 lds4<__nv_bfloat16>(const __nv_bfloat16* p) {
  const uint2 u = *reinterpret_cast<const uint2*>(p);
  float4 r;
  r.x = __uint_as_float(u.x << 16);
  r.y = __uint_as_float(u.x & 0xffff0000u);
  r.z = __uint_as_float(u.y << 16);
  r.w = __uint_as_float(u.y & 0xffff0000u);
  return r;
}

__device__ __forceinline__ void acc4(float4& s1, float4& s2, const float4& v, const float4& sh) {
  float dx = v.x - sh.x, dy = v.y - sh.y, dz = v.z - sh.z, dw = v.w - sh.w;
  s1.x += dx; s1.y += dy; s1.z += dz; s1.w += dw;
  s2.x = fmaf(dx, dx, s2.x); s2.y = fmaf(dy, dy, s2.y);
  s2.z = fmaf(dz, dz, s2.z); s2.w = fmaf(dw, dw, s2.w);
}
__device__ __forceinline__ void add4(float4& a, const float4& b) { a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w; }

// tmH describes h as [rows][d_h] with a [rows per stage x 256] box.  Its row extent may be an upper bound:
// a stage that would reach past the chunk's last row is fetched row by row instead, so no load
// touches a row the chunk does not own.
template <typename T>
__global__ void __launch_bounds__(kFitThreads)
fit_partial_kernel(const __grid_constant__ CUtensorMap tmH, const T* __restrict__ h, int64_t ld,
                   const int32_t* __restrict__ cu, int n_s, int d_h, int chunks, int stages,
                   float2* __restrict__ partial, int32_t* __restrict__ status) {
  extern __shared__ __align__(1024) uint8_t fit_ring[];
  __shared__ uint64_t full[kFitMaxStages], empty[kFitMaxStages];
  __shared__ int abort_flag;
  __shared__ float4 sm1[kFitTy][kFitTx], sm2[kFitTy][kFitTx];
  constexpr int R = kFitRows * (4 / (int)sizeof(T));       // 32 KB per stage whatever the element type
  constexpr uint32_t pitch = kFitStripCols * sizeof(T);
  constexpr uint32_t stage_bytes = R * pitch;
  const int r = blockIdx.z, c = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int col0 = blockIdx.x * kFitStripCols;
  const int width = min(kFitStripCols, d_h - col0);
  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], kFitConsumers / 32); }
    abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&tmH);
  }
  __syncthreads();
  int a, b;
  fit_chunk_rows(cu[r] + n_s, cu[r + 1], chunks, c, a, b);
  const int n_it = (b > a) ? (b - a + R - 1) / R : 0;
  const int tx = threadIdx.x % kFitTx, ty = (threadIdx.x / kFitTx) % kFitTy;
  const bool active = tx * 4 < width;
  float4 sh = make_float4(0.f, 0.f, 0.f, 0.f);

  if (warp == kFitConsumers / 32) {
    // ------------------------------------------------------------ producer
    const uint64_t pol = ptx::l2_policy_evict_first();
    int issued = 0;
    bool ok = true;
    for (int it = 0; it < n_it; ++it) {
      const int s = it % stages;
      if (it >= stages) {
        const uint32_t par = ((uint32_t)(it / stages) & 1u) ^ 1u;
        ok = ptx::mbar_wait(&empty[s], par, kFitWaitPolls) && !*(volatile int*)&abort_flag;
        if (!ok) break;
      }
      const int row = a + it * R;
      const int rows_here = min(R, b - row);
      uint8_t* dst = fit_ring + (size_t)s * stage_bytes;
      if (rows_here == R) {
        if (lane == 0) {
          ptx::mbar_arrive_expect_tx(&full[s], stage_bytes);
          ptx::tma_load_2d_hint(dst, &tmH, &full[s], col0, row, pol);
        }
      } else {
        const uint32_t row_bytes = (uint32_t)width * sizeof(T);
        if (lane == 0) ptx::mbar_arrive_expect_tx(&full[s], (uint32_t)rows_here * row_bytes);
        __syncwarp();
        for (int rr = lane; rr < rows_here; rr += 32)
          ptx::bulk_load(dst + (size_t)rr * pitch, h + (int64_t)(row + rr) * ld + col0, row_bytes, &full[s]);
      }
      issued = it + 1;
    }
    if (!ok) {
      if (lane == 0) abort_flag = 1;
      for (int it = max(issued - stages, 0); it < issued; ++it)      // let the copies in flight land
        ptx::mbar_wait(&full[it % stages], (uint32_t)(it / stages) & 1u, kFitWaitPolls);
    }
  } else {
    // ------------------------------------------------------------ consumers
    float4 s1 = make_float4(0.f, 0.f, 0.f, 0.f), s2 = s1, t1 = s1, t2 = s1;
    for (int it = 0; it < n_it; ++it) {
      const int s = it % stages;
      if (!ptx::mbar_wait(&full[s], (uint32_t)(it / stages) & 1u, kFitWaitPolls) || *(volatile int*)&abort_flag) {
        abort_flag = 1;
        break;
      }
      const T* st = reinterpret_cast<const T*>(fit_ring + (size_t)s * stage_bytes);
      const int rows_here = min(R, b - (a + it * R));
      if (active) {
        if (it == 0) sh = lds4<T>(st + tx * 4);     // shift: the chunk's first row (same for all row lanes)
        if (rows_here == R) {
#pragma unroll
          for (int sub = 0; sub < R; sub += kFitRows) {      // 16 loads in flight, then 16 updates
            float4 v[kFitRows / kFitTy];
#pragma unroll
            for (int j = 0; j < kFitRows / kFitTy; ++j)
              v[j] = lds4<T>(st + (size_t)(sub + ty + j * kFitTy) * kFitStripCols + tx * 4);
#pragma unroll
            for (int j = 0; j < kFitRows / kFitTy; ++j) acc4(s1, s2, v[j], sh);
          }
        } else {
          for (int row = ty; row < rows_here; row += kFitTy)
            acc4(s1, s2, lds4<T>(st + (size_t)row * kFitStripCols + tx * 4), sh);
        }
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&empty[s]);
      if ((it + 1) % kFitFlushStages == 0) {        // short fp32 runs: the rounding error stays that of a few dozen terms
        add4(t1, s1); add4(t2, s2);
        s1 = make_float4(0.f, 0.f, 0.f, 0.f); s2 = s1;
      }
    }
    add4(t1, s1); add4(t2, s2);
    sm1[ty][tx] = t1;
    sm2[ty][tx] = t2;
  }
  __syncthreads();
  const bool failed = abort_flag != 0;
  if (threadIdx.x == 0 && failed && status) {
    atomicExch(&status[0], GVOTE_ERR_TIMEOUT);
    atomicExch(&status[1], 7);
  }
  if (threadIdx.x < kFitTx && active) {
    double t1[4] = {0, 0, 0, 0}, t2[4] = {0, 0, 0, 0};
#pragma unroll
    for (int j = 0; j < kFitTy; ++j) {
      float4 u = sm1[j][tx], w = sm2[j][tx];
      t1[0] += u.x; t1[1] += u.y; t1[2] += u.z; t1[3] += u.w;
      t2[0] += w.x; t2[1] += w.y; t2[2] += w.z; t2[3] += w.w;
    }
    const int n = b - a;
    const float shv[4] = {sh.x, sh.y, sh.z, sh.w};
    float2* out = partial + ((int64_t)(r * chunks + c)) * d_h + col0 + tx * 4;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      double mean = 0.0, m2 = 0.0;
      if (n > 0) {
        mean = (double)shv[j] + t1[j] / n;
        m2 = t2[j] - t1[j] * t1[j] / n;
      }
      out[j] = failed ? make_float2(nanf(""), nanf("")) : make_float2((float)mean, (float)fmax(m2, 0.0));
    }
  }
}

// Merge of the chunks of a request (see fit_merge_lane).  A CTA covers 32 channels; eight row lanes
// each fold every eighth chunk, then lane 0 adds the eight partial results.
__global__ void __launch_bounds__(256)
fit_finalize_kernel(const float2* __restrict__ partial, const int32_t* __restrict__ cu, int n_s, int d_h, int chunks,
                    float* __restrict__ mu, float* __restrict__ var) {
  __shared__ FitMoments sm[8][32];
  const int r = blockIdx.y;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int col = blockIdx.x * 32 + tx;
  const int first = cu[r] + n_s, last = cu[r + 1];
  FitMoments acc{0.0, 0.0, 0.0};
  double ref = 0.0;
  if (col < d_h) {
    ref = (double)partial[((int64_t)r * chunks) * d_h + col].x;
    acc = fit_merge_lane(partial, r, chunks, d_h, col, first, last, ty, 8, ref);
  }
  sm[ty][tx] = acc;
  __syncthreads();
  if (ty == 0 && col < d_h) {
    for (int j = 1; j < 8; ++j) { acc.n += sm[j][tx].n; acc.a += sm[j][tx].a; acc.bc += sm[j][tx].bc; }
    fit_merge_finish(acc, ref, mu[(int64_t)r * d_h + col], var[(int64_t)r * d_h + col]);
  }
}

// ---------------------------------------------------------------------------------- streaming fit
// Running moments per request and channel, fp64: state[r][0][c] = rows seen, [1][c] = mean, [2][c] =
// sum of squared deviations.  One block of rows is reduced by fit_partial_kernel as usual; this kernel
// merges the block's chunks and folds them into the state with the pairwise update of Chan, Golub
// and LeVeque.
__global__ void __launch_bounds__(256)
fit_state_update_kernel(const float2* __restrict__ partial, const int32_t* __restrict__ cu, int d_h, int chunks,
                        double* __restrict__ state) {
  __shared__ FitMoments sm[8][32];
  const int r = blockIdx.y;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int col = blockIdx.x * 32 + tx;
  const int first = cu[r], last = cu[r + 1];
  FitMoments acc{0.0, 0.0, 0.0};
  double ref = 0.0;
  if (col < d_h && last > first) {
    ref = (double)partial[((int64_t)r * chunks) * d_h + col].x;
    acc = fit_merge_lane(partial, r, chunks, d_h, col, first, last, ty, 8, ref);
  }
  sm[ty][tx] = acc;
  __syncthreads();
  if (ty == 0 && col < d_h && last > first) {
    for (int j = 1; j < 8; ++j) { acc.n += sm[j][tx].n; acc.a += sm[j][tx].a; acc.bc += sm[j][tx].bc; }
    const double nb = acc.n, mean_b = ref + acc.a / acc.n, m2_b = fmax(acc.bc - acc.a * acc.a / acc.n, 0.0);
    double* st = state + (int64_t)r * 3 * d_h;
    const double na = st[col];
    if (na <= 0.0) {
      st[col] = nb; st[d_h + col] = mean_b; st[2 * d_h + col] = m2_b;
    } else {
      const double n = na + nb, delta = mean_b - st[d_h + col];
      st[col] = n;
      st[d_h + col] += delta * (nb / n);
      st[2 * d_h + col] += m2_b + delta * delta * (na * nb / n);
    }
  }
}

__global__ void fit_state_finish_kernel(const double* __restrict__ state, int d_h, float* __restrict__ mu,
                                        float* __restrict__ var) {
  const int r = blockIdx.y, col = blockIdx.x * blockDim.x + threadIdx.x;
  if (col >= d_h) return;
  const double* st = state + (int64_t)r * 3 * d_h;
  mu[(int64_t)r * d_h + col] = (float)st[d_h + col];
  var[(int64_t)r * d_h + col] = (float)(st[2 * d_h + col] / (st[col] - 1.0));   // NaN/inf below two rows
}

}  // namespace

// `rows_bound`: an upper bound of the rows h holds (the packed token count, or batch x longest request).
int32_t launch_fit_partial(const gvote_params* p, const void* h, int64_t ld, const int32_t* cu, int32_t batch,
                           int64_t rows_bound, int fit_chunks, float2* partial, int32_t* status, cudaStream_t st) {
  const int strips = (int)ceil_div(p->d_h, kFitStripCols);
  const int elem = p->h_dtype == GVOTE_DTYPE_F32 ? 4 : 2;
  if (rows_bound < 1) rows_bound = 1;
  CUtensorMap tmH;
  {
    const uint64_t dims[2] = {(uint64_t)p->d_h, (uint64_t)rows_bound};
    const uint64_t strides[1] = {(uint64_t)ld * elem};
    const uint32_t box[2] = {(uint32_t)kFitStripCols, (uint32_t)(kFitRows * (4 / elem))};
    if (!encode_tensor_map_plain(&tmH, h, elem, 2, dims, strides, box)) return GVOTE_ERR_UNSUPPORTED_SHAPE;
  }
  // 96 KB of stages per CTA: what keeps one CTA per SM at the HBM rate
  const size_t stage_bytes = (size_t)kFitRows * (4 / elem) * kFitStripCols * elem;
  int stages = (int)((96 * 1024) / stage_bytes);
  if (stages > kFitMaxStages) stages = kFitMaxStages;
  const size_t smem = stages * stage_bytes;
  dim3 grid(strips, fit_chunks, batch);
  {
    LaunchScope scope_("fit_partial_kernel", st);
    if (p->h_dtype == GVOTE_DTYPE_F32) {
      GVOTE_CUDA_CHECK(cudaFuncSetAttribute(fit_partial_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      launch_on(fit_partial_kernel<float>, grid, dim3(kFitThreads), smem, st, tmH, (const float*)h, ld, cu, p->n_s, p->d_h, fit_chunks,
                                                                 stages, partial, status);
    } else {
      GVOTE_CUDA_CHECK(cudaFuncSetAttribute(fit_partial_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      launch_on(fit_partial_kernel<__nv_bfloat16>, grid, dim3(kFitThreads), smem, st, tmH, (const __nv_bfloat16*)h, ld, cu, p->n_s,
                                                                         p->d_h, fit_chunks, stages, partial, status);
    }
  }
  GVOTE_LAUNCH_CHECK("fit_partial_kernel");
  return GVOTE_OK;
}

int32_t launch_fit(const gvote_params* p, const void* h, int64_t ld, const int32_t* cu, int32_t batch,
                   int64_t rows_bound, int fit_chunks, float2* partial, int32_t* status, float* mu, float* var,
                   cudaStream_t st) {
  const int32_t rc = launch_fit_partial(p, h, ld, cu, batch, rows_bound, fit_chunks, partial, status, st);
  if (rc != GVOTE_OK) return rc;
  dim3 g2((unsigned)ceil_div(p->d_h, 32), batch);
  {
    LaunchScope scope_("fit_finalize_kernel", st);
    fit_finalize_kernel<<<g2, 256, 0, st>>>(partial, cu, p->n_s, p->d_h, fit_chunks, mu, var);
  }
  GVOTE_LAUNCH_CHECK("fit_finalize_kernel");
  return GVOTE_OK;
}

int32_t launch_fit_state_update(const gvote_params* p, const void* h, int64_t ld, const int32_t* cu, int32_t batch,
                                int64_t rows_bound, int fit_chunks, float2* partial, int32_t* status, double* state,
                                cudaStream_t st) {
  gvote_params q = *p;
  q.n_s = 0;                                   // which rows to leave out is the caller's choice here
  const int32_t rc = launch_fit_partial(&q, h, ld, cu, batch, rows_bound, fit_chunks, partial, status, st);
  if (rc != GVOTE_OK) return rc;
  dim3 g2((unsigned)ceil_div(p->d_h, 32), batch);
  {
    LaunchScope scope_("fit_state_update_kernel", st);
    fit_state_update_kernel<<<g2, 256, 0, st>>>(partial, cu, p->d_h, fit_chunks, state);
  }
  GVOTE_LAUNCH_CHECK("fit_state_update_kernel");
  return GVOTE_OK;
}

// One CTA per SM of a 148-SM part streams at the HBM rate when the batch is a single request (all
// chunks alike); a batch of requests of different lengths gets eight times as many, so that the
// longest chunk is a small part of the whole.  At least two stages of rows per chunk.
int fit_chunk_count(const gvote_params* p, int32_t batch, int64_t max_N) {
  const int64_t strips = ceil_div(p->d_h, kFitStripCols);
  int64_t chunks = (batch == 1 ? 148 : 1184) / (strips * batch);
  const int64_t by_rows = ceil_div(max_N > 0 ? max_N : 1, 2 * kFitRows);
  if (chunks > by_rows) chunks = by_rows;
  if (chunks < 1) chunks = 1;
  return (int)chunks;
}

int32_t launch_fit_state_finish(const gvote_params* p, const double* state, int32_t batch, float* mu, float* var,
                                cudaStream_t st) {
  dim3 g((unsigned)ceil_div(p->d_h, 256), batch);
  {
    LaunchScope scope_("fit_state_finish_kernel", st);
    fit_state_finish_kernel<<<g, 256, 0, st>>>(state, p->d_h, mu, var);
  }
  GVOTE_LAUNCH_CHECK("fit_state_finish_kernel");
  return GVOTE_OK;
}

}  // namespace gvote

// ---------------------------------------------------------------------------------- no-allocation variant
// gvote_fit_static: the same two kernels as gvote_fit, with the per-chunk (mean, M2) partials kept
// in a fixed array that is part of the loaded library image instead of a caller workspace.  It is
// meant for callers that cannot obtain device memory at the point where they need the fit: code
// running inside a memory-pool callback, a serving loop whose allocator is frozen after warm-up,
// or a host thread that must not take the allocator's lock.

namespace gvote {
namespace {

constexpr size_t kStaticFitEntries = GVOTE_FIT_STATIC_MAX_ENTRIES;   // float2 entries, 1 MiB in all
static __device__ __align__(256) float2 g_fit_static_scratch[kStaticFitEntries];

// In host code the array's name only stands for the symbol; the address a kernel can use has to
// be asked for, once per device, while that device is current.
constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
float2* g_static_ptr[kMaxDevices] = {};

int32_t static_scratch_for_current_device(float2** out) {
  int dev = -1;
  GVOTE_CUDA_CHECK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return GVOTE_ERR_UNSUPPORTED_SHAPE;
  std::lock_guard<std::mutex> lk(g_static_mu);
  if (!g_static_ptr[dev]) {
    void* ptr = nullptr;
    GVOTE_CUDA_CHECK(cudaGetSymbolAddress(&ptr, g_fit_static_scratch));
    if (!ptr) return GVOTE_ERR_CUDA;
    g_static_ptr[dev] = static_cast<float2*>(ptr);
  }
  *out = g_static_ptr[dev];
  return GVOTE_OK;
}

}  // namespace
}  // namespace gvote

extern "C" int32_t gvote_fit_static(const gvote_params* p, const void* h, int64_t h_row_stride,
                                    const int32_t* cu_seqlens, int32_t batch, int64_t max_N, float* mu, float* var,
                                    void* stream) {
  using namespace gvote;
  const int32_t pv = validate_params(p);
  if (pv != GVOTE_OK) return pv;
  if (batch < 1 || max_N < 0) return GVOTE_ERR_INVALID_ARG;
  if (!h || !cu_seqlens || !mu || !var) return GVOTE_ERR_INVALID_ARG;
  if (!aligned16(h) || !aligned16(cu_seqlens) || !aligned16(mu) || !aligned16(var)) return GVOTE_ERR_UNALIGNED;
  if (h_row_stride < p->d_h || h_row_stride % 8 != 0) return GVOTE_ERR_UNALIGNED;
  if (max_N - p->n_s < 2) return GVOTE_ERR_INVALID_ARG;
  // one chunk per request is the least the kernels can run with
  const int64_t per_chunk = (int64_t)batch * p->d_h;
  if (per_chunk > (int64_t)kStaticFitEntries) return GVOTE_ERR_UNSUPPORTED_SHAPE;
  // as many row chunks as the fit wants, as few as the fixed array holds
  int64_t chunks = fit_chunk_count(p, batch, max_N);
  const int64_t fit_in_array = (int64_t)kStaticFitEntries / per_chunk;
  if (chunks > fit_in_array) chunks = fit_in_array;
  float2* scratch = nullptr;
  const int32_t sv = static_scratch_for_current_device(&scratch);
  if (sv != GVOTE_OK) return sv;
  // every entry the merge kernel reads is written by the partial kernel of the same call, so the
  // array needs no clearing between calls
  // no status word here: a wait that ran out shows as NaN in mu and var
  return launch_fit(p, h, h_row_stride, cu_seqlens, batch, (int64_t)batch * max_N, (int)chunks, scratch, nullptr, mu, var,
                    (cudaStream_t)stream);
}
