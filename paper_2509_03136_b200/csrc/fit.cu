// Step 2 of the GVote scheme (Algorithm 1, line 4): per-channel mean and unbiased variance of the
// hidden states along the sequence axis, skipping the first n_s sink tokens of every request.
//
// The hidden-state matrix is the largest tensor the pass touches (16 KiB per token at d_h = 4096
// in fp32), so this is a pure HBM stream: each CTA owns a strip of 256 channels and a chunk of
// rows, every thread keeps shifted first and second moments of four channels in registers, and
// one (mean, M2) pair per channel and chunk goes to scratch.  A second, tiny kernel merges the
// chunks with Chan's parallel-variance update in fp64.
#include <mutex>

#include "common.cuh"

namespace gvote {
namespace {

constexpr int kFitTx = 64;   // column threads (x4 channels each)
constexpr int kFitTy = 4;    // row lanes

template <typename T>
__device__ __forceinline__ float4 load4(const T* p);
template <>
__device__ __forceinline__ float4 load4<float>(const float* p) {
  return __ldcs(reinterpret_cast<const float4*>(p));
}
template <>
__device__ __forceinline__ float4 load4<__nv_bfloat16>(const __nv_bfloat16* p) {
  uint2 u = __ldcs(reinterpret_cast<const uint2*>(p));
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

template <typename T>
__global__ void __launch_bounds__(kFitTx* kFitTy)
fit_partial_kernel(const T* __restrict__ h, int64_t ld, const int32_t* __restrict__ cu, int n_s, int d_h,
                   int chunks, float2* __restrict__ partial) {
  const int r = blockIdx.z, c = blockIdx.y;
  const int tx = threadIdx.x, ty = threadIdx.y;
  const int col = (blockIdx.x * kFitTx + tx) * 4;
  const bool active = col < d_h;
  int a, b;
  fit_chunk_rows(cu[r] + n_s, cu[r + 1], chunks, c, a, b);

  float4 s1 = make_float4(0.f, 0.f, 0.f, 0.f), s2 = s1, sh = s1;
  if (active && a < b) {
    const T* base = h + col;
    sh = load4<T>(base + (int64_t)a * ld);   // shift: the chunk's first row (same for all row lanes)
    int i = a + ty;
    for (; i + 3 * kFitTy < b; i += 4 * kFitTy) {
      float4 v0 = load4<T>(base + (int64_t)i * ld);
      float4 v1 = load4<T>(base + (int64_t)(i + kFitTy) * ld);
      float4 v2 = load4<T>(base + (int64_t)(i + 2 * kFitTy) * ld);
      float4 v3 = load4<T>(base + (int64_t)(i + 3 * kFitTy) * ld);
      acc4(s1, s2, v0, sh); acc4(s1, s2, v1, sh); acc4(s1, s2, v2, sh); acc4(s1, s2, v3, sh);
    }
    for (; i < b; i += kFitTy) {
      float4 v = load4<T>(base + (int64_t)i * ld);
      acc4(s1, s2, v, sh);
    }
  }
  __shared__ float4 sm1[kFitTy][kFitTx], sm2[kFitTy][kFitTx];
  sm1[ty][tx] = s1;
  sm2[ty][tx] = s2;
  __syncthreads();
  if (ty == 0 && active) {
    double t1[4] = {0, 0, 0, 0}, t2[4] = {0, 0, 0, 0};
#pragma unroll
    for (int j = 0; j < kFitTy; ++j) {
      float4 u = sm1[j][tx], w = sm2[j][tx];
      t1[0] += u.x; t1[1] += u.y; t1[2] += u.z; t1[3] += u.w;
      t2[0] += w.x; t2[1] += w.y; t2[2] += w.z; t2[3] += w.w;
    }
    const int n = b - a;
    const float shv[4] = {sh.x, sh.y, sh.z, sh.w};
    float2* out = partial + ((int64_t)(r * chunks + c)) * d_h + col;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      double mean = 0.0, m2 = 0.0;
      if (n > 0) {
        mean = (double)shv[j] + t1[j] / n;
        m2 = t2[j] - t1[j] * t1[j] / n;
      }
      out[j] = make_float2((float)mean, (float)fmax(m2, 0.0));
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

int32_t launch_fit_partial(const gvote_params* p, const void* h, int64_t ld, const int32_t* cu, int32_t batch,
                           int fit_chunks, float2* partial, cudaStream_t st) {
  const int strips = (int)ceil_div(p->d_h, kFitStripCols);
  dim3 grid(strips, fit_chunks, batch), block(kFitTx, kFitTy);
  {
    LaunchScope scope_("fit_partial_kernel", st);
    if (p->h_dtype == GVOTE_DTYPE_F32) {
      fit_partial_kernel<float><<<grid, block, 0, st>>>((const float*)h, ld, cu, p->n_s, p->d_h, fit_chunks, partial);
    } else {
      fit_partial_kernel<__nv_bfloat16><<<grid, block, 0, st>>>((const __nv_bfloat16*)h, ld, cu, p->n_s, p->d_h,
                                                                fit_chunks, partial);
    }
  }
  GVOTE_LAUNCH_CHECK("fit_partial_kernel");
  return GVOTE_OK;
}

int32_t launch_fit(const gvote_params* p, const void* h, int64_t ld, const int32_t* cu, int32_t batch,
                   int fit_chunks, float2* partial, float* mu, float* var, cudaStream_t st) {
  const int32_t rc = launch_fit_partial(p, h, ld, cu, batch, fit_chunks, partial, st);
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
                                int fit_chunks, float2* partial, double* state, cudaStream_t st) {
  gvote_params q = *p;
  q.n_s = 0;                                   // which rows to leave out is the caller's choice here
  const int32_t rc = launch_fit_partial(&q, h, ld, cu, batch, fit_chunks, partial, st);
  if (rc != GVOTE_OK) return rc;
  dim3 g2((unsigned)ceil_div(p->d_h, 32), batch);
  {
    LaunchScope scope_("fit_state_update_kernel", st);
    fit_state_update_kernel<<<g2, 256, 0, st>>>(partial, cu, p->d_h, fit_chunks, state);
  }
  GVOTE_LAUNCH_CHECK("fit_state_update_kernel");
  return GVOTE_OK;
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
  // as many row chunks as fill the GPU, as few as the fixed array holds, at least 32 rows each
  const int64_t strips = ceil_div(p->d_h, kFitStripCols);
  int64_t chunks = 1184 / (strips * batch);
  const int64_t fit_in_array = (int64_t)kStaticFitEntries / per_chunk;
  const int64_t by_rows = ceil_div(max_N > 0 ? max_N : 1, 32);
  if (chunks > fit_in_array) chunks = fit_in_array;
  if (chunks > by_rows) chunks = by_rows;
  if (chunks < 1) chunks = 1;
  float2* scratch = nullptr;
  const int32_t sv = static_scratch_for_current_device(&scratch);
  if (sv != GVOTE_OK) return sv;
  // every entry the merge kernel reads is written by the partial kernel of the same call, so the
  // array needs no clearing between calls
  return launch_fit(p, h, h_row_stride, cu_seqlens, batch, (int)chunks, scratch, mu, var, (cudaStream_t)stream);
}
