// Algorithm 1: the current query Q0, AverageCosSin, and the synthetic queries Q~ = RoPE(H~ W_q, P).
//
// Per request the S+1 rows X = [h_last; H~] are rounded to bf16, multiplied by the stored weight
// W_q [n_q_heads*d_k, d_h] with fp32 accumulation, the bias is added, and each head's d_k-vector
// is rotated with rotate-half RoPE: row 0 with the exact cos/sin of position N-1, rows 1..S with
// the cos/sin averaged over positions N..N+n_f-1.  The result is rounded to bf16, the operand
// type of the score contraction.
#include "common.cuh"

namespace gvote {
namespace {

// ---------------------------------------------------------------------------------- X staging
template <typename T>
__device__ __forceinline__ float to_f32(T v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T>
__global__ void xstage_kernel(const float* __restrict__ H, const T* __restrict__ h_last, int64_t h_last_ld,
                              const int32_t* __restrict__ cu_rows, int d_h, int S,
                              __nv_bfloat16* __restrict__ X) {
  const int r = blockIdx.z, row = blockIdx.y;
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= d_h) return;
  float v;
  if (row == 0) {
    // the current query is the request's last row; a request without rows has none (zeros stand in)
    const bool empty = cu_rows && cu_rows[r + 1] <= cu_rows[r];
    const int64_t src_row = cu_rows ? (int64_t)cu_rows[r + 1] - 1 : (int64_t)r;
    v = empty ? 0.f : to_f32<T>(h_last[src_row * h_last_ld + c]);
  } else {
    v = H[((int64_t)r * S + (row - 1)) * d_h + c];
  }
  X[((int64_t)r * (S + 1) + row) * d_h + c] = __float2bfloat16_rn(v);
}

// ---------------------------------------------------------------------------------- RoPE tables
// table[r][0..3][j] = cos((N-1) w_j), sin((N-1) w_j), mean_i cos((N+i) w_j), mean_i sin((N+i) w_j).
// The means use the closed form of a sum of equally spaced angles:
//   sum_{i<n} e^{i(a + i w)} = e^{i(a + (n-1) w/2)} * sin(n w/2) / sin(w/2).
__global__ void rope_table_kernel(const int32_t* __restrict__ cu, const int32_t* __restrict__ seq_len, int d_k,
                                  double theta, int n_f, float* __restrict__ table) {
  const int r = blockIdx.x, half = d_k / 2;
  for (int j = threadIdx.x; j < half; j += blockDim.x) {
    const double N = seq_len ? (double)seq_len[r] : (double)(cu[r + 1] - cu[r]);   // tokens seen so far
    const double w = pow(theta, -2.0 * (double)j / (double)d_k);
    double s0, c0, sm, cm;
    sincos((N - 1.0) * w, &s0, &c0);
    sincos((N + 0.5 * (double)(n_f - 1)) * w, &sm, &cm);
    const double den = sin(0.5 * w);
    const double ratio = (den != 0.0) ? sin(0.5 * (double)n_f * w) / ((double)n_f * den) : 1.0;
    float* t = table + (int64_t)r * 4 * half;
    t[j] = (float)c0;
    t[half + j] = (float)s0;
    t[2 * half + j] = (float)(ratio * cm);
    t[3 * half + j] = (float)(ratio * sm);
  }
}

// ---------------------------------------------------------------------------------- GEMM (SIMT)
// The tensor-core kernel lives in project_umma.cu; this one takes over when a tensor map cannot be
// built for W_q or X.  out[row][f] = sum_c X[row][c] * W[f][c].  One warp per output feature, kProjRows rows per CTA;
// the X chunk is staged in shared memory and shared by the CTA's warps.
constexpr int kProjWarps = 8;
constexpr int kProjRows = 40;
constexpr int kProjChunk = 256;   // columns per staging step (8 per lane)

__global__ void __launch_bounds__(kProjWarps * 32)
project_simt_kernel(const __nv_bfloat16* __restrict__ X, const __nv_bfloat16* __restrict__ W, int64_t wq_ld,
                    int rows_total, int d_h, int F, float* __restrict__ out) {
  __shared__ __align__(16) __nv_bfloat16 xs[kProjRows][kProjChunk];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int f = blockIdx.x * kProjWarps + warp;
  const int row0 = blockIdx.y * kProjRows;
  const int nrows = min(kProjRows, rows_total - row0);
  float acc[kProjRows];
#pragma unroll
  for (int i = 0; i < kProjRows; ++i) acc[i] = 0.f;

  for (int c0 = 0; c0 < d_h; c0 += kProjChunk) {
    __syncthreads();
    // stage X[row0..row0+nrows)[c0..c0+chunk) ; d_h is a multiple of 8 so 16-byte pieces are whole
    for (int idx = threadIdx.x; idx < nrows * (kProjChunk / 8); idx += blockDim.x) {
      const int rr = idx / (kProjChunk / 8), piece = idx % (kProjChunk / 8);
      const int c = c0 + piece * 8;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (c < d_h) v = *reinterpret_cast<const uint4*>(X + (int64_t)(row0 + rr) * d_h + c);
      *reinterpret_cast<uint4*>(&xs[rr][piece * 8]) = v;
    }
    __syncthreads();
    const int c = c0 + lane * 8;
    if (f < F && c < d_h) {
      const uint4 wv = __ldg(reinterpret_cast<const uint4*>(W + (int64_t)f * wq_ld + c));
      const __nv_bfloat162* w2 = reinterpret_cast<const __nv_bfloat162*>(&wv);
      float wf[8];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 t = __bfloat1622float2(w2[j]);
        wf[2 * j] = t.x; wf[2 * j + 1] = t.y;
      }
#pragma unroll
      for (int i = 0; i < kProjRows; ++i) {
        if (i < nrows) {
          const uint4 xv = *reinterpret_cast<const uint4*>(&xs[i][lane * 8]);
          const __nv_bfloat162* x2 = reinterpret_cast<const __nv_bfloat162*>(&xv);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float2 t = __bfloat1622float2(x2[j]);
            acc[i] = fmaf(t.x, wf[2 * j], acc[i]);
            acc[i] = fmaf(t.y, wf[2 * j + 1], acc[i]);
          }
        }
      }
    }
  }
#pragma unroll
  for (int i = 0; i < kProjRows; ++i) {
    float v = acc[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (lane == 0 && i < nrows && f < F) out[(int64_t)(row0 + i) * F + f] = v;
  }
}

// ---------------------------------------------------------------------------------- finish
// Sum the split-K partials, add the bias, rotate, round to bf16.  Output rows are grouped per KV
// head: first the S synthetic rows of each of its G query heads, then the G current-query rows.
__global__ void project_finish_kernel(const float* __restrict__ qf, int splits, int64_t split_stride,
                                      const float* __restrict__ bias, const float* __restrict__ table, int S,
                                      int Hq, int G, int d_k, __nv_bfloat16* __restrict__ Q) {
  const int r = blockIdx.z, row = blockIdx.y;
  const int half = d_k / 2;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;   // over Hq * half
  if (idx >= Hq * half) return;
  const int g = idx / half, j = idx % half;
  const int F = Hq * d_k;
  const int64_t src = ((int64_t)r * (S + 1) + row) * F + (int64_t)g * d_k;
  float x1 = 0.f, x2 = 0.f;
  for (int s = 0; s < splits; ++s) {
    x1 += qf[s * split_stride + src + j];
    x2 += qf[s * split_stride + src + half + j];
  }
  if (bias) {
    x1 += bias[g * d_k + j];
    x2 += bias[g * d_k + half + j];
  }
  const float* t = table + (int64_t)r * 4 * half + (row == 0 ? 0 : 2 * half);
  const float c = t[j], s = t[half + j];
  const float y1 = x1 * c - x2 * s;
  const float y2 = x2 * c + x1 * s;
  const int kh = g / G, gl = g % G;
  const int grow = (row == 0) ? (G * S + gl) : (gl * S + row - 1);
  __nv_bfloat16* dst = Q + (((int64_t)r * (Hq / G) + kh) * (G * (S + 1)) + grow) * d_k;
  dst[j] = __float2bfloat16_rn(y1);
  dst[half + j] = __float2bfloat16_rn(y2);
}

}  // namespace

int32_t launch_project_umma(const gvote_params* p, const __nv_bfloat16* X, const __nv_bfloat16* W, int64_t wq_ld,
                            int rows_total, int splits, float* part, int32_t* status, cudaStream_t st);

int32_t launch_project_staged(const gvote_params* p, const __nv_bfloat16* X, const float* rope_table, const void* W_q,
                              int64_t wq_ld, const float* b_q, int32_t batch, const WorkspaceMap& m, char* ws,
                              __nv_bfloat16* Q, cudaStream_t st) {
  const int d_h = p->d_h, S = p->S, F = p->n_q_heads * p->d_k;
  const int rows_total = batch * (S + 1);
  float* qf = reinterpret_cast<float*>(ws + m.q_f32);
  int32_t* status = reinterpret_cast<int32_t*>(ws + m.status);

  // tensor-core path; the SIMT kernel serves operands a TMA tensor map cannot describe
  int splits = m.proj_splits;
  const int32_t rc = launch_project_umma(p, X, (const __nv_bfloat16*)W_q, wq_ld, rows_total, splits, qf, status, st);
  if (rc == GVOTE_ERR_UNSUPPORTED_SHAPE) {
    splits = 1;
    dim3 gp((unsigned)ceil_div(F, kProjWarps), (unsigned)ceil_div(rows_total, kProjRows));
    {
      LaunchScope scope_("project_simt_kernel", st);
      project_simt_kernel<<<gp, kProjWarps * 32, 0, st>>>(X, (const __nv_bfloat16*)W_q, wq_ld, rows_total, d_h, F, qf);
    }
    GVOTE_LAUNCH_CHECK("project_simt_kernel");
  } else if (rc != GVOTE_OK) {
    return rc;
  }

  dim3 gf((unsigned)ceil_div((int64_t)p->n_q_heads * (p->d_k / 2), 128), S + 1, batch);
  {
    LaunchScope scope_("project_finish_kernel", st);
    launch_on(project_finish_kernel, gf, dim3(128), 0, st, qf, splits, (int64_t)rows_total * F, b_q, rope_table, S, p->n_q_heads,
                                              p->n_q_heads / p->n_kv_heads, p->d_k, Q);
  }
  GVOTE_LAUNCH_CHECK("project_finish_kernel");
  return GVOTE_OK;
}

int32_t launch_project(const gvote_params* p, const float* H_tilde, const void* h_last, int64_t h_last_ld,
                       const int32_t* h_last_rows_from_cu, const void* W_q, int64_t wq_ld, const float* b_q,
                       const int32_t* cu, int32_t batch, const WorkspaceMap& m, char* ws, __nv_bfloat16* Q,
                       cudaStream_t st, const int32_t* seq_len) {
  const int d_h = p->d_h, S = p->S;
  __nv_bfloat16* X = reinterpret_cast<__nv_bfloat16*>(ws + m.x_bf16);
  float* table = reinterpret_cast<float*>(ws + m.rope);

  dim3 gx((unsigned)ceil_div(d_h, 256), S + 1, batch);
  {
    LaunchScope scope_("xstage_kernel", st);
    if (p->h_dtype == GVOTE_DTYPE_F32)
      xstage_kernel<float><<<gx, 256, 0, st>>>(H_tilde, (const float*)h_last, h_last_ld, h_last_rows_from_cu, d_h, S, X);
    else
      xstage_kernel<__nv_bfloat16><<<gx, 256, 0, st>>>(H_tilde, (const __nv_bfloat16*)h_last, h_last_ld,
                                                       h_last_rows_from_cu, d_h, S, X);
  }
  GVOTE_LAUNCH_CHECK("xstage_kernel");
  {
    LaunchScope scope_("rope_table_kernel", st);
    rope_table_kernel<<<batch, 64, 0, st>>>(cu, seq_len, p->d_k, p->rope_theta, p->n_f, table);
  }
  GVOTE_LAUNCH_CHECK("rope_table_kernel");
  return launch_project_staged(p, X, table, W_q, wq_ld, b_q, batch, m, ws, Q, st);
}

}  // namespace gvote
