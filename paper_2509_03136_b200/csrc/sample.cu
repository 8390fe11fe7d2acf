// Step 3 of the GVote scheme (Section 3.2; the sampling step of Algorithm 1): S synthetic hidden states per request drawn
// from N(mu, diag(var)).  Randomness is counter based (Philox4x32-10, Salmon et al., SC'11) so
// that any draw can be recomputed from (seed, layer, request, sample, channel) alone: key =
// (seed low word, seed high word), counter = (channel div 4, sample, layer, request); the four
// output words of a block feed channels 4b..4b+3 through two Box-Muller pairs.
#include "common.cuh"

namespace gvote {
namespace {

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                              uint32_t k1, uint32_t out[4]) {
  constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
    const uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += W0; k1 += W1;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// u in (0,1): top 23 bits plus half a step; exact in fp32.
__device__ __forceinline__ float u01(uint32_t x) { return ((float)(x >> 9) + 0.5f) * 1.1920928955078125e-07f; }

__device__ __forceinline__ void box_muller(uint32_t xa, uint32_t xb, float& z0, float& z1) {
  const float r = sqrtf(-2.0f * logf(u01(xa)));
  float s, c;
  sincospif(2.0f * u01(xb), &s, &c);
  z0 = r * c;
  z1 = r * s;
}

__global__ void sample_kernel(const float* __restrict__ mu, const float* __restrict__ var, int d_h, int S,
                              uint32_t k0, uint32_t k1, uint32_t layer, float* __restrict__ H,
                              uint32_t* __restrict__ raw) {
  const int r = blockIdx.z, s = blockIdx.y;
  const int blk = blockIdx.x * blockDim.x + threadIdx.x;   // block of 4 channels
  const int c = blk * 4;
  if (c >= d_h) return;
  uint32_t w[4];
  philox4x32_10((uint32_t)blk, (uint32_t)s, layer, (uint32_t)r, k0, k1, w);
  float z[4];
  box_muller(w[0], w[1], z[0], z[1]);
  box_muller(w[2], w[3], z[2], z[3]);
  const int64_t o = ((int64_t)r * S + s) * d_h + c;
  const float* m = mu + (int64_t)r * d_h + c;
  const float* v = var + (int64_t)r * d_h + c;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    if (c + j < d_h) {
      H[o + j] = fmaf(sqrtf(v[j]), z[j], m[j]);
      if (raw) raw[o + j] = w[j];
    }
  }
}


// ---------------------------------------------------------------------------------- fused middle of the pass
// One launch between the fit's streaming kernel and the projection: a CTA owns 32 channels of one
// request.  (1) Eight lanes per channel merge the fit's per-chunk moments into mu and var.  (2) The
// S draws of those channels are made exactly as in sample_kernel and go straight to the bf16 rows
// 1..S of the projection input X; row 0 is the current query's hidden state.  (3) The first CTA of a
// request also fills its RoPE table: cos/sin at position N-1 and their means over positions
// N..N+n_f-1, by the closed form of a sum of equally spaced angles,
//   sum_{i<n} e^{i(a + i w)} = e^{i(a + (n-1) w/2)} * sin(n w/2) / sin(w/2).
template <typename T>
__global__ void __launch_bounds__(256)
prep_kernel(const float2* __restrict__ partial, int chunks, const T* __restrict__ h_last, int64_t h_last_ld,
            const int32_t* __restrict__ cu_rows, const int32_t* __restrict__ cu, int n_s, int d_h, int S, int d_k,
            double theta, int n_f, uint32_t k0, uint32_t k1, uint32_t layer, float* __restrict__ mu,
            float* __restrict__ var, __nv_bfloat16* __restrict__ X, float* __restrict__ table) {
  __shared__ FitMoments sm[8][32];
  __shared__ float s_mu[32], s_sd[32];
  const int r = blockIdx.y;
  const int tid = threadIdx.x, tx = tid & 31, ty = tid >> 5;
  const int col0 = blockIdx.x * 32, col = col0 + tx;
  const int first = cu[r] + n_s, last = cu[r + 1];

  FitMoments acc{0.0, 0.0, 0.0};
  double ref = 0.0;
  if (col < d_h) {
    ref = (double)partial[((int64_t)r * chunks) * d_h + col].x;
    acc = fit_merge_lane(partial, r, chunks, d_h, col, first, last, ty, 8, ref);
  }
  sm[ty][tx] = acc;
  __syncthreads();
  if (ty == 0) {
    float m = 0.f, v = 0.f;
    if (col < d_h) {
      for (int j = 1; j < 8; ++j) { acc.n += sm[j][tx].n; acc.a += sm[j][tx].a; acc.bc += sm[j][tx].bc; }
      fit_merge_finish(acc, ref, m, v);
      mu[(int64_t)r * d_h + col] = m;
      var[(int64_t)r * d_h + col] = v;
      // the current query is the request's last row; a request without rows has none (zeros stand in)
      const bool empty = cu_rows && cu_rows[r + 1] <= cu_rows[r];
      const int64_t src_row = cu_rows ? (int64_t)cu_rows[r + 1] - 1 : (int64_t)r;
      float x0;
      if (empty) x0 = 0.f;
      else if (sizeof(T) == 4) x0 = reinterpret_cast<const float*>(h_last)[src_row * h_last_ld + col];
      else x0 = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(h_last)[src_row * h_last_ld + col]);
      X[((int64_t)r * (S + 1)) * d_h + col] = __float2bfloat16_rn(x0);
    }
    s_mu[tx] = m;
    s_sd[tx] = sqrtf(v);
  }
  __syncthreads();

  // eight Philox blocks (4 channels each) x 32 samples per sweep
  const int blk = tid & 7, c = col0 + blk * 4;
  if (c < d_h) {
    for (int s = tid >> 3; s < S; s += 32) {
      uint32_t w[4];
      philox4x32_10((uint32_t)(c >> 2), (uint32_t)s, layer, (uint32_t)r, k0, k1, w);
      float z[4];
      box_muller(w[0], w[1], z[0], z[1]);
      box_muller(w[2], w[3], z[2], z[3]);
      __nv_bfloat162 lo, hi;
      lo.x = __float2bfloat16_rn(fmaf(s_sd[blk * 4 + 0], z[0], s_mu[blk * 4 + 0]));
      lo.y = __float2bfloat16_rn(fmaf(s_sd[blk * 4 + 1], z[1], s_mu[blk * 4 + 1]));
      hi.x = __float2bfloat16_rn(fmaf(s_sd[blk * 4 + 2], z[2], s_mu[blk * 4 + 2]));
      hi.y = __float2bfloat16_rn(fmaf(s_sd[blk * 4 + 3], z[3], s_mu[blk * 4 + 3]));
      uint2 pk;
      pk.x = *reinterpret_cast<uint32_t*>(&lo);
      pk.y = *reinterpret_cast<uint32_t*>(&hi);
      *reinterpret_cast<uint2*>(X + ((int64_t)r * (S + 1) + 1 + s) * d_h + c) = pk;
    }
  }

  if (blockIdx.x == 0) {
    const int half = d_k / 2;
    const double N = (double)(cu[r + 1] - cu[r]);
    for (int j = tid; j < half; j += blockDim.x) {
      const double w = pow(theta, -2.0 * (double)j / (double)d_k);
      double s0, c0, sm_, cm_;
      sincos((N - 1.0) * w, &s0, &c0);
      sincos((N + 0.5 * (double)(n_f - 1)) * w, &sm_, &cm_);
      const double den = sin(0.5 * w);
      const double ratio = (den != 0.0) ? sin(0.5 * (double)n_f * w) / ((double)n_f * den) : 1.0;
      float* t = table + (int64_t)r * 4 * half;
      t[j] = (float)c0;
      t[half + j] = (float)s0;
      t[2 * half + j] = (float)(ratio * cm_);
      t[3 * half + j] = (float)(ratio * sm_);
    }
  }
}

}  // namespace

int32_t launch_sample(const gvote_params* p, const float* mu, const float* var, int32_t batch, float* H_tilde,
                      uint32_t* raw, cudaStream_t st) {
  const int blocks4 = (int)ceil_div(p->d_h, 4);
  dim3 grid((unsigned)ceil_div(blocks4, 128), p->S, batch);
  {
    LaunchScope scope_("sample_kernel", st);
  sample_kernel<<<grid, 128, 0, st>>>(mu, var, p->d_h, p->S, (uint32_t)(p->seed & 0xffffffffu),
                                      (uint32_t)(p->seed >> 32), p->layer_id, H_tilde, raw);
  }
  GVOTE_LAUNCH_CHECK("sample_kernel");
  return GVOTE_OK;
}

}  // namespace gvote

namespace gvote {

int32_t launch_prep(const gvote_params* p, const float2* partial, int fit_chunks, const void* h_last,
                    int64_t h_last_ld, const int32_t* h_last_rows_from_cu, const int32_t* cu, int32_t batch,
                    float* mu, float* var, __nv_bfloat16* X, float* rope_table, cudaStream_t st) {
  dim3 grid((unsigned)ceil_div(p->d_h, 32), (unsigned)batch);
  const uint32_t k0 = (uint32_t)(p->seed & 0xffffffffu), k1 = (uint32_t)(p->seed >> 32);
  {
    LaunchScope scope_("prep_kernel", st);
    if (p->h_dtype == GVOTE_DTYPE_F32)
      launch_on(prep_kernel<float>, grid, dim3(256), 0, st, partial, fit_chunks, (const float*)h_last, h_last_ld,
                                               h_last_rows_from_cu, cu, p->n_s, p->d_h, p->S, p->d_k, p->rope_theta,
                                               p->n_f, k0, k1, p->layer_id, mu, var, X, rope_table);
    else
      launch_on(prep_kernel<__nv_bfloat16>, grid, dim3(256), 0, st, partial, fit_chunks, (const __nv_bfloat16*)h_last, h_last_ld,
                                                       h_last_rows_from_cu, cu, p->n_s, p->d_h, p->S, p->d_k,
                                                       p->rope_theta, p->n_f, k0, k1, p->layer_id, mu, var, X,
                                                       rope_table);
  }
  GVOTE_LAUNCH_CHECK("prep_kernel");
  return GVOTE_OK;
}

}  // namespace gvote
