// Step 3 of the GVote scheme (Algorithm 1, line 5): S synthetic hidden states per request drawn
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
