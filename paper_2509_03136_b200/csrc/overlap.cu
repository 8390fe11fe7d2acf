// Section 3.3 of the paper judges a set of kept keys by how much of a real query's attention it
// captures.  gvote_overlap applies that yardstick to the pass's own output: for every query head, the
// share of the current query's softmax weights (Eq. 1) that falls on the keys its KV head keeps.
//
// Two small kernels.  overlap_partial_kernel gives each CTA 1024 keys of one query head: it computes the
// logits q.k / sqrt(d_k) in fp32 (four keys per thread), the chunk maximum m, and the chunk's sums of
// exp(l - m) over all keys and over the kept keys.  overlap_merge_kernel rescales the chunks to the row
// maximum and divides: overlap = sum_kept / sum_all.
#include "common.cuh"

namespace gvote {
namespace {

constexpr int kOvThreads = 256;
constexpr int kOvKeys = kOverlapKeys;      // keys per CTA

__global__ void __launch_bounds__(kOvThreads)
overlap_partial_kernel(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K, int64_t k_tok,
                       int64_t k_head, const uint32_t* __restrict__ mask, const int32_t* __restrict__ cu, int Hq,
                       int G, int S, int d_k, float scale, int64_t row_words, int chunks,
                       float4* __restrict__ partial) {
  __shared__ float qf[512];
  __shared__ float red[3][kOvThreads / 32];
  const int r = blockIdx.z, g = blockIdx.y, c = blockIdx.x;
  const int start = cu[r], N = cu[r + 1] - start;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float4* out = partial + ((int64_t)r * Hq + g) * chunks + c;
  const int n0 = c * kOvKeys;
  if (n0 >= N) { if (tid == 0) *out = make_float4(-INFINITY, 0.f, 0.f, 0.f); return; }
  const int kh = g / G, gl = g % G;
  // the current query's row of head g sits after the G*S synthetic rows of its head group
  const __nv_bfloat16* qrow = Q + (((int64_t)r * (Hq / G) + kh) * (G * (S + 1)) + G * S + gl) * d_k;
  for (int i = tid; i < d_k; i += kOvThreads) qf[i] = __bfloat162float(qrow[i]);
  __syncthreads();
  const __nv_bfloat16* krows = K + (int64_t)kh * k_head + (int64_t)start * k_tok;
  const uint32_t* mrow = mask + (int64_t)kh * row_words + mask_word_offset(start, r);
  float l[4];
  bool kept[4];
  float mx = -INFINITY;
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const int n = n0 + u * kOvThreads + tid;
    l[u] = -INFINITY;
    kept[u] = false;
    if (n < N) {
      const uint4* kp = reinterpret_cast<const uint4*>(krows + (int64_t)n * k_tok);
      float acc = 0.f;
      for (int cc = 0; cc < d_k / 8; ++cc) {
        const uint4 v = __ldg(kp + cc);
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float2 f = __bfloat1622float2(h[j]);
          acc = fmaf(qf[cc * 8 + 2 * j], f.x, acc);
          acc = fmaf(qf[cc * 8 + 2 * j + 1], f.y, acc);
        }
      }
      l[u] = acc * scale;
      kept[u] = (mrow[n >> 5] >> (n & 31)) & 1u;
      mx = fmaxf(mx, l[u]);
    }
  }
  mx = warp_max(mx);
  if (lane == 0) red[0][warp] = mx;
  __syncthreads();
  mx = red[0][0];
#pragma unroll
  for (int w = 1; w < kOvThreads / 32; ++w) mx = fmaxf(mx, red[0][w]);
  float s_all = 0.f, s_kept = 0.f;
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const float e = l[u] == -INFINITY ? 0.f : expf(l[u] - mx);
    s_all += e;
    if (kept[u]) s_kept += e;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    s_all += __shfl_xor_sync(0xffffffffu, s_all, o);
    s_kept += __shfl_xor_sync(0xffffffffu, s_kept, o);
  }
  if (lane == 0) { red[1][warp] = s_all; red[2][warp] = s_kept; }
  __syncthreads();
  if (tid == 0) {
    float a = 0.f, k = 0.f;
    for (int w = 0; w < kOvThreads / 32; ++w) { a += red[1][w]; k += red[2][w]; }
    *out = make_float4(mx, a, k, 0.f);
  }
}

__global__ void overlap_merge_kernel(const float4* __restrict__ partial, int Hq, int chunks, float* __restrict__ overlap) {
  const int r = blockIdx.y, g = blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= Hq) return;
  const float4* p = partial + ((int64_t)r * Hq + g) * chunks;
  float M = -INFINITY;
  for (int c = 0; c < chunks; ++c) M = fmaxf(M, p[c].x);
  double all = 0.0, kept = 0.0;
  for (int c = 0; c < chunks; ++c) {
    if (p[c].x == -INFINITY) continue;
    const double w = exp((double)p[c].x - (double)M);
    all += w * (double)p[c].y;
    kept += w * (double)p[c].z;
  }
  overlap[r * Hq + g] = all > 0.0 ? (float)(kept / all) : 0.f;
}

}  // namespace

int32_t launch_overlap(const gvote_params* p, const __nv_bfloat16* Q, const __nv_bfloat16* K, int64_t k_tok,
                       int64_t k_head, const uint32_t* mask, const int32_t* cu, int32_t batch, int64_t max_N,
                       float* overlap, const WorkspaceMap& m, char* ws, cudaStream_t st) {
  const int Hq = p->n_q_heads, G = Hq / p->n_kv_heads;
  const int chunks = (int)ceil_div(max_N > 0 ? max_N : 1, kOvKeys);
  float4* partial = reinterpret_cast<float4*>(ws + m.ov_partial);
  const float scale = (float)(1.0 / sqrt((double)p->d_k));
  dim3 g1((unsigned)chunks, (unsigned)Hq, (unsigned)batch);
  {
    LaunchScope scope_("overlap_partial_kernel", st);
    overlap_partial_kernel<<<g1, kOvThreads, 0, st>>>(Q, K, k_tok, k_head, mask, cu, Hq, G, p->S, p->d_k, scale,
                                                      m.row_words, chunks, partial);
  }
  GVOTE_LAUNCH_CHECK("overlap_partial_kernel");
  dim3 g2((unsigned)ceil_div(Hq, 64), (unsigned)batch);
  {
    LaunchScope scope_("overlap_merge_kernel", st);
    overlap_merge_kernel<<<g2, 64, 0, st>>>(partial, Hq, chunks, overlap);
  }
  GVOTE_LAUNCH_CHECK("overlap_merge_kernel");
  return GVOTE_OK;
}

}  // namespace gvote
