// Top-K retrieval over the datastore's hidden states (Section 4.3, Eq. 3): sim = cosine similarity between the
// query's hidden state and each historical invocation's, the K most similar entries become the candidates of
// the suffix match.
//
// cosine_scores_kernel: one warp per datastore entry, 16-byte loads of its bf16 row, fp32 dot product and squared
// norm, the query in shared memory: one pass over N x d x 2 bytes, bound by HBM.
// The K best scores are then taken by the row Top-K kernels (topk.cu).
#include "kernels.h"

namespace ts {

static constexpr int kCosThreads = 256;
static constexpr int kCosRowsPerWarp = 8;     // the query is staged once per CTA for 64 entries

// q_dev != nullptr: the query as fp32 [d]; else the bf16 (hi[, lo]) planes of a row of the last step's hidden state
__global__ void __launch_bounds__(kCosThreads)
cosine_scores_kernel(const __nv_bfloat16 *H, int N, int d, const float *q_dev, const __nv_bfloat16 *q_planes,
                     int plane_stride, int planes, float *scores) {
  extern __shared__ float q[];
  __shared__ float red[kCosThreads / 32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float qq = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    float v;
    if (q_dev) v = q_dev[i];
    else v = __bfloat162float(q_planes[i]) + (planes == 2 ? __bfloat162float(q_planes[plane_stride + i]) : 0.f);
    q[i] = v;
    qq += v * v;
  }
  qq = warp_sum(qq);
  if (lane == 0) red[warp] = qq;
  __syncthreads();
  qq = 0.f;
  for (int w = 0; w < kCosThreads / 32; ++w) qq += red[w];
  for (int r = 0; r < kCosRowsPerWarp; ++r) {
    const int e = (blockIdx.x * kCosRowsPerWarp + r) * (kCosThreads / 32) + warp;
    if (e >= N) return;
    const uint4 *row = reinterpret_cast<const uint4 *>(H + (size_t)e * d);   // 8 bf16 per load; d is a multiple of 8
    float dot = 0.f, hh = 0.f;
    for (int c = lane; c < d / 8; c += 32) {
      const uint4 raw = __ldcs(row + c);                                     // streamed once
      const __nv_bfloat162 *p = reinterpret_cast<const __nv_bfloat162 *>(&raw);
      const float4 q0 = *reinterpret_cast<const float4 *>(q + c * 8), q1 = *reinterpret_cast<const float4 *>(q + c * 8 + 4);
      const float a0 = __low2float(p[0]), b0 = __high2float(p[0]), a1 = __low2float(p[1]), b1 = __high2float(p[1]);
      const float a2 = __low2float(p[2]), b2 = __high2float(p[2]), a3 = __low2float(p[3]), b3 = __high2float(p[3]);
      dot += a0 * q0.x + b0 * q0.y + a1 * q0.z + b1 * q0.w + a2 * q1.x + b2 * q1.y + a3 * q1.z + b3 * q1.w;
      hh += a0 * a0 + b0 * b0 + a1 * a1 + b1 * b1 + a2 * a2 + b2 * b2 + a3 * a3 + b3 * b3;
    }
    dot = warp_sum(dot);
    hh = warp_sum(hh);
    if (lane == 0) scores[e] = (hh > 0.f && qq > 0.f) ? dot * rsqrtf(hh) * rsqrtf(qq) : -2.f;   // a zero vector ranks last
  }
}

cudaError_t launch_topk_cosine(const __nv_bfloat16 *H, int N, int d, const float *q_dev, const __nv_bfloat16 *q_planes,
                               int plane_stride, int planes, int K, float *scores, cudaStream_t st) {
  static PerDeviceOnce once;
  int dev_ = -1;
  if (once.needed(&dev_)) {
    cudaError_t e = cudaFuncSetAttribute(cosine_scores_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
    if (e != cudaSuccess) return e;
    once.done(dev_);
  }
  const int per = kCosThreads / 32 * kCosRowsPerWarp;
  cosine_scores_kernel<<<(N + per - 1) / per, kCosThreads, (size_t)d * 4, st>>>(H, N, d, q_dev, q_planes, plane_stride,
                                                                                planes, scores);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  // candidates live behind the K result pairs: scores[N + 2K ...], 2 floats per candidate
  float2 *cand = reinterpret_cast<float2 *>(scores + N + 2 * K + ((N + 2 * K) & 1));
  return launch_topk_rows(scores, 1, N, K, cand, scores + N, st);
}

}  // namespace ts
