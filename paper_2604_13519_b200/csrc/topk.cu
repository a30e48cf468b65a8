// Row-wise Top-K of a [rows][cols] fp32 matrix (largest value first, lowest column on ties), used for the retrieval
// scores (one row) and for the per-position Top-K of the verify logits that feeds the successor table of the
// Token-Recycling-style drafter.
#include "kernels.h"

namespace ts {

// Selection in two levels, both with the same rule (largest score, lowest index on ties): every CTA of the first
// kernel holds a slice of kSlice scores in shared memory and takes its K best in K rounds; the second kernel (one
// CTA per row) takes the K best of the slices' candidates.  cand: [rows][slices][K] (column as int bits, value)
// pairs; out: [rows][K] pairs.
static constexpr int kSlice = 4096;
static constexpr int kSelThreads = 256;

__device__ __forceinline__ void block_argmax(float &v, int &idx, float *bv, int *bi) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, v, o);
    const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
    if (ov > v || (ov == v && oi < idx)) { v = ov; idx = oi; }
  }
  __syncthreads();
  if (lane == 0) { bv[warp] = v; bi[warp] = idx; }
  __syncthreads();
  v = bv[0]; idx = bi[0];
  for (int w = 1; w < kSelThreads / 32; ++w)
    if (bv[w] > v || (bv[w] == v && bi[w] < idx)) { v = bv[w]; idx = bi[w]; }
}

__global__ void __launch_bounds__(kSelThreads)
topk_slice_kernel(const float *x, int N, int K, float2 *cand) {
  __shared__ float s[kSlice];
  __shared__ float bv[kSelThreads / 32];
  __shared__ int bi[kSelThreads / 32];
  const float *scores = x + (size_t)blockIdx.y * N;          // this CTA's row
  cand += (size_t)blockIdx.y * gridDim.x * K;
  const int base = blockIdx.x * kSlice;
  for (int i = threadIdx.x; i < kSlice; i += blockDim.x) s[i] = base + i < N ? scores[base + i] : -INFINITY;
  __syncthreads();
  for (int j = 0; j < K; ++j) {
    float v = -INFINITY;
    int idx = 0x7FFFFFFF;
    for (int i = threadIdx.x; i < kSlice; i += blockDim.x)
      if (s[i] > v) { v = s[i]; idx = base + i; }        // ascending i: the first of equal scores stays
    block_argmax(v, idx, bv, bi);
    if (threadIdx.x == 0) {
      cand[(size_t)blockIdx.x * K + j] = make_float2(__int_as_float(idx), v);
      if (idx != 0x7FFFFFFF) s[idx - base] = -INFINITY;  // struck out (a slice with fewer than K entries yields -inf pairs)
    }
    __syncthreads();
  }
}

__global__ void __launch_bounds__(kSelThreads)
topk_final_kernel(float2 *cand, int n_cand, int K, float *out) {
  __shared__ float bv[kSelThreads / 32];
  __shared__ int bi[kSelThreads / 32];
  __shared__ int taken_slot;
  cand += (size_t)blockIdx.x * n_cand;
  out += (size_t)blockIdx.x * 2 * K;
  for (int j = 0; j < K; ++j) {
    float v = -INFINITY;
    int idx = 0x7FFFFFFF, slot = -1;
    for (int i = threadIdx.x; i < n_cand; i += blockDim.x) {
      const float2 c = cand[i];
      const int ci = __float_as_int(c.x);
      if (c.y > v || (c.y == v && ci < idx)) { v = c.y; idx = ci; slot = i; }
    }
    const int my_idx = idx;
    block_argmax(v, idx, bv, bi);
    if (my_idx == idx && slot >= 0) taken_slot = slot;   // indices are unique among live candidates
    __syncthreads();
    if (threadIdx.x == 0) {
      out[2 * j] = __int_as_float(idx);
      out[2 * j + 1] = v;
      if (idx != 0x7FFFFFFF) cand[taken_slot] = make_float2(__int_as_float(0x7FFFFFFF), -INFINITY);
    }
    __syncthreads();
  }
}

cudaError_t launch_topk_rows(const float *x, int n_rows, int n_cols, int K, float2 *cand, float *out, cudaStream_t st) {
  if (K < 1 || K > kSlice || n_rows < 1 || n_cols < 1) return cudaErrorInvalidValue;
  const int slices = (n_cols + kSlice - 1) / kSlice;
  topk_slice_kernel<<<dim3(slices, n_rows), kSelThreads, 0, st>>>(x, n_cols, K, cand);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  topk_final_kernel<<<n_rows, kSelThreads, 0, st>>>(cand, slices * K, K, out);
  return cudaGetLastError();
}

}  // namespace ts
