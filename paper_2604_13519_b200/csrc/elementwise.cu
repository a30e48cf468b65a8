// Memory-light kernels of the verify step: embedding gather + RMSNorm, residual add + RMSNorm (which
// also folds the split-K partial sums of the preceding projection), rotary embedding + paged KV
// append, and the acceptance kernel (per-row argmax, longest accepted draft prefix, new lengths).
#include "kernels.h"

namespace ts {

static constexpr int kNormThreads = 256;

__device__ __forceinline__ float block_sum(float v, float *red) {
  v = warp_sum(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  if (l == 0) red[w] = v;
  __syncthreads();
  float t = (l < (int)(blockDim.x >> 5)) ? red[l] : 0.f;
  t = warp_sum(t);
  __syncthreads();
  return t;
}

// One CTA per row.  MODE 0: x = embedding row.  MODE 1: x += sum of partial slabs.
template <int MODE>
__global__ void __launch_bounds__(kNormThreads)
norm_kernel(const int32_t *tokens, const __nv_bfloat16 *embed, const float *part, int n_splits, int part_rows,
            const float *gain, float eps, int d, float *x, __nv_bfloat16 *h, int h_rows, int planes) {
  __shared__ float red[32];
  pdl_wait();
  const int m = blockIdx.x;
  float *xr = x + (size_t)m * d;
  float ss = 0.f;
  for (int c = threadIdx.x * 4; c < d; c += kNormThreads * 4) {
    float4 v;
    if (MODE == 0) {
      const __nv_bfloat16 *e = embed + (size_t)tokens[m] * d + c;
      const uint2 raw = *reinterpret_cast<const uint2 *>(e);
      const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162 *>(&raw.x);
      const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162 *>(&raw.y);
      v = make_float4(__low2float(a), __high2float(a), __low2float(b), __high2float(b));
    } else {
      v = *reinterpret_cast<const float4 *>(xr + c);
      for (int s = 0; s < n_splits; ++s) {
        const float4 p = *reinterpret_cast<const float4 *>(part + ((size_t)s * part_rows + m) * d + c);
        v.x += p.x; v.y += p.y; v.z += p.z; v.w += p.w;
      }
    }
    *reinterpret_cast<float4 *>(xr + c) = v;
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  const float tot = block_sum(ss, red);
  const float r = rsqrtf(tot / (float)d + eps);
  pdl_launch_dependents();
  for (int c = threadIdx.x * 4; c < d; c += kNormThreads * 4) {
    const float4 v = *reinterpret_cast<const float4 *>(xr + c);
    const float4 gn = *reinterpret_cast<const float4 *>(gain + c);
    const float o[4] = {v.x * r * gn.x, v.y * r * gn.y, v.z * r * gn.z, v.w * r * gn.w};
    __nv_bfloat16 hi[4], lo[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) split_bf16(o[j], hi[j], lo[j]);
    *reinterpret_cast<uint2 *>(h + (size_t)m * d + c) = *reinterpret_cast<uint2 *>(hi);
    if (planes == 2) *reinterpret_cast<uint2 *>(h + ((size_t)h_rows + m) * d + c) = *reinterpret_cast<uint2 *>(lo);
  }
}

template <typename K, typename... Args>
static cudaError_t launch_pdl(K kernel, dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

cudaError_t launch_embed_norm(const StepIn &in, const __nv_bfloat16 *embed, const float *gain, float eps,
                              int d, float *x, __nv_bfloat16 *h, int h_rows, int planes, cudaStream_t st) {
  return launch_pdl(norm_kernel<0>, dim3(in.M), dim3(kNormThreads), 0, st, in.tokens, embed,
                    (const float *)nullptr, 0, 0, gain, eps, d, x, h, h_rows, planes);
}

cudaError_t launch_add_norm(int M, int d, const float *part, int n_splits, int part_rows, const float *gain,
                            float eps, float *x, __nv_bfloat16 *h, int h_rows, int planes, cudaStream_t st) {
  return launch_pdl(norm_kernel<1>, dim3(M), dim3(kNormThreads), 0, st, (const int32_t *)nullptr,
                    (const __nv_bfloat16 *)nullptr, part, n_splits, part_rows, gain, eps, d, x, h, h_rows,
                    planes);
}

__device__ __forceinline__ __half to_half_sat(float x) {
  return __float2half_rn(fminf(fmaxf(x, -65504.f), 65504.f));
}

// grid = (M, Hq + 2*Hkv); one CTA of hd/2 threads per (row, head).  Thread i handles the rotary pair
// (i, i + hd/2) of q or k heads, or elements (i, i + hd/2) of a v head.
__global__ void rope_kv_kernel(StepIn in, const float *part, int n_splits, int part_rows, int Hq, int Hkv, int hd,
                               const float2 *rope_tab, __half *q_out, __half *k_pages, __half *v_pages) {
  pdl_wait();
  const int m = blockIdx.x, head = blockIdx.y, i = threadIdx.x, half = hd >> 1;
  const int N = (Hq + 2 * Hkv) * hd;
  const int col = head * hd + i;
  float a = 0.f, b = 0.f;
  for (int s = 0; s < n_splits; ++s) {
    const float *p = part + ((size_t)s * part_rows + m) * N;
    a += p[col];
    b += p[col + half];
  }
  pdl_launch_dependents();
  const int pos = in.pos[m];
  if (head < Hq + Hkv) {
    const float2 cs = rope_tab[(size_t)pos * half + i];
    const float ra = a * cs.x - b * cs.y;
    const float rb = b * cs.x + a * cs.y;
    a = ra; b = rb;
  }
  if (head < Hq) {
    __half *q = q_out + ((size_t)m * Hq + head) * hd;
    q[i] = to_half_sat(a);
    q[i + half] = to_half_sat(b);
  } else {
    const int seq = in.row_seq[m];
    const int page = in.block_tab[(size_t)seq * in.pages_per_seq + (pos >> 4)];
    const bool is_k = head < Hq + Hkv;
    const int kh = is_k ? head - Hq : head - Hq - Hkv;
    __half *dst = (is_k ? k_pages : v_pages) + (((size_t)page * Hkv + kh) * 16 + (pos & 15)) * hd;
    dst[i] = to_half_sat(a);
    dst[i + half] = to_half_sat(b);
  }
}

cudaError_t launch_rope_kv(const StepIn &in, const float *part, int n_splits, int part_rows, int Hq, int Hkv,
                           int hd, const float2 *rope_tab, __half *q_out, __half *k_pages, __half *v_pages,
                           cudaStream_t st) {
  return launch_pdl(rope_kv_kernel, dim3(in.M, Hq + 2 * Hkv), dim3(hd / 2), 0, st, in, part, n_splits,
                    part_rows, Hq, Hkv, hd, rope_tab, q_out, k_pages, v_pages);
}

// One CTA per sequence.  Step 1: every warp reduces the per-tile maxima of some rows to the row's
// argmax (lowest id among equal maxima).  Step 2: thread 0 walks the draft: row j predicted the
// token that row j+1 was fed; the accepted length is the number of leading agreements.
__global__ void __launch_bounds__(256)
accept_kernel(AcceptArgs a) {
  pdl_wait();
  const int seq = blockIdx.x;
  const int r0 = a.in.cu_rows[seq], r1 = a.in.cu_rows[seq + 1];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int r = r0 + warp; r < r1; r += 8) {
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    const float2 *p = a.amax + (size_t)r * a.n_part;
    for (int t = lane; t < a.n_part; t += 32) {
      const float2 e = p[t];
      const int idx = __float_as_int(e.y);
      if (e.x > bv || (e.x == bv && idx < bi)) { bv = e.x; bi = idx; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    if (lane == 0) a.argmax[r] = bi;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const int k = r1 - r0;
    int l = 0;
    while (l < k - 1 && a.argmax[r0 + l] == a.in.tokens[r0 + l + 1]) ++l;
    a.accept_len[seq] = l;
    int32_t *em = a.emitted + (size_t)seq * a.k_max;
    for (int j = 0; j < l; ++j) em[j] = a.in.tokens[r0 + j + 1];
    em[l] = a.argmax[r0 + l];
    a.new_len[seq] = a.in.seq_len[seq] + l + 1;   // rejected rows stay in their pages, uncounted
    a.new_pending[seq] = a.argmax[r0 + l];
  }
}

cudaError_t launch_accept(const AcceptArgs &a, cudaStream_t st) {
  return launch_pdl(accept_kernel, dim3(a.in.B), dim3(256), 0, st, a);
}

}  // namespace ts
