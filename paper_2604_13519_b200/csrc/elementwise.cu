// Memory-light kernels of the verify step: embedding gather + RMSNorm, residual add + RMSNorm (which
// also folds the split-K partial sums of the preceding projection), rotary embedding + paged KV
// append, and the acceptance kernel (per-row argmax, longest accepted draft prefix, new lengths).
#include <algorithm>

#include "kernels.h"

namespace ts {

static constexpr int kNormMaxThreads = 1024;
static constexpr int kNormMaxSplits = 12;   // split-K slabs folded in one pass (the GEMM launcher's cap)

__device__ __forceinline__ float block_sum(float v, float *red) {
  v = warp_sum(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  if (l == 0) red[w] = v;
  __syncthreads();
  float t = (l < (int)((blockDim.x + 31) >> 5)) ? red[l] : 0.f;
  t = warp_sum(t);
  __syncthreads();
  return t;
}

// One CTA per row.  MODE 0: x = embedding row (and the row's argmax slot is cleared for the LM-head epilogue).
// MODE 1: x += sum of the split-K partial slabs of the preceding projection.  Then h = x * rsqrt(mean(x^2) + eps) * g
// as bf16 (hi[, lo]) planes.  A thread owns one float4 of the row (d / 4 threads; wider rows loop), issues the loads it
// needs together -- the gain before the dependency wait, the residual and the slabs after it -- and keeps its sum in
// registers across the block reduction, so that nothing is read back.  (Spreading a row over a cluster of CTAs with
// the sums of squares exchanged through distributed shared memory was measured and is not faster: the kernel's time
// is the latency of its first access after the wait and of its exit, not the bytes one SM pulls from L2.)
template <int MODE>
__global__ void __launch_bounds__(kNormMaxThreads)
norm_kernel(const int32_t *tokens, const __nv_bfloat16 *embed, const float *part, int n_splits, int part_rows,
            const float *gain, float eps, int d, float *x, __nv_bfloat16 *h, int h_rows, int planes,
            unsigned long long *amax, unsigned long long *stamp, BoundsCheck bc) {
  __shared__ float red[32];
  if (threadIdx.x == 0) stamp_min(stamp);
  pdl_launch_dependents();   // the dependent kernel waits for this one's end before touching its data
  const int m = blockIdx.x;
  const int c0 = threadIdx.x * 4;
  const bool one_pass = d <= (int)blockDim.x * 4;   // the whole row lives in the CTA's registers
  float4 gn = make_float4(0.f, 0.f, 0.f, 0.f);
  if (c0 < d) gn = *reinterpret_cast<const float4 *>(gain + c0);   // (weights do not depend on the previous kernel)
  pdl_wait();
  if (threadIdx.x == 0) stamp_waited(stamp);
  float *xr = x + (size_t)m * d;
  float ss = 0.f;
  float4 keep = make_float4(0.f, 0.f, 0.f, 0.f);
  if (MODE == 0 && threadIdx.x == 0) amax[m] = 0ull;
  for (int c = c0; c < d; c += blockDim.x * 4) {
    float4 v;
    if (MODE == 0) {
      const int tok = tokens[m];
      const __nv_bfloat16 *e = embed + (size_t)(ts_in_range(bc, CHK_TOKEN, tok, bc.vocab) ? tok : 0) * d + c;
      const uint2 raw = *reinterpret_cast<const uint2 *>(e);
      const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162 *>(&raw.x);
      const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162 *>(&raw.y);
      v = make_float4(__low2float(a), __high2float(a), __low2float(b), __high2float(b));
    } else {
      // all loads first (a 1024-thread CTA has 64 registers per thread: nine slabs -- what the projections of the
      // large shapes use -- and the residual fit; further slabs take a second round), then the sum in slab order
      constexpr int kFirst = 9;
      float4 p[kFirst];
      v = *reinterpret_cast<const float4 *>(xr + c);
#pragma unroll
      for (int s = 0; s < kFirst; ++s)
        if (s < n_splits) p[s] = *reinterpret_cast<const float4 *>(part + ((size_t)s * part_rows + m) * d + c);
#pragma unroll
      for (int s = 0; s < kFirst; ++s)
        if (s < n_splits) { v.x += p[s].x; v.y += p[s].y; v.z += p[s].z; v.w += p[s].w; }
      if (n_splits > kFirst) {
#pragma unroll
        for (int s = kFirst; s < kNormMaxSplits; ++s)
          if (s < n_splits) p[s - kFirst] = *reinterpret_cast<const float4 *>(part + ((size_t)s * part_rows + m) * d + c);
#pragma unroll
        for (int s = kFirst; s < kNormMaxSplits; ++s)
          if (s < n_splits) { v.x += p[s - kFirst].x; v.y += p[s - kFirst].y; v.z += p[s - kFirst].z; v.w += p[s - kFirst].w; }
      }
    }
    *reinterpret_cast<float4 *>(xr + c) = v;
    keep = v;
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  const float tot = block_sum(ss, red);
  const float r = rsqrtf(tot / (float)d + eps);
  for (int c = c0; c < d; c += blockDim.x * 4) {
    float4 v = keep, gg = gn;
    if (!one_pass) {
      v = *reinterpret_cast<const float4 *>(xr + c);
      gg = *reinterpret_cast<const float4 *>(gain + c);
    }
    const float o[4] = {v.x * r * gg.x, v.y * r * gg.y, v.z * r * gg.z, v.w * r * gg.w};
    __nv_bfloat16 hi[4], lo[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) split_bf16(o[j], hi[j], lo[j]);
    *reinterpret_cast<uint2 *>(h + (size_t)m * d + c) = *reinterpret_cast<uint2 *>(hi);
    if (planes == 2) *reinterpret_cast<uint2 *>(h + ((size_t)h_rows + m) * d + c) = *reinterpret_cast<uint2 *>(lo);
  }
  if (stamp) { __syncthreads(); if (threadIdx.x == 0) stamp_max(stamp + 3); }
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

static int norm_threads(int d) { return std::min(kNormMaxThreads, (d / 4 + 31) / 32 * 32); }

cudaError_t launch_embed_norm(const StepIn &in, const __nv_bfloat16 *embed, const float *gain, float eps,
                              int d, float *x, __nv_bfloat16 *h, int h_rows, int planes,
                              unsigned long long *amax, cudaStream_t st) {
  return launch_pdl(norm_kernel<0>, dim3(in.M), dim3(norm_threads(d)), 0, st, in.tokens, embed,
                    (const float *)nullptr, 0, 0, gain, eps, d, x, h, h_rows, planes, amax, (unsigned long long *)nullptr, in.ck);
}

cudaError_t launch_add_norm(int M, int d, const float *part, int n_splits, int part_rows, const float *gain,
                            float eps, float *x, __nv_bfloat16 *h, int h_rows, int planes, cudaStream_t st,
                            unsigned long long *stamp) {
  if (n_splits > kNormMaxSplits) return cudaErrorInvalidValue;
  return launch_pdl(norm_kernel<1>, dim3(M), dim3(norm_threads(d)), 0, st, (const int32_t *)nullptr,
                    (const __nv_bfloat16 *)nullptr, part, n_splits, part_rows, gain, eps, d, x, h, h_rows,
                    planes, (unsigned long long *)nullptr, stamp, BoundsCheck{});
}

__device__ __forceinline__ __half to_half_sat(float x) {
  return __float2half_rn(fminf(fmaxf(x, -65504.f), 65504.f));
}

static constexpr int kRopeWideRows = 128;   // steps of at least this many rows take the wide kernel (no faster below)

// grid = (M, Hq + 2*Hkv); one CTA of hd/2 threads per (row, head).  Thread i handles the rotary pair
// (i, i + hd/2) of q or k heads, or elements (i, i + hd/2) of a v head.  Every load is issued before the first use
// (the slabs, the row's position, sequence and slot): the kernel is two round trips to L2, not one per slab.
__global__ void rope_kv_kernel(StepIn in, const float *part, int n_splits, int part_rows, int Hq, int Hkv, int hd,
                               const float2 *rope_tab, __half *q_out, __half *q_lo_out, __half *k_pages, __half *v_pages,
                               unsigned long long *stamp) {
  if (threadIdx.x == 0) stamp_min(stamp);
  pdl_launch_dependents();   // the dependent kernel waits for this one's end before touching its data
  const int m = blockIdx.x, head = blockIdx.y, i = threadIdx.x, half = hd >> 1;
  const int N = (Hq + 2 * Hkv) * hd;
  // the step's integer inputs were copied in before the step's first kernel: they may be read before the wait
  const int pos = in.pos[m], seq = in.row_seq[m], slot = in.slot[m];
  const int page = (head >= Hq) ? in.block_tab[(size_t)seq * in.pages_per_seq + (slot >> 4)] : 0;
  const bool pos_ok = ts_in_range(in.ck, CHK_POSITION, pos, in.ck.max_ctx);
  const bool page_ok = ts_in_range(in.ck, CHK_PAGE_APPEND, page, in.ck.max_pages);
  float2 cs = make_float2(1.f, 0.f);
  if (head < Hq + Hkv && pos_ok) cs = rope_tab[(size_t)pos * half + i];
  pdl_wait();
  if (threadIdx.x == 0) stamp_waited(stamp);
  // the QKV weight rows are stored with rotary partners adjacent: feature 2i = element i, 2i+1 = element i + hd/2
  const int col = head * hd + 2 * i;
  float2 p[kNormMaxSplits];
#pragma unroll
  for (int s = 0; s < kNormMaxSplits; ++s)
    if (s < n_splits) p[s] = *reinterpret_cast<const float2 *>(part + ((size_t)s * part_rows + m) * N + col);
  float a = 0.f, b = 0.f;
#pragma unroll
  for (int s = 0; s < kNormMaxSplits; ++s)
    if (s < n_splits) { a += p[s].x; b += p[s].y; }
  if (head < Hq + Hkv) {
    const float ra = a * cs.x - b * cs.y;
    const float rb = b * cs.x + a * cs.y;
    a = ra; b = rb;
  }
  if (head < Hq) {
    // the query as an fp16 pair (value, rounding remainder): the score product adds both, so the 11 bits of fp16
    // do not limit the scores (the remainder of a saturated value is dropped)
    const size_t qo = ((size_t)m * Hq + head) * hd;
    const __half ha = to_half_sat(a), hb = to_half_sat(b);
    q_out[qo + i] = ha;
    q_out[qo + i + half] = hb;
    if (q_lo_out) {
      q_lo_out[qo + i] = __float2half_rn(fabsf(a) <= 65504.f ? a - __half2float(ha) : 0.f);
      q_lo_out[qo + i + half] = __float2half_rn(fabsf(b) <= 65504.f ? b - __half2float(hb) : 0.f);
    }
  } else if (page_ok) {
    const bool is_k = head < Hq + Hkv;
    const int kh = is_k ? head - Hq : head - Hq - Hkv;
    __half *dst = (is_k ? k_pages : v_pages) + (((size_t)page * Hkv + kh) * 16 + (slot & 15)) * hd;
    dst[i] = to_half_sat(a);
    dst[i + half] = to_half_sat(b);
  }
  if (threadIdx.x == 0) stamp_max(stamp ? stamp + 3 : nullptr);
}

// The same for steps of many rows: grid = (M, ceil(heads / 16)), block = (hd / 8, 16): a thread handles FOUR
// neighbouring rotary pairs of one head (32 bytes per slab in one load, 8-byte stores), so a 256-row step is 768 CTAs
// of 256 threads instead of 12 288 CTAs of 64 -- less than one wave of resident threads instead of nearly three.  The
// sums are taken in the same order as above: the results are the same bits.
__global__ void rope_kv_wide_kernel(StepIn in, const float *part, int n_splits, int part_rows, int Hq, int Hkv, int hd,
                                    const float2 *rope_tab, __half *q_out, __half *q_lo_out, __half *k_pages,
                                    __half *v_pages, unsigned long long *stamp) {
  if (threadIdx.x == 0 && threadIdx.y == 0) stamp_min(stamp);
  pdl_launch_dependents();   // the dependent kernel waits for this one's end before touching its data
  const int m = blockIdx.x, head = blockIdx.y * blockDim.y + threadIdx.y, i0 = 4 * threadIdx.x, half = hd >> 1;
  const int n_heads = Hq + 2 * Hkv, N = n_heads * hd;
  const bool live = head < n_heads;
  // the step's integer inputs were copied in before the step's first kernel: they may be read before the wait
  const int pos = in.pos[m], seq = in.row_seq[m], slot = in.slot[m];
  const int page = (live && head >= Hq) ? in.block_tab[(size_t)seq * in.pages_per_seq + (slot >> 4)] : 0;
  const bool pos_ok = ts_in_range(in.ck, CHK_POSITION, pos, in.ck.max_ctx);
  const bool page_ok = ts_in_range(in.ck, CHK_PAGE_APPEND, page, in.ck.max_pages);
  float2 cs[4] = {make_float2(1.f, 0.f), make_float2(1.f, 0.f), make_float2(1.f, 0.f), make_float2(1.f, 0.f)};
  if (live && head < Hq + Hkv && pos_ok) {
    const float4 *t = reinterpret_cast<const float4 *>(rope_tab + (size_t)pos * half + i0);
    const float4 t0 = t[0], t1 = t[1];
    cs[0] = make_float2(t0.x, t0.y); cs[1] = make_float2(t0.z, t0.w);
    cs[2] = make_float2(t1.x, t1.y); cs[3] = make_float2(t1.z, t1.w);
  }
  pdl_wait();
  if (threadIdx.x == 0 && threadIdx.y == 0) stamp_waited(stamp);
  if (live) {
    // the QKV weight rows are stored with rotary partners adjacent: feature 2i = element i, 2i+1 = element i + hd/2
    const int col = head * hd + 2 * i0;
    float4 p[kNormMaxSplits][2];
#pragma unroll
    for (int s = 0; s < kNormMaxSplits; ++s)
      if (s < n_splits) {
        const float4 *src = reinterpret_cast<const float4 *>(part + ((size_t)s * part_rows + m) * N + col);
        p[s][0] = src[0];
        p[s][1] = src[1];
      }
    float a[4] = {0.f, 0.f, 0.f, 0.f}, b[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int s = 0; s < kNormMaxSplits; ++s)
      if (s < n_splits) {
        a[0] += p[s][0].x; b[0] += p[s][0].y; a[1] += p[s][0].z; b[1] += p[s][0].w;
        a[2] += p[s][1].x; b[2] += p[s][1].y; a[3] += p[s][1].z; b[3] += p[s][1].w;
      }
    if (head < Hq + Hkv) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float ra = a[j] * cs[j].x - b[j] * cs[j].y;
        const float rb = b[j] * cs[j].x + a[j] * cs[j].y;
        a[j] = ra; b[j] = rb;
      }
    }
    __align__(8) __half ha[4], hb[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) { ha[j] = to_half_sat(a[j]); hb[j] = to_half_sat(b[j]); }
    if (head < Hq) {
      // the query as an fp16 pair (value, rounding remainder), as in rope_kv_kernel
      const size_t qo = ((size_t)m * Hq + head) * hd + i0;
      *reinterpret_cast<uint2 *>(q_out + qo) = *reinterpret_cast<const uint2 *>(ha);
      *reinterpret_cast<uint2 *>(q_out + qo + half) = *reinterpret_cast<const uint2 *>(hb);
      if (q_lo_out) {
        __align__(8) __half la[4], lb[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          la[j] = __float2half_rn(fabsf(a[j]) <= 65504.f ? a[j] - __half2float(ha[j]) : 0.f);
          lb[j] = __float2half_rn(fabsf(b[j]) <= 65504.f ? b[j] - __half2float(hb[j]) : 0.f);
        }
        *reinterpret_cast<uint2 *>(q_lo_out + qo) = *reinterpret_cast<const uint2 *>(la);
        *reinterpret_cast<uint2 *>(q_lo_out + qo + half) = *reinterpret_cast<const uint2 *>(lb);
      }
    } else if (page_ok) {
      const bool is_k = head < Hq + Hkv;
      const int kh = is_k ? head - Hq : head - Hq - Hkv;
      __half *dst = (is_k ? k_pages : v_pages) + (((size_t)page * Hkv + kh) * 16 + (slot & 15)) * hd + i0;
      *reinterpret_cast<uint2 *>(dst) = *reinterpret_cast<const uint2 *>(ha);
      *reinterpret_cast<uint2 *>(dst + half) = *reinterpret_cast<const uint2 *>(hb);
    }
  }
  if (threadIdx.x == 0 && threadIdx.y == 0) stamp_max(stamp ? stamp + 3 : nullptr);
}

cudaError_t launch_rope_kv(const StepIn &in, const float *part, int n_splits, int part_rows, int Hq, int Hkv,
                           int hd, const float2 *rope_tab, __half *q_out, __half *q_lo_out, __half *k_pages,
                           __half *v_pages, cudaStream_t st, unsigned long long *stamp) {
  if (in.M >= kRopeWideRows && hd % 8 == 0)
    return launch_pdl(rope_kv_wide_kernel, dim3(in.M, (Hq + 2 * Hkv + 15) / 16), dim3(hd / 8, 16), 0, st, in, part,
                      n_splits, part_rows, Hq, Hkv, hd, rope_tab, q_out, q_lo_out, k_pages, v_pages, stamp);
  return launch_pdl(rope_kv_kernel, dim3(in.M, Hq + 2 * Hkv), dim3(hd / 2), 0, st, in, part, n_splits,
                    part_rows, Hq, Hkv, hd, rope_tab, q_out, q_lo_out, k_pages, v_pages, stamp);
}

// One CTA per source row; thread i moves 16 bytes.  Block (tile, kb) of the stored matrix starts at row
// w_block(tile, kb) * 128 of a [.][64] array.
__global__ void retile_kernel(const __nv_bfloat16 *src, int r0, int K, RowMap rm, __nv_bfloat16 *dst) {
  const int r = r0 + blockIdx.x;
  int row;
  if (rm.hd) {
    const int e = r % rm.hd, half = rm.hd >> 1;
    row = rm.base + (r / rm.hd) * rm.hd + (e < half ? 2 * e : 2 * (e - half) + 1);
  } else {
    row = rm.base + r * rm.mul;
  }
  const int tile = row >> 7, rr = row & 127, KB = K >> 6;
  const uint4 *s = reinterpret_cast<const uint4 *>(src + (size_t)blockIdx.x * K);
  for (int i = threadIdx.x; i < K / 8; i += blockDim.x) {
    const int kb = i >> 3, c = i & 7;
    uint4 *d = reinterpret_cast<uint4 *>(dst + ((size_t)w_block(tile, kb, rm.tiles, KB) * 128 + rr) * 64) + c;
    *d = s[i];
  }
}

cudaError_t launch_retile(const __nv_bfloat16 *src, int n_rows, int r0, int K, RowMap rm, __nv_bfloat16 *dst,
                          cudaStream_t st) {
  if (n_rows <= 0) return cudaSuccess;
  retile_kernel<<<n_rows, 256, 0, st>>>(src, r0, K, rm, dst);
  return cudaGetLastError();
}

// One CTA per sequence.  Each row's argmax was reduced by the LM-head epilogue into a packed
// (ordered value bits, ~token id) word, so the largest word is the largest logit with the lowest id.
// Thread 0 then walks the draft from the root: at row u the model predicted t_u; the walk moves to the
// lowest-numbered child of u that was fed t_u and stops when there is none.  In a chain (parent of row j
// = j - 1) this is the number of leading agreements between the drafts and the predictions.
__global__ void __launch_bounds__(64)
accept_kernel(AcceptArgs a) {
  pdl_launch_dependents();   // the dependent kernel waits for this one's end before touching its data
  pdl_wait();
  const int seq = blockIdx.x;
  const int r0 = a.in.cu_rows[seq], r1 = a.in.cu_rows[seq + 1];
  for (int r = r0 + threadIdx.x; r < r1; r += blockDim.x) {
    a.argmax[r] = (int32_t)(0xFFFFFFFFu - (uint32_t)(a.amax[r] & 0xFFFFFFFFull));
    // (a row's parent precedes it in its chunk; -1 marks the root)
    ts_in_range(a.in.ck, CHK_PARENT, (long long)a.in.parent[r] + 1, r - r0 + 1);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const int k = r1 - r0;
    int32_t *em = a.emitted + (size_t)seq * a.k_max;
    int32_t *path = a.path + (size_t)seq * a.k_max;
    int l = 0, u = 0;
    path[0] = 0;
    for (;;) {
      const int32_t t = a.argmax[r0 + u];
      int c = u + 1;
      while (c < k && !(a.in.parent[r0 + c] == u && a.in.tokens[r0 + c] == t)) ++c;
      if (c >= k) break;
      em[l] = t;
      u = c;
      path[++l] = u;
    }
    a.accept_len[seq] = l;
    em[l] = a.argmax[r0 + u];
    a.new_len[seq] = a.in.seq_len[seq] + l + 1;   // rejected rows stay in their pages, uncounted
    a.new_pending[seq] = a.argmax[r0 + u];
  }
}

// grid = (B, layers, kv heads), hd threads.  Path entry j (chunk row path[j]) moves from cache slot len + path[j]
// to slot len + j.  path is increasing with path[j] >= j, so going through j in ascending order never overwrites
// a row that is still to be moved; thread i moves element i of every row, so no barrier is needed.
__global__ void kv_compact_kernel(CompactArgs a) {
  pdl_launch_dependents();
  pdl_wait();
  const int seq = blockIdx.x, layer = blockIdx.y, kh = blockIdx.z, i = threadIdx.x;
  const int l = a.accept_len[seq], len = a.in.seq_len[seq];
  const int32_t *path = a.path + (size_t)seq * a.k_max;
  const int32_t *btab = a.in.block_tab + (size_t)seq * a.in.pages_per_seq;
  __half *kp = a.kv_pool + (uint64_t)layer * a.layer_stride;
  for (int j = 1; j <= l; ++j) {
    const int src = len + path[j], dst = len + j;
    if (src == dst) continue;
    const int ps = btab[src >> 4], pd = btab[dst >> 4];
    if (!ts_in_range(a.in.ck, CHK_PAGE_COMPACT, ps, a.in.ck.max_pages) ||
        !ts_in_range(a.in.ck, CHK_PAGE_COMPACT, pd, a.in.ck.max_pages))
      continue;
    const size_t so = (((size_t)ps * a.Hkv + kh) * 16 + (src & 15)) * a.hd + i;
    const size_t dof = (((size_t)pd * a.Hkv + kh) * 16 + (dst & 15)) * a.hd + i;
    kp[dof] = kp[so];
    kp[a.v_offset + dof] = kp[a.v_offset + so];
  }
}

cudaError_t launch_kv_compact(const CompactArgs &a, cudaStream_t st) {
  return launch_pdl(kv_compact_kernel, dim3(a.in.B, a.n_layers, a.Hkv), dim3(a.hd), 0, st, a);
}

cudaError_t launch_accept(const AcceptArgs &a, cudaStream_t st) {
  return launch_pdl(accept_kernel, dim3(a.in.B), dim3(64), 0, st, a);
}

}  // namespace ts
