// Paged grouped-query attention for the verify chunk: each of the k_i new rows of a sequence attends
// to the sequence's cached context plus the chunk rows up to itself (causal inside the chunk).
//
// Work decomposition: a CTA owns (KV split, kv head, tile of 64 packed query rows).  The G query
// heads that share a kv head are packed together with the chunk positions into rows r = j*G + g, so
// one pass over a K/V page serves all of them.  K/V blocks of 64 positions (4 pages) are staged in
// shared memory with 16-byte cp.async copies into an XOR-swizzled layout, double buffered; the
// cache, the queries and the softmax weights are fp16 (11 significant bits; same bytes per element
// as bf16), which keeps the first layers' attention output inside the logit tolerance; the products
// run on mma.sync m16n8k16 with fp16 operands and fp32 accumulation, ldmatrix operand fetches; the
// softmax is the streaming (running max / running sum) form in the log2 domain with quad shuffles.
// Each split writes an unnormalised partial output with its (max, sum); a second kernel merges the
// splits and emits bf16 (hi[, lo]) rows for the output projection.
#include <cuda_fp16.h>

#include "kernels.h"

namespace ts {

static constexpr int kRowsPerCta = 64;
static constexpr int kBlk = 64;  // kv positions per staged block

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid) {
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_f16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_f16(float a, float b) {
  __half2 v = __floats2half2_rn(a, b);
  return *reinterpret_cast<uint32_t *>(&v);
}
// byte offset of 16-byte chunk c of row r in a [rows][HD] fp16 tile with the XOR swizzle
template <int HD>
__device__ __forceinline__ uint32_t swz(int r, int c) {
  return (uint32_t)(r * (HD * 2) + ((c ^ (r & 7)) << 4));
}

template <int HD>
__global__ void __launch_bounds__(128)
attn_split_kernel(const AttnArgs a) {
  constexpr int CH = HD / 8;         // 16-byte chunks per row
  constexpr int TILE = kBlk * HD * 2;
  extern __shared__ __align__(128) uint8_t sm[];
  uint8_t *sQ = sm, *sK = sm + TILE, *sV = sm + 3 * TILE;   // K and V: two stages each

  // Everything this kernel reads (the row-tile table included) may come from the kernel before it.
  pdl_launch_dependents();   // the dependent kernel waits for this one's end before touching its data
  pdl_wait();
  const int split = blockIdx.x, kh = blockIdx.y, tile = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = a.Hq / a.Hkv;
  const int seq = a.tile_seq[tile], row0 = a.tile_row0[tile];
  const int r_beg = a.in.cu_rows[seq];
  const int k_i = a.in.cu_rows[seq + 1] - r_beg;
  const int len = a.in.seq_len[seq];
  const int R = k_i * G;
  const int rows_here = min(kRowsPerCta, R - row0);
  const int total = len + k_i;
  const int nblk = (total + kBlk - 1) / kBlk;
  const int bps = (nblk + a.n_splits - 1) / a.n_splits;
  const int j_max = (row0 + rows_here - 1) / G;
  const int b0 = split * bps;
  const int b1 = min(min(nblk, b0 + bps), (len + j_max + 1 + kBlk - 1) / kBlk);
  const int32_t *btab = a.in.block_tab + (size_t)seq * a.in.pages_per_seq;

  // this thread's two rows of the warp's 16-row tile
  const int rl = warp * 16 + (lane >> 2), rh = rl + 8;
  const int prl = row0 + rl, prh = row0 + rh;             // packed row indices
  const bool vl = rl < rows_here, vh = rh < rows_here;
  const int lim_l = len + (vl ? prl / G : 0), lim_h = len + (vh ? prh / G : 0);   // last visible position

  auto out_base = [&](int pr) -> size_t {
    const int j = pr / G, gq = pr % G;
    return ((size_t)(r_beg + j) * a.Hq + kh * G + gq) * a.n_splits + split;
  };

  if (b0 >= b1) {   // nothing visible in this split: mark it empty
    if ((lane & 3) == 0) {
      if (vl) a.part_ml[out_base(prl)] = make_float2(-INFINITY, 0.f);
      if (vh) a.part_ml[out_base(prh)] = make_float2(-INFINITY, 0.f);
    }
    return;
  }

  // ---- stage Q (64 packed rows) ---------------------------------------------------------------
  for (int idx = threadIdx.x; idx < kRowsPerCta * CH; idx += 128) {
    const int r = idx / CH, c = idx % CH;
    const int pr = row0 + r;
    const bool valid = r < rows_here;
    const int j = valid ? pr / G : 0, gq = valid ? pr % G : 0;
    const __half *src = a.q + ((size_t)(r_beg + j) * a.Hq + kh * G + gq) * HD + c * 8;
    cp_async16(smem_u32(sQ) + swz<HD>(r, c), src, valid);
  }
  auto load_block = [&](int b, int stage) {
    const uint32_t dK = smem_u32(sK) + stage * TILE, dV = smem_u32(sV) + stage * TILE;
    for (int idx = threadIdx.x; idx < kBlk * CH; idx += 128) {
      const int r = idx / CH, c = idx % CH;
      const int pos = b * kBlk + r;
      const bool valid = pos < total;
      const int page = valid ? btab[pos >> 4] : 0;
      const size_t off = (((size_t)page * a.Hkv + kh) * 16 + (pos & 15)) * HD + c * 8;
      cp_async16(dK + swz<HD>(r, c), a.k_pages + off, valid);
      cp_async16(dV + swz<HD>(r, c), a.v_pages + off, valid);
    }
  };
  load_block(b0, 0);
  cp_async_commit();

  uint32_t qa[HD / 16][4];
  float o[HD / 8][4];
#pragma unroll
  for (int t = 0; t < HD / 8; ++t) o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f;
  float m_l = -INFINITY, m_h = -INFINITY, l_l = 0.f, l_h = 0.f;
  const float scale = rsqrtf((float)HD) * 1.4426950408889634f;
  const bool warp_active = warp * 16 < rows_here;

  for (int b = b0; b < b1; ++b) {
    const int stage = (b - b0) & 1;
    if (b + 1 < b1) load_block(b + 1, stage ^ 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    if (b == b0) {
#pragma unroll
      for (int ks = 0; ks < HD / 16; ++ks) {
        const int mat = lane >> 3;
        ldsm_x4(smem_u32(sQ) + swz<HD>(warp * 16 + (lane & 7) + 8 * (mat & 1), ks * 2 + (mat >> 1)), qa[ks][0],
                qa[ks][1], qa[ks][2], qa[ks][3]);
      }
    }
    if (warp_active) {
      const uint32_t bK = smem_u32(sK) + stage * TILE, bV = smem_u32(sV) + stage * TILE;
      float s[8][4];
#pragma unroll
      for (int t = 0; t < 8; ++t) s[t][0] = s[t][1] = s[t][2] = s[t][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < HD / 16; ++ks) {
#pragma unroll
        for (int n2 = 0; n2 < 4; ++n2) {
          const int mat = lane >> 3;
          uint32_t k0, k1, k2, k3;
          ldsm_x4(bK + swz<HD>(n2 * 16 + (lane & 7) + 8 * (mat >> 1), ks * 2 + (mat & 1)), k0, k1, k2, k3);
          mma_f16(s[2 * n2], qa[ks], k0, k1);
          mma_f16(s[2 * n2 + 1], qa[ks], k2, k3);
        }
      }
      // mask, running max
      const int pbase = b * kBlk + (lane & 3) * 2;
      float mx_l = -INFINITY, mx_h = -INFINITY;
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        const int p0 = pbase + t * 8;
        s[t][0] = (p0 <= lim_l) ? s[t][0] * scale : -INFINITY;
        s[t][1] = (p0 + 1 <= lim_l) ? s[t][1] * scale : -INFINITY;
        s[t][2] = (p0 <= lim_h) ? s[t][2] * scale : -INFINITY;
        s[t][3] = (p0 + 1 <= lim_h) ? s[t][3] * scale : -INFINITY;
        mx_l = fmaxf(mx_l, fmaxf(s[t][0], s[t][1]));
        mx_h = fmaxf(mx_h, fmaxf(s[t][2], s[t][3]));
      }
      mx_l = fmaxf(mx_l, __shfl_xor_sync(0xffffffffu, mx_l, 1));
      mx_l = fmaxf(mx_l, __shfl_xor_sync(0xffffffffu, mx_l, 2));
      mx_h = fmaxf(mx_h, __shfl_xor_sync(0xffffffffu, mx_h, 1));
      mx_h = fmaxf(mx_h, __shfl_xor_sync(0xffffffffu, mx_h, 2));
      const float mn_l = fmaxf(m_l, mx_l), mn_h = fmaxf(m_h, mx_h);
      const float ref_l = (mn_l == -INFINITY) ? 0.f : mn_l, ref_h = (mn_h == -INFINITY) ? 0.f : mn_h;
      const float f_l = exp2f(m_l - ref_l), f_h = exp2f(m_h - ref_h);   // exp2(-inf) = 0 on the first block
      m_l = mn_l; m_h = mn_h;
      l_l *= f_l; l_h *= f_h;
#pragma unroll
      for (int t = 0; t < HD / 8; ++t) { o[t][0] *= f_l; o[t][1] *= f_l; o[t][2] *= f_h; o[t][3] *= f_h; }
      uint32_t pa[4][4];
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        const float p0 = exp2f(s[t][0] - ref_l), p1 = exp2f(s[t][1] - ref_l);
        const float p2 = exp2f(s[t][2] - ref_h), p3 = exp2f(s[t][3] - ref_h);
        l_l += p0 + p1;
        l_h += p2 + p3;
        pa[t >> 1][(t & 1) * 2 + 0] = pack_f16(p0, p1);
        pa[t >> 1][(t & 1) * 2 + 1] = pack_f16(p2, p3);
      }
#pragma unroll
      for (int kt = 0; kt < 4; ++kt) {
#pragma unroll
        for (int d2 = 0; d2 < HD / 16; ++d2) {
          const int mat = lane >> 3;
          uint32_t v0, v1, v2, v3;
          ldsm_x4_t(bV + swz<HD>(kt * 16 + (lane & 7) + 8 * (mat & 1), d2 * 2 + (mat >> 1)), v0, v1, v2, v3);
          mma_f16(o[2 * d2], pa[kt], v0, v1);
          mma_f16(o[2 * d2 + 1], pa[kt], v2, v3);
        }
      }
    }
    __syncthreads();
  }
  cp_async_wait<0>();

  l_l += __shfl_xor_sync(0xffffffffu, l_l, 1);
  l_l += __shfl_xor_sync(0xffffffffu, l_l, 2);
  l_h += __shfl_xor_sync(0xffffffffu, l_h, 1);
  l_h += __shfl_xor_sync(0xffffffffu, l_h, 2);
  if (vl) {
    const size_t ob = out_base(prl);
    if ((lane & 3) == 0) a.part_ml[ob] = make_float2(m_l, l_l);
    float *dst = a.part_o + ob * HD + (lane & 3) * 2;
#pragma unroll
    for (int t = 0; t < HD / 8; ++t) *reinterpret_cast<float2 *>(dst + t * 8) = make_float2(o[t][0], o[t][1]);
  }
  if (vh) {
    const size_t ob = out_base(prh);
    if ((lane & 3) == 0) a.part_ml[ob] = make_float2(m_h, l_h);
    float *dst = a.part_o + ob * HD + (lane & 3) * 2;
#pragma unroll
    for (int t = 0; t < HD / 8; ++t) *reinterpret_cast<float2 *>(dst + t * 8) = make_float2(o[t][2], o[t][3]);
  }
}

// grid = (M, Hq), hd threads: merge the splits of one (row, query head).  Every thread issues the loads of its
// output element for all splits at once, together with the splits' (max, sum) pairs (lane s of each warp takes
// split s and turns it into a normalised weight), so the kernel costs one round trip to L2.  NS = compile-time bound
// on the number of splits.
template <int NS>
__global__ void attn_combine_kernel(const AttnArgs a) {
  pdl_launch_dependents();   // the dependent kernel waits for this one's end before touching its data
  pdl_wait();
  const int m = blockIdx.x, h = blockIdx.y, d = threadIdx.x, lane = threadIdx.x & 31;
  const size_t base = ((size_t)m * a.Hq + h) * a.n_splits;
  const float2 ml = lane < a.n_splits ? a.part_ml[base + lane] : make_float2(-INFINITY, 0.f);
  // (an empty split never wrote its slot; whatever is read there is dropped by its zero weight below)
  float t[NS];
#pragma unroll
  for (int s = 0; s < NS; ++s) t[s] = (s < a.n_splits) ? a.part_o[(base + s) * a.hd + d] : 0.f;
  float mx = ml.y > 0.f ? ml.x : -INFINITY;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  float w = ml.y > 0.f ? exp2f(ml.x - mx) : 0.f;
  const float den = warp_sum(w * ml.y);
  w *= 1.f / den;
  float num = 0.f;
#pragma unroll
  for (int s = 0; s < NS; ++s) {
    const float ws = __shfl_sync(0xffffffffu, w, s);
    if (ws != 0.f) num += ws * t[s];
  }
  __nv_bfloat16 hi, lo;
  split_bf16(num, hi, lo);
  const size_t col = (size_t)h * a.hd + d;
  const size_t ld = (size_t)a.Hq * a.hd;
  a.out[(size_t)m * ld + col] = hi;
  if (a.planes == 2) a.out[((size_t)a.out_rows + m) * ld + col] = lo;
}

template <typename K>
static cudaError_t launch_attn_pdl(K kernel, dim3 grid, dim3 block, size_t smem, cudaStream_t st, const AttnArgs &a) {
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
  return cudaLaunchKernelEx(&cfg, kernel, a);
}

cudaError_t launch_attention_split(const AttnArgs &a, cudaStream_t st) {
  static PerDeviceOnce once;
  int dev_ = -1;
  if (once.needed(&dev_)) {
    cudaError_t e = cudaFuncSetAttribute(attn_split_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         5 * kBlk * 128 * 2);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_split_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             5 * kBlk * 64 * 2);
    if (e != cudaSuccess) return e;
    once.done(dev_);
  }
  const dim3 grid(a.n_splits, a.Hkv, a.n_row_tiles_total);
  const size_t smem = (size_t)5 * kBlk * a.hd * 2;
  return (a.hd == 128) ? launch_attn_pdl(attn_split_kernel<128>, grid, dim3(128), smem, st, a)
                       : launch_attn_pdl(attn_split_kernel<64>, grid, dim3(128), smem, st, a);
}

cudaError_t launch_attention_combine(const AttnArgs &a, cudaStream_t st) {
  if (a.n_splits < 1 || a.n_splits > kAttnMaxSplits) return cudaErrorInvalidValue;
  const dim3 grid(a.in.M, a.Hq), block(a.hd);
  if (a.n_splits <= 2) return launch_attn_pdl(attn_combine_kernel<2>, grid, block, 0, st, a);
  if (a.n_splits <= 4) return launch_attn_pdl(attn_combine_kernel<4>, grid, block, 0, st, a);
  if (a.n_splits <= 8) return launch_attn_pdl(attn_combine_kernel<8>, grid, block, 0, st, a);
  if (a.n_splits <= 16) return launch_attn_pdl(attn_combine_kernel<16>, grid, block, 0, st, a);
  return launch_attn_pdl(attn_combine_kernel<32>, grid, block, 0, st, a);
}

}  // namespace ts
