// The whole verify step for a small number of rows (M <= 64) as ONE persistent cooperative kernel.
//
// At batch 1 the step is bound by streaming 15 GB of weights and the context's K/V once.  Separate
// kernels stall that stream at every boundary, so here one CTA per SM walks all phases of the step:
//
//   embed | per layer: QKV proj (+rotary, KV append) | attention | merge | O proj (+residual) |
//         gate-up proj (+SwiGLU) | down proj (+residual) | LM head (+argmax) | accept
//
// Warp roles:  warp 0  weight producer: TMA loads of 128x64 weight blocks into a shared-memory ring.
//                      Weights depend on nothing, so this warp runs ahead of every phase boundary.
//              warp 1  activation producer: TMA loads of the (hi, lo) activation rows of each k-block
//                      once the phase that writes them has completed on every CTA.
//              warp 2  tcgen05.mma issue (weights = operand A, 128 rows; activations = operand B),
//                      fp32 accumulators in tensor memory, four buffers.
//              warps 3..10  workers: epilogues out of tensor memory, tile fix-up, attention
//                      (mma.sync on fp16 K/V staged with cp.async), merge, acceptance.
//
// Projections are cut stream-K style (schedule.h): every CTA owns an equal run of (tile, k-block)
// units; a tile shared by several CTAs is finished by the last one to arrive, which adds the parked
// partial sums in CTA order and applies the epilogue.  Phases are separated by a grid-wide counter
// barrier.  RMSNorm is folded away: residual epilogues emit the un-normalised activations (times the
// gain) together with per-tile sums of squares, and the consuming projection scales its accumulator
// rows by rsqrt(mean square + eps), which is the same product.
//
// Every wait is bounded.  A wait that expires records an error word that all other waits watch, so
// the grid drains and exits normally (tensor memory freed) and the host reports a device timeout.
#include <cuda_fp16.h>

#include <algorithm>

#include "kernels.h"
#include "schedule.h"

namespace ts {

static constexpr int kThreads = 352;
static constexpr int kWorkerWarp0 = 3;
static constexpr int kWorkers = 256;
static constexpr int kBlockK = 64;
static constexpr int kTileN = 128;
static constexpr int kWBytes = kTileN * kBlockK * 2;
static constexpr int kMaxRing = 12;
static constexpr int kMaxMc = 64;
static constexpr int kAccBufs = 4;      // accumulator buffers in tensor memory (4 x 128 columns at most)
static constexpr int kAttnRows = 128;   // packed (position, query head) rows per attention unit
static constexpr int kAttnBlk = 64;     // kv positions per staged block

enum : int { OP_QKV = 0, OP_O = 1, OP_GU = 2, OP_D = 3, OP_LM = 4, OP_EMBED = 5 };

struct __align__(16) FusedCtl {
  uint64_t full[kMaxRing];
  uint64_t empty[kMaxRing];
  uint64_t tmem_full[kAccBufs];
  uint64_t tmem_empty[kAccBufs];
  uint32_t tmem_base;
  int flag;
  int attn_epoch;            // attention phases this CTA has finished (ring slots under the staging area are free)
  int row_pos[kMaxMc];       // absolute position of each row
  int row_page[kMaxMc];      // KV page holding that position
  float r_s[kMaxMc];
  float ss_acc[2][4][kMaxMc];
};

// ---- small device helpers ---------------------------------------------------------------------------
__device__ __forceinline__ int ld_acquire(const int *p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void worker_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ bool worker_all(bool ok) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %1, 0;\n\tbar.red.and.pred q, 1, 256, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(r)
      : "r"((uint32_t)ok)
      : "memory");
  return r != 0;
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

// Bounded mbarrier wait that also gives up when another CTA has reported an error.
__device__ __forceinline__ bool mbar_wait_err(uint32_t bar, uint32_t parity, const int *err) {
  uint64_t t0 = 0;
  for (uint32_t it = 0;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 255u) == 255u) {
      if (*reinterpret_cast<const volatile int *>(err) != 0) return false;
      const uint64_t now = global_timer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > 2000000000ull) return false;
      __nanosleep(32);
    }
  }
}

// Wait until the grid-wide phase counter reaches `target` (single thread).
__device__ __forceinline__ bool grid_wait(const int *ctr, int target, const int *err) {
  uint64_t t0 = 0;
  for (uint32_t it = 0;; ++it) {
    if (ld_acquire(ctr) >= target) return true;
    if ((it & 63u) == 63u) {
      if (*reinterpret_cast<const volatile int *>(err) != 0) return false;
      const uint64_t now = global_timer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > 2000000000ull) return false;
    }
    __nanosleep(20);
  }
}

struct OpInfo {
  int op, layer;
  int T, KB;          // tiles, k-blocks
  int map_w, map_a;   // tensor-map indices
  int phase;          // grid phase index of this projection
  int use;            // how many times this op's tile counters were used before (monotonic counters)
  int cnt_base;       // first tile counter
};

__device__ __forceinline__ OpInfo gemm_op(const FusedArgs &a, int g) {
  OpInfo o;
  const int L = a.n_layers;
  if (g < 4 * L) {
    o.layer = g >> 2;
    o.op = g & 3;
  } else {
    o.layer = 0;
    o.op = OP_LM;
  }
  o.use = o.layer;
  const int am = 4 * L + 1 + 3 * a.mc_index;
  switch (o.op) {
    case OP_QKV: o.T = a.Nqkv / kTileN; o.KB = a.d / kBlockK; o.map_a = am + 0; o.phase = 1 + 6 * o.layer; o.cnt_base = 0; break;
    case OP_O: o.T = a.d / kTileN; o.KB = a.Nq / kBlockK; o.map_a = am + 1; o.phase = 4 + 6 * o.layer; o.cnt_base = a.Nqkv / kTileN; break;
    case OP_GU: o.T = 2 * a.F / kTileN; o.KB = a.d / kBlockK; o.map_a = am + 0; o.phase = 5 + 6 * o.layer;
      o.cnt_base = (a.Nqkv + a.d) / kTileN; break;
    case OP_D: o.T = a.d / kTileN; o.KB = a.F / kBlockK; o.map_a = am + 2; o.phase = 6 + 6 * o.layer;
      o.cnt_base = (a.Nqkv + a.d + 2 * a.F) / kTileN; break;
    default: o.T = a.V / kTileN; o.KB = a.d / kBlockK; o.map_a = am + 0; o.phase = 1 + 6 * L;
      o.cnt_base = (a.Nqkv + 2 * a.d + 2 * a.F) / kTileN; break;
  }
  o.map_w = (o.op == OP_LM) ? 4 * L : 4 * o.layer + o.op;
  return o;
}

// ---- epilogues ----------------------------------------------------------------------------------------
// One warp holds 16 rows (c0 .. c0+15) of 32 consecutive output features: lane <-> feature.
// All global loads of an epilogue come before its first store: the compiler must assume that a store
// aliases a later load, so interleaving them would put one L2 round trip per row on the critical path.
__device__ __forceinline__ void epilogue16(const FusedArgs &a, const OpInfo &o, FusedCtl *ctl, int tile, int q, int lane,
                                           int c0, float (&v)[16], int ss_buf) {
  const int n = tile * kTileN + q * 32 + lane;
  const int M = a.in.M;
  if (o.op == OP_QKV) {
    // weight rows are stored with rotary partners adjacent: feature 2i = element i, 2i+1 = element i + hd/2
    const int hd = a.hd, half = hd >> 1;
    const int head = n / hd, e = n - head * hd, i = e >> 1, odd = e & 1;
    const int elem = odd ? i + half : i;
    const bool rot = head < a.Hq + a.Hkv;
    float2 cs[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const int m = min(c0 + j, M - 1);
      cs[j] = rot ? a.rope[(size_t)ctl->row_pos[m] * half + i] : make_float2(1.f, 0.f);
    }
    const bool is_q = head < a.Hq, is_k = head < a.Hq + a.Hkv;
    const int kh = is_k ? head - a.Hq : head - a.Hq - a.Hkv;
    __half *kv = a.kv_pool + (size_t)o.layer * a.kv_layer_stride + (is_k ? 0 : a.kv_v_offset);
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const int m = c0 + j;
      if (m >= M) break;
      const float val = v[j] * ctl->r_s[m];
      const float other = __shfl_xor_sync(0xffffffffu, val, 1);
      const float out = odd ? (val * cs[j].x + other * cs[j].y) : (val * cs[j].x - other * cs[j].y);
      const __half hv = __float2half_rn(fminf(fmaxf(out, -65504.f), 65504.f));
      if (is_q) {
        a.q[((size_t)m * a.Hq + head) * hd + elem] = hv;
      } else {
        const int pos = ctl->row_pos[m];
        kv[(((size_t)ctl->row_page[m] * a.Hkv + kh) * 16 + (pos & 15)) * hd + elem] = hv;
      }
    }
  } else if (o.op == OP_O || o.op == OP_D || o.op == OP_EMBED) {
    const int d = a.d;
    // gain of the norm that follows: g2[l] after O, g1[l+1] (or the final gain) after down, g1[0] after embed
    const float *gain = a.gains + (size_t)a.gain_stride *
        (o.op == OP_O ? 2 * o.layer + 1 : (o.op == OP_EMBED ? 0 : (o.layer + 1 < a.n_layers ? 2 * o.layer + 2 : 2 * a.n_layers)));
    const float gn = gain[n];
    float xo[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) xo[j] = (o.op != OP_EMBED && c0 + j < M) ? __ldcg(a.x + (size_t)(c0 + j) * d + n) : 0.f;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const int m = c0 + j;
      if (m >= M) break;
      const float xn = v[j] + xo[j];
      a.x[(size_t)m * d + n] = xn;
      __nv_bfloat16 hi, lo;
      split_bf16(xn * gn, hi, lo);
      a.h[(size_t)m * d + n] = hi;
      if (a.planes == 2) a.h[((size_t)a.R + m) * d + n] = lo;
      const float s = warp_sum(xn * xn);
      if (lane == 0) ctl->ss_acc[ss_buf][q][m] = s;
    }
  } else if (o.op == OP_GU) {
    const int f = n >> 1, F = a.F;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const int m = c0 + j;
      if (m >= M) break;
      const float val = v[j] * ctl->r_s[m];
      const float other = __shfl_xor_sync(0xffffffffu, val, 1);
      const float gate = (lane & 1) ? other : val;
      const float up = (lane & 1) ? val : other;
      const float act = gate / (1.f + __expf(-gate)) * up;
      __nv_bfloat16 hi, lo;
      split_bf16(act, hi, lo);
      if ((lane & 1) == 0) a.act[(size_t)m * F + f] = hi;
      else if (a.planes == 2) a.act[((size_t)a.R + m) * F + f] = lo;
    }
  } else {  // OP_LM
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const int m = c0 + j;
      if (m >= M) break;
      const float val = v[j] * ctl->r_s[m];
      a.logits[(size_t)m * a.V + n] = val;
      float bv = val;
      int bi = n;
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, s);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, s);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
      }
      if (lane == 0) {   // order-preserving map of the float; ties resolve to the lowest id
        uint32_t u = __float_as_uint(bv);
        u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
        atomicMax(a.amax + m, ((unsigned long long)u << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)bi));
      }
    }
  }
}

// After a residual-type tile: fold the four feature quarters' sums of squares into the tile's slot.
__device__ __forceinline__ void finish_ss(const FusedArgs &a, FusedCtl *ctl, int tile, int wtid, int ss_buf) {
  worker_sync();
  if (wtid < a.in.M)
    a.ss_part[(size_t)tile * a.R + wtid] = ctl->ss_acc[ss_buf][0][wtid] + ctl->ss_acc[ss_buf][1][wtid] +
                                           ctl->ss_acc[ss_buf][2][wtid] + ctl->ss_acc[ss_buf][3][wtid];
}

// Per-row scale of the RMSNorm that precedes this projection: rsqrt(mean(x^2) + eps).
__device__ __forceinline__ void compute_row_scale(const FusedArgs &a, FusedCtl *ctl, int wtid) {
  if (wtid < a.in.M) {
    const int Td = a.d / kTileN;
    float s = 0.f;
    for (int t = 0; t < Td; ++t) s += __ldcg(a.ss_part + (size_t)t * a.R + wtid);
    ctl->r_s[wtid] = rsqrtf(s / (float)a.d + a.eps);
  }
  worker_sync();
}

// ---- attention (workers) --------------------------------------------------------------------------------
__device__ __forceinline__ void cp_async16z(uint32_t dst, const void *src, bool valid) {
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm4t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_h2(float x, float y) {
  __half2 v = __floats2half2_rn(x, y);
  return *reinterpret_cast<uint32_t *>(&v);
}
template <int HD>
__device__ __forceinline__ uint32_t swz(int r, int c) {
  return (uint32_t)(r * (HD * 2) + ((c ^ (r & 7)) << 4));
}

// One unit: (row tile, kv head, split).  256 worker threads; warp w owns packed rows 16w .. 16w+15.
// K/V blocks of 64 positions are double buffered; scores are taken 32 positions at a time, each with its
// own running-softmax update, which halves the score registers.
template <int HD>
__device__ __noinline__ void attn_unit(const FusedArgs &a, int layer, uint8_t *sm, int tile, int kh, int split, int widx,
                                       int lane, int wtid) {
  constexpr int CH = HD / 8;
  constexpr int QB = kAttnRows * HD * 2;
  constexpr int TB = kAttnBlk * HD * 2;
  uint8_t *sQ = sm, *sK = sm + QB, *sV = sm + QB + 2 * TB;
  const int G = a.Hq / a.Hkv;
  const int seq = a.tile_seq[tile], row0 = a.tile_row0[tile];
  const int r_beg = a.in.cu_rows[seq];
  const int k_i = a.in.cu_rows[seq + 1] - r_beg;
  const int len = a.in.seq_len[seq];
  const int R = k_i * G;
  const int rows_here = min(kAttnRows, R - row0);
  const int total = len + k_i;
  const int j_max = (row0 + rows_here - 1) / G;
  int p0, p1;
  split_pages((total + 15) >> 4, a.attn_splits, split, &p0, &p1);
  const int pos_beg = p0 << 4;
  const int pos_end = min(min(p1 << 4, total), len + j_max + 1);
  const int32_t *btab = a.in.block_tab + (size_t)seq * a.in.pages_per_seq;
  const __half *kp = a.kv_pool + (size_t)layer * a.kv_layer_stride;
  const __half *vp = kp + a.kv_v_offset;

  const int rl = widx * 16 + (lane >> 2), rh = rl + 8;
  const int prl = row0 + rl, prh = row0 + rh;
  const bool vl = rl < rows_here, vh = rh < rows_here;
  const int lim_l = min(len + (vl ? prl / G : 0), pos_end - 1), lim_h = min(len + (vh ? prh / G : 0), pos_end - 1);
  auto out_base = [&](int pr) -> size_t {
    const int j = pr / G, gq = pr % G;
    return ((size_t)(r_beg + j) * a.Hq + kh * G + gq) * a.attn_splits + split;
  };
  if (pos_beg >= pos_end) {   // nothing visible in this split: mark it empty
    if ((lane & 3) == 0) {
      if (vl) a.attn_ml[out_base(prl)] = make_float2(-INFINITY, 0.f);
      if (vh) a.attn_ml[out_base(prh)] = make_float2(-INFINITY, 0.f);
    }
    return;
  }
  const int nblk = (pos_end - pos_beg + kAttnBlk - 1) / kAttnBlk;

  worker_sync();   // the previous unit's readers are done with the staging buffers
  for (int idx = wtid; idx < kAttnRows * CH; idx += kWorkers) {
    const int r = idx / CH, c = idx % CH;
    const int pr = row0 + r;
    const bool valid = r < rows_here;
    const int j = valid ? pr / G : 0, gq = valid ? pr % G : 0;
    const __half *src = a.q + ((size_t)(r_beg + j) * a.Hq + kh * G + gq) * HD + c * 8;
    cp_async16z(smem_u32(sQ) + swz<HD>(r, c), src, valid);
  }
  auto load_block = [&](int b, int stage) {
    const uint32_t dK = smem_u32(sK) + stage * TB, dV = smem_u32(sV) + stage * TB;
    for (int idx = wtid; idx < kAttnBlk * CH; idx += kWorkers) {
      const int r = idx / CH, c = idx % CH;
      const int pos = pos_beg + b * kAttnBlk + r;
      const bool valid = pos < pos_end;
      const int page = valid ? btab[pos >> 4] : 0;
      const size_t off = (((size_t)page * a.Hkv + kh) * 16 + (pos & 15)) * HD + c * 8;
      cp_async16z(dK + swz<HD>(r, c), kp + off, valid);
      cp_async16z(dV + swz<HD>(r, c), vp + off, valid);
    }
  };
  load_block(0, 0);
  cp_commit();

  float o[HD / 8][4];
#pragma unroll
  for (int t = 0; t < HD / 8; ++t) o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f;
  float m_l = -INFINITY, m_h = -INFINITY, l_l = 0.f, l_h = 0.f;
  const float scale = rsqrtf((float)HD) * 1.4426950408889634f;
  const bool warp_active = widx * 16 < rows_here;

  for (int b = 0; b < nblk; ++b) {
    const int stage = b & 1;
    if (b + 1 < nblk) load_block(b + 1, stage ^ 1);
    cp_commit();
    cp_wait<1>();
    worker_sync();
    if (warp_active) {
      const uint32_t bK = smem_u32(sK) + stage * TB, bV = smem_u32(sV) + stage * TB;
      const int mat = lane >> 3;
#pragma unroll 1
      for (int sb = 0; sb < 2; ++sb) {
        float s[4][4];
#pragma unroll
        for (int t = 0; t < 4; ++t) s[t][0] = s[t][1] = s[t][2] = s[t][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
          uint32_t qa[4];   // Q fragment of this k-slice, re-read from shared memory to keep registers free
          ldsm4(smem_u32(sQ) + swz<HD>(widx * 16 + (lane & 7) + 8 * (mat & 1), ks * 2 + (mat >> 1)), qa[0], qa[1], qa[2], qa[3]);
#pragma unroll
          for (int n2 = 0; n2 < 2; ++n2) {
            uint32_t k0, k1, k2, k3;
            ldsm4(bK + swz<HD>(sb * 32 + n2 * 16 + (lane & 7) + 8 * (mat >> 1), ks * 2 + (mat & 1)), k0, k1, k2, k3);
            mma16816(s[2 * n2], qa, k0, k1);
            mma16816(s[2 * n2 + 1], qa, k2, k3);
          }
        }
        const int pbase = pos_beg + b * kAttnBlk + sb * 32 + (lane & 3) * 2;
        float mx_l = -INFINITY, mx_h = -INFINITY;
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          const int q0 = pbase + t * 8;
          s[t][0] = (q0 <= lim_l) ? s[t][0] * scale : -INFINITY;
          s[t][1] = (q0 + 1 <= lim_l) ? s[t][1] * scale : -INFINITY;
          s[t][2] = (q0 <= lim_h) ? s[t][2] * scale : -INFINITY;
          s[t][3] = (q0 + 1 <= lim_h) ? s[t][3] * scale : -INFINITY;
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
        uint32_t pa[2][4];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          const float e0 = exp2f(s[t][0] - ref_l), e1 = exp2f(s[t][1] - ref_l);
          const float e2 = exp2f(s[t][2] - ref_h), e3 = exp2f(s[t][3] - ref_h);
          l_l += e0 + e1;
          l_h += e2 + e3;
          pa[t >> 1][(t & 1) * 2 + 0] = pack_h2(e0, e1);
          pa[t >> 1][(t & 1) * 2 + 1] = pack_h2(e2, e3);
        }
#pragma unroll
        for (int kt = 0; kt < 2; ++kt) {
#pragma unroll
          for (int d2 = 0; d2 < HD / 16; ++d2) {
            uint32_t v0, v1, v2, v3;
            ldsm4t(bV + swz<HD>(sb * 32 + kt * 16 + (lane & 7) + 8 * (mat & 1), d2 * 2 + (mat >> 1)), v0, v1, v2, v3);
            mma16816(o[2 * d2], pa[kt], v0, v1);
            mma16816(o[2 * d2 + 1], pa[kt], v2, v3);
          }
        }
      }
    }
    worker_sync();
  }
  cp_wait<0>();

  l_l += __shfl_xor_sync(0xffffffffu, l_l, 1);
  l_l += __shfl_xor_sync(0xffffffffu, l_l, 2);
  l_h += __shfl_xor_sync(0xffffffffu, l_h, 1);
  l_h += __shfl_xor_sync(0xffffffffu, l_h, 2);
  if (vl) {
    const size_t ob = out_base(prl);
    if ((lane & 3) == 0) a.attn_ml[ob] = make_float2(m_l, l_l);
    float *dst = a.attn_o + ob * HD + (lane & 3) * 2;
#pragma unroll
    for (int t = 0; t < HD / 8; ++t) *reinterpret_cast<float2 *>(dst + t * 8) = make_float2(o[t][0], o[t][1]);
  }
  if (vh) {
    const size_t ob = out_base(prh);
    if ((lane & 3) == 0) a.attn_ml[ob] = make_float2(m_h, l_h);
    float *dst = a.attn_o + ob * HD + (lane & 3) * 2;
#pragma unroll
    for (int t = 0; t < HD / 8; ++t) *reinterpret_cast<float2 *>(dst + t * 8) = make_float2(o[t][2], o[t][3]);
  }
}

// Merge the splits of one (row, query head): one warp per pair, lane <-> split for the weights.
template <int HD>
__device__ __forceinline__ void merge_unit(const FusedArgs &a, int m, int h, int lane) {
  constexpr int EPL = HD / 32;   // output elements per lane
  const int S = a.attn_splits;
  const size_t base = ((size_t)m * a.Hq + h) * S;
  float2 ml = make_float2(-INFINITY, 0.f);
  if (lane < S) ml = __ldcg(a.attn_ml + base + lane);
  float mx = ml.y > 0.f ? ml.x : -INFINITY;
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, s));
  float w = ml.y > 0.f ? exp2f(ml.x - mx) : 0.f;
  const float den = warp_sum(w * ml.y);
  w /= den;
  float acc[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
  for (int s = 0; s < S; ++s) {
    const float ws = __shfl_sync(0xffffffffu, w, s);
    if (ws != 0.f) {
      const float *src = a.attn_o + (base + s) * HD + lane * EPL;
      if constexpr (EPL == 4) {
        const float4 t = __ldcg(reinterpret_cast<const float4 *>(src));
        acc[0] += ws * t.x; acc[1] += ws * t.y; acc[2] += ws * t.z; acc[3] += ws * t.w;
      } else {
        const float2 t = __ldcg(reinterpret_cast<const float2 *>(src));
        acc[0] += ws * t.x; acc[1] += ws * t.y;
      }
    }
  }
  const size_t ld = (size_t)a.Hq * HD;
  const size_t col = (size_t)h * HD + lane * EPL;
  __nv_bfloat16 hi[EPL], lo[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) split_bf16(acc[e], hi[e], lo[e]);
  if constexpr (EPL == 4) {
    *reinterpret_cast<uint2 *>(a.attn + (size_t)m * ld + col) = *reinterpret_cast<uint2 *>(hi);
    if (a.planes == 2) *reinterpret_cast<uint2 *>(a.attn + ((size_t)a.R + m) * ld + col) = *reinterpret_cast<uint2 *>(lo);
  } else {
    *reinterpret_cast<uint32_t *>(a.attn + (size_t)m * ld + col) = *reinterpret_cast<uint32_t *>(hi);
    if (a.planes == 2)
      *reinterpret_cast<uint32_t *>(a.attn + ((size_t)a.R + m) * ld + col) = *reinterpret_cast<uint32_t *>(lo);
  }
}

// ---- the kernel -------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 1) fused_verify_kernel(const __grid_constant__ FusedArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int a_bytes = a.planes * a.Mc * kBlockK * 2;
  const int stage_bytes = kWBytes + a_bytes;
  const int R = a.ring;
  // The attention staging area lies over the last ring slots (from slot `first_overlay` on): a projection
  // streams through every slot, attention borrows the tail of the ring while no projection needs it.
  const size_t attn_off = ((size_t)R * stage_bytes - (size_t)a.attn_smem_bytes) & ~(size_t)1023;
  uint8_t *attn_sm = smem + attn_off;
  const int first_overlay = (int)(attn_off / (size_t)stage_bytes);
  FusedCtl *ctl = reinterpret_cast<FusedCtl *>(smem + (size_t)R * stage_bytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t c = blockIdx.x, n = gridDim.x;
  const int ncols = a.planes * a.Mc;        // accumulator columns of one buffer
  uint32_t alloc_cols = 32;
  while (alloc_cols < (uint32_t)(kAccBufs * ncols)) alloc_cols <<= 1;
  int *ctr = a.sync, *err = a.err;
  const int n_gemms = 4 * a.n_layers + (a.skip_lm ? 0 : 1);

  if (threadIdx.x == 0) {
    for (int s = 0; s < R; ++s) {
      mbar_init(smem_u32(&ctl->full[s]), 2);    // weight producer + activation producer
      mbar_init(smem_u32(&ctl->empty[s]), 1);   // tcgen05.commit
    }
    for (int b = 0; b < kAccBufs; ++b) {
      mbar_init(smem_u32(&ctl->tmem_full[b]), 1);
      mbar_init(smem_u32(&ctl->tmem_empty[b]), 8);   // one arrival per worker warp
    }
    ctl->flag = 0;
    ctl->attn_epoch = 0;
    fence_barrier_init();
  }
  if (warp == 2) {
    tmem_alloc(smem_u32(&ctl->tmem_base), alloc_cols);
    tmem_relinquish();
  }
  if (threadIdx.x >= kWorkerWarp0 * 32 && (int)threadIdx.x - kWorkerWarp0 * 32 < a.in.M) {
    const int m = threadIdx.x - kWorkerWarp0 * 32;
    const int pos = a.in.pos[m];
    ctl->row_pos[m] = pos;
    ctl->row_page[m] = a.in.block_tab[(size_t)a.in.row_seq[m] * a.in.pages_per_seq + (pos >> 4)];
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;

  if (warp == 0) {
    // ================================================================ weight producer
    if (lane == 0) {
      const uint64_t pol_w = policy_evict_first();
      uint32_t round_par = 0;
      int slot = 0;
      bool ok = true;
      for (int g = 0; g < n_gemms && ok; ++g) {
        const OpInfo o = gemm_op(a, g);
        // a slot under the attention staging area may be refilled only once every attention phase that
        // precedes this projection has finished on this CTA
        const int need = o.op == OP_QKV ? o.layer : (o.op == OP_LM ? a.n_layers : o.layer + 1);
        SegmentIter sit(c, o.T, o.KB, n);
        Segment sg;
        while (ok && sit.next(&sg)) {
          for (int kb = sg.kb0; kb < sg.kb1; ++kb) {
            const int s = slot;
            const uint32_t par = round_par ^ 1;
            if (++slot == R) { slot = 0; round_par ^= 1; }
            const uint32_t ebar = smem_u32(&ctl->empty[s]);
            const bool borrowed = s >= first_overlay;
            uint64_t t0 = 0;
            for (uint32_t spin = 0;
                 !(mbar_try_wait(ebar, par) && (!borrowed || *reinterpret_cast<volatile int *>(&ctl->attn_epoch) >= need));
                 ++spin) {
              if ((spin & 255u) == 255u) {
                const uint64_t now = global_timer_ns();
                if (t0 == 0) t0 = now;
                if (*reinterpret_cast<const volatile int *>(err) != 0 || now - t0 > 2000000000ull) { ok = false; break; }
              }
            }
            if (!ok) { atomicCAS(err, 0, DEV_TIMEOUT_EMPTY); break; }
            const uint32_t bar = smem_u32(&ctl->full[s]);
            mbar_expect_tx(bar, kWBytes);
            // one block of the stored matrix = 16 contiguous KB = rows (tile * KB + kb) * 128 .. of a [.][64] array
            tma_load_2d(smem_u32(smem + (size_t)s * stage_bytes), &a.maps[o.map_w], 0, (sg.tile * o.KB + kb) * kTileN, bar, pol_w);
          }
        }
      }
      if (!ok) {   // let the copies in flight land before the CTA exits
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    // ================================================================ activation producer
    if (lane == 0) {
      const uint64_t pol_a = policy_evict_last();
      uint32_t round_par = 0;
      int slot = 0;
      bool ok = true;
      for (int g = 0; g < n_gemms && ok; ++g) {
        const OpInfo o = gemm_op(a, g);
        SegmentIter sit(c, o.T, o.KB, n);
        Segment sg;
        bool first = true;
        while (ok && sit.next(&sg)) {
          if (first) {
            ok = grid_wait(ctr, o.phase * (int)n, err);
            if (!ok) { atomicCAS(err, 0, DEV_TIMEOUT_GRID); break; }
            fence_proxy_async_all();   // other CTAs' generic-proxy stores -> this CTA's TMA reads
            first = false;
          }
          for (int kb = sg.kb0; kb < sg.kb1; ++kb) {
            const int s = slot;
            const uint32_t par = round_par ^ 1;
            if (++slot == R) { slot = 0; round_par ^= 1; }
            // (a borrowed slot is free by now: this phase's activations exist only after the attention before it)
            if (!mbar_wait_err(smem_u32(&ctl->empty[s]), par, err)) { ok = false; atomicCAS(err, 0, DEV_TIMEOUT_EMPTY); break; }
            const uint32_t bar = smem_u32(&ctl->full[s]);
            mbar_expect_tx(bar, a_bytes);
            tma_load_3d(smem_u32(smem + (size_t)s * stage_bytes + kWBytes), &a.maps[o.map_a], kb * kBlockK, 0, 0, bar, pol_a);
          }
        }
      }
      if (!ok) {
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
      }
    }
  } else if (warp == 2) {
    // ================================================================ MMA issue
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(kTileN, ncols);
      uint32_t seg = 0, round_par = 0;
      int slot = 0;
      bool ok = true;
      for (int g = 0; g < n_gemms && ok; ++g) {
        const OpInfo o = gemm_op(a, g);
        SegmentIter sit(c, o.T, o.KB, n);
        Segment sg;
        while (ok && sit.next(&sg)) {
          const uint32_t buf = seg % kAccBufs;
          if (!mbar_wait_err(smem_u32(&ctl->tmem_empty[buf]), ((seg / kAccBufs) & 1) ^ 1, err)) { ok = false; break; }
          tc_fence_after();
          const uint32_t dcol = tmem_base + buf * ncols;
          for (int kb = sg.kb0; kb < sg.kb1; ++kb) {
            const int s = slot;
            const uint32_t par = round_par;
            if (++slot == R) { slot = 0; round_par ^= 1; }
            if (!mbar_wait_err(smem_u32(&ctl->full[s]), par, err)) { ok = false; break; }
            if (a.phase_t && sg.index == 0 && kb == sg.kb0)
              atomicMax(a.phase_t + 2 * a.n_phases + o.phase, (unsigned long long)global_timer_ns());
            tc_fence_after();
            const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
            const uint64_t da = umma_desc_sw128(sa), db = umma_desc_sw128(sa + kWBytes);
#pragma unroll
            for (int kk = 0; kk < kBlockK / 16; ++kk)
              umma_bf16(dcol, da + 2 * kk, db + 2 * kk, idesc, (kb > sg.kb0 || kk > 0) ? 1u : 0u);
            umma_commit(smem_u32(&ctl->empty[s]));
          }
          if (!ok) break;
          umma_commit(smem_u32(&ctl->tmem_full[buf]));
          ++seg;
        }
        if (a.phase_t && ok) atomicMax(a.phase_t + a.n_phases + o.phase, (unsigned long long)global_timer_ns());
      }
      if (!ok) atomicCAS(err, 0, DEV_TIMEOUT_FULL);
    }
  } else {
    // ================================================================ workers
    const int widx = warp - kWorkerWarp0;          // 0..7
    const int wtid = threadIdx.x - kWorkerWarp0 * 32;
    const int q = warp & 3;                        // tensor-memory lane quarter this warp may read
    const int half = widx >> 2;
    const uint32_t tq = tmem_base + ((uint32_t)(q * 32) << 16);
    uint32_t seg = 0;
    int ss_buf = 0;
    int phase = 0;      // phases completed by this CTA
    bool ok = true;

    auto phase_done = [&]() {   // all workers' stores of this phase are complete -> arrive grid-wide
      worker_sync();
      if (wtid == 0) {
        if (a.phase_t) atomicMax(a.phase_t + phase, (unsigned long long)global_timer_ns());
        __threadfence();
        atomicAdd(ctr, 1);
      }
      ++phase;
    };
    auto wait_phases = [&](int n_phases) -> bool {   // every CTA has completed n_phases phases
      if (wtid == 0) {
        const bool w = grid_wait(ctr, n_phases * (int)n, err);
        if (!w) atomicCAS(err, 0, DEV_TIMEOUT_GRID);
        __threadfence();
        ctl->flag = w ? 1 : 0;
      }
      worker_sync();
      const bool w = ctl->flag != 0;
      worker_sync();
      return w;
    };

    // ---- one projection phase ------------------------------------------------------------------
    auto run_gemm = [&](int g) {
      const OpInfo o = gemm_op(a, g);
      // Every CTA waits here, busy or idle: the phase counter is a plain sum of arrivals, which is a
      // barrier only if nobody can arrive for this phase before all have arrived for the previous one.
      if (!wait_phases(o.phase)) { ok = false; return; }
      if (o.op == OP_QKV || o.op == OP_GU || o.op == OP_LM) compute_row_scale(a, ctl, wtid);
      SegmentIter sit(c, o.T, o.KB, n);
      Segment sg;
      const bool resid = (o.op == OP_O || o.op == OP_D);
      while (sit.next(&sg)) {
        const uint32_t buf = seg % kAccBufs;
        const bool got = mbar_wait_err(smem_u32(&ctl->tmem_full[buf]), (seg / kAccBufs) & 1, err);
        if (!worker_all(got)) { ok = false; return; }
        tc_fence_after();
        const TileCover tc = tile_cover(sg.tile, o.T, o.KB, n);
        const bool direct = tc.n_seg == 1;
        float *slab = a.slab + ((size_t)c * 2 + (sg.index == 0 ? 0 : 1)) * (size_t)(a.Mc * kTileN);
        for (int c0 = 16 * half; c0 < a.Mc; c0 += 32) {
          if (c0 >= a.in.M) break;
          uint32_t r[16], r2[16];
          float v[16];
          tmem_ld16(tq + buf * ncols + c0, r);
          if (a.planes == 2) tmem_ld16(tq + buf * ncols + a.Mc + c0, r2);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(r[j]) + (a.planes == 2 ? __uint_as_float(r2[j]) : 0.f);
          if (direct) {
            epilogue16(a, o, ctl, sg.tile, q, lane, c0, v, ss_buf);
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j)
              if (c0 + j < a.in.M) slab[(size_t)(c0 + j) * kTileN + q * 32 + lane] = v[j];
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctl->tmem_empty[buf]));
        ++seg;
        if (direct) {
          if (resid) { finish_ss(a, ctl, sg.tile, wtid, ss_buf); ss_buf ^= 1; }
          continue;
        }
        // partial tile: park, count, and let the last arriver finish the tile
        worker_sync();
        if (wtid == 0) {
          __threadfence();
          const int old = atomicAdd(a.sync + 8 + o.cnt_base + sg.tile, 1);
          const bool last = (old + 1) == tc.n_seg * (o.use + 1);
          if (last) __threadfence();
          ctl->flag = last ? 1 : 0;
        }
        worker_sync();
        const bool last = ctl->flag != 0;
        worker_sync();
        if (!last) continue;
        for (int c0 = 16 * half; c0 < a.Mc; c0 += 32) {
          if (c0 >= a.in.M) break;
          float v[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] = 0.f;
          // fixed CTA order, so the sum does not depend on which CTA finishes the tile; the loads of three
          // parked pieces are in flight together
          for (int s = 0; s < tc.n_seg; s += 3) {
            float t[3][16];
#pragma unroll
            for (int u = 0; u < 3; ++u) {
              const int cc = tc.c_first + min(s + u, tc.n_seg - 1);
              const float *src = a.slab + ((size_t)cc * 2 + slab_slot_of(cc, sg.tile, o.T, o.KB, n)) * (size_t)(a.Mc * kTileN) +
                                 q * 32 + lane;
#pragma unroll
              for (int j = 0; j < 16; ++j) t[u][j] = (c0 + j < a.in.M) ? __ldcg(src + (size_t)(c0 + j) * kTileN) : 0.f;
            }
#pragma unroll
            for (int u = 0; u < 3; ++u)
              if (s + u < tc.n_seg) {
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] += t[u][j];
              }
          }
          epilogue16(a, o, ctl, sg.tile, q, lane, c0, v, ss_buf);
        }
        if (resid) { finish_ss(a, ctl, sg.tile, wtid, ss_buf); ss_buf ^= 1; }
      }
    };

    // ---- phase 0: embedding rows -> x, un-normalised activations, sums of squares -----------------
    {
      OpInfo o{};
      o.op = OP_EMBED; o.layer = 0;
      const int Td = a.d / kTileN;
      if (c == 0 && wtid < a.in.M) a.amax[wtid] = 0ull;
      for (int tile = (int)c; tile < Td; tile += (int)n) {
        for (int c0 = 16 * half; c0 < a.Mc; c0 += 32) {
          if (c0 >= a.in.M) break;
          float v[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int m = c0 + j;
            v[j] = (m < a.in.M) ? __bfloat162float(a.embed[(size_t)a.in.tokens[m] * a.d + tile * kTileN + q * 32 + lane]) : 0.f;
          }
          epilogue16(a, o, ctl, tile, q, lane, c0, v, ss_buf);
        }
        finish_ss(a, ctl, tile, wtid, ss_buf);
        ss_buf ^= 1;
      }
      phase_done();
    }

    for (int l = 0; l < a.n_layers && ok; ++l) {
      run_gemm(4 * l + OP_QKV);
      if (!ok) break;
      phase_done();
      // ---- attention ----------------------------------------------------------------------------
      if (!wait_phases(phase)) { ok = false; break; }
      {
        const int n_units = a.n_attn_tiles * a.Hkv * a.attn_splits;
        for (int u = (int)c; u < n_units; u += (int)n) {
          const int split = u % a.attn_splits;
          const int kh = (u / a.attn_splits) % a.Hkv;
          const int tile = u / (a.attn_splits * a.Hkv);
          if (a.hd == 128) attn_unit<128>(a, l, attn_sm, tile, kh, split, widx, lane, wtid);
          else attn_unit<64>(a, l, attn_sm, tile, kh, split, widx, lane, wtid);
        }
      }
      fence_proxy_async_all();   // generic-proxy use of the staging area is over before TMA writes there again
      worker_sync();
      if (wtid == 0) *reinterpret_cast<volatile int *>(&ctl->attn_epoch) = l + 1;
      phase_done();
      // ---- merge --------------------------------------------------------------------------------
      if (!wait_phases(phase)) { ok = false; break; }
      {
        const int n_units = a.in.M * a.Hq;
        for (int u = (int)c * 8 + widx; u < n_units; u += (int)n * 8) {
          if (a.hd == 128) merge_unit<128>(a, u / a.Hq, u % a.Hq, lane);
          else merge_unit<64>(a, u / a.Hq, u % a.Hq, lane);
        }
      }
      phase_done();
      run_gemm(4 * l + OP_O);
      if (!ok) break;
      phase_done();
      run_gemm(4 * l + OP_GU);
      if (!ok) break;
      phase_done();
      run_gemm(4 * l + OP_D);
      if (!ok) break;
      phase_done();
    }
    if (ok && !a.skip_lm) {
      run_gemm(4 * a.n_layers);
      if (ok) {
        phase_done();
        // ---- acceptance: one CTA per sequence ---------------------------------------------------
        if ((int)c < a.in.B && wait_phases(phase)) {
          const int r0 = a.in.cu_rows[c], r1 = a.in.cu_rows[c + 1];
          for (int r = r0 + wtid; r < r1; r += kWorkers)
            a.out_argmax[r] = (int32_t)(0xFFFFFFFFu - (uint32_t)(__ldcg(a.amax + r) & 0xFFFFFFFFull));
          worker_sync();
          if (wtid == 0) {
            const int k = r1 - r0;
            int acc = 0;
            while (acc < k - 1 && a.out_argmax[r0 + acc] == a.in.tokens[r0 + acc + 1]) ++acc;
            a.out_accept[c] = acc;
            int32_t *em = a.out_emitted + (size_t)c * a.k_max;
            for (int j = 0; j < acc; ++j) em[j] = a.in.tokens[r0 + j + 1];
            em[acc] = a.out_argmax[r0 + acc];
            a.out_newlen[c] = a.in.seq_len[c] + acc + 1;   // rejected rows stay in their pages, uncounted
            a.out_newpend[c] = a.out_argmax[r0 + acc];
          }
        }
      }
    }
  }

  // ---- exit: free tensor memory; the last CTA out rewinds the counters for the next launch ----------
  tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    tc_fence_after();
    tmem_dealloc(tmem_base, alloc_cols);
  }
  if (threadIdx.x == 0) {
    __threadfence();
    const int old = atomicAdd(a.sync + 2, 1);
    if (old == (int)n - 1 && *reinterpret_cast<volatile int *>(err) == 0) {
      for (int i = 0; i < a.n_counters; ++i) a.sync[8 + i] = 0;
      a.sync[0] = 0;
      a.sync[2] = 0;
      __threadfence();
    }
  }
}

// ---- host side ----------------------------------------------------------------------------------------------
size_t fused_attn_smem_bytes(int hd) { return (size_t)kAttnRows * hd * 2 + (size_t)4 * kAttnBlk * hd * 2; }

int fused_ring_stages(int planes, int Mc, int hd, size_t smem_limit) {
  const size_t stage = kWBytes + (size_t)planes * Mc * kBlockK * 2;
  const size_t fixed = 1024 + sizeof(FusedCtl) + 256;
  if (smem_limit < fixed + fused_attn_smem_bytes(hd) + 2 * stage) return 0;
  return (int)std::min<size_t>(kMaxRing, (smem_limit - fixed) / stage);
}

cudaError_t launch_fused(FusedArgs a, size_t smem_limit, cudaStream_t st) {
  static bool attr_done = false;
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(fused_verify_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_limit);
    if (e != cudaSuccess) return e;
    attr_done = true;
  }
  a.ring = fused_ring_stages(a.planes, a.Mc, a.hd, smem_limit);
  if (a.ring < 2) return cudaErrorInvalidConfiguration;
  a.attn_smem_bytes = (int)fused_attn_smem_bytes(a.hd);
  const size_t stage = kWBytes + (size_t)a.planes * a.Mc * kBlockK * 2;
  const size_t smem = 1024 + (size_t)a.ring * stage + sizeof(FusedCtl) + 256;
  void *params[] = {&a};
  return cudaLaunchCooperativeKernel((const void *)fused_verify_kernel, dim3(a.n_ctas), dim3(kThreads), params, smem, st);
}

}  // namespace ts
