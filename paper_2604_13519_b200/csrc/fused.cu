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
//              warps 3..10  workers: epilogues out of tensor memory, tile fix-up, the softmax of attention
//                      (both attention products run on tcgen05 as well, see below), merge, acceptance.
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
static constexpr int kKvStages = 4;     // K/V blocks in flight per CTA during attention

enum : int { OP_QKV = 0, OP_O = 1, OP_GU = 2, OP_D = 3, OP_LM = 4, OP_EMBED = 5 };

struct __align__(16) FusedCtl {
  uint64_t full[kMaxRing];
  uint64_t empty[kMaxRing];
  uint64_t tmem_full[kAccBufs];
  uint64_t tmem_empty[kAccBufs];
  uint32_t tmem_base;
  int flag;
  int attn_epoch;            // attention phases this CTA has finished (ring slots under the staging area are free)
  // attention pipeline: K/V stages (TMA -> MMA), Q tile, score / probability / output-block buffers
  uint64_t kv_full[kKvStages], kv_empty[kKvStages], q_full;
  uint64_t s_full[2], s_empty[2], p_full[2], o_full[2], o_empty[2];
  float l_half[kAttnRows];
  int row_pos[kMaxMc];       // absolute position of each row
  int row_page[kMaxMc];      // KV page holding that position
  float r_s[kMaxMc];
  float ss_acc[2][4][kMaxMc];
  FusedArgs args;            // copy of the kernel arguments: cheap to read from the out-of-line device functions
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

// ---- attention ----------------------------------------------------------------------------------------------
// One unit = (128-row tile of packed (position, query head) rows, kv head, split of the KV positions).
// Both products run on tcgen05:  S = Q K^T  (A = Q tile, B = K block, both K-major fp16 in shared memory,
// D = 128 x 64 fp32 in tensor memory), then the worker threads (one row each) take the running max, write
// P = exp2(S - max) back to tensor memory as fp16, and  O_blk = P V  (A = P from tensor memory, B = the V block
// read MN-major from the same [position][64 elements] image K uses).  The workers add O_blk into registers
// with the usual running-softmax rescale.  K/V blocks of 64 positions arrive by TMA straight from the pages.
struct AttnUnit {
  int tile, kh, split;
  int seq, row0, rows_here, r_beg, len, G;
  int pos_beg, pos_end, nblk;
};

__device__ __forceinline__ AttnUnit attn_unit_info(const FusedArgs &a, int u) {
  AttnUnit t;
  t.split = u % a.attn_splits;
  t.kh = (u / a.attn_splits) % a.Hkv;
  t.tile = u / (a.attn_splits * a.Hkv);
  t.G = a.Hq / a.Hkv;
  t.seq = a.tile_seq[t.tile];
  t.row0 = a.tile_row0[t.tile];
  t.r_beg = a.in.cu_rows[t.seq];
  const int k_i = a.in.cu_rows[t.seq + 1] - t.r_beg;
  t.len = a.in.seq_len[t.seq];
  t.rows_here = min(kAttnRows, k_i * t.G - t.row0);
  const int total = t.len + k_i;
  const int j_max = (t.row0 + t.rows_here - 1) / t.G;
  // (nothing beyond the last row's own position is visible)
  split_positions(t.len, min(total, t.len + j_max + 1), a.attn_splits, t.split, 4, &t.pos_beg, &t.pos_end);
  t.nblk = t.pos_end > t.pos_beg ? (t.pos_end - t.pos_beg + kAttnBlk - 1) / kAttnBlk : 0;
  return t;
}

// tensor-memory columns of the attention phase (they lie over the projection accumulators, which are idle then)
static constexpr int kColS = 0;      // two score buffers of 64 columns
static constexpr int kColP = 128;    // two probability buffers of 32 columns (fp16 pairs)
static constexpr int kColO = 192;    // two output-block buffers of head_dim columns

__device__ __forceinline__ void cp_async16z(uint32_t dst, const void *src, bool valid) {
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_commit_wait_all() {
  asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ uint32_t pack_h2(float x, float y) {
  __half2 v = __floats2half2_rn(x, y);
  return *reinterpret_cast<uint32_t *>(&v);
}

// Worker side of one unit.  Thread <-> row (tensor-memory lane q*32 + lane); the two warps that share a lane
// quarter split the exponentials (32 positions each) and the output columns (head_dim / 2 each).
// `blk` counts K/V blocks over all units of this CTA (buffer index and barrier parity come from it).
template <int HD>
__device__ __noinline__ bool attn_unit_workers(const FusedArgs &a, FusedCtl *ctl, const AttnUnit &t, uint8_t *sQ, uint32_t tmem_base,
                                               int q, int half, int lane, int wtid, uint32_t &blk, uint32_t unit_no,
                                               const int *err) {
  constexpr int CH = HD / 8;          // 16-byte chunks per row
  constexpr int OC = HD / 2;          // output columns per thread
  const int row = q * 32 + lane;      // row of the tile
  const int pr = t.row0 + row;        // packed row of the sequence
  const bool valid = row < t.rows_here;
  const int j = valid ? pr / t.G : 0, gq = valid ? pr % t.G : 0;
  const size_t ob = ((size_t)(t.r_beg + j) * a.Hq + t.kh * t.G + gq) * a.attn_splits + t.split;
  if (t.nblk == 0) {   // nothing visible in this split: mark it empty
    if (valid && half == 0) a.attn_ml[ob] = make_float2(-INFINITY, 0.f);
    return true;
  }
  // ---- stage Q: [128 rows][64 elements] images with the 128-byte swizzle, one per 64-element half ----------
  for (int idx = wtid; idx < kAttnRows * CH; idx += kWorkers) {
    const int r = idx / CH, c = idx % CH;
    const int prr = t.row0 + r;
    const bool v = r < t.rows_here;
    const int jj = v ? prr / t.G : 0, gg = v ? prr % t.G : 0;
    const __half *src = a.q + ((size_t)(t.r_beg + jj) * a.Hq + t.kh * t.G + gg) * HD + c * 8;
    const uint32_t dst = smem_u32(sQ) + (c >> 3) * (kAttnRows * 128) + r * 128 + (((c & 7) ^ (r & 7)) << 4);
    cp_async16z(dst, src, v);
  }
  cp_commit_wait_all();
  fence_proxy_async_all();   // generic-proxy writes -> tcgen05 (async proxy) reads
  worker_sync();
  if (wtid == 0) mbar_arrive(smem_u32(&ctl->q_full));

  const uint32_t tq = tmem_base + ((uint32_t)(q * 32) << 16);
  const int lim = min(t.len + j, t.pos_end - 1);   // last visible position of this row
  const float scale = rsqrtf((float)HD) * 1.4426950408889634f;
  float acc[OC];
#pragma unroll
  for (int i = 0; i < OC; ++i) acc[i] = 0.f;
  float m_run = -INFINITY, l_run = 0.f, f_pending = 0.f;
  bool ok = true;

  auto consume_o = [&](uint32_t bi, float f) {   // acc = acc * f + O_blk
    const uint32_t buf = bi & 1;
    if (ok && !mbar_wait_err(smem_u32(&ctl->o_full[buf]), (bi >> 1) & 1, err)) { ok = false; atomicCAS((int *)err, 0, DEV_TIMEOUT_TMEM); }
    tc_fence_after();
#pragma unroll
    for (int i = 0; i < OC / 16; ++i) {
      uint32_t r[16];
      tmem_ld16(tq + kColO + buf * HD + half * OC + i * 16, r);
      tmem_wait_ld();
#pragma unroll
      for (int e = 0; e < 16; ++e) acc[i * 16 + e] = acc[i * 16 + e] * f + __uint_as_float(r[e]);
    }
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&ctl->o_empty[buf]));
  };

  for (int b = 0; b < t.nblk; ++b, ++blk) {
    const uint32_t buf = blk & 1;
    if (ok && !mbar_wait_err(smem_u32(&ctl->s_full[buf]), (blk >> 1) & 1, err)) { ok = false; atomicCAS((int *)err, 0, DEV_TIMEOUT_TMEM); }
    tc_fence_after();
    const int p_base = t.pos_beg + b * kAttnBlk;
    float mine[32];
    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint32_t r[16];
      tmem_ld16(tq + kColS + buf * 64 + i * 16, r);
      tmem_wait_ld();
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        const float sv = (p_base + i * 16 + e <= lim) ? __uint_as_float(r[e]) * scale : -INFINITY;
        mx = fmaxf(mx, sv);
        if ((i >> 1) == half) mine[(i & 1) * 16 + e] = sv;
      }
    }
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&ctl->s_empty[buf]));
    const float m_new = fmaxf(m_run, mx);
    const float ref = (m_new == -INFINITY) ? 0.f : m_new;
    const float f = exp2f(m_run - ref);   // exp2(-inf) = 0 on the first block
    m_run = m_new;
    uint32_t pk[16];
    float sum = 0.f;
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      const float e0 = exp2f(mine[2 * e] - ref), e1 = exp2f(mine[2 * e + 1] - ref);
      sum += e0 + e1;
      pk[e] = pack_h2(e0, e1);
    }
    l_run = l_run * f + sum;
    // the P buffer is free: the product that read it two blocks ago was seen complete when its O_blk was taken
    tmem_st16(tq + kColP + buf * 32 + half * 16, pk);
    tmem_wait_st();
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&ctl->p_full[buf]));
    if (b > 0) consume_o(blk - 1, f_pending);
    f_pending = f;
  }
  consume_o(blk - 1, f_pending);
  if (!worker_all(ok)) return false;

  // ---- partial result of this split: un-normalised output, running max (log2 domain), sum -----------------
  if (half == 1) ctl->l_half[row] = l_run;
  worker_sync();
  if (valid) {
    if (half == 0) a.attn_ml[ob] = make_float2(m_run, l_run + ctl->l_half[row]);
    float4 *dst = reinterpret_cast<float4 *>(a.attn_o + ob * HD + half * OC);
#pragma unroll
    for (int i = 0; i < OC / 4; ++i) dst[i] = make_float4(acc[4 * i], acc[4 * i + 1], acc[4 * i + 2], acc[4 * i + 3]);
  }
  return true;
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
  // eight splits' loads in flight at a time (an empty split never wrote its slot: it is not read)
  for (int s0 = 0; s0 < S; s0 += 8) {
    float ws[8];
    float t[8][EPL];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      ws[u] = __shfl_sync(0xffffffffu, w, (s0 + u) & 31);
      if (s0 + u >= S) ws[u] = 0.f;
      const float *src = a.attn_o + (base + s0 + u) * HD + lane * EPL;
      if constexpr (EPL == 4) {
        float4 x4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (ws[u] != 0.f) x4 = __ldcg(reinterpret_cast<const float4 *>(src));
        t[u][0] = x4.x; t[u][1] = x4.y; t[u][2] = x4.z; t[u][3] = x4.w;
      } else {
        float2 x2 = make_float2(0.f, 0.f);
        if (ws[u] != 0.f) x2 = __ldcg(reinterpret_cast<const float2 *>(src));
        t[u][0] = x2.x; t[u][1] = x2.y;
      }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u)
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[e] += ws[u] * t[u][e];
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
  // all of tensor memory: the projection accumulators (kAccBufs * ncols columns) and, over them, the
  // attention buffers (kColO + 2 * head_dim columns)
  const uint32_t alloc_cols = 512;
  int *ctr = a.sync, *err = a.err;
  const int n_gemms = 4 * a.n_layers + (a.skip_lm ? 0 : 1);

  for (int i = threadIdx.x; i < (int)(sizeof(FusedArgs) / 4); i += kThreads)
    reinterpret_cast<uint32_t *>(&ctl->args)[i] = reinterpret_cast<const uint32_t *>(&a)[i];
  if (threadIdx.x == 0) {
    for (int s = 0; s < R; ++s) {
      mbar_init(smem_u32(&ctl->full[s]), 2);    // weight producer + activation producer
      mbar_init(smem_u32(&ctl->empty[s]), 1);   // tcgen05.commit
    }
    for (int b = 0; b < kAccBufs; ++b) {
      mbar_init(smem_u32(&ctl->tmem_full[b]), 1);
      mbar_init(smem_u32(&ctl->tmem_empty[b]), 8);   // one arrival per worker warp
    }
    for (int b = 0; b < kKvStages; ++b) {
      mbar_init(smem_u32(&ctl->kv_full[b]), 1);    // producer's expect_tx arrival
      mbar_init(smem_u32(&ctl->kv_empty[b]), 1);   // tcgen05.commit after P V
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&ctl->s_full[b]), 1);
      mbar_init(smem_u32(&ctl->s_empty[b]), 8);
      mbar_init(smem_u32(&ctl->p_full[b]), 8);
      mbar_init(smem_u32(&ctl->o_full[b]), 1);
      mbar_init(smem_u32(&ctl->o_empty[b]), 8);
    }
    mbar_init(smem_u32(&ctl->q_full), 1);
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
            // one block of the stored matrix = 16 contiguous KB = rows w_block(tile, kb) * 128 .. of a [.][64] array
            tma_load_2d(smem_u32(smem + (size_t)s * stage_bytes), &a.maps[o.map_w], 0, w_block(sg.tile, kb, o.T, o.KB) * kTileN, bar, pol_w);
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
      uint32_t blk = 0;
      for (int g = 0; g < n_gemms && ok; ++g) {
        const OpInfo o = gemm_op(a, g);
        if (o.op == OP_O) {
          // ---- attention of this layer: stream the K/V blocks of this CTA's units ---------------------
          ok = grid_wait(ctr, (o.phase - 2) * (int)n, err);   // the QKV phase (rotary, KV append) is complete everywhere
          if (!ok) { atomicCAS(err, 0, DEV_TIMEOUT_GRID); break; }
          fence_proxy_async_all();
          const int n_units = a.n_attn_tiles * a.Hkv * a.attn_splits;
          const int halves = a.hd / 64;
          const uint32_t kv_bytes = 2u * kAttnBlk * a.hd * 2;
          for (int u = (int)c; u < n_units && ok; u += (int)n) {
            const AttnUnit t = attn_unit_info(a, u);
            const int32_t *btab = a.in.block_tab + (size_t)t.seq * a.in.pages_per_seq;
            for (int b = 0; b < t.nblk; ++b, ++blk) {
              const uint32_t st = blk % kKvStages;
              if (!mbar_wait_err(smem_u32(&ctl->kv_empty[st]), ((blk / kKvStages) & 1) ^ 1, err)) { ok = false; atomicCAS(err, 0, DEV_TIMEOUT_EMPTY); break; }
              const uint32_t bar = smem_u32(&ctl->kv_full[st]);
              mbar_expect_tx(bar, kv_bytes);
              uint8_t *sK = attn_sm + kAttnRows * a.hd * 2 + st * kv_bytes, *sV = sK + kAttnBlk * a.hd * 2;
              for (int pg = 0; pg < kAttnBlk / 16; ++pg) {
                // a page past the split's end is never visible; load the last visible page again instead
                const int pos = min(t.pos_beg + b * kAttnBlk + pg * 16, t.pos_end - 1);
                const int page = btab[pos >> 4];
                for (int hh = 0; hh < halves; ++hh) {
                  const uint32_t off = hh * (kAttnBlk * 128) + pg * 2048;
                  tma_load_5d(smem_u32(sK + off), &a.maps[a.map_kv], hh * 64, 0, t.kh, page, 2 * o.layer, bar, pol_a);
                  tma_load_5d(smem_u32(sV + off), &a.maps[a.map_kv], hh * 64, 0, t.kh, page, 2 * o.layer + 1, bar, pol_a);
                }
              }
            }
          }
          if (!ok) break;
        }
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
      uint32_t blk = 0, unit_no = 0;
      const uint32_t idesc_qk = umma_idesc_f16(kAttnRows, kAttnBlk, 0);
      const uint32_t idesc_pv = umma_idesc_f16(kAttnRows, (uint32_t)a.hd, 1);
      for (int g = 0; g < n_gemms && ok; ++g) {
        const OpInfo o = gemm_op(a, g);
        if (o.op == OP_O) {
          // ---- attention of this layer --------------------------------------------------------------
          const int n_units = a.n_attn_tiles * a.Hkv * a.attn_splits;
          const int halves = a.hd / 64;
          const uint32_t kv_bytes = 2u * kAttnBlk * a.hd * 2;
          const uint32_t sQ = smem_u32(attn_sm);
          auto issue_pv = [&](uint32_t bi) -> bool {   // O_blk = P V for block number bi
            const uint32_t pb = bi & 1;
            if (!mbar_wait_err(smem_u32(&ctl->p_full[pb]), (bi >> 1) & 1, err)) return false;
            if (!mbar_wait_err(smem_u32(&ctl->o_empty[pb]), ((bi >> 1) & 1) ^ 1, err)) return false;
            tc_fence_after();
            const uint32_t vst = bi % kKvStages;
            const uint32_t sV = sQ + kAttnRows * a.hd * 2 + vst * kv_bytes + kAttnBlk * a.hd * 2;
#pragma unroll
            for (int ks = 0; ks < kAttnBlk / 16; ++ks)   // 16 positions per instruction
              umma_f16_ts(tmem_base + kColO + pb * a.hd, tmem_base + kColP + pb * 32 + ks * 8,
                          umma_desc_sw128_mn(sV + ks * 2048, kAttnBlk * 128), idesc_pv, ks > 0 ? 1u : 0u);
            umma_commit(smem_u32(&ctl->o_full[pb]));
            umma_commit(smem_u32(&ctl->kv_empty[vst]));
            return true;
          };
          for (int u = (int)c; u < n_units && ok; u += (int)n) {
            const AttnUnit t = attn_unit_info(a, u);
            if (t.nblk == 0) continue;
            if (!mbar_wait_err(smem_u32(&ctl->q_full), unit_no & 1, err)) { ok = false; break; }
            ++unit_no;
            for (int b = 0; b < t.nblk && ok; ++b, ++blk) {
              const uint32_t kst = blk % kKvStages, st = blk & 1;
              if (!mbar_wait_err(smem_u32(&ctl->kv_full[kst]), (blk / kKvStages) & 1, err)) { ok = false; break; }
              if (!mbar_wait_err(smem_u32(&ctl->s_empty[st]), ((blk >> 1) & 1) ^ 1, err)) { ok = false; break; }
              tc_fence_after();
              const uint32_t sK = sQ + kAttnRows * a.hd * 2 + kst * kv_bytes;
              for (int hh = 0; hh < halves; ++hh) {
                const uint64_t dq = umma_desc_sw128(sQ + hh * (kAttnRows * 128)), dk = umma_desc_sw128(sK + hh * (kAttnBlk * 128));
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                  umma_bf16(tmem_base + kColS + st * 64, dq + 2 * kk, dk + 2 * kk, idesc_qk, (hh | kk) != 0 ? 1u : 0u);
              }
              umma_commit(smem_u32(&ctl->s_full[st]));
              if (b > 0) ok = issue_pv(blk - 1);
            }
            if (ok) ok = issue_pv(blk - 1);
          }
          if (!ok) break;
        }
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
    uint32_t seg = 0, attn_blk = 0;
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
        for (int u = (int)c; u < n_units && ok; u += (int)n) {
          const AttnUnit t = attn_unit_info(a, u);
          ok = (a.hd == 128) ? attn_unit_workers<128>(ctl->args, ctl, t, attn_sm, tmem_base, q, half, lane, wtid, attn_blk, 0, err)
                             : attn_unit_workers<64>(ctl->args, ctl, t, attn_sm, tmem_base, q, half, lane, wtid, attn_blk, 0, err);
        }
        if (!ok) break;
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
// Q tile + kKvStages stages of (K block, V block)
size_t fused_attn_smem_bytes(int hd) { return (size_t)kAttnRows * hd * 2 + (size_t)kKvStages * 2 * kAttnBlk * hd * 2; }

int fused_ring_stages(int planes, int Mc, int hd, size_t smem_limit) {
  const size_t stage = kWBytes + (size_t)planes * Mc * kBlockK * 2;
  const size_t fixed = 1024 + sizeof(FusedCtl) + 256;
  if (smem_limit < fixed + 2 * stage) return 0;
  const size_t ring = std::min<size_t>(kMaxRing, (smem_limit - fixed) / stage);
  return ring * stage >= fused_attn_smem_bytes(hd) ? (int)ring : 0;   // the attention staging area lies over the ring
}

cudaError_t launch_fused(FusedArgs a, size_t smem_limit, cudaStream_t st) {
  static PerDeviceOnce once;
  int dev_ = -1;
  if (once.needed(&dev_)) {
    cudaError_t e = cudaFuncSetAttribute(fused_verify_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_limit);
    if (e != cudaSuccess) return e;
    once.done(dev_);
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
