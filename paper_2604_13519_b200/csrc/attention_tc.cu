// Paged grouped-query attention of the verify chunk on the 5th-generation tensor cores, as a kernel of its own.
//
// One unit = (128-row tile of packed (position, query head) rows, kv head, leaf of the KV positions); a CTA takes one
// unit when the step has no more units than SMs, else it walks several (tensor memory, barriers and the K/V ring are
// set up once and the ring keeps running across units).
//   warp 0   K/V producer: TMA loads of 64-position blocks straight from the pages (5-d tensor map over the pool)
//   warp 1   tensor memory allocation + tcgen05.mma issue:  S = Q K^T  (the unit's queries sit in tensor memory as
//            the row operand -- re-reading a 128-row query tile from shared memory for every 64-position block was
//            what bounded the kernel -- the K block K-major in shared memory, 128 x 64 fp32 result in tensor
//            memory), then  O_blk = P V  with P read from tensor memory (fp16) and the V block read MN-major from
//            the same [position][64 elements] image K uses
//   warps 2..5  one row per thread: maximum over the block's 64 scores, P = exp2(S - reference maximum) written back
//            to tensor memory as an fp16 (value, rounding remainder) pair -- the second product adds both, so the 11
//            bits of fp16 do not limit the weights (a single fp16 P was the largest error of the whole step).  The
//            output sums stay in tensor memory (every P V adds to them); the reference maximum follows the running
//            one in steps, and only then is the row of sums multiplied down
// Each leaf writes an un-normalised partial output with its (max, sum); attn_merge_kernel adds a row's leaves.
// Every wait is bounded; on expiry the CTA records an error word and leaves through the normal exit.
#include <cuda_fp16.h>

#include <algorithm>

#include "kernels.h"
#include "schedule.h"

namespace ts {

static constexpr int kAttnRows = 128;   // packed rows per unit
static constexpr int kAttnBlk = 64;     // kv positions per block
static constexpr int kKvStages = 6;     // K/V blocks in the ring (three are held by issued products, the rest are in flight)
static constexpr int kTcThreads = 192;
static constexpr int kWorkers = 128;
static constexpr int kWorkerWarp0 = 2;

struct __align__(16) AttnCtl {
  uint64_t kv_full[kKvStages], kv_empty[kKvStages], q_full;
  uint64_t s_full[2], s_empty[2], p_full[2], pv_done[2], o_free;
  uint32_t tmem_base;
};

__device__ __forceinline__ void worker_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ bool worker_all(bool ok) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %1, 0;\n\tbar.red.and.pred q, 1, 128, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(r)
      : "r"((uint32_t)ok)
      : "memory");
  return r != 0;
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
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

struct AttnUnit {
  int tile, kh, leaf;
  int seq, row0, rows_here, r_beg, len, G;
  int pos_beg, pos_end, nblk;
};

// The j-th unit of CTA c out of G: units are listed longest first and dealt out in rounds of G, every other round in
// reverse CTA order, so that the CTA given the longest unit of one round gets the shortest of the next.
__device__ __forceinline__ int attn_unit_of(int c, int j, int G) { return j * G + ((j & 1) ? G - 1 - c : c); }

// Unit u works on pair u / Hkv (a row tile and one leaf of its sequence) for kv head u % Hkv.  The leaf's positions
// are [leaf * leaf_len, (leaf + 1) * leaf_len), cut off at the end of the chunk: absolute positions, so the blocks a
// row meets, and their order, do not depend on where the chunk starts or how long it is.
__device__ __forceinline__ AttnUnit attn_unit_info(const AttnTcArgs &a, int u) {
  AttnUnit t;
  const int pair = u / a.Hkv;
  t.kh = u - pair * a.Hkv;
  t.tile = a.unit_tile[pair];
  t.leaf = a.unit_leaf[pair];
  t.G = a.Hq / a.Hkv;
  t.seq = a.tile_seq[t.tile];
  if (!ts_in_range(a.in.ck, CHK_UNIT, t.seq, a.in.B) || !ts_in_range(a.in.ck, CHK_UNIT, t.leaf, a.n_slots)) {
    t.seq = 0;   // (debug build: the failed check is on record; go on with indices that are in range)
    t.leaf = 0;
  }
  t.row0 = a.tile_row0[t.tile];
  t.r_beg = a.in.cu_rows[t.seq];
  const int k_i = a.in.cu_rows[t.seq + 1] - t.r_beg;
  t.len = a.in.seq_len[t.seq];
  t.rows_here = min(kAttnRows, k_i * t.G - t.row0);
  t.pos_beg = t.leaf * a.leaf_len;
  t.pos_end = min(t.pos_beg + a.leaf_len, t.len + k_i);
  t.nblk = t.pos_end > t.pos_beg ? (t.pos_end - t.pos_beg + kAttnBlk - 1) / kAttnBlk : 0;
  return t;
}

// tensor-memory columns of the attention phase (they lie over the projection accumulators, which are idle then)
static constexpr int kColS = 0;      // two score buffers of 64 columns
static constexpr int kColP = 128;    // two probability buffers of 32 columns (fp16, two per column)
static constexpr int kColO = 192;    // the output sums: head_dim columns, accumulated over the unit's blocks
static constexpr int kColPL = 448;   // the probabilities' rounding remainders: two buffers of 32 columns
static constexpr int kColQ = 320;    // the unit's queries, fp16 pairs: head_dim / 2 columns of values, then as many of remainders
static constexpr float kRescaleStep = 8.f;   // the reference maximum follows the running one in steps of 2^8

// 2^x for x <= 0 (and 0 for -inf); tiny results flush to zero
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float y;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
  return y;
}
__device__ __forceinline__ uint32_t pack_h2(float x, float y) {
  __half2 v = __floats2half2_rn(x, y);
  return *reinterpret_cast<uint32_t *>(&v);
}

// Worker side of one unit.  Thread <-> row (tensor-memory lane q*32 + lane): it takes the row maximum over the
// block's 64 scores, writes the 64 probabilities back as fp16 and, rarely, rescales the row's output sums.
// `blk` counts K/V blocks over all units of this CTA (buffer index and barrier parity come from it).
template <int HD>
__device__ __forceinline__ bool attn_unit_workers(const AttnTcArgs &a, AttnCtl *ctl, const AttnUnit &t, uint32_t tmem_base,
                                                  int q, int lane, int wtid, uint32_t &blk, bool &waited, const int *err) {
  const int row = q * 32 + lane;      // row of the tile
  const int pr = t.row0 + row;        // packed row of the sequence
  const bool valid = row < t.rows_here;
  const int j = valid ? pr / t.G : 0, gq = valid ? pr % t.G : 0;
  const size_t ob = ((size_t)(t.r_beg + j) * a.Hq + t.kh * t.G + gq) * a.n_slots + t.leaf;
  // (a step input like the unit tables: read before the dependency wait)
  const unsigned long long anc = ((unsigned long long)a.in.anc[2 * (t.r_beg + j) + 1] << 32) | a.in.anc[2 * (t.r_beg + j)];
  // the rotated queries come from the previous kernel; everything above was on the device before the step began
  if (!waited) {
    pdl_wait();
    waited = true;
    if (wtid == 0) stamp_waited(a.stamp);
  }
  if (t.nblk == 0) {   // no position in this leaf: mark it empty
    if (valid) a.attn_ml[ob] = make_float2(-INFINITY, 0.f);
    return true;
  }
  // ---- stage Q into tensor memory: the score product reads its row operand there (thread <-> row, an fp16 pair
  // per column: head_dim / 2 columns of values, then as many of rounding remainders), so per block only the keys
  // and values come through shared memory.  Every score product of the CTA's previous unit has completed (its
  // last scores were read before that unit's sums were drained), so the columns may be overwritten.
  const uint32_t tq = tmem_base + ((uint32_t)(q * 32) << 16);
  {
    const size_t so = ((size_t)(t.r_beg + j) * a.Hq + t.kh * t.G + gq) * HD;
    // all loads of both planes are issued before the first use: one round trip to L2, where the previous kernel has
    // just written the rows
    // (32 bytes per lane and load: the lanes of a warp read 32 different rows)
    uint32_t v[2][HD / 2];
    if (valid) {
#pragma unroll
      for (int c = 0; c < HD / 16; ++c) {
        ld_global_v8(a.q + so + c * 16, &v[0][c * 8]);
        ld_global_v8(a.q_lo + so + c * 16, &v[1][c * 8]);
      }
    } else {
#pragma unroll
      for (int c = 0; c < HD / 2; ++c) v[0][c] = v[1][c] = 0u;
    }
#pragma unroll
    for (int pl = 0; pl < 2; ++pl) {
#pragma unroll
      for (int c4 = 0; c4 < HD / 32; ++c4) {
        uint32_t r[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) r[e] = v[pl][c4 * 16 + e];
        tmem_st16(tq + kColQ + pl * (HD / 2) + c4 * 16, r);
      }
    }
    tmem_wait_st();
  }
  tc_fence_before();
  worker_sync();
  if (wtid == 0) mbar_arrive(smem_u32(&ctl->q_full));

  // Visibility: the whole cache, and of the chunk the rows named by this row's mask (itself and its ancestors in
  // the draft tree; in a chain, rows 0..j), up to the end of this split.
  const int lim_all = min(t.len, t.pos_end) - 1;   // every row sees every position up to here
  const float scale = rsqrtf((float)HD) * 1.4426950408889634f;
  // The output sums stay in tensor memory: every product P V adds to them.  Probabilities are taken against a
  // reference maximum m_ref that follows the running maximum lazily: only when a block's maximum exceeds it by
  // more than kRescaleStep (in the log2 domain) is the row of sums multiplied down and m_ref raised, so in most
  // blocks the softmax thread never touches the sums.  Until then probabilities may reach 2^kRescaleStep: well
  // inside fp16, and the sums are fp32.
  float m_ref = -INFINITY, l_run = 0.f;
  bool ok = true;

  for (int b = 0; b < t.nblk; ++b, ++blk) {
    const uint32_t buf = blk & 1;
    if (ok && !mbar_wait_err(smem_u32(&ctl->s_full[buf]), (blk >> 1) & 1, err)) { ok = false; atomicCAS((int *)err, 0, DEV_TIMEOUT_TMEM); }
    tc_fence_after();
    const int p_base = t.pos_beg + b * kAttnBlk;
    float sc[64];
    {
      uint32_t r0[16], r1[16], r2[16], r3[16];
      tmem_ld16(tq + kColS + buf * 64, r0);
      tmem_ld16(tq + kColS + buf * 64 + 16, r1);
      tmem_ld16(tq + kColS + buf * 64 + 32, r2);
      tmem_ld16(tq + kColS + buf * 64 + 48, r3);
      tmem_wait_ld();
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        sc[e] = __uint_as_float(r0[e]); sc[16 + e] = __uint_as_float(r1[e]);
        sc[32 + e] = __uint_as_float(r2[e]); sc[48 + e] = __uint_as_float(r3[e]);
      }
    }
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&ctl->s_empty[buf]));
    // a block every row sees whole needs no mask (all but the last blocks of a sequence's last split)
    if (p_base + kAttnBlk - 1 > lim_all) {
      // bit e of `vis`: position p_base + e is visible to this row (cache positions all, chunk rows by the mask,
      // nothing at or past the split's end)
      const int rel0 = p_base - t.len;                 // chunk row of the block's first position (negative: cache)
      unsigned long long vis;
      if (rel0 >= 0) vis = rel0 < 64 ? anc >> rel0 : 0ull;
      else if (rel0 > -64) vis = (anc << (-rel0)) | ((1ull << (-rel0)) - 1ull);
      else vis = ~0ull;
      const int n_in = t.pos_end - p_base;             // positions of the block inside the split
      if (n_in < 64) vis &= n_in > 0 ? (1ull << n_in) - 1ull : 0ull;
      const uint32_t vlo = (uint32_t)vis, vhi = (uint32_t)(vis >> 32);
#pragma unroll
      for (int e = 0; e < 32; ++e) {
        sc[e] = (vlo >> e) & 1u ? sc[e] : -INFINITY;
        sc[32 + e] = (vhi >> e) & 1u ? sc[32 + e] : -INFINITY;
      }
    }
    float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
    for (int e = 0; e < 64; e += 8) {   // three-input maxima: half the instructions of pairwise ones
      mx0 = max3(mx0, sc[e], sc[e + 1]); mx1 = max3(mx1, sc[e + 2], sc[e + 3]);
      mx2 = max3(mx2, sc[e + 4], sc[e + 5]); mx3 = max3(mx3, sc[e + 6], sc[e + 7]);
    }
    // block maximum in the log2 domain: scores times log2(e)/sqrt(head_dim), folded into one multiply-add per score
    const float m_blk = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * scale;
    const bool raise = m_blk > m_ref + kRescaleStep;   // (also the first finite maximum: m_ref starts at -inf)
    const float m_old = m_ref;
    if (raise) m_ref = m_blk;
    const float ref = (m_ref == -INFINITY) ? 0.f : m_ref;
    float sum0 = 0.f, sum1 = 0.f;
    uint32_t pk0[16], pk1[16], pl0[16], pl1[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      const float e0 = ex2_approx(fmaf(sc[2 * e], scale, -ref));
      const float e1 = ex2_approx(fmaf(sc[2 * e + 1], scale, -ref));
      const float e2 = ex2_approx(fmaf(sc[32 + 2 * e], scale, -ref));
      const float e3 = ex2_approx(fmaf(sc[32 + 2 * e + 1], scale, -ref));
      sum0 += e0 + e2; sum1 += e1 + e3;
      const __half2 h01 = __floats2half2_rn(e0, e1), h23 = __floats2half2_rn(e2, e3);
      pk0[e] = *reinterpret_cast<const uint32_t *>(&h01);
      pk1[e] = *reinterpret_cast<const uint32_t *>(&h23);
      pl0[e] = pack_h2(e0 - __low2float(h01), e1 - __high2float(h01));
      pl1[e] = pack_h2(e2 - __low2float(h23), e3 - __high2float(h23));
    }
    // This block's P buffer last fed product b - 2, which is complete: the scores of this block were committed after
    // it by the same thread, and a commit covers everything issued before it.  Only multiplying the sums down needs
    // more -- product b - 1 complete -- so that is the only case that waits.  The products of even and of odd blocks
    // complete phases of barriers of their own: a waiter is then never more than one phase behind (product b - 3,
    // the previous one on the same barrier, is known complete), which a parity wait needs.
    float f = 1.f;
    if (b > 0 && __any_sync(0xffffffffu, raise)) {       // tensor-memory accesses are warp-wide: lanes that stay use f = 1
      if (ok && !mbar_wait_err(smem_u32(&ctl->pv_done[(blk - 1) & 1u]), ((blk - 1) >> 1) & 1u, err)) { ok = false; atomicCAS((int *)err, 0, DEV_TIMEOUT_TMEM); }
      tc_fence_after();
      if (raise) f = ex2_approx(m_old - ref);            // exp2(-inf) = 0: nothing was summed before the first finite maximum
#pragma unroll
      for (int i = 0; i < HD / 32; ++i) {
        uint32_t r0[16], r1[16];
        tmem_ld16(tq + kColO + i * 32, r0);
        tmem_ld16(tq + kColO + i * 32 + 16, r1);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          r0[e] = __float_as_uint(__uint_as_float(r0[e]) * f);
          r1[e] = __float_as_uint(__uint_as_float(r1[e]) * f);
        }
        tmem_st16(tq + kColO + i * 32, r0);
        tmem_st16(tq + kColO + i * 32 + 16, r1);
      }
    }
    l_run = l_run * f + (sum0 + sum1);
    tmem_st16(tq + kColP + buf * 32, pk0);
    tmem_st16(tq + kColP + buf * 32 + 16, pk1);
    tmem_st16(tq + kColPL + buf * 32, pl0);
    tmem_st16(tq + kColPL + buf * 32 + 16, pl1);
    tmem_wait_st();
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&ctl->p_full[buf]));
    // (no CTA-wide barrier per block: a failed wait has set the error word, which ends every other wait)
  }
  // the unit's last product (and with it every earlier one)
  if (ok && !mbar_wait_err(smem_u32(&ctl->pv_done[(blk - 1) & 1u]), ((blk - 1) >> 1) & 1u, err)) { ok = false; atomicCAS((int *)err, 0, DEV_TIMEOUT_TMEM); }
  tc_fence_after();
  if (!worker_all(ok)) return false;

  // ---- partial result of this split: un-normalised output, its reference maximum (log2 domain), sum -------
  {
    float *dst = a.attn_o + ob * HD;
    if (valid) a.attn_ml[ob] = make_float2(m_ref, l_run);
#pragma unroll
    for (int i = 0; i < HD / 32; ++i) {
      uint32_t r0[16], r1[16];
      tmem_ld16(tq + kColO + i * 32, r0);      // (warp-wide: rows past the tile's end read too, and write nothing)
      tmem_ld16(tq + kColO + i * 32 + 16, r1);
      tmem_wait_ld();
      if (valid) {   // whole 32-byte sectors per lane: the lanes of a warp write 32 different rows
        st_global_v8(dst + i * 32, r0);
        st_global_v8(dst + i * 32 + 8, r0 + 8);
        st_global_v8(dst + i * 32 + 16, r1);
        st_global_v8(dst + i * 32 + 24, r1 + 8);
      }
    }
  }
  // the output sums are in registers / on their way to memory: the next unit's first product may overwrite them, and
  // its queries may be written over this unit's (every score product of this unit has completed)
  tc_fence_before();
  __syncwarp();
  if (lane == 0) mbar_arrive(smem_u32(&ctl->o_free));
  return true;
}

template <int HD>
__global__ void __launch_bounds__(kTcThreads, 1) attn_tc_kernel(const __grid_constant__ AttnTcArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  constexpr uint32_t kKvBytes = 2u * kAttnBlk * HD * 2, kHalves = HD / 64;
  AttnCtl *ctl = reinterpret_cast<AttnCtl *>(smem + kKvStages * kKvBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int *err = a.err;

  if (threadIdx.x == 0) {
    for (int b = 0; b < kKvStages; ++b) {
      mbar_init(smem_u32(&ctl->kv_full[b]), 1);
      mbar_init(smem_u32(&ctl->kv_empty[b]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&ctl->s_full[b]), 1);
      mbar_init(smem_u32(&ctl->s_empty[b]), 4);
      mbar_init(smem_u32(&ctl->p_full[b]), 4);
      mbar_init(smem_u32(&ctl->pv_done[b]), 1);
    }
    mbar_init(smem_u32(&ctl->q_full), 1);
    mbar_init(smem_u32(&ctl->o_free), 4);   // one arrival per worker warp
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&ctl->tmem_base), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  if (threadIdx.x == 0) stamp_min(a.stamp);
  pdl_launch_dependents();   // (this CTA holds its tensor memory; the dependent waits for this kernel's end anyway)
  // The step's integer inputs were copied in before the step's first kernel started, so they may be read here.
  // This CTA's units: attn_unit_of(blockIdx.x, 0, 1, 2, ...).  The three roles walk the units as three loops coupled only by the barriers, whose
  // phases are counted over all blocks (`gb`) and units (`un`) of the CTA.
  const int n_total = a.n_units * a.Hkv;

  if (warp == 0) {
    // ---------------------------------------------------------------- K/V producer
    // (the whole warp walks the loops and the waits; an elected lane issues a block's sixteen copies -- a lone lane
    // in a divergent branch needs about 50 cycles per copy instruction, more than half of a block's time)
    {
      const uint64_t pol = policy_evict_first();
      uint32_t gb = 0;
      bool waited = false, ok = true;
      for (int j = 0; j * (int)gridDim.x < n_total && ok; ++j) {
        const int u = attn_unit_of((int)blockIdx.x, j, (int)gridDim.x);
        if (u >= n_total) continue;
        const AttnUnit t = attn_unit_info(a, u);
        const int32_t *btab = a.in.block_tab + (size_t)t.seq * a.in.pages_per_seq;
        for (int b = 0; b < t.nblk; ++b, ++gb) {
          // blocks wholly inside the cache of earlier steps do not depend on the previous kernel: the ring is filled
          // with them before the dependency wait; the chunk's own K/V rows come from the previous kernel
          if (!waited && (gb >= (uint32_t)kKvStages || t.pos_beg + (b + 1) * kAttnBlk > t.len)) { pdl_wait(); waited = true; }
          const uint32_t st = gb % kKvStages;
          if (gb >= (uint32_t)kKvStages &&
              !__all_sync(0xffffffffu, mbar_wait_err(smem_u32(&ctl->kv_empty[st]), ((gb / kKvStages) & 1) ^ 1, err))) {
            if (lane == 0) atomicCAS(a.err, 0, DEV_TIMEOUT_EMPTY);
            ok = false;
            break;
          }
          const uint32_t bar = smem_u32(&ctl->kv_full[st]);
          uint8_t *sK = smem + st * kKvBytes, *sV = sK + kAttnBlk * HD * 2;
          // lane pg looks its page up (a page past the unit's end is never visible: the last visible page is loaded
          // again instead); the elected lane gets the four ids by shuffle
          int page = 0;
          if (lane < kAttnBlk / 16) {
            const int pos = min(t.pos_beg + b * kAttnBlk + lane * 16, t.pos_end - 1);
            page = btab[pos >> 4];
            if (!ts_in_range(a.in.ck, CHK_PAGE_ATTN, page, a.in.ck.max_pages)) page = 0;
          }
          int pages[kAttnBlk / 16];
#pragma unroll
          for (int pg = 0; pg < kAttnBlk / 16; ++pg) pages[pg] = __shfl_sync(0xffffffffu, page, pg);
          if (elect_one()) {
            mbar_expect_tx(bar, kKvBytes);
#pragma unroll
            for (int pg = 0; pg < kAttnBlk / 16; ++pg) {
#pragma unroll
              for (int hh = 0; hh < (int)kHalves; ++hh) {
                const uint32_t off = hh * (kAttnBlk * 128) + pg * 2048;
                tma_load_5d(smem_u32(sK + off), a.map_kv, hh * 64, 0, t.kh, pages[pg], 2 * a.layer, bar, pol);
                tma_load_5d(smem_u32(sV + off), a.map_kv, hh * 64, 0, t.kh, pages[pg], 2 * a.layer + 1, bar, pol);
              }
            }
          }
          __syncwarp();
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issue
    // The whole warp walks the loops and the waits together; one elected lane issues each tensor-core instruction and
    // each commit (the loop state is then the same in every lane, which lets the compiler keep descriptors and
    // addresses in uniform registers: a lone lane issued an instruction every ~50 cycles, too slow for 20 small
    // instructions per 64-position block).
    {
      const uint32_t idesc_qk = umma_idesc_f16(kAttnRows, kAttnBlk, 0);
      const uint32_t idesc_pv = umma_idesc_f16(kAttnRows, HD, 1);
      const uint32_t sKV = smem_u32(smem);
      bool ok = true;
      uint32_t gb = 0, un = 0;
      // a wait that ran out in one lane ends the loops of all lanes together (elect.sync names the full warp)
      auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
        return __all_sync(0xffffffffu, mbar_wait_err(bar, parity, err));
      };
      // O (+)= P V for block bi; `first`: the unit's first block starts the sums afresh, which needs the workers to
      // have read the previous unit's sums out
      auto issue_pv = [&](uint32_t bi, bool first) -> bool {
        const uint32_t pb = bi & 1, vst = bi % kKvStages;
        if (!wait_all(smem_u32(&ctl->p_full[pb]), (bi >> 1) & 1)) return false;
        if (first && un > 0 && !wait_all(smem_u32(&ctl->o_free), (un - 1) & 1)) return false;
        tc_fence_after();
        const uint32_t sV = sKV + vst * kKvBytes + kAttnBlk * HD * 2;
#pragma unroll
        for (int ks = 0; ks < kAttnBlk / 16; ++ks) {   // 16 positions per instruction: values, then remainders
          if (elect_one())
            umma_f16_ts(tmem_base + kColO, tmem_base + kColP + pb * 32 + ks * 8,
                        umma_desc_sw128_mn(sV + ks * 2048, kAttnBlk * 128), idesc_pv, (!first || ks != 0) ? 1u : 0u);
          if (elect_one())
            umma_f16_ts(tmem_base + kColO, tmem_base + kColPL + pb * 32 + ks * 8,
                        umma_desc_sw128_mn(sV + ks * 2048, kAttnBlk * 128), idesc_pv, 1u);
        }
        if (elect_one()) {
          umma_commit(smem_u32(&ctl->pv_done[pb]));
          umma_commit(smem_u32(&ctl->kv_empty[vst]));
        }
        __syncwarp();
        return true;
      };
      // S = Q K^T + Q_lo K^T for block g (counted over the CTA's blocks): the remainder plane of the queries goes
      // through the same keys into the same sums; the queries are read from tensor memory (8 columns = 16 elements
      // per instruction)
      auto issue_qk = [&](uint32_t g) -> bool {
        const uint32_t kst = g % kKvStages, st = g & 1;
        if (!wait_all(smem_u32(&ctl->kv_full[kst]), (g / kKvStages) & 1)) return false;
        if (!wait_all(smem_u32(&ctl->s_empty[st]), ((g >> 1) & 1) ^ 1)) return false;
        tc_fence_after();
        const uint32_t sK = sKV + kst * kKvBytes;
#pragma unroll
        for (int pl = 0; pl < 2; ++pl) {
#pragma unroll
          for (int hh = 0; hh < (int)kHalves; ++hh) {
            const uint64_t dk = umma_desc_sw128(sK + hh * (kAttnBlk * 128));
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              if (elect_one())
                umma_f16_ts(tmem_base + kColS + st * 64, tmem_base + kColQ + pl * (HD / 2) + hh * 32 + kk * 8, dk + 2 * kk,
                            idesc_qk, (pl | hh | kk) != 0 ? 1u : 0u);
          }
        }
        if (elect_one()) umma_commit(smem_u32(&ctl->s_full[st]));
        __syncwarp();
        return true;
      };
      // Issue order within a unit: S(0), then for every block b: S(b + 1), O += P(b) V(b).  The scores run one block
      // ahead of the block the workers are on, so a worker finds its scores complete when it gets to them, and the
      // product of block b waits only for that block's probabilities.
      for (int j = 0; j * (int)gridDim.x < n_total && ok; ++j) {
        const int u = attn_unit_of((int)blockIdx.x, j, (int)gridDim.x);
        if (u >= n_total) continue;
        const AttnUnit t = attn_unit_info(a, u);
        if (t.nblk == 0) continue;
        ok = wait_all(smem_u32(&ctl->q_full), un & 1);
        if (ok) ok = issue_qk(gb);
        for (int b = 0; ok && b < t.nblk; ++b, ++gb) {
          if (b + 1 < t.nblk) ok = issue_qk(gb + 1);
          if (ok) ok = issue_pv(gb, b == 0);
        }
        ++un;
      }
      if (!ok && lane == 0) atomicCAS(a.err, 0, DEV_TIMEOUT_FULL);
    }
  } else {
    // ---------------------------------------------------------------- workers
    uint32_t blk = 0;
    bool ok = true, waited = false;
    for (int j = 0; j * (int)gridDim.x < n_total && ok; ++j) {
      const int u = attn_unit_of((int)blockIdx.x, j, (int)gridDim.x);
      if (u >= n_total) continue;
      const AttnUnit t = attn_unit_info(a, u);
      ok = attn_unit_workers<HD>(a, ctl, t, tmem_base, warp & 3, lane, (int)threadIdx.x - kWorkerWarp0 * 32, blk, waited, err);
    }
    if (!waited) pdl_wait();
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
  if (threadIdx.x == 0 && a.stamp) stamp_max(a.stamp + 3);
}

// grid = (M, Hq / 4), 4 warps: a warp adds the leaves of one (row, query head) and emits the normalised row as bf16
// (hi[, lo]); lane i owns hd / 32 consecutive elements.  The row's sequence has n_leaves = ceil((cached length +
// chunk rows) / leaf_len) leaves, all of them written (a leaf the row cannot see carries sum 0 and gets weight 0).
// Lane s turns leaf s's (max, sum) into a weight; every lane loads its elements of all leaves at once (one round trip
// to L2, 16 bytes per lane and leaf) and adds them in leaf order.  NS = compile-time bound on the number of leaves.
template <int NS, int VW>
__global__ void attn_merge_kernel(const AttnTcArgs a) {
  if (threadIdx.x == 0) stamp_min(a.stamp_merge);
  pdl_launch_dependents();   // the dependent kernel waits for this one's end before touching its data
  const int m = blockIdx.x, h = blockIdx.y * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  int nl = a.in.row_leaves[m];   // (a step input, on the device before the step's first kernel)
  if (!ts_in_range(a.in.ck, CHK_LEAVES, nl, a.n_slots + 1)) nl = 0;
  pdl_wait();
  if (threadIdx.x == 0) stamp_waited(a.stamp_merge);
  if (h >= a.Hq) return;
  const size_t base = ((size_t)m * a.Hq + h) * a.n_slots;
  const float2 ml = lane < nl ? a.attn_ml[base + lane] : make_float2(-INFINITY, 0.f);
  float t[NS][VW];
#pragma unroll
  for (int s = 0; s < NS; ++s) {
    if (s < nl) {
      const float *src = a.attn_o + (base + s) * a.hd + lane * VW;
      if constexpr (VW == 4) {
        const float4 v = *reinterpret_cast<const float4 *>(src);
        t[s][0] = v.x; t[s][1] = v.y; t[s][2] = v.z; t[s][3] = v.w;
      } else {
        const float2 v = *reinterpret_cast<const float2 *>(src);
        t[s][0] = v.x; t[s][1] = v.y;
      }
    } else {
#pragma unroll
      for (int e = 0; e < VW; ++e) t[s][e] = 0.f;
    }
  }
  float mx = ml.y > 0.f ? ml.x : -INFINITY;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  float w = ml.y > 0.f ? exp2f(ml.x - mx) : 0.f;
  // the denominator: leaf by leaf in leaf order (a shuffle tree would pair lanes differently as leaves are added)
  float den = 0.f, num[VW];
#pragma unroll
  for (int e = 0; e < VW; ++e) num[e] = 0.f;
#pragma unroll
  for (int s = 0; s < NS; ++s) {
    const float ws = __shfl_sync(0xffffffffu, w, s);
    const float ls = __shfl_sync(0xffffffffu, ml.y, s);
    if (ws != 0.f) {
      den += ws * ls;
#pragma unroll
      for (int e = 0; e < VW; ++e) num[e] += ws * t[s][e];
    }
  }
  const float inv = 1.f / den;
  __align__(8) __nv_bfloat16 hi[VW], lo[VW];
#pragma unroll
  for (int e = 0; e < VW; ++e) split_bf16(num[e] * inv, hi[e], lo[e]);
  const size_t col = (size_t)h * a.hd + lane * VW;
  const size_t ld = (size_t)a.Hq * a.hd;
  __nv_bfloat16 *o_hi = a.out + (size_t)m * ld + col, *o_lo = a.out + ((size_t)a.out_rows + m) * ld + col;
  if constexpr (VW == 4) {
    *reinterpret_cast<uint2 *>(o_hi) = *reinterpret_cast<const uint2 *>(hi);
    if (a.planes == 2) *reinterpret_cast<uint2 *>(o_lo) = *reinterpret_cast<const uint2 *>(lo);
  } else {
    *reinterpret_cast<uint32_t *>(o_hi) = *reinterpret_cast<const uint32_t *>(hi);
    if (a.planes == 2) *reinterpret_cast<uint32_t *>(o_lo) = *reinterpret_cast<const uint32_t *>(lo);
  }
  if (threadIdx.x == 0 && a.stamp_merge) stamp_max(a.stamp_merge + 3);
}

template <typename K>
static cudaError_t launch_merge_pdl(K kernel, const AttnTcArgs &a, cudaStream_t st) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(a.in.M, (a.Hq + 3) / 4);
  cfg.blockDim = dim3(128);
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, a);
}

cudaError_t launch_attention_tc_merge(const AttnTcArgs &a, cudaStream_t st) {
  if (a.n_slots < 1 || a.n_slots > kAttnMaxSplits) return cudaErrorInvalidValue;
  if (a.hd == 128) {
    if (a.n_slots <= 2) return launch_merge_pdl(attn_merge_kernel<2, 4>, a, st);
    if (a.n_slots <= 4) return launch_merge_pdl(attn_merge_kernel<4, 4>, a, st);
    if (a.n_slots <= 8) return launch_merge_pdl(attn_merge_kernel<8, 4>, a, st);
    if (a.n_slots <= 16) return launch_merge_pdl(attn_merge_kernel<16, 4>, a, st);
    return launch_merge_pdl(attn_merge_kernel<32, 4>, a, st);
  }
  if (a.n_slots <= 2) return launch_merge_pdl(attn_merge_kernel<2, 2>, a, st);
  if (a.n_slots <= 4) return launch_merge_pdl(attn_merge_kernel<4, 2>, a, st);
  if (a.n_slots <= 8) return launch_merge_pdl(attn_merge_kernel<8, 2>, a, st);
  if (a.n_slots <= 16) return launch_merge_pdl(attn_merge_kernel<16, 2>, a, st);
  return launch_merge_pdl(attn_merge_kernel<32, 2>, a, st);
}

static size_t attn_tc_smem(int hd) {
  return 1024 + (size_t)kKvStages * 2 * kAttnBlk * hd * 2 + sizeof(AttnCtl) + 64;
}

cudaError_t launch_attention_tc(const AttnTcArgs &a, cudaStream_t st) {
  static PerDeviceOnce once;
  int dev_ = -1;
  if (once.needed(&dev_)) {
    cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_tc_smem(128));
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_tc_smem(64));
    if (e != cudaSuccess) return e;
    once.done(dev_);
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(std::min(a.n_units * a.Hkv, a.max_ctas));
  cfg.blockDim = dim3(kTcThreads);
  cfg.dynamicSmemBytes = attn_tc_smem(a.hd);
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return (a.hd == 128) ? cudaLaunchKernelEx(&cfg, attn_tc_kernel<128>, a) : cudaLaunchKernelEx(&cfg, attn_tc_kernel<64>, a);
}

}  // namespace ts
