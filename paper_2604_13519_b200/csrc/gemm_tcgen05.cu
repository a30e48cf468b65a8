// Weight-streaming GEMM for the verify step's dense projections (QKV, O, gate-up, down, LM head):
//     out[m][n] = sum_k act[m][k] * W[n][k]
// with few rows m (the verified positions) and a large weight matrix read exactly once.
//
// The weight matrix is stored as contiguous 128 x 64 blocks (one TMA box each).
// Operands are swapped with respect to the usual layout so that the 128-row dimension of the
// tensor-core instruction runs over output features: a CTA owns 128 rows of W (operand A, K-major,
// 16 KB per 64-wide k-block) and a chunk of up to 128 activation rows (operand B).  Activations can
// be fed as a (hi, lo) bf16 pair stacked along the instruction's N dimension, so one MMA multiplies
// the weight tile with both halves; the epilogue adds the two column groups.  The accumulator lives
// in tensor memory: lane = output feature, column = activation row.
//
// Roles: warp 0 = TMA producer, warp 1 = TMEM allocation + MMA issue, warps 2..5 = epilogue.
// Every wait is bounded; on expiry the CTA records an error word and leaves through the normal exit.
#include "kernels.h"

namespace ts {

static constexpr int kBlockK = 64;                 // k-block: 64 bf16 = 128 bytes per row
static constexpr int kTileN = 128;                 // weight rows per CTA
static constexpr int kWBytes = kTileN * kBlockK * 2;
static constexpr int kMaxStages = 8;

struct __align__(8) GemmSmemCtl {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t tmem_full;
  uint32_t tmem_base;
  uint32_t abort_flag;
};

template <int EPI>
__global__ void __launch_bounds__(192, 1)
gemm_ws_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_a,
               const GemmArgs g) {
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte alignment is required by the 128-byte swizzle pattern
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int a_bytes = g.planes * g.Mc * kBlockK * 2;
  const int stage_bytes = kWBytes + a_bytes;
  GemmSmemCtl *ctl = reinterpret_cast<GemmSmemCtl *>(smem + (size_t)g.stages * stage_bytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * kTileN;
  const int split = blockIdx.y;
  const int m0 = blockIdx.z * g.Mc;
  // balanced cut of the k-blocks into gridDim.y runs
  const int kb0 = (int)(((long long)split * g.n_kblocks) / (int)gridDim.y);
  const int kb1 = (int)(((long long)(split + 1) * g.n_kblocks) / (int)gridDim.y);
  const int nkb = kb1 - kb0;
  const uint32_t ncols = g.planes * g.Mc;
  uint32_t alloc_cols = 32;
  while (alloc_cols < ncols) alloc_cols <<= 1;

  if (warp == 0 && lane == 0) {
    tma_prefetch_desc(&tmap_w);
    tma_prefetch_desc(&tmap_a);
    for (int s = 0; s < g.stages; ++s) {
      mbar_init(smem_u32(&ctl->full[s]), 1);
      mbar_init(smem_u32(&ctl->empty[s]), 1);
    }
    mbar_init(smem_u32(&ctl->tmem_full), 1);
    ctl->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&ctl->tmem_base), alloc_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  if (threadIdx.x == 0) stamp_min(g.stamp);
  // Let the next kernel launch now: it waits (griddepcontrol.wait) for this one to finish before it touches
  // dependent data, so only its launch latency and its own prologue (weight prefetch) move forward.  Placed after
  // this CTA holds its resources, so a waiting dependent can never starve an earlier kernel.
  pdl_launch_dependents();

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0 && nkb > 0) {
      const uint64_t pol_w = policy_evict_first(), pol_a = policy_evict_last();
      const int pre = min(g.stages, nkb);
      // weights do not depend on the previous kernel: start streaming them before the
      // programmatic-dependency wait, activations after it
      for (int it = 0; it < pre; ++it) {
        uint32_t bar = smem_u32(&ctl->full[it]);
        mbar_expect_tx(bar, stage_bytes);
        tma_load_2d(smem_u32(smem + (size_t)it * stage_bytes), &tmap_w, 0, w_block(blockIdx.x, kb0 + it, (g.N + kTileN - 1) / kTileN, g.n_kblocks) * kTileN, bar, pol_w);
      }
      pdl_wait();
      stamp_waited(g.stamp);
      for (int it = 0; it < pre; ++it) {
        uint32_t bar = smem_u32(&ctl->full[it]);
        tma_load_3d(smem_u32(smem + (size_t)it * stage_bytes + kWBytes), &tmap_a, (kb0 + it) * kBlockK, m0, 0,
                    bar, pol_a);
      }
      // slot and round parity are carried along: an integer division per k-block would be a large part of
      // this single thread's time budget per block
      int s = (pre == g.stages) ? 0 : pre;
      uint32_t ph = (pre == g.stages) ? 1 : 0;
      for (int it = pre; it < nkb; ++it) {
        if (!mbar_wait(smem_u32(&ctl->empty[s]), ph ^ 1)) {
          atomicExch(g.err, DEV_TIMEOUT_EMPTY);
          break;
        }
        uint32_t bar = smem_u32(&ctl->full[s]);
        mbar_expect_tx(bar, stage_bytes);
        uint32_t dst = smem_u32(smem + (size_t)s * stage_bytes);
        tma_load_2d(dst, &tmap_w, 0, w_block(blockIdx.x, kb0 + it, (g.N + kTileN - 1) / kTileN, g.n_kblocks) * kTileN, bar, pol_w);
        tma_load_3d(dst + kWBytes, &tmap_a, (kb0 + it) * kBlockK, m0, 0, bar, pol_a);
        if (++s == g.stages) { s = 0; ph ^= 1; }
      }
    } else if (lane == 0) {
      pdl_wait();
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issue
    // The whole warp walks the loop and the waits; one elected lane issues the instructions of a k-block and its
    // commit (a lone lane in a divergent branch needs about 50 cycles per tensor-core instruction, this form 22).
    {
      const uint32_t idesc = umma_idesc_bf16(kTileN, ncols);
      bool ok = true;
      int s = 0;
      uint32_t ph = 0;
      for (int it = 0; it < nkb; ++it) {
        if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&ctl->full[s]), ph))) {   // (all lanes leave together)
          if (lane == 0) atomicExch(g.err, DEV_TIMEOUT_FULL);
          ok = false;
          break;
        }
        tc_fence_after();
        const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
        const uint64_t da = umma_desc_sw128(sa), db = umma_desc_sw128(sa + kWBytes);
        if (elect_one()) {
#pragma unroll
          for (int kk = 0; kk < kBlockK / 16; ++kk) {
            // 16 bf16 along K = 32 bytes = 2 descriptor address units
            umma_bf16(tmem_base, da + 2 * kk, db + 2 * kk, idesc, (it | kk) != 0);
          }
          umma_commit(smem_u32(&ctl->empty[s]));
        }
        __syncwarp();
        if (++s == g.stages) { s = 0; ph ^= 1; }
      }
      if (elect_one()) {
        if (!ok) ctl->abort_flag = 1;
        umma_commit(smem_u32(&ctl->tmem_full));
      }
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    pdl_wait();   // outputs of this kernel may still be read by the previous one's consumers
    bool ok = true;
    if (nkb > 0) {
      ok = mbar_wait(smem_u32(&ctl->tmem_full), 0);
      if (!ok && lane == 0) atomicExch(g.err, DEV_TIMEOUT_TMEM);
    }
    tc_fence_after();
    ok = ok && (ctl->abort_flag == 0);
    const int q = warp & 3;                       // TMEM lane quarter this warp may read
    const int n = n0 + q * 32 + lane;
    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
    if (ok) {
      for (int c0 = 0; c0 < g.Mc; c0 += 16) {
        if (m0 + c0 >= g.M) break;
        uint32_t r[16], r2[16];
        float v[16];
        if (nkb > 0) {
          tmem_ld16(taddr + c0, r);
          if (g.planes == 2) tmem_ld16(taddr + g.Mc + c0, r2);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 16; ++j)
            v[j] = __uint_as_float(r[j]) + (g.planes == 2 ? __uint_as_float(r2[j]) : 0.f);
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] = 0.f;
        }
        if constexpr (EPI == EPI_PARTIAL) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int m = m0 + c0 + j;
            if (m < g.M && n < g.N) g.out[((size_t)split * g.out_rows + m) * g.N + n] = v[j];
          }
        } else if constexpr (EPI == EPI_LOGITS) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int m = m0 + c0 + j;
            if (m < g.M && n < g.N) g.out[(size_t)m * g.N + n] = v[j];
            float bv = (n < g.N) ? v[j] : -INFINITY;
            int bi = n;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
              float ov = __shfl_xor_sync(0xffffffffu, bv, o);
              int oi = __shfl_xor_sync(0xffffffffu, bi, o);
              if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
            }
            if (lane == 0 && m < g.M) {
              // order-preserving map of the float to an unsigned word; ties resolve to the lowest id
              uint32_t u = __float_as_uint(bv);
              u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
              atomicMax(g.amax + m, ((unsigned long long)u << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)bi));
            }
          }
        } else {  // EPI_SWIGLU: even feature row = gate_f, odd = up_f, f = n / 2
          const int f = n >> 1;
          const int F = g.N >> 1;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int m = m0 + c0 + j;
            const float other = __shfl_xor_sync(0xffffffffu, v[j], 1);
            const float gate = (lane & 1) ? other : v[j];
            const float up = (lane & 1) ? v[j] : other;
            const float a = gate / (1.f + __expf(-gate)) * up;
            __nv_bfloat16 hi, lo;
            split_bf16(a, hi, lo);
            if (m < g.M && n < g.N) {
              if ((lane & 1) == 0) g.act_out[(size_t)m * F + f] = hi;
              else if (g.out_planes == 2) g.act_out[((size_t)g.act_rows + m) * F + f] = lo;
            }
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, alloc_cols);
  }
  if (threadIdx.x == 0 && g.stamp) stamp_max(g.stamp + 3);
}

static size_t gemm_smem_bytes(int stages, int planes, int Mc) {
  return (size_t)stages * (kWBytes + planes * Mc * kBlockK * 2) + sizeof(GemmSmemCtl) + 1024;
}

int gemm_pick_stages(int planes, int Mc, size_t smem_budget) {
  int s = kMaxStages;
  while (s > 2 && gemm_smem_bytes(s, planes, Mc) > smem_budget) --s;
  return s;
}

template <int EPI>
static cudaError_t launch_one(const CUtensorMap &tw, const CUtensorMap &ta, const GemmArgs &g, dim3 grid,
                              size_t smem, cudaStream_t st, bool pdl) {
  static PerDeviceOnce once;
  int dev_ = -1;
  if (once.needed(&dev_)) {
    cudaError_t e = cudaFuncSetAttribute(gemm_ws_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         227 * 1024);
    if (e != cudaSuccess) return e;
    once.done(dev_);
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(192);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, gemm_ws_kernel<EPI>, tw, ta, g);
}

cudaError_t launch_gemm(int epi, const CUtensorMap &tw, const CUtensorMap &ta, GemmArgs g, int n_splits,
                        size_t smem_budget, cudaStream_t st, bool pdl) {
  g.stages = gemm_pick_stages(g.planes, g.Mc, smem_budget);
  const size_t smem = gemm_smem_bytes(g.stages, g.planes, g.Mc);
  dim3 grid((g.N + kTileN - 1) / kTileN, n_splits, (g.M + g.Mc - 1) / g.Mc);
  switch (epi) {
    case EPI_PARTIAL: return launch_one<EPI_PARTIAL>(tw, ta, g, grid, smem, st, pdl);
    case EPI_SWIGLU: return launch_one<EPI_SWIGLU>(tw, ta, g, grid, smem, st, pdl);
    default: return launch_one<EPI_LOGITS>(tw, ta, g, grid, smem, st, pdl);
  }
}

}  // namespace ts
