// The dense projections of the verify step for MANY rows (batched steps: more than 64 rows), where the work is bound by
// the tensor cores and by the bytes an SM pulls from L2 per flop, no longer by streaming the weights:
//     out[m][n] = sum_k act[m][k] * W[n][k]
// Orientation: a CTA owns a chunk of 128 activation rows (operand A of the tensor-core instruction, its 128-row
// dimension) and 256 weight rows (operand B, the instruction's N dimension); the accumulator in tensor memory is
// 128 lanes (rows) x 256 fp32 columns (features).  The (hi, lo) bf16 planes of the activations are two instructions
// into the SAME accumulator, so per 64-wide k-block a CTA brings in 32 KB of activations and 32 KB of weights for
// 8.4 MFLOP -- two thirds of the bytes per flop of the weight-streaming kernel (gemm_tcgen05.cu), which at these sizes
// is what sets the pace.  The weight matrix keeps its storage (contiguous 128 x 64 blocks, one TMA box each): a CTA's
// 256 weight rows are two such boxes.  One CTA per SM (three 64 KB stages).
//
// Roles: warp 0 = TMA producer, warp 1 = TMEM allocation + MMA issue, warps 2..9 = epilogue (thread <-> row, two
// warps per row quarter, half of the columns each).
// Every wait is bounded; on expiry the CTA records an error word and leaves through the normal exit.
#include <algorithm>
#include <functional>
#include <map>
#include <mutex>
#include <tuple>
#include <vector>

#include "kernels.h"

namespace ts {

static constexpr int kBlockK = 64;                 // k-block: 64 bf16 = 128 bytes per row
static constexpr int kRowsM = 128;                 // activation rows per CTA
static constexpr int kBoxN = 128;                  // weight rows per stored block (one TMA box)
static constexpr int kTileN = 256;                 // weight rows per CTA
static constexpr int kBoxBytes = kBoxN * kBlockK * 2;
static constexpr int kMaxStages = 4;

struct __align__(8) RowsSmemCtl {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t tmem_full;
  uint32_t tmem_base;
  uint32_t abort_flag;
};

template <int EPI>
__global__ void __launch_bounds__(320, 1)
gemm_rows_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_a,
                 const GemmArgs g) {
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte alignment is required by the 128-byte swizzle pattern
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int a_bytes = g.planes * kRowsM * kBlockK * 2;
  const int stage_bytes = a_bytes + 2 * kBoxBytes;
  RowsSmemCtl *ctl = reinterpret_cast<RowsSmemCtl *>(smem + (size_t)g.stages * stage_bytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // grid = (row chunks, weight tiles, K slices): the row chunks of one (tile, slice) are neighbours in launch order, so
  // they run at the same time and all but the first find the weight blocks in L2
  // the first n_wide tiles hold two stored 128-row weight blocks, the tiles after them one (the launcher mixes the
  // widths so that the last wave of CTAs is short instead of nearly empty)
  const int tile = blockIdx.y;
  const int blk0 = tile < g.n_wide ? 2 * tile : g.n_wide + tile;   // the tile's first weight block
  const int n0 = blk0 * kBoxN;
  const int nb = tile < g.n_wide ? kTileN : kBoxN;
  const int split = blockIdx.z;
  const int m0 = blockIdx.x * kRowsM;
  // balanced cut of the k-blocks into gridDim.z runs
  const int kb0 = (int)(((long long)split * g.n_kblocks) / (int)gridDim.z);
  const int kb1 = (int)(((long long)(split + 1) * g.n_kblocks) / (int)gridDim.z);
  const int nkb = kb1 - kb0;
  const int tx_bytes = a_bytes + (nb / kBoxN) * kBoxBytes;

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
    tmem_alloc(smem_u32(&ctl->tmem_base), kTileN);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  if (threadIdx.x == 0) stamp_min(g.stamp);
  // (placed after this CTA holds its resources, so a waiting dependent can never starve an earlier kernel)
  pdl_launch_dependents();

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0 && nkb > 0) {
      const uint64_t pol_w = policy_evict_first(), pol_a = policy_evict_last();
      // block (128-row block j, k-block kb) of the stored matrix = rows w_block(j, kb) * 128 .. of a [.][64] array
      auto load_w = [&](int s, int kb) {
        const uint32_t bar = smem_u32(&ctl->full[s]);
        const uint32_t dst = smem_u32(smem + (size_t)s * stage_bytes + a_bytes);
        for (int j = 0; j < nb / kBoxN; ++j)
          tma_load_2d(dst + j * kBoxBytes, &tmap_w, 0, w_block(blk0 + j, kb, g.N / kBoxN, g.n_kblocks) * kBoxN, bar, pol_w);
      };
      const int pre = min(g.stages, nkb);
      // weights do not depend on the previous kernel: start them before the programmatic-dependency wait
      for (int it = 0; it < pre; ++it) {
        mbar_expect_tx(smem_u32(&ctl->full[it]), tx_bytes);
        load_w(it, kb0 + it);
      }
      pdl_wait();
      stamp_waited(g.stamp);
      for (int it = 0; it < pre; ++it)
        tma_load_3d(smem_u32(smem + (size_t)it * stage_bytes), &tmap_a, (kb0 + it) * kBlockK, m0, 0,
                    smem_u32(&ctl->full[it]), pol_a);
      int s = (pre == g.stages) ? 0 : pre;
      uint32_t ph = (pre == g.stages) ? 1 : 0;
      for (int it = pre; it < nkb; ++it) {
        if (!mbar_wait(smem_u32(&ctl->empty[s]), ph ^ 1)) {
          atomicExch(g.err, DEV_TIMEOUT_EMPTY);
          break;
        }
        mbar_expect_tx(smem_u32(&ctl->full[s]), tx_bytes);
        load_w(s, kb0 + it);
        tma_load_3d(smem_u32(smem + (size_t)s * stage_bytes), &tmap_a, (kb0 + it) * kBlockK, m0, 0,
                    smem_u32(&ctl->full[s]), pol_a);
        if (++s == g.stages) { s = 0; ph ^= 1; }
      }
    } else if (lane == 0) {
      pdl_wait();
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issue
    // The whole warp walks the loop and the waits; one elected lane issues the instructions of a k-block and its commit.
    {
      const uint32_t idesc = umma_idesc_bf16(kRowsM, (uint32_t)nb);
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
        const uint64_t db = umma_desc_sw128(sa + a_bytes);
        if (elect_one()) {
          // the value plane and the remainder plane of the activations into the same sums
          for (int pl = 0; pl < g.planes; ++pl) {
            const uint64_t da = umma_desc_sw128(sa + pl * (kRowsM * kBlockK * 2));
#pragma unroll
            for (int kk = 0; kk < kBlockK / 16; ++kk)   // 16 bf16 along K = 32 bytes = 2 descriptor address units
              umma_bf16(tmem_base, da + 2 * kk, db + 2 * kk, idesc, (it | kk | pl) != 0);
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
    // ------------------------------------------------------------------ epilogue (warps 2..9): thread <-> row
    pdl_wait();   // outputs of this kernel may still be read by the previous one's consumers
    bool ok = true;
    if (nkb > 0) {
      ok = mbar_wait(smem_u32(&ctl->tmem_full), 0);
      if (!ok && lane == 0) atomicExch(g.err, DEV_TIMEOUT_TMEM);
    }
    tc_fence_after();
    ok = ok && (*reinterpret_cast<volatile uint32_t *>(&ctl->abort_flag) == 0);
    const int q = warp & 3;                       // TMEM lane quarter this warp may read
    const int m = m0 + q * 32 + lane;             // this thread's row
    const bool row_ok = m < g.M;
    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
    float best = -INFINITY;
    int best_n = 0;
    // Results leave through shared memory so that global stores are whole lines: a thread owns a ROW of the
    // accumulator, so storing from registers makes the 32 lanes of a warp write 32 different lines per instruction
    // (4 us for the 128 KB of a tile).  Each warp stages 32 rows x 128 bytes (16-byte chunks, slot = chunk ^ (row & 7):
    // conflict-free both ways) in the ring's shared memory -- free by now: every load was consumed by a product that
    // has completed -- and writes them back 4 rows x 128 bytes per instruction.
    // Eight epilogue warps: warps 2..5 take the first half of the tile's columns, warps 6..9 the second (two warps
    // per tensor-memory lane quarter).
    const int eh = (warp - 2) >> 2, c_beg = eh * (nb >> 1), c_end = c_beg + (nb >> 1);
    const uint32_t stg = smem_u32(smem) + (warp - 2) * 4096;
    const int rr = lane >> 3, slot = lane & 7;   // read-back: rows rr, rr + 4, ...; 16-byte slot of the row
    if (ok) {
      if constexpr (EPI != EPI_SWIGLU) {
        for (int c0 = c_beg; c0 < c_end; c0 += 32) {
          uint32_t r[32];
          if (nkb > 0) {
            tmem_ld16(taddr + c0, *reinterpret_cast<uint32_t(*)[16]>(r));     // (warp-wide: rows past the end read too)
            tmem_ld16(taddr + c0 + 16, *reinterpret_cast<uint32_t(*)[16]>(r + 16));
            tmem_wait_ld();
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) r[j] = 0u;
          }
          const int n = n0 + c0;
          if constexpr (EPI == EPI_LOGITS) {
            if (row_ok) {
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                const float v = __uint_as_float(r[j]);
                if (v > best) { best = v; best_n = n + j; }   // (ascending ids: a tie keeps the lower one)
              }
            }
          }
#pragma unroll
          for (int c = 0; c < 8; ++c)
            st_shared_v4(stg + lane * 128 + ((c ^ (lane & 7)) << 4), r[4 * c], r[4 * c + 1], r[4 * c + 2], r[4 * c + 3]);
          __syncwarp();
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int R = i * 4 + rr, mr = m0 + q * 32 + R;
            const uint4 v = ld_shared_v4(stg + R * 128 + ((slot ^ (R & 7)) << 4));
            if (mr < g.M) {
              float *dst = (EPI == EPI_PARTIAL ? g.out + ((size_t)split * g.out_rows + mr) * g.N : g.out + (size_t)mr * g.N) + n + slot * 4;
              *reinterpret_cast<uint4 *>(dst) = v;
            }
          }
          __syncwarp();
        }
      } else {
        // EPI_SWIGLU: even feature = gate_f, odd = up_f, f = n / 2.  64 accumulator columns give 32 features: 64 bytes
        // of the value plane (slots 0..3 of the staged row) and 64 of the remainder plane (slots 4..7).
        const int F = g.N >> 1;
        for (int c0 = c_beg; c0 < c_end; c0 += 64) {
          uint32_t hi[16], lo[16];   // 32 features per plane, two bf16 per word
#pragma unroll
          for (int part = 0; part < 4; ++part) {
            uint32_t r[16];
            if (nkb > 0) {
              tmem_ld16(taddr + c0 + part * 16, r);
              tmem_wait_ld();
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j) r[j] = 0u;
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              __nv_bfloat16 h0, l0, h1, l1;
              const float g0 = __uint_as_float(r[4 * j]), u0 = __uint_as_float(r[4 * j + 1]);
              const float g1 = __uint_as_float(r[4 * j + 2]), u1 = __uint_as_float(r[4 * j + 3]);
              split_bf16(g0 / (1.f + __expf(-g0)) * u0, h0, l0);
              split_bf16(g1 / (1.f + __expf(-g1)) * u1, h1, l1);
              hi[part * 4 + j] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
              lo[part * 4 + j] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
            }
          }
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            st_shared_v4(stg + lane * 128 + ((c ^ (lane & 7)) << 4), hi[4 * c], hi[4 * c + 1], hi[4 * c + 2], hi[4 * c + 3]);
            st_shared_v4(stg + lane * 128 + (((c + 4) ^ (lane & 7)) << 4), lo[4 * c], lo[4 * c + 1], lo[4 * c + 2], lo[4 * c + 3]);
          }
          __syncwarp();
          const int f = (n0 + c0) >> 1;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int R = i * 4 + rr, mr = m0 + q * 32 + R;
            const uint4 v = ld_shared_v4(stg + R * 128 + ((slot ^ (R & 7)) << 4));
            if (mr < g.M && (slot < 4 || g.out_planes == 2)) {
              __nv_bfloat16 *dst = g.act_out + ((size_t)(slot < 4 ? 0 : g.act_rows) + mr) * F + f + (slot & 3) * 8;
              *reinterpret_cast<uint4 *>(dst) = v;
            }
          }
          __syncwarp();
        }
      }
      if constexpr (EPI == EPI_LOGITS) {
        if (row_ok) {
          // order-preserving map of the float to an unsigned word; ties resolve to the lowest id
          uint32_t u = __float_as_uint(best);
          u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
          atomicMax(g.amax + m, ((unsigned long long)u << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)best_n));
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTileN);
  }
  if (threadIdx.x == 0 && g.stamp) stamp_max(g.stamp + 3);
}

static size_t rows_smem_bytes(int stages, int planes) {
  return (size_t)stages * (planes * kRowsM * kBlockK * 2 + 2 * kBoxBytes) + sizeof(RowsSmemCtl) + 1024;
}

template <int EPI>
static cudaError_t launch_rows_one(const CUtensorMap &tw, const CUtensorMap &ta, const GemmArgs &g, dim3 grid,
                                   size_t smem, cudaStream_t st, bool pdl) {
  static PerDeviceOnce once;
  int dev_ = -1;
  if (once.needed(&dev_)) {
    cudaError_t e = cudaFuncSetAttribute(gemm_rows_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    once.done(dev_);
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(320);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, gemm_rows_kernel<EPI>, tw, ta, g);
}

int gemm_rows_tiles(int N) { return (N + kTileN - 1) / kTileN; }

// How many of a projection's `blocks` stored weight blocks go into 256-row tiles (two blocks) when the launch has
// `chunks` row chunks and one CTA per SM: the rest become 128-row tiles, launched last.  A 128-row tile costs about
// 0.6 of a 256-row one (half the flops, three quarters of the bytes through shared memory).  The CTAs start in launch
// order on whichever SM frees up first; the count with the shortest finish wins, ties go to fewer narrow tiles.
static int pick_wide_tiles(int blocks, int chunks, int n_sms) {
  static std::mutex mu;
  static std::map<std::tuple<int, int, int>, int> memo;
  std::lock_guard<std::mutex> lk(mu);
  const auto key = std::make_tuple(blocks, chunks, n_sms);
  auto it = memo.find(key);
  if (it != memo.end()) return it->second;
  const int x_max = blocks / 2;
  int best_x = x_max;
  double best_t = 1e30;
  std::vector<double> sm(n_sms);
  for (int x = x_max; x >= 0 && x >= x_max - 2 * n_sms; --x) {
    std::fill(sm.begin(), sm.end(), 0.0);
    std::make_heap(sm.begin(), sm.end(), std::greater<double>());
    const int tiles = x + (blocks - 2 * x);
    for (int t = 0; t < tiles; ++t)
      for (int c = 0; c < chunks; ++c) {
        std::pop_heap(sm.begin(), sm.end(), std::greater<double>());
        sm.back() += t < x ? 1.0 : 0.6;
        std::push_heap(sm.begin(), sm.end(), std::greater<double>());
      }
    const double finish = *std::max_element(sm.begin(), sm.end());
    if (finish < best_t - 1e-9) { best_t = finish; best_x = x; }
  }
  memo[key] = best_x;
  return best_x;
}

// `ta` must be the activation map whose box holds 128 rows.  N must be a multiple of 128.
cudaError_t launch_gemm_rows(int epi, const CUtensorMap &tw, const CUtensorMap &ta, GemmArgs g, int n_splits,
                             size_t smem_limit, int n_sms, cudaStream_t st, bool pdl) {
  if (n_splits < 1 || n_splits > g.n_kblocks || g.N % kBoxN) return cudaErrorInvalidValue;
  g.Mc = kRowsM;
  g.stages = kMaxStages;
  while (g.stages > 2 && rows_smem_bytes(g.stages, g.planes) > smem_limit) --g.stages;
  const size_t smem = rows_smem_bytes(g.stages, g.planes);
  if (smem > smem_limit) return cudaErrorInvalidConfiguration;
  const int blocks = g.N / kBoxN, chunks = (g.M + kRowsM - 1) / kRowsM;
  // split-K launches are already cut to fill their waves; the others may mix tile widths
  g.n_wide = n_splits > 1 ? blocks / 2 : pick_wide_tiles(blocks, chunks, n_sms);
  dim3 grid(chunks, g.n_wide + (blocks - 2 * g.n_wide), n_splits);
  switch (epi) {
    case EPI_PARTIAL: return launch_rows_one<EPI_PARTIAL>(tw, ta, g, grid, smem, st, pdl);
    case EPI_SWIGLU: return launch_rows_one<EPI_SWIGLU>(tw, ta, g, grid, smem, st, pdl);
    default: return launch_rows_one<EPI_LOGITS>(tw, ta, g, grid, smem, st, pdl);
  }
}

}  // namespace ts
