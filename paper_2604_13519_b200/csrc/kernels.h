// Internal interface between the model orchestration (model.cu) and the kernels.
#pragma once
#include <cuda.h>          // CUtensorMap (types only; the driver entry point is resolved at run time)
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "common.cuh"

namespace ts {

// A function attribute (the opt-in to large dynamic shared memory) is set per DEVICE, so "done once" has to be kept
// per device ordinal: bit d of the mask = done on device d.  Setting an attribute twice is harmless, so a race
// between two threads on their first launch costs a repeated call and nothing else.
struct PerDeviceOnce {
  std::atomic<uint64_t> mask{0};
  // true if the caller still has to do the set-up on the current device; *dev receives its ordinal (-1 = unknown)
  bool needed(int *dev) {
    if (cudaGetDevice(dev) != cudaSuccess || *dev < 0 || *dev >= 64) { *dev = -1; return true; }
    return !((mask.load(std::memory_order_acquire) >> *dev) & 1ull);
  }
  void done(int dev) { if (dev >= 0) mask.fetch_or(1ull << dev, std::memory_order_release); }
};

enum : int { EPI_PARTIAL = 0, EPI_SWIGLU = 1, EPI_LOGITS = 2 };

struct GemmArgs {
  int N, K, M;          // output features, reduction length, valid activation rows
  int Mc;               // activation rows per CTA (16, 32, 64 or 128)
  int planes;           // 1 = bf16 activations, 2 = (hi, lo) pair
  int n_kblocks;        // K / 64
  int kb_per_split;     // k-blocks per split-K slice
  int stages;           // filled in by the launcher
  int n_wide;           // many-rows kernel: weight tiles of 256 rows (the tiles after them have 128); filled in by the launcher
  float *out;           // EPI_PARTIAL: [splits][out_rows][N]; EPI_LOGITS: [M][N]
  int out_rows;
  __nv_bfloat16 *act_out;  // EPI_SWIGLU: [out_planes][act_rows][N/2]
  int act_rows;
  int out_planes;
  unsigned long long *amax;  // EPI_LOGITS: [M] packed (ordered logit bits << 32 | ~token id), atomicMax
  int *err;             // device status word
  unsigned long long *stamp;   // optional clock stamps of this launch (null = none)
};

int gemm_pick_stages(int planes, int Mc, size_t smem_budget);
cudaError_t launch_gemm(int epi, const CUtensorMap &tw, const CUtensorMap &ta, GemmArgs g, int n_splits,
                        size_t smem_budget, cudaStream_t st, bool pdl);

// The same projections for many rows (gemm_rows_tcgen05.cu): 128 activation rows x 256 weight rows per CTA, one CTA
// per SM.  `ta` must be the activation map whose box holds 128 rows; g.Mc and g.stages are set by the launcher.
int gemm_rows_tiles(int N);
cudaError_t launch_gemm_rows(int epi, const CUtensorMap &tw, const CUtensorMap &ta, GemmArgs g, int n_splits,
                             size_t smem_limit, int n_sms, cudaStream_t st, bool pdl);

// Per-step inputs resident in device memory (all int32).
struct StepIn {
  const int32_t *tokens;     // [M] chunk ids, rows of sequence i at cu_rows[i]..cu_rows[i+1]
  const int32_t *pos;        // [M] absolute (rotary) position of each row
  const int32_t *slot;       // [M] cache slot the row's K/V go to: cached length + the row's index in its chunk (equal
                             // to pos in a chain; in a draft tree pos is the depth and siblings need slots of their own)
  const int32_t *row_seq;    // [M] sequence index of each row
  const int32_t *cu_rows;    // [B+1]
  const int32_t *seq_len;    // [B] tokens already in the cache
  const int32_t *block_tab;  // [B][pages_per_seq] page ids
  const int32_t *parent;     // [M] parent of each row inside its chunk (row index relative to the chunk; -1 = root)
  const uint32_t *anc;       // [M][2] low / high word of the row's visibility mask over its chunk: bit i = row i of
                             // the chunk is the row itself or one of its ancestors (a chain: bits 0..j)
  const int32_t *row_leaves; // [M] attention leaves of the row's sequence: ceil((cached length + chunk rows) / leaf length)
  int pages_per_seq;
  int B, M;
  BoundsCheck ck;            // ranges for the debug build's index checks
};

// x[m] = E[tokens[m]]; h = rmsnorm(x) * gain -> bf16 (hi[, lo])
cudaError_t launch_embed_norm(const StepIn &in, const __nv_bfloat16 *embed, const float *gain, float eps,
                              int d, float *x, __nv_bfloat16 *h, int h_rows, int planes,
                              unsigned long long *amax, cudaStream_t st);
// x[m] += sum_s part[s][m]; h = rmsnorm(x) * gain -> bf16 (hi[, lo])
cudaError_t launch_add_norm(int M, int d, const float *part, int n_splits, int part_rows, const float *gain,
                            float eps, float *x, __nv_bfloat16 *h, int h_rows, int planes, cudaStream_t st,
                            unsigned long long *stamp = nullptr);
// qkv = sum of split-K partials; rotary on q and k; q -> fp16 [M][Hq][hd] (and, if q_lo_out is given, the rounding
// remainder of every element as a second fp16 array of the same shape); k, v -> fp16 pages
cudaError_t launch_rope_kv(const StepIn &in, const float *part, int n_splits, int part_rows, int Hq, int Hkv,
                           int hd, const float2 *rope_tab, __half *q_out, __half *q_lo_out, __half *k_pages,
                           __half *v_pages, cudaStream_t st, unsigned long long *stamp = nullptr);

constexpr int kAttnMaxSplits = 32;   // KV splits per (row tile, kv head): one lane of the merge kernel each

struct AttnArgs {
  StepIn in;
  const __half *q;               // [M][Hq][hd] rotated queries, fp16
  const __half *k_pages;         // [page][Hkv][16][hd], fp16
  const __half *v_pages;
  int Hq, Hkv, hd;
  int n_splits;                  // KV splits per (sequence, kv head, row tile)
  int n_row_tiles_total;         // sum over sequences of row tiles
  const int32_t *tile_seq;       // [n_row_tiles_total] sequence of each row tile
  const int32_t *tile_row0;      // [n_row_tiles_total] first packed row (j*G+g index) of the tile
  float *part_o;                 // [M*Hq][n_splits][hd] unnormalised partial outputs
  float2 *part_ml;               // [M*Hq][n_splits] (running max in log2 domain, sum)
  __nv_bfloat16 *out;            // [planes][out_rows][Hq*hd]
  int out_rows, planes;
};
cudaError_t launch_attention_split(const AttnArgs &a, cudaStream_t st);
cudaError_t launch_attention_combine(const AttnArgs &a, cudaStream_t st);

// tcgen05 attention as a kernel of its own (attention_tc.cu): one CTA per (128-row tile, leaf, kv head).
// A leaf is a run of leaf_len KV positions starting at an absolute multiple of leaf_len (a model constant, a
// multiple of 64): leaf L of a sequence holds positions [L * leaf_len, (L + 1) * leaf_len), whatever the cached
// length or the chunk length.  Every leaf yields one partial result per row, and the merge adds a row's leaves in
// leaf order, so the bits of a row's attention output are a function of its position and its prefix only: the same
// token gets the same logits whether it is verified alone (vanilla decoding) or as row j of a chunk.
struct AttnTcArgs {
  StepIn in;
  int Hq, Hkv, hd, layer;
  int leaf_len;                  // KV positions per leaf
  int n_units;                   // (tile, leaf) pairs of this step: n_units * Hkv units of work
  int max_ctas;                  // CTAs launched at most (one per SM); a CTA walks units blockIdx.x, + gridDim.x, ...
  int n_slots;                   // partial results kept per (row, query head): the most leaves any sequence has
  const int32_t *unit_tile;      // [n_units] tile of each pair
  const int32_t *unit_leaf;      // [n_units] leaf of each pair
  const int32_t *tile_seq;       // [tiles] sequence of each 128-row tile of packed rows
  const int32_t *tile_row0;      // [tiles] first packed row of the tile
  const __half *q, *q_lo;        // [M][Hq][hd] rotated queries as an fp16 pair: value and rounding remainder
  const CUtensorMap *map_kv;     // device copy of the 5-d map over the paged KV pool
  float *attn_o;                 // [M*Hq][n_slots][hd] unnormalised partial outputs
  float2 *attn_ml;               // [M*Hq][n_slots] (reference maximum in the log2 domain, sum)
  __nv_bfloat16 *out;            // [planes][out_rows][Hq*hd] merged, normalised rows as bf16 (hi[, lo])
  int out_rows, planes;
  int *err;                      // device status word
  unsigned long long *stamp, *stamp_merge;   // optional clock stamps of the attention and the merge launch
};
cudaError_t launch_attention_tc(const AttnTcArgs &a, cudaStream_t st);
cudaError_t launch_attention_tc_merge(const AttnTcArgs &a, cudaStream_t st);

// per-row argmax over the LM-head tiles, longest accepted prefix per sequence, new lengths
struct AcceptArgs {
  StepIn in;
  const unsigned long long *amax;   // [M] packed per-row maxima written by the LM-head epilogue
  int32_t *argmax;         // [M]
  int32_t *accept_len;     // [B]
  int32_t *emitted;        // [B][k_max]
  int32_t *new_len;        // [B]  cache length after the commit
  int32_t *new_pending;    // [B]
  int32_t *path;           // [B][k_max] chunk rows of the accepted path, root first (accept_len + 1 entries)
  int k_max;
};
cudaError_t launch_accept(const AcceptArgs &a, cudaStream_t st);

// Speculative-sampling acceptance (sampling.cu): per-row softmax statistics, accept tests, the step's one sample.
struct SampleArgs {
  StepIn in;
  float *logits;                    // [M][V] (refused tokens are masked for the draw and restored)
  const unsigned long long *amax;   // [M] packed per-row maxima (argmax is still reported)
  const float *uni;                 // [M] uniforms in [0, 1): row c of a chunk decides node c, the root row's draws the sample
  float *part;                      // [M][16] scratch: per-slice sums of exp((l - max) / T)
  int V;
  float inv_t;                      // 1 / temperature
  int32_t *argmax, *accept_len, *emitted, *new_len, *new_pending, *path;
  int k_max;
};
cudaError_t launch_sample_accept(const SampleArgs &a, cudaStream_t st);

// Cosine Top-K over datastore hidden states (retrieval.cu).  scores: [N + 2K] floats; the result pairs (index as int
// bits, score), best first, follow the N scores.  The query is q_dev (fp32 [d]) or, if null, bf16 planes of a row.
cudaError_t launch_topk_cosine(const __nv_bfloat16 *H, int N, int d, const float *q_dev, const __nv_bfloat16 *q_planes,
                               int plane_stride, int planes, int K, float *scores, cudaStream_t st);

// Row-wise Top-K (topk.cu): out[r][j] = (column as int bits, value) of the j-th largest entry of row r, lowest column
// on ties.  cand: scratch of n_rows * ceil(n_cols / 4096) * K pairs.
cudaError_t launch_topk_rows(const float *x, int n_rows, int n_cols, int K, float2 *cand, float *out, cudaStream_t st);

// After a tree step: move the K/V rows of the accepted path to consecutive cache positions len, len+1, ...
struct CompactArgs {
  StepIn in;
  const int32_t *accept_len;   // [B]
  const int32_t *path;         // [B][k_max]
  int k_max;
  __half *kv_pool;             // layer l: K pages at kv_pool + l * layer_stride, V pages v_offset further
  uint64_t layer_stride, v_offset;
  int n_layers, Hkv, hd;
};
cudaError_t launch_kv_compact(const CompactArgs &a, cudaStream_t st);

// Where a source row of an uploaded matrix goes in the stored matrix: row r -> base + r * mul, or, with
// hd != 0, base + (r / hd) * hd + p(r % hd) with p(e) = 2e for e < hd/2 and 2(e - hd/2) + 1 otherwise.
struct RowMap { int base, mul, hd, tiles; };   // tiles = 128-row blocks of the whole stored matrix
// Index of block (128-row tile, 64-wide k-block) of a stored projection matrix, in units of 128 x 64 blocks: k-block
// major, so that the CTAs of one launch, which walk the k-blocks of neighbouring tiles in step, read one contiguous
// region of memory at a time instead of as many regions a tile's length apart as there are CTAs.
__host__ __device__ inline int w_block(int tile, int kb, int tiles, int kblocks) { (void)kblocks; return kb * tiles + tile; }
// Scatter n_rows source rows (row-major, K columns, first one being row r0 of the uploaded matrix) into the
// 128 x 64-block storage of the stored matrix.
cudaError_t launch_retile(const __nv_bfloat16 *src, int n_rows, int r0, int K, RowMap rm, __nv_bfloat16 *dst,
                          cudaStream_t st);

// ---- fused single-kernel step (fused.cu) ---------------------------------------------------------------
struct FusedArgs {
  // model shape
  int n_layers, d, Nqkv, Nq, F, V, Hq, Hkv, hd;
  float eps;
  // step
  StepIn in;
  int Mc, mc_index, planes;      // activation rows per MMA (16, 32 or 64), its index, 1 or 2 planes
  int n_ctas, ring, attn_smem_bytes, skip_lm, k_max;
  int n_attn_tiles, attn_splits;
  const int32_t *tile_seq;       // [n_attn_tiles] sequence of each 128-row tile of packed rows
  const int32_t *tile_row0;      // [n_attn_tiles] first packed row of the tile
  // tensor maps in device memory: 4 per layer (qkv, o, gate-up, down), LM head, then per row-chunk
  // size three activation maps (h, attn, act)
  const CUtensorMap *maps;
  int map_kv;                    // index of the 5-d map over the paged KV pool (64 elements x 16 positions x head x page x layer*2)
  const __nv_bfloat16 *embed;
  const float *gains;            // g1[0], g2[0], g1[1], ..., gf; gain_stride floats apart
  int gain_stride;
  const float2 *rope;
  __half *kv_pool;
  unsigned long long kv_layer_stride, kv_v_offset;   // in fp16 elements
  // workspace
  float *x;                      // [R][d] residual stream
  __nv_bfloat16 *h, *attn, *act; // [planes][R][.]
  int R;
  __half *q;                     // [R][Hq*hd]
  float *slab;                   // [n_ctas][2][Mc][128] parked partial tiles
  float *ss_part;                // [d/128][R] per-tile sums of squares of x
  float *attn_o;                 // [M*Hq][splits][hd]
  float2 *attn_ml;               // [M*Hq][splits]
  float *logits;                 // [M][V]
  unsigned long long *amax;      // [M]
  int *sync;                     // [0] phase counter, [2] exit counter, [8..] tile counters (all zero between launches)
  int *err;                      // device status word shared with the other kernels
  int n_counters;
  // optional clocks (ns, latest over the CTAs), three rows of n_phases: phase end; last MMA of the phase
  // issued; first weight+activation block of the phase ready
  unsigned long long *phase_t;
  int n_phases;
  // results
  int32_t *out_argmax, *out_accept, *out_emitted, *out_newlen, *out_newpend;
};
size_t fused_attn_smem_bytes(int hd);
int fused_ring_stages(int planes, int Mc, int hd, size_t smem_limit);
cudaError_t launch_fused(FusedArgs a, size_t smem_limit, cudaStream_t st);

}  // namespace ts
