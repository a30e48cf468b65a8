// Internal interface between the model orchestration (model.cu) and the kernels.
#pragma once
#include <cuda.h>          // CUtensorMap (types only; the driver entry point is resolved at run time)
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"

namespace ts {

enum : int { EPI_PARTIAL = 0, EPI_SWIGLU = 1, EPI_LOGITS = 2 };

struct GemmArgs {
  int N, K, M;          // output features, reduction length, valid activation rows
  int Mc;               // activation rows per CTA (16, 32, 64 or 128)
  int planes;           // 1 = bf16 activations, 2 = (hi, lo) pair
  int n_kblocks;        // K / 64
  int kb_per_split;     // k-blocks per split-K slice
  int stages;           // filled in by the launcher
  float *out;           // EPI_PARTIAL: [splits][out_rows][N]; EPI_LOGITS: [M][N]
  int out_rows;
  __nv_bfloat16 *act_out;  // EPI_SWIGLU: [out_planes][act_rows][N/2]
  int act_rows;
  int out_planes;
  unsigned long long *amax;  // EPI_LOGITS: [M] packed (ordered logit bits << 32 | ~token id), atomicMax
  int *err;             // device status word
};

int gemm_pick_stages(int planes, int Mc, size_t smem_budget);
cudaError_t launch_gemm(int epi, const CUtensorMap &tw, const CUtensorMap &ta, GemmArgs g, int n_splits,
                        size_t smem_budget, cudaStream_t st, bool pdl);

// Per-step inputs resident in device memory (all int32).
struct StepIn {
  const int32_t *tokens;     // [M] chunk ids, rows of sequence i at cu_rows[i]..cu_rows[i+1]
  const int32_t *pos;        // [M] absolute position of each row
  const int32_t *row_seq;    // [M] sequence index of each row
  const int32_t *cu_rows;    // [B+1]
  const int32_t *seq_len;    // [B] tokens already in the cache
  const int32_t *block_tab;  // [B][pages_per_seq] page ids
  int pages_per_seq;
  int B, M;
};

// x[m] = E[tokens[m]]; h = rmsnorm(x) * gain -> bf16 (hi[, lo])
cudaError_t launch_embed_norm(const StepIn &in, const __nv_bfloat16 *embed, const float *gain, float eps,
                              int d, float *x, __nv_bfloat16 *h, int h_rows, int planes,
                              unsigned long long *amax, cudaStream_t st);
// x[m] += sum_s part[s][m]; h = rmsnorm(x) * gain -> bf16 (hi[, lo])
cudaError_t launch_add_norm(int M, int d, const float *part, int n_splits, int part_rows, const float *gain,
                            float eps, float *x, __nv_bfloat16 *h, int h_rows, int planes, cudaStream_t st);
// qkv = sum of split-K partials; rotary on q and k; q -> fp16 [M][Hq][hd]; k, v -> fp16 pages
cudaError_t launch_rope_kv(const StepIn &in, const float *part, int n_splits, int part_rows, int Hq, int Hkv,
                           int hd, const float2 *rope_tab, __half *q_out, __half *k_pages, __half *v_pages,
                           cudaStream_t st);

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

// per-row argmax over the LM-head tiles, longest accepted prefix per sequence, new lengths
struct AcceptArgs {
  StepIn in;
  const unsigned long long *amax;   // [M] packed per-row maxima written by the LM-head epilogue
  int32_t *argmax;         // [M]
  int32_t *accept_len;     // [B]
  int32_t *emitted;        // [B][k_max]
  int32_t *new_len;        // [B]  cache length after the commit
  int32_t *new_pending;    // [B]
  int k_max;
};
cudaError_t launch_accept(const AcceptArgs &a, cudaStream_t st);

}  // namespace ts
