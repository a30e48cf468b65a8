// ts_attention_static: the paged grouped-query attention of the verify chunk for callers that
// must not allocate device memory.  The split-KV partial outputs, their (max, sum) pairs and the
// row-tile tables normally live in the workspace the caller sizes and allocates for a model; here
// they live in one file-scope device array that is part of the loaded library image.
//
// The array's name is a host-side stand-in in host code: the device address is looked up once per
// device with cudaGetSymbolAddress (with that device current) and only that address is handed to
// the kernels.  Nothing is copied from host memory: the row-tile table is built on the device, from
// the caller's device copy of the row offsets, by a small kernel ahead of the attention kernels.
#include <algorithm>
#include <mutex>

#include "kernels.h"
#include "toolspec.h"

namespace ts {
ts_status set_error(ts_status code, const char *fmt, ...);   // model.cu
}

namespace {

constexpr size_t kPartOBytes = (size_t)TS_STATIC_ATTN_SCRATCH_MIB << 20;   // unnormalised partial outputs
constexpr size_t kPartMlBytes = kPartOBytes / (64 * 4) * 8;                // one float2 per (row, head, split); hd >= 64
constexpr int kMaxTiles = 512;
constexpr size_t kTileBytes = 2 * kMaxTiles * sizeof(int32_t);
constexpr size_t kScratchBytes = kPartOBytes + kPartMlBytes + kTileBytes;
constexpr int kMaxDevices = 64;
constexpr int kMaxAttnSplits = ts::kAttnMaxSplits;

static __device__ __align__(256) unsigned char g_attn_scratch[kScratchBytes];

// Row-tile table of the attention kernel: tile t covers packed rows [row0, row0 + 64) of sequence seq; a
// sequence of k rows and G query heads per kv head has ceil(k * G / 64) tiles.  One thread: a few hundred
// entries at most.  Entries past max_tiles are not written (the host has checked the count already).
__global__ void static_tile_table_kernel(const int32_t *cu_rows, int batch, int G, int max_tiles, int32_t *tile_seq,
                                         int32_t *tile_row0) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  int t = 0;
  for (int i = 0; i < batch; ++i) {
    const int k = cu_rows[i + 1] - cu_rows[i];
    for (int r0 = 0; r0 < k * G && t < max_tiles; r0 += 64, ++t) {
      tile_seq[t] = i;
      tile_row0[t] = r0;
    }
  }
}

std::mutex g_mu;
unsigned char *g_dev_ptr[kMaxDevices];   // device address of g_attn_scratch, per device
int g_sms[kMaxDevices];

}  // namespace

extern "C" ts_status ts_attention_static(const ts_attention_args *a, void *stream) {
  using ts::set_error;
  if (!a) return set_error(TS_ERR_ARG, "null argument");
  if (!a->cu_rows_host || !a->seq_len_host || !a->cu_rows || !a->seq_len || !a->block_table || !a->q ||
      !a->k_pages || !a->v_pages || !a->out)
    return set_error(TS_ERR_ARG, "null pointer in ts_attention_args");
  if (a->head_dim != 64 && a->head_dim != 128) return set_error(TS_ERR_ARG, "head_dim must be 64 or 128");
  if (a->n_q_heads < 1 || a->n_kv_heads < 1 || a->n_q_heads % a->n_kv_heads)
    return set_error(TS_ERR_ARG, "q heads must be a positive multiple of kv heads");
  if (a->batch < 1 || a->pages_per_seq < 1) return set_error(TS_ERR_ARG, "batch / pages_per_seq out of range");
  if (a->planes != 1 && a->planes != 2) return set_error(TS_ERR_ARG, "planes must be 1 or 2");
  const int G = a->n_q_heads / a->n_kv_heads;
  int tiles = 0, max_total = 0;
  if (a->cu_rows_host[0] != 0) return set_error(TS_ERR_ARG, "cu_rows must start at 0");
  for (int i = 0; i < a->batch; ++i) {
    const int k = a->cu_rows_host[i + 1] - a->cu_rows_host[i];
    if (k < 1 || k > TS_K_MAX) return set_error(TS_ERR_K_TOO_LARGE, "sequence %d: %d rows, at most %d", i, k, TS_K_MAX);
    if (a->seq_len_host[i] < 0) return set_error(TS_ERR_ARG, "negative cache length");
    const long long total = (long long)a->seq_len_host[i] + k;
    if ((total + TS_PAGE_SIZE - 1) / TS_PAGE_SIZE > a->pages_per_seq)
      return set_error(TS_ERR_ARG, "sequence %d needs more pages than pages_per_seq", i);
    tiles += (k * G + 63) / 64;
    max_total = total > max_total ? (int)total : max_total;
  }
  const int M = a->cu_rows_host[a->batch];
  if (M > a->out_rows) return set_error(TS_ERR_ARG, "out_rows smaller than the number of rows");
  if (tiles > kMaxTiles)
    return set_error(TS_ERR_K_TOO_LARGE, "%d row tiles exceed the static limit of %d", tiles, kMaxTiles);
  const size_t per_split = (size_t)M * a->n_q_heads * a->head_dim * sizeof(float);
  if (per_split > kPartOBytes)
    return set_error(TS_ERR_K_TOO_LARGE,
                     "rows x heads x head_dim x 4 = %zu bytes exceeds the %d MiB static scratch of ts_attention_static",
                     per_split, TS_STATIC_ATTN_SCRATCH_MIB);

  // ---- set-up, once per device: device address of the scratch array, SM count ---------------------
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return set_error(TS_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
  if (dev < 0 || dev >= kMaxDevices) return set_error(TS_ERR_ARG, "device ordinal %d not supported", dev);
  unsigned char *base = nullptr;
  int n_sms = 0;
  {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_dev_ptr[dev]) {
      void *p = nullptr;
      e = cudaGetSymbolAddress(&p, g_attn_scratch);
      if (e != cudaSuccess) return set_error(TS_ERR_CUDA, "cudaGetSymbolAddress(scratch): %s", cudaGetErrorString(e));
      int sms = 0;
      e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
      if (e != cudaSuccess) return set_error(TS_ERR_CUDA, "cudaDeviceGetAttribute: %s", cudaGetErrorString(e));
      g_sms[dev] = sms;
      g_dev_ptr[dev] = static_cast<unsigned char *>(p);
    }
    base = g_dev_ptr[dev];
    n_sms = g_sms[dev];
  }

  // same split rule as the verify step: about two CTAs per SM, one 64-position block per split at least
  const int nblk = (max_total + 63) / 64;
  int s = (2 * n_sms + a->n_kv_heads * tiles - 1) / (a->n_kv_heads * tiles);
  s = std::max(1, std::min(std::min(s, kMaxAttnSplits), nblk));
  s = (int)std::min<size_t>((size_t)s, kPartOBytes / per_split);

  cudaStream_t st = (cudaStream_t)stream;
  int32_t *tile_seq = reinterpret_cast<int32_t *>(base + kPartOBytes + kPartMlBytes);
  static_tile_table_kernel<<<1, 32, 0, st>>>((const int32_t *)a->cu_rows, a->batch, G, kMaxTiles, tile_seq,
                                             tile_seq + kMaxTiles);
  e = cudaGetLastError();
  if (e != cudaSuccess) return set_error(TS_ERR_CUDA, "tile-table launch: %s", cudaGetErrorString(e));

  ts::AttnArgs aa{};
  aa.in.cu_rows = a->cu_rows; aa.in.seq_len = a->seq_len; aa.in.block_tab = a->block_table;
  aa.in.pages_per_seq = a->pages_per_seq; aa.in.B = a->batch; aa.in.M = M;
  aa.q = (const __half *)a->q; aa.k_pages = (const __half *)a->k_pages; aa.v_pages = (const __half *)a->v_pages;
  aa.Hq = a->n_q_heads; aa.Hkv = a->n_kv_heads; aa.hd = a->head_dim;
  aa.n_splits = s; aa.n_row_tiles_total = tiles;
  aa.part_o = reinterpret_cast<float *>(base);
  aa.part_ml = reinterpret_cast<float2 *>(base + kPartOBytes);
  aa.tile_seq = tile_seq;
  aa.tile_row0 = tile_seq + kMaxTiles;
  aa.out = (__nv_bfloat16 *)a->out; aa.out_rows = a->out_rows; aa.planes = a->planes;
  e = ts::launch_attention_split(aa, st);
  if (e != cudaSuccess) return set_error(TS_ERR_CUDA, "attention launch: %s", cudaGetErrorString(e));
  e = ts::launch_attention_combine(aa, st);
  if (e != cudaSuccess) return set_error(TS_ERR_CUDA, "attention merge launch: %s", cudaGetErrorString(e));
  return TS_OK;
}
