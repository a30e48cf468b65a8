// Host side of the library: handles, buffer layout, weight upload, the verify step's kernel sequence,
// sessions (page lists, drafter state) and every extern "C" entry point declared in toolspec.h.
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <string>
#include <array>
#include <unordered_map>
#include <vector>

#include "drafter.h"
#include "kernels.h"
#include "schedule.h"
#include "toolspec.h"

namespace {

thread_local std::string g_err;

ts_status fail(ts_status code, const char *fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  g_err = buf;
  return code;
}

#define CU_TRY(expr)                                                                          \
  do {                                                                                        \
    cudaError_t e__ = (expr);                                                                 \
    if (e__ != cudaSuccess)                                                                   \
      return fail(TS_ERR_CUDA, "%s failed: %s (%s:%d)", #expr, cudaGetErrorString(e__), __FILE__, __LINE__); \
  } while (0)

inline uint64_t align_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

constexpr int kMaxSplits = 12;
constexpr int kMaxToolCandidates = 8;   // tool names verified in parallel while the name is open
constexpr int kMaxAttnSplits = ts::kAttnMaxSplits;
constexpr int kMcOptions[4] = {16, 32, 64, 128};
constexpr int kMaxFusedCtas = 256;   // the fused kernel runs one CTA per SM
constexpr int kFusedMaxRows = 64;    // most rows per step the fused kernel takes
constexpr bool kAutoPrefersFused = false;   // path = 0 picks the faster of the two on the 8B batch-1 step

struct Layout {
  // weights buffer (byte offsets)
  uint64_t embed, lm_head, gf;
  std::vector<uint64_t> wqkv, wo, wgu, wd, g1, g2;
  uint64_t weights_bytes;
  // kv pool
  uint64_t kv_layer_stride, kv_v_offset, kv_bytes;   // in fp16 elements / bytes
  // workspace (byte offsets)
  uint64_t x, h, part, q, attn_o, attn_ml, attn, act, logits, amax, rope, d_in, d_out, workspace_bytes;
  // fused single-kernel path
  uint64_t maps, slab, ss_part, sync, phase_t, stamps;
  int max_stamps;
  int n_maps, n_counters, n_phases, max_tiles128, o_tile128_seq, o_tile128_row0;
  int max_units, o_unit_tile, o_unit_leaf, o_row_leaves;   // attention units (see AttnTcArgs)
  // step io (int32 offsets inside d_in / h_in)
  int o_tokens, o_pos, o_rowseq, o_cu, o_len, o_tile_seq, o_tile_row0, o_btab, in_ints;
  int o_parent, o_anc, o_path, o_uni, o_topk, o_slot;
  uint64_t samp_stats, topk_cand;
  // step out (int32 offsets)
  int o_argmax, o_accept, o_emitted, o_newlen, o_newpend, o_err, out_ints;
  int rows_alloc, pages_per_seq, max_tiles, Nqkv, n_vocab_tiles;
  uint64_t host_io_bytes;
};

bool config_ok(const ts_model_config &c, const char **why) {
#define REQ(cond, msg) if (!(cond)) { *why = msg; return false; }
  REQ(c.n_layers > 0 && c.d_model > 0 && c.vocab > 0 && c.d_ffn > 0, "non-positive dimension");
  REQ(c.head_dim == 64 || c.head_dim == 128, "head_dim must be 64 or 128");
  REQ(c.n_q_heads > 0 && c.n_kv_heads > 0 && c.n_q_heads % c.n_kv_heads == 0, "q heads not a multiple of kv heads");
  REQ(c.d_model % 128 == 0 && c.d_ffn % 64 == 0 && c.vocab % 128 == 0, "d_model, vocab must be multiples of 128, d_ffn of 64");
  REQ(((c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim) % 128 == 0, "QKV width must be a multiple of 128");
  REQ((c.n_q_heads * c.head_dim) % 64 == 0, "attention width must be a multiple of 64");
  REQ(c.k_max >= 1 && c.k_max <= TS_K_MAX, "k_max out of range");
  REQ(c.max_batch >= 1 && c.max_rows >= c.k_max && c.max_rows <= c.max_batch * c.k_max, "max_rows out of range");
  REQ(c.max_ctx >= c.k_max && c.max_pages >= 1, "max_ctx / max_pages out of range");
  REQ(c.act_split == 0 || c.act_split == 1, "act_split must be 0 or 1");
  REQ(c.path >= 0 && c.path <= 2, "path must be 0 (auto), 1 (separate kernels) or 2 (fused kernel)");
  REQ(c.rope_theta > 1.f && c.rms_eps > 0.f, "rope_theta / rms_eps out of range");
#undef REQ
  return true;
}

void make_layout(const ts_model_config &c, Layout *L) {
  const uint64_t d = c.d_model, F = c.d_ffn, V = c.vocab, hd = c.head_dim;
  L->Nqkv = (c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim;
  const uint64_t Nq = (uint64_t)c.n_q_heads * hd;
  uint64_t o = 0;
  auto take = [&](uint64_t bytes) { uint64_t r = o; o = align_up(o + bytes, 1024); return r; };
  L->embed = take(V * d * 2);
  L->lm_head = take(V * d * 2);
  L->wqkv.resize(c.n_layers); L->wo.resize(c.n_layers); L->wgu.resize(c.n_layers); L->wd.resize(c.n_layers);
  L->g1.resize(c.n_layers); L->g2.resize(c.n_layers);
  for (int l = 0; l < c.n_layers; ++l) {
    L->wqkv[l] = take((uint64_t)L->Nqkv * d * 2);
    L->wo[l] = take(d * Nq * 2);
    L->wgu[l] = take(2 * F * d * 2);
    L->wd[l] = take(d * F * 2);
  }
  for (int l = 0; l < c.n_layers; ++l) { L->g1[l] = take(d * 4); L->g2[l] = take(d * 4); }
  L->gf = take(d * 4);
  L->weights_bytes = o;

  const uint64_t page_elems = (uint64_t)c.n_kv_heads * TS_PAGE_SIZE * hd;
  L->kv_v_offset = (uint64_t)c.max_pages * page_elems;
  L->kv_layer_stride = 2 * L->kv_v_offset;
  L->kv_bytes = (uint64_t)c.n_layers * L->kv_layer_stride * 2;

  L->rows_alloc = (int)align_up(c.max_rows, 128);
  L->pages_per_seq = (c.max_ctx + TS_PAGE_SIZE - 1) / TS_PAGE_SIZE;
  const int G = c.n_q_heads / c.n_kv_heads;
  L->max_tiles = c.max_batch * ((c.k_max * G + 63) / 64);
  L->n_vocab_tiles = c.vocab / 128;
  const uint64_t R = L->rows_alloc, planes = c.act_split ? 2 : 1;
  o = 0;
  L->x = take(R * d * 4);
  L->h = take(planes * R * d * 2);
  const uint64_t part_cols = std::max<uint64_t>(L->Nqkv, d);
  L->part = take((uint64_t)kMaxSplits * R * part_cols * 4);
  L->q = take(2 * R * Nq * 2);   // rotated queries, fp16: values [R][Nq], then their rounding remainders [R][Nq]
  L->attn_o = take(R * c.n_q_heads * kMaxAttnSplits * hd * 4);
  L->attn_ml = take(R * c.n_q_heads * kMaxAttnSplits * 8);
  L->attn = take(planes * R * Nq * 2);
  L->act = take(planes * R * F * 2);
  L->logits = take(R * V * 4);
  L->amax = take(R * 8);
  L->samp_stats = take(R * 16 * 4);
  L->topk_cand = take(R * (uint64_t)((c.vocab + 4095) / 4096) * TS_TOPK * 8);
  L->rope = take((uint64_t)c.max_ctx * (hd / 2) * 8);
  int io = 0;
  auto itake = [&](int n) { int r = io; io += (n + 3) / 4 * 4; return r; };
  L->o_tokens = itake(c.max_rows); L->o_pos = itake(c.max_rows); L->o_rowseq = itake(c.max_rows);
  L->o_cu = itake(c.max_batch + 1); L->o_len = itake(c.max_batch);
  L->o_tile_seq = itake(L->max_tiles); L->o_tile_row0 = itake(L->max_tiles);
  L->max_tiles128 = c.max_batch * ((c.k_max * G + 127) / 128);
  L->o_tile128_seq = itake(L->max_tiles128); L->o_tile128_row0 = itake(L->max_tiles128);
  L->max_units = L->max_tiles128 * kMaxAttnSplits;
  L->o_unit_tile = itake(L->max_units); L->o_unit_leaf = itake(L->max_units);
  L->o_row_leaves = itake(c.max_rows);
  L->o_parent = itake(c.max_rows); L->o_anc = itake(2 * c.max_rows); L->o_uni = itake(c.max_rows);
  L->o_slot = itake(c.max_rows);
  L->o_btab = itake(c.max_batch * L->pages_per_seq);   // (last: only the used part is copied per step)
  L->in_ints = io;
  io = 0;
  L->o_argmax = itake(c.max_rows); L->o_accept = itake(c.max_batch); L->o_emitted = itake(c.max_batch * c.k_max);
  L->o_newlen = itake(c.max_batch); L->o_newpend = itake(c.max_batch); L->o_err = itake(4);
  L->o_path = itake(c.max_batch * c.k_max);
  L->o_topk = itake(c.max_rows * TS_TOPK * 2);   // (id bits, value) pairs, written by the Top-K kernel
  L->out_ints = io;
  L->d_in = take((uint64_t)L->in_ints * 4);
  L->d_out = take((uint64_t)L->out_ints * 4);
  L->n_maps = 4 * c.n_layers + 1 + 3 * 3 + 1;
  L->maps = take((uint64_t)L->n_maps * sizeof(CUtensorMap));
  L->slab = take((uint64_t)kMaxFusedCtas * 2 * kFusedMaxRows * 128 * 4);
  L->ss_part = take((uint64_t)(d / 128) * R * 4);
  L->n_counters = (int)((L->Nqkv + 2 * d + 2 * F + V) / 128);
  L->sync = take((uint64_t)(8 + L->n_counters) * 4);
  L->n_phases = 6 * c.n_layers + 3;
  L->phase_t = take((uint64_t)3 * L->n_phases * 8);
  L->max_stamps = 9 * c.n_layers + 16;
  L->stamps = take((uint64_t)L->max_stamps * 4 * 8);
  L->workspace_bytes = o;
  L->host_io_bytes = align_up((uint64_t)(L->in_ints + L->out_ints) * 4, 4096);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

}  // namespace

namespace ts {
// records the thread's last error text for entry points that live in other translation units
ts_status set_error(ts_status code, const char *fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  g_err = buf;
  return code;
}
}  // namespace ts

struct ts_model {
  ts_model_config c{};
  ts_buffers b{};
  Layout L{};
  cudaStream_t st = nullptr;
  int planes = 1, n_sms = 148;
  int leaf_len = 64;   // KV positions per attention leaf: a constant of the model (see AttnTcArgs), set by ts_init_model
  size_t gemm_smem_budget = 100 * 1024;
  std::vector<CUtensorMap> tm_qkv, tm_o, tm_gu, tm_d;
  CUtensorMap tm_lm{}, tm_h[4]{}, tm_attn[4]{}, tm_act[4]{};
  std::vector<int32_t> free_pages;
  std::vector<ts_session *> sessions;   // live sessions over this model (detached on destroy)
  // last staged step
  int last_B = 0, last_M = 0, last_tiles = 0, last_tiles128 = 0, last_units = 0, last_slots = 1;
  uint32_t last_flags = 0;
  bool have_step = false;
  int64_t launches = 0, h2d = 0, d2h = 0;
  bool use_pdl = true;
  int32_t inject_err = 0;                      // test support: status code the next step is made to report
  bool fused_ok = false, last_fused = false;   // device can run the fused kernel; the staged step uses it
  bool last_tree = false;                      // the staged step verifies a draft tree (not a chain)
  bool last_sample = false;                    // the staged step accepts by speculative sampling
  float last_inv_t = 1.f;                      // 1 / temperature of that step
  size_t smem_optin = 0;
  // per-kernel timing pass (ts_profile_step): one event after every launch
  bool profiling = false;
  std::vector<cudaEvent_t> prof_ev;
  std::vector<int> prof_cls;
  // device-clock timeline (ts_debug_timeline): four stamps per launch of the step being recorded
  bool timeline = false;
  int stamp_idx = 0;
  std::vector<int> stamp_cls;
  unsigned long long *stamp_slot() const {
    return (timeline && stamp_idx < L.max_stamps) ? (unsigned long long *)WS(L.stamps) + 4 * (size_t)stamp_idx : nullptr;
  }
  void launched(int cls) {
    ++launches;
    if (timeline) { stamp_cls.push_back(cls); ++stamp_idx; }
    if (profiling) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) == cudaSuccess) {
        cudaEventRecord(e, st);
        prof_ev.push_back(e);
        prof_cls.push_back(cls);
      }
    }
  }

  uint8_t *W(uint64_t off) const { return (uint8_t *)b.weights + off; }
  uint8_t *WS(uint64_t off) const { return (uint8_t *)b.workspace + off; }
  int32_t *h_in() const { return (int32_t *)b.host_io; }
  int32_t *h_out() const { return (int32_t *)b.host_io + L.in_ints; }
  int32_t *d_in() const { return (int32_t *)WS(L.d_in); }
  int32_t *d_out() const { return (int32_t *)WS(L.d_out); }
  __half *k_pages(int l) const { return (__half *)b.kv_pool + (uint64_t)l * L.kv_layer_stride; }
  __half *v_pages(int l) const { return k_pages(l) + L.kv_v_offset; }
};

struct ts_session {
  ts_model *m = nullptr;
  const ts_schema *schema = nullptr;
  const ts_datastore *store = nullptr;
  ts_draft_config cfg{};
  ts::Fsm fsm;
  std::vector<int32_t> y, ranks, pages, last_chunk;
  std::vector<int32_t> prompt;                                         // kept for the context suffix match
  bool general_sd = false;                                             // drafts for q_v / q_o: context match, then recycled successors
  std::unordered_map<int32_t, std::array<int32_t, TS_TOPK>> successors;  // token -> the model's last Top-K after it
  bool have_ranks = false;
  int32_t cache_len = -1, pending = -1;
  bool finished = false;
};

namespace {

ts_status make_map(EncodeTiledFn enc, CUtensorMap *out, void *base, int rank, const uint64_t *dims,
                   const uint32_t *box) {
  cuuint64_t gdim[3], gstride[2];
  cuuint32_t bx[3], es[3] = {1, 1, 1};
  for (int i = 0; i < rank; ++i) { gdim[i] = dims[i]; bx[i] = box[i]; }
  gstride[0] = dims[0] * 2;
  if (rank == 3) gstride[1] = dims[0] * dims[1] * 2;
  CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, base, gdim, gstride, bx, es,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(TS_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
  return TS_OK;
}

// Weights are stored block by block: the 128 x 64 block (tile t, k-block kb) of an [N][K] matrix is the
// contiguous 16 KB at rows (t * K/64 + kb) * 128 .. of a [.][64] array.  One block is one TMA box and one run
// of DRAM pages.
ts_status weight_map(EncodeTiledFn enc, CUtensorMap *out, void *base, uint64_t N, uint64_t K) {
  const uint64_t dims[2] = {64, N * (K / 64)};
  const uint32_t box[2] = {64, 128};
  return make_map(enc, out, base, 2, dims, box);
}

ts_status act_maps(EncodeTiledFn enc, CUtensorMap *out4, void *base, uint64_t K, uint64_t rows, int planes) {
  for (int i = 0; i < 4; ++i) {
    const uint64_t dims[3] = {K, rows, (uint64_t)planes};
    const uint32_t box[3] = {64, (uint32_t)kMcOptions[i], (uint32_t)planes};
    ts_status s = make_map(enc, &out4[i], base, 3, dims, box);
    if (s) return s;
  }
  return TS_OK;
}

int pick_mc_index(int M) {
  for (int i = 0; i < 3; ++i)
    if (M <= kMcOptions[i]) return i;
  return 3;
}

// split-K factor: two CTAs fit on an SM, so the grid runs in waves of 2 * n_sms CTAs; take the smallest factor
// (at least 4 k-blocks per slice) whose last wave is at least 95% full, else the one that fills its waves best
int pick_splits(const ts_model *m, int n_tiles, int m_chunks, int n_kblocks, bool allow, int ctas_per_sm = 2) {
  if (!allow) return 1;
  const int ctas = std::max(1, n_tiles * m_chunks), slots = ctas_per_sm * m->n_sms;
  const int s_max = std::max(1, std::min(kMaxSplits, n_kblocks / 4));
  int best = 1;
  double best_eff = 0.0;
  for (int s = 1; s <= s_max; ++s) {
    const int waves = (ctas * s + slots - 1) / slots;
    const double eff = (double)(ctas * s) / ((double)waves * slots);
    if (eff > best_eff + 1e-9) { best_eff = eff; best = s; }
    if (eff >= 0.95) return s;
  }
  return best;
}

// split-K factor of the many-rows kernel (one CTA per SM, 128 x 256 output tile per CTA).  A CTA there costs about
// 13 k-blocks' worth of time besides its k-blocks (set-up, the first loads, 128 KB of partial sums written out), and
// every slice adds a slab of partial sums that the next kernel reads back: take the factor with the smallest
//   waves * (k-blocks per CTA + 13) + 2.5 * slices
// (measured on the 8B shape with 256 rows: 9 slices of 7 k-blocks in two waves took 29.5 us for the O projection,
// 4 slices of 16 in one wave 21 us, and the norm after it reads 4 slabs instead of 9).
int pick_splits_rows(const ts_model *m, int n_tiles, int m_chunks, int n_kblocks, bool allow) {
  if (!allow) return 1;
  const int ctas = std::max(1, n_tiles * m_chunks);
  const int s_max = std::max(1, std::min(kMaxSplits, n_kblocks / 4));
  int best = 1;
  double best_cost = 1e30;
  for (int s = 1; s <= s_max; ++s) {
    const int waves = (ctas * s + m->n_sms - 1) / m->n_sms;
    const double cost = waves * ((double)n_kblocks / s + 13.0) + 2.5 * s;
    if (cost < best_cost - 1e-9) { best_cost = cost; best = s; }
  }
  return best;
}

struct GemmPlan { int splits, kb_per_split; };

ts_status run_gemm(ts_model *m, int epi, const CUtensorMap &tw, const CUtensorMap *ta4, int N, int K, int M,
                   float *out, __nv_bfloat16 *act_out, unsigned long long *amax, GemmPlan *plan) {
  const int mi = pick_mc_index(M);
  ts::GemmArgs g{};
  g.N = N; g.K = K; g.M = M; g.Mc = kMcOptions[mi]; g.planes = m->planes;
  g.n_kblocks = K / 64;
  // Up to 64 rows the step is bound by streaming the weights (weight-major kernel, two CTAs per SM); beyond, by the
  // tensor cores and the bytes per flop an SM pulls from L2 (row-major kernel, 256 weight rows per CTA, one CTA per SM)
  const bool many_rows = M > 64;
  const int m_chunks = (M + g.Mc - 1) / g.Mc;
  int splits = many_rows ? pick_splits_rows(m, ts::gemm_rows_tiles(N), m_chunks, g.n_kblocks, epi == ts::EPI_PARTIAL)
                         : pick_splits(m, N / 128, m_chunks, g.n_kblocks, epi == ts::EPI_PARTIAL);
  g.kb_per_split = (g.n_kblocks + splits - 1) / splits;   // (the kernel cuts K into `splits` balanced runs)
  g.out = out; g.out_rows = m->L.rows_alloc;
  g.act_out = act_out; g.act_rows = m->L.rows_alloc; g.out_planes = m->planes;
  g.amax = amax;
  g.err = m->d_out() + m->L.o_err;
  g.stamp = m->stamp_slot();
  if (plan) { plan->splits = splits; plan->kb_per_split = g.kb_per_split; }
  if (many_rows)
    CU_TRY(ts::launch_gemm_rows(epi, tw, ta4[3], g, splits, m->smem_optin, m->n_sms, m->st, m->use_pdl && !m->profiling));
  else
    CU_TRY(ts::launch_gemm(epi, tw, ta4[mi], g, splits, m->gemm_smem_budget, m->st, m->use_pdl && !m->profiling));
  m->launched(0);
  return TS_OK;
}

// The staged step as one persistent kernel (fused.cu).
ts_status run_step_fused(ts_model *m) {
  const ts_model_config &c = m->c;
  const Layout &L = m->L;
  int32_t *di = m->d_in();
  int32_t *dout = m->d_out();
  ts::FusedArgs a{};
  a.n_layers = c.n_layers; a.d = c.d_model; a.Nqkv = L.Nqkv; a.Nq = c.n_q_heads * c.head_dim; a.F = c.d_ffn;
  a.V = c.vocab; a.Hq = c.n_q_heads; a.Hkv = c.n_kv_heads; a.hd = c.head_dim; a.eps = c.rms_eps;
  a.in.tokens = di + L.o_tokens; a.in.pos = di + L.o_pos; a.in.row_seq = di + L.o_rowseq; a.in.cu_rows = di + L.o_cu;
  a.in.seq_len = di + L.o_len; a.in.block_tab = di + L.o_btab; a.in.pages_per_seq = L.pages_per_seq;
  a.in.parent = di + L.o_parent; a.in.anc = (const uint32_t *)(di + L.o_anc); a.in.slot = di + L.o_slot;
  a.in.row_leaves = di + L.o_row_leaves;
  a.in.B = m->last_B; a.in.M = m->last_M;
  a.mc_index = pick_mc_index(m->last_M); a.Mc = kMcOptions[a.mc_index]; a.planes = m->planes;
  a.n_ctas = m->n_sms; a.skip_lm = (m->last_flags & TS_FLAG_SKIP_LM_HEAD) ? 1 : 0;
  a.k_max = c.k_max;
  a.n_attn_tiles = m->last_tiles128;
  {
    // (from the cached lengths and the model's k_max, not from this step's k, so that the cut does not change with the
    // number of rows verified)
    int max_total = 0;
    const int32_t *hi = m->h_in();
    for (int i = 0; i < m->last_B; ++i) max_total = std::max(max_total, hi[L.o_len + i] + c.k_max);
    const int nblk = (max_total + 63) / 64;
    const int G = c.n_q_heads / c.n_kv_heads;
    const int s = m->n_sms / std::max(1, c.n_kv_heads * m->last_B * ((c.k_max * G + 127) / 128));
    a.attn_splits = std::max(1, std::min(std::min(s, kMaxAttnSplits), nblk));
  }
  a.tile_seq = di + L.o_tile128_seq; a.tile_row0 = di + L.o_tile128_row0;
  a.maps = (const CUtensorMap *)m->WS(L.maps);
  a.map_kv = L.n_maps - 1;
  a.embed = (const __nv_bfloat16 *)m->W(L.embed);
  a.gains = (const float *)m->W(L.g1[0]);
  a.gain_stride = (int)(align_up((uint64_t)c.d_model * 4, 1024) / 4);
  a.rope = (const float2 *)m->WS(L.rope);
  a.kv_pool = (__half *)m->b.kv_pool; a.kv_layer_stride = L.kv_layer_stride; a.kv_v_offset = L.kv_v_offset;
  a.x = (float *)m->WS(L.x); a.h = (__nv_bfloat16 *)m->WS(L.h); a.attn = (__nv_bfloat16 *)m->WS(L.attn);
  a.act = (__nv_bfloat16 *)m->WS(L.act); a.R = L.rows_alloc; a.q = (__half *)m->WS(L.q);
  a.slab = (float *)m->WS(L.slab); a.ss_part = (float *)m->WS(L.ss_part);
  a.attn_o = (float *)m->WS(L.attn_o); a.attn_ml = (float2 *)m->WS(L.attn_ml);
  a.logits = (float *)m->WS(L.logits); a.amax = (unsigned long long *)m->WS(L.amax);
  a.sync = (int *)m->WS(L.sync); a.err = dout + L.o_err; a.n_counters = L.n_counters;
  a.phase_t = m->profiling ? (unsigned long long *)m->WS(L.phase_t) : nullptr;
  a.n_phases = L.n_phases;
  a.out_argmax = dout + L.o_argmax; a.out_accept = dout + L.o_accept; a.out_emitted = dout + L.o_emitted;
  a.out_newlen = dout + L.o_newlen; a.out_newpend = dout + L.o_newpend;
  CU_TRY(ts::launch_fused(a, m->smem_optin, m->st));
  m->launched(6);
  return TS_OK;
}

ts_status run_step(ts_model *m) {
  if (m->last_fused) return run_step_fused(m);
  const ts_model_config &c = m->c;
  const Layout &L = m->L;
  const int M = m->last_M, B = m->last_B;
  const int d = c.d_model, F = c.d_ffn, Nq = c.n_q_heads * c.head_dim;
  ts::StepIn in{};
  int32_t *di = m->d_in();
  in.tokens = di + L.o_tokens; in.pos = di + L.o_pos; in.row_seq = di + L.o_rowseq; in.cu_rows = di + L.o_cu;
  in.seq_len = di + L.o_len; in.block_tab = di + L.o_btab; in.pages_per_seq = L.pages_per_seq;
  in.parent = di + L.o_parent; in.anc = (const uint32_t *)(di + L.o_anc); in.slot = di + L.o_slot;
  in.row_leaves = di + L.o_row_leaves;
  in.B = B; in.M = M;
  in.ck.err = m->d_out() + L.o_err; in.ck.vocab = c.vocab; in.ck.max_pages = c.max_pages; in.ck.max_ctx = c.max_ctx;
  float *x = (float *)m->WS(L.x);
  __nv_bfloat16 *h = (__nv_bfloat16 *)m->WS(L.h);
  float *part = (float *)m->WS(L.part);
  __half *q = (__half *)m->WS(L.q);
  __nv_bfloat16 *attn = (__nv_bfloat16 *)m->WS(L.attn);
  __nv_bfloat16 *act = (__nv_bfloat16 *)m->WS(L.act);
  const float2 *rope = (const float2 *)m->WS(L.rope);
  const int R = L.rows_alloc;

  ts::AttnArgs aa{};
  aa.in = in; aa.q = q; aa.Hq = c.n_q_heads; aa.Hkv = c.n_kv_heads; aa.hd = c.head_dim;
  aa.n_row_tiles_total = m->last_tiles;
  aa.tile_seq = di + L.o_tile_seq; aa.tile_row0 = di + L.o_tile_row0;
  aa.part_o = (float *)m->WS(L.attn_o); aa.part_ml = (float2 *)m->WS(L.attn_ml);
  aa.out = attn; aa.out_rows = R; aa.planes = m->planes;
  {
    // enough CTAs for about two per SM, each split at least one 64-position block
    int max_total = 0;
    const int32_t *hi = m->h_in();
    for (int i = 0; i < B; ++i)
      max_total = std::max(max_total, hi[L.o_len + i] + (hi[L.o_cu + i + 1] - hi[L.o_cu + i]));
    const int nblk = (max_total + 63) / 64;
    int s = (2 * m->n_sms + c.n_kv_heads * m->last_tiles - 1) / (c.n_kv_heads * m->last_tiles);
    aa.n_splits = std::max(1, std::min(std::min(s, kMaxAttnSplits), nblk));
  }

  ts::AttnTcArgs at{};
  at.in = in; at.Hq = c.n_q_heads; at.Hkv = c.n_kv_heads; at.hd = c.head_dim;
  at.leaf_len = m->leaf_len; at.n_units = m->last_units; at.n_slots = m->last_slots; at.max_ctas = m->n_sms;
  at.unit_tile = di + L.o_unit_tile; at.unit_leaf = di + L.o_unit_leaf;
  at.tile_seq = di + L.o_tile128_seq; at.tile_row0 = di + L.o_tile128_row0;
  at.q = q; at.q_lo = q + (size_t)R * Nq; at.map_kv = (const CUtensorMap *)m->WS(L.maps) + (L.n_maps - 1);
  at.attn_o = aa.part_o; at.attn_ml = aa.part_ml; at.err = m->d_out() + L.o_err;
  at.out = attn; at.out_rows = R; at.planes = m->planes;
  CU_TRY(ts::launch_embed_norm(in, (const __nv_bfloat16 *)m->W(L.embed), (const float *)m->W(L.g1[0]), c.rms_eps,
                               d, x, h, R, m->planes, (unsigned long long *)m->WS(L.amax), m->st));
  m->launched(3);
  GemmPlan plan{};
  for (int l = 0; l < c.n_layers; ++l) {
    if (l > 0) {
      CU_TRY(ts::launch_add_norm(M, d, part, plan.splits, R, (const float *)m->W(L.g1[l]), c.rms_eps, x, h, R,
                                 m->planes, m->st, m->stamp_slot()));
      m->launched(3);
    }
    ts_status s = run_gemm(m, ts::EPI_PARTIAL, m->tm_qkv[l], m->tm_h, L.Nqkv, d, M, part, nullptr, nullptr, &plan);
    if (s) return s;
    CU_TRY(ts::launch_rope_kv(in, part, plan.splits, R, c.n_q_heads, c.n_kv_heads, c.head_dim, rope, q,
                              q + (size_t)R * Nq, m->k_pages(l), m->v_pages(l), m->st, m->stamp_slot()));
    m->launched(4);
    aa.k_pages = m->k_pages(l); aa.v_pages = m->v_pages(l);
    if (m->fused_ok) {   // tensor-memory attention (needs the same device features as the persistent kernel)
      at.layer = l;
      at.stamp = m->stamp_slot();
      CU_TRY(ts::launch_attention_tc(at, m->st));
      m->launched(1);
      at.stamp_merge = m->stamp_slot();
      CU_TRY(ts::launch_attention_tc_merge(at, m->st));
    } else {
      CU_TRY(ts::launch_attention_split(aa, m->st));
      m->launched(1);
      CU_TRY(ts::launch_attention_combine(aa, m->st));
    }
    m->launched(2);
    s = run_gemm(m, ts::EPI_PARTIAL, m->tm_o[l], m->tm_attn, d, Nq, M, part, nullptr, nullptr, &plan);
    if (s) return s;
    CU_TRY(ts::launch_add_norm(M, d, part, plan.splits, R, (const float *)m->W(L.g2[l]), c.rms_eps, x, h, R,
                               m->planes, m->st, m->stamp_slot()));
    m->launched(3);
    // (gate-up keeps its SwiGLU epilogue and so cannot split K: 192 tiles run as 1.3 waves.  Splitting K
    // three ways with a separate SwiGLU kernel filled the waves but cost as much as it saved.)
    s = run_gemm(m, ts::EPI_SWIGLU, m->tm_gu[l], m->tm_h, 2 * F, d, M, nullptr, act, nullptr, nullptr);
    if (s) return s;
    s = run_gemm(m, ts::EPI_PARTIAL, m->tm_d[l], m->tm_act, d, F, M, part, nullptr, nullptr, &plan);
    if (s) return s;
  }
  if (m->last_flags & TS_FLAG_SKIP_LM_HEAD) return TS_OK;
  CU_TRY(ts::launch_add_norm(M, d, part, plan.splits, R, (const float *)m->W(L.gf), c.rms_eps, x, h, R, m->planes,
                             m->st, m->stamp_slot()));
  m->launched(3);
  unsigned long long *amax = (unsigned long long *)m->WS(L.amax);
  ts_status s = run_gemm(m, ts::EPI_LOGITS, m->tm_lm, m->tm_h, c.vocab, d, M, (float *)m->WS(L.logits), nullptr,
                         amax, nullptr);
  if (s) return s;
  int32_t *dout = m->d_out();
  if (m->last_flags & TS_FLAG_WANT_TOPK) {   // per-position Top-K of the logits, for the successor tables
    CU_TRY(ts::launch_topk_rows((const float *)m->WS(L.logits), M, c.vocab, TS_TOPK, (float2 *)m->WS(L.topk_cand),
                                (float *)(dout + L.o_topk), m->st));
    m->launched(5);
    m->launched(5);
  }
  if (m->last_sample) {
    ts::SampleArgs sa{};
    sa.in = in; sa.logits = (float *)m->WS(L.logits); sa.amax = amax;
    sa.uni = (const float *)(di + L.o_uni); sa.part = (float *)m->WS(L.samp_stats);
    sa.V = c.vocab; sa.inv_t = m->last_inv_t; sa.k_max = c.k_max;
    sa.argmax = dout + L.o_argmax; sa.accept_len = dout + L.o_accept; sa.emitted = dout + L.o_emitted;
    sa.new_len = dout + L.o_newlen; sa.new_pending = dout + L.o_newpend; sa.path = dout + L.o_path;
    CU_TRY(ts::launch_sample_accept(sa, m->st));
    m->launched(5);
    m->launched(5);
  } else {
    ts::AcceptArgs ac{};
    ac.in = in; ac.amax = amax;
    ac.argmax = dout + L.o_argmax; ac.accept_len = dout + L.o_accept; ac.emitted = dout + L.o_emitted;
    ac.new_len = dout + L.o_newlen; ac.new_pending = dout + L.o_newpend; ac.k_max = c.k_max;
    ac.path = dout + L.o_path;
    CU_TRY(ts::launch_accept(ac, m->st));
    m->launched(5);
  }
  if (m->last_tree) {   // the accepted path's K/V rows become the next cache positions
    ts::CompactArgs ca{};
    ca.in = in; ca.accept_len = dout + L.o_accept; ca.path = dout + L.o_path; ca.k_max = c.k_max;
    ca.kv_pool = (__half *)m->b.kv_pool; ca.layer_stride = L.kv_layer_stride; ca.v_offset = L.kv_v_offset;
    ca.n_layers = c.n_layers; ca.Hkv = c.n_kv_heads; ca.hd = c.head_dim;
    CU_TRY(ts::launch_kv_compact(ca, m->st));
    m->launched(5);
  }
  return TS_OK;
}

ts_status ensure_pages(ts_session *s, int tokens) {
  ts_model *m = s->m;
  const int need = (tokens + TS_PAGE_SIZE - 1) / TS_PAGE_SIZE;
  if (need > m->L.pages_per_seq) return fail(TS_ERR_ARG, "sequence of %d tokens exceeds max_ctx %d", tokens, m->c.max_ctx);
  while ((int)s->pages.size() < need) {
    if (m->free_pages.empty()) return fail(TS_ERR_OOM_PAGES, "KV page pool exhausted (%d pages)", m->c.max_pages);
    s->pages.push_back(m->free_pages.back());
    m->free_pages.pop_back();
  }
  return TS_OK;
}

// Stage one step: rows[i] = chunk ids of sequence i.  Copies inputs, runs, copies results back, syncs.
// parents (optional): parents[i][j] = chunk row that row j of sequence i hangs from (-1 for row 0); a chain if null.
ts_status stage_and_run(ts_model *m, ts_session *const *ss, int B, const std::vector<std::vector<int32_t>> &rows,
                        uint32_t flags, const std::vector<std::vector<int32_t>> *parents = nullptr,
                        const float *uniforms = nullptr, float temperature = 0.f) {
  const ts_model_config &c = m->c;
  const Layout &L = m->L;
  int32_t *hi = m->h_in();
  const int G = c.n_q_heads / c.n_kv_heads;
  int M = 0, tiles = 0, tiles128 = 0;
  hi[L.o_cu] = 0;
  for (int i = 0; i < B; ++i) {
    ts_session *s = ss[i];
    const int k = (int)rows[i].size();
    if (k < 1 || k > c.k_max) return fail(TS_ERR_K_TOO_LARGE, "sequence %d: chunk of %d rows, k_max is %d", i, k, c.k_max);
    if (M + k > c.max_rows) return fail(TS_ERR_K_TOO_LARGE, "step has more than max_rows = %d rows", c.max_rows);
    if (s->cache_len + k > c.max_ctx) return fail(TS_ERR_ARG, "sequence %d would exceed max_ctx", i);
    for (int t : rows[i])
      if (t < 0 || t >= c.vocab) return fail(TS_ERR_TOKEN_RANGE, "token id %d outside [0, %d)", t, c.vocab);
    ts_status st = ensure_pages(s, s->cache_len + k);
    if (st) return st;
    if (parents && k > 64) return fail(TS_ERR_K_TOO_LARGE, "sequence %d: a draft tree holds at most 64 rows", i);
    uint64_t anc[64];
    int depth[64];
    for (int j = 0; j < k; ++j) {
      const int par = parents ? (*parents)[i][j] : j - 1;
      if (parents) {
        if ((j == 0) != (par == -1) || par >= j || par < -1)
          return fail(TS_ERR_ARG, "sequence %d: parent of row %d must be an earlier row (-1 only for row 0)", i, j);
        depth[j] = j == 0 ? 0 : depth[par] + 1;
        anc[j] = (j == 0 ? 0ull : anc[par]) | (1ull << j);
        // the residual walk of speculative sampling removes a refused child's token from the distribution: two
        // children of one node carrying the same token would remove it twice
        if (uniforms)
          for (int e = 1; e < j; ++e)
            if ((*parents)[i][e] == par && rows[i][e] == rows[i][j])
              return fail(TS_ERR_ARG, "sequence %d: rows %d and %d are children of row %d with the same token", i, e, j, par);
      }
      const uint64_t mask = parents ? anc[j] : (j >= 63 ? ~0ull : ((2ull << j) - 1ull));
      hi[L.o_tokens + M + j] = rows[i][j];
      hi[L.o_pos + M + j] = s->cache_len + (parents ? depth[j] : j);
      hi[L.o_rowseq + M + j] = i;
      hi[L.o_slot + M + j] = s->cache_len + j;
      hi[L.o_parent + M + j] = par;
      hi[L.o_anc + 2 * (M + j)] = (int32_t)(uint32_t)(mask & 0xFFFFFFFFull);
      hi[L.o_anc + 2 * (M + j) + 1] = (int32_t)(uint32_t)(mask >> 32);
    }
    hi[L.o_len + i] = s->cache_len;
    for (int r0 = 0; r0 < k * G; r0 += 64) {
      hi[L.o_tile_seq + tiles] = i;
      hi[L.o_tile_row0 + tiles] = r0;
      ++tiles;
    }
    tiles128 += (k * G + 127) / 128;
    std::memcpy(hi + L.o_btab + (size_t)i * L.pages_per_seq, s->pages.data(), s->pages.size() * sizeof(int32_t));
    M += k;
    hi[L.o_cu + i + 1] = M;
  }
  {
    // 128-row tiles, longest sequence first: the attention kernel's CTAs are handed out in tile order, so the long
    // units start first and the short ones fill the tail
    std::vector<int> order(B);
    for (int i = 0; i < B; ++i) order[i] = i;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
      return hi[L.o_len + a] + (hi[L.o_cu + a + 1] - hi[L.o_cu + a]) > hi[L.o_len + b] + (hi[L.o_cu + b + 1] - hi[L.o_cu + b]);
    });
    int t = 0;
    // (tile, leaf) pairs of the attention kernel: leaf L of a sequence is the absolute positions [L, L + 1) * leaf_len
    struct Unit { int tile, leaf, nblk; };
    std::vector<Unit> units;
    int slots = 1;
    for (int i : order) {
      const int k = hi[L.o_cu + i + 1] - hi[L.o_cu + i], total = hi[L.o_len + i] + k;
      const int n_leaves = (total + m->leaf_len - 1) / m->leaf_len;
      slots = std::max(slots, n_leaves);
      for (int r = hi[L.o_cu + i]; r < hi[L.o_cu + i + 1]; ++r) hi[L.o_row_leaves + r] = n_leaves;
      for (int r0 = 0; r0 < k * G; r0 += 128) {
        hi[L.o_tile128_seq + t] = i;
        hi[L.o_tile128_row0 + t] = r0;
        for (int lf = 0; lf < n_leaves; ++lf)
          units.push_back({t, lf, (std::min(total, (lf + 1) * m->leaf_len) - lf * m->leaf_len + 63) / 64});
        ++t;
      }
    }
    // whole leaves first, the shorter last leaves at the end, where they fill the tail of the last wave
    std::stable_sort(units.begin(), units.end(), [](const Unit &a, const Unit &b) { return a.nblk > b.nblk; });
    if ((int)units.size() > L.max_units) return fail(TS_ERR_ARG, "internal: %zu attention units exceed %d", units.size(), L.max_units);
    for (size_t u = 0; u < units.size(); ++u) {
      hi[L.o_unit_tile + u] = units[u].tile;
      hi[L.o_unit_leaf + u] = units[u].leaf;
    }
    m->last_units = (int)units.size();
    m->last_slots = slots;
  }
  const bool can_fuse = m->fused_ok && M <= kFusedMaxRows;
  if (c.path == 2 && !can_fuse)
    return fail(TS_ERR_K_TOO_LARGE, "the fused kernel takes at most %d rows on a device that supports it (step has %d)",
                kFusedMaxRows, M);
  m->last_tree = parents != nullptr;
  if (m->last_tree && (c.path == 2 || !m->fused_ok))
    return fail(TS_ERR_UNIMPLEMENTED, "draft trees need the one-kernel-per-stage path with tensor-memory attention");
  m->last_sample = uniforms != nullptr;
  if (m->last_sample) {
    if (c.path == 2) return fail(TS_ERR_UNIMPLEMENTED, "sampling acceptance needs the one-kernel-per-stage path");
    m->last_inv_t = 1.f / temperature;
    // the kernel reads uni[node c] for node c and the root's for the draw; a chain's caller gives value j for draft
    // j + 1 and its chunk's last value for the draw
    float *un = reinterpret_cast<float *>(hi + L.o_uni);
    if (m->last_tree) {
      std::memcpy(un, uniforms, sizeof(float) * M);
    } else {
      for (int i = 0, r = 0; i < B; ++i) {
        const int k = hi[L.o_cu + i + 1] - hi[L.o_cu + i];
        un[r] = uniforms[r + k - 1];
        for (int j = 1; j < k; ++j) un[r + j] = uniforms[r + j - 1];
        r += k;
      }
    }
  }
  if ((flags & TS_FLAG_WANT_TOPK) && c.path == 2)
    return fail(TS_ERR_UNIMPLEMENTED, "the per-position Top-K needs the one-kernel-per-stage path");
  m->last_fused = !m->last_tree && !m->last_sample && !(flags & TS_FLAG_WANT_TOPK) && can_fuse &&
                  (c.path == 2 || (c.path == 0 && kAutoPrefersFused));
  m->last_B = B; m->last_M = M; m->last_tiles = tiles; m->last_tiles128 = tiles128; m->last_flags = flags;
  m->have_step = true;
  const size_t in_bytes = (size_t)(L.o_btab + (size_t)B * L.pages_per_seq) * 4;
  CU_TRY(cudaMemcpyAsync(m->d_in(), hi, in_bytes, cudaMemcpyHostToDevice, m->st));
  m->h2d += (int64_t)in_bytes;
  ts_status st = run_step(m);
  if (st) return st;
  if (m->inject_err) {
    // test support (ts_debug_inject_device_error): after the step's last kernel, write the status word an expired
    // device-side wait would have left; the code below must then treat the step as failed
    m->h_out()[L.o_err + 1] = m->inject_err;
    m->inject_err = 0;
    CU_TRY(cudaMemcpyAsync(m->d_out() + L.o_err, m->h_out() + L.o_err + 1, 4, cudaMemcpyHostToDevice, m->st));
  }
  const size_t out_bytes = (size_t)L.out_ints * 4;
  CU_TRY(cudaMemcpyAsync(m->h_out(), m->d_out(), out_bytes, cudaMemcpyDeviceToHost, m->st));
  m->d2h += (int64_t)out_bytes;
  CU_TRY(cudaStreamSynchronize(m->st));
  const int dev_err = m->h_out()[L.o_err];
  if (dev_err != 0) {
    cudaMemsetAsync(m->d_out() + L.o_err, 0, 4, m->st);
    cudaMemsetAsync(m->WS(L.sync), 0, (size_t)(8 + L.n_counters) * 4, m->st);   // the fused kernel left its counters mid-step
    if (dev_err >= ts::DEV_BOUNDS)
      return fail(TS_ERR_DEVICE_BOUNDS, "an index check of the debug build failed on the device (check %d)", dev_err - ts::DEV_BOUNDS);
    return fail(TS_ERR_DEVICE_TIMEOUT, "a bounded device-side wait expired (code %d)", dev_err);
  }
  return TS_OK;
}

// y <- y (+) ids, delta per id, stop at the first finishing id.  Returns ids consumed.
int commit_ids(ts_session *s, const int32_t *ids, int n) {
  int used = 0;
  for (int j = 0; j < n && !s->finished; ++j) {
    s->y.push_back(ids[j]);
    if (s->schema) s->fsm.step(ids[j]);
    ++used;
    const bool done = (s->schema && s->fsm.kind == ts::Q_DONE) ||
                      (s->schema && ids[j] == s->schema->v.eos) ||
                      (int)s->y.size() >= s->cfg.max_new_tokens;
    if (done) s->finished = true;
  }
  return used;
}

int guess_tool(const ts_session *s) {
  const ts_schema *sc = s->schema;
  const ts::TrieNode &node = sc->trie[s->fsm.stage == ts::ST_NAME ? s->fsm.node : 0];
  if (node.tools.empty()) return -1;
  if (s->have_ranks && s->store) {
    for (int32_t cnd : s->ranks) {
      const int32_t t = s->store->tool_of[cnd];
      if (t >= 0 && std::binary_search(node.tools.begin(), node.tools.end(), t)) return t;
    }
  }
  int best = node.tools[0];
  if (s->store) {
    for (int32_t t : node.tools) {
      const int64_t ft = t < (int32_t)s->store->freq.size() ? s->store->freq[t] : 0;
      const int64_t fb = best < (int32_t)s->store->freq.size() ? s->store->freq[best] : 0;
      if (ft > fb) best = t;
    }
  }
  return best;
}

}  // namespace

// =====================================================================================================
extern "C" {

const char *ts_last_error(void) { return g_err.c_str(); }

ts_status ts_query_buffer_sizes(const ts_model_config *cfg, ts_buffer_sizes *out) {
  if (!cfg || !out) return fail(TS_ERR_ARG, "null argument");
  const char *why = "";
  if (!config_ok(*cfg, &why)) return fail(TS_ERR_ARG, "bad configuration: %s", why);
  Layout L;
  make_layout(*cfg, &L);
  out->weights_bytes = L.weights_bytes;
  out->kv_pool_bytes = L.kv_bytes;
  out->workspace_bytes = L.workspace_bytes;
  out->host_io_bytes = L.host_io_bytes;
  return TS_OK;
}

ts_status ts_init_model(const ts_model_config *cfg, const ts_buffers *bufs, void *stream, ts_model **out) {
  if (!cfg || !bufs || !out) return fail(TS_ERR_ARG, "null argument");
  const char *why = "";
  if (!config_ok(*cfg, &why)) return fail(TS_ERR_ARG, "bad configuration: %s", why);
  if (!bufs->weights || !bufs->kv_pool || !bufs->workspace || !bufs->host_io) return fail(TS_ERR_ARG, "null buffer");
  if (((uintptr_t)bufs->weights | (uintptr_t)bufs->kv_pool | (uintptr_t)bufs->workspace) & 1023)
    return fail(TS_ERR_ARG, "device buffers must be 1024-byte aligned");
  int dev = 0;
  CU_TRY(cudaGetDevice(&dev));
  cudaDeviceProp prop;
  CU_TRY(cudaGetDeviceProperties(&prop, dev));
  if (prop.major != 10) return fail(TS_ERR_CUDA, "device is sm_%d%d; this library is built for sm_100a only", prop.major, prop.minor);
  void *fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  CU_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
  if (!fn || qres != cudaDriverEntryPointSuccess) return fail(TS_ERR_CUDA, "cuTensorMapEncodeTiled not available");
  EncodeTiledFn enc = (EncodeTiledFn)fn;

  ts_model *m = new ts_model();
  m->c = *cfg; m->b = *bufs; m->st = (cudaStream_t)stream;
  m->planes = cfg->act_split ? 2 : 1;
  m->n_sms = prop.multiProcessorCount;
  make_layout(*cfg, &m->L);
  const Layout &L = m->L;
  const ts_model_config &c = m->c;
  auto bail = [&](ts_status s) { delete m; return s; };

  cudaError_t e = cudaMemsetAsync(bufs->workspace, 0, L.workspace_bytes, m->st);
  if (e != cudaSuccess) return bail(fail(TS_ERR_CUDA, "cudaMemsetAsync(workspace): %s", cudaGetErrorString(e)));
  {
    // rotary table in double precision: (cos, sin) of pos * theta^(-2i/hd)
    const int half = c.head_dim / 2;
    std::vector<float2> tab((size_t)c.max_ctx * half);
    std::vector<double> inv(half);
    for (int i = 0; i < half; ++i) inv[i] = std::pow((double)c.rope_theta, -2.0 * i / c.head_dim);
    for (int p = 0; p < c.max_ctx; ++p)
      for (int i = 0; i < half; ++i) {
        const double ang = (double)p * inv[i];
        tab[(size_t)p * half + i] = make_float2((float)std::cos(ang), (float)std::sin(ang));
      }
    e = cudaMemcpyAsync(m->WS(L.rope), tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice, m->st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(m->st);
    if (e != cudaSuccess) return bail(fail(TS_ERR_CUDA, "rotary table upload: %s", cudaGetErrorString(e)));
  }
  const uint64_t d = c.d_model, F = c.d_ffn, Nq = (uint64_t)c.n_q_heads * c.head_dim;
  m->tm_qkv.resize(c.n_layers); m->tm_o.resize(c.n_layers); m->tm_gu.resize(c.n_layers); m->tm_d.resize(c.n_layers);
  ts_status s = TS_OK;
  for (int l = 0; l < c.n_layers && !s; ++l) {
    s = weight_map(enc, &m->tm_qkv[l], m->W(L.wqkv[l]), L.Nqkv, d);
    if (!s) s = weight_map(enc, &m->tm_o[l], m->W(L.wo[l]), d, Nq);
    if (!s) s = weight_map(enc, &m->tm_gu[l], m->W(L.wgu[l]), 2 * F, d);
    if (!s) s = weight_map(enc, &m->tm_d[l], m->W(L.wd[l]), d, F);
  }
  if (!s) s = weight_map(enc, &m->tm_lm, m->W(L.lm_head), c.vocab, d);
  if (!s) s = act_maps(enc, m->tm_h, m->WS(L.h), d, L.rows_alloc, m->planes);
  if (!s) s = act_maps(enc, m->tm_attn, m->WS(L.attn), Nq, L.rows_alloc, m->planes);
  if (!s) s = act_maps(enc, m->tm_act, m->WS(L.act), F, L.rows_alloc, m->planes);
  if (s) return bail(s);
  {
    // the fused kernel reads its tensor maps from device memory
    std::vector<CUtensorMap> maps(L.n_maps);
    for (int l = 0; l < c.n_layers; ++l) {
      maps[4 * l + 0] = m->tm_qkv[l]; maps[4 * l + 1] = m->tm_o[l]; maps[4 * l + 2] = m->tm_gu[l]; maps[4 * l + 3] = m->tm_d[l];
    }
    maps[4 * c.n_layers] = m->tm_lm;
    for (int i = 0; i < 3; ++i) {
      maps[4 * c.n_layers + 1 + 3 * i + 0] = m->tm_h[i];
      maps[4 * c.n_layers + 1 + 3 * i + 1] = m->tm_attn[i];
      maps[4 * c.n_layers + 1 + 3 * i + 2] = m->tm_act[i];
    }
    {
      // paged KV pool as a 5-d tensor: 64-element half of a head row, 16 positions of a page, kv head, page,
      // (layer, K|V); one box = one page of one head = 16 rows of 128 bytes
      const uint64_t hd = c.head_dim, page_bytes = (uint64_t)c.n_kv_heads * TS_PAGE_SIZE * hd * 2;
      cuuint64_t gdim[5] = {hd, TS_PAGE_SIZE, (cuuint64_t)c.n_kv_heads, (cuuint64_t)c.max_pages, (cuuint64_t)2 * c.n_layers};
      cuuint64_t gstr[4] = {hd * 2, TS_PAGE_SIZE * hd * 2, page_bytes, (cuuint64_t)c.max_pages * page_bytes};
      cuuint32_t box[5] = {64, TS_PAGE_SIZE, 1, 1, 1}, es[5] = {1, 1, 1, 1, 1};
      CUresult r = enc(&maps[L.n_maps - 1], CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 5, bufs->kv_pool, gdim, gstr, box, es,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
      if (r != CUDA_SUCCESS) return bail(fail(TS_ERR_CUDA, "cuTensorMapEncodeTiled(kv pool) failed with code %d", (int)r));
    }
    // Attention multiplies masked positions by zero, so every cache position that can be read must hold a
    // finite value: start from an all-zero pool.
    e = cudaMemsetAsync(bufs->kv_pool, 0, L.kv_bytes, m->st);
    if (e != cudaSuccess) return bail(fail(TS_ERR_CUDA, "cudaMemsetAsync(kv pool): %s", cudaGetErrorString(e)));
    e = cudaMemcpyAsync(m->WS(L.maps), maps.data(), maps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice, m->st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(m->st);
    if (e != cudaSuccess) return bail(fail(TS_ERR_CUDA, "tensor map upload: %s", cudaGetErrorString(e)));
    int coop = 0, optin = 0;
    cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
    cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    m->smem_optin = (size_t)optin;
    m->fused_ok = coop != 0 && m->n_sms <= kMaxFusedCtas &&
                  ts::fused_ring_stages(m->planes, kFusedMaxRows, c.head_dim, m->smem_optin) >= 2;
  }
  {
    // Attention leaf length.  A constant of the model, NOT of the step: a row's bits must not depend on the step's
    // shape.  Chosen so that a full batch at full context gives about one unit of work per SM -- groups = (sequence,
    // row tile, kv head) triples of a full step, leaves per group = 95% of the SMs / groups, at least 4 and at most
    // 16 -- in whole 64-position blocks: a batch-1 model gets many short leaves (its few groups must
    // cover the SMs), a batched one a few long ones (a leaf costs a fixed start-up and one partial result per row;
    // four per full-length sequence still let ragged batches be dealt out evenly over the SMs).
    const int G = c.n_q_heads / c.n_kv_heads;
    const int groups = c.max_batch * ((c.k_max * G + 127) / 128) * c.n_kv_heads;
    // (at most 16: the merge kernel is unrolled over 2, 4, 8, 16 or 32 leaves, and 17 leaves cost it a fifth more
    // than 15 while the attention kernel gains nothing)
    const int want = std::max(4, std::min(16, (int)(0.95 * m->n_sms) / std::max(1, groups)));
    const int blocks = (c.max_ctx + 63) / 64;
    int leaf_blocks = std::max(1, (blocks + want - 1) / want);
    while ((blocks + leaf_blocks - 1) / leaf_blocks > kMaxAttnSplits) ++leaf_blocks;
    m->leaf_len = 64 * leaf_blocks;
  }
  m->free_pages.resize(c.max_pages);
  for (int i = 0; i < c.max_pages; ++i) m->free_pages[i] = c.max_pages - 1 - i;   // hand out 0, 1, 2, ...
  *out = m;
  return TS_OK;
}

ts_status ts_model_destroy(ts_model *m) {
  if (!m) return TS_OK;
  cudaStreamSynchronize(m->st);
  for (ts_session *s : m->sessions) {   // sessions outlive the model as host-only sessions
    s->m = nullptr;
    s->pages.clear();
  }
  delete m;
  return TS_OK;
}

ts_status ts_load_tensor(ts_model *m, int32_t kind, int32_t layer, const void *host, int64_t rows, int64_t cols) {
  if (!m || !host) return fail(TS_ERR_ARG, "null argument");
  const ts_model_config &c = m->c;
  const Layout &L = m->L;
  const int64_t d = c.d_model, F = c.d_ffn, hd = c.head_dim, Nq = (int64_t)c.n_q_heads * hd, Nkv = (int64_t)c.n_kv_heads * hd;
  const bool global = kind == TS_W_EMBED || kind == TS_W_LM_HEAD || kind == TS_W_FINAL_GAIN;
  if (!global && (layer < 0 || layer >= c.n_layers)) return fail(TS_ERR_ARG, "layer %d out of range", layer);
  int64_t er = 0, ec = 0;
  uint8_t *dst = nullptr;
  size_t esz = 2;
  ts::RowMap rm{0, 1, 0, 0};
  switch (kind) {
    case TS_W_EMBED: er = c.vocab; ec = d; dst = m->W(L.embed); break;
    case TS_W_LM_HEAD: er = c.vocab; ec = d; dst = m->W(L.lm_head); rm.tiles = (c.vocab + 127) / 128; break;
    case TS_W_FINAL_GAIN: er = 1; ec = d; dst = m->W(L.gf); esz = 4; break;
    case TS_W_GAIN1: er = 1; ec = d; dst = m->W(L.g1[layer]); esz = 4; break;
    case TS_W_GAIN2: er = 1; ec = d; dst = m->W(L.g2[layer]); esz = 4; break;
    case TS_W_Q: er = Nq; ec = d; dst = m->W(L.wqkv[layer]); rm.base = 0; rm.hd = (int)hd; rm.tiles = L.Nqkv / 128; break;
    case TS_W_K: er = Nkv; ec = d; dst = m->W(L.wqkv[layer]); rm.base = (int)Nq; rm.hd = (int)hd; rm.tiles = L.Nqkv / 128; break;
    case TS_W_V: er = Nkv; ec = d; dst = m->W(L.wqkv[layer]); rm.base = (int)(Nq + Nkv); rm.hd = (int)hd; rm.tiles = L.Nqkv / 128; break;
    case TS_W_O: er = d; ec = Nq; dst = m->W(L.wo[layer]); rm.tiles = (int)(d / 128); break;
    case TS_W_GATE: er = F; ec = d; dst = m->W(L.wgu[layer]); rm.mul = 2; rm.tiles = (int)(2 * F / 128); break;               // even rows
    case TS_W_UP: er = F; ec = d; dst = m->W(L.wgu[layer]); rm.mul = 2; rm.base = 1; rm.tiles = (int)(2 * F / 128); break;    // odd rows
    case TS_W_DOWN: er = d; ec = F; dst = m->W(L.wd[layer]); rm.tiles = (int)(d / 128); break;
    default: return fail(TS_ERR_ARG, "unknown tensor kind %d", kind);
  }
  if (rows != er || cols != ec) return fail(TS_ERR_ARG, "tensor kind %d: expected %lld x %lld, got %lld x %lld", kind,
                                            (long long)er, (long long)ec, (long long)rows, (long long)cols);
  const size_t row_bytes = (size_t)ec * esz;
  if (esz == 4 || kind == TS_W_EMBED) {   // gains and the embedding table stay row-major
    CU_TRY(cudaMemcpyAsync(dst, host, row_bytes * (size_t)er, cudaMemcpyDefault, m->st));
    CU_TRY(cudaStreamSynchronize(m->st));
    return TS_OK;
  }
  // Projection matrices: rows go to their place in the stored matrix (Q, K, V concatenated, with rotary
  // partners i and i + hd/2 on adjacent rows 2i and 2i+1; gate and up rows interleaved) and the matrix is
  // stored as 128 x 64 blocks.  Host sources pass through a staging area inside the workspace.
  cudaPointerAttributes pa{};
  const bool on_device = cudaPointerGetAttributes(&pa, host) == cudaSuccess && pa.type == cudaMemoryTypeDevice;
  cudaGetLastError();
  const size_t stage_bytes = (size_t)L.rows_alloc * (size_t)c.vocab * 4;   // the logits area doubles as staging
  const int64_t rows_per_chunk = on_device ? er : std::max<int64_t>(1, (int64_t)(stage_bytes / row_bytes));
  for (int64_t r0 = 0; r0 < er; r0 += rows_per_chunk) {
    const int64_t nr = std::min(rows_per_chunk, er - r0);
    const void *src = (const uint8_t *)host + (size_t)r0 * row_bytes;
    if (!on_device) {
      CU_TRY(cudaMemcpyAsync(m->WS(L.logits), src, (size_t)nr * row_bytes, cudaMemcpyHostToDevice, m->st));
      src = m->WS(L.logits);
    }
    CU_TRY(ts::launch_retile((const __nv_bfloat16 *)src, (int)nr, (int)r0, (int)ec, rm, (__nv_bfloat16 *)dst, m->st));
    CU_TRY(cudaStreamSynchronize(m->st));
  }
  m->have_step = false;   // the staging area held the last step's logits
  return TS_OK;
}

// ---- schema ------------------------------------------------------------------------------------------
ts_status ts_schema_create(const ts_vocab_layout *v, ts_schema **out) {
  if (!v || !out) return fail(TS_ERR_ARG, "null argument");
  const int32_t lens[5] = {v->pfx_len, v->mid_len, v->kvsep_len, v->nxt_len, v->end_len};
  for (int i = 0; i < 5; ++i)
    if (lens[i] < (i == 0 ? 0 : 1) || lens[i] > 8) return fail(TS_ERR_ARG, "scaffolding string length out of range");
  ts_schema *s = new ts_schema();
  s->v = *v;
  s->trie.emplace_back();
  *out = s;
  return TS_OK;
}

ts_status ts_schema_add_tool(ts_schema *s, const int32_t *name, int32_t name_len, const int32_t *key_tokens,
                             const int32_t *key_offsets, int32_t n_keys) {
  if (!s || !name || !key_tokens || !key_offsets) return fail(TS_ERR_ARG, "null argument");
  if (name_len < 1 || n_keys < 1) return fail(TS_ERR_ARG, "a tool needs a name and at least one key");
  ts::ToolDef t;
  t.name.assign(name, name + name_len);
  for (int k = 0; k < n_keys; ++k) {
    if (key_offsets[k + 1] <= key_offsets[k]) return fail(TS_ERR_ARG, "empty key");
    t.keys.emplace_back(key_tokens + key_offsets[k], key_tokens + key_offsets[k + 1]);
  }
  int32_t node = 0;
  const int32_t id = (int32_t)s->tools.size();
  {
    // reject duplicates
    int32_t n = s->walk(t.name);
    if (n >= 0 && s->trie[n].tool_exact >= 0) return fail(TS_ERR_ARG, "duplicate tool name");
  }
  s->trie[0].tools.push_back(id);
  if (s->trie[0].min_tool < 0) s->trie[0].min_tool = id;
  for (int32_t tok : t.name) {
    int32_t nx = s->child(node, tok);
    if (nx < 0) {
      nx = (int32_t)s->trie.size();
      s->trie.emplace_back();
      auto &v = s->trie[node].next;
      v.insert(std::lower_bound(v.begin(), v.end(), std::make_pair(tok, INT32_MIN)), {tok, nx});
    }
    node = nx;
    s->trie[node].tools.push_back(id);
    if (s->trie[node].min_tool < 0) s->trie[node].min_tool = id;
  }
  s->trie[node].tool_exact = id;
  s->tools.push_back(std::move(t));
  return TS_OK;
}

ts_status ts_schema_destroy(ts_schema *s) { delete s; return TS_OK; }

// ---- datastore -----------------------------------------------------------------------------------------
ts_status ts_datastore_create(int32_t n_tools, ts_datastore **out) {
  if (!out || n_tools < 0) return fail(TS_ERR_ARG, "bad argument");
  ts_datastore *d = new ts_datastore();
  d->freq.assign(n_tools, 0);
  *out = d;
  return TS_OK;
}

ts_status ts_datastore_attach_hidden(ts_datastore *d, void *hidden_dev, int32_t capacity, int32_t d_model) {
  if (!d) return fail(TS_ERR_ARG, "null argument");
  if (!hidden_dev) { d->hidden_dev = nullptr; d->hidden_capacity = d->hidden_width = 0; return TS_OK; }
  if (capacity < d->n_entries() || capacity < 1) return fail(TS_ERR_ARG, "capacity %d below the %d entries held", capacity, d->n_entries());
  if (d_model < 8 || d_model % 8) return fail(TS_ERR_ARG, "d_model must be a positive multiple of 8");
  if ((uintptr_t)hidden_dev & 15) return fail(TS_ERR_ARG, "hidden-state matrix must be 16-byte aligned");
  d->hidden_dev = hidden_dev; d->hidden_capacity = capacity; d->hidden_width = d_model;
  return TS_OK;
}

ts_status ts_datastore_add_hidden(ts_datastore *d, ts_model *m, int32_t row, const int32_t *tokens, int32_t n,
                                  int32_t tool_id) {
  if (!d || !m || (!tokens && n > 0) || n < 0) return fail(TS_ERR_ARG, "bad argument");
  if (!d->hidden_dev) return fail(TS_ERR_STATE, "no hidden-state matrix attached (ts_datastore_attach_hidden)");
  if (d->n_entries() >= d->hidden_capacity) return fail(TS_ERR_STATE, "hidden-state matrix is full (%d rows)", d->hidden_capacity);
  if (d->hidden_width != m->c.d_model) return fail(TS_ERR_ARG, "hidden states are %d wide, the model %d", d->hidden_width, m->c.d_model);
  if (!m->have_step || (m->last_flags & TS_FLAG_SKIP_LM_HEAD) || m->last_fused)
    return fail(TS_ERR_STATE, "the last step left no final hidden state (it must run the LM head on the one-kernel-per-stage path)");
  if (row < 0 || row >= m->last_M) return fail(TS_ERR_ARG, "row outside the last step");
  // the first activation plane of the LM head's input IS the hidden state rounded to bf16
  const size_t wbytes = (size_t)m->c.d_model * 2;
  CU_TRY(cudaMemcpyAsync((uint8_t *)d->hidden_dev + (size_t)d->n_entries() * wbytes, m->WS(m->L.h) + (size_t)row * wbytes,
                         wbytes, cudaMemcpyDeviceToDevice, m->st));
  d->tokens.insert(d->tokens.end(), tokens, tokens + n);
  d->offset.push_back((int64_t)d->tokens.size());
  d->tool_of.push_back(tool_id);
  if (tool_id >= 0 && tool_id < (int32_t)d->freq.size()) ++d->freq[tool_id];
  return TS_OK;
}

ts_status ts_datastore_add(ts_datastore *d, const int32_t *tokens, int32_t n, int32_t tool_id) {
  if (!d || (!tokens && n > 0) || n < 0) return fail(TS_ERR_ARG, "bad argument");
  if (d->hidden_dev) return fail(TS_ERR_STATE, "hidden states are attached: add entries with ts_datastore_add_hidden");
  d->tokens.insert(d->tokens.end(), tokens, tokens + n);
  d->offset.push_back((int64_t)d->tokens.size());
  d->tool_of.push_back(tool_id);
  if (tool_id >= 0 && tool_id < (int32_t)d->freq.size()) ++d->freq[tool_id];
  return TS_OK;
}

ts_status ts_datastore_destroy(ts_datastore *d) { delete d; return TS_OK; }

// ---- sessions ------------------------------------------------------------------------------------------
ts_status ts_session_create(ts_model *model, const ts_schema *schema, const ts_datastore *store,
                            const ts_draft_config *cfg, ts_session **out) {
  if (!out || !cfg) return fail(TS_ERR_ARG, "null argument");
  if (cfg->n_cap < 0 || cfg->max_new_tokens < 1) return fail(TS_ERR_ARG, "bad draft configuration");
  ts_session *s = new ts_session();
  s->m = model; s->schema = schema; s->store = store; s->cfg = *cfg;
  s->fsm.s = schema;
  if (model) model->sessions.push_back(s);
  *out = s;
  return TS_OK;
}

ts_status ts_session_set_ranks(ts_session *s, const int32_t *ranks, int32_t n) {
  if (!s || n < 0 || (n > 0 && !ranks)) return fail(TS_ERR_ARG, "bad argument");
  if (n > 0 && !s->store) return fail(TS_ERR_STATE, "session has no datastore");
  for (int i = 0; i < n; ++i)
    if (ranks[i] < 0 || ranks[i] >= s->store->n_entries()) return fail(TS_ERR_ARG, "rank entry %d out of range", ranks[i]);
  s->ranks.assign(ranks, ranks + n);
  s->have_ranks = n > 0;
  return TS_OK;
}

ts_status ts_session_enable_general_sd(ts_session *s, int32_t on) {
  if (!s) return fail(TS_ERR_ARG, "null argument");
  s->general_sd = on != 0;
  return TS_OK;
}

ts_status ts_session_set_successors(ts_session *s, int32_t token, const int32_t *ids) {
  if (!s || !ids || token < 0) return fail(TS_ERR_ARG, "bad argument");
  std::array<int32_t, TS_TOPK> a;
  for (int t = 0; t < TS_TOPK; ++t) a[t] = ids[t];
  s->successors[token] = a;
  return TS_OK;
}

ts_status ts_session_successors(const ts_session *s, int32_t token, int32_t *ids, int32_t *found) {
  if (!s || !ids || !found) return fail(TS_ERR_ARG, "null argument");
  auto it = s->successors.find(token);
  *found = it != s->successors.end();
  if (*found) for (int t = 0; t < TS_TOPK; ++t) ids[t] = it->second[t];
  return TS_OK;
}

ts_status ts_last_topk(ts_model *m, int32_t row, int32_t *ids, float *values) {
  if (!m || !ids) return fail(TS_ERR_ARG, "null argument");
  if (!m->have_step || !(m->last_flags & TS_FLAG_WANT_TOPK)) return fail(TS_ERR_STATE, "the last step was not asked for the Top-K");
  if (row < 0 || row >= m->last_M) return fail(TS_ERR_ARG, "row outside the last step");
  const int32_t *ho = m->h_out() + m->L.o_topk + (size_t)row * TS_TOPK * 2;
  for (int t = 0; t < TS_TOPK; ++t) {
    ids[t] = ho[2 * t];
    if (values) std::memcpy(&values[t], &ho[2 * t + 1], 4);
  }
  return TS_OK;
}

ts_status ts_session_destroy(ts_session *s) {
  if (!s) return TS_OK;
  if (s->m) {
    for (int32_t p : s->pages) s->m->free_pages.push_back(p);
    auto &v = s->m->sessions;
    v.erase(std::remove(v.begin(), v.end(), s), v.end());
  }
  delete s;
  return TS_OK;
}

ts_status ts_prefill(ts_model *m, ts_session *s, const int32_t *tokens, int32_t n) {
  if (!s || !tokens || n < 1) return fail(TS_ERR_ARG, "bad argument");
  if (s->m != m) return fail(TS_ERR_ARG, "session belongs to another model");
  if (s->cache_len >= 0) return fail(TS_ERR_STATE, "session already has a context");
  if (s->schema)
    for (int i = 0; i < n; ++i) s->fsm.step(tokens[i]);
  s->prompt.assign(tokens, tokens + n);
  s->cache_len = 0;
  if (m) {
    std::vector<std::vector<int32_t>> rows(1);
    for (int i = 0; i < n - 1; i += m->c.k_max) {
      const int k = std::min(m->c.k_max, n - 1 - i);
      rows[0].assign(tokens + i, tokens + i + k);
      ts_status st = stage_and_run(m, &s, 1, rows, TS_FLAG_SKIP_LM_HEAD);
      if (st) { s->cache_len = -1; return st; }
      s->cache_len += k;
    }
  } else {
    s->cache_len = n - 1;
  }
  s->pending = tokens[n - 1];
  return TS_OK;
}

ts_status ts_draft(ts_session *s, int32_t max_draft, int32_t *out_tokens, int32_t *out_n, int32_t *out_source) {
  if (!s || !out_n || !out_source || (max_draft > 0 && !out_tokens)) return fail(TS_ERR_ARG, "null argument");
  *out_n = 0; *out_source = 0;
  if (max_draft <= 0 || s->finished) return TS_OK;
  std::vector<int32_t> d;
  if (s->store) {
    const int n = std::min(s->cfg.n_cap, max_draft);
    ts::suffix_match(s->y, *s->store, s->have_ranks ? &s->ranks : nullptr, n, &d);
    if (!d.empty()) *out_source = 2;
  }
  if (d.empty() && s->schema) {
    int guess = -1;
    if (s->fsm.kind == ts::Q_T && s->fsm.stage != ts::ST_MID) guess = guess_tool(s);
    s->fsm.draft(guess, &d);
    if ((int)d.size() > max_draft) d.resize(max_draft);
    if (!d.empty()) *out_source = 1;
  }
  std::memcpy(out_tokens, d.data(), d.size() * sizeof(int32_t));
  *out_n = (int32_t)d.size();
  return TS_OK;
}

ts_status ts_draft_tree(ts_session *s, int32_t max_nodes, int32_t *out_tokens, int32_t *out_parents, int32_t *out_n,
                        int32_t *out_source) {
  if (!s || !out_n || !out_source || (max_nodes > 1 && (!out_tokens || !out_parents)))
    return fail(TS_ERR_ARG, "null argument");
  *out_n = 0; *out_source = 0;
  if (max_nodes > TS_K_MAX) return fail(TS_ERR_K_TOO_LARGE, "a draft tree holds at most %d nodes", TS_K_MAX);
  const int max_draft = max_nodes - 1;
  if (max_draft <= 0 || s->finished) return TS_OK;
  std::vector<std::vector<int32_t>> cands;
  int source = 0;
  if (s->store) {
    const int32_t caps[4] = {s->cfg.n_cap, 16, 8, 8};   // Appendix B.2: continuation lengths in candidate order
    ts::suffix_matches(s->y, *s->store, s->have_ranks ? &s->ranks : nullptr, caps, 4, max_draft, &cands);
    if (!cands.empty()) source = 2;
  }
  if (cands.empty() && s->schema) {
    std::vector<int32_t> d;
    if (s->fsm.kind == ts::Q_T && s->fsm.stage != ts::ST_MID) {
      // one chain per tool whose name extends what was emitted so far: the guessed tool first, then ascending ids
      const int guess = guess_tool(s);
      if (guess >= 0) {
        const ts::TrieNode &node = s->schema->trie[s->fsm.stage == ts::ST_NAME ? s->fsm.node : 0];
        std::vector<int32_t> order{guess};
        for (int32_t t : node.tools)
          if (t != guess && (int)order.size() < kMaxToolCandidates) order.push_back(t);
        for (int32_t t : order) {
          s->fsm.draft(t, &d);
          if ((int)d.size() > max_draft) d.resize(max_draft);
          cands.push_back(d);
        }
      } else {
        s->fsm.draft(-1, &d);
        if ((int)d.size() > max_draft) d.resize(max_draft);
        if (!d.empty()) cands.push_back(d);
      }
    } else {
      s->fsm.draft(-1, &d);
      if ((int)d.size() > max_draft) d.resize(max_draft);
      if (!d.empty()) cands.push_back(d);
    }
    if (!cands.empty()) source = 1;
  }
  std::vector<int32_t> toks, par;
  if (cands.empty() && s->general_sd) {
    // open-ended states: a suffix match inside the context itself, else the static tree over recycled successors
    std::vector<int32_t> ctx(s->prompt);
    ctx.insert(ctx.end(), s->y.begin(), s->y.end());
    std::vector<int32_t> d;
    ts::context_match(ctx, std::min(s->cfg.n_cap, max_draft), &d);
    if (!d.empty()) {
      cands.push_back(d);
      source = 3;
    } else {
      ts::recycled_tree(s->pending, s->successors, max_nodes, &toks, &par);
      if (!toks.empty()) source = 4;
    }
  }
  if (source != 4) ts::pack_candidates(cands, max_nodes, &toks, &par);
  std::memcpy(out_tokens, toks.data(), toks.size() * sizeof(int32_t));
  std::memcpy(out_parents, par.data(), par.size() * sizeof(int32_t));
  *out_n = (int32_t)toks.size();
  *out_source = toks.empty() ? 0 : source;
  return TS_OK;
}

namespace {
// ts_verify and ts_verify_tree: draft_parents = nullptr for chains
ts_status verify_impl(ts_model *m, ts_session *const *ss, int32_t B, const int32_t *draft_tokens,
                      const int32_t *draft_parents, const int32_t *draft_offsets, uint32_t flags,
                      ts_verify_result *out, int32_t *path_out, const float *uniforms = nullptr,
                      float temperature = 0.f) {
  if (!m || !ss || !draft_offsets || !out) return fail(TS_ERR_ARG, "null argument");
  if (B < 1 || B > m->c.max_batch) return fail(TS_ERR_ARG, "batch %d outside [1, %d]", B, m->c.max_batch);
  std::vector<std::vector<int32_t>> rows(B), parents(B);
  for (int i = 0; i < B; ++i) {
    ts_session *s = ss[i];
    if (!s || s->m != m) return fail(TS_ERR_ARG, "session %d is null or belongs to another model", i);
    if (s->cache_len < 0 || s->pending < 0) return fail(TS_ERR_STATE, "session %d has no context (call ts_prefill)", i);
    if (s->finished) return fail(TS_ERR_STATE, "session %d is finished", i);
    for (int j = 0; j < i; ++j)
      if (ss[j] == s) return fail(TS_ERR_ARG, "session listed twice");
    const int n = draft_offsets[i + 1] - draft_offsets[i];
    if (n < 0) return fail(TS_ERR_ARG, "draft_offsets not ascending");
    if (n > 0 && !draft_tokens) return fail(TS_ERR_ARG, "null draft_tokens");
    rows[i].reserve(n + 1);
    rows[i].push_back(s->pending);
    for (int j = 0; j < n; ++j) rows[i].push_back(draft_tokens[draft_offsets[i] + j]);
    if (draft_parents) {
      parents[i].push_back(-1);
      for (int j = 0; j < n; ++j) parents[i].push_back(draft_parents[draft_offsets[i] + j]);
    }
  }
  for (int i = 0; i < B; ++i) ss[i]->last_chunk.clear();   // this step overwrites the rows of the previous one
  ts_status st = stage_and_run(m, ss, B, rows, flags, draft_parents ? &parents : nullptr, uniforms, temperature);
  if (st) return st;
  const Layout &L = m->L;
  const int32_t *ho = m->h_out();
  int row = 0;
  for (int i = 0; i < B; ++i) {
    ts_verify_result &r = out[i];
    std::memset(&r, 0, sizeof r);
    r.k = (int32_t)rows[i].size();
    r.first_row = row;
    ss[i]->last_chunk = rows[i];
    if (flags & TS_FLAG_SKIP_LM_HEAD) ss[i]->last_chunk.clear();   // no acceptance ran: nothing to commit
    if (!(flags & TS_FLAG_SKIP_LM_HEAD)) {
      r.accept_len = ho[L.o_accept + i];
      r.n_emitted = r.accept_len + 1;
      for (int j = 0; j < r.n_emitted; ++j) r.emitted[j] = ho[L.o_emitted + i * m->c.k_max + j];
      for (int j = 0; j < r.k; ++j) r.argmax[j] = ho[L.o_argmax + row + j];
      if (path_out) {
        for (int j = 0; j < TS_K_MAX; ++j)
          path_out[i * TS_K_MAX + j] = j <= r.accept_len ? ho[L.o_path + i * m->c.k_max + j] : -1;
      }
      if ((flags & TS_FLAG_WANT_TOPK) && ss[i]->general_sd) {
        // successor table: what the model ranked highest after each token it was fed in this step (all rows)
        for (int j = 0; j < r.k; ++j) {
          std::array<int32_t, TS_TOPK> ids;
          for (int t = 0; t < TS_TOPK; ++t) ids[t] = ho[L.o_topk + ((row + j) * TS_TOPK + t) * 2];
          ss[i]->successors[rows[i][j]] = ids;
        }
      }
      if (draft_parents) {
        // the cache now holds the accepted path's rows at consecutive positions: record what sits there, so that
        // a later forced commit is checked against the right ids
        std::vector<int32_t> kept;
        for (int j = 0; j <= r.accept_len; ++j) kept.push_back(rows[i][ho[L.o_path + i * m->c.k_max + j]]);
        ss[i]->last_chunk = kept;
      }
    }
    row += r.k;
  }
  return TS_OK;
}
}  // namespace

ts_status ts_verify(ts_model *m, ts_session *const *ss, int32_t B, const int32_t *draft_tokens,
                    const int32_t *draft_offsets, uint32_t flags, ts_verify_result *out) {
  return verify_impl(m, ss, B, draft_tokens, nullptr, draft_offsets, flags, out, nullptr);
}

ts_status ts_verify_sampled(ts_model *m, ts_session *const *ss, int32_t B, const int32_t *draft_tokens,
                            const int32_t *draft_offsets, float temperature, const float *uniforms, uint32_t flags,
                            ts_verify_result *out) {
  if (!uniforms) return fail(TS_ERR_ARG, "null uniforms");
  if (!(temperature > 0.f) || !(temperature < 1e4f)) return fail(TS_ERR_ARG, "temperature must be in (0, 1e4)");
  if (flags & TS_FLAG_SKIP_LM_HEAD) return fail(TS_ERR_ARG, "sampling acceptance needs the logits");
  if (draft_offsets && B >= 1 && B <= 4096) {
    const int M = draft_offsets[B] - draft_offsets[0] + B;
    for (int r = 0; r < M; ++r)
      if (!(uniforms[r] >= 0.f && uniforms[r] < 1.f)) return fail(TS_ERR_ARG, "uniform %d outside [0, 1)", r);
  }
  return verify_impl(m, ss, B, draft_tokens, nullptr, draft_offsets, flags, out, nullptr, uniforms, temperature);
}

ts_status ts_verify_tree_sampled(ts_model *m, ts_session *const *ss, int32_t B, const int32_t *draft_tokens,
                                 const int32_t *draft_parents, const int32_t *draft_offsets, float temperature,
                                 const float *uniforms, uint32_t flags, ts_verify_result *out, int32_t *path_out) {
  if (!uniforms) return fail(TS_ERR_ARG, "null uniforms");
  if (!(temperature > 0.f) || !(temperature < 1e4f)) return fail(TS_ERR_ARG, "temperature must be in (0, 1e4)");
  if (flags & TS_FLAG_SKIP_LM_HEAD) return fail(TS_ERR_ARG, "sampling acceptance needs the logits");
  if (!draft_parents && draft_offsets && B >= 1 && draft_offsets[B] > draft_offsets[0])
    return fail(TS_ERR_ARG, "null draft_parents");
  if (draft_offsets && B >= 1 && B <= 4096) {
    const int M = draft_offsets[B] - draft_offsets[0] + B;
    for (int r = 0; r < M; ++r)
      if (!(uniforms[r] >= 0.f && uniforms[r] < 1.f)) return fail(TS_ERR_ARG, "uniform %d outside [0, 1)", r);
  }
  static const int32_t none = 0;
  return verify_impl(m, ss, B, draft_tokens, draft_parents ? draft_parents : &none, draft_offsets, flags, out, path_out,
                     uniforms, temperature);
}

ts_status ts_verify_tree(ts_model *m, ts_session *const *ss, int32_t B, const int32_t *draft_tokens,
                         const int32_t *draft_parents, const int32_t *draft_offsets, uint32_t flags,
                         ts_verify_result *out, int32_t *path_out) {
  if (!draft_parents && draft_offsets && B >= 1 && draft_offsets[B] > draft_offsets[0])
    return fail(TS_ERR_ARG, "null draft_parents");
  if (flags & TS_FLAG_SKIP_LM_HEAD) return fail(TS_ERR_ARG, "a draft tree cannot be run without acceptance");
  static const int32_t none = 0;
  return verify_impl(m, ss, B, draft_tokens, draft_parents ? draft_parents : &none, draft_offsets, flags, out, path_out);
}

ts_status ts_verify_replay(ts_model *m) {
  if (!m) return fail(TS_ERR_ARG, "null argument");
  if (!m->have_step) return fail(TS_ERR_STATE, "no step has been staged yet");
  return run_step(m);
}

ts_status ts_profile_step(ts_model *m, float *ms_by_class, int32_t *launches_by_class, int32_t n_classes) {
  if (!m || !ms_by_class || !launches_by_class || n_classes < 6) return fail(TS_ERR_ARG, "bad argument");
  if (!m->have_step) return fail(TS_ERR_STATE, "no step has been staged yet");
  for (int i = 0; i < n_classes; ++i) { ms_by_class[i] = 0.f; launches_by_class[i] = 0; }
  if (m->last_fused) {
    // one kernel: class 6 is its event time; the phase classes come from the device-side phase-end stamps
    const Layout &L = m->L;
    const int n_ph = (m->last_flags & TS_FLAG_SKIP_LM_HEAD) ? 6 * m->c.n_layers + 1 : 6 * m->c.n_layers + 2;
    CU_TRY(cudaMemsetAsync(m->WS(L.phase_t), 0, (size_t)3 * L.n_phases * 8, m->st));
    cudaEvent_t e0, e1;
    CU_TRY(cudaEventCreate(&e0));
    CU_TRY(cudaEventCreate(&e1));
    CU_TRY(cudaEventRecord(e0, m->st));
    m->profiling = true;
    ts_status st = run_step(m);
    m->profiling = false;
    for (cudaEvent_t ev : m->prof_ev) cudaEventDestroy(ev);
    m->prof_ev.clear();
    m->prof_cls.clear();
    cudaEventRecord(e1, m->st);
    std::vector<unsigned long long> t(L.n_phases);
    cudaError_t e = cudaMemcpyAsync(t.data(), m->WS(L.phase_t), (size_t)L.n_phases * 8, cudaMemcpyDeviceToHost, m->st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(m->st);
    float total = 0.f;
    if (e == cudaSuccess) cudaEventElapsedTime(&total, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (st) return st;
    if (e != cudaSuccess) return fail(TS_ERR_CUDA, "profile step: %s", cudaGetErrorString(e));
    for (int p = 1; p < n_ph; ++p) {
      if (t[p] == 0 || t[p - 1] == 0) continue;
      const float ms = (float)((double)(t[p] - t[p - 1]) * 1e-6);
      const int r = (p - 1) % 6;   // 0 qkv, 1 attention, 2 merge, 3 o, 4 gate-up, 5 down; the last phase is the LM head
      const int cls = (p == 6 * m->c.n_layers + 1) ? 0 : (r == 1 ? 1 : (r == 2 ? 2 : 0));
      ms_by_class[cls] += ms;
      ++launches_by_class[cls];
    }
    if (n_classes > 6) { ms_by_class[6] = total; launches_by_class[6] = 1; }
    return TS_OK;
  }
  cudaEvent_t start;
  CU_TRY(cudaEventCreate(&start));
  CU_TRY(cudaEventRecord(start, m->st));
  m->profiling = true;
  ts_status st = run_step(m);
  m->profiling = false;
  cudaError_t e = cudaStreamSynchronize(m->st);
  cudaEvent_t prev = start;
  for (size_t i = 0; i < m->prof_ev.size(); ++i) {
    float ms = 0.f;
    if (e == cudaSuccess && cudaEventElapsedTime(&ms, prev, m->prof_ev[i]) == cudaSuccess) {
      ms_by_class[m->prof_cls[i]] += ms;
      ++launches_by_class[m->prof_cls[i]];
    }
    prev = m->prof_ev[i];
  }
  cudaEventDestroy(start);
  for (cudaEvent_t ev : m->prof_ev) cudaEventDestroy(ev);
  m->prof_ev.clear();
  m->prof_cls.clear();
  if (st) return st;
  if (e != cudaSuccess) return fail(TS_ERR_CUDA, "profile step: %s", cudaGetErrorString(e));
  return TS_OK;
}

ts_status ts_commit_forced(ts_session *s, const int32_t *emitted, int32_t n) {
  if (!s || !emitted || n < 1) return fail(TS_ERR_ARG, "bad argument");
  if (s->finished) return fail(TS_ERR_STATE, "session is finished");
  if (s->cache_len < 0) return fail(TS_ERR_STATE, "session has no context");
  if (s->m) {
    // The cache keeps the pending token and the first n - 1 emitted ids: the K/V rows at those positions were
    // written by the last verification (after a tree step: the accepted path, moved to consecutive slots), so the
    // ids must be the ones that step was fed there.  One commit per verification.
    if (s->last_chunk.empty())
      return fail(TS_ERR_STATE, "nothing to commit: no verification since the last commit (or since the context was set)");
    if (n > (int)s->last_chunk.size())
      return fail(TS_ERR_ARG, "%d ids to commit, but the last verification holds only %zu rows in the cache", n,
                  s->last_chunk.size());
    for (int j = 0; j + 1 < n; ++j)
      if (emitted[j] != s->last_chunk[j + 1])
        return fail(TS_ERR_ARG, "emitted id %d (%d) is not the id verified at that row (%d)", j, emitted[j],
                    s->last_chunk[j + 1]);
    s->last_chunk.clear();
  }
  const int used = commit_ids(s, emitted, n);
  s->cache_len += used;
  s->pending = emitted[used - 1];
  return TS_OK;
}

ts_status ts_commit(ts_session *s, const ts_verify_result *r) {
  if (!s || !r) return fail(TS_ERR_ARG, "null argument");
  if (r->n_emitted < 1 || r->n_emitted > TS_K_MAX) return fail(TS_ERR_ARG, "result carries no emitted ids");
  return ts_commit_forced(s, r->emitted, r->n_emitted);
}

ts_status ts_session_state(const ts_session *s, ts_session_info *out) {
  if (!s || !out) return fail(TS_ERR_ARG, "null argument");
  out->cache_len = s->cache_len; out->pending = s->pending; out->n_output = (int32_t)s->y.size();
  out->finished = s->finished ? 1 : 0;
  out->fsm_kind = s->fsm.kind; out->fsm_tool = s->fsm.tool; out->fsm_key = s->fsm.key;
  out->n_pages = (int32_t)s->pages.size();
  return TS_OK;
}

ts_status ts_session_output(const ts_session *s, int32_t *out, int32_t cap, int32_t *n) {
  if (!s || !n || (cap > 0 && !out)) return fail(TS_ERR_ARG, "null argument");
  *n = (int32_t)s->y.size();
  std::memcpy(out, s->y.data(), sizeof(int32_t) * std::min<size_t>(cap, s->y.size()));
  return TS_OK;
}

// ---- test / benchmark support -------------------------------------------------------------------------
static ts_status kv_transfer(ts_model *m, ts_session *s, int layer, void *k, void *v, int n_tokens, bool to_device) {
  if (!m || !s || (n_tokens > 0 && (!k || !v))) return fail(TS_ERR_ARG, "null argument");
  if (s->m != m) return fail(TS_ERR_ARG, "session belongs to another model");
  if (layer < 0 || layer >= m->c.n_layers || n_tokens < 0) return fail(TS_ERR_ARG, "bad layer / length");
  if (to_device) {
    ts_status st = ensure_pages(s, n_tokens);
    if (st) return st;
  } else if ((n_tokens + TS_PAGE_SIZE - 1) / TS_PAGE_SIZE > (int)s->pages.size()) {
    return fail(TS_ERR_ARG, "session holds fewer than %d tokens", n_tokens);
  }
  const int Hkv = m->c.n_kv_heads, hd = m->c.head_dim;
  const size_t page_elems = (size_t)Hkv * TS_PAGE_SIZE * hd;
  const int n_pages = (n_tokens + TS_PAGE_SIZE - 1) / TS_PAGE_SIZE;
  // one staging image of all pages, so that the copies of a layer are issued back to back and awaited once
  std::vector<__half> stage((size_t)n_pages * page_elems);
  for (int which = 0; which < 2; ++which) {
    float *host = (float *)(which ? v : k);
    __half *pool = which ? m->v_pages(layer) : m->k_pages(layer);
    if (to_device) {
      std::fill(stage.begin(), stage.end(), __float2half(0.f));
      for (int t = 0; t < n_tokens; ++t) {
        __half *pg = stage.data() + (size_t)(t / TS_PAGE_SIZE) * page_elems;
        for (int hh = 0; hh < Hkv; ++hh) {
          const float *src = host + ((size_t)t * Hkv + hh) * hd;
          __half *dst = pg + ((size_t)hh * TS_PAGE_SIZE + (t % TS_PAGE_SIZE)) * hd;
          for (int e = 0; e < hd; ++e) dst[e] = __float2half_rn(std::min(std::max(src[e], -65504.f), 65504.f));
        }
      }
      for (int p = 0; p < n_pages; ++p)
        CU_TRY(cudaMemcpyAsync(pool + (size_t)s->pages[p] * page_elems, stage.data() + (size_t)p * page_elems,
                               page_elems * 2, cudaMemcpyHostToDevice, m->st));
      CU_TRY(cudaStreamSynchronize(m->st));
    } else {
      for (int p = 0; p < n_pages; ++p)
        CU_TRY(cudaMemcpyAsync(stage.data() + (size_t)p * page_elems, pool + (size_t)s->pages[p] * page_elems,
                               page_elems * 2, cudaMemcpyDeviceToHost, m->st));
      CU_TRY(cudaStreamSynchronize(m->st));
      for (int t = 0; t < n_tokens; ++t) {
        const __half *pg = stage.data() + (size_t)(t / TS_PAGE_SIZE) * page_elems;
        for (int hh = 0; hh < Hkv; ++hh) {
          float *dst = host + ((size_t)t * Hkv + hh) * hd;
          const __half *src = pg + ((size_t)hh * TS_PAGE_SIZE + (t % TS_PAGE_SIZE)) * hd;
          for (int e = 0; e < hd; ++e) dst[e] = __half2float(src[e]);
        }
      }
    }
  }
  return TS_OK;
}

ts_status ts_debug_import_kv(ts_model *m, ts_session *s, int32_t layer, const float *k, const float *v, int32_t n) {
  return kv_transfer(m, s, layer, (void *)k, (void *)v, n, true);
}
ts_status ts_debug_export_kv(ts_model *m, ts_session *s, int32_t layer, float *k, float *v, int32_t n) {
  return kv_transfer(m, s, layer, k, v, n, false);
}

ts_status ts_debug_set_cache(ts_session *s, int32_t cache_len, int32_t pending) {
  if (!s || cache_len < 0 || pending < 0) return fail(TS_ERR_ARG, "bad argument");
  if (s->m) {
    if (pending >= s->m->c.vocab) return fail(TS_ERR_TOKEN_RANGE, "pending id out of range");
    ts_status st = ensure_pages(s, cache_len);
    if (st) return st;
  }
  s->cache_len = cache_len;
  s->pending = pending;
  s->last_chunk.clear();   // whatever was verified before does not describe this context
  return TS_OK;
}

ts_status ts_debug_restart(ts_session *s, int32_t cache_len, int32_t pending) {
  ts_status st = ts_debug_set_cache(s, cache_len, pending);
  if (st) return st;
  s->y.clear();
  s->last_chunk.clear();
  s->successors.clear();
  s->finished = false;
  s->fsm.reset();
  return TS_OK;
}

ts_status ts_read_logits(ts_model *m, int32_t row0, int32_t n_rows, float *host_out) {
  if (!m || !host_out) return fail(TS_ERR_ARG, "null argument");
  if (!m->have_step || (m->last_flags & TS_FLAG_SKIP_LM_HEAD)) return fail(TS_ERR_STATE, "last step produced no logits");
  if (row0 < 0 || n_rows < 0 || row0 + n_rows > m->last_M) return fail(TS_ERR_ARG, "rows outside the last step");
  const size_t V = m->c.vocab;
  CU_TRY(cudaMemcpyAsync(host_out, (float *)m->WS(m->L.logits) + (size_t)row0 * V, (size_t)n_rows * V * 4,
                         cudaMemcpyDeviceToHost, m->st));
  CU_TRY(cudaStreamSynchronize(m->st));
  return TS_OK;
}

ts_status ts_last_hidden(ts_model *m, int32_t row, float *host_out) {
  if (!m || !host_out) return fail(TS_ERR_ARG, "null argument");
  if (!m->have_step || (m->last_flags & TS_FLAG_SKIP_LM_HEAD) || m->last_fused)
    return fail(TS_ERR_STATE, "the last step left no final hidden state (it must run the LM head on the one-kernel-per-stage path)");
  if (row < 0 || row >= m->last_M) return fail(TS_ERR_ARG, "row outside the last step");
  const size_t d = m->c.d_model, R = m->L.rows_alloc;
  std::vector<__nv_bfloat16> tmp(2 * d);
  const __nv_bfloat16 *h = (const __nv_bfloat16 *)m->WS(m->L.h);
  CU_TRY(cudaMemcpyAsync(tmp.data(), h + (size_t)row * d, d * 2, cudaMemcpyDeviceToHost, m->st));
  if (m->planes == 2)
    CU_TRY(cudaMemcpyAsync(tmp.data() + d, h + (R + (size_t)row) * d, d * 2, cudaMemcpyDeviceToHost, m->st));
  CU_TRY(cudaStreamSynchronize(m->st));
  for (size_t i = 0; i < d; ++i)
    host_out[i] = __bfloat162float(tmp[i]) + (m->planes == 2 ? __bfloat162float(tmp[d + i]) : 0.f);
  return TS_OK;
}

ts_status ts_topk_cosine(ts_model *m, const void *hidden_dev, int32_t n_entries, const float *query_dev, int32_t row,
                         int32_t K, float *scores_dev, int32_t *out_index, float *out_score) {
  if (!m || !hidden_dev || !scores_dev || !out_index) return fail(TS_ERR_ARG, "null argument");
  if (n_entries < 1 || K < 1 || K > 64 || K > n_entries) return fail(TS_ERR_ARG, "K must be in [1, min(64, n_entries)]");
  if (m->c.d_model % 8 || m->c.d_model > 16384) return fail(TS_ERR_ARG, "d_model must be a multiple of 8, at most 16384");
  const __nv_bfloat16 *planes = nullptr;
  if (!query_dev) {
    if (!m->have_step || (m->last_flags & TS_FLAG_SKIP_LM_HEAD) || m->last_fused)
      return fail(TS_ERR_STATE, "no final hidden state: pass a query, or run a step with the LM head on the one-kernel-per-stage path first");
    if (row < 0 || row >= m->last_M) return fail(TS_ERR_ARG, "row outside the last step");
    planes = (const __nv_bfloat16 *)m->WS(m->L.h) + (size_t)row * m->c.d_model;
  }
  CU_TRY(ts::launch_topk_cosine((const __nv_bfloat16 *)hidden_dev, n_entries, m->c.d_model, query_dev, planes,
                                (int)(m->L.rows_alloc * m->c.d_model), m->planes, K, scores_dev, m->st));
  std::vector<float> res(2 * (size_t)K);
  CU_TRY(cudaMemcpyAsync(res.data(), scores_dev + n_entries, res.size() * 4, cudaMemcpyDeviceToHost, m->st));
  CU_TRY(cudaStreamSynchronize(m->st));
  for (int j = 0; j < K; ++j) {
    int32_t idx;
    std::memcpy(&idx, &res[2 * j], 4);
    out_index[j] = idx;
    if (out_score) out_score[j] = res[2 * j + 1];
  }
  return TS_OK;
}

ts_status ts_session_retrieve(ts_model *m, ts_session *s, int32_t row, int32_t K, float *scores_dev, int32_t *out_index,
                              float *out_score, int32_t *out_k) {
  if (!m || !s || !scores_dev || !out_index || !out_k) return fail(TS_ERR_ARG, "null argument");
  if (s->m != m) return fail(TS_ERR_ARG, "session belongs to another model");
  const ts_datastore *d = s->store;
  if (!d) return fail(TS_ERR_STATE, "session has no datastore");
  if (!d->hidden_dev) return fail(TS_ERR_STATE, "the datastore has no hidden states attached");
  if (d->n_entries() < 1) return fail(TS_ERR_STATE, "the datastore is empty");
  if (d->hidden_width != m->c.d_model) return fail(TS_ERR_ARG, "hidden states are %d wide, the model %d", d->hidden_width, m->c.d_model);
  if (K < 1) return fail(TS_ERR_ARG, "K must be positive");
  const int32_t k = std::min(std::min(K, d->n_entries()), 64);
  ts_status st = ts_topk_cosine(m, d->hidden_dev, d->n_entries(), nullptr, row, k, scores_dev, out_index, out_score);
  if (st) return st;
  *out_k = k;
  return ts_session_set_ranks(s, out_index, k);
}

ts_status ts_debug_read_buffer(ts_model *m, int32_t which, void *host_out, uint64_t bytes) {
  if (!m || !host_out) return fail(TS_ERR_ARG, "null argument");
  const Layout &L = m->L;
  const uint64_t R = L.rows_alloc, P = m->planes, d = m->c.d_model, Nq = (uint64_t)m->c.n_q_heads * m->c.head_dim;
  uint64_t off = 0, cap = 0;
  switch (which) {
    case 0: off = L.x; cap = R * d * 4; break;
    case 1: off = L.h; cap = P * R * d * 2; break;
    case 2: off = L.q; cap = R * Nq * 2; break;
    case 3: off = L.attn; cap = P * R * Nq * 2; break;
    case 4: off = L.act; cap = P * R * (uint64_t)m->c.d_ffn * 2; break;
    default: return fail(TS_ERR_ARG, "unknown buffer %d", which);
  }
  if (bytes > cap) return fail(TS_ERR_ARG, "buffer %d holds %llu bytes", which, (unsigned long long)cap);
  CU_TRY(cudaMemcpyAsync(host_out, m->WS(off), bytes, cudaMemcpyDeviceToHost, m->st));
  CU_TRY(cudaStreamSynchronize(m->st));
  return TS_OK;
}

ts_status ts_debug_phase_clocks(ts_model *m, uint64_t *out, int32_t cap, int32_t *n_phases) {
  if (!m || !n_phases || (cap > 0 && !out)) return fail(TS_ERR_ARG, "null argument");
  *n_phases = m->L.n_phases;
  const size_t n = std::min<size_t>((size_t)std::max(cap, 0), (size_t)3 * m->L.n_phases);
  CU_TRY(cudaMemcpyAsync(out, m->WS(m->L.phase_t), n * 8, cudaMemcpyDeviceToHost, m->st));
  CU_TRY(cudaStreamSynchronize(m->st));
  return TS_OK;
}

ts_status ts_debug_schedule(int32_t n_tiles, int32_t n_kblocks, int32_t n_ctas, int32_t cta, int32_t cap,
                            int32_t *segments, int32_t *n_segments) {
  if (n_tiles < 1 || n_kblocks < 1 || n_ctas < 1 || cta < 0 || cta >= n_ctas || !n_segments || (cap > 0 && !segments))
    return fail(TS_ERR_ARG, "bad argument");
  ts::SegmentIter it((uint32_t)cta, n_tiles, n_kblocks, (uint32_t)n_ctas);
  ts::Segment sg;
  int n = 0;
  while (it.next(&sg)) {
    if (n < cap) {
      const ts::TileCover tc = ts::tile_cover(sg.tile, n_tiles, n_kblocks, (uint32_t)n_ctas);
      int32_t *o = segments + 6 * n;
      o[0] = sg.tile; o[1] = sg.kb0; o[2] = sg.kb1;
      o[3] = ts::slab_slot_of(cta, sg.tile, n_tiles, n_kblocks, (uint32_t)n_ctas);
      o[4] = tc.c_first; o[5] = tc.n_seg;
    }
    ++n;
  }
  *n_segments = n;
  return TS_OK;
}

ts_status ts_debug_timeline(ts_model *m, uint64_t *stamps, int32_t *classes, int32_t cap, int32_t *n_launches) {
  if (!m || !n_launches || (cap > 0 && (!stamps || !classes))) return fail(TS_ERR_ARG, "null argument");
  if (!m->have_step) return fail(TS_ERR_STATE, "no step has been staged yet");
  if (m->last_fused) return fail(TS_ERR_UNIMPLEMENTED, "the persistent kernel has its own clocks (ts_debug_phase_clocks)");
  const Layout &L = m->L;
  std::vector<unsigned long long> init((size_t)L.max_stamps * 4);
  for (int i = 0; i < L.max_stamps; ++i) { init[4 * i] = init[4 * i + 1] = ~0ull; init[4 * i + 2] = init[4 * i + 3] = 0ull; }
  CU_TRY(cudaMemcpyAsync(m->WS(L.stamps), init.data(), init.size() * 8, cudaMemcpyHostToDevice, m->st));
  CU_TRY(cudaStreamSynchronize(m->st));
  m->timeline = true; m->stamp_idx = 0; m->stamp_cls.clear();
  ts_status st = run_step(m);
  m->timeline = false;
  if (st) return st;
  CU_TRY(cudaMemcpyAsync(init.data(), m->WS(L.stamps), init.size() * 8, cudaMemcpyDeviceToHost, m->st));
  CU_TRY(cudaStreamSynchronize(m->st));
  const int n = std::min<int>((int)m->stamp_cls.size(), L.max_stamps);
  *n_launches = n;
  for (int i = 0; i < n && i < cap; ++i) {
    classes[i] = m->stamp_cls[i];
    for (int j = 0; j < 4; ++j) stamps[4 * i + j] = init[4 * (size_t)i + j];
  }
  return TS_OK;
}

ts_status ts_debug_inject_device_error(ts_model *m, int32_t code) {
  if (!m || code <= 0) return fail(TS_ERR_ARG, "bad argument");
  m->inject_err = code;
  return TS_OK;
}

ts_status ts_model_counters(const ts_model *m, int64_t *launches, int64_t *h2d, int64_t *d2h) {
  if (!m) return fail(TS_ERR_ARG, "null argument");
  if (launches) *launches = m->launches;
  if (h2d) *h2d = m->h2d;
  if (d2h) *d2h = m->d2h;
  return TS_OK;
}

}  // extern "C"
