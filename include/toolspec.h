/*
 * toolspec.h — C ABI of the B200-native verify path of ToolSpec (schema-aware, retrieval-augmented
 * speculative decoding for tool calling).
 *
 * The calls follow the loop body of the paper's Algorithm 1:
 *     draft (SuffixMatch, else SchemaAwareDraft)  ->  ts_draft      (host C++)
 *     Verification (one forward over the packed chunk) + SelectLongestAcceptedPrefix
 *                                                  ->  ts_verify     (sm_100a CUDA kernels)
 *     y <- y (+) accepted span;  q <- delta(q, span) ->  ts_commit     (host C++)
 * One candidate chain per step (causal mask inside the chunk) and greedy acceptance: the accepted
 * length is the longest draft prefix equal to the per-position argmax of the target model, and one
 * bonus token (the argmax after the last accepted draft) is always emitted, so an empty draft is
 * exactly one vanilla decoding step.
 *
 * Conventions
 *   - Every function returns a ts_status (0 = TS_OK, negative = error).  No exception crosses the
 *     boundary.  ts_last_error() returns a thread-local description of the last failure.
 *   - Handles (ts_model, ts_schema, ts_datastore, ts_session) are opaque, owned by the library and
 *     released with the matching *_destroy.  A handle is not thread-safe.
 *   - The library allocates NO device memory.  The caller allocates the four buffers whose sizes
 *     ts_query_buffer_sizes() reports (three in device memory, one in pinned host memory) and
 *     keeps them alive until ts_model_destroy().  All device work is enqueued on the cudaStream_t
 *     given to ts_init_model (passed as void*).
 *   - "host" / "device" below says where a pointer must point.  Token ids are int32.
 *   - Without a usable CUDA device every call that needs one fails with TS_ERR_CUDA; there is no
 *     CPU fallback for the verify path.
 */
#ifndef TOOLSPEC_H_
#define TOOLSPEC_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TS_K_MAX 64          /* most rows (pending token + drafts) one sequence may verify per step */
#define TS_PAGE_SIZE 16      /* tokens per KV page */

typedef int32_t ts_status;
enum {
  TS_OK = 0,
  TS_ERR_ARG = -1,            /* null pointer, size out of range, inconsistent configuration */
  TS_ERR_STATE = -2,          /* call not valid in the handle's current state */
  TS_ERR_OOM_PAGES = -3,      /* KV page pool exhausted */
  TS_ERR_K_TOO_LARGE = -4,    /* chunk longer than k_max, or more rows than max_rows */
  TS_ERR_TOKEN_RANGE = -5,    /* token id outside [0, vocab) */
  TS_ERR_DEVICE_TIMEOUT = -6, /* a bounded device-side wait expired; the context stays usable */
  TS_ERR_CUDA = -7,           /* CUDA runtime/driver error, or no device */
  TS_ERR_UNIMPLEMENTED = -8,
  TS_ERR_DEVICE_BOUNDS = -9   /* debug build of the library only (compiled with TS_DEBUG_BOUNDS): a kernel found an index
                                 from the step's inputs outside its range and skipped the access; the context stays
                                 usable */
};

typedef struct ts_model ts_model;
typedef struct ts_schema ts_schema;
typedef struct ts_datastore ts_datastore;
typedef struct ts_session ts_session;

/* Decoder shape and capacity limits.  The layer recipe is pre-norm RMSNorm, rotary embedding in
 * the rotate-half pairing, grouped-query attention, SwiGLU MLP, untied LM head, no biases. */
typedef struct {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
  float rope_theta, rms_eps;
  int32_t max_pages;   /* KV pages in the pool (each TS_PAGE_SIZE tokens, all layers; fp16 elements) */
  int32_t max_batch;   /* most sequences per ts_verify call */
  int32_t k_max;       /* most rows per sequence per call, <= TS_K_MAX */
  int32_t max_rows;    /* most rows per call summed over the batch */
  int32_t max_ctx;     /* most tokens per sequence (cache + chunk) */
  int32_t act_split;   /* 1: GEMM activations are fed as a bf16 (hi, lo) pair; 0: hi only */
  int32_t path;        /* 0: the library chooses; 1: one kernel per stage; 2: the single persistent kernel
                          (steps of at most 64 rows; a larger step fails with TS_ERR_K_TOO_LARGE) */
} ts_model_config;

typedef struct {
  uint64_t weights_bytes;    /* device */
  uint64_t kv_pool_bytes;    /* device */
  uint64_t workspace_bytes;  /* device */
  uint64_t host_io_bytes;    /* pinned host */
} ts_buffer_sizes;

typedef struct {
  void *weights, *kv_pool, *workspace; /* device, 1024-byte aligned, sizes as queried */
  void *host_io;                       /* pinned host */
} ts_buffers;

/* Sizes of the caller-allocated buffers for a configuration.  Host-only; needs no device. */
ts_status ts_query_buffer_sizes(const ts_model_config *cfg, ts_buffer_sizes *out);

/* ts_init_model — create the target model M of Algorithm 1 ("Require: target model M") over
 * caller-owned buffers.  Zeroes the workspace and the KV pool (cache positions that were never
 * written must read as finite numbers), builds the TMA descriptors and the rotary table.
 * Weights are loaded afterwards with ts_load_tensor.  `stream` is a cudaStream_t (0 = default).
 * Errors: TS_ERR_ARG (bad shape: head_dim not 64/128, dims not multiples of 128, ...),
 * TS_ERR_CUDA. */
ts_status ts_init_model(const ts_model_config *cfg, const ts_buffers *bufs, void *stream,
                        ts_model **out);

enum { TS_W_EMBED = 0, TS_W_LM_HEAD = 1, TS_W_FINAL_GAIN = 2, TS_W_Q = 3, TS_W_K = 4, TS_W_V = 5,
       TS_W_O = 6, TS_W_GATE = 7, TS_W_UP = 8, TS_W_DOWN = 9, TS_W_GAIN1 = 10, TS_W_GAIN2 = 11 };

/* Upload one tensor.  Matrices are bf16, row-major [out_features][in_features]; gains are
 * float32 [d_model]; the source may be host or device memory (the copy direction is inferred).
 * `layer` is ignored for the three global tensors.  The library lays the matrix out for its
 * kernels (Q,K,V rows concatenated with rotary partners adjacent; gate and up rows interleaved;
 * every projection matrix stored as contiguous 128 x 64 blocks).  Uses the workspace as staging,
 * so the last step's logits are gone afterwards.  Synchronous.
 * Errors: TS_ERR_ARG on a shape that does not match the configuration. */
ts_status ts_load_tensor(ts_model *m, int32_t kind, int32_t layer, const void *host_data,
                         int64_t rows, int64_t cols);

ts_status ts_model_destroy(ts_model *m);

/* ---- schema (Section 4.2: the parsed tool schema S; here supplied already parsed) -------------- */

/* Fixed scaffolding strings of the tool-call format, as token ids:
 *   <tool_call>  pfx name mid  key kvsep value  ( nxt key kvsep value )*  end
 * e.g. pfx = {"name": "   mid = ", "parameters": {"   kvsep = ": "   nxt = ", "   end = "}}
 * Each string has 1..8 ids; scaffolding ids must not occur inside names or keys. */
typedef struct {
  int32_t vocab, eos, tool_call;
  int32_t pfx[8], mid[8], kvsep[8], nxt[8], end[8];
  int32_t pfx_len, mid_len, kvsep_len, nxt_len, end_len;
} ts_vocab_layout;

ts_status ts_schema_create(const ts_vocab_layout *layout, ts_schema **out);
/* key_tokens: all keys' ids concatenated; key_offsets[n_keys+1] delimits them (declared order). */
ts_status ts_schema_add_tool(ts_schema *s, const int32_t *name, int32_t name_len,
                             const int32_t *key_tokens, const int32_t *key_offsets, int32_t n_keys);
ts_status ts_schema_destroy(ts_schema *s);

/* ---- datastore (Section 4.3: H = {(h_j, y_j)}, historical invocations y_j with the hidden state h_j of the
 * question that led to each) --------------------------------------------------------------------------------- */
ts_status ts_datastore_create(int32_t n_tools, ts_datastore **out);
/* Append one historical invocation y_j (host ids, copied) and the tool it called (-1 = unknown), without a hidden
 * state.  Not allowed while a session created over this datastore is between ts_draft calls of a step, and not
 * once hidden states are attached (TS_ERR_STATE: every entry then needs its h_j, see ts_datastore_add_hidden). */
ts_status ts_datastore_add(ts_datastore *d, const int32_t *tokens, int32_t n, int32_t tool_id);
/* Give the datastore the memory for its hidden states: hidden_dev is device memory owned by the caller, bf16
 * [capacity][d_model] row-major, 16-byte aligned, kept alive until the datastore is destroyed or another matrix is
 * attached; row j belongs to entry j.  The library allocates nothing and writes only rows it is told to.  Rows of
 * entries that exist already must hold their states (e.g. a store restored from disk); capacity >= entries.
 * hidden_dev = NULL detaches.  Errors: TS_ERR_ARG. */
ts_status ts_datastore_attach_hidden(ts_datastore *d, void *hidden_dev, int32_t capacity, int32_t d_model);
/* Append (h_j, y_j): y_j as ts_datastore_add, and h_j = the final-norm hidden state (the LM head's input) of row
 * `row` of model m's last step, rounded to bf16, copied device to device into row j of the attached matrix on the
 * model's stream.  The paper takes the question's hidden state at its final token: after ts_prefill of the
 * question, that is row 0 of the session's first ts_verify.  Errors: TS_ERR_STATE (no matrix attached, matrix
 * full, or the last step left no hidden state: it must run the LM head on the one-kernel-per-stage path),
 * TS_ERR_ARG (row outside the step, width mismatch). */
ts_status ts_datastore_add_hidden(ts_datastore *d, ts_model *m, int32_t row, const int32_t *tokens, int32_t n,
                                  int32_t tool_id);
ts_status ts_datastore_destroy(ts_datastore *d);

/* ---- session: one sequence being decoded -------------------------------------------------------- */
typedef struct {
  int32_t n_cap;           /* longest retrieved continuation (paper: 32 for the first candidate) */
  int32_t max_new_tokens;  /* generation budget */
} ts_draft_config;

/* `model` may be NULL for a host-only session (ts_draft / ts_commit_forced only). */
ts_status ts_session_create(ts_model *model, const ts_schema *schema, const ts_datastore *store,
                            const ts_draft_config *cfg, ts_session **out);
/* Install the ranked candidate list I_k (indices into the datastore, best first) that Eq. 3's
 * Top-K would produce.  n = 0 restores the default: every entry, in insertion order. */
ts_status ts_session_set_ranks(ts_session *s, const int32_t *ranks, int32_t n);
ts_status ts_session_destroy(ts_session *s);

/* Feed the prompt: the KV of tokens[0..n-2] is computed with the verify kernels (chunks of k_max,
 * LM head skipped) and tokens[n-1] becomes the pending token; every prompt id also passes through
 * the FSM's delta.  With a host-only session only the FSM part happens. */
ts_status ts_prefill(ts_model *m, ts_session *s, const int32_t *tokens, int32_t n);

/* ts_draft — drafting part of Algorithm 1's loop body.  Retrieval first (Eq. 4: suffix lengths
 * 7, 6, 5 of the generated output, candidates in rank order, first match position), and only if it
 * yields nothing the schema FSM's deterministic filling (Eq. 2).  Writes at most max_draft ids to
 * out_tokens (host, capacity max_draft), their count to *out_n (0 is not an error) and the source
 * to *out_source: 0 none, 1 schema FSM, 2 retrieval.  Host only. */
ts_status ts_draft(ts_session *s, int32_t max_draft, int32_t *out_tokens, int32_t *out_n,
                   int32_t *out_source);

typedef struct {
  int32_t k;                   /* rows verified for this sequence = 1 + number of drafts */
  int32_t accept_len;          /* l: drafts accepted, 0 <= l <= k-1 */
  int32_t n_emitted;           /* l + 1 */
  int32_t emitted[TS_K_MAX];   /* d_1..d_l followed by the bonus token t_l */
  int32_t argmax[TS_K_MAX];    /* t_0..t_{k-1}: per-row argmax, lowest id on ties */
  int32_t first_row;           /* index of this sequence's first row in the step's logits */
} ts_verify_result;

#define TS_FLAG_SKIP_LM_HEAD 1u  /* no logits, no acceptance: rows only extend the KV cache */
#define TS_FLAG_WANT_TOPK 2u     /* also take the TS_TOPK highest logits of every row (ts_last_topk; successor tables) */
#define TS_TOPK 8

/* ts_verify — Verification + SelectLongestAcceptedPrefix for B sequences in one batched forward.
 * Sequence i's chunk is [pending_i, draft_tokens[draft_offsets[i] .. draft_offsets[i+1])], k_i rows
 * at positions len_i .. len_i+k_i-1.  Allocates KV pages as needed, copies the step's inputs to the
 * device, enqueues every kernel of the step, copies the result back and synchronises the stream.
 * The sessions are not advanced: ts_commit does that.  out: host, B entries.
 * Errors: TS_ERR_K_TOO_LARGE, TS_ERR_TOKEN_RANGE, TS_ERR_OOM_PAGES, TS_ERR_STATE (finished or
 * unprefilled session), TS_ERR_DEVICE_TIMEOUT, TS_ERR_CUDA. */
ts_status ts_verify(ts_model *m, ts_session *const *sessions, int32_t B,
                    const int32_t *draft_tokens, const int32_t *draft_offsets, uint32_t flags,
                    ts_verify_result *out);

/* ts_draft_tree — the candidate set B of Algorithm 1 packed as a tree (PackDraftsAsTree).  Retrieval first: up to
 * four continuations of the suffix match, taken in the order (L = 7, 6, 5; candidate rank; match position), a
 * position already taken at a longer L skipped, of at most n_cap, 16, 8 and 8 ids (Appendix B.2's lengths).  If
 * retrieval yields nothing: the schema drafts (Section 4.2) -- with the tool name still open, one chain per tool
 * whose name extends the ids emitted so far (Eq. 2; the tool ts_draft would guess first, then ascending tool id,
 * at most 8 tools); otherwise ts_draft's single chain.  The chains are merged into a token trie: node 0 is the
 * pending token, nodes are numbered in creation order, nothing is added once the chunk holds max_nodes nodes
 * (<= TS_K_MAX).  out_tokens[j], out_parents[j]: token and parent node of node j + 1, in the form ts_verify_tree
 * takes; *out_n = nodes after the root; *out_source: 0 none, 1 schema, 2 retrieval.  The first root-to-leaf path
 * is ts_draft's chain.  Host only; never fails on "no draft". */
ts_status ts_draft_tree(ts_session *s, int32_t max_nodes, int32_t *out_tokens, int32_t *out_parents,
                        int32_t *out_n, int32_t *out_source);

/* General speculative drafting for the open-ended states q_v and q_o (Section 4.2 defers them to a general method and
 * names Token Recycling; Appendix A.1: a pre-defined static tree there; the ablation of Section 5.3 falls back to a
 * suffix match inside the input context).  Off by default.  When on, ts_draft_tree, after retrieval and the schema
 * both yield nothing, (source 3) matches the last 7, 6, 5 ids of the context (prompt followed by the output) against
 * an earlier occurrence in the context, earliest first, and drafts its continuation (at most n_cap ids); failing
 * that, (source 4) builds the static tree over recycled successors: 17 slots in breadth-first order (four successors
 * of the pending token; 3, 2, 1, 1 below them; then 2, 1, 1; then a chain of two), slot i carrying the rank-th entry
 * of its parent's successor list.  A token's successor list is the TS_TOPK ids the model ranked highest right after
 * it, refreshed by every ts_verify / ts_verify_tree call that carries TS_FLAG_WANT_TOPK, from all rows of the chunk. */
ts_status ts_session_enable_general_sd(ts_session *s, int32_t on);
/* Install / read one successor list (TS_TOPK ids, best first); *found = 0 if the token has none. */
ts_status ts_session_set_successors(ts_session *s, int32_t token, const int32_t *ids);
ts_status ts_session_successors(const ts_session *s, int32_t token, int32_t *ids, int32_t *found);
/* The TS_TOPK highest logits of row `row` of the last step (run with TS_FLAG_WANT_TOPK): ids best first, lowest id on
 * ties; values may be NULL. */
ts_status ts_last_topk(ts_model *m, int32_t row, int32_t *ids, float *values);

/* ts_verify_tree — PackDraftsAsTree's output verified in one forward pass under the tree-structured attention
 * mask (Appendix A.1 "Parallel Verification"; Algorithm 1: Verification, SelectLongestAcceptedPrefix).
 * Sequence i's chunk has node 0 = its pending token and node j+1 = draft_tokens[draft_offsets[i] + j], whose
 * parent is node draft_parents[draft_offsets[i] + j], a value in [0, j] (a parent precedes its children; a
 * chain is parents 0, 1, 2, ...).  At most 64 nodes per sequence.  A node attends to the cache and to its
 * ancestors and itself; its rotary position is cache length + depth; its K/V rows go to cache slot
 * cache length + node index.  Acceptance walks from the root: at node u with model token t_u it moves to the
 * lowest-numbered child of u whose token is t_u, and stops when there is none.  out[i]: accept_len = nodes on
 * the path after the root, emitted = their tokens followed by the model's token at the last node, argmax = t_u
 * for every node.  path_out (host, B x TS_K_MAX, may be NULL): node indices of the path, root first, -1 after
 * the end.  Before returning, the K/V rows of the path are moved to consecutive slots (cache length + 0, 1, ..),
 * so ts_commit advances the session exactly as after ts_verify.  The rows of rejected nodes are lost.
 * Runs on the one-kernel-per-stage path only (TS_ERR_UNIMPLEMENTED with path = 2 or without tensor-memory
 * attention); flags must not contain TS_FLAG_SKIP_LM_HEAD.  Other errors as ts_verify, plus TS_ERR_ARG for a
 * parent outside [0, j]. */
ts_status ts_verify_tree(ts_model *m, ts_session *const *sessions, int32_t B,
                         const int32_t *draft_tokens, const int32_t *draft_parents,
                         const int32_t *draft_offsets, uint32_t flags, ts_verify_result *out,
                         int32_t *path_out);

/* ts_verify_sampled — ts_verify with speculative sampling as the acceptance rule (Appendix B.2) at temperature
 * T > 0 instead of the greedy match.  The drafts are deterministic, so the draft distribution is a point mass on
 * the drafted id x: row j accepts draft j + 1 = x with probability p_j(x), p_j = softmax(logits_j / T); the first
 * rejection emits one sample of p_j with x removed (renormalised) and ends the step; if all drafts pass, one sample
 * of the last row's p is emitted.  The emitted ids are then distributed as token-by-token sampling from the model.
 * uniforms (host): one value in [0, 1) per chunk row, rows in the order of the chunks (draft_offsets[B] + B values);
 * within a chunk of k rows, value j < k - 1 decides draft j + 1 (accepted iff it is below p_j(x)) and value k - 1
 * draws the step's one sample: the smallest id whose running sum of weights exp((l - max) / T), in id order,
 * exceeds it times the total.  The library draws no random numbers.  out[i] as ts_verify (argmax still reports
 * the per-row argmax).  Runs on the one-kernel-per-stage path (TS_ERR_UNIMPLEMENTED with path = 2); TS_ERR_ARG for
 * a temperature outside (0, 1e4) or a uniform outside [0, 1).  Other errors as ts_verify. */
ts_status ts_verify_sampled(ts_model *m, ts_session *const *sessions, int32_t B,
                            const int32_t *draft_tokens, const int32_t *draft_offsets, float temperature,
                            const float *uniforms, uint32_t flags, ts_verify_result *out);

/* ts_verify_tree_sampled — the paper's full verification: a draft tree (ts_verify_tree) accepted by speculative
 * sampling (ts_verify_sampled).  At a node the children are tried in node order against the residual: child c with
 * token x is accepted with probability r(x) / R, r being the node's p = softmax(logits / T) with the tokens of the
 * children already refused removed and R its total; if none is accepted (or the node is a leaf) one sample of the
 * residual is emitted and the step ends.  uniforms: one value in [0, 1) per chunk node, chunk after chunk: value c of
 * a chunk decides its node c (c >= 1), value 0 draws the sample.  The children of a node must carry distinct tokens
 * (a trie, as ts_draft_tree builds): TS_ERR_ARG otherwise.  Arguments, result, path and compaction as
 * ts_verify_tree; other errors as ts_verify_tree and ts_verify_sampled. */
ts_status ts_verify_tree_sampled(ts_model *m, ts_session *const *sessions, int32_t B,
                                 const int32_t *draft_tokens, const int32_t *draft_parents,
                                 const int32_t *draft_offsets, float temperature, const float *uniforms,
                                 uint32_t flags, ts_verify_result *out, int32_t *path_out);

/* Enqueue again the device work of the last ts_verify call on its inputs, which are still resident
 * in device memory; no host<->device copy, no synchronisation.  The step is idempotent because
 * sessions advance only in ts_commit.  For timing the kernels alone. */
ts_status ts_verify_replay(ts_model *m);

/* Run the last step once more and return, per class, the summed milliseconds and a count:
 * 0 projection GEMM, 1 attention, 2 attention merge, 3 norm / residual, 4 rotary + KV append,
 * 5 acceptance, 6 the persistent kernel as a whole.  n_classes >= 6 (class 6 is written if
 * n_classes > 6).  With separate kernels an event follows every launch (no overlap between
 * kernels) and the count is the launches; with the persistent kernel classes 0..2 are sums of
 * its phases (time between the grid-wide ends of consecutive phases, read from device-side
 * clocks) and the count is the phases.  Synchronises the stream.  For the benchmark. */
ts_status ts_profile_step(ts_model *m, float *ms_by_class, int32_t *launches_by_class,
                          int32_t n_classes);

/* ts_commit — y <- y (+) emitted, q <- delta(q, .) applied id by id (bonus token included), cache
 * length and pending token advanced; stops at the first id that finishes the generation (call
 * complete, EOS, or max_new_tokens) and drops the rest.  Host only.  One commit per verification: with
 * a model behind the session, TS_ERR_STATE if no ts_verify* call has run since the last commit (or since
 * ts_debug_set_cache / ts_debug_restart). */
ts_status ts_commit(ts_session *s, const ts_verify_result *r);
/* Same, with an emitted span chosen by the caller (n >= 1): the cache keeps the pending token and
 * the first n-1 ids, which must be the ids the last verification was fed at rows 1 .. n-1 (after a tree
 * step: along the accepted path) -- their K/V rows are what the cache holds there.  TS_ERR_ARG if n
 * exceeds those rows or an id differs; the last id is free (it becomes the pending token).  A host-only
 * session (no model) has no cache and takes any span. */
ts_status ts_commit_forced(ts_session *s, const int32_t *emitted, int32_t n);

typedef struct {
  int32_t cache_len, pending, n_output, finished;
  int32_t fsm_kind;    /* 0 q_o, 1 q_t, 2 q_p, 3 q_v, 4 done */
  int32_t fsm_tool;    /* chosen tool or -1 */
  int32_t fsm_key;     /* index of the current key */
  int32_t n_pages;
} ts_session_info;
ts_status ts_session_state(const ts_session *s, ts_session_info *out);
/* Copy the generated output y (at most cap ids) to out (host); *n receives |y|. */
ts_status ts_session_output(const ts_session *s, int32_t *out, int32_t cap, int32_t *n);

/* ts_topk_cosine — Top-K of Eq. 3 (Section 4.3): the K datastore entries whose hidden state is most similar (cosine)
 * to the query's; their indices, best first, are what ts_session_set_ranks takes as the candidate order of the
 * suffix match (the paper uses K = 10).  hidden_dev: device, bf16 [n_entries][d_model] row-major, 16-byte aligned,
 * owned by the caller (the paper stores the hidden representation of each historical question at its final token).
 * query_dev: device fp32 [d_model], or NULL to use the final-norm hidden state of row `row` of the last step (row 0
 * of a session's first step is its question's last token).  scores_dev: device scratch of
 * TS_TOPK_SCRATCH_FLOATS(n_entries, K) floats, 8-byte aligned, owned by the caller, overwritten.  out_index / out_score: host, K entries (out_score may be NULL).  Ties go to the
 * lower index; an entry or query of zero norm scores -2 (ranks last).  Synchronises the model's stream.
 * Errors: TS_ERR_ARG (K outside [1, min(64, n_entries)], bad row), TS_ERR_STATE (no hidden state available). */
#define TS_TOPK_SCRATCH_FLOATS(n, k) ((n) + 2 * (k) + 1 + 2 * (k) * (((n) + 4095) / 4096))
ts_status ts_topk_cosine(ts_model *m, const void *hidden_dev, int32_t n_entries, const float *query_dev,
                         int32_t row, int32_t K, float *scores_dev, int32_t *out_index, float *out_score);
/* ts_session_retrieve — the once-per-query part of Algorithm 1: compute h_x, retrieve the Top-K index set I_k (Eq. 3)
 * from the session's datastore, and make it the candidate order of the suffix match.  h_x is the final-norm hidden
 * state of row `row` of model m's last step (row 0 of the session's first step = the question's last token); the
 * similarity runs over the hidden states attached to the datastore (ts_topk_cosine over rows [0, entries)); the K
 * indices, best first, are installed as by ts_session_set_ranks and also written to out_index (host, K entries;
 * out_score may be NULL).  K is lowered to the number of entries.  scores_dev: device scratch as in ts_topk_cosine.
 * Errors: TS_ERR_STATE (no datastore, no hidden states attached, empty datastore, no hidden state in the last
 * step), TS_ERR_ARG. */
ts_status ts_session_retrieve(ts_model *m, ts_session *s, int32_t row, int32_t K, float *scores_dev,
                              int32_t *out_index, float *out_score, int32_t *out_k);
/* The final-norm hidden state (the LM head's input) of row `row` of the last step, as fp32 [d_model] on the host:
 * what a caller stores per question to build the datastore's hidden states.  TS_ERR_STATE if the last step skipped
 * the LM head or ran as the persistent kernel. */
ts_status ts_last_hidden(ts_model *m, int32_t row, float *host_out);

/* ---- test / benchmark support ------------------------------------------------------------------- */
/* Overwrite the session's cache for one layer with n_tokens rows of host float32 K and V
 * ([n_tokens][n_kv_heads][head_dim]); values are rounded to the cache's storage type (fp16,
 * saturating).  After all layers were imported with the same n_tokens call
 * ts_debug_set_cache(s, n_tokens, pending) to make them the session's context. */
ts_status ts_debug_import_kv(ts_model *m, ts_session *s, int32_t layer, const float *k,
                             const float *v, int32_t n_tokens);
/* Read the first n_tokens cached rows of one layer back as float32. */
ts_status ts_debug_export_kv(ts_model *m, ts_session *s, int32_t layer, float *k, float *v,
                             int32_t n_tokens);
ts_status ts_debug_set_cache(ts_session *s, int32_t cache_len, int32_t pending);
/* ts_debug_set_cache, and the session forgets what it generated: output, FSM state (back to q_o), successor lists,
 * the finished mark.  For replaying a context with another decoding strategy (benchmark traces). */
ts_status ts_debug_restart(ts_session *s, int32_t cache_len, int32_t pending);
/* Copy rows [row0, row0+n_rows) of the last step's float32 logits [rows][vocab] to host memory. */
ts_status ts_read_logits(ts_model *m, int32_t row0, int32_t n_rows, float *host_out);
/* Copy the first `bytes` bytes of an internal activation buffer of the last step to host memory:
 * 0 residual stream x (float32 [rows_alloc][d_model]); 1 projection input activations (bf16
 * [planes][rows_alloc][d_model]; normalised with separate kernels, x times gain before the
 * row scale with the persistent kernel); 2 rotated queries (fp16 [rows_alloc][n_q_heads*head_dim], rounded values;
 * the rounding remainders the attention kernel adds to them are kept beside them and are not returned);
 * 3 attention output (bf16 [planes][rows_alloc][n_q_heads*head_dim]); 4 SwiGLU output (bf16
 * [planes][rows_alloc][d_ffn]).  rows_alloc = max_rows rounded up to 128; planes = 1 + act_split. */
ts_status ts_debug_read_buffer(ts_model *m, int32_t which, void *host_out, uint64_t bytes);
/* Device-side clocks (nanoseconds of the GPU's global timer, latest over the CTAs) that the
 * persistent kernel left during the last ts_profile_step: three rows of *n_phases entries —
 * end of each phase, last MMA of the phase issued, first operand block of the phase ready.
 * Copies at most cap values to out (host).  Phases: 0 embedding, then per layer QKV, attention,
 * merge, O, gate-up, down, then the LM head. */
ts_status ts_debug_phase_clocks(ts_model *m, uint64_t *out, int32_t cap, int32_t *n_phases);
/* The persistent kernel's partition of a projection with n_tiles output tiles of 128 features and
 * n_kblocks blocks of 64 reduction columns over n_ctas CTAs, evaluated on the host for CTA `cta`:
 * writes up to cap records {tile, first k-block, end k-block, parking slot, first CTA of the tile,
 * CTAs sharing the tile} to segments (host, 6 int32 each) and the record count to *n_segments.
 * Host only; for testing the index arithmetic without a GPU. */
ts_status ts_debug_schedule(int32_t n_tiles, int32_t n_kblocks, int32_t n_ctas, int32_t cta, int32_t cap,
                            int32_t *segments, int32_t *n_segments);
/* Timeline of the last step under its normal launch configuration (programmatic dependent launch on, kernels
 * overlapping as in production): the step is run once more with every kernel leaving four device-clock stamps
 * (nanoseconds of the GPU's global timer): earliest CTA start, earliest and latest return from the dependency wait,
 * latest CTA end.  stamps: host, 4 values per launch in launch order; classes: host, the launch's class as in
 * ts_profile_step; at most cap launches are written, *n_launches receives their number.  A launch without stamps
 * (acceptance, Top-K, sampling) reports ~0, ~0, 0, 0.  One-kernel-per-stage path only.  Synchronises the stream. */
ts_status ts_debug_timeline(ts_model *m, uint64_t *stamps, int32_t *classes, int32_t cap, int32_t *n_launches);
/* Make the NEXT step (ts_verify*, ts_prefill chunk) report `code` (> 0) in its device status word, as a bounded
 * device-side wait that expired would: the word is written on the model's stream after the step's last kernel and
 * before the results are read back, so no kernel sees it and nothing is left waiting.  That step then fails with
 * TS_ERR_DEVICE_TIMEOUT (codes below 64) or TS_ERR_DEVICE_BOUNDS (64 + the number of a debug-build index check), the
 * library clears the word and the persistent kernel's counters, and later steps run normally.  For testing the
 * host's handling of a device timeout, or of a failed index check, without making a GPU wait or go out of range. */
ts_status ts_debug_inject_device_error(ts_model *m, int32_t code);
/* Counters: kernels launched since ts_init_model, bytes copied host->device and device->host by
 * ts_verify since then. */
ts_status ts_model_counters(const ts_model *m, int64_t *launches, int64_t *h2d_bytes,
                            int64_t *d2h_bytes);

/* ---- attention without device allocation -------------------------------------------------------- */
/* The paper has no counterpart to this call; it exists for deployment reasons only.
 *
 * Some hosts of this library are not allowed to obtain device memory themselves: a plugin inside
 * a serving process whose memory pool is owned (and fully reserved) by the host application, a
 * callback that runs where cudaMalloc is forbidden, or a process working under a fixed memory
 * budget.  Such a caller cannot size and allocate the workspace that ts_init_model needs.
 * ts_attention_static runs the attention stage of the verify step (rows of the chunk against the
 * paged cache plus the chunk itself, causal inside the chunk) as two kernels of its own -- a split-KV
 * kernel on mma.sync tensor-core instructions and a merge kernel; ts_verify on a B200 runs a
 * tensor-memory kernel instead, so results agree to rounding, not bit for bit -- with all of its
 * scratch memory (per-split partial outputs, their running max / sum, the row-tile table, which a
 * third small kernel builds from cu_rows on the device) in a fixed array of TS_STATIC_ATTN_SCRATCH_MIB MiB (plus about 0.5 MiB of
 * bookkeeping) that is part of the library image.  Every GPU on which the library is loaded
 * holds that array until the process exits.  The call itself allocates nothing, on the host
 * heap or on the device.
 *
 * Arguments: the *_host arrays are read on the host during the call; everything else is device
 * memory owned by the caller and must stay valid until the stream has run the work.
 *   q            fp16 [rows][n_q_heads][head_dim], rotary already applied, rows = cu_rows[batch]
 *   k_pages,
 *   v_pages      fp16 [page][n_kv_heads][TS_PAGE_SIZE][head_dim]; must already hold the chunk rows
 *   block_table  int32 [batch][pages_per_seq]: page ids of each sequence, in position order
 *   cu_rows      int32 [batch+1] row offsets (cu_rows[0] = 0), on the device and on the host
 *   seq_len      int32 [batch] tokens in the cache before the chunk, on the device and on the host
 *                (the host copies are only checked against the limits; the kernels read the device
 *                copies, which must hold the same values)
 *   out          bf16 [planes][out_rows][n_q_heads*head_dim]: plane 0 the rounded result, plane 1
 *                (planes = 2) the rounding remainder, as the output projection consumes them
 * Limits: head_dim 64 or 128; at most TS_K_MAX rows per sequence; rows * n_q_heads * head_dim * 4
 * bytes must fit the scratch array (the number of KV splits is lowered to fit before that);
 * at most 512 row tiles of 64 packed rows.  Beyond them the call fails with TS_ERR_K_TOO_LARGE
 * and a message naming the limit; nothing is launched.
 * First use: the first call on each device looks up the array's device address (that device
 * must be current) and keeps it, so it must not be made while a stream is being captured.  No
 * statement is made about capturing later calls.
 * Sharing: every call on a device uses the same array, which keeps whatever the previous call
 * left there.  No part of it has to start at zero: each call writes every word it later reads.
 * Two calls whose kernels overlap on the GPU (different streams, no ordering between them) race
 * on the array and both results are undefined; order them on one stream or with events.
 * Asynchronous: work is enqueued on `stream` (a cudaStream_t, 0 = default); errors found later
 * surface through the stream as usual.  Errors: TS_ERR_ARG, TS_ERR_K_TOO_LARGE, TS_ERR_CUDA. */
#define TS_STATIC_ATTN_SCRATCH_MIB 16
typedef struct {
  int32_t n_q_heads, n_kv_heads, head_dim;
  int32_t batch, pages_per_seq;
  int32_t out_rows, planes;
  const int32_t *cu_rows_host, *seq_len_host;        /* host */
  const int32_t *cu_rows, *seq_len, *block_table;    /* device */
  const void *q, *k_pages, *v_pages;                 /* device */
  void *out;                                         /* device */
} ts_attention_args;
ts_status ts_attention_static(const ts_attention_args *a, void *stream);

const char *ts_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* TOOLSPEC_H_ */
