// Host-side drafting structures: tool schema with a name trie, the schema finite-state machine
// (Section 4.2 of the paper), and the datastore of historical invocations with a 5-gram index for
// suffix matching (Section 4.3, Eq. 4).
#pragma once
#include <cstdint>
#include <string>
#include <array>
#include <unordered_map>
#include <vector>

#include "toolspec.h"

namespace ts {

struct ToolDef {
  std::vector<int32_t> name;
  std::vector<std::vector<int32_t>> keys;
};

struct TrieNode {
  std::vector<std::pair<int32_t, int32_t>> next;  // (token, child), kept sorted by token
  int32_t tool_exact = -1;                        // tool whose full name ends here
  int32_t min_tool = -1;                          // lowest tool id in this subtree
  std::vector<int32_t> tools;                     // every tool id in this subtree (ascending)
};

}  // namespace ts

struct ts_schema {
  ts_vocab_layout v{};
  std::vector<ts::ToolDef> tools;
  std::vector<ts::TrieNode> trie;  // node 0 = root
  int32_t child(int32_t node, int32_t token) const;
  int32_t walk(const std::vector<int32_t> &prefix) const;  // -1 if no tool has this prefix
};

struct ts_datastore {
  std::vector<int32_t> tokens;       // all entries concatenated
  std::vector<int64_t> offset{0};    // entry e = tokens[offset[e] .. offset[e+1])
  std::vector<int32_t> tool_of;
  std::vector<int64_t> freq;         // per tool
  // hidden states h_j of the entries (Section 4.3: H = {(h_j, y_j)}): a caller-owned device matrix, bf16
  // [hidden_capacity][hidden_width] row-major, row j = entry j; null until attached
  void *hidden_dev = nullptr;
  int32_t hidden_capacity = 0, hidden_width = 0;
  // index over every position m with a 5-gram ending at m and a non-empty continuation
  struct Posting { uint64_t key; int32_t entry; int32_t m; };
  mutable std::vector<Posting> index;
  mutable int64_t indexed_entries = 0;
  void ensure_index() const;
  int32_t n_entries() const { return (int32_t)tool_of.size(); }
  const int32_t *entry(int32_t e, int32_t *len) const {
    *len = (int32_t)(offset[e + 1] - offset[e]);
    return tokens.data() + offset[e];
  }
};

namespace ts {

enum FsmKind : int32_t { Q_O = 0, Q_T = 1, Q_P = 2, Q_V = 3, Q_DONE = 4 };
enum FsmStage : int32_t { ST_NONE = 0, ST_PFX, ST_NAME, ST_MID, ST_KEY, ST_SEP, ST_VAL, ST_NXT, ST_END };

// State of the schema FSM F = (Q, Sigma_schema, delta, q0), q0 = q_o.
struct Fsm {
  const ts_schema *s = nullptr;
  int32_t kind = Q_O, stage = ST_NONE, i = 0, tool = -1, key = 0, node = 0;
  int32_t name_len = 0;
  void reset() { kind = Q_O; stage = ST_NONE; i = 0; tool = -1; key = 0; node = 0; name_len = 0; }
  void step(int32_t token);                         // delta
  // deterministic schema filling from the current state; guess = tool to assume while the name is open
  void draft(int32_t guess, std::vector<int32_t> *out) const;
 private:
  void to_o(int32_t token);
  int expect(const int32_t *seq, int32_t len, int32_t token);  // -1 mismatch, 0 more, 1 complete
};

// Eq. 4 over the store: returns the continuation (possibly empty).
void suffix_match(const std::vector<int32_t> &y, const ts_datastore &d, const std::vector<int32_t> *ranks,
                  int32_t n, std::vector<int32_t> *out);

// The retrieval candidate set: hits in the order (L descending, candidate rank ascending, position ascending), a
// position already taken at a longer L skipped; hit i contributes at most caps[i] ids (and at most max_draft);
// at most n_caps continuations.  The first one equals suffix_match's draft for n = min(caps[0], max_draft).
void suffix_matches(const std::vector<int32_t> &y, const ts_datastore &d, const std::vector<int32_t> *ranks,
                    const int32_t *caps, int32_t n_caps, int32_t max_draft, std::vector<std::vector<int32_t>> *out);

// PackDraftsAsTree: merge candidate chains into a token trie, nodes numbered in creation order (node 0 = the
// pending token), no node added once the chunk holds max_nodes nodes.  tokens: nodes 1..; parents: parent of
// node j + 1 at index j.
void pack_candidates(const std::vector<std::vector<int32_t>> &cands, int32_t max_nodes, std::vector<int32_t> *tokens,
                     std::vector<int32_t> *parents);

// Suffix match inside the context itself (prompt followed by the generated output), as the paper's ablation without
// schema and retrieval falls back to: L = 7, 6, 5 ids at the end of the context, the earliest earlier occurrence,
// continuation of at most n ids.
void context_match(const std::vector<int32_t> &ctx, int32_t n, std::vector<int32_t> *out);

// Static draft tree over recycled successors: node slots in breadth-first order, slot i hangs from slot
// kRecycleTree[i].parent and carries the rank-th successor of that slot's token (slot 0 = the pending token).  A
// slot whose parent is missing or whose parent's token has no table entry is left out; nodes are numbered in
// creation order; nothing is added once the chunk holds max_nodes nodes.
struct RecycleSlot { int8_t parent, rank; };
extern const RecycleSlot kRecycleTree[17];
void recycled_tree(int32_t pending, const std::unordered_map<int32_t, std::array<int32_t, TS_TOPK>> &table,
                   int32_t max_nodes, std::vector<int32_t> *tokens, std::vector<int32_t> *parents);

}  // namespace ts
