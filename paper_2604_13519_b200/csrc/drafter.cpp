#include "drafter.h"

#include <algorithm>
#include <cstring>

int32_t ts_schema::child(int32_t node, int32_t token) const {
  const auto &nx = trie[node].next;
  auto it = std::lower_bound(nx.begin(), nx.end(), std::make_pair(token, INT32_MIN));
  return (it != nx.end() && it->first == token) ? it->second : -1;
}

int32_t ts_schema::walk(const std::vector<int32_t> &prefix) const {
  int32_t n = 0;
  for (int32_t t : prefix) {
    n = child(n, t);
    if (n < 0) return -1;
  }
  return n;
}

namespace ts {

void Fsm::to_o(int32_t token) {
  reset();
  if (token == s->v.tool_call) {
    kind = Q_T;
    stage = s->v.pfx_len > 0 ? ST_PFX : ST_NAME;
  }
}

int Fsm::expect(const int32_t *seq, int32_t len, int32_t token) {
  if (token != seq[i]) return -1;
  ++i;
  return i == len ? 1 : 0;
}

void Fsm::step(int32_t token) {
  const ts_vocab_layout &v = s->v;
  switch (kind) {
    case Q_DONE:
      return;
    case Q_O:
      to_o(token);
      return;
    case Q_T:
      if (stage == ST_PFX) {
        int r = expect(v.pfx, v.pfx_len, token);
        if (r < 0) to_o(token);
        else if (r > 0) { stage = ST_NAME; i = 0; node = 0; name_len = 0; }
      } else if (stage == ST_NAME) {
        int32_t exact = s->trie[node].tool_exact;
        int32_t nx = s->child(node, token);
        if (token == v.mid[0] && exact >= 0) {
          tool = exact; stage = ST_MID; i = 1;
          if (i == v.mid_len) { kind = Q_P; stage = ST_KEY; i = 0; key = 0; }
        } else if (nx >= 0) {
          node = nx; ++name_len;
        } else {
          to_o(token);
        }
      } else {  // ST_MID
        int r = expect(v.mid, v.mid_len, token);
        if (r < 0) to_o(token);
        else if (r > 0) { kind = Q_P; stage = ST_KEY; i = 0; key = 0; }
      }
      return;
    case Q_P:
      if (stage == ST_KEY) {
        const auto &k = s->tools[tool].keys[key];
        int r = expect(k.data(), (int32_t)k.size(), token);
        if (r < 0) to_o(token);
        else if (r > 0) { stage = ST_SEP; i = 0; }
      } else {
        int r = expect(v.kvsep, v.kvsep_len, token);
        if (r < 0) to_o(token);
        else if (r > 0) { kind = Q_V; stage = ST_VAL; i = 0; }
      }
      return;
    case Q_V:
      if (stage == ST_VAL) {
        if (token == v.nxt[0]) {
          if (key + 1 < (int32_t)s->tools[tool].keys.size()) {
            stage = ST_NXT; i = 1;
            if (i == v.nxt_len) { kind = Q_P; stage = ST_KEY; i = 0; ++key; }
          } else {
            to_o(token);
          }
        } else if (token == v.end[0]) {
          stage = ST_END; i = 1;
          if (i == v.end_len) kind = Q_DONE;
        }
      } else if (stage == ST_NXT) {
        int r = expect(v.nxt, v.nxt_len, token);
        if (r < 0) to_o(token);
        else if (r > 0) { kind = Q_P; stage = ST_KEY; i = 0; ++key; }
      } else {
        int r = expect(v.end, v.end_len, token);
        if (r < 0) to_o(token);
        else if (r > 0) kind = Q_DONE;
      }
      return;
  }
}

static void append(std::vector<int32_t> *out, const int32_t *p, int32_t from, int32_t to) {
  for (int32_t j = from; j < to; ++j) out->push_back(p[j]);
}
static void append(std::vector<int32_t> *out, const std::vector<int32_t> &v, int32_t from = 0) {
  for (size_t j = (size_t)from; j < v.size(); ++j) out->push_back(v[j]);
}

void Fsm::draft(int32_t guess, std::vector<int32_t> *out) const {
  const ts_vocab_layout &v = s->v;
  out->clear();
  if (kind == Q_T) {
    if (stage == ST_MID) {
      append(out, v.mid, i, v.mid_len);
      append(out, s->tools[tool].keys[0]);
      append(out, v.kvsep, 0, v.kvsep_len);
      return;
    }
    if (stage == ST_PFX) append(out, v.pfx, i, v.pfx_len);
    if (guess < 0) return;
    const ToolDef &t = s->tools[guess];
    append(out, t.name, stage == ST_PFX ? 0 : name_len);
    append(out, v.mid, 0, v.mid_len);
    append(out, t.keys[0]);
    append(out, v.kvsep, 0, v.kvsep_len);
  } else if (kind == Q_P) {
    if (stage == ST_KEY) {
      append(out, s->tools[tool].keys[key], i);
      append(out, v.kvsep, 0, v.kvsep_len);
    } else {
      append(out, v.kvsep, i, v.kvsep_len);
    }
  } else if (kind == Q_V) {
    if (stage == ST_NXT) {
      append(out, v.nxt, i, v.nxt_len);
      append(out, s->tools[tool].keys[key + 1]);
      append(out, v.kvsep, 0, v.kvsep_len);
    } else if (stage == ST_END) {
      append(out, v.end, i, v.end_len);
    }
  }
}

static inline uint64_t gram_key(const int32_t *p) {  // hash of 5 ids
  uint64_t h = 0x9E3779B97F4A7C15ull;
  for (int j = 0; j < 5; ++j) {
    h ^= (uint64_t)(uint32_t)p[j] + 0x9E3779B97F4A7C15ull + (h << 6) + (h >> 2);
    h *= 0xBF58476D1CE4E5B9ull;
  }
  return h;
}

}  // namespace ts

void ts_datastore::ensure_index() const {
  if (indexed_entries == n_entries()) return;
  size_t old = index.size();
  for (int64_t e = indexed_entries; e < n_entries(); ++e) {
    int32_t len;
    const int32_t *p = entry((int32_t)e, &len);
    for (int32_t m = 5; m < len; ++m) index.push_back({ts::gram_key(p + m - 5), (int32_t)e, m});
  }
  auto cmp = [](const Posting &a, const Posting &b) {
    if (a.key != b.key) return a.key < b.key;
    if (a.entry != b.entry) return a.entry < b.entry;
    return a.m < b.m;
  };
  std::sort(index.begin() + old, index.end(), cmp);
  std::inplace_merge(index.begin(), index.begin() + old, index.end(), cmp);
  indexed_entries = n_entries();
}

namespace ts {

// longest-first over L = 7, 6, 5; candidates in rank order; match positions ascending
void suffix_match(const std::vector<int32_t> &y, const ts_datastore &d, const std::vector<int32_t> *ranks,
                  int32_t n, std::vector<int32_t> *out) {
  out->clear();
  const int32_t ny = (int32_t)y.size();
  if (n <= 0 || ny < 5 || d.n_entries() == 0) return;
  const int32_t *tail = y.data() + ny;  // tail[-L .. -1] is the suffix
  auto matches = [&](const int32_t *p, int32_t m, int32_t L) {
    return m >= L && std::memcmp(p + m - L, tail - L, sizeof(int32_t) * L) == 0;
  };
  auto emit = [&](const int32_t *p, int32_t len, int32_t m) {
    for (int32_t j = m; j < len && j < m + n; ++j) out->push_back(p[j]);
  };
  if (ranks) {
    for (int32_t L = 7; L >= 5; --L) {
      if (ny < L) continue;
      for (int32_t c : *ranks) {
        int32_t len;
        const int32_t *p = d.entry(c, &len);
        for (int32_t m = L; m < len; ++m)
          if (matches(p, m, L)) { emit(p, len, m); return; }
      }
    }
    return;
  }
  d.ensure_index();
  ts_datastore::Posting probe{gram_key(tail - 5), INT32_MIN, INT32_MIN};
  auto lo = std::lower_bound(d.index.begin(), d.index.end(), probe,
                             [](const ts_datastore::Posting &a, const ts_datastore::Posting &b) {
                               if (a.key != b.key) return a.key < b.key;
                               if (a.entry != b.entry) return a.entry < b.entry;
                               return a.m < b.m;
                             });
  for (int32_t L = 7; L >= 5; --L) {
    if (ny < L) continue;
    for (auto it = lo; it != d.index.end() && it->key == probe.key; ++it) {
      int32_t len;
      const int32_t *p = d.entry(it->entry, &len);
      if (matches(p, it->m, L)) { emit(p, len, it->m); return; }
    }
  }
}

void suffix_matches(const std::vector<int32_t> &y, const ts_datastore &d, const std::vector<int32_t> *ranks,
                    const int32_t *caps, int32_t n_caps, int32_t max_draft, std::vector<std::vector<int32_t>> *out) {
  out->clear();
  const int32_t ny = (int32_t)y.size();
  if (max_draft <= 0 || n_caps <= 0 || ny < 5 || d.n_entries() == 0) return;
  const int32_t *tail = y.data() + ny;
  auto matches = [&](const int32_t *p, int32_t m, int32_t L) {
    return m >= L && std::memcmp(p + m - L, tail - L, sizeof(int32_t) * L) == 0;
  };
  std::vector<std::pair<int32_t, int32_t>> taken;   // (entry, m) of the hits so far: at most n_caps
  auto take = [&](int32_t c, const int32_t *p, int32_t len, int32_t m) -> bool {   // true once the set is full
    for (const auto &t : taken)
      if (t.first == c && t.second == m) return false;
    taken.push_back({c, m});
    const int32_t n = std::min(caps[out->size()], max_draft);
    out->emplace_back(p + m, p + std::min(len, m + n));
    return (int32_t)out->size() == n_caps;
  };
  if (ranks) {
    for (int32_t L = 7; L >= 5; --L) {
      if (ny < L) continue;
      for (int32_t c : *ranks) {
        int32_t len;
        const int32_t *p = d.entry(c, &len);
        for (int32_t m = L; m < len; ++m)
          if (matches(p, m, L) && take(c, p, len, m)) return;
      }
    }
    return;
  }
  d.ensure_index();
  ts_datastore::Posting probe{gram_key(tail - 5), INT32_MIN, INT32_MIN};
  auto lo = std::lower_bound(d.index.begin(), d.index.end(), probe,
                             [](const ts_datastore::Posting &a, const ts_datastore::Posting &b) {
                               if (a.key != b.key) return a.key < b.key;
                               if (a.entry != b.entry) return a.entry < b.entry;
                               return a.m < b.m;
                             });
  for (int32_t L = 7; L >= 5; --L) {
    if (ny < L) continue;
    for (auto it = lo; it != d.index.end() && it->key == probe.key; ++it) {
      int32_t len;
      const int32_t *p = d.entry(it->entry, &len);
      if (matches(p, it->m, L) && take(it->entry, p, len, it->m)) return;
    }
  }
}

void pack_candidates(const std::vector<std::vector<int32_t>> &cands, int32_t max_nodes, std::vector<int32_t> *tokens,
                     std::vector<int32_t> *parents) {
  tokens->clear();
  parents->clear();
  // children of node u are found by scanning the nodes created so far (a chunk has at most 64 nodes)
  for (const auto &cand : cands) {
    int32_t u = 0;
    for (int32_t t : cand) {
      int32_t nxt = -1;
      for (size_t j = 0; j < tokens->size(); ++j)
        if ((*parents)[j] == u && (*tokens)[j] == t) { nxt = (int32_t)j + 1; break; }
      if (nxt < 0) {
        if ((int32_t)tokens->size() + 1 >= max_nodes) break;
        tokens->push_back(t);
        parents->push_back(u);
        nxt = (int32_t)tokens->size();
      }
      u = nxt;
    }
  }
}

void context_match(const std::vector<int32_t> &ctx, int32_t n, std::vector<int32_t> *out) {
  out->clear();
  const int32_t len = (int32_t)ctx.size();
  if (n <= 0) return;
  for (int32_t L = 7; L >= 5; --L) {
    if (len <= L) continue;
    const int32_t *tail = ctx.data() + len - L;
    for (int32_t m = L; m < len; ++m) {   // m = len would be the suffix matching itself
      if (std::memcmp(ctx.data() + m - L, tail, sizeof(int32_t) * L) == 0) {
        out->assign(ctx.begin() + m, ctx.begin() + std::min(len, m + n));
        return;
      }
    }
  }
}

// breadth-first: four successors of the pending token; 3, 2, 1, 1 below them; then 2, 1, 1; then a chain of two
const RecycleSlot kRecycleTree[17] = {{0, 0}, {0, 1}, {0, 2}, {0, 3}, {1, 0}, {1, 1}, {1, 2}, {2, 0}, {2, 1}, {3, 0},
                                      {4, 0}, {5, 0}, {5, 1}, {6, 0}, {8, 0}, {12, 0}, {16, 0}};

void recycled_tree(int32_t pending, const std::unordered_map<int32_t, std::array<int32_t, TS_TOPK>> &table,
                   int32_t max_nodes, std::vector<int32_t> *tokens, std::vector<int32_t> *parents) {
  tokens->clear();
  parents->clear();
  int32_t node_of[18], tok_of[18];   // per slot: node number (-1 = left out) and token
  node_of[0] = 0; tok_of[0] = pending;
  for (int i = 1; i <= 17; ++i) {
    node_of[i] = -1; tok_of[i] = -1;
    const RecycleSlot sl = kRecycleTree[i - 1];
    if (node_of[sl.parent] < 0 || (int32_t)tokens->size() + 1 >= max_nodes) continue;
    auto it = table.find(tok_of[sl.parent]);
    if (it == table.end()) continue;
    tok_of[i] = it->second[sl.rank];
    tokens->push_back(tok_of[i]);
    parents->push_back(node_of[sl.parent]);
    node_of[i] = (int32_t)tokens->size();
  }
}

}  // namespace ts
