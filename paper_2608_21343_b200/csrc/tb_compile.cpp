// Host-side graph compiler: phrase lists -> flat arc/state arrays (Sec. 2.1 para. 1-2, the
// potential rule above Eq. 1, Sec. 2.2 para. 2).  Sort-based: the case-folded phrases are
// sorted lexicographically, which makes the distinct prefixes of every length appear in
// breadth-first order (a state's children in ascending class order), so states and arcs are
// numbered directly without building a pointer tree.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <limits>
#include <new>
#include <numeric>
#include <string>
#include <unordered_map>
#include <utility>

#include "tb_internal.h"

namespace {

struct Folded {
  const int32_t* tok;  // into the caller's array
  const float* w;      // may be null
  int32_t len;
};

inline size_t align16(size_t x) { return (x + 15) & ~size_t(15); }

template <typename T>
int32_t append_section(std::vector<unsigned char>& blob, const std::vector<T>& v) {
  size_t off = align16(blob.size());
  blob.resize(off + v.size() * sizeof(T));
  if (!v.empty()) std::memcpy(blob.data() + off, v.data(), v.size() * sizeof(T));
  return static_cast<int32_t>(off);
}

}  // namespace

uint64_t tb_hash_class_map(const int32_t* case_class, int32_t vocab) {
  uint64_t h = 1469598103934665603ull ^ static_cast<uint64_t>(vocab);
  for (int32_t v = 0; v < vocab; ++v) {
    uint64_t c = case_class ? static_cast<uint64_t>(case_class[v]) : static_cast<uint64_t>(v);
    h = (h ^ c) * 1099511628211ull;
  }
  return h;
}

extern "C" const char* tb_strerror(int code) {
  switch (code) {
    case TB_OK: return "ok";
    case TB_ERR_INVALID_ARG: return "invalid argument";
    case TB_ERR_OOM: return "out of memory";
    case TB_ERR_CUDA: return "CUDA runtime error";
    case TB_ERR_ARENA_FULL: return "graph arena full";
    case TB_ERR_BAD_SLOT: return "slot index out of range";
    case TB_ERR_DEVICE_STATUS: return "a kernel recorded a violated bound";
    case TB_ERR_IO: return "file could not be opened, read or written";
    default: return "unknown error";
  }
}

// TB_COMPILE_PAGEABLE: while one of these lives, this thread's images go to the heap.
struct PoolBypass {
  bool on;
  explicit PoolBypass(bool o) : on(o) { if (on) tb_pinned_bypass(true); }
  ~PoolBypass() { if (on) tb_pinned_bypass(false); }
};

// What every front end shares: from the flat arc / state arrays to the device blob (Sec. 2.2 para. 2), with the
// per-state records, token-expanded arcs and resolved lists the kernels read.
static void finalize_graph(tb_graph* g, const int32_t* case_class, int32_t vocab, int32_t n_classes, float lambda) {
  const int32_t N = g->n_states;
  g->case_class.resize(vocab);
  for (int32_t v = 0; v < vocab; ++v) g->case_class[v] = case_class ? case_class[v] : v;
  g->class_map_hash = tb_hash_class_map(case_class, vocab);

  // ---- device blob ---------------------------------------------------------------------------
  std::vector<unsigned char> blob;   // built here, then moved into its final place in one piece
  g->off_arc_begin = append_section(blob, g->state_arc_begin);
  g->off_fail = append_section(blob, g->state_fail);
  g->off_bw = append_section(blob, g->state_bw);
  g->off_arc_cls = append_section(blob, g->arc_class);
  g->off_arc_w = append_section(blob, g->arc_w);
  g->off_arc_dst = append_section(blob, g->arc_dst);
  g->off_final = append_section(blob, g->state_final);
  {  // the tokens of every class, in ascending id order
    std::vector<int32_t> ctb(n_classes + 1, 0), ctk(vocab);
    for (int32_t v = 0; v < vocab; ++v) ctb[g->case_class[v] + 1]++;
    for (int32_t c = 0; c < n_classes; ++c) ctb[c + 1] += ctb[c];
    std::vector<int32_t> fill(ctb.begin(), ctb.end() - 1);
    for (int32_t v = 0; v < vocab; ++v) ctk[fill[g->case_class[v]]++] = v;

    // resolved lists (see TbRsRec): the walk the kernels would do, done once here in float
    float root_w_max = 0.0f;
    for (int32_t a = g->state_arc_begin[0]; a < g->state_arc_begin[1]; ++a) root_w_max = std::max(root_w_max, std::fabs(g->arc_w[a]));
    std::vector<TbRsRec> rrecs(N);
    std::vector<TbRsEnt> rents;
    std::vector<int32_t> seen(n_classes, -1);   // class -> state that listed it during the current walk
    bool fits = 2 * (vocab + 1) <= (1 << TB_RS_TOK_BITS) && N < (1 << (32 - TB_RS_TOK_BITS));
    g->d_max = 0.0f;
    for (int32_t s = 0; s < N; ++s) {
      float acc = 0.0f;
      const size_t first = rents.size();
      for (int32_t u = s; u != 0; u = g->state_fail[u]) {
        if (fits) {
          for (int32_t a = g->state_arc_begin[u]; a < g->state_arc_begin[u + 1]; ++a) {
            const int32_t c = g->arc_class[a];
            if (seen[c] == s) continue;           // shadowed by a chain state closer to s
            seen[c] = s;
            const float bonus = acc + g->arc_w[a];
            const float lb = lambda * bonus;
            for (int32_t j = ctb[c]; j < ctb[c + 1]; ++j)
              rents.push_back({(static_cast<uint32_t>(g->arc_dst[a]) << TB_RS_TOK_BITS) | static_cast<uint32_t>(2 * ctk[j]), lb});
          }
          if (rents.size() > TB_RS_MAX_ENTRIES) fits = false;
        }
        acc = acc + g->state_bw[u];
      }
      g->d_max = std::max(g->d_max, std::fabs(acc));
      if (fits) {
        std::sort(rents.begin() + first, rents.end(), [](const TbRsEnt& x, const TbRsEnt& y) {
          return (x.dst_tok & ((1u << TB_RS_TOK_BITS) - 1)) < (y.dst_tok & ((1u << TB_RS_TOK_BITS) - 1));
        });
        while ((rents.size() - first) % 4 != 0)   // sentinels: the blank column with lb = -inf
          rents.push_back({static_cast<uint32_t>(2 * vocab), -std::numeric_limits<float>::infinity()});
      }
      rrecs[s].begin = static_cast<int32_t>(first);
      rrecs[s].count = static_cast<int32_t>(rents.size() - first);
      rrecs[s].D = acc;
      rrecs[s].bmag = std::fabs(lambda) * (std::fabs(acc) + root_w_max);
    }
    if (fits) {
      // (the kernels read these lists and nothing else beyond the flat arrays: the image carries no per-state records)
      g->off_strec = g->off_tokent = 0;
      g->n_tokent = 0;
      g->off_rsrec = append_section(blob, rrecs);
      g->off_rsent = append_section(blob, rents);
      g->n_rsent = static_cast<int32_t>(rents.size());
    } else {
      // too large for resolved lists: per-state records and token-expanded arcs, which the kernels walk instead
      std::vector<TbStateRec> recs(N);
      std::vector<TbTokEnt> ents;
      for (int32_t u = 0; u < N; ++u) {
        recs[u].tok_begin = static_cast<int32_t>(ents.size());
        for (int32_t a = g->state_arc_begin[u]; a < g->state_arc_begin[u + 1]; ++a) {
          const int32_t c = g->arc_class[a];
          for (int32_t j = ctb[c]; j < ctb[c + 1]; ++j)
            ents.push_back({static_cast<uint32_t>(ctk[j]) | (static_cast<uint32_t>(c) << 16), g->arc_w[a], g->arc_dst[a], 0});
        }
        recs[u].tok_end = static_cast<int32_t>(ents.size());
        recs[u].fail = g->state_fail[u];
        recs[u].bw = g->state_bw[u];
      }
      g->off_strec = append_section(blob, recs);
      g->off_tokent = append_section(blob, ents);
      g->n_tokent = static_cast<int32_t>(ents.size());
      g->off_rsrec = g->off_rsent = 0;
      g->n_rsent = -1;
    }
  }
  blob.resize(align16(blob.size()) + 16);  // tail padding so vector loads may overrun a section
  g->blob = TbImage();
  g->blob.assign(blob.begin(), blob.end());
  g->pinned = tb_pinned_owns(g->blob.data());
}

static int compile_impl(const int32_t* phrase_tokens, const int64_t* phrase_offsets, int32_t n_phrases,
                        const float* token_weights, const int32_t* case_class, int32_t vocab, float lambda,
                        tb_graph* g) {
  // ---- validation -------------------------------------------------------------------------
  int32_t n_classes = vocab;
  if (case_class) {
    n_classes = 0;
    for (int32_t v = 0; v < vocab; ++v) {
      if (case_class[v] < 0) return TB_ERR_INVALID_ARG;
      n_classes = std::max(n_classes, case_class[v] + 1);
    }
  }
  if (n_phrases > 0 && phrase_offsets[0] != 0) return TB_ERR_INVALID_ARG;
  std::vector<Folded> ph;
  ph.reserve(n_phrases);
  int32_t max_len = 0;
  for (int32_t p = 0; p < n_phrases; ++p) {
    int64_t b = phrase_offsets[p], e = phrase_offsets[p + 1];
    if (e < b) return TB_ERR_INVALID_ARG;
    if (e - b > TB_MAX_PHRASE_LEN) return TB_ERR_INVALID_ARG;
    for (int64_t i = b; i < e; ++i) {
      if (phrase_tokens[i] < 0 || phrase_tokens[i] >= vocab) return TB_ERR_INVALID_ARG;
      if (token_weights && !(std::isfinite(token_weights[i]) && token_weights[i] >= 0.0f)) return TB_ERR_INVALID_ARG;
    }
    if (e == b) continue;  // empty phrases are skipped
    ph.push_back({phrase_tokens + b, token_weights ? token_weights + b : nullptr, static_cast<int32_t>(e - b)});
    max_len = std::max(max_len, static_cast<int32_t>(e - b));
  }
  auto cls_of = [&](int32_t tok) { return case_class ? case_class[tok] : tok; };

  // ---- sort the folded phrases, longest-common-prefix with the predecessor -----------------
  const size_t P = ph.size();
  std::vector<uint32_t> order(P);
  std::iota(order.begin(), order.end(), 0u);
  std::sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) {
    const Folded &x = ph[a], &y = ph[b];
    int32_t n = std::min(x.len, y.len);
    for (int32_t i = 0; i < n; ++i) {
      int32_t cx = cls_of(x.tok[i]), cy = cls_of(y.tok[i]);
      if (cx != cy) return cx < cy;
    }
    return x.len < y.len;
  });
  std::vector<int32_t> lcp(P, 0);
  std::vector<size_t> node_base(P + 1, 0);  // where phrase i's node ids start in `node_of`
  for (size_t i = 0; i < P; ++i) {
    const Folded& x = ph[order[i]];
    node_base[i + 1] = node_base[i] + x.len;
    if (i == 0) continue;
    const Folded& y = ph[order[i - 1]];
    int32_t n = std::min(x.len, y.len), l = 0;
    while (l < n && cls_of(x.tok[l]) == cls_of(y.tok[l])) ++l;
    lcp[i] = l;
  }

  // ---- states: distinct prefixes, depth by depth = breadth-first order ----------------------
  std::vector<int32_t> node_of(node_base[P]);   // node id of phrase i's prefix of length d+1
  std::vector<int32_t> parent(1, -1), cls(1, -1);
  std::vector<uint8_t> depth(1, 0), is_end(1, 0);
  std::vector<double> wt(1, 0.0);
  for (int32_t d = 1; d <= max_len; ++d) {
    for (size_t i = 0; i < P; ++i) {
      const Folded& x = ph[order[i]];
      if (x.len < d) continue;
      double w = x.w ? static_cast<double>(x.w[d - 1]) : 1.0;
      int32_t id;
      if (lcp[i] >= d) {  // same prefix as the predecessor, which therefore has this node
        id = node_of[node_base[i - 1] + d - 1];
        wt[id] = std::max(wt[id], w);
      } else {
        id = static_cast<int32_t>(parent.size());
        parent.push_back(d == 1 ? 0 : node_of[node_base[i] + d - 2]);
        cls.push_back(cls_of(x.tok[d - 1]));
        depth.push_back(static_cast<uint8_t>(d));
        is_end.push_back(0);
        wt.push_back(w);
      }
      node_of[node_base[i] + d - 1] = id;
      if (x.len == d) is_end[id] = 1;
    }
  }
  const int32_t N = static_cast<int32_t>(parent.size());
  const int32_t A = N - 1;

  // ---- arcs: arc a enters state a+1; a state's arcs are contiguous --------------------------
  g->n_states = N; g->n_arcs = A; g->n_classes = n_classes; g->vocab = vocab;
  g->max_depth = max_len; g->lambda = lambda;
  g->state_arc_begin.assign(N + 1, 0);
  g->arc_class.resize(A); g->arc_dst.resize(A); g->arc_w.resize(A);
  g->state_fail.assign(N, 0); g->state_bw.assign(N, 0.0f); g->state_final.assign(N, 0.0f);
  g->state_depth.assign(depth.begin(), depth.end());
  for (int32_t id = 1; id < N; ++id) {
    g->state_arc_begin[parent[id] + 1]++;
    g->arc_class[id - 1] = cls[id];
    g->arc_dst[id - 1] = id;
  }
  for (int32_t u = 0; u < N; ++u) g->state_arc_begin[u + 1] += g->state_arc_begin[u];

  auto find_arc = [&](int32_t u, int32_t c) -> int32_t {
    const int32_t* b = g->arc_class.data() + g->state_arc_begin[u];
    const int32_t* e = g->arc_class.data() + g->state_arc_begin[u + 1];
    const int32_t* it = std::lower_bound(b, e, c);
    return (it != e && *it == c) ? static_cast<int32_t>(it - g->arc_class.data()) : -1;
  };

  // ---- suffix links (ids ascend breadth-first, so the parent's link is ready) ---------------
  for (int32_t id = 1; id < N; ++id) {
    int32_t f = 0;
    if (parent[id] != 0) {
      int32_t q = g->state_fail[parent[id]];
      for (;;) {
        int32_t a = find_arc(q, cls[id]);
        if (a >= 0) { f = g->arc_dst[a]; break; }
        if (q == 0) break;
        q = g->state_fail[q];
      }
    }
    g->state_fail[id] = f;
  }

  // ---- potentials in double, stored values rounded once --------------------------------------
  // loan: credit of the partial match since the last completed phrase (returned on back-off);
  // outp: everything banked on arriving at a state (phrases ending there, own or as suffixes).
  std::vector<double> loan(N, 0.0), outp(N, 0.0);
  for (int32_t id = 1; id < N; ++id) {
    double through = loan[parent[id]] + wt[id];
    loan[id] = is_end[id] ? 0.0 : through;
    outp[id] = (is_end[id] ? through : 0.0) + outp[g->state_fail[id]];
  }
  for (int32_t id = 0; id < N; ++id) {
    g->state_final[id] = static_cast<float>(-loan[id]);
    if (id) {
      g->state_bw[id] = static_cast<float>(loan[g->state_fail[id]] - loan[id]);
      g->arc_w[id - 1] = static_cast<float>(loan[id] - loan[parent[id]] + outp[id]);
    }
  }
  finalize_graph(g, case_class, vocab, n_classes, lambda);
  return TB_OK;
}

extern "C" int tb_graph_compile(const int32_t* phrase_tokens, const int64_t* phrase_offsets, int32_t n_phrases,
                                const float* token_weights, const int32_t* case_class, int32_t vocab,
                                float lambda, uint32_t flags, tb_graph** out) {
  TbRange range_("tb_graph_compile");
  if (!out) return TB_ERR_INVALID_ARG;
  *out = nullptr;
  if ((flags & ~static_cast<uint32_t>(TB_COMPILE_PAGEABLE)) != 0 || vocab < 1 || vocab > TB_MAX_VOCAB || n_phrases < 0 || !std::isfinite(lambda)) return TB_ERR_INVALID_ARG;
  PoolBypass bypass((flags & TB_COMPILE_PAGEABLE) != 0);
  if (n_phrases > 0 && (!phrase_offsets || (phrase_offsets[n_phrases] > 0 && !phrase_tokens))) return TB_ERR_INVALID_ARG;
  try {
    tb_graph* g = new tb_graph();
    int rc = compile_impl(phrase_tokens, phrase_offsets, n_phrases, token_weights, case_class, vocab, lambda, g);
    if (rc != TB_OK) { delete g; return rc; }
    *out = g;
    return TB_OK;
  } catch (const std::bad_alloc&) {
    return TB_ERR_OOM;
  }
}

// ---- variative, case-insensitive front end (Sec. 2.1 para. 4-7, Eq. 1) -----------------------------
namespace {

inline unsigned char lower_ascii(unsigned char b) { return (b >= 'A' && b <= 'Z') ? static_cast<unsigned char>(b + 32) : b; }

// One class per distinct lower-cased spelling, numbered by the lowest token id that has it.
int classes_of_pieces(const uint8_t* piece_chars, const int64_t* piece_offsets, int32_t vocab,
                      std::vector<int32_t>& cls, std::vector<std::string>& spell,
                      std::unordered_map<std::string, int32_t>& id_of) {
  if (!piece_offsets || piece_offsets[0] != 0) return TB_ERR_INVALID_ARG;
  cls.resize(vocab);
  for (int32_t v = 0; v < vocab; ++v) {
    const int64_t b = piece_offsets[v], e = piece_offsets[v + 1];
    if (e <= b || e - b > TB_MAX_PIECE_LEN || !piece_chars) return TB_ERR_INVALID_ARG;
    std::string c(static_cast<size_t>(e - b), '\0');
    for (int64_t i = b; i < e; ++i) c[static_cast<size_t>(i - b)] = static_cast<char>(lower_ascii(piece_chars[i]));
    auto it = id_of.find(c);
    if (it == id_of.end()) {
      it = id_of.emplace(c, static_cast<int32_t>(spell.size())).first;
      spell.push_back(c);
    }
    cls[v] = it->second;
  }
  return TB_OK;
}

struct CharPhrase {
  std::string canon;
  std::vector<double> share;   // Eq. 1: this phrase's share for each of its characters
};

int compile_variative_impl(const uint8_t* phrase_chars, const int64_t* phrase_offsets, int32_t n_phrases,
                           const float* phrase_weights, const uint8_t* piece_chars, const int64_t* piece_offsets,
                           int32_t vocab, float tau, float lambda, tb_graph* g) {
  std::vector<int32_t> cls;
  std::vector<std::string> spell;
  std::unordered_map<std::string, int32_t> id_of;
  int rc = classes_of_pieces(piece_chars, piece_offsets, vocab, cls, spell, id_of);
  if (rc != TB_OK) return rc;
  const int32_t n_classes = static_cast<int32_t>(spell.size());
  size_t longest = 0;
  for (const std::string& c : spell) longest = std::max(longest, c.size());
  if (n_phrases > 0 && phrase_offsets[0] != 0) return TB_ERR_INVALID_ARG;

  // ---- phrases: lower-cased, cut greedily (longest spelling first) into the scoring backbone, Eq. 1 per token ----
  std::vector<CharPhrase> ph;
  size_t max_len = 0;
  for (int32_t p = 0; p < n_phrases; ++p) {
    const int64_t b = phrase_offsets[p], e = phrase_offsets[p + 1];
    if (e < b || e - b > 255) return TB_ERR_INVALID_ARG;
    if (e == b) continue;
    const double w = phrase_weights ? static_cast<double>(phrase_weights[p]) : 1.0;
    if (!(std::isfinite(w) && w >= 0.0)) return TB_ERR_INVALID_ARG;
    CharPhrase cp;
    cp.canon.resize(static_cast<size_t>(e - b));
    for (int64_t i = b; i < e; ++i) cp.canon[static_cast<size_t>(i - b)] = static_cast<char>(lower_ascii(phrase_chars[i]));
    const size_t L = cp.canon.size();
    cp.share.reserve(L);
    for (size_t i = 0; i < L;) {
      size_t m = std::min(longest, L - i);
      for (; m >= 1; --m)
        if (id_of.count(cp.canon.substr(i, m))) break;
      if (m == 0) return TB_ERR_INVALID_ARG;            // a character no piece spells
      const double top = std::pow(static_cast<double>(m), static_cast<double>(tau));
      double z = 0.0;
      std::vector<double> ex(m);
      for (size_t j = 0; j < m; ++j) {
        ex[j] = std::exp(std::pow(static_cast<double>(j + 1), static_cast<double>(tau)) - top);
        z = z + ex[j];
      }
      for (size_t j = 0; j < m; ++j) cp.share.push_back(w * ex[j] / z);
      i += m;
    }
    max_len = std::max(max_len, L);
    ph.push_back(std::move(cp));
  }

  // ---- states: the distinct character prefixes, depth by depth over the sorted phrases = breadth first,
  //      a state's children in ascending character order -------------------------------------------------
  const size_t P = ph.size();
  std::vector<uint32_t> order(P);
  std::iota(order.begin(), order.end(), 0u);
  std::sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) {
    const std::string &x = ph[a].canon, &y = ph[b].canon;
    const size_t n = std::min(x.size(), y.size());
    for (size_t i = 0; i < n; ++i)
      if (x[i] != y[i]) return static_cast<unsigned char>(x[i]) < static_cast<unsigned char>(y[i]);
    return x.size() < y.size();
  });
  std::vector<size_t> lcp(P, 0), node_base(P + 1, 0);
  for (size_t i = 0; i < P; ++i) {
    const std::string& x = ph[order[i]].canon;
    node_base[i + 1] = node_base[i] + x.size();
    if (i == 0) continue;
    const std::string& y = ph[order[i - 1]].canon;
    size_t l = 0;
    while (l < x.size() && l < y.size() && x[l] == y[l]) ++l;
    lcp[i] = l;
  }
  std::vector<int32_t> node_of(node_base[P]);
  std::vector<int32_t> parent(1, -1), first_child(1, -1), n_child(1, 0);
  std::vector<unsigned char> ch(1, 0);
  std::vector<uint8_t> depth(1, 0), is_end(1, 0);
  std::vector<double> wt(1, 0.0);
  for (size_t d = 1; d <= max_len; ++d) {
    for (size_t i = 0; i < P; ++i) {
      const CharPhrase& x = ph[order[i]];
      if (x.canon.size() < d) continue;
      int32_t id;
      if (lcp[i] >= d) {
        id = node_of[node_base[i - 1] + d - 1];
        wt[id] = std::max(wt[id], x.share[d - 1]);
      } else {
        id = static_cast<int32_t>(parent.size());
        const int32_t par = d == 1 ? 0 : node_of[node_base[i] + d - 2];
        parent.push_back(par); first_child.push_back(-1); n_child.push_back(0);
        ch.push_back(static_cast<unsigned char>(x.canon[d - 1]));
        depth.push_back(static_cast<uint8_t>(d)); is_end.push_back(0); wt.push_back(x.share[d - 1]);
        if (first_child[par] < 0) first_child[par] = id;
        n_child[par]++;
      }
      node_of[node_base[i] + d - 1] = id;
      if (x.canon.size() == d) is_end[id] = 1;
    }
  }
  const int32_t N = static_cast<int32_t>(parent.size());
  auto child_on = [&](int32_t u, unsigned char b) -> int32_t {
    for (int32_t v = first_child[u], e = v + n_child[u]; v >= 0 && v < e; ++v)
      if (ch[v] == b) return v;
    return -1;
  };

  // ---- suffix links over the characters, potentials as in the tree compiler ---------------------------------
  std::vector<int32_t> fail(N, 0);
  for (int32_t id = 1; id < N; ++id) {
    if (parent[id] == 0) continue;
    int32_t q = fail[parent[id]];
    for (;;) {
      const int32_t v = child_on(q, ch[id]);
      if (v >= 0) { fail[id] = v; break; }
      if (q == 0) break;
      q = fail[q];
    }
  }
  std::vector<double> loan(N, 0.0), outp(N, 0.0);
  for (int32_t id = 1; id < N; ++id) {
    const double through = loan[parent[id]] + wt[id];
    loan[id] = is_end[id] ? 0.0 : through;
    outp[id] = (is_end[id] ? through : 0.0) + outp[fail[id]];
  }

  // ---- arcs: from every state, every class whose spelling continues the state's path; an arc over several
  //      characters collects what the single-character arcs along it would (same total for every segmentation) ----
  g->n_states = N; g->n_classes = n_classes; g->vocab = vocab;
  g->max_depth = static_cast<int32_t>(max_len); g->lambda = lambda;
  g->state_arc_begin.assign(N + 1, 0);
  g->arc_class.clear(); g->arc_dst.clear(); g->arc_w.clear();
  g->state_fail = fail;
  g->state_bw.assign(N, 0.0f); g->state_final.assign(N, 0.0f);
  g->state_depth.assign(depth.begin(), depth.end());
  struct Found { int32_t cls, dst; double w; };
  struct Frame { int32_t node; size_t len; double banked; };
  std::vector<Found> found;
  std::vector<std::pair<Frame, int32_t>> todo;   // (frame, next child to visit)
  std::string path;
  for (int32_t u = 0; u < N; ++u) {
    found.clear(); todo.clear();
    path.assign(longest, '\0');
    // depth-first over the descendants within the longest spelling; `path` holds the characters of the current branch
    todo.push_back({{u, 0, 0.0}, first_child[u]});
    while (!todo.empty()) {
      auto& top = todo.back();
      const Frame f = top.first;
      const int32_t v = top.second;
      if (v < 0 || v >= first_child[f.node] + n_child[f.node]) { todo.pop_back(); continue; }
      top.second = v + 1;
      path[f.len] = static_cast<char>(ch[v]);
      const double got = f.banked + outp[v];
      auto it = id_of.find(path.substr(0, f.len + 1));
      if (it != id_of.end()) found.push_back({it->second, v, loan[v] - loan[u] + got});
      if (f.len + 1 < longest && n_child[v] > 0) todo.push_back({{v, f.len + 1, got}, first_child[v]});
    }
    std::sort(found.begin(), found.end(), [](const Found& a, const Found& b) { return a.cls < b.cls; });
    for (const Found& f : found) {
      g->arc_class.push_back(f.cls); g->arc_dst.push_back(f.dst); g->arc_w.push_back(static_cast<float>(f.w));
    }
    g->state_arc_begin[u + 1] = static_cast<int32_t>(g->arc_class.size());
  }
  g->n_arcs = static_cast<int32_t>(g->arc_class.size());
  for (int32_t id = 0; id < N; ++id) {
    g->state_final[id] = static_cast<float>(-loan[id]);
    if (id) g->state_bw[id] = static_cast<float>(loan[fail[id]] - loan[id]);
  }
  finalize_graph(g, cls.data(), vocab, n_classes, lambda);
  return TB_OK;
}

}  // namespace

extern "C" int tb_piece_classes(const uint8_t* piece_chars, const int64_t* piece_offsets, int32_t vocab,
                                int32_t* out_case_class, int32_t* out_n_classes) {
  if (vocab < 1 || vocab > TB_MAX_VOCAB || !out_case_class) return TB_ERR_INVALID_ARG;
  try {
    std::vector<int32_t> cls;
    std::vector<std::string> spell;
    std::unordered_map<std::string, int32_t> id_of;
    int rc = classes_of_pieces(piece_chars, piece_offsets, vocab, cls, spell, id_of);
    if (rc != TB_OK) return rc;
    std::memcpy(out_case_class, cls.data(), sizeof(int32_t) * static_cast<size_t>(vocab));
    if (out_n_classes) *out_n_classes = static_cast<int32_t>(spell.size());
    return TB_OK;
  } catch (const std::bad_alloc&) {
    return TB_ERR_OOM;
  }
}

extern "C" int tb_graph_compile_variative(const uint8_t* phrase_chars, const int64_t* phrase_offsets, int32_t n_phrases,
                                          const float* phrase_weights, const uint8_t* piece_chars,
                                          const int64_t* piece_offsets, int32_t vocab, float tau, float lambda,
                                          uint32_t flags, tb_graph** out) {
  TbRange range_("tb_graph_compile_variative");
  if (!out) return TB_ERR_INVALID_ARG;
  *out = nullptr;
  if ((flags & ~static_cast<uint32_t>(TB_COMPILE_PAGEABLE)) != 0 || vocab < 1 || vocab > TB_MAX_VOCAB || n_phrases < 0 || !std::isfinite(lambda) ||
      !std::isfinite(tau) || tau < 0.0f)
    return TB_ERR_INVALID_ARG;
  PoolBypass bypass((flags & TB_COMPILE_PAGEABLE) != 0);
  if (n_phrases > 0 && (!phrase_offsets || (phrase_offsets[n_phrases] > 0 && !phrase_chars))) return TB_ERR_INVALID_ARG;
  try {
    tb_graph* g = new tb_graph();
    int rc = compile_variative_impl(phrase_chars, phrase_offsets, n_phrases, phrase_weights, piece_chars, piece_offsets,
                                    vocab, tau, lambda, g);
    if (rc != TB_OK) { delete g; return rc; }
    *out = g;
    return TB_OK;
  } catch (const std::bad_alloc&) {
    return TB_ERR_OOM;
  }
}

extern "C" int tb_graph_view_get(const tb_graph* g, tb_graph_view* out) {
  if (!g || !out) return TB_ERR_INVALID_ARG;
  out->n_states = g->n_states; out->n_arcs = g->n_arcs; out->n_classes = g->n_classes;
  out->vocab = g->vocab; out->max_depth = g->max_depth; out->lambda = g->lambda;
  out->state_arc_begin = g->state_arc_begin.data(); out->arc_class = g->arc_class.data();
  out->arc_dst = g->arc_dst.data(); out->arc_w = g->arc_w.data();
  out->state_fail = g->state_fail.data(); out->state_bw = g->state_bw.data();
  out->state_final = g->state_final.data(); out->state_depth = g->state_depth.data();
  out->case_class = g->case_class.data();
  return TB_OK;
}

extern "C" void tb_graph_free(tb_graph* g) {
  if (g && g->refs.fetch_sub(1) == 1) delete g;   // a cache may still hold the graph
}
