// Model lifecycle off the device (Sec. 2.2 para. 5: the cost that remains is compiling and transferring the
// models when streams are created; a three-level cache hides it).  This file holds the two host levels:
//   disk   -- a compiled graph written to / read from a file (tb_graph_save / tb_graph_load), for large or
//             repeated lists that should not be compiled again in a later process;
//   memory -- compiled graphs kept in host memory under the content of the list they were compiled from
//             (tb_cache_*), so that a stream that brings a list seen before only pays the copy into the arena.
// The third level, registration with the decoder before a session, lives with the arena (tb_batch_register_model).
#include <cstdio>
#include <cstring>
#include <list>
#include <mutex>
#include <new>
#include <string>
#include <unordered_map>

#include "tb_internal.h"

namespace {

constexpr uint32_t kMagic = 0x31474254u;   // "TBG1"
constexpr uint32_t kVersion = 4;

// FNV-1a style checksum over 8-byte words (the tail byte by byte): detects damage, is not cryptographic
uint64_t fnv1a(const void* p, size_t n, uint64_t h = 1469598103934665603ull) {
  const unsigned char* b = static_cast<const unsigned char*>(p);
  size_t i = 0;
  for (; i + 8 <= n; i += 8) {
    uint64_t w;
    std::memcpy(&w, b + i, 8);
    h = (h ^ w) * 1099511628211ull;
    h ^= h >> 29;
  }
  for (; i < n; ++i) h = (h ^ b[i]) * 1099511628211ull;
  return h;
}

struct FileHeader {
  uint32_t magic, version;
  int32_t n_states, n_arcs, n_classes, vocab, max_depth;
  float lambda;
  uint64_t class_map_hash;
  int32_t off_arc_begin, off_fail, off_bw, off_arc_cls, off_arc_w, off_arc_dst, off_strec, off_tokent, n_tokent;
  int32_t off_rsrec, off_rsent, n_rsent;
  float d_max;
  int32_t off_final;
  uint64_t blob_bytes;
  uint64_t payload_hash;   // of the header (this field taken as zero) followed by everything after it
};

template <typename Vec>
void put(std::string& out, const Vec& v) {
  out.append(reinterpret_cast<const char*>(v.data()), v.size() * sizeof(typename Vec::value_type));
}
template <typename Vec>
bool take(const unsigned char*& p, const unsigned char* end, Vec& v, size_t n) {
  using T = typename Vec::value_type;
  if (static_cast<size_t>(end - p) < n * sizeof(T)) return false;
  v.resize(n);
  if (n) std::memcpy(v.data(), p, n * sizeof(T));
  p += n * sizeof(T);
  return true;
}

// Checksum of a file: the header with its checksum field zero, then the payload.
uint64_t file_hash(const FileHeader& h0, const std::string& payload) {
  std::string all(reinterpret_cast<const char*>(&h0), sizeof h0);
  all.append(payload);
  return fnv1a(all.data(), all.size());
}

size_t graph_bytes(const tb_graph* g) {
  return sizeof(tb_graph) + g->blob.size() + 4 * (g->state_arc_begin.size() + g->arc_class.size() + g->arc_dst.size() +
         g->state_fail.size() + g->case_class.size() + g->arc_w.size() + g->state_bw.size() + g->state_final.size()) +
         g->state_depth.size();
}

}  // namespace

extern "C" int tb_graph_save(const tb_graph* g, const char* path) {
  if (!g || !path) return TB_ERR_INVALID_ARG;
  try {
    std::string payload;
    put(payload, g->state_arc_begin); put(payload, g->arc_class); put(payload, g->arc_dst); put(payload, g->arc_w);
    put(payload, g->state_fail); put(payload, g->state_bw); put(payload, g->state_final); put(payload, g->state_depth);
    put(payload, g->case_class); put(payload, g->blob);
    FileHeader h;
    std::memset(&h, 0, sizeof h);
    h.magic = kMagic; h.version = kVersion;
    h.n_states = g->n_states; h.n_arcs = g->n_arcs; h.n_classes = g->n_classes; h.vocab = g->vocab;
    h.max_depth = g->max_depth; h.lambda = g->lambda; h.class_map_hash = g->class_map_hash;
    h.off_arc_begin = g->off_arc_begin; h.off_fail = g->off_fail; h.off_bw = g->off_bw; h.off_arc_cls = g->off_arc_cls;
    h.off_arc_w = g->off_arc_w; h.off_arc_dst = g->off_arc_dst; h.off_strec = g->off_strec; h.off_tokent = g->off_tokent;
    h.n_tokent = g->n_tokent; h.off_rsrec = g->off_rsrec; h.off_rsent = g->off_rsent; h.n_rsent = g->n_rsent;
    h.d_max = g->d_max; h.off_final = g->off_final; h.blob_bytes = g->blob.size();
    h.payload_hash = 0;
    h.payload_hash = file_hash(h, payload);                  // header (with this field zero) and payload together
    std::FILE* f = std::fopen(path, "wb");
    if (!f) return TB_ERR_IO;
    bool ok = std::fwrite(&h, sizeof h, 1, f) == 1;
    ok = ok && (payload.empty() || std::fwrite(payload.data(), payload.size(), 1, f) == 1);
    ok = (std::fclose(f) == 0) && ok;
    return ok ? TB_OK : TB_ERR_IO;
  } catch (const std::bad_alloc&) {
    return TB_ERR_OOM;
  }
}

extern "C" int tb_graph_load(const char* path, tb_graph** out) {
  TbRange range_("tb_graph_load");
  if (!out) return TB_ERR_INVALID_ARG;
  *out = nullptr;
  if (!path) return TB_ERR_INVALID_ARG;
  std::FILE* f = std::fopen(path, "rb");
  if (!f) return TB_ERR_IO;
  tb_graph* g = nullptr;
  try {
    FileHeader h;
    std::string payload;
    bool ok = std::fread(&h, sizeof h, 1, f) == 1;
    if (ok) {
      char buf[1 << 16];
      size_t n;
      while ((n = std::fread(buf, 1, sizeof buf, f)) > 0) payload.append(buf, n);
      ok = std::ferror(f) == 0;
    }
    std::fclose(f);
    f = nullptr;
    if (!ok) return TB_ERR_IO;
    // a file that is not one of ours, was cut short or was altered is refused as a whole
    if (h.magic != kMagic || h.version != kVersion) return TB_ERR_INVALID_ARG;
    if (h.n_states < 1 || h.n_arcs < 0 || h.vocab < 1 || h.vocab > TB_MAX_VOCAB || h.n_classes < 1) return TB_ERR_INVALID_ARG;
    {
      FileHeader h0 = h;
      h0.payload_hash = 0;
      if (h.payload_hash != file_hash(h0, payload)) return TB_ERR_INVALID_ARG;
    }
    if (h.max_depth < 0 || h.max_depth > TB_MAX_PHRASE_LEN || h.n_tokent < 0) return TB_ERR_INVALID_ARG;
    g = new tb_graph();
    const unsigned char* p = reinterpret_cast<const unsigned char*>(payload.data());
    const unsigned char* end = p + payload.size();
    const size_t N = static_cast<size_t>(h.n_states), A = static_cast<size_t>(h.n_arcs);
    ok = take(p, end, g->state_arc_begin, N + 1) && take(p, end, g->arc_class, A) && take(p, end, g->arc_dst, A) &&
         take(p, end, g->arc_w, A) && take(p, end, g->state_fail, N) && take(p, end, g->state_bw, N) &&
         take(p, end, g->state_final, N) && take(p, end, g->state_depth, N) &&
         take(p, end, g->case_class, static_cast<size_t>(h.vocab)) && take(p, end, g->blob, static_cast<size_t>(h.blob_bytes)) &&
         p == end;
    if (!ok) { delete g; return TB_ERR_INVALID_ARG; }
    g->n_states = h.n_states; g->n_arcs = h.n_arcs; g->n_classes = h.n_classes; g->vocab = h.vocab;
    g->max_depth = h.max_depth; g->lambda = h.lambda; g->class_map_hash = h.class_map_hash;
    g->off_arc_begin = h.off_arc_begin; g->off_fail = h.off_fail; g->off_bw = h.off_bw; g->off_arc_cls = h.off_arc_cls;
    g->off_arc_w = h.off_arc_w; g->off_arc_dst = h.off_arc_dst; g->off_strec = h.off_strec; g->off_tokent = h.off_tokent;
    g->n_tokent = h.n_tokent; g->off_rsrec = h.off_rsrec; g->off_rsent = h.off_rsent; g->n_rsent = h.n_rsent;
    g->d_max = h.d_max; g->off_final = h.off_final;
    // the sections named by the header must lie inside the blob
    const int64_t B = static_cast<int64_t>(g->blob.size());
    const int32_t offs[] = {g->off_arc_begin, g->off_fail, g->off_bw, g->off_arc_cls, g->off_arc_w, g->off_arc_dst,
                            g->off_strec, g->off_tokent, g->off_rsrec, g->off_rsent, g->off_final};
    for (int32_t o : offs)
      if (o < 0 || o > B || (o & 15)) { delete g; return TB_ERR_INVALID_ARG; }
    // ... with their whole extent, and what the kernels index with must stay inside the arrays
    {
      const int64_t Ns = h.n_states, As = h.n_arcs, Te = h.n_tokent, Re = h.n_rsent;
      bool in = g->off_arc_begin + 4 * (Ns + 1) <= B && g->off_fail + 4 * Ns <= B && g->off_bw + 4 * Ns <= B &&
                g->off_arc_cls + 4 * As <= B && g->off_arc_w + 4 * As <= B && g->off_arc_dst + 4 * As <= B &&
                g->off_final + 4 * Ns <= B;
      // a graph carries either resolved lists or per-state records with token-expanded arcs, never both
      if (Re >= 0) in = in && g->off_rsrec + 16 * Ns <= B && g->off_rsent + 8 * Re <= B && Te == 0 && g->off_strec == 0 && g->off_tokent == 0;
      else in = in && g->off_strec + 16 * Ns <= B && g->off_tokent + 16 * Te <= B;
      in = in && g->state_arc_begin[0] == 0 && g->state_arc_begin[Ns] == As;
      for (int64_t u = 0; in && u < Ns; ++u)
        in = g->state_arc_begin[u] <= g->state_arc_begin[u + 1] && g->state_fail[u] >= 0 && g->state_fail[u] < Ns;
      for (int64_t a = 0; in && a < As; ++a)
        in = g->arc_dst[a] >= 0 && g->arc_dst[a] < Ns && g->arc_class[a] >= 0 && g->arc_class[a] < h.n_classes;
      if (!in) { delete g; return TB_ERR_INVALID_ARG; }
      // the device-side copies of the same tables, and the derived records
      const unsigned char* bl = g->blob.data();
      auto i32 = [&](int32_t off, int64_t i) { int32_t v; std::memcpy(&v, bl + off + 4 * i, 4); return v; };
      in = i32(g->off_arc_begin, 0) == 0 && i32(g->off_arc_begin, Ns) == As;
      for (int64_t u = 0; in && u < Ns; ++u) {
        const int32_t f = i32(g->off_fail, u);
        in = i32(g->off_arc_begin, u) <= i32(g->off_arc_begin, u + 1) && f >= 0 && f < Ns;
        if (Re < 0) {
          TbStateRec sr;
          std::memcpy(&sr, bl + g->off_strec + 16 * u, 16);
          in = in && sr.tok_begin >= 0 && sr.tok_begin <= sr.tok_end && sr.tok_end <= Te && sr.fail >= 0 && sr.fail < Ns;
        }
      }
      for (int64_t a = 0; in && a < As; ++a) {
        const int32_t d = i32(g->off_arc_dst, a), c = i32(g->off_arc_cls, a);
        in = d >= 0 && d < Ns && c >= 0 && c < h.n_classes;
      }
      for (int64_t e = 0; in && e < Te; ++e) {
        TbTokEnt te;
        std::memcpy(&te, bl + g->off_tokent + 16 * e, 16);
        in = static_cast<int32_t>(te.tok_cls & 0xffffu) < h.vocab && te.dst >= 0 && te.dst < Ns;
      }
      if (Re >= 0) {
        in = in && Re <= TB_RS_MAX_ENTRIES && h.vocab + 1 <= (1 << (TB_RS_TOK_BITS - 1));
        for (int64_t u = 0; in && u < Ns; ++u) {
          TbRsRec rr;
          std::memcpy(&rr, bl + g->off_rsrec + 16 * u, 16);
          in = rr.begin >= 0 && rr.count >= 0 && static_cast<int64_t>(rr.begin) + rr.count <= Re;
        }
        for (int64_t e = 0; in && e < Re; ++e) {
          TbRsEnt re;
          std::memcpy(&re, bl + g->off_rsent + 8 * e, 8);
          const uint32_t tok2 = re.dst_tok & ((1u << TB_RS_TOK_BITS) - 1), dst = re.dst_tok >> TB_RS_TOK_BITS;
          in = tok2 <= 2u * static_cast<uint32_t>(h.vocab) && (tok2 & 1u) == 0 && dst < static_cast<uint32_t>(Ns);
        }
      }
      if (!in) { delete g; return TB_ERR_INVALID_ARG; }
    }
    if (g->class_map_hash != tb_hash_class_map(g->case_class.data(), g->vocab)) { delete g; return TB_ERR_INVALID_ARG; }
    g->pinned = tb_pinned_owns(g->blob.data());
    *out = g;
    return TB_OK;
  } catch (const std::bad_alloc&) {
    if (f) std::fclose(f);
    delete g;
    return TB_ERR_OOM;
  }
}

// ---- memory level ---------------------------------------------------------------------------------------------
struct tb_cache {
  struct Entry { std::string key; tb_graph* g; size_t bytes; };
  std::mutex mu;
  std::list<Entry> lru;                                           // front = most recently used
  std::unordered_map<std::string, std::list<Entry>::iterator> map;
  size_t capacity = 0, used = 0;
  int64_t hits = 0, misses = 0, evictions = 0;
};

extern "C" int tb_cache_create(size_t capacity_bytes, tb_cache** out) {
  if (!out || capacity_bytes == 0) return TB_ERR_INVALID_ARG;
  tb_cache* c = new (std::nothrow) tb_cache();
  if (!c) return TB_ERR_OOM;
  c->capacity = capacity_bytes;
  *out = c;
  return TB_OK;
}

extern "C" void tb_cache_destroy(tb_cache* c) {
  if (!c) return;
  for (auto& e : c->lru) tb_graph_free(e.g);
  delete c;
}

extern "C" int tb_cache_stats(tb_cache* c, int64_t* hits, int64_t* misses, int64_t* evictions, size_t* bytes_used,
                              int64_t* entries) {
  if (!c) return TB_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(c->mu);
  if (hits) *hits = c->hits;
  if (misses) *misses = c->misses;
  if (evictions) *evictions = c->evictions;
  if (bytes_used) *bytes_used = c->used;
  if (entries) *entries = static_cast<int64_t>(c->lru.size());
  return TB_OK;
}

// A hit hands out the cached graph with one more reference and makes it the most recently used.
static bool cache_lookup(tb_cache* c, const std::string& key, tb_graph** out) {
  std::lock_guard<std::mutex> lk(c->mu);
  auto it = c->map.find(key);
  if (it == c->map.end()) return false;
  c->lru.splice(c->lru.begin(), c->lru, it->second);
  it->second->g->refs.fetch_add(1);
  *out = it->second->g;
  c->hits++;
  return true;
}

// Keeps a freshly compiled graph (the caller keeps its own reference), dropping the least recently used ones first.
static void cache_insert(tb_cache* c, const std::string& key, tb_graph* g) {
  const size_t bytes = graph_bytes(g) + key.size();
  std::lock_guard<std::mutex> lk(c->mu);
  c->misses++;
  if (bytes > c->capacity || c->map.find(key) != c->map.end()) return;
  while (c->used + bytes > c->capacity && !c->lru.empty()) {
    auto& last = c->lru.back();
    c->used -= last.bytes;
    c->map.erase(last.key);
    tb_graph_free(last.g);
    c->lru.pop_back();
    c->evictions++;
  }
  g->refs.fetch_add(1);
  tb_graph_pin(g);                                              // it will be bound again: binds then copy from it in place
  c->lru.push_front({key, g, bytes});
  c->map[key] = c->lru.begin();
  c->used += bytes;
}

extern "C" int tb_cache_compile(tb_cache* c, const int32_t* phrase_tokens, const int64_t* phrase_offsets, int32_t n_phrases,
                                const float* token_weights, const int32_t* case_class, int32_t vocab, float lambda,
                                uint32_t flags, tb_graph** out, int32_t* out_hit) {
  TbRange range_("tb_cache_compile");
  if (!c || !out) return TB_ERR_INVALID_ARG;
  *out = nullptr;
  if (out_hit) *out_hit = 0;
  if (n_phrases < 0 || vocab < 1 || vocab > TB_MAX_VOCAB || (n_phrases > 0 && !phrase_offsets)) return TB_ERR_INVALID_ARG;
  if (n_phrases > 0 && (phrase_offsets[0] != 0 || phrase_offsets[n_phrases] < 0 ||
                        (phrase_offsets[n_phrases] > 0 && !phrase_tokens)))
    return TB_ERR_INVALID_ARG;
  try {
    // the key is the content of everything the compiler reads
    const size_t n_tok = n_phrases > 0 ? static_cast<size_t>(phrase_offsets[n_phrases]) : 0;
    std::string key;
    const uint64_t cm = tb_hash_class_map(case_class, vocab);
    const int32_t head[4] = {vocab, n_phrases, static_cast<int32_t>(flags), token_weights ? 1 : 0};
    key.append(reinterpret_cast<const char*>(head), sizeof head);
    key.append(reinterpret_cast<const char*>(&lambda), sizeof lambda);
    key.append(reinterpret_cast<const char*>(&cm), sizeof cm);
    if (n_phrases > 0) key.append(reinterpret_cast<const char*>(phrase_offsets), sizeof(int64_t) * (static_cast<size_t>(n_phrases) + 1));
    if (n_tok) key.append(reinterpret_cast<const char*>(phrase_tokens), sizeof(int32_t) * n_tok);
    if (n_tok && token_weights) key.append(reinterpret_cast<const char*>(token_weights), sizeof(float) * n_tok);
    if (cache_lookup(c, key, out)) { if (out_hit) *out_hit = 1; return TB_OK; }
    tb_graph* g = nullptr;
    int rc = tb_graph_compile(phrase_tokens, phrase_offsets, n_phrases, token_weights, case_class, vocab, lambda, flags, &g);
    if (rc != TB_OK) return rc;
    cache_insert(c, key, g);
    *out = g;
    return TB_OK;
  } catch (const std::bad_alloc&) {
    return TB_ERR_OOM;
  }
}

extern "C" int tb_cache_compile_variative(tb_cache* c, const uint8_t* phrase_chars, const int64_t* phrase_offsets,
                                          int32_t n_phrases, const float* phrase_weights, const uint8_t* piece_chars,
                                          const int64_t* piece_offsets, int32_t vocab, float tau, float lambda,
                                          uint32_t flags, tb_graph** out, int32_t* out_hit) {
  if (!c || !out) return TB_ERR_INVALID_ARG;
  *out = nullptr;
  if (out_hit) *out_hit = 0;
  if (n_phrases < 0 || vocab < 1 || vocab > TB_MAX_VOCAB || !piece_offsets || piece_offsets[0] != 0 ||
      piece_offsets[vocab] <= 0 || !piece_chars || (n_phrases > 0 && !phrase_offsets))
    return TB_ERR_INVALID_ARG;
  if (n_phrases > 0 && (phrase_offsets[0] != 0 || phrase_offsets[n_phrases] < 0 ||
                        (phrase_offsets[n_phrases] > 0 && !phrase_chars)))
    return TB_ERR_INVALID_ARG;
  try {
    const size_t n_ch = n_phrases > 0 ? static_cast<size_t>(phrase_offsets[n_phrases]) : 0;
    const size_t n_pc = static_cast<size_t>(piece_offsets[vocab]);
    std::string key("variative", 9);
    const int32_t head[4] = {vocab, n_phrases, static_cast<int32_t>(flags), phrase_weights ? 1 : 0};
    key.append(reinterpret_cast<const char*>(head), sizeof head);
    key.append(reinterpret_cast<const char*>(&tau), sizeof tau);
    key.append(reinterpret_cast<const char*>(&lambda), sizeof lambda);
    // the vocabulary enters by a checksum of its spellings and boundaries (it is large and the same for every list)
    const uint64_t vh = fnv1a(piece_offsets, sizeof(int64_t) * (static_cast<size_t>(vocab) + 1), fnv1a(piece_chars, n_pc));
    key.append(reinterpret_cast<const char*>(&vh), sizeof vh);
    if (n_phrases > 0) key.append(reinterpret_cast<const char*>(phrase_offsets), sizeof(int64_t) * (static_cast<size_t>(n_phrases) + 1));
    if (n_ch) key.append(reinterpret_cast<const char*>(phrase_chars), n_ch);
    if (n_phrases > 0 && phrase_weights) key.append(reinterpret_cast<const char*>(phrase_weights), sizeof(float) * static_cast<size_t>(n_phrases));
    if (cache_lookup(c, key, out)) { if (out_hit) *out_hit = 1; return TB_OK; }
    tb_graph* g = nullptr;
    int rc = tb_graph_compile_variative(phrase_chars, phrase_offsets, n_phrases, phrase_weights, piece_chars, piece_offsets,
                                        vocab, tau, lambda, flags, &g);
    if (rc != TB_OK) return rc;
    cache_insert(c, key, g);
    *out = g;
    return TB_OK;
  } catch (const std::bad_alloc&) {
    return TB_ERR_OOM;
  }
}
