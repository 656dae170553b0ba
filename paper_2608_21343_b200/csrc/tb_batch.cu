// Batch object: the merged multi-model storage (one device arena for all bound graphs behind a
// per-slot offset table, Sec. 2.2 para. 2), graph add / swap / remove (Sec. 2.2 para. 4) with
// asynchronous host-to-device copies through pinned staging, and the C-ABI entry points that
// validate arguments and launch the decode kernels.
#include <cstring>
#include <atomic>
#include <iterator>
#include <map>
#include <mutex>
#include <new>
#include <vector>

#include "tb_launch.h"

namespace {

constexpr size_t kArenaAlign = 256;
constexpr int kStagingRing = 4;
constexpr size_t kGroupBytes = 4u << 20;   // graphs a group bind packs into one copy (larger groups go in parts)

struct DeviceGuard {  // makes the batch's device current for the duration of a call
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; cudaGetLastError(); return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) { ok = false; cudaGetLastError(); }
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

// First-fit free list over the arena with coalescing.  Live graphs never move: a slot keeps its
// block until it is re-bound, so no decode in flight ever sees its arrays shift.  (The paper
// compacts the merged tensors on removal; with a free list the physical offsets of the other
// models stay put and the slot index plays the role of the stable model id.)
struct ArenaAllocator {
  std::map<size_t, size_t> free_blocks;  // offset -> size
  size_t capacity = 0;
  void init(size_t bytes) { capacity = bytes; free_blocks.clear(); if (bytes) free_blocks[0] = bytes; }
  bool alloc(size_t bytes, size_t* off) {
    for (auto it = free_blocks.begin(); it != free_blocks.end(); ++it) {
      if (it->second >= bytes) {
        *off = it->first;
        size_t rest = it->second - bytes, start = it->first;
        free_blocks.erase(it);
        if (rest) free_blocks[start + bytes] = rest;
        return true;
      }
    }
    return false;
  }
  void release(size_t off, size_t bytes) {
    auto next = free_blocks.lower_bound(off);
    if (next != free_blocks.begin()) {
      auto prev = std::prev(next);
      if (prev->first + prev->second == off) { off = prev->first; bytes += prev->second; free_blocks.erase(prev); }
    }
    if (next != free_blocks.end() && off + bytes == next->first) { bytes += next->second; free_blocks.erase(next); }
    free_blocks[off] = bytes;
  }
};

struct Staging {
  unsigned char* host = nullptr;
  size_t cap = 0;
  cudaEvent_t done = nullptr;
  bool pending = false;
  tb_graph* held = nullptr;   // a pinned graph whose blob the pending copy reads: released once the copy is done
  std::vector<tb_graph*> held_more;   // the same for a group bind (tb_batch_bind_streams)
};

inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace

tb_graph::~tb_graph() {
  if (registered) { cudaHostUnregister(blob.data()); cudaGetLastError(); }
}

void tb_graph_pin(tb_graph* g) {
  if (!g || g->pinned || g->blob.empty()) return;
  // (portable: whichever device's batch binds the graph later may copy from it)
  if (cudaHostRegister(g->blob.data(), g->blob.size(), cudaHostRegisterPortable) == cudaSuccess) g->pinned = g->registered = true;
  else cudaGetLastError();
}

// ---- the pool of page-locked memory for graph images (see tb_internal.h) ---------------------------------------
namespace {
constexpr size_t kPoolChunk = static_cast<size_t>(32) << 20;     // allocated from the driver in pieces of this size
constexpr size_t kPoolMax = static_cast<size_t>(1) << 30;        // the pool never takes more than this
constexpr size_t kPoolLargest = static_cast<size_t>(16) << 20;   // larger images stay on the heap
struct PinnedPool {
  std::mutex mu;
  struct Chunk {
    unsigned char* base;
    unsigned char* dev_base;                                       // the same memory as kernels address it, or null
    size_t bytes;
    std::map<size_t, size_t> free_blocks;                          // offset -> bytes, neighbours coalesced
  };
  std::vector<Chunk> chunks;
  size_t total = 0;
  std::atomic<bool> armed{false};
  bool closed = false;                                             // the driver refused a chunk: no further attempts
};
thread_local bool g_pool_bypass = false;
PinnedPool& pinned_pool() {
  static PinnedPool* pool = new PinnedPool();                      // (never destroyed: graphs may be freed during exit)
  return *pool;
}
}  // namespace

void tb_pinned_bypass(bool on) { g_pool_bypass = on; }

void tb_pinned_pool_arm() {
  PinnedPool& pool = pinned_pool();
  if (pool.armed.exchange(true)) return;
  // the first piece is taken now (page-locking 32 MB takes tens of milliseconds, which belongs to start-up and not
  // to the first compile after it)
  void* p = tb_pinned_alloc(kArenaAlign);
  if (p) tb_pinned_free(p, kArenaAlign);
}

void* tb_pinned_alloc(size_t bytes) {
  PinnedPool& pool = pinned_pool();
  if (!pool.armed.load() || g_pool_bypass || bytes == 0 || bytes > kPoolLargest) return nullptr;
  const size_t want = round_up(bytes, kArenaAlign);
  std::lock_guard<std::mutex> lock(pool.mu);
  for (int pass = 0; pass < 2; ++pass) {
    for (auto& c : pool.chunks)
      for (auto it = c.free_blocks.begin(); it != c.free_blocks.end(); ++it) {
        if (it->second < want) continue;
        const size_t off = it->first, rest = it->second - want;
        c.free_blocks.erase(it);
        if (rest) c.free_blocks[off + want] = rest;
        return c.base + off;
      }
    if (pass == 1 || pool.closed || pool.total + kPoolChunk > kPoolMax) return nullptr;
    void* base = nullptr;
    bool mapped = true;
    if (cudaHostAlloc(&base, kPoolChunk, cudaHostAllocPortable | cudaHostAllocMapped) != cudaSuccess) {
      cudaGetLastError();
      mapped = false;                                                // (page-locked without a device mapping still serves the copies)
      if (cudaHostAlloc(&base, kPoolChunk, cudaHostAllocPortable) != cudaSuccess) {
        cudaGetLastError();
        pool.closed = true;
        return nullptr;
      }
    }
    PinnedPool::Chunk c;
    c.base = static_cast<unsigned char*>(base); c.bytes = kPoolChunk;
    // kernels may read the piece in place (a bind that the decoding kernel carries out itself) where the device
    // addresses it like the host does -- unified addressing --, which is what makes the address good on every device
    void* dev = nullptr;
    if (!mapped || cudaHostGetDevicePointer(&dev, base, 0) != cudaSuccess) { cudaGetLastError(); dev = nullptr; }
    c.dev_base = dev == base ? static_cast<unsigned char*>(dev) : nullptr;
    c.free_blocks[0] = kPoolChunk;
    pool.chunks.push_back(std::move(c));
    pool.total += kPoolChunk;
  }
  return nullptr;
}

bool tb_pinned_owns(const void* p) {
  PinnedPool& pool = pinned_pool();
  if (!pool.armed.load() || !p) return false;
  std::lock_guard<std::mutex> lock(pool.mu);
  const unsigned char* q = static_cast<const unsigned char*>(p);
  for (auto& c : pool.chunks)
    if (q >= c.base && q < c.base + c.bytes) return true;
  return false;
}

const unsigned char* tb_pinned_device_ptr(const void* p) {
  PinnedPool& pool = pinned_pool();
  if (!pool.armed.load() || !p) return nullptr;
  std::lock_guard<std::mutex> lock(pool.mu);
  const unsigned char* q = static_cast<const unsigned char*>(p);
  for (auto& c : pool.chunks)
    if (q >= c.base && q < c.base + c.bytes) return c.dev_base ? c.dev_base + (q - c.base) : nullptr;
  return nullptr;
}

bool tb_pinned_free(void* p, size_t bytes) {
  PinnedPool& pool = pinned_pool();
  if (!pool.armed.load() || !p) return false;
  std::lock_guard<std::mutex> lock(pool.mu);
  unsigned char* q = static_cast<unsigned char*>(p);
  for (auto& c : pool.chunks) {
    if (q < c.base || q >= c.base + c.bytes) continue;
    size_t off = static_cast<size_t>(q - c.base), n = round_up(bytes, kArenaAlign);
    auto next = c.free_blocks.lower_bound(off);
    if (next != c.free_blocks.begin()) {
      auto prev = std::prev(next);
      if (prev->first + prev->second == off) { off = prev->first; n += prev->second; c.free_blocks.erase(prev); }
    }
    if (next != c.free_blocks.end() && off + n == next->first) { n += next->second; c.free_blocks.erase(next); }
    c.free_blocks[off] = n;
    return true;
  }
  return false;
}

struct tb_batch {
  int device = 0;
  int32_t vocab = 0, n_classes = 0, n_slots = 0, max_beam = 0, max_tree_steps = 0;
  uint64_t class_map_hash = 0;
  unsigned char* arena = nullptr;
  size_t arena_bytes = 0;
  TbSlotRec* d_slots = nullptr;
  TbSlotState* d_sstate = nullptr;
  int32_t* d_cls = nullptr;
  uint32_t flags = 0;
  int32_t* d_status = nullptr;
  int2* d_tree = nullptr;
  unsigned long long* d_hyp_hash = nullptr;   // [2][n_slots * max_beam]: token-sequence hash of every beam hypothesis, ping-pong
  int32_t* d_hyp_len = nullptr;               // [2][n_slots * max_beam]: its length
  int64_t beam_steps = 0;                     // steps since tb_beam_reset (selects the ping-pong half)
  float beam_prune_delta = -1.0f;             // >= 0: prune at frame starts (tb_batch_set_beam_prune)
  int32_t tree_steps = 0, tree_B = 0, tree_K = 0;
  TbTopEnt* d_top = nullptr;                  // rows reduced ahead of a multi-step beam launch (grown on demand)
  size_t d_top_bytes = 0;
  int32_t* d_slot_pos = nullptr;              // [n_slots] steps every slot has taken since its last reset (streaming beam decoding)
  int32_t chunk_K = 0;                        // beam width of the streaming calls since the last reset of all slots (0: none yet)
  ArenaAllocator alloc;
  std::vector<std::pair<size_t, size_t>> slot_block;  // (offset, bytes); bytes == 0: none
  std::vector<int32_t> slot_cache_bytes;               // bytes of the sections the pipelined kernel caches
  std::vector<uint8_t> slot_resolved;                  // the bound graph carries resolved per-state lists (1 for an unbound slot)
  std::vector<int32_t> slot_n_states;
  // models registered ahead of a session (Sec. 2.2 para. 5, decoder-level registration): uploaded once, bound to
  // slots by id without a copy
  struct Model {
    bool live = false;
    size_t off = 0, bytes = 0;
    TbSlotRec rec;
    int32_t n_states = 0, cache_bytes = 0, users = 0;
    uint8_t resolved = 1;
  };
  std::vector<Model> models;
  TbSlotRec* d_model_recs = nullptr;                   // the registered models' records on the device, by model id
  int32_t model_recs_cap = 0;
  std::vector<int32_t> slot_model;                     // registered model a slot is bound to, else -1
  Staging staging[kStagingRing];
  int next_staging = 0;
  void* seg_scratch = nullptr;      // working memory of the two-segment greedy decode (grown on demand)
  size_t seg_scratch_bytes = 0;
  // working memory of the segmented greedy decode: zeroed when allocated and whenever the shape it is laid out for
  // changes; never freed or moved once a stream capture has used it (a captured graph keeps the pointer)
  void* sg_scratch = nullptr;
  size_t sg_scratch_bytes = 0;
  int32_t sg_shape[4] = {0, 0, 0, 0};   // streams, frames, rows per frame, segments of the layout in place
  bool sg_captured = false;
  int32_t plan_G = 0, plan_H = 0, plan_NB = 0;   // tb_batch_set_greedy_plan (0: automatic)
  int32_t last_kernel = 0, last_NB = 0, last_G = 0;
  int32_t n_sm = 0, max_smem = 0;
  int64_t n_pulled_binds = 0, n_copied_binds = 0;   // tb_stream_chunk_binds: binds carried out by the chunk's launch / ahead of it
};

static void destroy_batch(tb_batch* b) {
  if (!b) return;
  cudaDeviceSynchronize();
  cudaFree(b->arena); cudaFree(b->d_slots); cudaFree(b->d_sstate); cudaFree(b->d_cls);
  cudaFree(b->d_status); cudaFree(b->d_tree); cudaFree(b->seg_scratch); cudaFree(b->sg_scratch); cudaFree(b->d_hyp_hash); cudaFree(b->d_hyp_len); cudaFree(b->d_model_recs); cudaFree(b->d_slot_pos); cudaFree(b->d_top);
  for (auto& s : b->staging) {
    if (s.held) tb_graph_free(s.held);
    for (tb_graph* h : s.held_more) tb_graph_free(h);
    if (s.host) cudaFreeHost(s.host);
    if (s.done) cudaEventDestroy(s.done);
  }
  cudaGetLastError();
  delete b;
}

extern "C" int tb_batch_create(int32_t vocab, const int32_t* case_class, int32_t n_slots, int32_t max_beam,
                               int32_t max_tree_steps, size_t arena_bytes, int device, tb_batch** out) {
  if (!out) return TB_ERR_INVALID_ARG;
  *out = nullptr;
  if (vocab < 1 || vocab > TB_MAX_VOCAB || n_slots < 1 || max_beam < 1 || max_beam > TB_MAX_BEAM ||
      max_tree_steps < 0 || arena_bytes == 0)
    return TB_ERR_INVALID_ARG;
  std::vector<int32_t> cls(vocab);
  int32_t n_classes = 0;
  for (int32_t v = 0; v < vocab; ++v) {
    cls[v] = case_class ? case_class[v] : v;
    if (cls[v] < 0) return TB_ERR_INVALID_ARG;
    n_classes = cls[v] + 1 > n_classes ? cls[v] + 1 : n_classes;
  }
  DeviceGuard guard(device);
  if (!guard.ok) return TB_ERR_CUDA;
  tb_batch* b = new (std::nothrow) tb_batch();
  if (!b) return TB_ERR_OOM;
  b->device = device; b->vocab = vocab; b->n_classes = n_classes; b->n_slots = n_slots;
  b->max_beam = max_beam; b->max_tree_steps = max_tree_steps;
  b->class_map_hash = tb_hash_class_map(case_class, vocab);
  b->arena_bytes = round_up(arena_bytes, kArenaAlign);
  b->alloc.init(b->arena_bytes);
  b->slot_block.assign(n_slots, {0, 0});
  b->slot_cache_bytes.assign(n_slots, 0);
  b->slot_resolved.assign(n_slots, 1);
  b->slot_n_states.assign(n_slots, 0);
  b->slot_model.assign(n_slots, -1);
  bool ok = true;
  ok = ok && cudaMalloc(&b->arena, b->arena_bytes) == cudaSuccess;
  ok = ok && cudaMalloc(&b->d_slots, sizeof(TbSlotRec) * n_slots) == cudaSuccess;
  ok = ok && cudaMalloc(&b->d_sstate, sizeof(TbSlotState) * n_slots) == cudaSuccess;
  ok = ok && cudaMalloc(&b->d_cls, sizeof(int32_t) * vocab) == cudaSuccess;
  ok = ok && cudaMalloc(&b->d_status, sizeof(int32_t)) == cudaSuccess;
  if (ok && max_tree_steps > 0)
    ok = cudaMalloc(&b->d_tree, sizeof(int2) * static_cast<size_t>(max_tree_steps) * n_slots * max_beam) == cudaSuccess;
  const size_t n_hyp = static_cast<size_t>(n_slots) * max_beam;
  ok = ok && cudaMalloc(&b->d_hyp_hash, 2 * n_hyp * sizeof(unsigned long long)) == cudaSuccess;
  ok = ok && cudaMalloc(&b->d_hyp_len, 2 * n_hyp * sizeof(int32_t)) == cudaSuccess;
  ok = ok && cudaMalloc(&b->d_slot_pos, static_cast<size_t>(n_slots) * sizeof(int32_t)) == cudaSuccess;
  ok = ok && cudaMemset(b->d_slot_pos, 0, static_cast<size_t>(n_slots) * sizeof(int32_t)) == cudaSuccess;
  if (!ok) { cudaGetLastError(); destroy_batch(b); return TB_ERR_OOM; }
  ok = ok && cudaMemset(b->d_hyp_hash, 0, 2 * n_hyp * sizeof(unsigned long long)) == cudaSuccess;
  ok = ok && cudaMemset(b->d_hyp_len, 0, 2 * n_hyp * sizeof(int32_t)) == cudaSuccess;
  // every slot starts unbound: n_states = 0, streaming state = {-1, 0, 0, 0, 0, 0}
  std::vector<TbSlotState> init(n_slots);
  for (auto& s : init) { std::memset(&s, 0, sizeof s); s.state = -1; }
  ok = ok && cudaMemset(b->d_slots, 0, sizeof(TbSlotRec) * n_slots) == cudaSuccess;
  ok = ok && cudaMemcpy(b->d_sstate, init.data(), sizeof(TbSlotState) * n_slots, cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(b->d_cls, cls.data(), sizeof(int32_t) * vocab, cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemset(b->d_status, 0, sizeof(int32_t)) == cudaSuccess;
  for (auto& s : b->staging) ok = ok && cudaEventCreateWithFlags(&s.done, cudaEventDisableTiming) == cudaSuccess;
  if (!ok) { cudaGetLastError(); destroy_batch(b); return TB_ERR_CUDA; }
  tb_pinned_pool_arm();   // from now on this process keeps the images of the graphs it compiles in page-locked memory
  *out = b;
  return TB_OK;
}

extern "C" void tb_batch_destroy(tb_batch* b) {
  if (!b) return;
  DeviceGuard guard(b->device);
  destroy_batch(b);
}

// The slot record of graph g when its blob sits at byte offset `off` of the arena.
static void fill_record(const tb_graph* g, size_t off, TbSlotRec* rec_out) {
  TbSlotRec& rec = *rec_out;
  std::memset(&rec, 0, sizeof rec);
  rec.blob_off = static_cast<int64_t>(off);
  rec.off_arc_begin = g->off_arc_begin; rec.off_fail = g->off_fail; rec.off_bw = g->off_bw;
  rec.off_arc_cls = g->off_arc_cls; rec.off_arc_w = g->off_arc_w; rec.off_arc_dst = g->off_arc_dst;
  rec.off_strec = g->off_strec; rec.off_tokent = g->off_tokent;
  rec.off_final = g->off_final;
  rec.n_tokent = g->n_tokent; rec.blob_bytes = static_cast<int32_t>(g->blob.size());
  rec.off_rsrec = g->off_rsrec; rec.off_rsent = g->off_rsent; rec.n_rsent = g->n_rsent; rec.d_max = g->d_max;
  rec.n_states = g->n_states; rec.n_arcs = g->n_arcs; rec.max_depth = g->max_depth; rec.lambda = g->lambda;
}

// Copies a graph's blob into a fresh arena block (through the pinned staging ring, on `stream`) and fills the
// slot record that points at it.
static int upload_graph(tb_batch* b, const tb_graph* g, cudaStream_t stream, size_t* off_out, size_t* bytes_out,
                        TbSlotRec* rec_out) {
  if (g->vocab != b->vocab || g->class_map_hash != b->class_map_hash) return TB_ERR_INVALID_ARG;
  size_t off = 0;
  const size_t bytes = round_up(g->blob.size(), kArenaAlign);
  if (!b->alloc.alloc(bytes, &off)) return TB_ERR_ARENA_FULL;
  // pinned staging: wait only if this ring entry's previous copy has not finished yet
  Staging& s = b->staging[b->next_staging];
  b->next_staging = (b->next_staging + 1) % kStagingRing;
  bool ok = true;
  if (s.pending) { ok = cudaEventSynchronize(s.done) == cudaSuccess; s.pending = false; }
  if (s.held) { tb_graph_free(s.held); s.held = nullptr; }
  for (tb_graph* h : s.held_more) tb_graph_free(h);
  s.held_more.clear();
  if (ok && g->pinned) {
    // the blob's pages are locked: the copy engine reads it in place; the graph is held until the copy is done
    ok = cudaMemcpyAsync(b->arena + off, g->blob.data(), g->blob.size(), cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok = ok && cudaEventRecord(s.done, stream) == cudaSuccess;
    if (ok) { s.pending = true; s.held = const_cast<tb_graph*>(g); s.held->refs.fetch_add(1); }
  } else if (ok && s.cap < g->blob.size()) {
    if (s.host) cudaFreeHost(s.host);
    s.host = nullptr; s.cap = 0;
    size_t want = round_up(g->blob.size() * 2, 1 << 16);
    ok = cudaMallocHost(&s.host, want) == cudaSuccess;
    if (ok) s.cap = want;
  }
  if (ok && !g->pinned) {
    std::memcpy(s.host, g->blob.data(), g->blob.size());
    ok = cudaMemcpyAsync(b->arena + off, s.host, g->blob.size(), cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok = ok && cudaEventRecord(s.done, stream) == cudaSuccess;
    s.pending = ok;
  }
  if (!ok) { cudaGetLastError(); b->alloc.release(off, bytes); return TB_ERR_CUDA; }
  fill_record(g, off, rec_out);
  *off_out = off; *bytes_out = bytes;
  return TB_OK;
}

// what the pipelined kernel caches in shared memory: the resolved lists, else the state records + token arcs
static int32_t cache_bytes_of(const tb_graph* g) {
  return static_cast<int32_t>(g->blob.size()) - (g->n_rsent >= 0 ? g->off_rsrec : g->off_strec);
}

// The slot lets go of what it was bound to: its own block goes back to the free list (anything that reuses it is
// enqueued on the same stream after the decode calls that still read it), a registered model loses a user.
static void release_slot(tb_batch* b, int32_t slot) {
  auto& blk = b->slot_block[slot];
  if (blk.second) b->alloc.release(blk.first, blk.second);
  blk = {0, 0};
  const int32_t m = b->slot_model[slot];
  if (m >= 0) b->models[m].users--;
  b->slot_model[slot] = -1;
}

static bool prepare_pulled_binds(tb_batch* b, int32_t n, const int32_t* slots, const tb_graph* const* graphs, cudaStream_t stream,
                                 TbInlineBinds* ib, Staging** used, std::vector<tb_graph*>* let_go);

// Binds of up to TB_INLINE_BINDS graphs whose images lie in the page-locked pool, carried out by one launch that
// reads the images in place (no copy is enqueued; the graphs are held until the launch's event).  False, with nothing
// changed, when the group has to go the ordinary way.
static bool bind_by_pull(tb_batch* b, int32_t n, const int32_t* slots, const tb_graph* const* graphs, cudaStream_t stream) {
  if (b->flags & TB_FLAG_COPIED_BINDS) return false;
  bool any = false;
  for (int32_t i = 0; i < n && graphs; ++i) any = any || graphs[i] != nullptr;
  if (!any) return false;                              // (slots that only lose their graph need no image: the small launch does)
  TbInlineBinds ib;
  Staging* used = nullptr;
  std::vector<tb_graph*> let_go;
  if (!prepare_pulled_binds(b, n, slots, graphs, stream, &ib, &used, &let_go)) return false;
  int rc = tb_launch_pull_binds(ib, b->d_sstate, stream);
  if (rc == TB_OK && cudaEventRecord(used->done, stream) == cudaSuccess) used->pending = true;
  else { cudaGetLastError(); cudaStreamSynchronize(stream); }     // (no event, or no launch: nothing reads the graphs once this returns)
  if (rc != TB_OK) {
    // the launch did not happen: the copies and the small launch do the same job from the same blocks
    bool ok = true;
    for (int32_t i = 0; i < n; ++i)
      if (graphs[i]) ok = ok && cudaMemcpyAsync(b->arena + ib.rec[i].blob_off, graphs[i]->blob.data(), graphs[i]->blob.size(), cudaMemcpyHostToDevice, stream) == cudaSuccess;
    for (int32_t i = 0; i < n; ++i) ok = ok && tb_launch_publish_slot(b->d_slots, b->d_sstate, slots[i], ib.rec[i], stream) == TB_OK;
    if (!ok) cudaGetLastError();
    cudaStreamSynchronize(stream);
  }
  for (tb_graph* h : let_go) tb_graph_free(h);
  return true;
}

extern "C" int tb_batch_bind_stream(tb_batch* b, int32_t slot, const tb_graph* g, void* stream_) {
  TbRange range_("tb_batch_bind_stream");
  if (!b) return TB_ERR_INVALID_ARG;
  if (slot < 0 || slot >= b->n_slots) return TB_ERR_BAD_SLOT;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  DeviceGuard guard(b->device);
  if (!guard.ok) return TB_ERR_CUDA;
  if (g && bind_by_pull(b, 1, &slot, &g, stream)) return TB_OK;
  TbSlotRec rec;
  std::memset(&rec, 0, sizeof rec);
  size_t off = 0, bytes = 0;
  if (g) {
    int rc = upload_graph(b, g, stream, &off, &bytes, &rec);
    if (rc != TB_OK) return rc;
  }
  int rc = tb_launch_publish_slot(b->d_slots, b->d_sstate, slot, rec, stream);
  if (rc != TB_OK) { if (bytes) b->alloc.release(off, bytes); return rc; }
  release_slot(b, slot);
  b->slot_block[slot] = {off, bytes};
  b->slot_n_states[slot] = g ? g->n_states : 0;
  b->slot_cache_bytes[slot] = !g ? 0 : cache_bytes_of(g);
  b->slot_resolved[slot] = (!g || g->n_rsent >= 0) ? 1 : 0;
  return TB_OK;
}

// Several slots at once (the streams that start between two chunks): the graphs go into ONE arena block, packed
// next to each other in one pinned staging block together with their slot records, so that the whole update is one
// host-to-device copy and one small launch, whatever the number of streams.
extern "C" int tb_batch_bind_streams(tb_batch* b, int32_t n, const int32_t* slots, const tb_graph* const* graphs,
                                     void* stream_) {
  TbRange range_("tb_batch_bind_streams");
  if (!b || n < 0 || (n > 0 && (!slots || !graphs))) return TB_ERR_INVALID_ARG;
  if (n == 0) return TB_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  // everything is checked before anything changes
  std::vector<uint8_t> seen(static_cast<size_t>(b->n_slots), 0);
  size_t total = 0;
  int32_t first_part = n;                                             // a group beyond a few MB goes in several parts
  for (int32_t i = 0; i < n; ++i) {
    if (slots[i] < 0 || slots[i] >= b->n_slots) return TB_ERR_BAD_SLOT;
    if (seen[slots[i]]) return TB_ERR_INVALID_ARG;
    seen[slots[i]] = 1;
    const tb_graph* g = graphs[i];
    if (g && (g->vocab != b->vocab || g->class_map_hash != b->class_map_hash)) return TB_ERR_INVALID_ARG;
    if (g && first_part == n) {
      if (total > 0 && total + g->blob.size() > kGroupBytes) first_part = i;
      else total += round_up(g->blob.size(), kArenaAlign);
    }
  }
  if (first_part < n) {
    // (the parts' staging blocks stay small; an error in a later part leaves the earlier parts bound)
    int rc = tb_batch_bind_streams(b, first_part, slots, graphs, stream_);
    if (rc == TB_OK) rc = tb_batch_bind_streams(b, n - first_part, slots + first_part, graphs + first_part, stream_);
    return rc;
  }
  const size_t tail_off = total;                                      // records, then slot indices, behind the graphs
  const size_t tail = round_up(static_cast<size_t>(n) * (sizeof(TbSlotRec) + sizeof(int32_t)), kArenaAlign);
  DeviceGuard guard(b->device);
  if (!guard.ok) return TB_ERR_CUDA;
  // graphs in the page-locked pool: a launch reads their images in place, TB_INLINE_BINDS binds at a time (what is left when a
  // group cannot go that way -- a graph on the heap, no room -- goes the ordinary way below)
  {
    int32_t done = 0;
    while (done < n) {
      const int32_t m = n - done < TB_INLINE_BINDS ? n - done : TB_INLINE_BINDS;
      if (!bind_by_pull(b, m, slots + done, graphs + done, stream)) break;
      done += m;
    }
    if (done == n) return TB_OK;
    if (done > 0) return tb_batch_bind_streams(b, n - done, slots + done, graphs + done, stream_);
  }
  size_t base = 0;
  if (!b->alloc.alloc(total + tail, &base)) {
    // no contiguous room for the group (a fragmented or nearly full arena): one by one, each in the first hole that fits
    for (int32_t i = 0; i < n; ++i) {
      const int rc = tb_batch_bind_stream(b, slots[i], graphs[i], stream_);
      if (rc != TB_OK) return rc;
    }
    return TB_OK;
  }
  Staging& s = b->staging[b->next_staging];
  b->next_staging = (b->next_staging + 1) % kStagingRing;
  bool ok = true;
  if (s.pending) { ok = cudaEventSynchronize(s.done) == cudaSuccess; s.pending = false; }
  // the graphs this entry's last copies read are let go when the call returns: after this call's copies and launch
  // have been issued, not before them
  struct LetGo {
    std::vector<tb_graph*> graphs;
    ~LetGo() { for (tb_graph* h : graphs) tb_graph_free(h); }
  } let_go;
  let_go.graphs.swap(s.held_more);
  if (s.held) { let_go.graphs.push_back(s.held); s.held = nullptr; }
  // graphs whose image is page-locked (those kept by a cache) are copied from where they are; only
  // the others pass through the staging block, which also carries the records
  bool any_pinned = false;
  for (int32_t i = 0; i < n; ++i) any_pinned = any_pinned || (graphs[i] && graphs[i]->pinned);
  if (ok && s.cap < total + tail) {
    if (s.host) cudaFreeHost(s.host);
    s.host = nullptr; s.cap = 0;
    const size_t want = round_up((total + tail) * 2, 1 << 20);
    ok = cudaMallocHost(&s.host, want) == cudaSuccess;
    if (ok) s.cap = want;
  }
  if (!ok) { cudaGetLastError(); b->alloc.release(base, total + tail); return TB_ERR_CUDA; }
  TbSlotRec* recs = reinterpret_cast<TbSlotRec*>(s.host + tail_off);
  int32_t* slot_of = reinterpret_cast<int32_t*>(s.host + tail_off + static_cast<size_t>(n) * sizeof(TbSlotRec));
  std::vector<std::pair<size_t, size_t>> blocks(static_cast<size_t>(n), {0, 0});
  size_t at = 0;
  // page-locked images that lie next to each other in host memory (graphs compiled one after the other sit side by
  // side in the pool, at the spacing the arena uses) travel in one copy
  const unsigned char* run_src = nullptr;
  size_t run_at = 0, run_span = 0, run_bytes = 0;
  auto flush_run = [&]() {
    if (run_src) ok = ok && cudaMemcpyAsync(b->arena + base + run_at, run_src, run_bytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    run_src = nullptr;
  };
  for (int32_t i = 0; i < n; ++i) {
    const tb_graph* g = graphs[i];
    slot_of[i] = slots[i];
    if (!g) { std::memset(&recs[i], 0, sizeof(TbSlotRec)); continue; }
    if (g->pinned) {
      if (!(run_src && !g->registered && g->blob.data() == run_src + run_span && at == run_at + run_span)) {
        flush_run();
        run_src = g->blob.data(); run_at = at; run_span = 0;
      }
      run_bytes = run_span + g->blob.size();
      run_span += round_up(g->blob.size(), kArenaAlign);
      if (g->registered) flush_run();                                  // (registered memory ends with the image)
      tb_graph* h = const_cast<tb_graph*>(g); h->refs.fetch_add(1); s.held_more.push_back(h);
    } else {
      flush_run();
      std::memcpy(s.host + at, g->blob.data(), g->blob.size());
      if (any_pinned)   // (a mixed group: every staged graph is its own copy)
        ok = ok && cudaMemcpyAsync(b->arena + base + at, s.host + at, g->blob.size(), cudaMemcpyHostToDevice, stream) == cudaSuccess;
    }
    fill_record(g, base + at, &recs[i]);
    blocks[i] = {base + at, round_up(g->blob.size(), kArenaAlign)};
    at += blocks[i].second;
  }
  flush_run();
  if (any_pinned) ok = ok && cudaMemcpyAsync(b->arena + base + tail_off, s.host + tail_off, tail, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  else ok = ok && cudaMemcpyAsync(b->arena + base, s.host, total + tail, cudaMemcpyHostToDevice, stream) == cudaSuccess;   // graphs and records in one copy
  ok = ok && cudaEventRecord(s.done, stream) == cudaSuccess;
  s.pending = ok;
  int rc = ok ? tb_launch_publish_slots(b->d_slots, b->d_sstate, n, reinterpret_cast<const TbSlotRec*>(b->arena + base + tail_off),
                                        reinterpret_cast<const int32_t*>(b->arena + base + tail_off + static_cast<size_t>(n) * sizeof(TbSlotRec)),
                                        stream)
              : TB_ERR_CUDA;
  if (rc != TB_OK) { cudaGetLastError(); b->alloc.release(base, total + tail); return rc; }
  // the records' part of the block is free again (whatever reuses it is enqueued after the launch that reads it)
  b->alloc.release(base + tail_off, tail);
  for (int32_t i = 0; i < n; ++i) {
    const tb_graph* g = graphs[i];
    release_slot(b, slots[i]);
    b->slot_block[slots[i]] = blocks[i];
    b->slot_n_states[slots[i]] = g ? g->n_states : 0;
    b->slot_cache_bytes[slots[i]] = !g ? 0 : cache_bytes_of(g);
    b->slot_resolved[slots[i]] = (!g || g->n_rsent >= 0) ? 1 : 0;
  }
  return TB_OK;
}

// A group of binds prepared for the streaming chunk launch that follows to carry out itself (see TbInlineBinds): room in
// the arena, the records, the host's bookkeeping -- no copy, no launch.  Taken when every graph's image sits in the
// page-locked pool at an address the device can read, the group is small enough for the launch's parameters, and the
// stream is not being captured (a captured launch would keep the host addresses).  Returns false, with nothing
// changed, when the group has to go the ordinary way (tb_batch_bind_streams, which also reports what is wrong with it).
// *used: the staging entry that holds the graphs until the launch is done; the caller records its event after the
// launch.  let_go: graphs of that entry's previous use, to be released after the launch has been issued.
static bool prepare_pulled_binds(tb_batch* b, int32_t n, const int32_t* slots, const tb_graph* const* graphs, cudaStream_t stream,
                                 TbInlineBinds* ib, Staging** used, std::vector<tb_graph*>* let_go) {
  if (n < 1 || n > TB_INLINE_BINDS || !slots || !graphs) return false;
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess) { cudaGetLastError(); return false; }
  if (cap != cudaStreamCaptureStatusNone) return false;
  size_t total = 0;
  for (int32_t i = 0; i < n; ++i) {
    if (slots[i] < 0 || slots[i] >= b->n_slots) return false;
    for (int32_t j = 0; j < i; ++j)
      if (slots[j] == slots[i]) return false;
    const tb_graph* g = graphs[i];
    ib->slot[i] = slots[i]; ib->src[i] = nullptr; ib->bytes[i] = 0;
    if (!g) continue;
    if (g->vocab != b->vocab || g->class_map_hash != b->class_map_hash) return false;
    if (!g->pinned || g->registered || g->blob.size() > static_cast<size_t>(INT32_MAX)) return false;
    ib->src[i] = tb_pinned_device_ptr(g->blob.data());
    if (!ib->src[i]) return false;
    ib->bytes[i] = static_cast<int32_t>(g->blob.size());
    total += round_up(g->blob.size(), kArenaAlign);
  }
  size_t base = 0;
  if (total > 0 && !b->alloc.alloc(total, &base)) return false;
  Staging& s = b->staging[b->next_staging];
  b->next_staging = (b->next_staging + 1) % kStagingRing;
  if (s.pending) {
    if (cudaEventSynchronize(s.done) != cudaSuccess) { cudaGetLastError(); if (total) b->alloc.release(base, total); return false; }
    s.pending = false;
  }
  let_go->swap(s.held_more);
  if (s.held) { let_go->push_back(s.held); s.held = nullptr; }
  size_t at = 0;
  for (int32_t i = 0; i < n; ++i) {
    const tb_graph* g = graphs[i];
    std::pair<size_t, size_t> block{0, 0};
    if (g) {
      fill_record(g, base + at, &ib->rec[i]);
      block = {base + at, round_up(g->blob.size(), kArenaAlign)};
      at += block.second;
      tb_graph* h = const_cast<tb_graph*>(g); h->refs.fetch_add(1); s.held_more.push_back(h);
    } else {
      std::memset(&ib->rec[i], 0, sizeof(TbSlotRec));
    }
    release_slot(b, slots[i]);                       // (after the group's room was taken: the new blocks are none of the old)
    b->slot_block[slots[i]] = block;
    b->slot_n_states[slots[i]] = g ? g->n_states : 0;
    b->slot_cache_bytes[slots[i]] = !g ? 0 : cache_bytes_of(g);
    b->slot_resolved[slots[i]] = (!g || g->n_rsent >= 0) ? 1 : 0;
  }
  ib->n = n; ib->arena = b->arena; ib->slots = b->d_slots;
  *used = &s;
  return true;
}

extern "C" int tb_batch_register_model(tb_batch* b, const tb_graph* g, int32_t* out_model_id, void* stream_) {
  TbRange range_("tb_batch_register_model");
  if (!b || !g || !out_model_id) return TB_ERR_INVALID_ARG;
  *out_model_id = -1;
  DeviceGuard guard(b->device);
  if (!guard.ok) return TB_ERR_CUDA;
  tb_batch::Model m;
  int rc;
  rc = upload_graph(b, g, static_cast<cudaStream_t>(stream_), &m.off, &m.bytes, &m.rec);
  if (rc != TB_OK) return rc;
  m.live = true; m.n_states = g->n_states; m.cache_bytes = cache_bytes_of(g); m.resolved = g->n_rsent >= 0 ? 1 : 0;
  int32_t id = -1;
  for (size_t i = 0; i < b->models.size(); ++i)
    if (!b->models[i].live) { id = static_cast<int32_t>(i); break; }
  try {
    if (id < 0) { b->models.emplace_back(); id = static_cast<int32_t>(b->models.size()) - 1; }
  } catch (const std::bad_alloc&) {
    b->alloc.release(m.off, m.bytes);
    return TB_ERR_OOM;
  }
  // the record also goes into the device table that tb_batch_bind_models reads (grown in powers of two; the old
  // table is freed after a device-wide wait inside cudaFree, registration is not on the decoding loop)
  if (id >= b->model_recs_cap) {
    int32_t cap = b->model_recs_cap ? b->model_recs_cap : 256;
    while (cap <= id) cap *= 2;
    TbSlotRec* bigger = nullptr;
    bool ok = cudaMalloc(&bigger, sizeof(TbSlotRec) * cap) == cudaSuccess;
    ok = ok && cudaMemset(bigger, 0, sizeof(TbSlotRec) * cap) == cudaSuccess;
    // records published on `stream` by earlier registrations must have landed before the table is copied (the
    // caller's stream does not synchronise with the legacy stream the copy below runs on)
    ok = ok && cudaStreamSynchronize(static_cast<cudaStream_t>(stream_)) == cudaSuccess;
    if (ok && b->model_recs_cap)
      ok = cudaMemcpy(bigger, b->d_model_recs, sizeof(TbSlotRec) * b->model_recs_cap, cudaMemcpyDeviceToDevice) == cudaSuccess;
    if (!ok) { cudaGetLastError(); cudaFree(bigger); b->alloc.release(m.off, m.bytes); return TB_ERR_OOM; }
    cudaFree(b->d_model_recs);
    b->d_model_recs = bigger; b->model_recs_cap = cap;
  }
  rc = tb_launch_publish_model(b->d_model_recs, id, m.rec, static_cast<cudaStream_t>(stream_));
  if (rc != TB_OK) { b->alloc.release(m.off, m.bytes); return rc; }
  b->models[id] = m;
  *out_model_id = id;
  return TB_OK;
}

extern "C" int tb_batch_bind_models(tb_batch* b, int32_t n, const int32_t* slots, const int32_t* model_ids, void* stream_) {
  TbRange range_("tb_batch_bind_models");
  if (!b || n < 0 || (n > 0 && (!slots || !model_ids))) return TB_ERR_INVALID_ARG;
  // everything is checked before anything is changed
  std::vector<uint8_t> seen(static_cast<size_t>(b->n_slots), 0);
  for (int32_t i = 0; i < n; ++i) {
    if (slots[i] < 0 || slots[i] >= b->n_slots) return TB_ERR_BAD_SLOT;
    if (seen[slots[i]]) return TB_ERR_INVALID_ARG;           // a slot twice in one call
    seen[slots[i]] = 1;
    const int32_t m = model_ids[i];
    if (m < -1 || m >= static_cast<int32_t>(b->models.size()) || (m >= 0 && !b->models[m].live)) return TB_ERR_INVALID_ARG;
  }
  DeviceGuard guard(b->device);
  if (!guard.ok) return TB_ERR_CUDA;
  for (int32_t i0 = 0; i0 < n; i0 += TB_BIND_PAIRS) {
    const int32_t cnt = n - i0 < TB_BIND_PAIRS ? n - i0 : TB_BIND_PAIRS;
    int rc = tb_launch_bind_models(b->d_slots, b->d_sstate, b->d_model_recs, cnt, slots + i0, model_ids + i0,
                                   static_cast<cudaStream_t>(stream_));
    if (rc != TB_OK) return rc;
    for (int32_t i = i0; i < i0 + cnt; ++i) {
      const int32_t slot = slots[i], m = model_ids[i];
      release_slot(b, slot);
      if (m >= 0) {
        b->models[m].users++;
        b->slot_model[slot] = m;
        b->slot_n_states[slot] = b->models[m].n_states; b->slot_cache_bytes[slot] = b->models[m].cache_bytes;
        b->slot_resolved[slot] = b->models[m].resolved;
      } else {
        b->slot_n_states[slot] = 0; b->slot_cache_bytes[slot] = 0; b->slot_resolved[slot] = 1;
      }
    }
  }
  return TB_OK;
}

extern "C" int tb_batch_bind_model(tb_batch* b, int32_t slot, int32_t model_id, void* stream_) {
  if (!b) return TB_ERR_INVALID_ARG;
  if (slot < 0 || slot >= b->n_slots) return TB_ERR_BAD_SLOT;
  if (model_id < -1 || model_id >= static_cast<int32_t>(b->models.size()) || (model_id >= 0 && !b->models[model_id].live))
    return TB_ERR_INVALID_ARG;
  DeviceGuard guard(b->device);
  if (!guard.ok) return TB_ERR_CUDA;
  TbSlotRec rec;
  std::memset(&rec, 0, sizeof rec);
  if (model_id >= 0) rec = b->models[model_id].rec;
  int rc = tb_launch_publish_slot(b->d_slots, b->d_sstate, slot, rec, static_cast<cudaStream_t>(stream_));
  if (rc != TB_OK) return rc;
  release_slot(b, slot);
  if (model_id >= 0) {
    const tb_batch::Model& m = b->models[model_id];
    b->models[model_id].users++;
    b->slot_model[slot] = model_id;
    b->slot_n_states[slot] = m.n_states; b->slot_cache_bytes[slot] = m.cache_bytes; b->slot_resolved[slot] = m.resolved;
  } else {
    b->slot_n_states[slot] = 0; b->slot_cache_bytes[slot] = 0; b->slot_resolved[slot] = 1;
  }
  return TB_OK;
}

extern "C" int tb_batch_unregister_model(tb_batch* b, int32_t model_id) {
  if (!b || model_id < 0 || model_id >= static_cast<int32_t>(b->models.size()) || !b->models[model_id].live)
    return TB_ERR_INVALID_ARG;
  tb_batch::Model& m = b->models[model_id];
  if (m.users > 0) return TB_ERR_INVALID_ARG;          // still bound to a slot
  b->alloc.release(m.off, m.bytes);
  m = tb_batch::Model();
  return TB_OK;
}

extern "C" int tb_batch_status(tb_batch* b, int32_t* device_status, void* stream_) {
  if (!b || !device_status) return TB_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  DeviceGuard guard(b->device);
  if (!guard.ok) return TB_ERR_CUDA;
  int32_t st = 0;
  bool ok = cudaMemcpyAsync(&st, b->d_status, sizeof st, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
  ok = ok && cudaMemsetAsync(b->d_status, 0, sizeof st, stream) == cudaSuccess;
  ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
  if (!ok) { cudaGetLastError(); return TB_ERR_CUDA; }
  *device_status = st;
  return st == 0 ? TB_OK : TB_ERR_DEVICE_STATUS;
}

static int fill_decode_params(tb_batch* b, const void* logits, int dtype, int32_t n, int32_t frames, int32_t S,
                              int32_t n_dur, const int64_t* strides, TbDecodeParams* p) {
  if (!b || !logits || !strides || (dtype != TB_BF16 && dtype != TB_F32)) return TB_ERR_INVALID_ARG;
  if (n < 1 || n > b->n_slots || frames < 1 || S < 1 || n_dur < 0 || n_dur > 32) return TB_ERR_INVALID_ARG;
  if (static_cast<int64_t>(frames) * S > INT32_MAX) return TB_ERR_INVALID_ARG;
  std::memset(p, 0, sizeof *p);
  p->logits = logits; p->dtype = dtype; p->n_streams = n; p->frames = frames; p->S = S; p->V = b->vocab;
  p->n_dur = n_dur; p->C = b->n_classes;
  p->sb = strides[0]; p->st = strides[1]; p->ss = strides[2]; p->sv = strides[3];
  p->out_cap = frames * S;
  p->slots = b->d_slots; p->sstate = b->d_sstate; p->arena = b->arena; p->cls = b->d_cls; p->status = b->d_status;
  return TB_OK;
}

extern "C" int tb_greedy_decode(tb_batch* b, const void* logits, int dtype, int32_t B, int32_t T, int32_t S,
                                const int64_t* strides, const int32_t* lengths, int32_t* out_tokens,
                                int32_t* out_frames, int32_t* out_counts, float* out_scores, int32_t* out_states,
                                void* stream_) {
  TbRange range_("tb_greedy_decode");
  TbDecodeParams p;
  int rc = fill_decode_params(b, logits, dtype, B, T, S, 0, strides, &p);
  if (rc != TB_OK) return rc;
  if (!out_tokens || !out_frames || !out_counts || !out_scores || !out_states) return TB_ERR_INVALID_ARG;
  p.lengths = lengths; p.persistent = 0;
  p.out_tokens = out_tokens; p.out_frames = out_frames; p.out_counts = out_counts;
  p.out_scores = out_scores; p.out_states = out_states;
  DeviceGuard guard(b->device);
  if (!guard.ok) return TB_ERR_CUDA;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  p.normalize = (b->flags & TB_FLAG_LOG_SOFTMAX) ? 1 : 0;
  if (!(b->flags & TB_FLAG_GENERAL_KERNELS)) {
    int32_t max_cache = 0, max_states = 0, all_resolved = 1;
    for (int32_t i = 0; i < B; ++i) {
      max_cache = b->slot_cache_bytes[i] > max_cache ? b->slot_cache_bytes[i] : max_cache;
      max_states = b->slot_n_states[i] > max_states ? b->slot_n_states[i] : max_states;
      if (!b->slot_resolved[i]) all_resolved = 0;
    }
    // Working memory is never allocated while the caller's stream is being captured into a graph (allocation is
    // not allowed there): the decode then runs with the block it has, or on a path that needs none.
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess) { cudaGetLastError(); cap = cudaStreamCaptureStatusNone; }
    const bool capturing = cap != cudaStreamCaptureStatusNone;
    if (!(b->flags & TB_FLAG_ONE_BLOCK_PER_STREAM)) {
      if (b->n_sm == 0) {
        cudaDeviceGetAttribute(&b->n_sm, cudaDevAttrMultiProcessorCount, b->device);
        cudaDeviceGetAttribute(&b->max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, b->device);
        cudaGetLastError();
      }
      TbSegPlan plan;
      plan.force_G = b->plan_G; plan.force_H = b->plan_H; plan.force_NB = b->plan_NB;
      plan.test_timeout = (b->flags & TB_FLAG_TEST_WAIT_TIMEOUT) ? 1 : 0;
      if (plan.test_timeout && plan.force_G == 0) { plan.force_G = 2; plan.force_H = 8; }   // the self-test always takes this kernel
      if (b->n_sm > 0 && tb_greedy_seg_plan(p, max_cache, all_resolved, b->n_sm, b->max_smem, &plan)) {
        const int32_t nseg = plan.NB * plan.G;
        const size_t want = tb_greedy_seg_scratch_bytes(B, T, S, nseg);
        bool ok = true;
        if (want > b->sg_scratch_bytes) {
          ok = !capturing && !b->sg_captured && want <= (static_cast<size_t>(4) << 30);
          if (ok) {
            cudaFree(b->sg_scratch);                    // (waits for earlier work: one decode per batch at a time)
            b->sg_scratch = nullptr; b->sg_scratch_bytes = 0; b->sg_shape[0] = 0;
            if (cudaMalloc(&b->sg_scratch, want) == cudaSuccess) b->sg_scratch_bytes = want;
            else { cudaGetLastError(); ok = false; }
          }
        }
        if (ok && (b->sg_shape[0] != B || b->sg_shape[1] != T || b->sg_shape[2] != S || b->sg_shape[3] != nseg)) {
          // another layout: what the last one left (launch numbers, records) would be misread
          if (cudaMemsetAsync(b->sg_scratch, 0, want, stream) != cudaSuccess) { cudaGetLastError(); ok = false; }
          else { b->sg_shape[0] = B; b->sg_shape[1] = T; b->sg_shape[2] = S; b->sg_shape[3] = nseg; }
        }
        if (ok) {
          if (capturing) b->sg_captured = true;
          rc = tb_launch_greedy_seg(p, max_cache, plan, b->sg_scratch, stream);
          if (rc == TB_OK) { b->last_kernel = TB_KERNEL_SEGMENTED; b->last_NB = plan.NB; b->last_G = plan.G; }
          return rc;
        }
      }
    }
    // the two-segment decode keeps what its second segment produces in scratch memory of the batch; growing it
    // frees the old block first (cudaFree waits for earlier work), so one decode per batch at a time
    const size_t want = tb_greedy_fast_scratch_bytes(B, T, S);
    if (!capturing && want > b->seg_scratch_bytes && want <= (static_cast<size_t>(1) << 30)) {
      cudaFree(b->seg_scratch);
      b->seg_scratch = nullptr; b->seg_scratch_bytes = 0;
      if (cudaMalloc(&b->seg_scratch, want) == cudaSuccess) b->seg_scratch_bytes = want;
      else cudaGetLastError();
    }
    rc = tb_launch_greedy_fast(p, max_cache, max_states, all_resolved, b->seg_scratch, b->seg_scratch_bytes, stream);
    if (rc == TB_OK) { b->last_kernel = TB_KERNEL_PIPELINED; b->last_NB = 1; b->last_G = 0; }
    if (rc != 1) return rc;
  }
  rc = tb_launch_decode_general(p, stream);
  if (rc == TB_OK) { b->last_kernel = TB_KERNEL_GENERAL; b->last_NB = 1; b->last_G = 0; }
  return rc;
}

extern "C" int tb_batch_set_greedy_plan(tb_batch* b, int32_t deciders_per_block, int32_t helpers_per_block,
                                        int32_t blocks_per_stream) {
  if (!b || deciders_per_block < 0 || helpers_per_block < 0 || blocks_per_stream < 0) return TB_ERR_INVALID_ARG;
  if ((deciders_per_block == 0) != (helpers_per_block == 0)) return TB_ERR_INVALID_ARG;
  if (deciders_per_block > 4 || (deciders_per_block + helpers_per_block) > 20) return TB_ERR_INVALID_ARG;
  b->plan_G = deciders_per_block; b->plan_H = helpers_per_block; b->plan_NB = blocks_per_stream;
  return TB_OK;
}

extern "C" int tb_batch_last_greedy_kernel(const tb_batch* b, int32_t* kernel, int32_t* blocks_per_stream,
                                           int32_t* deciders_per_block) {
  if (!b) return TB_ERR_INVALID_ARG;
  if (kernel) *kernel = b->last_kernel;
  if (blocks_per_stream) *blocks_per_stream = b->last_NB;
  if (deciders_per_block) *deciders_per_block = b->last_G;
  return TB_OK;
}

extern "C" int tb_batch_set_beam_prune(tb_batch* b, float delta) {
  if (!b || delta != delta) return TB_ERR_INVALID_ARG;
  b->beam_prune_delta = delta >= 0.0f ? delta : -1.0f;
  return TB_OK;
}

extern "C" int tb_apply_final_weights(tb_batch* b, int32_t B, int32_t K, float* scores, const int32_t* states,
                                      void* stream_) {
  if (!b || !scores || !states || B < 1 || B > b->n_slots || K < 1) return TB_ERR_INVALID_ARG;
  DeviceGuard guard(b->device);
  if (!guard.ok) return TB_ERR_CUDA;
  return tb_launch_final_weights(b->d_slots, b->arena, B, K, scores, states, b->d_status, static_cast<cudaStream_t>(stream_));
}

extern "C" int tb_batch_set_flags(tb_batch* b, uint32_t flags) {
  if (!b || (flags & ~static_cast<uint32_t>(TB_FLAG_GENERAL_KERNELS | TB_FLAG_ONE_BLOCK_PER_STREAM | TB_FLAG_TEST_WAIT_TIMEOUT | TB_FLAG_LOG_SOFTMAX |
                                              TB_FLAG_BEAM_WHOLE_ROWS | TB_FLAG_COPIED_BINDS))) return TB_ERR_INVALID_ARG;
  b->flags = flags;
  return TB_OK;
}

static int stream_chunk_params(tb_batch* b, const void* logits, int dtype, int32_t n_slots, int32_t chunk, int32_t S, int32_t n_dur,
                               const int64_t* strides, const int32_t* valid_frames, int32_t* out_tokens, int32_t* out_frames,
                               int32_t* out_durs, int32_t* out_counts, float* out_scores, int32_t* out_states,
                               int32_t* out_cursors, TbDecodeParams* p) {
  int rc = fill_decode_params(b, logits, dtype, n_slots, chunk, S, n_dur, strides, p);
  if (rc != TB_OK) return rc;
  if (!valid_frames || !out_tokens || !out_frames || !out_counts || !out_scores || !out_states) return TB_ERR_INVALID_ARG;
  p->lengths = valid_frames; p->persistent = 1;
  p->normalize = (b->flags & TB_FLAG_LOG_SOFTMAX) ? 1 : 0;
  if (p->normalize && n_dur != 0) return TB_ERR_INVALID_ARG;   // normalisation is defined for the token logits of an RNNT row
  p->out_tokens = out_tokens; p->out_frames = out_frames; p->out_durs = out_durs; p->out_counts = out_counts;
  p->out_scores = out_scores; p->out_states = out_states; p->out_cursors = out_cursors;
  return TB_OK;
}

extern "C" int tb_stream_chunk(tb_batch* b, const void* logits, int dtype, int32_t n_slots, int32_t chunk,
                               int32_t S, int32_t n_dur, const int64_t* strides, const int32_t* valid_frames,
                               int32_t* out_tokens, int32_t* out_frames, int32_t* out_durs, int32_t* out_counts,
                               float* out_scores, int32_t* out_states, int32_t* out_cursors, void* stream_) {
  TbRange range_("tb_stream_chunk");
  TbDecodeParams p;
  const int rc = stream_chunk_params(b, logits, dtype, n_slots, chunk, S, n_dur, strides, valid_frames, out_tokens, out_frames,
                                     out_durs, out_counts, out_scores, out_states, out_cursors, &p);
  if (rc != TB_OK) return rc;
  DeviceGuard guard(b->device);
  if (!guard.ok) return TB_ERR_CUDA;
  return tb_launch_decode_general(p, static_cast<cudaStream_t>(stream_));
}

extern "C" int tb_stream_chunk_binds(tb_batch* b, int32_t n_binds, const int32_t* bind_slots, const tb_graph* const* bind_graphs,
                                     const void* logits, int dtype, int32_t n_slots, int32_t chunk, int32_t S, int32_t n_dur,
                                     const int64_t* strides, const int32_t* valid_frames, int32_t* out_tokens,
                                     int32_t* out_frames, int32_t* out_durs, int32_t* out_counts, float* out_scores,
                                     int32_t* out_states, int32_t* out_cursors, void* stream_) {
  TbRange range_("tb_stream_chunk_binds");
  if (!b || n_binds < 0) return TB_ERR_INVALID_ARG;
  // the chunk's arguments are checked before any bind changes anything
  TbDecodeParams p;
  int rc = stream_chunk_params(b, logits, dtype, n_slots, chunk, S, n_dur, strides, valid_frames, out_tokens, out_frames,
                               out_durs, out_counts, out_scores, out_states, out_cursors, &p);
  if (rc != TB_OK) return rc;
  DeviceGuard guard(b->device);
  if (!guard.ok) return TB_ERR_CUDA;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (n_binds > 0) {
    // every bound slot must be one the chunk decodes, or its bind could not ride on the chunk's launch
    bool in_chunk = true;
    for (int32_t i = 0; i < n_binds && bind_slots; ++i) in_chunk = in_chunk && bind_slots[i] < n_slots;
    TbInlineBinds ib;
    Staging* used = nullptr;
    std::vector<tb_graph*> let_go;
    if (in_chunk && !(b->flags & TB_FLAG_COPIED_BINDS) &&
        prepare_pulled_binds(b, n_binds, bind_slots, bind_graphs, stream, &ib, &used, &let_go)) {
      rc = tb_launch_decode_general(p, stream, &ib);
      if (rc == TB_OK && cudaEventRecord(used->done, stream) == cudaSuccess) used->pending = true;
      else if (rc == TB_OK) { cudaGetLastError(); cudaStreamSynchronize(stream); }   // (no event: the graphs are let go only after the launch is done)
      if (rc != TB_OK) {
        // the launch did not happen: the slots it would have bound are left unbound, on both sides
        for (int32_t i = 0; i < n_binds; ++i) {
          release_slot(b, bind_slots[i]);
          b->slot_n_states[bind_slots[i]] = 0; b->slot_cache_bytes[bind_slots[i]] = 0; b->slot_resolved[bind_slots[i]] = 1;
          cudaMemsetAsync(b->d_slots + bind_slots[i], 0, sizeof(TbSlotRec), stream);
        }
        cudaGetLastError();
      } else {
        b->n_pulled_binds += n_binds;
      }
      for (tb_graph* h : let_go) tb_graph_free(h);
      return rc;
    }
    rc = tb_batch_bind_streams(b, n_binds, bind_slots, bind_graphs, stream_);
    if (rc != TB_OK) return rc;
    b->n_copied_binds += n_binds;
  }
  return tb_launch_decode_general(p, stream);
}

extern "C" int tb_batch_bind_counts(const tb_batch* b, int64_t* out_pulled, int64_t* out_copied) {
  if (!b || !out_pulled || !out_copied) return TB_ERR_INVALID_ARG;
  *out_pulled = b->n_pulled_binds; *out_copied = b->n_copied_binds;
  return TB_OK;
}

// The beam pre-pass for a launch that covers T * E rows per stream: reduces every row to its few best root-boosted
// tokens (tb_launch_beam_topm) into memory of the batch and points the step parameters at the result.  Skipped (the
// steps then look at whole rows) when the batch asks for it, when the memory would have to grow while the stream is
// being captured, or when it cannot be had.
static void beam_prepass(tb_batch* b, TbBeamParams* p, int32_t T, int32_t E, int64_t frame_stride, int64_t row_stride,
                         const int32_t* n_frames, cudaStream_t stream) {
  p->top_base = nullptr; p->top_row = nullptr; p->top_m = 0;
  if (b->flags & (TB_FLAG_GENERAL_KERNELS | TB_FLAG_BEAM_WHOLE_ROWS)) return;
  if (2 * (b->vocab + 1) > (1 << TB_RS_TOK_BITS) || b->vocab > 0xFFFE) return;   // (the steps' token view has the same limit)
  const int32_t M = 2 * p->K + 8;
  const size_t want = static_cast<size_t>(p->B) * T * E * (M + 1) * sizeof(TbTopEnt);
  if (want > b->d_top_bytes) {
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess) { cudaGetLastError(); return; }
    if (cap != cudaStreamCaptureStatusNone || want > (static_cast<size_t>(2) << 30)) return;
    cudaFree(b->d_top);
    b->d_top = nullptr; b->d_top_bytes = 0;
    if (cudaMalloc(&b->d_top, want) != cudaSuccess) { cudaGetLastError(); return; }
    b->d_top_bytes = want;
  }
  if (tb_launch_beam_topm(p->logits, p->dtype, p->B, T, E, p->V, p->C, p->stream_stride, frame_stride, row_stride, n_frames,
                          b->d_slots, b->arena, b->d_cls, M, b->d_top, stream) != TB_OK)
    return;
  p->top_base = b->d_top; p->top_m = M;
}

extern "C" int tb_beam_reset(tb_batch* b) {
  if (!b) return TB_ERR_INVALID_ARG;
  b->tree_steps = 0; b->tree_B = 0; b->tree_K = 0;
  b->chunk_K = 0;   // (a streaming session, if one was under way, is over: its per-slot trees are reused by the batch-wide one)
  // every hypothesis starts from the empty token sequence: the first step after this ignores the stored records
  b->beam_steps = 0;
  return TB_OK;
}

extern "C" int tb_beam_step(tb_batch* b, const void* logits, int dtype, int32_t B, int32_t K, int64_t stream_stride,
                            int64_t hyp_stride, int32_t new_frame, float* scores, int32_t* states, uint8_t* live,
                            int32_t* out_parent, int32_t* out_token, void* stream_) {
  TbRange range_("tb_beam_step");
  if (!b || !logits || !scores || !states || !live || !out_parent || !out_token) return TB_ERR_INVALID_ARG;
  if ((dtype != TB_BF16 && dtype != TB_F32) || B < 1 || B > b->n_slots || K < 1 || K > b->max_beam) return TB_ERR_INVALID_ARG;
  if (b->chunk_K != 0) return TB_ERR_INVALID_ARG;   // a streaming session is under way: tb_beam_reset ends it
  if (b->d_tree) {
    if (b->tree_steps >= b->max_tree_steps) return TB_ERR_INVALID_ARG;
    if (b->tree_steps > 0 && (b->tree_B != B || b->tree_K != K)) return TB_ERR_INVALID_ARG;
  }
  TbBeamParams p;
  std::memset(&p, 0, sizeof p);
  p.logits = logits; p.dtype = dtype; p.B = B; p.K = K; p.V = b->vocab; p.C = b->n_classes;
  if (new_frame < 0 || new_frame > TB_FRAME_NEW_MERGE) return TB_ERR_INVALID_ARG;
  {
    const size_t n_hyp = static_cast<size_t>(b->n_slots) * b->max_beam;
    const size_t in = (b->beam_steps & 1) ? n_hyp : 0, out = (b->beam_steps & 1) ? 0 : n_hyp;
    p.hash_in = b->d_hyp_hash + in; p.hash_out = b->d_hyp_hash + out;
    p.len_in = b->d_hyp_len + in; p.len_out = b->d_hyp_len + out;
    p.merge = new_frame == TB_FRAME_NEW_MERGE ? 1 : 0;
    p.fresh = b->beam_steps == 0 ? 1 : 0;
    p.prune_delta = new_frame != 0 ? b->beam_prune_delta : -1.0f;
  }
  p.new_frame = new_frame != 0; p.step = b->tree_steps; p.stream_stride = stream_stride; p.hyp_stride = hyp_stride;
  p.scores = scores; p.states = states; p.live = live; p.out_parent = out_parent; p.out_token = out_token;
  p.tree = b->d_tree; p.slots = b->d_slots; p.arena = b->arena; p.cls = b->d_cls; p.status = b->d_status;
  DeviceGuard guard(b->device);
  if (!guard.ok) return TB_ERR_CUDA;
  int rc = tb_launch_beam_step(p, static_cast<cudaStream_t>(stream_));
  if (rc == TB_OK) b->beam_steps++;
  if (rc == TB_OK && b->d_tree) { b->tree_steps++; b->tree_B = B; b->tree_K = K; }
  return rc;
}

extern "C" int tb_beam_frames(tb_batch* b, const void* logits, int dtype, int32_t B, int32_t K, int32_t T, int32_t E,
                              int64_t stream_stride, int64_t frame_stride, int64_t row_stride, int32_t merge,
                              float* scores, int32_t* states, uint8_t* live, int32_t* out_parent, int32_t* out_token,
                              void* stream_) {
  TbRange range_("tb_beam_frames");
  if (!b || !logits || !scores || !states || !live || !out_parent || !out_token) return TB_ERR_INVALID_ARG;
  if ((dtype != TB_BF16 && dtype != TB_F32) || B < 1 || B > b->n_slots || K < 1 || K > b->max_beam || T < 1 || E < 1 ||
      static_cast<int64_t>(T) * E > (1 << 24))
    return TB_ERR_INVALID_ARG;
  const int32_t n_steps = T * E;
  if (b->chunk_K != 0) return TB_ERR_INVALID_ARG;   // a streaming session is under way: tb_beam_reset ends it
  if (b->d_tree) {
    if (b->tree_steps + n_steps > b->max_tree_steps) return TB_ERR_INVALID_ARG;
    if (b->tree_steps > 0 && (b->tree_B != B || b->tree_K != K)) return TB_ERR_INVALID_ARG;
  }
  TbBeamParams p;
  std::memset(&p, 0, sizeof p);
  p.logits = logits; p.dtype = dtype; p.B = B; p.K = K; p.V = b->vocab; p.C = b->n_classes;
  {
    const size_t n_hyp = static_cast<size_t>(b->n_slots) * b->max_beam;
    const size_t in = (b->beam_steps & 1) ? n_hyp : 0, out = (b->beam_steps & 1) ? 0 : n_hyp;
    p.hash_in = b->d_hyp_hash + in; p.hash_out = b->d_hyp_hash + out;
    p.len_in = b->d_hyp_len + in; p.len_out = b->d_hyp_len + out;
    p.merge = merge ? 1 : 0;
    p.fresh = b->beam_steps == 0 ? 1 : 0;
    p.prune_delta = b->beam_prune_delta;
  }
  p.new_frame = 1; p.step = b->tree_steps; p.stream_stride = stream_stride; p.hyp_stride = 0;
  p.scores = scores; p.states = states; p.live = live; p.out_parent = out_parent; p.out_token = out_token;
  p.tree = b->d_tree; p.slots = b->d_slots; p.arena = b->arena; p.cls = b->d_cls; p.status = b->d_status;
  DeviceGuard guard(b->device);
  if (!guard.ok) return TB_ERR_CUDA;
  beam_prepass(b, &p, T, E, frame_stride, row_stride, nullptr, static_cast<cudaStream_t>(stream_));
  int rc = tb_launch_beam_frames(p, T, E, frame_stride, row_stride, static_cast<cudaStream_t>(stream_));
  if (rc == TB_OK) b->beam_steps += n_steps;
  if (rc == TB_OK && b->d_tree) { b->tree_steps += n_steps; b->tree_B = B; b->tree_K = K; }
  return rc;
}

// ---- streaming beam decoding, slot by slot (Sec. 2.3) --------------------------------------------------------

// tb_beam_reset_slots, and tb_beam_start_slots (which also sets up the slots' rows of the caller's arrays).
static int beam_reset_slots(tb_batch* b, int32_t n, const int32_t* slots, int32_t K, float* scores, int32_t* states,
                            uint8_t* live, void* stream_) {
  if (!b || n < 0 || (n > 0 && !slots)) return TB_ERR_INVALID_ARG;
  for (int32_t i = 0; i < n; ++i) if (slots[i] < 0 || slots[i] >= b->n_slots) return TB_ERR_BAD_SLOT;
  DeviceGuard guard(b->device);
  if (!guard.ok) return TB_ERR_CUDA;
  const size_t n_hyp = static_cast<size_t>(b->n_slots) * b->max_beam;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (n == 0) {   // every slot
    b->chunk_K = 0;
    return tb_launch_beam_reset_slots(b->d_slot_pos, b->d_hyp_hash, b->d_hyp_len, n_hyp, b->max_beam, b->n_slots, nullptr, 1,
                                      b->d_slots, K, scores, states, live, stream);   // (every record of both halves, whatever the width)
  }
  for (int32_t at = 0; at < n; at += TB_BIND_PAIRS) {
    const int32_t m = n - at < TB_BIND_PAIRS ? n - at : TB_BIND_PAIRS;
    // a slot's records sit at slot * (the session's beam width): the width of the chunks so far, else the one given
    const int32_t stride = b->chunk_K > 0 ? b->chunk_K : (K > 0 ? K : b->max_beam);
    const int rc = tb_launch_beam_reset_slots(b->d_slot_pos, b->d_hyp_hash, b->d_hyp_len, n_hyp, stride, m, slots + at, 0,
                                              b->d_slots, K, scores, states, live, stream);
    if (rc != TB_OK) return rc;
  }
  return TB_OK;
}

extern "C" int tb_beam_reset_slots(tb_batch* b, int32_t n, const int32_t* slots, void* stream_) {
  return beam_reset_slots(b, n, slots, 0, nullptr, nullptr, nullptr, stream_);
}

extern "C" int tb_beam_start_slots(tb_batch* b, int32_t n, const int32_t* slots, int32_t K, float* scores, int32_t* states,
                                   uint8_t* live, void* stream_) {
  if (!b || !scores || !states || !live || K < 1 || K > b->max_beam) return TB_ERR_INVALID_ARG;
  return beam_reset_slots(b, n, slots, K, scores, states, live, stream_);
}

extern "C" int tb_beam_chunk(tb_batch* b, const void* logits, int dtype, int32_t n_slots, int32_t K, int32_t chunk, int32_t E,
                             int64_t stream_stride, int64_t frame_stride, int64_t row_stride, int32_t merge,
                             const int32_t* n_frames, float* scores, int32_t* states, uint8_t* live, int32_t* out_parent,
                             int32_t* out_token, void* stream_) {
  TbRange range_("tb_beam_chunk");
  if (!b || !logits || !scores || !states || !live || !out_parent || !out_token) return TB_ERR_INVALID_ARG;
  if ((dtype != TB_BF16 && dtype != TB_F32) || n_slots < 1 || n_slots > b->n_slots || K < 1 || K > b->max_beam || chunk < 1 ||
      E < 1 || static_cast<int64_t>(chunk) * E > (1 << 24))
    return TB_ERR_INVALID_ARG;
  if (!b->d_tree || b->max_tree_steps < 1) return TB_ERR_INVALID_ARG;            // streaming needs the hypothesis tree
  if (b->chunk_K != 0 && b->chunk_K != K) return TB_ERR_INVALID_ARG;             // one beam width between resets of all slots
  if (b->tree_steps != 0) return TB_ERR_INVALID_ARG;                             // the tree is in use by tb_beam_step / tb_beam_frames
  TbBeamParams p;
  std::memset(&p, 0, sizeof p);
  p.logits = logits; p.dtype = dtype; p.B = n_slots; p.K = K; p.V = b->vocab; p.C = b->n_classes;
  p.merge = merge ? 1 : 0; p.prune_delta = b->beam_prune_delta; p.new_frame = 1;
  p.stream_stride = stream_stride; p.hyp_stride = 0;
  p.scores = scores; p.states = states; p.live = live; p.out_parent = out_parent; p.out_token = out_token;
  p.tree = b->d_tree;
  // each slot's ring: the tree buffer holds max_tree_steps * n_slots * max_beam entries, i.e. per slot
  // max_tree_steps * max_beam / K steps of K entries (an entry index never leaves the slot's share)
  p.tree_cap = static_cast<int32_t>(static_cast<int64_t>(b->max_tree_steps) * b->max_beam / K);
  p.slots = b->d_slots; p.arena = b->arena; p.cls = b->d_cls; p.status = b->d_status;
  DeviceGuard guard(b->device);
  if (!guard.ok) return TB_ERR_CUDA;
  const size_t n_hyp = static_cast<size_t>(b->n_slots) * b->max_beam;
  beam_prepass(b, &p, chunk, E, frame_stride, row_stride, n_frames, static_cast<cudaStream_t>(stream_));
  const int rc = tb_launch_beam_chunk(p, chunk, E, frame_stride, row_stride, n_frames, b->d_slot_pos, b->d_hyp_hash,
                                      b->d_hyp_len, n_hyp, static_cast<cudaStream_t>(stream_));
  if (rc == TB_OK) b->chunk_K = K;
  return rc;
}

extern "C" int tb_beam_backtrace_slots(tb_batch* b, int32_t n_slots, int32_t K, int32_t max_len, int32_t* out_tokens,
                                       int32_t* out_lens, void* stream_) {
  TbRange range_("tb_beam_backtrace_slots");
  if (!b || !out_tokens || !out_lens || max_len < 1 || n_slots < 1 || n_slots > b->n_slots) return TB_ERR_INVALID_ARG;
  if (!b->d_tree || b->chunk_K != K) return TB_ERR_INVALID_ARG;
  DeviceGuard guard(b->device);
  if (!guard.ok) return TB_ERR_CUDA;
  const int32_t cap = static_cast<int32_t>(static_cast<int64_t>(b->max_tree_steps) * b->max_beam / K);
  return tb_launch_beam_backtrace_slots(b->d_tree, cap, b->d_slot_pos, n_slots, K, b->vocab, max_len, out_tokens, out_lens,
                                        b->d_status, b->d_hyp_len, static_cast<size_t>(b->n_slots) * b->max_beam, nullptr,
                                        static_cast<cudaStream_t>(stream_));
}

extern "C" int tb_beam_backtrace_slot_list(tb_batch* b, int32_t n, const int32_t* slots, int32_t K, int32_t max_len,
                                           int32_t* out_tokens, int32_t* out_lens, void* stream_) {
  TbRange range_("tb_beam_backtrace_slot_list");
  if (!b || !out_tokens || !out_lens || max_len < 1 || n < 1 || !slots) return TB_ERR_INVALID_ARG;
  for (int32_t i = 0; i < n; ++i) if (slots[i] < 0 || slots[i] >= b->n_slots) return TB_ERR_BAD_SLOT;
  if (!b->d_tree || b->chunk_K != K) return TB_ERR_INVALID_ARG;
  DeviceGuard guard(b->device);
  if (!guard.ok) return TB_ERR_CUDA;
  const int32_t cap = static_cast<int32_t>(static_cast<int64_t>(b->max_tree_steps) * b->max_beam / K);
  for (int32_t at = 0; at < n; at += TB_BIND_PAIRS) {
    const int32_t m = n - at < TB_BIND_PAIRS ? n - at : TB_BIND_PAIRS;
    const int rc = tb_launch_beam_backtrace_slots(b->d_tree, cap, b->d_slot_pos, m, K, b->vocab, max_len,
                                                  out_tokens + static_cast<int64_t>(at) * K * max_len, out_lens + static_cast<int64_t>(at) * K,
                                                  b->d_status, b->d_hyp_len, static_cast<size_t>(b->n_slots) * b->max_beam, slots + at,
                                                  static_cast<cudaStream_t>(stream_));
    if (rc != TB_OK) return rc;
  }
  return TB_OK;
}

extern "C" int tb_apply_final_weights_slots(tb_batch* b, int32_t n, const int32_t* slots, int32_t K, float* scores,
                                            const int32_t* states, void* stream_) {
  if (!b || n < 1 || !slots || K < 1 || !scores || !states) return TB_ERR_INVALID_ARG;
  for (int32_t i = 0; i < n; ++i) if (slots[i] < 0 || slots[i] >= b->n_slots) return TB_ERR_BAD_SLOT;
  DeviceGuard guard(b->device);
  if (!guard.ok) return TB_ERR_CUDA;
  for (int32_t at = 0; at < n; at += TB_BIND_PAIRS) {
    const int32_t m = n - at < TB_BIND_PAIRS ? n - at : TB_BIND_PAIRS;
    const int rc = tb_launch_final_weights_slots(b->d_slots, b->arena, m, slots + at, K, scores, states, b->d_status,
                                                 static_cast<cudaStream_t>(stream_));
    if (rc != TB_OK) return rc;
  }
  return TB_OK;
}

extern "C" int tb_beam_backtrace(tb_batch* b, int32_t B, int32_t K, int32_t max_len, int32_t* out_tokens,
                                 int32_t* out_lens, void* stream_) {
  TbRange range_("tb_beam_backtrace");
  if (!b || !out_tokens || !out_lens || max_len < 1) return TB_ERR_INVALID_ARG;
  if (!b->d_tree || b->tree_steps == 0 || b->tree_B != B || b->tree_K != K) return TB_ERR_INVALID_ARG;
  DeviceGuard guard(b->device);
  if (!guard.ok) return TB_ERR_CUDA;
  // the sequence records the last step wrote: their lengths are the transcripts' lengths
  const size_t n_hyp = static_cast<size_t>(b->n_slots) * b->max_beam;
  const int32_t* len_cur = b->beam_steps > 0 ? b->d_hyp_len + (((b->beam_steps - 1) & 1) ? 0 : n_hyp) : nullptr;
  return tb_launch_beam_backtrace(b->d_tree, b->tree_steps, B, K, b->vocab, max_len, out_tokens, out_lens, len_cur,
                                  static_cast<cudaStream_t>(stream_));
}
