// Internal declarations shared by the host compiler, the batch/arena code and the kernels.
#ifndef TB_INTERNAL_H_
#define TB_INTERNAL_H_

#include <atomic>
#include <cstddef>
#include <cstdint>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "tb.h"

// A named range around a library call for timeline tools (NVTX; costs a pointer test when no tool is attached).
struct TbRange {
  explicit TbRange(const char* name) { nvtxRangePushA(name); }
  ~TbRange() { nvtxRangePop(); }
  TbRange(const TbRange&) = delete;
  TbRange& operator=(const TbRange&) = delete;
};

// Page-locked host memory for graph images.  A process that decodes (one that has created a batch) keeps the device
// image of every graph it compiles or loads in one pool of page-locked memory, so that a bind is a plain
// host-to-device copy from where the image already is: no staging copy on the path between "a stream starts" and
// "its first chunk is decoded".  Before the first batch exists (a process that only compiles), when the pool is full,
// or without a device, the image lives on the heap and binds go through the batch's staging ring.
void tb_pinned_pool_arm();                       // called when a batch has been created
void* tb_pinned_alloc(size_t bytes);             // nullptr: not from the pool (use the heap)
bool tb_pinned_free(void* p, size_t bytes);      // false: p is not the pool's
bool tb_pinned_owns(const void* p);
// The address at which kernels of the current device can read the pool memory at host address p (the pool's pieces
// are mapped into the device's address space when they are taken), or null when p is not the pool's or not mapped.
const unsigned char* tb_pinned_device_ptr(const void* p);
void tb_pinned_bypass(bool on);                  // this thread's next images go to the heap (TB_COMPILE_PAGEABLE)

template <typename T>
struct TbImageAlloc {
  using value_type = T;
  TbImageAlloc() = default;
  template <typename U> TbImageAlloc(const TbImageAlloc<U>&) {}
  T* allocate(size_t n) {
    void* p = tb_pinned_alloc(n * sizeof(T));
    if (!p) p = ::operator new(n * sizeof(T));
    return static_cast<T*>(p);
  }
  void deallocate(T* p, size_t n) {
    if (!tb_pinned_free(p, n * sizeof(T))) ::operator delete(p);
  }
  template <typename U> bool operator==(const TbImageAlloc<U>&) const { return true; }
  template <typename U> bool operator!=(const TbImageAlloc<U>&) const { return false; }
};
using TbImage = std::vector<unsigned char, TbImageAlloc<unsigned char>>;

// A compiled graph: the canonical flat arrays (what tb_graph_view exposes) plus the
// position-independent byte blob that is copied into the device arena.
struct tb_graph {
  int32_t n_states = 0, n_arcs = 0, n_classes = 0, vocab = 0, max_depth = 0;
  float lambda = 1.0f;
  std::vector<int32_t> state_arc_begin, arc_class, arc_dst, state_fail, case_class;
  std::vector<float> arc_w, state_bw, state_final;
  std::vector<uint8_t> state_depth;
  uint64_t class_map_hash = 0;  // to reject a bind against a batch with another class map
  // Device blob: sections at 16-byte aligned offsets, all ids graph-local.
  TbImage blob;                                        // (allocated once, at its final size: see TbImageAlloc)
  int32_t off_arc_begin = 0, off_fail = 0, off_bw = 0, off_arc_cls = 0, off_arc_w = 0, off_arc_dst = 0;
  int32_t off_final = 0;                               // state_final as a blob section (end-of-stream weights)
  int32_t off_strec = 0, off_tokent = 0, n_tokent = 0;
  int32_t off_rsrec = 0, off_rsent = 0, n_rsent = 0;  // resolved per-state lists (n_rsent < 0: not built)
  float d_max = 0.0f;                                  // largest |sum of suffix-link weights| over all states
  std::atomic<int32_t> refs{1};                        // holders: the caller's handle, one per cache that keeps the graph, one per copy in flight
  bool pinned = false;                                 // the blob's pages are locked (it sits in the pool, or tb_graph_pin registered it): binds copy straight from it
  bool registered = false;                             // ... by tb_graph_pin: to be unregistered
  ~tb_graph();
};

// Page-locks the blob of a graph that will be bound again and again (graphs kept by a cache) if it is not in the
// page-locked pool already, so that a bind can hand it to the copy engine directly instead of going through the
// staging ring.  Does nothing without a device.
void tb_graph_pin(tb_graph* g);

// Two derived sections of the blob serve the pipelined kernel.  TbStateRec packs what a
// suffix-link walk needs from one state into one 16-byte load; TbTokEnt lists, per state, its
// outgoing arcs expanded to tokens (every case sibling of the arc's class), so that the tokens
// a state boosts can be scored without going through the class -> tokens table.
struct TbStateRec {
  int32_t tok_begin, tok_end;  // range in the TbTokEnt section
  int32_t fail;                // suffix-link target
  float bw;                    // suffix-link weight
};
struct TbTokEnt {
  uint32_t tok_cls;            // token | class << 16
  float w;                     // arc weight
  int32_t dst;                 // arc target
  int32_t pad;
};
static_assert(sizeof(TbStateRec) == 16 && sizeof(TbTokEnt) == 16, "16-byte records");

// Resolved lists: for every state, all tokens that the non-root part of its suffix chain boosts,
// shadowing already applied (the chain state closest to the state wins a class), sorted by token
// id, each with its finished additive term lb = fl(lambda * fl(acc + w)) (acc = suffix-link
// weights crossed before the arc's chain state, added in walk order) and the arc's target.  With
// them a state change costs the pipelined kernel one record load instead of a chain walk.  Built
// only for graphs whose lists stay small (TB_RS_MAX_ENTRIES) and whose ids fit the packing.
// Every list is padded to a multiple of four entries with sentinels {token = vocab (the blank
// column), lb = -inf, target 0}, which can never be selected, so that readers may take four
// entries at a time without a bounds test.
struct TbRsRec {
  int32_t begin, count;  // range in the TbRsEnt section (count includes the padding)
  float D;               // sum of the suffix-link weights of the whole chain, in walk order
  float bmag;            // |lambda| * (|D| + largest root arc weight): scale of the rounding margin
};
struct TbRsEnt {
  uint32_t dst_tok;      // target state << 12 | 2 * token (the token's byte offset in a bf16 row)
  float lb;
};
static_assert(sizeof(TbRsRec) == 16 && sizeof(TbRsEnt) == 8, "record sizes");
#define TB_RS_MAX_ENTRIES (1 << 18)
#define TB_RS_TOK_BITS 12   /* 2 * token < 4096, i.e. vocab + 1 <= 2048 */

uint64_t tb_hash_class_map(const int32_t* case_class, int32_t vocab);

// One row of the device offset table: where a slot's arrays start inside the arena (byte
// offsets from the arena base) and the scalars a walk needs.  n_states == 0 marks an unbound
// slot (model id -1).
struct TbSlotRec {
  int64_t blob_off;  // byte offset of the graph's blob inside the arena
  int32_t off_arc_begin, off_fail, off_bw, off_arc_cls, off_arc_w, off_arc_dst, off_strec, off_tokent;  // within the blob
  int32_t n_states, n_arcs, max_depth;
  float lambda;
  int32_t n_tokent, blob_bytes;
  int32_t off_rsrec, off_rsent, n_rsent;  // resolved lists; n_rsent < 0: the graph has none
  float d_max;
  int32_t off_final;   // per-state final weights (within the blob)
  int32_t pad[11];
};
static_assert(sizeof(TbSlotRec) == 128, "slot record is 128 bytes");

// Per-slot streaming state kept on the device between tb_stream_chunk calls.
struct TbSlotState {
  int32_t state;       // graph state, -1 when unbound
  int32_t t;           // frame cursor, relative to the stream's first frame
  int32_t k;           // symbols already emitted in frame t
  float score;
  int32_t n_emitted;
  int32_t chunk_base;  // frames covered by earlier chunks since the last bind
  int32_t pad0, pad1;
};
static_assert(sizeof(TbSlotState) == 32, "slot state is 32 bytes");

#endif  // TB_INTERNAL_H_
