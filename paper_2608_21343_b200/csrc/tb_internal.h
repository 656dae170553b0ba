// Internal declarations shared by the host compiler, the batch/arena code and the kernels.
#ifndef TB_INTERNAL_H_
#define TB_INTERNAL_H_

#include <cstddef>
#include <cstdint>
#include <vector>

#include "tb.h"

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
  std::vector<unsigned char> blob;
  int64_t off_arc_begin = 0, off_fail = 0, off_bw = 0, off_arc_cls = 0, off_arc_w = 0, off_arc_dst = 0;
};

uint64_t tb_hash_class_map(const int32_t* case_class, int32_t vocab);

// One row of the device offset table: where a slot's arrays start inside the arena (byte
// offsets from the arena base) and the scalars a walk needs.  n_states == 0 marks an unbound
// slot (model id -1).
struct TbSlotRec {
  int64_t off_arc_begin, off_fail, off_bw, off_arc_cls, off_arc_w, off_arc_dst;
  int32_t n_states, n_arcs, max_depth;
  float lambda;
};
static_assert(sizeof(TbSlotRec) == 64, "slot record is one 64-byte line");

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
