// Kernel parameter blocks and launch entry points (host side of the kernels).
#ifndef TB_LAUNCH_H_
#define TB_LAUNCH_H_

#include <cstddef>
#include <cuda_runtime.h>

#include "tb_internal.h"

struct TbDecodeParams {
  const void* logits;        // device
  int dtype;                 // TB_BF16 / TB_F32
  int32_t n_streams, frames, S, V, n_dur, C;
  int64_t sb, st, ss, sv;    // element strides: stream, frame, row-in-frame, token
  const int32_t* lengths;    // device [n_streams] or null
  int32_t persistent;        // 0: offline greedy (fresh state); 1: streaming (TbSlotState)
  int32_t tokview;           // set by the launcher: shared memory is sized for the token view of resolved lists
  int32_t normalize;         // every visited row is scored by its log-softmax (general kernel: before the bonus is added; pipelined kernels: the normaliser comes off the selected value)
  int32_t* out_tokens; int32_t* out_frames; int32_t* out_durs; int32_t* out_counts;
  float* out_scores; int32_t* out_states; int32_t* out_cursors;
  int32_t out_cap;           // tokens per stream the output arrays can hold
  const TbSlotRec* slots; TbSlotState* sstate; const unsigned char* arena;
  const int32_t* cls;        // device [V] token -> class
  int32_t* status;
};

// What the beam pre-pass leaves per logit row: the top_m tokens (blank excluded) with the largest root-boosted value
// y = fl(x + fl(lambda * w_root(class))), best first (ties: lowest token), and in entry top_m the value y of the next one
// (-inf if there is none) together with the row's blank logit in x.
struct TbTopEnt {
  float y;
  float x;            // the token's logit (entry top_m: the blank logit)
  uint32_t tok_cls;   // token | class << 16
};

struct TbBeamParams {
  const void* logits; int dtype;
  int32_t B, K, V, C, new_frame, step;
  int32_t tokview;           // set by the launcher, as in TbDecodeParams
  int64_t stream_stride, hyp_stride;
  float* scores; int32_t* states; uint8_t* live; int32_t* out_parent; int32_t* out_token;
  int2* tree;                // [steps, B, K] (parent, token) or null
  // identity of every hypothesis' token sequence (64-bit hash and length), read from *_in, written to *_out
  const unsigned long long* hash_in; unsigned long long* hash_out; const int32_t* len_in; int32_t* len_out;
  int32_t merge;             // at this frame start, hypotheses with equal token sequences are merged first
  float prune_delta;         // >= 0: at a frame start, hypotheses scoring below best - prune_delta are dropped
  int32_t tv_ready;          // set inside a multi-step launch: the block's root tables in shared memory are filled already
  int32_t fresh;             // first step after a reset: every hypothesis has the empty sequence, *_in is not read
  // streaming (tb_beam_chunk): every slot keeps its own ring of tree_cap steps, tree[slot][step % tree_cap][K]; 0: the
  // tree is [steps, B, K] for the whole batch
  int32_t tree_cap;
  // rows reduced ahead of the steps (tb_launch_beam_topm): per row top_m + 1 entries of 12 bytes, see TbTopEnt; null: none.
  // top_rows: this step's row (set per step inside a multi-step launch); top_base / strides: where the launch finds them
  const struct TbTopEnt* top_row;
  const struct TbTopEnt* top_base;
  int32_t top_m;
  const TbSlotRec* slots; const unsigned char* arena; const int32_t* cls; int32_t* status;
  // first / one-past-last byte of the logits tensor of a multi-step launch (set by the launcher; null: not known)
  const unsigned char* tensor_lo; const unsigned char* tensor_hi;
  int32_t rec_cache_bytes;   // shared memory set aside for a copy of the stream's list records (narrow beams; 0: none)
};

// Binds that a streaming chunk launch carries out itself (tb_stream_chunk_binds): the block of slot[i] first copies
// the graph image of bytes[i] bytes from src[i] -- page-locked host memory, read in place -- to its arena block
// (rec[i].blob_off), stores rec[i] as the slot's record and starts the slot's stream afresh; all other blocks start
// at once.  bytes 0: the slot becomes unbound (rec all zero).
#define TB_INLINE_BINDS 16
struct TbInlineBinds {
  int32_t n;
  int32_t slot[TB_INLINE_BINDS];
  int32_t bytes[TB_INLINE_BINDS];
  const unsigned char* src[TB_INLINE_BINDS];
  unsigned char* arena;       // (writable views of what the decode parameters hold as read-only)
  TbSlotRec* slots;
  TbSlotRec rec[TB_INLINE_BINDS];
};

int tb_launch_decode_general(const TbDecodeParams& p, cudaStream_t stream, const TbInlineBinds* binds = nullptr);
// The same binds carried out by a launch of their own (tb_batch_bind_stream(s) for graphs in the page-locked pool).
int tb_launch_pull_binds(const TbInlineBinds& binds, TbSlotState* sstate, cudaStream_t stream);
// Returns TB_OK when it launched, 1 when the call is outside what the pipelined kernel covers.
// max_cache_bytes: the largest cacheable list section among the slots decoded; max_states: their largest state count.
// all_resolved: non-zero when every bound graph among them carries resolved per-state lists.
// scratch / scratch_bytes: device memory for the two-segment decode (tb_greedy_fast_scratch_bytes says how
// much a call needs); with less than that the kernel decodes every stream as one segment.
size_t tb_greedy_fast_scratch_bytes(int32_t n_streams, int32_t frames, int32_t S);
int tb_launch_greedy_fast(const TbDecodeParams& p, int32_t max_cache_bytes, int32_t max_states, int32_t all_resolved,
                          void* scratch, size_t scratch_bytes, cudaStream_t stream);
// The segmented kernel (tb_greedy_seg.cu): every stream cut into NB * G segments, NB blocks per stream with G decider
// warps and H helper warps each.  force_*: non-zero values override the automatic choice (tuning).
struct TbSegPlan {
  int32_t G = 0, H = 0, NB = 0, smem = 0;
  int32_t force_G = 0, force_H = 0, force_NB = 0;
  int32_t test_timeout = 0;   // self-test: one frame is withheld and the waits are short, so a wait runs out
};
bool tb_greedy_seg_plan(const TbDecodeParams& p, int32_t max_cache_bytes, int32_t all_resolved, int32_t n_sm,
                        int32_t max_smem, TbSegPlan* plan);
size_t tb_greedy_seg_scratch_bytes(int32_t n_streams, int32_t frames, int32_t S, int32_t nseg_max);
int tb_launch_greedy_seg(const TbDecodeParams& p, int32_t max_cache_bytes, const TbSegPlan& plan, void* scratch,
                         cudaStream_t stream);
int tb_launch_beam_step(const TbBeamParams& p, cudaStream_t stream);
int tb_launch_beam_frames(const TbBeamParams& p, int32_t T, int32_t E, int64_t frame_stride, int64_t row_stride,
                          cudaStream_t stream);
// Streaming beam decoding, slot by slot (tb_beam_chunk and friends).  slot_pos: device [n_slots], steps each slot has
// taken since its last reset; hash / len: both halves of the per-hypothesis sequence records, n_hyp entries apart.
int tb_launch_beam_chunk(const TbBeamParams& p, int32_t T, int32_t E, int64_t frame_stride, int64_t row_stride,
                         const int32_t* n_frames, int32_t* slot_pos, unsigned long long* hash, int32_t* len, size_t n_hyp,
                         cudaStream_t stream);
int tb_launch_beam_reset_slots(int32_t* slot_pos, unsigned long long* hash, int32_t* len, size_t n_hyp, int32_t rec_stride,
                               int32_t n, const int32_t* slots, int32_t all_slots, const TbSlotRec* slot_recs, int32_t K,
                               float* scores, int32_t* states, uint8_t* live, cudaStream_t stream);
int tb_launch_beam_backtrace_slots(const int2* tree, int32_t tree_cap, const int32_t* slot_pos, int32_t n_slots, int32_t K,
                                   int32_t V, int32_t max_len, int32_t* out_tokens, int32_t* out_lens, int32_t* status,
                                   const int32_t* len_base, size_t n_hyp, const int32_t* slot_list, cudaStream_t stream);
int tb_launch_final_weights_slots(const TbSlotRec* slots, const unsigned char* arena, int32_t n, const int32_t* slot_list,
                                  int32_t K, float* scores, const int32_t* states, int32_t* status, cudaStream_t stream);
// Reduces every row of [B, T, E] (element strides given) to its TbTopEnt entries: out[((b * T + t) * E + e) * (top_m + 1)].
// n_frames: device [B] or null (rows of frames at or beyond it are skipped).
int tb_launch_beam_topm(const void* logits, int dtype, int32_t B, int32_t T, int32_t E, int32_t V, int32_t C,
                        int64_t stream_stride, int64_t frame_stride, int64_t row_stride, const int32_t* n_frames,
                        const TbSlotRec* slots, const unsigned char* arena, const int32_t* cls, int32_t top_m,
                        TbTopEnt* out, cudaStream_t stream);
int tb_launch_beam_backtrace(const int2* tree, int32_t n_steps, int32_t B, int32_t K, int32_t V, int32_t max_len,
                             int32_t* out_tokens, int32_t* out_lens, const int32_t* len_cur, cudaStream_t stream);
// Registered models: their records live in a device table; tb_launch_bind_models points up to TB_BIND_PAIRS slots at
// models of that table (id -1: unbound) and resets the slots' streaming state, in one launch.
#define TB_BIND_PAIRS 256
int tb_launch_publish_model(TbSlotRec* model_recs, int32_t model_id, const TbSlotRec& rec, cudaStream_t stream);
int tb_launch_bind_models(TbSlotRec* slots, TbSlotState* sstate, const TbSlotRec* model_recs, int32_t n,
                          const int32_t* slot_of, const int32_t* model_of, cudaStream_t stream);
int tb_launch_final_weights(const TbSlotRec* slots, const unsigned char* arena, int32_t B, int32_t K, float* scores,
                            const int32_t* states, int32_t* status, cudaStream_t stream);
// n slots at once: recs / slot_of are device arrays (uploaded together with the graphs they describe).
int tb_launch_publish_slots(TbSlotRec* slots, TbSlotState* sstate, int32_t n, const TbSlotRec* recs, const int32_t* slot_of,
                            cudaStream_t stream);
int tb_launch_publish_slot(TbSlotRec* slots, TbSlotState* sstate, int32_t slot, const TbSlotRec& rec,
                           cudaStream_t stream);

#endif  // TB_LAUNCH_H_
