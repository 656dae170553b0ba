/*
 * tb.h -- C ABI of the B200 phrase-boosting decode library.
 *
 * The library implements the hot path of per-stream shallow-fusion phrase boosting inside
 * batched Transducer (RNNT / TDT) decoding: every stream of a batch owns a compiled
 * case-insensitive boosting graph; each decode step turns the hypothesis's graph state into
 * a bonus over the vocabulary, adds lambda * bonus to the joint logits, selects tokens
 * (argmax, or top-K over beam x vocabulary) and advances the graph state; blank leaves the
 * state unchanged.
 *
 * Conventions
 *   - Every call returns an int: TB_OK (0) or a negative TB_ERR_* code; tb_strerror() names
 *     it.  No exception crosses this boundary.  The library keeps no global state, with one
 *     exception that its own comment describes: the fixed device array of tb_greedy_decode_noalloc.
 *   - "host" pointers are read or written by the CPU during the call.  "device" pointers are
 *     caller-owned device memory on the batch's GPU; the library never frees or resizes
 *     them.  The library owns only what tb_batch_create allocates (graph arena, slot table,
 *     per-slot decode state, hypothesis tree, status word).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  GPU
 *     work is enqueued on it and returns before it has run; device outputs may be read after
 *     the stream has been synchronised.  All calls on one batch must be issued to one
 *     stream, or be ordered by the caller, because a re-bind may reuse arena space that
 *     earlier decode calls read.
 *   - Token ids are 0..vocab-1, blank = vocab.  Graph states are graph-local (root = 0); a
 *     slot without a graph reports state -1.
 *   - Logits must not contain NaN (the selection is then undefined); infinities are fine.
 *   - Arithmetic contract: a candidate's value is fl(x + fl(lambda * bonus)) in float32 (a
 *     rounded multiply, then a rounded add, never fused); blank and unbound slots use x
 *     itself; bf16 logits are widened exactly.  Ties go to the lowest token id.
 */
#ifndef TB_H_
#define TB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TB_OK 0
#define TB_ERR_INVALID_ARG (-1)   /* a bad pointer, size, token, weight, stride, dtype */
#define TB_ERR_OOM (-2)           /* host or device allocation failed */
#define TB_ERR_CUDA (-3)          /* a CUDA runtime call failed */
#define TB_ERR_ARENA_FULL (-4)    /* the graph does not fit into the arena's free space */
#define TB_ERR_BAD_SLOT (-5)      /* slot index outside the batch */
#define TB_ERR_DEVICE_STATUS (-6) /* a kernel recorded a violated bound (see tb_batch_status) */
#define TB_ERR_IO (-7)            /* a file could not be opened, read or written */

#define TB_BF16 0 /* logits are bfloat16 */
#define TB_F32 1  /* logits are float32 */

/* Bits of the device status word (tb_batch_status). */
#define TB_STATUS_WALK_TOO_DEEP 1   /* a suffix-link walk exceeded the graph's depth bound */
#define TB_STATUS_BAD_STATE 2       /* a graph state outside [0, n_states) was met */
#define TB_STATUS_STEP_LIMIT 4      /* a decode loop hit its static iteration bound */
#define TB_STATUS_WAIT_TIMEOUT 8    /* a bounded wait inside a kernel ran out */

/* tb_beam_step, new_frame */
#define TB_FRAME_SAME 0       /* another row of the current frame */
#define TB_FRAME_NEW 1        /* first row of a frame: every hypothesis with a score becomes live */
#define TB_FRAME_NEW_MERGE 2  /* as TB_FRAME_NEW, after hypotheses with equal token sequences were merged */

/* tb_graph_compile, tb_graph_compile_variative, tb_cache_compile(_variative): flags */
#define TB_COMPILE_PAGEABLE 1           /* keep the graph's device blob in ordinary host memory even when the process has its pool of
                                           page-locked memory (see tb_cache_compile): for lists compiled in bulk and seldom bound; a
                                           bind then stages the blob through page-locked memory of the batch */

/* tb_batch_set_flags */
#define TB_FLAG_GENERAL_KERNELS 1       /* always use the general decode kernel (any layout), never a pipelined one */
#define TB_FLAG_ONE_BLOCK_PER_STREAM 2  /* pipelined greedy decode: never the segmented kernel, one block per stream */
#define TB_FLAG_LOG_SOFTMAX 8           /* tb_greedy_decode and tb_stream_chunk (RNNT rows) score every visited row by its log-softmax:
                                           L = m + log(sum_v exp(x_v - m)) over the row's vocab+1 entries, computed in float inside
                                           the selection kernel (Sec. 2.2 para. 3: one fused scoring operation).  The general kernel
                                           (any layout; streaming chunks) takes L off every entry before the bonus is added:
                                           value(v) = fl(fl(x_v - L) + fl(lambda * bonus)).  The pipelined kernels (packed bf16 rows)
                                           take it off after the selection, L being common to a row's candidates: the row is
                                           decided on fl(x_v + fl(lambda * bonus)) exactly as without the flag, and adds
                                           fl(that value - L) to the score.  Either way tokens can differ from a decode in exact
                                           arithmetic only where two candidates are closer than the float roundings, and scores
                                           by a few float roundings per visited row */
#define TB_FLAG_BEAM_WHOLE_ROWS 16      /* tb_beam_frames / tb_beam_chunk: no pre-pass that reduces every row to its best tokens; every
                                           step looks at all vocab+1 entries of its row (identical results) */
#define TB_FLAG_COPIED_BINDS 32         /* tb_stream_chunk_binds: always bind ahead of the chunk's launch (copies + a small launch), never
                                           inside it */
#define TB_FLAG_TEST_WAIT_TIMEOUT 4     /* self-test of the kernels' bounded waits: tb_greedy_decode (segmented kernel) withholds one
                                           frame's summaries and waits only briefly, so the wait runs out: the call returns,
                                           TB_STATUS_WAIT_TIMEOUT is set, the outputs of that call are undefined */

/* tb_batch_last_greedy_kernel */
#define TB_KERNEL_GENERAL 1     /* one block per stream, a block-wide argmax per visited row */
#define TB_KERNEL_PIPELINED 2   /* one block per stream: rows staged in shared memory, at most two segments */
#define TB_KERNEL_SEGMENTED 3   /* streams cut into segments decoded by many small pipelines on all SMs, then stitched */

/* Limits of this build. */
#define TB_MAX_VOCAB 8192           /* non-blank tokens */
#define TB_MAX_PHRASE_LEN 255       /* tokens per phrase (graph depth is stored in a byte) */
#define TB_MAX_PIECE_LEN 32         /* characters (bytes) per vocabulary piece, variative compile */
#define TB_MAX_BEAM 32
#define TB_NOALLOC_MAX_STREAMS 256 /* streams per tb_greedy_decode_noalloc call */

typedef struct tb_graph tb_graph; /* immutable compiled graph, host memory */
typedef struct tb_batch tb_batch; /* device arena + slot table + per-slot state */
typedef struct tb_cache tb_cache; /* compiled graphs kept in host memory, by the content of their lists */

/*
 * Read-only view of a compiled graph as flat arrays in host memory: the arc arrays (label =
 * case class, target state, weight) and state arrays (outgoing-arc range, suffix-link
 * target, suffix-link weight, final weight) of Sec. 2.2 para. 2.  States are numbered
 * breadth-first from root = 0 with a state's children in ascending class order, so arcs are
 * sorted by (source state, class).  The pointers stay valid until tb_graph_free.
 */
typedef struct {
  int32_t n_states, n_arcs, n_classes, vocab, max_depth;
  float lambda;
  const int32_t *state_arc_begin; /* [n_states+1] */
  const int32_t *arc_class;       /* [n_arcs] ascending within a state */
  const int32_t *arc_dst;         /* [n_arcs] */
  const float *arc_w;             /* [n_arcs] */
  const int32_t *state_fail;      /* [n_states] suffix-link target */
  const float *state_bw;          /* [n_states] suffix-link weight */
  const float *state_final;       /* [n_states] final weight; charged by tb_apply_final_weights only */
  const uint8_t *state_depth;     /* [n_states] */
  const int32_t *case_class;      /* [vocab] token -> class */
} tb_graph_view;

const char *tb_strerror(int code);

/*
 * Compile one phrase list into a boosting graph (host only, no GPU needed).
 * Sec. 2.1 para. 1-2 (phrase tree with suffix links; one arc per case class stands for all
 * case variants of a token), the potential rule above Eq. 1 (arc score = destination potential
 * minus source potential; one token per arc, so Eq. 1's split is Delta = w_k), Sec. 2.2 para. 2
 * (array layout).
 *   phrase_tokens  host int32 [phrase_offsets[n_phrases]]: the phrases' tokens, back to back
 *   phrase_offsets host int64 [n_phrases+1], non-decreasing, first entry 0
 *   token_weights  host float [as phrase_tokens] or NULL (= 1.0): score of each phrase token;
 *                  must be finite and >= 0; where phrases share a prefix the largest weight
 *                  given to a position wins; phrases equal after case folding are merged
 *   case_class     host int32 [vocab] or NULL (= identity, case-sensitive): tokens with the
 *                  same class are case variants of each other; classes are >= 0
 *   lambda         boosting weight of this list (Sec. 2.2 para. 2), finite
 *   flags          0, or TB_COMPILE_PAGEABLE
 *   out            receives the graph; free it with tb_graph_free
 * Empty phrases are skipped.  Errors: TB_ERR_INVALID_ARG (token outside [0, vocab), bad
 * weight or class, phrase longer than TB_MAX_PHRASE_LEN, vocab outside [1, TB_MAX_VOCAB]),
 * TB_ERR_OOM.
 */
int tb_graph_compile(const int32_t *phrase_tokens, const int64_t *phrase_offsets, int32_t n_phrases,
                     const float *token_weights, const int32_t *case_class, int32_t vocab, float lambda,
                     uint32_t flags, tb_graph **out);

/*
 * Token -> class map of a piece vocabulary for case-insensitive matching (Sec. 2.1 para. 5: a piece
 * counts wherever its lower-cased spelling matches): pieces with the same lower-cased spelling
 * (ASCII letters are folded, other bytes compared as they are) share a class; classes are numbered in
 * order of the lowest token id that has them.  Pass the result to tb_batch_create for a batch that
 * binds graphs made by tb_graph_compile_variative over the same vocabulary.
 *   piece_chars    host bytes [piece_offsets[vocab]]: the pieces' spellings, back to back
 *   piece_offsets  host int64 [vocab+1], increasing, first entry 0; every piece 1..TB_MAX_PIECE_LEN bytes
 *   out_case_class host int32 [vocab], written;  out_n_classes host int32 or NULL
 * Errors: TB_ERR_INVALID_ARG, TB_ERR_OOM.
 */
int tb_piece_classes(const uint8_t *piece_chars, const int64_t *piece_offsets, int32_t vocab,
                     int32_t *out_case_class, int32_t *out_n_classes);

/*
 * Compile one phrase list, given as text, into a variative case-insensitive boosting graph (host
 * only).  Sec. 2.1 para. 4-7 and Eq. 1: the lower-cased phrase is a chain of its characters; every
 * piece whose lower-cased spelling covers a contiguous stretch of the chain is an arc over it, so
 * the graph accepts every casing and every segmentation of the phrase; states carry a cumulative
 * potential and an arc scores the difference of the potentials of its ends.  The potentials come
 * from the greedy segmentation of the lower-cased phrase (here: longest spelling first): a token of
 * m characters with score w gives its character i (0-based) the share
 * w * exp((i+1)^tau) / sum_j exp((j+1)^tau).  Phrases sharing a prefix share its states, a state
 * taking the largest share given to it.  Suffix links and their weights are those of
 * tb_graph_compile, taken over the characters; an arc over several characters weighs what the
 * single-character arcs along it weigh together, so all spellings of a phrase earn the same total.
 * The result has the same array layout and is bound, decoded and freed like any other graph; its
 * classes are those of tb_piece_classes.
 *   phrase_chars   host bytes [phrase_offsets[n_phrases]]: the phrases' text, any casing, back to back
 *   phrase_offsets host int64 [n_phrases+1], non-decreasing, first entry 0; at most 255 bytes per phrase
 *   phrase_weights host float [n_phrases] or NULL (= 1.0): score w of every token of the phrase's
 *                  greedy segmentation; finite and >= 0
 *   piece_chars, piece_offsets, vocab  the piece vocabulary, as for tb_piece_classes; every
 *                  character of every phrase must be the spelling of some piece
 *   tau            Eq. 1's exponent, finite and >= 0 (0: uniform split; large: all at the token's end)
 *   lambda, flags, out  as for tb_graph_compile
 * Empty phrases are skipped.  Errors: TB_ERR_INVALID_ARG, TB_ERR_OOM.
 */
int tb_graph_compile_variative(const uint8_t *phrase_chars, const int64_t *phrase_offsets, int32_t n_phrases,
                               const float *phrase_weights, const uint8_t *piece_chars,
                               const int64_t *piece_offsets, int32_t vocab, float tau, float lambda,
                               uint32_t flags, tb_graph **out);

/* Fill *out with pointers into g (host).  TB_ERR_INVALID_ARG on NULL. */
int tb_graph_view_get(const tb_graph *g, tb_graph_view *out);

/* Free a graph.  Safe right after tb_batch_bind_stream returned: bind copies what it needs. */
void tb_graph_free(tb_graph *g);

/*
 * The host levels of the three-level cache of Sec. 2.2 para. 5 (the cost that remains with per-stream lists is
 * compiling and transferring the models when streams are created).
 *
 * Disk: tb_graph_save writes a compiled graph (its arrays and its device blob) to `path`; tb_graph_load
 * reads one back, identical in every array to the graph that was saved.  A file that is not such a file,
 * was cut short or altered (magic, version, sizes, a checksum over the contents, the class map) is refused
 * with TB_ERR_INVALID_ARG; a file that cannot be opened, read or written gives TB_ERR_IO.  Files are only
 * meant for the machine and build that wrote them (native byte order, this build's blob layout).
 */
int tb_graph_save(const tb_graph *g, const char *path);
int tb_graph_load(const char *path, tb_graph **out);

/*
 * Memory: a cache of compiled graphs in host memory, keyed by the content of everything the compiler
 * reads (tokens, offsets, weights, class map, vocab, lambda, flags).  tb_cache_compile returns the graph
 * tb_graph_compile would return for the same arguments -- from the cache when the same list was compiled
 * through this cache before (*out_hit = 1), otherwise by compiling it and keeping it (least recently used
 * graphs are dropped once `capacity_bytes` of host memory would be exceeded; a graph larger than that is
 * returned but not kept).  The returned graph is the caller's to release with tb_graph_free as usual; it
 * stays valid after the cache drops or is destroyed.  Calls on one cache may come from several threads.
 * Graphs kept by a cache have their device blob page-locked (when a CUDA device is present), so binding them
 * copies from the graph in place; the batch holds the graph until that copy is done.  The same holds for every graph
 * compiled or loaded after the process has created its first batch: their device blobs are placed in a pool of
 * page-locked host memory (up to 1 GB, in pieces of 32 MB; blobs over 16 MB and whatever does not fit stay on the heap
 * and are staged at bind time).  The pool's pieces are also mapped into the devices' address space, so that a
 * kernel can read a blob where it lies (tb_stream_chunk_binds uses that).
 *   out_hit  host int32 or NULL.   Errors: as tb_graph_compile.
 * tb_cache_stats: any pointer may be NULL.
 */
int tb_cache_create(size_t capacity_bytes, tb_cache **out);
void tb_cache_destroy(tb_cache *c);
int tb_cache_compile(tb_cache *c, const int32_t *phrase_tokens, const int64_t *phrase_offsets, int32_t n_phrases,
                     const float *token_weights, const int32_t *case_class, int32_t vocab, float lambda,
                     uint32_t flags, tb_graph **out, int32_t *out_hit);
/* The same for tb_graph_compile_variative (the key holds the phrases' text, weights, tau, lambda and a checksum of
 * the piece vocabulary). */
int tb_cache_compile_variative(tb_cache *c, const uint8_t *phrase_chars, const int64_t *phrase_offsets,
                               int32_t n_phrases, const float *phrase_weights, const uint8_t *piece_chars,
                               const int64_t *piece_offsets, int32_t vocab, float tau, float lambda, uint32_t flags,
                               tb_graph **out, int32_t *out_hit);
int tb_cache_stats(tb_cache *c, int64_t *hits, int64_t *misses, int64_t *evictions, size_t *bytes_used,
                   int64_t *entries);

/*
 * Create a batch on `device`: the merged multi-model storage of Sec. 2.2 para. 2 (one arena
 * holding every bound graph's arrays behind a per-slot offset table), plus per-slot decode
 * state.  All slots start unbound (model id -1).
 *   vocab, case_class  as for tb_graph_compile; one token -> class map per batch
 *   n_slots            number of stream slots (>= 1)
 *   max_beam           largest K tb_beam_step will be called with (1..TB_MAX_BEAM)
 *   max_tree_steps     capacity, in beam steps, of the hypothesis tree (0 = no tree)
 *   arena_bytes        size of the graph arena
 * Errors: TB_ERR_INVALID_ARG, TB_ERR_OOM, TB_ERR_CUDA.
 */
int tb_batch_create(int32_t vocab, const int32_t *case_class, int32_t n_slots, int32_t max_beam,
                    int32_t max_tree_steps, size_t arena_bytes, int device, tb_batch **out);

/* Free everything the batch owns (synchronises the device first). */
void tb_batch_destroy(tb_batch *b);

/*
 * Attach graph g to `slot`, or detach with g == NULL (model id -1: zero bonus, state -1;
 * Sec. 2.2 para. 3).  Adding and removing lists while other streams keep running is Sec. 2.2
 * para. 4; here the slot index is the stable id, and no other slot's graph moves or changes.
 * The graph reaches the arena on `stream`: a blob in the library's page-locked pool is read in place by a small
 * launch that also publishes the slot's record (no copy is enqueued); any other blob is copied with an asynchronous
 * host-to-device copy (from its own page-locked memory when a cache keeps it, else through page-locked staging
 * memory of the batch); the slot's offsets are published and its streaming state is reset (state =
 * root or -1, frame cursor 0, score 0) in stream order.  The previous graph's arena space is
 * reused by later binds.  g must have been compiled with the batch's vocab and class map.
 * Ordering: the previous graph's arena block goes back to the free list when this call returns, and a later bind
 * may overwrite it; a bind (this call, tb_batch_bind_streams, tb_batch_bind_model(s), tb_batch_register_model) must
 * therefore be enqueued on the same stream as, or be ordered by an event after, every decode call that still reads
 * the slot's previous graph.  Issuing all calls on one batch to one stream satisfies this.
 * Errors: TB_ERR_BAD_SLOT, TB_ERR_INVALID_ARG (vocab / class map mismatch),
 * TB_ERR_ARENA_FULL (nothing was changed), TB_ERR_CUDA.
 */
int tb_batch_bind_stream(tb_batch *b, int32_t slot, const tb_graph *g, void *stream);

/*
 * tb_batch_bind_stream for n slots at once (Sec. 2.2 para. 4: between two chunks several streams end and start): the
 * graphs are packed into one arena block; heap-held graphs travel, with all slot records, in ONE host-to-device copy,
 * page-locked graphs straight from where they are (one copy per run of graphs that are neighbours in the pool, which
 * graphs compiled one after the other usually are), followed by one small launch.  graphs[i] == NULL
 * unbinds slots[i].  A slot may appear once.  Everything is checked before anything changes.  A group of more than
 * 4 MB of graphs goes in parts of that size, and when the arena has no contiguous room for a part its slots are
 * bound one by one (an error then leaves the earlier ones bound).
 *   slots   host int32 [n];   graphs  host array of n graph pointers (each may be freed when the call returns)
 * Ordering: as for tb_batch_bind_stream -- a bind must be enqueued on the stream (or ordered by an event) after the
 * decode calls that still read the slots' previous graphs: their arena blocks go back to the free list at once and
 * the next bind may overwrite them.
 * Errors: TB_ERR_BAD_SLOT, TB_ERR_INVALID_ARG (a slot twice, vocab / class map mismatch), TB_ERR_ARENA_FULL, TB_ERR_CUDA.
 */
int tb_batch_bind_streams(tb_batch *b, int32_t n, const int32_t *slots, const tb_graph *const *graphs, void *stream);

/*
 * Decoder-level registration (Sec. 2.2 para. 5: models known before a recognition session are registered with
 * the decoder, which takes the update cost out of the decoding loop).  tb_batch_register_model copies the
 * graph into the arena once (asynchronously on `stream`, like a bind) and returns a model id >= 0;
 * tb_batch_bind_model then points a slot at that model: no compile, no copy, no allocation -- one small
 * kernel that writes the slot's record and resets its streaming state, ordered on `stream`.  Any number of
 * slots may be bound to one model; model id -1 unbinds the slot (as tb_batch_bind_stream with NULL).  A slot
 * bound either way can be re-bound either way.  tb_batch_unregister_model gives the model's arena block back;
 * it fails with TB_ERR_INVALID_ARG while a slot is still bound to the model.  The caller orders it after the
 * decode calls that may still read the model, as for re-binding a slot.
 * Errors: TB_ERR_INVALID_ARG (NULL, a graph for another vocabulary or class map, an id that is not
 * registered), TB_ERR_BAD_SLOT, TB_ERR_ARENA_FULL, TB_ERR_OOM, TB_ERR_CUDA.
 */
int tb_batch_register_model(tb_batch *b, const tb_graph *g, int32_t *out_model_id, void *stream);
int tb_batch_bind_model(tb_batch *b, int32_t slot, int32_t model_id, void *stream);
int tb_batch_unregister_model(tb_batch *b, int32_t model_id);
/*
 * tb_batch_bind_model for n (slot, model id) pairs at once: one small launch per 256 pairs, which is what takes the
 * update cost out of the decoding loop when many streams start together.  host int32 arrays; a slot may appear once.
 * All pairs are checked before anything changes (TB_ERR_BAD_SLOT, TB_ERR_INVALID_ARG).
 */
int tb_batch_bind_models(tb_batch *b, int32_t n, const int32_t *slots, const int32_t *model_ids, void *stream);

/*
 * Set behaviour flags of the batch (TB_FLAG_*; 0 = defaults).  With the defaults
 * tb_greedy_decode picks a pipelined kernel whenever the call fits it (bf16 logits, token
 * stride 1, the S rows of a frame contiguous, vocab <= 2048, S <= 4) -- the segmented one when every
 * bound graph carries resolved lists that fit a block's shared memory, else the one-block-per-stream
 * one -- and the general kernel otherwise; all give identical results.  The paper has no counterpart
 * of this call.
 * Errors: TB_ERR_INVALID_ARG (unknown bits).
 */
int tb_batch_set_flags(tb_batch *b, uint32_t flags);

/*
 * Tuning of the segmented greedy kernel (no counterpart in the paper): how many decider warps (1..4) and helper
 * warps a block holds, and how many blocks decode one stream; the stream is cut into blocks_per_stream *
 * deciders_per_block segments (Sec. 2.2 para. 3 asks for one advance per stream and step; segments are a way to run
 * several parts of a stream's decode at once, with identical results).  0 = chosen by the library from the GPU's
 * size and the call's shape; deciders and helpers are given together or not at all.
 * Errors: TB_ERR_INVALID_ARG.
 */
int tb_batch_set_greedy_plan(tb_batch *b, int32_t deciders_per_block, int32_t helpers_per_block,
                             int32_t blocks_per_stream);

/*
 * Which kernel the last successful tb_greedy_decode of this batch launched (TB_KERNEL_*; 0 before the first), and
 * for the segmented kernel its blocks per stream and deciders per block (host pointers, each may be NULL).  The
 * three kernels give identical results; a caller that depends on the speed of one can assert it here.
 */
int tb_batch_last_greedy_kernel(const tb_batch *b, int32_t *kernel, int32_t *blocks_per_stream,
                                int32_t *deciders_per_block);

/*
 * Copy the device status word to *device_status (host) after synchronising `stream`, and
 * clear it.  Returns TB_OK if it was 0, else TB_ERR_DEVICE_STATUS (bits: TB_STATUS_*).
 */
int tb_batch_status(tb_batch *b, int32_t *device_status, void *stream);

/*
 * Greedy RNNT decoding of B streams, slot i serving stream i, all on the device with no
 * host synchronisation per frame (Sec. 2.2 para. 3 for the boosted scores, Sec. 3.4 for greedy
 * label-looping decoding, Sec. 2.3 for GPU-resident execution).
 * Per stream: t = 0, k = 0, state = root; while t < length: take row (t, k), select the
 * argmax of the boosted row; blank: t++, k = 0; else emit (token, t), advance the state,
 * k++, and k == S closes the frame (t++, k = 0) adding nothing to the score.  The score is
 * the float32 sum, in step order, of the selected values.
 *   logits       device, dtype TB_BF16 or TB_F32, logical shape [B, T, S, vocab+1]
 *   strides      host int64 [4]: element strides of the four dimensions
 *   lengths      device int32 [B] or NULL (= T); values are clamped to [0, T]
 *   out_tokens   device int32 [B, T*S]: emitted tokens of stream i at [i*T*S ...]
 *   out_frames   device int32 [B, T*S]: frame of each emitted token
 *   out_counts   device int32 [B]: tokens emitted
 *   out_scores   device float [B]
 *   out_states   device int32 [B]: final graph state (-1 for unbound slots)
 * Does not read or change the slots' streaming state.  Working memory: the pipelined kernel
 * decodes long bound streams as two segments at once and merges them (the result is that of the
 * sequential decode, bit for bit); what the second segment produces passes through a device
 * block owned by the batch, which this call allocates or grows (freeing the old block, which
 * waits for the device) when B*T*S exceeds what an earlier call needed.  Hence one
 * tb_greedy_decode per batch at a time; if the block cannot be had, streams are decoded whole.
 * While `stream` is being captured into a CUDA graph nothing is allocated (the call works with
 * the block an earlier call left, or decodes the streams whole).
 * Errors: TB_ERR_INVALID_ARG (B > n_slots, bad dtype, NULL pointers, non-positive sizes),
 * TB_ERR_CUDA.
 */
int tb_greedy_decode(tb_batch *b, const void *logits, int dtype, int32_t B, int32_t T, int32_t S,
                     const int64_t *strides, const int32_t *lengths, int32_t *out_tokens,
                     int32_t *out_frames, int32_t *out_counts, float *out_scores, int32_t *out_states,
                     void *stream);

/*
 * One streaming chunk for slots 0..n_slots-1, RNNT (n_dur = 0) or TDT (n_dur > 0), resuming
 * from and updating each slot's persistent state {graph state, frame cursor, symbols in the
 * current frame, score, emitted count} (Sec. 2.3: decoding state is kept across chunk
 * boundaries; Sec. 2.2 para. 4: slots are re-bound between chunks).  The call covers the
 * slot's frames [c, c + chunk), c = the number of frames that earlier
 * tb_stream_chunk calls covered since the slot's last bind; frames at or beyond valid_frames[slot] are not
 * decoded; a cursor that a TDT duration moved beyond the chunk is carried over.
 * TDT row: vocab+1 token logits, then n_dur duration logits for durations 0..n_dur-1; the
 * duration is their argmax (lowest on ties); score += value[token] + x_dur[duration];
 * blank: t += max(duration, 1); token: emit, advance the state, then duration > 0 ?
 * t += duration : next row of the same frame (the S-th symbol closes the frame).
 *   logits        device [n_slots, chunk, S, vocab+1+n_dur], strides as above (host int64 [4])
 *   valid_frames  device int32 [n_slots]: total frames of the slot's stream known so far
 *   out_tokens / out_frames / out_durs  device int32 [n_slots, chunk*S]; out_durs may be NULL
 *   out_counts    device int32 [n_slots]: tokens emitted in this chunk
 *   out_scores    device float [n_slots]: running score
 *   out_states    device int32 [n_slots]: graph state after the chunk
 *   out_cursors   device int32 [n_slots] or NULL: frame cursor after the chunk
 * Errors: as tb_greedy_decode.
 */
int tb_stream_chunk(tb_batch *b, const void *logits, int dtype, int32_t n_slots, int32_t chunk, int32_t S,
                    int32_t n_dur, const int64_t *strides, const int32_t *valid_frames,
                    int32_t *out_tokens, int32_t *out_frames, int32_t *out_durs, int32_t *out_counts,
                    float *out_scores, int32_t *out_states, int32_t *out_cursors, void *stream);

/*
 * The streams that start with a chunk and the chunk itself in one call (Sec. 2.2 para. 4, Sec. 2.3): the result is
 * that of tb_batch_bind_streams(b, n_binds, bind_slots, bind_graphs, stream) followed by tb_stream_chunk with the
 * remaining arguments, both on `stream`.  The chunk's arguments are checked first: a chunk that would be refused
 * binds nothing.  n_binds may be 0 (bind_slots / bind_graphs are then not read).  If the binds fail the chunk is not
 * decoded.  Errors: those of the two calls.
 *
 * Up to 16 binds per call ride on the chunk's own launch: when every graph's image lies in the library's page-locked
 * memory (graphs compiled or loaded after the first tb_batch_create, without TB_COMPILE_PAGEABLE, not handed out by
 * a cache), the bound slots are among the chunk's n_slots, and `stream` is not being captured, the call reserves
 * the arena blocks, and the thread block that decodes a re-bound slot first reads the new image from host memory in
 * place into its arena block, stores the slot's record and starts the stream afresh, while all other slots' blocks
 * decode already: no copy is enqueued and no second launch is made.  The library holds the graphs until that
 * launch has completed, as for a copy.  Anything else goes the ordinary way (copies and a small launch ahead of the
 * chunk).  tb_batch_bind_counts tells how many binds went which way.
 */
int tb_batch_bind_counts(const tb_batch *b, int64_t *out_pulled, int64_t *out_copied);   /* binds of tb_stream_chunk_binds so far: inside the chunk's launch / ahead of it */
int tb_stream_chunk_binds(tb_batch *b, int32_t n_binds, const int32_t *bind_slots, const tb_graph *const *bind_graphs,
                          const void *logits, int dtype, int32_t n_slots, int32_t chunk, int32_t S, int32_t n_dur,
                          const int64_t *strides, const int32_t *valid_frames, int32_t *out_tokens, int32_t *out_frames,
                          int32_t *out_durs, int32_t *out_counts, float *out_scores, int32_t *out_states,
                          int32_t *out_cursors, void *stream);

/*
 * Forget the hypothesis tree (step counter = 0) and the per-hypothesis record of emitted token sequences (every
 * hypothesis starts from the empty sequence).  Call before the first step of an utterance (host bookkeeping only:
 * no device work, so it may sit inside a stream capture).  Across the chunks of one utterance simply keep calling
 * tb_beam_step: scores, states, liveness (the caller's arrays), the tree and the sequence records carry over.
 */
int tb_beam_reset(tb_batch *b);

/*
 * One beam expansion for streams 0..B-1 (Sec. 2.3 / Sec. 3.4 beam search; Sec. 2.2 para. 3 for
 * the scores), each hypothesis carrying its own graph state.
 * Per stream, candidates: each live hypothesis k with score > -inf and each token v in
 * 0..vocab scores fl(score_k + value_k(v)); each frozen hypothesis with score > -inf is
 * carried as one candidate with its score and token -1.  The K best in the order (score
 * descending, token ascending with the carried token counted as vocab+1, parent ascending)
 * become the new hypotheses, best first: score, state = token non-blank ? next(state_parent,
 * token) : state_parent, live = live_parent and token non-blank.  Unfilled places get score
 * -inf, state -1, live 0, parent -1, token -1.  (parent, token) is appended to the
 * hypothesis tree when the batch has one.
 *   logits         device; hypothesis k of stream i reads the vocab+1 contiguous elements
 *                  at element offset i*stream_stride + k*hyp_stride (hyp_stride 0: all
 *                  hypotheses of a stream share one row)
 *   new_frame      TB_FRAME_SAME, TB_FRAME_NEW (before expanding, every hypothesis with score > -inf becomes
 *                  live) or TB_FRAME_NEW_MERGE (Sec. 2.3, merging: first, hypotheses of a stream that have
 *                  emitted the same token sequence -- one transcript reached by different alignments -- are
 *                  merged: the first in slot order, i.e. the best of the previous step, stays, the others
 *                  become empty places; then as TB_FRAME_NEW).  Sequences are compared by length, graph
 *                  state and a 64-bit hash kept per hypothesis inside the batch from tb_beam_reset on.
 *   scores/states/live  device float / int32 / uint8 [B, K], updated in place
 *   out_parent/out_token  device int32 [B, K]
 * Errors: TB_ERR_INVALID_ARG (K > max_beam, tree full, ...), TB_ERR_CUDA.
 */
int tb_beam_step(tb_batch *b, const void *logits, int dtype, int32_t B, int32_t K, int64_t stream_stride,
                 int64_t hyp_stride, int32_t new_frame, float *scores, int32_t *states, uint8_t *live,
                 int32_t *out_parent, int32_t *out_token, void *stream);

/*
 * T frames of E expansions each in ONE launch (Sec. 2.3: fully GPU-based decoding without a host round trip per
 * step): exactly the sequence of tb_beam_step calls in which every hypothesis of stream i reads the row at element
 * offset i*stream_stride + t*frame_stride + e*row_stride (hyp_stride 0) and the first row of every frame is given
 * TB_FRAME_NEW, or TB_FRAME_NEW_MERGE when `merge` is non-zero; pruning as set by tb_batch_set_beam_prune.  Each
 * stream's block loops over its own expansions.  The tree receives T*E steps; out_parent / out_token hold those of
 * the last one.  A chunk of a longer utterance is one such call; the next call continues from the arrays.
 * Errors: as tb_beam_step (the tree must have room for T*E more steps).
 */
int tb_beam_frames(tb_batch *b, const void *logits, int dtype, int32_t B, int32_t K, int32_t T, int32_t E,
                   int64_t stream_stride, int64_t frame_stride, int64_t row_stride, int32_t merge, float *scores,
                   int32_t *states, uint8_t *live, int32_t *out_parent, int32_t *out_token, void *stream);

/*
 * Streaming beam decoding, slot by slot (Sec. 2.3: the hypotheses a stream holds at the end of a chunk -- their
 * place in the flattened tree, accumulated scores and graph states -- are kept and are what the next chunk continues,
 * merges and prunes; Sec. 2.2 para. 4: streams end and new ones start on their slots between chunks).
 * Every slot has its own hypothesis tree (a ring of max_tree_steps * max_beam / K steps inside the batch's tree
 * buffer) and its own position in it, so slots start, pause and end independently.  The caller's [n_slots, K] arrays
 * hold scores, graph states and liveness as for tb_beam_step.  A session: tb_beam_reset_slots(b, 0, NULL) for all
 * slots, or for the slots on which a new utterance starts (the caller also sets those slots' rows of the arrays:
 * score 0 / -inf..., state 0 or -1, as for an utterance's first tb_beam_step); then per chunk tb_beam_chunk; when a
 * stream has ended tb_apply_final_weights_slots and tb_beam_backtrace_slots give its result.  tb_beam_reset ends the
 * session (tb_beam_step / tb_beam_frames refuse to run during one, and tb_beam_chunk after them without a reset).
 *
 * tb_beam_reset_slots: n = 0 resets every slot; else `slots` is a host int32 array of n slot indices.  Device work
 *   on `stream` (position 0, empty token sequences).  Errors: TB_ERR_BAD_SLOT, TB_ERR_INVALID_ARG, TB_ERR_CUDA.
 * tb_beam_start_slots: tb_beam_reset_slots, which in the same launch also sets up those slots' rows of the caller's
 *   device arrays scores / states / live [n_slots, K] for an utterance's first step: hypothesis 0 with score 0 in state 0
 *   (state -1 on a slot without a graph, so call it after the slot's bind, on the same stream), the others with score
 *   -inf and state -1, live 0.  Errors: as tb_beam_reset_slots; TB_ERR_INVALID_ARG for K outside [1, max_beam].
 * tb_beam_chunk: for slot i, n_frames[i] (device int32 [n_slots], clamped to [0, chunk]; NULL: chunk) frames of E
 *   expansions, exactly as tb_beam_frames does them for a whole batch (every hypothesis of slot i reads the row at
 *   element offset i*stream_stride + t*frame_stride + e*row_stride; merge and pruning at frame starts); a slot with
 *   n_frames 0 is left alone (its out_parent / out_token rows are not written).  K must stay the same from one
 *   reset of all slots to the next.  Errors: TB_ERR_INVALID_ARG (no tree, K, a batch-wide tree in use), TB_ERR_CUDA.
 * tb_beam_backtrace_slots: as tb_beam_backtrace, each slot walked back to the start of its own utterance; an
 *   utterance longer than the slot's ring sets TB_STATUS_STEP_LIMIT and yields the tokens still in the ring.
 * tb_beam_backtrace_slot_list: the same for the n slots that `slots` (host int32 [n]) names, e.g. those whose streams
 *   have just ended: out_tokens device int32 [n, K, max_len], out_lens device int32 [n, K], row i for slots[i].
 *   Errors: TB_ERR_BAD_SLOT, TB_ERR_INVALID_ARG, TB_ERR_CUDA.
 * tb_apply_final_weights_slots: tb_apply_final_weights for the rows of the [n_slots, K] arrays that `slots` (host
 *   int32 [n]) names.
 */
int tb_beam_reset_slots(tb_batch *b, int32_t n, const int32_t *slots, void *stream);
int tb_beam_start_slots(tb_batch *b, int32_t n, const int32_t *slots, int32_t K, float *scores, int32_t *states, uint8_t *live,
                        void *stream);
int tb_beam_chunk(tb_batch *b, const void *logits, int dtype, int32_t n_slots, int32_t K, int32_t chunk, int32_t E,
                  int64_t stream_stride, int64_t frame_stride, int64_t row_stride, int32_t merge, const int32_t *n_frames,
                  float *scores, int32_t *states, uint8_t *live, int32_t *out_parent, int32_t *out_token, void *stream);
int tb_beam_backtrace_slots(tb_batch *b, int32_t n_slots, int32_t K, int32_t max_len, int32_t *out_tokens,
                            int32_t *out_lens, void *stream);
int tb_beam_backtrace_slot_list(tb_batch *b, int32_t n, const int32_t *slots, int32_t K, int32_t max_len, int32_t *out_tokens,
                                int32_t *out_lens, void *stream);
int tb_apply_final_weights_slots(tb_batch *b, int32_t n, const int32_t *slots, int32_t K, float *scores,
                                 const int32_t *states, void *stream);

/*
 * Pruning of the beam (Sec. 2.3 names it; the rule here is the usual threshold against the best hypothesis):
 * with delta >= 0, every tb_beam_step that starts a frame (TB_FRAME_NEW, TB_FRAME_NEW_MERGE) first -- after
 * the merge, if one was asked for -- turns every hypothesis of a stream whose score is below
 * fl(best score of the stream - delta) into an empty place.  A negative delta (the default) switches it off;
 * +inf prunes nothing.  Errors: TB_ERR_INVALID_ARG (NULL, NaN).
 */
int tb_batch_set_beam_prune(tb_batch *b, float delta);

/*
 * End of stream: charge every hypothesis the final weight of the graph state it stops in (Sec. 2.2 para. 2
 * lists a final weight per state; it is the loan of the unfinished partial match, negated, so a finished
 * hypothesis keeps the bonus of the phrases it completed and nothing else):
 * scores[i, k] = fl(scores[i, k] + fl(lambda_i * final(states[i, k]))) for stream i = 0..B-1 bound to a graph,
 * states[i, k] >= 0 and a score above -inf; everything else is left as it is.  Works on the [B, K] arrays of
 * tb_beam_step (re-rank afterwards if the order matters) and, with K = 1, on out_scores / out_states of
 * tb_greedy_decode or tb_stream_chunk.
 *   scores  device float [B, K], updated in place;  states  device int32 [B, K]
 * Errors: TB_ERR_INVALID_ARG, TB_ERR_CUDA; a state outside the graph sets TB_STATUS_BAD_STATE.
 */
int tb_apply_final_weights(tb_batch *b, int32_t B, int32_t K, float *scores, const int32_t *states, void *stream);

/*
 * Walk the hypothesis tree back from the hypotheses of the latest step and write each one's
 * non-blank tokens in emission order (Sec. 2.3: hypotheses live in a flattened tree).
 *   out_tokens  device int32 [B, K, max_len]; sequences longer than max_len are truncated
 *   out_lens    device int32 [B, K]: full lengths (0 for empty places)
 * Errors: TB_ERR_INVALID_ARG (no tree, no steps, K/B different from the steps recorded).
 */
int tb_beam_backtrace(tb_batch *b, int32_t B, int32_t K, int32_t max_len, int32_t *out_tokens,
                      int32_t *out_lens, void *stream);

/*
 * Unboosted greedy RNNT decoding that allocates nothing.  (The paper has no counterpart; this is
 * a service to one kind of caller.)
 *
 * Who needs it: code that is not allowed to allocate device memory at the moment it decodes --
 * a serving process whose device memory was divided up front among its models and that treats any
 * later cudaMalloc as a fault, or a latency-critical thread that cannot afford cudaMalloc because
 * it synchronises the device and would stall the other streams' decoding.  Such callers cannot use
 * tb_batch_create (it allocates the arena, the slot table and the status word), and without a
 * batch there is no graph, so this call decodes every stream as unbound (model id -1): per stream
 * exactly what tb_greedy_decode returns for a slot without a graph.
 *
 * The decode kernel's own working memory (one status word and one "unbound" slot record per
 * stream) lives in a fixed array inside the library, 33 KB, which every GPU that loads the library
 * holds until the process exits; hence the limit of TB_NOALLOC_MAX_STREAMS streams per call.  The
 * call makes no cudaMalloc / cudaFree and uses no allocating library routine.  Every call shares
 * that one array: the call clears what it needs to start from zero, in stream order, but two calls
 * that overlap on the GPU (different streams, or different host threads) race on it -- callers must
 * serialise their calls per device.  The first call on a device looks up the array's device address
 * (cudaGetSymbolAddress); make that first call outside any stream capture.
 *
 *   device       the GPU that holds the caller's buffers
 *   logits       device, dtype TB_BF16 or TB_F32, logical shape [B, T, S, vocab+1]
 *   strides      host int64 [4], element strides (any layout)
 *   lengths      device int32 [B] or NULL (= T)
 *   out_tokens / out_frames   device int32 [B, T*S]
 *   out_counts / out_states   device int32 [B] (states are all -1)
 *   out_scores   device float [B]
 *   out_status   device int32 [1] or NULL: receives the kernel's status word (TB_STATUS_* bits, 0 = fine)
 * Asynchronous on `stream` like the other decode calls.  Errors: TB_ERR_INVALID_ARG (B outside
 * [1, TB_NOALLOC_MAX_STREAMS], vocab outside [1, TB_MAX_VOCAB], bad dtype, NULL pointers, sizes
 * < 1), TB_ERR_CUDA.
 */
int tb_greedy_decode_noalloc(int device, const void *logits, int dtype, int32_t B, int32_t T, int32_t S,
                             int32_t vocab, const int64_t *strides, const int32_t *lengths,
                             int32_t *out_tokens, int32_t *out_frames, int32_t *out_counts, float *out_scores,
                             int32_t *out_states, int32_t *out_status, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* TB_H_ */
