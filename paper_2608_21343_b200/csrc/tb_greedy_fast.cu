// Pipelined greedy RNNT decode for packed bf16 logits: one persistent thread block per stream.
//
//   producer warp : streams the stream's frames (S rows each) from HBM into a shared-memory ring
//                   with bulk asynchronous copies (16-byte aligned supersets of each frame) that
//                   complete on an mbarrier;
//   helper warps  : reduce every row, ahead of time and independently of the graph state, to a
//                   summary {best root-boosted value y1, its token id1, an upper bound y2b on
//                   every other token's root-boosted value, the blank logit, ...};
//   decider warp  : the only sequential part -- walks the rows the decode visits, resolves each
//                   from its summary plus the few tokens boosted by the current non-root graph
//                   state, advances the graph state and the frame cursor, writes the outputs.
// The deciders share their warp scheduler with no helper: warps are spread over the SM's four
// schedulers by warp index, and every fourth warp that is neither a decider nor a producer just
// waits at the final barrier.
//
// Exactness.  Values follow the arithmetic contract (val = fl(x + fl(lambda * bonus)), ties to
// the lowest id).  y(v) = fl(x[v] + fl(lambda * w_root(cls v))) is the exact value of token v in
// the root state.  In a non-root state s every token whose class has no arc on the non-root part
// of the suffix chain ("plain" tokens) has value fl(x + fl(lambda * fl(D + w_root))) with D the
// summed suffix-link weights of the whole chain; in real arithmetic that is y + lambda*D, so the
// order among plain tokens is the order of y up to rounding.  The decider accepts the summary's
// winner as the best plain token only when y1 exceeds the bound on all other tokens by more
// than a margin tau that dominates every rounding error involved, or shows that no plain token
// can reach the best of {blank, the state's own tokens}; the tokens the chain boosts are always
// evaluated exactly; otherwise the whole row is rescanned exactly from shared memory.
//
// Long bound streams are decoded as two segments at once, each by a pipeline of its own (producer,
// helpers, decider, half of the ring), and merged at the end: see "segments" in the kernel.
//
// Every wait is bounded; a wait that runs out raises TB_STATUS_WAIT_TIMEOUT, makes all roles of
// the block leave their loops, and the block still waits (bounded) for its copies in flight.
#include "tb_fast_common.cuh"
#include "tb_launch.h"

namespace {

constexpr int kWarpsF = 20;     // warp 0 decider, warp 4 producer, warps 8/12/16 parked, 15 helpers
constexpr int kHelpers = kWarpsF - kWarpsF / 4;
constexpr int kThreadsF = kWarpsF * 32;
constexpr int kGroupDeep = 64;  // up to this many boosted tokens, the decider resolves eight rows per round, four lanes each
constexpr int kAllRowsDeep = 64; // all-rows mode in a state that just repeated itself: at most this many boosted tokens
constexpr int kStagesMax = 24;  // ring stages; each decider lane below this number owns one stage
constexpr uint32_t kSpinLimit = 1u << 20;
constexpr int kSegMinFrames = 128;  // streams at least this long are decoded as two segments (see the header)
constexpr int kSegWarm = 16;        // frames the second segment decodes before the first frame it answers for



// ---- mbarrier / bulk-copy primitives --------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait for the roles that are not latency critical: parks the warp between polls so that
// it does not take issue slots or shared-memory pipeline cycles from the decider.
__device__ __forceinline__ bool mbar_wait_parked(uint64_t* bar, uint32_t parity, volatile int* flags, int pipe, int32_t* status) {
  for (uint32_t it = 0; it < (kSpinLimit >> 2); ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    __nanosleep(256);
    if ((it & 7u) == 7u && flags[pipe]) return false;
  }
  flags[0] = 1; flags[1] = 1;
  atomicOr(status, TB_STATUS_WAIT_TIMEOUT);
  return false;
}
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst_smem)),
               "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

// Arrival without release ordering.  The decider uses it to hand a ring slot back: it has only
// read the slot, and every such read has completed (its value fed a ballot) before the arrival,
// so nothing needs to be made visible -- while a releasing arrival would also wait for the
// decider's earlier global stores (emitted tokens) to be acknowledged by the memory system.
__device__ __forceinline__ void mbar_arrive_relaxed_addr(uint32_t bar_addr) {
  asm volatile("mbarrier.arrive.relaxed.cta.shared::cta.b64 _, [%0];" ::"r"(bar_addr) : "memory");
}

struct Smem {  // byte offsets into dynamic shared memory, computed identically on host and device
  int ring, bars, summ, cls16, tokcb, rootcw, rootdst, lbuf, cls_seen, tokidx, emit, misc, cache, total;
  int lbuf_sz, cls_seen_sz, tokidx_sz;   // the deciders' private areas exist once per segment, this far apart
};
__host__ __device__ inline int up16(int x) { return (x + 15) & ~15; }
__host__ __device__ inline Smem carve(int nst, int slot_bytes, int V, int C, int cache_bytes, int npipes, int own_lists) {
  Smem s;
  int o = 0;
  s.ring = o; o += nst * slot_bytes;
  s.bars = o; o += up16(8 * (2 * nst));
  s.summ = o; o += nst * kSumStageBytes;
  s.cls16 = o; o += up16(2 * V);
  s.tokcb = o; o += up16(4 * V);            // lambda * root-arc weight of every token (0 without a root arc)
  s.rootcw = o; o += up16(4 * C);
  s.rootdst = o; o += up16(4 * C);
  // own_lists == 0: every bound graph's resolved lists are in the cache, no decider ever builds or stages a list
  s.lbuf_sz = own_lists ? up16(8 * (V + 4)) : 16; s.cls_seen_sz = own_lists ? up16(2 * C) : 0; s.tokidx_sz = up16(2 * V);
  s.lbuf = o; o += npipes * s.lbuf_sz;         // boosted-token list of the current state when it is not read from the cache
  s.cls_seen = o; o += npipes * s.cls_seen_sz; // class -> position in lbuf while a list is being built
  s.tokidx = o; o += npipes * s.tokidx_sz;     // token -> position in the current list (filled only for an exact rescan)
  s.emit = o; o += npipes * 32 * 8;            // emitted (token, frame) pairs waiting for a coalesced store
  s.misc = o; o += 96;
  s.cache = o; o += up16(cache_bytes);
  s.total = o;
  return s;
}

struct FastParams {
  TbDecodeParams d;
  int32_t nst, slot_bytes, cache_bytes;  // cache_bytes > 0: every bound graph's lists (resolved, else state records + token arcs) fit in shared memory
  const unsigned char* tensor_lo;        // first / one-past-last byte of the logits tensor
  const unsigned char* tensor_hi;
  // two-segment decode: per stream, what the second segment emits / adds to the score / its state at every frame start
  int32_t npipes;                        // 2: long bound streams are decoded as two segments
  int32_t own_lists;                     // 0: no graph of the batch needs a list built or staged outside the cache
  int32_t scr_cap;                       // frames * S
  int32_t* scr_tok;                      // [n_streams][2 * scr_cap]: tokens, then frames
  float* scr_val;                        // [n_streams][scr_cap]: value of every row the segment visits, in order
  int4* scr_trace;                       // [n_streams][frames + 1]: {state, tokens so far, values so far} at each frame start
};


// ---- decider ------------------------------------------------------------------------------------

// Chain walk for graphs without resolved lists: closest chain state first, a class already
// listed by a closer state is shadowed.  acc = suffix-link weights crossed so far, in walk order.
// The list is padded to a multiple of four with sentinels (blank column, lb = -inf).
__device__ __forceinline__ void build_list(const TbStateRec* strec, const TbTokEnt* tokent, int n_states, int max_depth,
                                           int s, float lam, float R, int V, TbRsEnt* lbuf, int16_t* cls_seen,
                                           const uint16_t* cls16, CurList& L, int lane, int32_t* status) {
  int n = 0;
  float acc = 0.0f;
  int u = s;
  if (u < 0 || u >= n_states) { if (lane == 0) atomicOr(status, TB_STATUS_BAD_STATE); u = 0; }
  TbStateRec rec{0, 0, 0, 0.0f};
  if (u != 0) rec = strec[u];
  for (int it = 0; u != 0; ++it) {
    if (it > max_depth + 1) { if (lane == 0) atomicOr(status, TB_STATUS_WALK_TOO_DEEP); break; }
    // the next chain state's record is requested before this state's arcs are: the two trips to L2 overlap
    const int nu = rec.fail;
    TbStateRec nrec = rec;
    if (nu > 0 && nu < n_states) nrec = strec[nu];
    const int n_start = n;
    TbTokEnt ahead{0u, 0.0f, 0, 0};
    if (rec.tok_begin + lane < rec.tok_end) ahead = tokent[rec.tok_begin + lane];
    for (int e0 = rec.tok_begin; e0 < rec.tok_end; e0 += 32) {
      const int e = e0 + lane;
      const bool have = e < rec.tok_end;
      const TbTokEnt ent = ahead;                           // (the next 32 arcs are requested before these are dealt with)
      if (e + 32 < rec.tok_end) ahead = tokent[e + 32];
      const int c = static_cast<int>(ent.tok_cls >> 16);
      const int seen = have ? cls_seen[c] : 0;
      const bool fresh = have && (seen < 0 || seen >= n_start);   // same class again only as a sibling from this state
      const unsigned mask = __ballot_sync(0xffffffffu, fresh);
      if (fresh) {
        const int pos = n + __popc(mask & ((1u << lane) - 1u));
        lbuf[pos].dst_tok = (static_cast<uint32_t>(ent.dst) << TB_RS_TOK_BITS) | (2u * (ent.tok_cls & 0xFFFFu));
        lbuf[pos].lb = __fmul_rn(lam, __fadd_rn(acc, ent.w));
        cls_seen[c] = static_cast<int16_t>(pos);
      }
      n += __popc(mask);
      __syncwarp();
    }
    acc = __fadd_rn(acc, rec.bw);
    u = (nu > 0 && nu < n_states) ? nu : 0;
    rec = nrec;
  }
  for (int i = lane; i < n; i += 32) cls_seen[cls16[(lbuf[i].dst_tok & kTokMask) >> 1]] = -1;   // leave the map clean
  const int n_pad = (n + 3) & ~3;
  if (lane < n_pad - n) { lbuf[n + lane].dst_tok = 2u * static_cast<uint32_t>(V); lbuf[n + lane].lb = -INFINITY; }
  __syncwarp();
  L.addr = smem_u32(lbuf); L.n = n_pad; L.sorted = false; L.D = acc;
  L.bmag = fabsf(lam) * (fabsf(acc) + R);
}

__device__ __forceinline__ void prog_publish(volatile int* flags, int v) { flags[2] = v; }


template <int NIT, bool NORM>
__global__ void __launch_bounds__(kThreadsF, 1) k_greedy_fast(FastParams P) {
  extern __shared__ __align__(128) unsigned char dyn[];
  const TbDecodeParams& p = P.d;
  const int V = p.V, C = p.C, S = p.S, W = V + 1, nst = P.nst;
  const Smem so = carve(nst, P.slot_bytes, V, C, P.cache_bytes, P.npipes, P.own_lists);
  unsigned char* ring = dyn + so.ring;
  uint64_t* full = reinterpret_cast<uint64_t*>(dyn + so.bars);
  uint64_t* freeb = full + nst;
  const uint32_t summ_a = smem_u32(dyn + so.summ);
  uint16_t* cls16 = reinterpret_cast<uint16_t*>(dyn + so.cls16);
  float* tokcb = reinterpret_cast<float*>(dyn + so.tokcb);
  float* rootcb = reinterpret_cast<float*>(dyn + so.ring + 256);   // per class, only while the tables are set up (the ring is not in use yet)
  float* rootcw = reinterpret_cast<float*>(dyn + so.rootcw);
  int32_t* rootdst = reinterpret_cast<int32_t*>(dyn + so.rootdst);
  volatile int* flags = reinterpret_cast<volatile int*>(dyn + so.misc);        // [2] stop flag per segment; [2] second segment's progress
  int* seg_res = reinterpret_cast<int*>(dyn + so.misc + 32);                     // what the two deciders leave for the final merge
  float* root_stats = reinterpret_cast<float*>(dyn + so.misc + 16);   // beta_min, beta_max, R

  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const TbSlotRec rec = p.slots[b];
  const bool bound = rec.n_states > 0;
  const bool resolved = bound && rec.n_rsent >= 0;
  const bool cached = bound && P.cache_bytes > 0;
  const GraphPtrs g = graph_of(p.arena, rec);
  const float lam = bound ? rec.lambda : 0.0f;
  const unsigned char* blob = p.arena + rec.blob_off;

  int end = p.lengths ? p.lengths[b] : p.frames;
  end = max(0, min(end, p.frames));
  if (bound && !P.own_lists && !(resolved && cached)) {      // the launch was laid out without room for this graph's lists
    if (tid == 0) {
      atomicOr(p.status, TB_STATUS_BAD_STATE);
      p.out_counts[b] = 0; p.out_scores[b] = 0.0f; p.out_states[b] = 0;
      if (p.out_cursors) p.out_cursors[b] = 0;
    }
    return;
  }

  // ---- set-up: tables, root vectors, graph cache, barriers ----------------------------------------
  for (int v = tid; v < V; v += kThreadsF) {
    cls16[v] = static_cast<uint16_t>(p.cls[v]);
    reinterpret_cast<int16_t*>(dyn + so.tokidx)[v] = -1;
    if (P.npipes == 2) reinterpret_cast<int16_t*>(dyn + so.tokidx + so.tokidx_sz)[v] = -1;
  }
  for (int c = tid; c < C; c += kThreadsF) {
    rootcb[c] = 0.0f; rootcw[c] = 0.0f; rootdst[c] = 0;
    if (P.own_lists) {
      reinterpret_cast<int16_t*>(dyn + so.cls_seen)[c] = -1;
      if (P.npipes == 2) reinterpret_cast<int16_t*>(dyn + so.cls_seen + so.cls_seen_sz)[c] = -1;
    }
  }
  for (int i = tid; i < nst * kSumStageBytes / 4; i += kThreadsF) reinterpret_cast<uint32_t*>(dyn + so.summ)[i] = 0u;   // no sequence word matches yet
  if (tid == 0) {
    flags[0] = 0; flags[1] = 0; flags[2] = 0;
    for (int i = 0; i < nst; ++i) { mbar_init(&full[i], 1); mbar_init(&freeb[i], S + 1); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (cached) {
    // the lists the decider reads are the tail of the blob: one contiguous 16-byte aligned range
    const int from = resolved ? rec.off_rsrec : rec.off_strec;
    const uint4* src = reinterpret_cast<const uint4*>(blob + from);
    uint4* dst = reinterpret_cast<uint4*>(dyn + so.cache);
    for (int i = tid; i < ((rec.blob_bytes - from) >> 4); i += kThreadsF) dst[i] = src[i];
  }
  __syncthreads();
  if (bound) {
    const int e = g.arc_begin[1];
    for (int a = g.arc_begin[0] + tid; a < e; a += kThreadsF) {
      const int c = g.arc_cls[a];
      const float wv = __fadd_rn(0.0f, g.arc_w[a]);        // the walk's fl(acc + w) with acc = 0
      rootcw[c] = wv; rootcb[c] = __fmul_rn(lam, wv); rootdst[c] = g.arc_dst[a];
    }
  }
  __syncthreads();
  for (int v = tid; v < V; v += kThreadsF) tokcb[v] = rootcb[cls16[v]];
  {
    // extremes of the root arcs' lambda * w (tokens without a root arc have beta = 0) and of |w|
    float bmin = 0.0f, bmax = 0.0f, R = 0.0f;
    if (bound) {
      const int e = g.arc_begin[1];
      for (int a = g.arc_begin[0] + tid; a < e; a += kThreadsF) {
        const float wv = __fadd_rn(0.0f, g.arc_w[a]);
        const float cb = __fmul_rn(lam, wv);
        bmin = fminf(bmin, cb); bmax = fmaxf(bmax, cb); R = fmaxf(R, fabsf(wv));
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      bmin = fminf(bmin, __shfl_xor_sync(0xffffffffu, bmin, off));
      bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, off));
      R = fmaxf(R, __shfl_xor_sync(0xffffffffu, R, off));
    }
    float* part = reinterpret_cast<float*>(dyn + so.ring);   // the ring is not in use yet (3 floats per warp)
    if (lane == 0) { part[3 * warp] = bmin; part[3 * warp + 1] = bmax; part[3 * warp + 2] = R; }
    __syncthreads();
    if (tid == 0) {
      for (int w2 = 1; w2 < kWarpsF; ++w2) {
        bmin = fminf(bmin, part[3 * w2]); bmax = fmaxf(bmax, part[3 * w2 + 1]); R = fmaxf(R, part[3 * w2 + 2]);
      }
      root_stats[0] = bmin; root_stats[1] = bmax; root_stats[2] = R;
    }
  }
  __syncthreads();

  const unsigned char* base = reinterpret_cast<const unsigned char*>(p.logits) + 2 * static_cast<int64_t>(b) * p.sb;
  const int64_t frame_stride_bytes = 2 * p.st;
  const int row_bytes = 2 * W;
  const int frame_bytes = S * row_bytes;
  const int lead0 = static_cast<int>(reinterpret_cast<uintptr_t>(base) & 15);
  const int lead_step = static_cast<int>(frame_stride_bytes & 15);

  // ---- segments ------------------------------------------------------------------------------------------
  // A long bound stream is decoded by two pipelines at once (each: producer, helpers, decider, a share of the
  // ring).  Pipeline 0 starts at frame 0.  Pipeline 1 starts kSegWarm frames before frame f_mid in the root
  // state and answers for the frames from f_mid on; from there it records, at every frame start, its graph
  // state and how much it has emitted.  The decode from a given (frame start, graph state) is a function of
  // those two alone, so once pipeline 0, which carries the true state, stands at a frame start >= f_mid in the
  // state pipeline 1 recorded there, the rest of pipeline 1's output is the true continuation; until then
  // pipeline 0 just keeps decoding.  The merge after the final barrier appends that continuation.
  // (an unbound stream has no graph state: its second pipeline starts exactly in the true state, with no
  // warm-up, and the two meet at f_mid; it is split as well because one pipeline's ring turns over too slowly
  // to keep the copies flowing)
  const bool seg = P.npipes == 2 && end >= kSegMinFrames;
  const int warm = bound ? kSegWarm : 0;
  const int f_mid = seg ? (end + warm) / 2 : end;
  // this warp's pipeline: warps 0 / 4 (decider, producer) and the first helpers belong to 0; warps 8 / 12 and the rest to 1
  const int vw = warp;
  const int hid_all = vw - 1 - (vw >> 2);                // helper index over the warps that are not multiples of 4
  const int nh0 = seg ? (kHelpers + 1) / 2 : kHelpers;
  const int pipe = !seg ? 0 : ((vw & 3) == 0 ? (vw >= 8 ? 1 : 0) : (hid_all >= nh0 ? 1 : 0));
  const int nst0 = seg ? nst / 2 : nst;
  const int pst_base = pipe ? nst0 : 0;                      // first ring stage of the pipeline
  const int pnst = pipe ? nst - nst0 : nst0;
  const int pf0 = pipe ? f_mid - warm : 0;                   // first frame the pipeline fetches and decodes
  unsigned char* pring = ring + static_cast<size_t>(pst_base) * P.slot_bytes;
  uint64_t* pfull = full + pst_base;
  uint64_t* pfree = freeb + pst_base;
  const uint32_t psumm_a = summ_a + pst_base * kSumStageBytes;

  if (vw == 4 || (seg && vw == 12)) {
    // ================================ producer ================================================
    int issued = pf0, st = 0, use = 0;
    for (int f = pf0; f < end; ++f) {
      if (flags[pipe]) break;
      if (use > 0 && !mbar_wait_parked(&pfree[st], (use - 1) & 1, flags, pipe, p.status)) break;
      const unsigned char* src = base + static_cast<int64_t>(f) * frame_stride_bytes;
      const int lead = static_cast<int>(reinterpret_cast<uintptr_t>(src) & 15);
      const unsigned char* a0 = src - lead;
      const uint32_t bytes = static_cast<uint32_t>(up16(lead + frame_bytes));
      unsigned char* dst = pring + static_cast<size_t>(st) * P.slot_bytes;
      if (a0 >= P.tensor_lo && a0 + bytes <= P.tensor_hi) {
        if (lane == 0) { mbar_arrive_expect_tx(&pfull[st], bytes); bulk_load(dst, a0, bytes, &pfull[st]); }
      } else {  // the aligned superset would leave the tensor: copy the frame's own elements
        const uint16_t* s16 = reinterpret_cast<const uint16_t*>(src);
        uint16_t* d16 = reinterpret_cast<uint16_t*>(dst + lead);
        for (int i = lane; i < S * W; i += 32) d16[i] = __ldg(s16 + i);
        __syncwarp();
        if (lane == 0) mbar_arrive(&pfull[st]);
      }
      issued = f + 1;
      if (++st == pnst) { st = 0; ++use; }
      __syncwarp();
    }
    // no copy may be in flight when the block exits
    for (int f = max(pf0, issued - pnst); f < issued; ++f) {
      const int fl = f - pf0, fs = fl % pnst;
      for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(&pfull[fs], (fl / pnst) & 1); ++it) {}
    }
  } else if ((vw & 3) != 0) {
    // ================================ helpers =================================================
    const int ph0 = pipe ? nh0 : 0, pnh = seg ? (pipe ? kHelpers - nh0 : nh0) : kHelpers;
    const int hid = hid_all - ph0;                        // 0 .. pnh-1 within the pipeline
    HelperCtx h;
    h.cls16 = cls16; h.tokcb = tokcb; h.rootcw = rootcw; h.rootdst = rootdst; h.V = V; h.nit = (V + 255) / 256;
    h.beta_min = root_stats[0]; h.beta_max = root_stats[1]; h.dbeta = __fsub_rn(root_stats[1], root_stats[0]);
    h.bmag_max = fabsf(lam) * ((bound ? rec.d_max : 0.0f) + root_stats[2]);
    // rows are dealt round-robin: this warp takes rows hid, hid + pnh, ... of the pipeline's frames, in order
    int fl = hid / S, k = hid - fl * S;                   // frame (counted from the pipeline's first) and row in frame
    int st = fl % pnst;
    uint32_t ph = (fl / pnst) & 1;
    int f = pf0 + fl;
    int lead = (lead0 + f * lead_step) & 15;
    for (; f < end;) {
      if (!mbar_wait_parked(&pfull[st], ph, flags, pipe, p.status)) break;
      const unsigned char* slot = pring + static_cast<size_t>(st) * P.slot_bytes;
      summarize_row<NIT, NORM>(h, slot, lead + k * row_bytes, psumm_a + st * kSumStageBytes + k * 32, static_cast<uint32_t>(f) + 1u, lane,
                               psumm_a + st * kSumStageBytes + kSMax * 32 + 4 * k);
      if (lane == 0) mbar_arrive(&pfree[st]);
      k += pnh;
      while (k >= S) {                                      // on to a later frame
        k -= S; ++f;
        lead = (lead + lead_step) & 15;
        if (++st == pnst) { st = 0; ph ^= 1u; }
      }
    }
  } else if (vw == 0 || (seg && vw == 8)) {
    // ================================ decider =================================================
    // Works in rounds over a window of eight frames.  The warp is eight groups of four lanes; group q
    // stands for frame t + q.  A round resolves rows in parallel under the current graph state and then
    // consumes as many of them, in decode order, as the state allows:
    //   shared mode (the usual case: the state's chain boosts a few tokens and the last token changed
    //     the state): group q resolves one row -- group 0 the current row (t, k), group q >= 1 row
    //     (t + q, 0), the row the decode reaches there if everything before it is blank; the four lanes
    //     share the boosted tokens and combine with two shuffles.  One ballot tells how many leading
    //     rows are blank; they are consumed at once and the first row that selects a token ends the
    //     round, because the graph state changes there.
    //   all-rows mode (no boosted tokens -- root state or unboosted stream -- or the last token left the
    //     state unchanged): lane ql of group q resolves row (t + q, ql) on its own, so a round can walk
    //     through tokens too, as long as they leave the state unchanged.
    //   wide mode (many boosted tokens): all 32 lanes share them and resolve the current row only.
    const float R = root_stats[2];
    const uint32_t ring_a = smem_u32(pring), freeb_a = smem_u32(pfree);
    const uint32_t summ_a = psumm_a;                        // (shadows the block-wide base: this pipeline's stages)
    const int nst = pnst;
    const uint32_t cache_a = smem_u32(dyn + so.cache);
    TbRsEnt* lbuf = reinterpret_cast<TbRsEnt*>(dyn + so.lbuf + pipe * so.lbuf_sz);
    int16_t* cls_seen = reinterpret_cast<int16_t*>(dyn + so.cls_seen + pipe * so.cls_seen_sz);
    int16_t* tokidx = reinterpret_cast<int16_t*>(dyn + so.tokidx + pipe * so.tokidx_sz);
    int2* emit_buf = reinterpret_cast<int2*>(dyn + so.emit + pipe * 256);
    const TbStateRec* strec = cached && !resolved ? reinterpret_cast<const TbStateRec*>(dyn + so.cache)
                                                  : reinterpret_cast<const TbStateRec*>(blob + rec.off_strec);
    const TbTokEnt* tokent = cached && !resolved ? reinterpret_cast<const TbTokEnt*>(dyn + so.cache + (rec.off_tokent - rec.off_strec))
                                                 : reinterpret_cast<const TbTokEnt*>(blob + rec.off_tokent);
    const TbRsRec* rsrec_g = reinterpret_cast<const TbRsRec*>(blob + rec.off_rsrec);
    const TbRsEnt* rsent_g = reinterpret_cast<const TbRsEnt*>(blob + rec.off_rsent);
    const uint32_t rsent_cache_a = cache_a + static_cast<uint32_t>(rec.off_rsent - rec.off_rsrec);

    CurList L;
    L.addr = smem_u32(lbuf); L.n = 0; L.sorted = true; L.D = 0.0f; L.bmag = fabsf(lam) * R;

    const int q = lane >> 2, ql = lane & 3;                 // group and lane within the group
    constexpr int kWin = 8;                                 // frames per window (the launcher guarantees nst >= kWin)
    int t = pf0, k = 0, s = bound ? 0 : -1, n_out = 0, st = 0, lead = (lead0 + pf0 * lead_step) & 15;
    float score = 0.0f;
    // pipeline 1 writes to scratch memory and keeps a log: rec_on
    const bool rec_on = pipe == 1, chk_on = seg && pipe == 0;
    const int out_cap = rec_on ? P.scr_cap : p.out_cap;
    int32_t* out_tok = rec_on ? P.scr_tok + 2 * static_cast<int64_t>(b) * P.scr_cap : p.out_tokens + static_cast<int64_t>(b) * p.out_cap;
    int32_t* out_frm = rec_on ? out_tok + P.scr_cap : p.out_frames + static_cast<int64_t>(b) * p.out_cap;
    float* vlog = rec_on ? P.scr_val + static_cast<int64_t>(b) * P.scr_cap : nullptr;
    int4* trace = seg ? P.scr_trace + static_cast<int64_t>(b) * (p.frames + 1) : nullptr;
    int nv = 0;                                             // values logged so far
    int tc = -1;                                            // pipeline 0: the frame start at which it met pipeline 1's record
    if (rec_on && pf0 >= f_mid && lane == 0) { trace[pf0] = make_int4(s, 0, 0, 0); __threadfence_block(); flags[2] = pf0 + 1; }
    const int max_rounds = p.frames * S + p.frames + 8;
    uint32_t spins = 0;
    bool failed = false, stable = false, no_allrows = false;
    const bool fast_ok = bound && cached && resolved;       // the branch-free round reads lists from the cache only
    for (int it = 0; t < end; ++it) {
      if (it >= max_rounds) { if (lane == 0) atomicOr(p.status, TB_STATUS_STEP_LIMIT); break; }
      // ---- mode and this lane's row --------------------------------------------------------------------
      const bool allrows = !no_allrows && (L.n == 0 || (stable && L.n <= kAllRowsDeep));
      const bool wide = !allrows && L.n > kGroupDeep;
      // ---- the usual round, without branches -----------------------------------------------------------
      // A lone warp pays tens of cycles for every branch whose condition was only just computed (nothing
      // else can issue while it resolves).  The usual round -- shared mode, lists in the cache -- is therefore
      // computed here as straight-line code with selects; everything unusual (a row that needs the rescan,
      // nothing ready, a state out of range) is collected in one
      // flag, and then the round falls through, having changed nothing, to the general code below.
      if (fast_ok && !allrows && !wide && !(chk_on && t >= f_mid)) {
      fast_again:
        const int rk = q == 0 ? k : 0;
        int stq = st + q; stq -= stq >= nst ? nst : 0;
        const uint32_t sum_a = summ_a + stq * kSumStageBytes + rk * 32u;
        const uint4 q1 = lds_v4_volatile(sum_a + 16u);
        const uint4 q0 = lds_v4_volatile(sum_a);
        const uint32_t row_a = ring_a + stq * P.slot_bytes + ((lead + q * lead_step) & 15) + rk * row_bytes;
        const bool ready = t + q < end && q1.w == static_cast<uint32_t>(t + q) + 1u;
        const float y1 = __uint_as_float(q0.x), y2b = __uint_as_float(q0.y), xb = __uint_as_float(q0.z), x1 = __uint_as_float(q0.w);
        const float lse = NORM ? lds_f32_volatile(summ_a + stq * kSumStageBytes + kSMax * 32u + 4u * rk) : 0.0f;
        const uint32_t id1x2 = 2u * (q1.z & 0xFFFFu);
        // this lane's entries ql, ql + 4, ...: the cached lists are sorted by token, so within a lane a strict
        // comparison keeps the lowest token among equal values; bit 0 of an entry word is free (2 * token) and
        // carries "this is the summary's winner" through the reduction
        float wv = -INFINITY;
        uint32_t wdt = 2u * static_cast<uint32_t>(V);
        {
          int i = ql;
          for (; i + 12 < L.n; i += 16) {                     // four entries in flight, compared as a tree
            const uint32_t ea = L.addr + 8u * i;
            const uint2 e0 = lds_v2_nv(ea), e1 = lds_v2_nv(ea + 32u), e2 = lds_v2_nv(ea + 64u), e3 = lds_v2_nv(ea + 96u);
            const uint32_t t0 = e0.x & kTokMask, t1 = e1.x & kTokMask, t2 = e2.x & kTokMask, t3 = e3.x & kTokMask;
            const float v0 = __fadd_rn(bf16_bits_to_float(lds_u16_nv(row_a + t0)), __uint_as_float(e0.y));
            const float v1 = __fadd_rn(bf16_bits_to_float(lds_u16_nv(row_a + t1)), __uint_as_float(e1.y));
            const float v2 = __fadd_rn(bf16_bits_to_float(lds_u16_nv(row_a + t2)), __uint_as_float(e2.y));
            const float v3 = __fadd_rn(bf16_bits_to_float(lds_u16_nv(row_a + t3)), __uint_as_float(e3.y));
            const uint32_t seen = ((t0 == id1x2 || t1 == id1x2 || t2 == id1x2 || t3 == id1x2) ? 1u : 0u) | (wdt & 1u);
            const bool b01 = v1 > v0, b23 = v3 > v2;
            const float va = b01 ? v1 : v0, vb = b23 ? v3 : v2;
            const uint32_t da = b01 ? e1.x : e0.x, db = b23 ? e3.x : e2.x;
            const bool bab = vb > va;
            const float vm = bab ? vb : va;
            const uint32_t dm = bab ? db : da;
            const bool bw = vm > wv;
            wv = bw ? vm : wv; wdt = (bw ? dm : wdt) | seen;
          }
          for (; i + 4 < L.n; i += 8) {                      // two entries in flight
            const uint2 e0 = lds_v2_nv(L.addr + 8u * i), e1 = lds_v2_nv(L.addr + 8u * (i + 4));
            const uint32_t x0 = lds_u16_nv(row_a + (e0.x & kTokMask)), x1r = lds_u16_nv(row_a + (e1.x & kTokMask));
            const float v0 = __fadd_rn(bf16_bits_to_float(x0), __uint_as_float(e0.y));
            const float v1 = __fadd_rn(bf16_bits_to_float(x1r), __uint_as_float(e1.y));
            const uint32_t d0 = e0.x | ((e0.x & kTokMask) == id1x2 ? 1u : 0u), d1 = e1.x | ((e1.x & kTokMask) == id1x2 ? 1u : 0u);
            const bool b01 = v1 > v0;                         // e1's token is the larger one
            const float vm = b01 ? v1 : v0; const uint32_t dm = b01 ? d1 : d0;
            const uint32_t seen = (d0 | d1 | wdt) & 1u;
            const bool bw = vm > wv;
            wv = bw ? vm : wv; wdt = (bw ? dm : wdt) | seen;
          }
          if (i < L.n) {
            const uint2 e0 = lds_v2_nv(L.addr + 8u * i);
            const float v0 = __fadd_rn(bf16_bits_to_float(lds_u16_nv(row_a + (e0.x & kTokMask))), __uint_as_float(e0.y));
            const uint32_t d0 = e0.x | ((e0.x & kTokMask) == id1x2 ? 1u : 0u);
            const uint32_t seen = (d0 | wdt) & 1u;
            const bool bw = v0 > wv;
            wv = bw ? v0 : wv; wdt = (bw ? d0 : wdt) | seen;
          }
        }
        // the group's best: every lane fetches the other three lanes' results at once and reduces them itself
        // (minima and maxima only; no predicate until the end).  Equal best values in two lanes -- the lowest
        // token would decide -- are left to the general code.
        bool tie;
        {
          const float o1 = __shfl_xor_sync(0xffffffffu, wv, 1), o2 = __shfl_xor_sync(0xffffffffu, wv, 2), o3 = __shfl_xor_sync(0xffffffffu, wv, 3);
          const uint32_t d1 = __shfl_xor_sync(0xffffffffu, wdt, 1), d2 = __shfl_xor_sync(0xffffffffu, wdt, 2), d3 = __shfl_xor_sync(0xffffffffu, wdt, 3);
          const float hi1 = fmaxf(wv, o1), lo1 = fminf(wv, o1), hi2 = fmaxf(o2, o3), lo2 = fminf(o2, o3);
          const float gm = fmaxf(hi1, hi2), second = fmaxf(fminf(hi1, hi2), fmaxf(lo1, lo2));
          tie = second == gm;
          const uint32_t seen = (wdt | d1 | d2 | d3) & 1u;
          const uint32_t dsel = wv == gm ? wdt : (o1 == gm ? d1 : (o2 == gm ? d2 : d3));
          wdt = (dsel & ~1u) | seen;
          wv = gm;
        }
        const bool in_deep = (wdt & 1u) != 0u;
        int wtok = static_cast<int>((wdt & kTokMask) >> 1);
        int wnext = static_cast<int>(wdt >> TB_RS_TOK_BITS);
        // the best plain token (see the general code): exact when it clears the others by the margin, else bounded
        const bool plain_ok = !in_deep && ((q1.z & kSumGap) != 0 || s <= 0);
        const float nd = __fadd_rn(x1, __fmul_rn(lam, __fadd_rn(L.D, __uint_as_float(q1.x))));
        const int id1 = static_cast<int>(id1x2 >> 1);
        const float ub = (in_deep ? y2b : y1) + lam * L.D;
        const float tau = (fabsf(y1) + 4.0f * L.bmag) * 3.814697265625e-6f + 1e-30f;
        const bool rescan = (q1.z & kSumOvf) != 0 || tie || (!plain_ok && !(fmaxf(wv, xb) > ub + tau)) || (plain_ok && nd == wv);
        const bool take_plain = plain_ok && nd > wv;
        wv = take_plain ? nd : wv; wtok = take_plain ? id1 : wtok; wnext = take_plain ? static_cast<int>(q1.y) : wnext;
        const bool is_blank = ready && !rescan && !(wv >= xb);
        const unsigned blank_m = __ballot_sync(0xffffffffu, is_blank) & 0x11111111u;
        const unsigned stop_m = ~blank_m & 0x11111111u;
        const int nb = stop_m ? (__ffs(stop_m) - 1) >> 2 : kWin;
        const int jl = 4 * min(nb, kWin - 1);
        const bool j_ready = __shfl_sync(0xffffffffu, ready, jl);
        const bool j_rescan = __shfl_sync(0xffffffffu, rescan, jl);
        const uint32_t j_tn = __shfl_sync(0xffffffffu, (static_cast<uint32_t>(wnext) << TB_RS_TOK_BITS) | static_cast<uint32_t>(wtok), jl);
        const int j_tok = static_cast<int>(j_tn & kTokMask), j_next = static_cast<int>(j_tn >> TB_RS_TOK_BITS);
        // what a row adds to the score: its selected value, less the row's normaliser when rows are normalised (the
        // normaliser is common to all candidates of a row, so it is taken off after the selection)
        const float xbs = NORM ? __fsub_rn(xb, lse) : xb;
        const float j_val = __shfl_sync(0xffffffffu, NORM ? __fsub_rn(wv, lse) : wv, jl);
        const float xb0 = __shfl_sync(0xffffffffu, xbs, 0), xb1 = __shfl_sync(0xffffffffu, xbs, 4);
        const float xb2 = __shfl_sync(0xffffffffu, xbs, 8), xb3 = __shfl_sync(0xffffffffu, xbs, 12);
        const float xb4 = __shfl_sync(0xffffffffu, xbs, 16), xb5 = __shfl_sync(0xffffffffu, xbs, 20);
        const float xb6 = __shfl_sync(0xffffffffu, xbs, 24), xb7 = __shfl_sync(0xffffffffu, xbs, 28);
        const bool took = nb < kWin && j_ready;             // the row after the blanks selects a token
        const bool rare = (nb == 0 && !took) || (took && j_rescan) || (took && (j_next < 0 || j_next >= rec.n_states));
        if (!rare) {
          // ---- commit ----
          score = nb > 0 ? __fadd_rn(score, xb0) : score;
          score = nb > 1 ? __fadd_rn(score, xb1) : score;
          score = nb > 2 ? __fadd_rn(score, xb2) : score;
          score = nb > 3 ? __fadd_rn(score, xb3) : score;
          score = nb > 4 ? __fadd_rn(score, xb4) : score;
          score = nb > 5 ? __fadd_rn(score, xb5) : score;
          score = nb > 6 ? __fadd_rn(score, xb6) : score;
          score = nb > 7 ? __fadd_rn(score, xb7) : score;
          score = took ? __fadd_rn(score, j_val) : score;
          if (lane == 0 && took) emit_buf[n_out & 31] = make_int2(j_tok, t + nb);
          {
            // a token that fills the staging block sends it out (every lane reads its slot in any case: no branch)
            const bool full_blk = took && (n_out & 31) == 31;
            __syncwarp();
            const int2 e = emit_buf[lane];
            const int o = (n_out & ~31) + lane;
            if (full_blk && o < out_cap) { out_tok[o] = e.x; out_frm[o] = e.y; }
            __syncwarp();
          }
          const int k_row = nb == 0 ? k : 0;
          const bool closes = took && k_row + 1 == S;       // the token fills its frame
          const int adv = nb + (closes ? 1 : 0);
          const int tnext = took ? j_next : s;
          n_out += took ? 1 : 0;
          if (rec_on) {
            if ((lane & 3) == 0 && q < nb) vlog[nv + q] = xbs;
            if (took && lane == 0) vlog[nv + nb] = j_val;
            if (lane < adv && t + lane + 1 >= f_mid)
              trace[t + lane + 1] = make_int4(lane >= nb ? tnext : s, n_out - ((took && lane < nb) ? 1 : 0), nv + lane + 1, 0);
            nv += nb + (took ? 1 : 0);
          }
          k = (took && !closes) ? k_row + 1 : 0;
          {
            int sr = st + lane; sr -= sr >= nst ? nst : 0;
            asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %1, 0;\n\t@p mbarrier.arrive.relaxed.cta.shared::cta.b64 _, [%0];\n\t}"
                         ::"r"(freeb_a + 8u * sr), "r"(lane < adv ? 1u : 0u) : "memory");
          }
          t += adv;
          st += adv; st -= st >= nst ? nst : 0;
          lead = (lead + adv * lead_step) & 15;
          stable = took ? tnext == s : stable;
          s = tnext;
          {
            const uint4 r4 = lds_v4(cache_a + 16u * static_cast<uint32_t>(max(s, 0)));   // the root's record is the empty list
            L.addr = rsent_cache_a + 8u * r4.x; L.n = static_cast<int>(r4.y);
            L.D = __uint_as_float(r4.z); L.bmag = __uint_as_float(r4.w); L.sorted = true;
          }
          if (rec_on) {
            __threadfence_block();
            if (lane == 0 && adv > 0) prog_publish(flags, t + 1);
          }
          spins = 0; no_allrows = false;
          // the next round is of the same kind more often than not: straight back, without the loop's bookkeeping
          if (L.n > 0 && L.n <= kGroupDeep && !stable && t < end && it + 1 < max_rounds && !(chk_on && t >= f_mid)) { ++it; goto fast_again; }
          continue;
        }
      }
      // ---- the same for an all-rows round (root state, unbound stream, or a state that repeats itself): every
      // lane its own row, and the whole list of the state, if it has one
      if (allrows && (fast_ok || !bound) && !(chk_on && t >= f_mid)) {
        int stq = st + q; stq -= stq >= nst ? nst : 0;
        const uint32_t sum_a = summ_a + stq * kSumStageBytes + min(ql, kSMax - 1) * 32u;
        const uint4 q1 = lds_v4_volatile(sum_a + 16u);
        const uint4 q0 = lds_v4_volatile(sum_a);
        const float xb = __uint_as_float(q0.z);
        const float lse = NORM ? lds_f32_volatile(summ_a + stq * kSumStageBytes + kSMax * 32u + 4u * min(ql, kSMax - 1)) : 0.0f;
        // the plain winner: at the root (no list) it is the row's winner
        float wv = __fadd_rn(__uint_as_float(q0.w), __fmul_rn(lam, __fadd_rn(L.D, __uint_as_float(q1.x))));
        int wtok = static_cast<int>(q1.z & 0xFFFFu), wnext = bound ? static_cast<int>(q1.y) : -1;
        bool rescan = (q1.z & kSumOvf) != 0;
        if (L.n > 0) {
          const uint32_t row_a = ring_a + stq * P.slot_bytes + ((lead + q * lead_step) & 15) + min(ql, kSMax - 1) * row_bytes;
          const uint32_t id1x2 = 2u * (q1.z & 0xFFFFu);
          float lv = -INFINITY;
          uint32_t ld = 2u * static_cast<uint32_t>(V);
          bool in_deep = false;
          int i = 0;
          for (; i + 3 < L.n; i += 4) {                       // sorted by token: strict comparisons, four in flight
            const uint32_t ea = L.addr + 8u * i;
            const uint2 e0 = lds_v2_nv(ea), e1 = lds_v2_nv(ea + 8u), e2 = lds_v2_nv(ea + 16u), e3 = lds_v2_nv(ea + 24u);
            const uint32_t t0 = e0.x & kTokMask, t1 = e1.x & kTokMask, t2 = e2.x & kTokMask, t3 = e3.x & kTokMask;
            const float v0 = __fadd_rn(bf16_bits_to_float(lds_u16_nv(row_a + t0)), __uint_as_float(e0.y));
            const float v1 = __fadd_rn(bf16_bits_to_float(lds_u16_nv(row_a + t1)), __uint_as_float(e1.y));
            const float v2 = __fadd_rn(bf16_bits_to_float(lds_u16_nv(row_a + t2)), __uint_as_float(e2.y));
            const float v3 = __fadd_rn(bf16_bits_to_float(lds_u16_nv(row_a + t3)), __uint_as_float(e3.y));
            in_deep |= t0 == id1x2 || t1 == id1x2 || t2 == id1x2 || t3 == id1x2;
            const bool b01 = v1 > v0, b23 = v3 > v2;
            const float va = b01 ? v1 : v0, vb = b23 ? v3 : v2;
            const uint32_t da = b01 ? e1.x : e0.x, db = b23 ? e3.x : e2.x;
            const bool bab = vb > va;
            const float vm = bab ? vb : va;
            const uint32_t dm = bab ? db : da;
            const bool bw = vm > lv;
            lv = bw ? vm : lv; ld = bw ? dm : ld;
          }                                                   // (cached lists are padded to multiples of four)
          const float y1 = __uint_as_float(q0.x), y2b = __uint_as_float(q0.y);
          const bool plain_ok = !in_deep && ((q1.z & kSumGap) != 0 || s <= 0);
          const float ub = (in_deep ? y2b : y1) + lam * L.D;
          const float tau = (fabsf(y1) + 4.0f * L.bmag) * 3.814697265625e-6f + 1e-30f;
          rescan = rescan || (!plain_ok && !(fmaxf(lv, xb) > ub + tau)) || (plain_ok && wv == lv);
          const bool take_plain = plain_ok && wv > lv;
          wv = take_plain ? wv : lv;
          wtok = take_plain ? wtok : static_cast<int>((ld & kTokMask) >> 1);
          wnext = take_plain ? wnext : static_cast<int>(ld >> TB_RS_TOK_BITS);
        }
        const bool ready = ql < S && (q > 0 || ql >= k) && t + q < end && q1.w == static_cast<uint32_t>(t + q) + 1u && !rescan;
        const unsigned ready_all = __ballot_sync(0xffffffffu, ready);
        const unsigned blank_all = __ballot_sync(0xffffffffu, ready && !(wv >= xb));
        const unsigned keep_all = __ballot_sync(0xffffffffu, wnext == s);
        const unsigned m1 = 0x11111111u;
        const unsigned smask = S >= 4 ? 0xFFFFFFFFu : (m1 << S) - m1;
        const unsigned pre = (1u << k) - 1u;
        const unsigned tok_all = ready_all & ~blank_all;
        const unsigned tokx = tok_all | pre;
        const unsigned a0 = tokx & m1, a1 = (tokx >> 1) & m1, a2 = (tokx >> 2) & m1;
        const unsigned vis = (m1 | (a0 << 1) | ((a0 & a1) << 2) | ((a0 & a1 & a2) << 3)) & smask & ~pre;
        const unsigned bad = vis & (~ready_all | (tok_all & ~keep_all));
        const int pb = bad ? __ffs(bad) - 1 : 32;
        const bool last_tok = pb < 32 && ((tok_all >> (pb & 31)) & 1u);
        const unsigned cm = (vis & (pb < 32 ? (1u << (pb & 31)) - 1u : 0xFFFFFFFFu)) | (last_tok ? 1u << (pb & 31) : 0u);
        const unsigned tm = cm & tok_all, bm = cm & blank_all;
        const int tn = __shfl_sync(0xffffffffu, wnext, pb & 31);
        const int tnext = last_tok ? tn : s;
        const int nt = __popc(tm);
        const bool rare = cm == 0u || (last_tok && bound && (tnext < 0 || tnext >= rec.n_states));
        if (!rare) {
          const unsigned cl = bm | (tm & (m1 << (S - 1)));
          const unsigned clf = (cl | (cl >> 1) | (cl >> 2) | (cl >> 3)) & m1;
          const int fq = __popc(clf);
          const int pos = fq < kWin ? __popc(((tm | (fq == 0 ? pre : 0u)) >> (4 * (fq & 7))) & 0xFu) : 0;
          const unsigned upto = 0xFFFFFFFFu >> (31 - lane);
          const bool mine_c = (cm >> lane) & 1u, mine_t = (tm >> lane) & 1u;
          const float val = NORM ? __fsub_rn(mine_t ? wv : xb, lse) : (mine_t ? wv : xb);
          if (rec_on) {
            if (mine_c) vlog[nv + __popc(cm & upto) - 1] = val;
            if (((cl >> lane) & 1u) && t + q + 1 >= f_mid)
              trace[t + q + 1] = make_int4((last_tok && lane == pb) ? tnext : s, n_out + __popc(tm & upto), nv + __popc(cm & upto), 0);
            nv += __popc(cm);
          }
          {
            // through the staging buffer; when these tokens fill the current block it goes out in between
            const int room = 32 - (n_out & 31), rank = __popc(tm & upto) - 1;
            if (mine_t && rank < room) emit_buf[(n_out + rank) & 31] = make_int2(wtok, t + q);
            __syncwarp();
            const int2 e = emit_buf[lane];
            const int o = (n_out & ~31) + lane;
            if (nt >= room && o < out_cap) { out_tok[o] = e.x; out_frm[o] = e.y; }
            __syncwarp();
            if (mine_t && rank >= room) emit_buf[(n_out + rank) & 31] = make_int2(wtok, t + q);
          }
          n_out += nt;
          // the score in visiting order; a row that was not consumed adds -0, which changes nothing
          const float valm = mine_c ? val : -0.0f;
#pragma unroll
          for (int i = 0; i < 32; ++i) score = __fadd_rn(score, __shfl_sync(0xffffffffu, valm, i));
          {
            int sr = st + lane; sr -= sr >= nst ? nst : 0;
            asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %1, 0;\n\t@p mbarrier.arrive.relaxed.cta.shared::cta.b64 _, [%0];\n\t}"
                         ::"r"(freeb_a + 8u * sr), "r"(lane < fq ? 1u : 0u) : "memory");
          }
          k = pos;
          t += fq;
          st += fq; st -= st >= nst ? nst : 0;
          lead = (lead + fq * lead_step) & 15;
          stable = last_tok ? false : stable;
          s = tnext;
          if (bound) {
            const uint4 r4 = lds_v4(cache_a + 16u * static_cast<uint32_t>(max(s, 0)));
            L.addr = rsent_cache_a + 8u * r4.x; L.n = static_cast<int>(r4.y);
            L.D = __uint_as_float(r4.z); L.bmag = __uint_as_float(r4.w); L.sorted = true;
          }
          if (rec_on) {
            __threadfence_block();
            if (lane == 0 && fq > 0) prog_publish(flags, t + 1);
          }
          spins = 0;
          continue;
        }
      }
      const int rq = wide ? 0 : q;                          // window frame of this lane
      const int rk = allrows ? ql : (rq == 0 ? k : 0);      // row of that frame
      int stq = st + rq; if (stq >= nst) stq -= nst;
      const uint32_t sum_a = summ_a + stq * kSumStageBytes + min(rk, kSMax - 1) * 32u;
      // the half with the sequence word is read first: when it matches, the other half is complete
      const uint4 q1 = lds_v4_volatile(sum_a + 16u);
      const uint4 q0 = lds_v4_volatile(sum_a);
      const uint32_t row_a = ring_a + stq * P.slot_bytes + ((lead + rq * lead_step) & 15) + rk * row_bytes;
      const bool in_row = rk < S && (rq > 0 || rk >= k);   // all-rows mode: rows before (t, k) are behind us
      const bool ready = in_row && t + rq < end && q1.w == static_cast<uint32_t>(t + rq) + 1u;
      const float y1 = __uint_as_float(q0.x), y2b = __uint_as_float(q0.y), xb = __uint_as_float(q0.z), x1 = __uint_as_float(q0.w);
      const float lse = NORM ? lds_f32_volatile(summ_a + stq * kSumStageBytes + kSMax * 32u + 4u * min(rk, kSMax - 1)) : 0.0f;
      const float xbs = NORM ? __fsub_rn(xb, lse) : xb;
      const uint32_t id1x2 = 2u * (q1.z & 0xFFFFu);
      bool rescan = (q1.z & kSumOvf) != 0;
      // ---- the tokens the state's chain boosts: exact values; the lanes that share a row split the list
      float wv = -INFINITY;
      uint32_t wdt = 2u * static_cast<uint32_t>(V);
      bool in_deep = false;
      {
        const int lstep = allrows ? 1 : (wide ? 32 : 4), l0 = allrows ? 0 : (wide ? lane : ql);
        int i = l0;
        if (L.sorted) {
          // a list sorted by token (all but those built by walking the chain): this lane's entries come in
          // ascending token order, so strict comparisons keep the lowest token among equal values; four entries
          // in flight, compared as a tree
          for (; i + 3 * lstep < L.n; i += 4 * lstep) {
            const uint32_t ea = L.addr + 8u * i;
            const uint2 e0 = lds_v2_nv(ea), e1 = lds_v2_nv(ea + 8u * lstep), e2 = lds_v2_nv(ea + 16u * lstep), e3 = lds_v2_nv(ea + 24u * lstep);
            const uint32_t t0 = e0.x & kTokMask, t1 = e1.x & kTokMask, t2 = e2.x & kTokMask, t3 = e3.x & kTokMask;
            const float v0 = __fadd_rn(bf16_bits_to_float(lds_u16_nv(row_a + t0)), __uint_as_float(e0.y));
            const float v1 = __fadd_rn(bf16_bits_to_float(lds_u16_nv(row_a + t1)), __uint_as_float(e1.y));
            const float v2 = __fadd_rn(bf16_bits_to_float(lds_u16_nv(row_a + t2)), __uint_as_float(e2.y));
            const float v3 = __fadd_rn(bf16_bits_to_float(lds_u16_nv(row_a + t3)), __uint_as_float(e3.y));
            in_deep |= t0 == id1x2 || t1 == id1x2 || t2 == id1x2 || t3 == id1x2;
            const bool b01 = v1 > v0, b23 = v3 > v2;
            const float va = b01 ? v1 : v0, vb = b23 ? v3 : v2;
            const uint32_t da = b01 ? e1.x : e0.x, db = b23 ? e3.x : e2.x;
            const bool bab = vb > va;
            const float vm = bab ? vb : va;
            const uint32_t dm = bab ? db : da;
            const bool bw = vm > wv;
            wv = bw ? vm : wv; wdt = bw ? dm : wdt;
          }
          for (; i < L.n; i += lstep) {
            const uint2 e0 = lds_v2_nv(L.addr + 8u * i);
            const float v0 = __fadd_rn(bf16_bits_to_float(lds_u16_nv(row_a + (e0.x & kTokMask))), __uint_as_float(e0.y));
            in_deep |= (e0.x & kTokMask) == id1x2;
            const bool bw = v0 > wv;
            wv = bw ? v0 : wv; wdt = bw ? e0.x : wdt;
          }
        }
        for (; i + lstep < L.n; i += 2 * lstep) {           // two entries in flight
          const uint2 e0 = lds_v2(L.addr + 8u * i), e1 = lds_v2(L.addr + 8u * (i + lstep));
          const uint32_t x0 = lds_u16(row_a + (e0.x & kTokMask)), x1r = lds_u16(row_a + (e1.x & kTokMask));
          const float v0 = __fadd_rn(bf16_bits_to_float(x0), __uint_as_float(e0.y));
          const float v1 = __fadd_rn(bf16_bits_to_float(x1r), __uint_as_float(e1.y));
          in_deep |= (e0.x & kTokMask) == id1x2 || (e1.x & kTokMask) == id1x2;
          if (v0 > wv || (v0 == wv && (e0.x & kTokMask) < (wdt & kTokMask))) { wv = v0; wdt = e0.x; }
          if (v1 > wv || (v1 == wv && (e1.x & kTokMask) < (wdt & kTokMask))) { wv = v1; wdt = e1.x; }
        }
        if (i < L.n) {
          const uint2 e0 = lds_v2(L.addr + 8u * i);
          const float v0 = __fadd_rn(bf16_bits_to_float(lds_u16(row_a + (e0.x & kTokMask))), __uint_as_float(e0.y));
          in_deep |= (e0.x & kTokMask) == id1x2;
          if (v0 > wv || (v0 == wv && (e0.x & kTokMask) < (wdt & kTokMask))) { wv = v0; wdt = e0.x; }
        }
      }
      // combine over the lanes that share the row
      if (L.n > 0 && !allrows) {
        if (wide) {
          const uint32_t key = fkey(wv);
          const uint32_t kmax = __reduce_max_sync(0xffffffffu, key);
          const uint32_t tmin = __reduce_min_sync(0xffffffffu, key == kmax ? (wdt & kTokMask) : 0xFFFFFFFFu);
          const unsigned who = __ballot_sync(0xffffffffu, key == kmax && (wdt & kTokMask) == tmin);
          const int src = __ffs(who) - 1;
          wv = __shfl_sync(0xffffffffu, wv, src); wdt = __shfl_sync(0xffffffffu, wdt, src);
          in_deep = __any_sync(0xffffffffu, in_deep);
        } else {
#pragma unroll
          for (int off = 1; off <= 2; off <<= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, wv, off);
            const uint32_t od = __shfl_xor_sync(0xffffffffu, wdt, off);
            const bool oi = __shfl_xor_sync(0xffffffffu, in_deep, off);
            if (ov > wv || (ov == wv && (od & kTokMask) < (wdt & kTokMask))) { wv = ov; wdt = od; }
            in_deep |= oi;
          }
        }
      }
      int wtok = static_cast<int>((wdt & kTokMask) >> 1);
      int wnext = static_cast<int>(wdt >> TB_RS_TOK_BITS);
      {
        // the best plain token: exact when the summary's winner is plain and clears the others by the
        // rounding margin (at the root it is exact by construction); else bounded from above
        const bool plain_ok = !in_deep && ((q1.z & kSumGap) != 0 || s <= 0);
        const float nd = __fadd_rn(x1, __fmul_rn(lam, __fadd_rn(L.D, __uint_as_float(q1.x))));
        const int id1 = static_cast<int>(id1x2 >> 1);
        if (plain_ok) {
          if (nd > wv || (nd == wv && id1 < wtok)) { wv = nd; wtok = id1; wnext = bound ? static_cast<int>(q1.y) : -1; }
        } else {
          const float ub = (in_deep ? y2b : y1) + lam * L.D;
          const float tau = (fabsf(y1) + 4.0f * L.bmag) * 3.814697265625e-6f + 1e-30f;
          if (!(fmaxf(wv, xb) > ub + tau)) {
            rescan = true;
          }
        }
      }
      const bool is_blank = ready && !rescan && !(wv >= xb);   // a tie with blank goes to the token
      const unsigned blank_all = __ballot_sync(0xffffffffu, is_blank);
      int tok = V;                                          // V: the round's last row selected no token
      float tval = 0.0f;
      int tnext = s, adv = 0;                               // adv: frames fully passed in this round
      bool progress = false;
      if (allrows) {
        // ---- walk the window row by row, through tokens too, while the state stays what it is ----------
        const unsigned ready_all = __ballot_sync(0xffffffffu, ready && !rescan);
        const unsigned keep_all = __ballot_sync(0xffffffffu, wnext == s);
        // Which rows the decode visits follows from the blank / token pattern alone while the state stays what
        // it is: in a frame, row j is visited when rows 0 .. j-1 selected tokens.  All of it is bit arithmetic
        // on the ballots (bit 4 q + j: row j of frame t + q); only the score is added up row by row.
        const unsigned m1 = 0x11111111u;
        const unsigned smask = S >= 4 ? 0xFFFFFFFFu : (m1 << S) - m1;          // rows j < S of every frame
        const unsigned pre = (1u << k) - 1u;                                   // rows of frame t behind the cursor
        const unsigned tok_all = ready_all & ~blank_all;
        const unsigned tokx = tok_all | pre;
        const unsigned a0 = tokx & m1, a1 = (tokx >> 1) & m1, a2 = (tokx >> 2) & m1;
        const unsigned vis = (m1 | (a0 << 1) | ((a0 & a1) << 2) | ((a0 & a1 & a2) << 3)) & smask & ~pre;
        // the walk ends before a row that is not ready (or needs the rescan) and after a token that changes the state
        const unsigned bad = vis & (~ready_all | (tok_all & ~keep_all));
        const int pb = bad ? __ffs(bad) - 1 : 32;
        const bool last_tok = pb < 32 && ((tok_all >> pb) & 1u);                // that token is consumed too
        const unsigned cm = (vis & (pb < 32 ? (1u << pb) - 1u : 0xFFFFFFFFu)) | (last_tok ? 1u << pb : 0u);
        const unsigned tm = cm & tok_all, bm = cm & blank_all;
        progress = cm != 0u;
        if (last_tok) { tok = __shfl_sync(0xffffffffu, wtok, pb); tnext = __shfl_sync(0xffffffffu, wnext, pb); }
        // frames closed: by a blank, or by a token in the frame's last row
        const unsigned cl = bm | (tm & (m1 << (S - 1)));
        const unsigned clf = (cl | (cl >> 1) | (cl >> 2) | (cl >> 3)) & m1;
        const int fq = __popc(clf);
        const int pos = fq < kWin ? __popc(((tm | (fq == 0 ? pre : 0u)) >> (4 * fq)) & 0xFu) : 0;
        const unsigned upto = 0xFFFFFFFFu >> (31 - lane);                       // bits 0 .. lane
        const bool mine_c = (cm >> lane) & 1u, mine_t = (tm >> lane) & 1u;
        const float val = NORM ? __fsub_rn(mine_t ? wv : xb, lse) : (mine_t ? wv : xb);
        if (rec_on) {
          if (mine_c) vlog[nv + __popc(cm & upto) - 1] = val;
          if (((cl >> lane) & 1u) && t + q + 1 >= f_mid)
            trace[t + q + 1] = make_int4((last_tok && lane == pb) ? tnext : s, n_out + __popc(tm & upto), nv + __popc(cm & upto), 0);
          nv += __popc(cm);
        }
        // emitted tokens, in order, through the staging buffer (at most one block boundary is crossed)
        const int nt = __popc(tm);
        if (nt > 0) {
          const int room = 32 - (n_out & 31);
          const int rank = __popc(tm & upto) - 1;
          if (mine_t && rank < room) emit_buf[(n_out + rank) & 31] = make_int2(wtok, t + q);
          if (nt >= room) {
            __syncwarp();
            const int2 e = emit_buf[lane];
            const int o = (n_out & ~31) + lane;
            if (o < out_cap) { out_tok[o] = e.x; out_frm[o] = e.y; }
            __syncwarp();
            if (mine_t && rank >= room) emit_buf[(n_out + rank) & 31] = make_int2(wtok, t + q);
          }
          n_out += nt;
        }
        for (unsigned m = cm; m; m &= m - 1u) score = __fadd_rn(score, __shfl_sync(0xffffffffu, val, __ffs(m) - 1));
        adv = fq; k = pos;
        if (!progress) {
          // the current row is not summarised yet (poll), or it needs the exact rescan (next round, shared mode)
          const unsigned resc_all = __ballot_sync(0xffffffffu, ready && rescan);
          if ((resc_all >> k) & 1u) no_allrows = true;
        }
      } else {
        // ---- the leading blanks, then the row after them --------------------------------------------------
        const unsigned blank_m = blank_all & 0x11111111u;   // one bit per group
        const unsigned stop_m = ~blank_m & 0x11111111u;
        int nb = stop_m ? (__ffs(stop_m) - 1) >> 2 : kWin;
        if (wide) nb = (blank_m & 1u) ? 1 : 0;
        const int jl = wide ? 0 : 4 * min(nb, kWin - 1);
        const float xb0 = __shfl_sync(0xffffffffu, xbs, 0), xb1 = __shfl_sync(0xffffffffu, xbs, 4);
        const bool j_ready = __shfl_sync(0xffffffffu, ready, jl);
        const bool j_rescan = __shfl_sync(0xffffffffu, rescan, jl);
        const int j_tok = __shfl_sync(0xffffffffu, wtok, jl);
        const float j_val = __shfl_sync(0xffffffffu, NORM ? __fsub_rn(wv, lse) : wv, jl);
        const float j_lse = NORM ? __shfl_sync(0xffffffffu, lse, jl) : 0.0f;
        const int j_next = __shfl_sync(0xffffffffu, wnext, jl);
        if (nb > 0) score = __fadd_rn(score, xb0);
        if (nb > 1) score = __fadd_rn(score, xb1);
        for (int r = 2; r < nb; ++r) score = __fadd_rn(score, __shfl_sync(0xffffffffu, xbs, 4 * r));
        adv = nb;
        progress = nb > 0;
        bool took = false;                                  // the row after the blanks was consumed too
        if (!(wide && nb == 1) && nb < kWin && j_ready) {
          progress = true;
          took = true;
          const int k_row = nb == 0 ? k : 0;                // symbols already emitted in that row's frame
          if (!j_rescan) {
            tok = j_tok; tval = j_val; tnext = j_next;
          } else {
            // exact evaluation of that row by the whole warp from shared memory
            const uint32_t rrow = __shfl_sync(0xffffffffu, row_a, jl);
            for (int i = lane; i < L.n; i += 32) { const int tk = (lds_v2(L.addr + 8u * i).x & kTokMask) >> 1; if (tk < V) tokidx[tk] = static_cast<int16_t>(i); }
            __syncwarp();
            ValId best{bf16_bits_to_float(lds_u16(rrow + 2u * V)), V};
            int bn = s;
            for (int tk = lane; tk < V; tk += 32) {
              const int i = tokidx[tk];
              float lbv; int nx;
              if (i >= 0) { const uint2 e = lds_v2(L.addr + 8u * i); lbv = __uint_as_float(e.y); nx = static_cast<int>(e.x >> TB_RS_TOK_BITS); }
              else { const int c = cls16[tk]; lbv = __fmul_rn(lam, __fadd_rn(L.D, rootcw[c])); nx = rootdst[c]; }
              const float x = bf16_bits_to_float(lds_u16(rrow + 2u * tk));
              const ValId c2{bound ? __fadd_rn(x, lbv) : x, tk};
              if (better(c2, best)) { best = c2; bn = bound ? nx : -1; }
            }
            __syncwarp();
            for (int i = lane; i < L.n; i += 32) { const int tk = (lds_v2(L.addr + 8u * i).x & kTokMask) >> 1; if (tk < V) tokidx[tk] = -1; }
            const Pick pk = warp_pick(best, bn);
            tok = pk.win.i; tval = NORM ? __fsub_rn(pk.win.v, j_lse) : pk.win.v; tnext = pk.next;
            if (tok == V) { score = __fadd_rn(score, tval); ++adv; }   // blank after all: that frame is passed too
          }
          if (tok != V) {
            score = __fadd_rn(score, tval);
            // emitted tokens are staged in shared memory and written out 32 at a time, coalesced
            if (lane == 0) emit_buf[n_out & 31] = make_int2(tok, t + nb);
            if ((n_out & 31) == 31) {
              __syncwarp();
              const int2 e = emit_buf[lane];
              const int o = (n_out & ~31) + lane;
              if (o < out_cap) { out_tok[o] = e.x; out_frm[o] = e.y; }
              __syncwarp();
            }
            ++n_out;
            k = k_row + 1;
            if (k == S) ++adv;                              // the frame closes by force
          }
        }
        if (rec_on) {
          // the values in visiting order, and the frame starts t + 1 .. t + adv this round reached
          if ((lane & 3) == 0 && q < nb) vlog[nv + q] = xbs;
          if (took && lane == 0) vlog[nv + nb] = tval;
          if (lane < adv && t + lane + 1 >= f_mid) {
            const bool viatok = lane >= nb && tok != V;     // reached because the token closed its frame
            trace[t + lane + 1] = make_int4(viatok ? tnext : s, n_out - ((tok != V && !viatok) ? 1 : 0), nv + lane + 1, 0);
          }
          nv += nb + (took ? 1 : 0);
        }
        if (adv > 0 && (tok == V || k == S)) k = 0;
      }
      if (!progress) {                                      // the current row is not summarised yet: poll
        if (++spins > kSpinLimit || ((spins & 255u) == 0u && flags[pipe])) {
          if (spins > kSpinLimit) { flags[0] = 1; flags[1] = 1; if (lane == 0) atomicOr(p.status, TB_STATUS_WAIT_TIMEOUT); }
          failed = true; break;
        }
        --it;                                               // a poll is not a round
        continue;
      }
      spins = 0;
      if (!allrows) no_allrows = false;
      // ---- hand the passed frames' slots back, move on -------------------------------------------------
      if (lane < adv) {                                     // lane r frees the slot of frame t + r
        const int sr = st + lane >= nst ? st + lane - nst : st + lane;
        mbar_arrive_relaxed_addr(freeb_a + 8u * sr);
      }
      t += adv;
      st += adv; if (st >= nst) st -= nst;
      lead = (lead + adv * lead_step) & 15;
      if (tok != V) stable = (tnext == s);                  // the last token left the state unchanged
      if (tok != V && bound && tnext != s) {
        s = tnext;
        if (s <= 0) {
          L.n = 0; L.D = 0.0f; L.bmag = fabsf(lam) * R; L.sorted = true;
        } else if (resolved) {
          if (s >= rec.n_states) { if (lane == 0) atomicOr(p.status, TB_STATUS_BAD_STATE); s = 0; }
          if (cached) {
            const uint4 r4 = lds_v4(cache_a + 16u * s);
            L.addr = rsent_cache_a + 8u * r4.x; L.n = static_cast<int>(r4.y);
            L.D = __uint_as_float(r4.z); L.bmag = __uint_as_float(r4.w);
          } else {
            const TbRsRec r4 = rsrec_g[s];
            for (int i = lane; i < r4.count && i < V + 4; i += 32) lbuf[i] = rsent_g[r4.begin + i];
            __syncwarp();
            L.addr = smem_u32(lbuf); L.n = r4.count; L.D = r4.D; L.bmag = r4.bmag;
          }
          L.sorted = true;
        } else {
          build_list(strec, tokent, rec.n_states, rec.max_depth, s, lam, R, V, lbuf, cls_seen, cls16, L, lane, p.status);
        }
      }
      if (rec_on && adv > 0) {                              // publish how far the record reaches
        __threadfence_block();
        if (lane == 0) flags[2] = t + 1;
      }
      if (chk_on && k == 0 && t >= f_mid && t < end && t < flags[2]) {
        // at a frame start pipeline 1 has recorded: the same graph state means the same decode from here on
        const int rec_state = *reinterpret_cast<const volatile int*>(trace + t);
        if (rec_state == s) { tc = t; break; }
      }
    }
    if ((n_out & 31) != 0) {                  // the tokens still staged
      __syncwarp();
      const int2 e = emit_buf[lane];
      const int o = (n_out & ~31) + lane;
      if (lane < (n_out & 31) && o < out_cap) { out_tok[o] = e.x; out_frm[o] = e.y; }
    }
    if (tc >= 0) flags[0] = 1;                // met the record: this pipeline's producer and helpers stop
    else if (chk_on && !failed && t >= end) flags[1] = 1;   // decoded everything itself: pipeline 1 is not needed
    else if (failed || t < end) { flags[0] = 1; flags[1] = 1; }   // left early: let the other roles stop too
    if (lane == 0) {
      if (!seg) {
        p.out_counts[b] = n_out; p.out_scores[b] = score; p.out_states[b] = s;
        if (p.out_cursors) p.out_cursors[b] = t;
      } else if (pipe == 0) {
        seg_res[0] = n_out; seg_res[1] = __float_as_int(score); seg_res[2] = s; seg_res[3] = tc; seg_res[4] = t;
      } else {
        seg_res[8] = n_out; seg_res[9] = nv; seg_res[10] = s; seg_res[11] = t;
      }
    }
  }
  __syncthreads();
  if (seg) {
    // ---- merge: pipeline 0's output, then pipeline 1's from the frame start where the two met ----------------
    const int nA = seg_res[0], tcm = seg_res[3];
    int count = nA, s_fin = seg_res[2], t_fin = seg_res[4];
    float score = __int_as_float(seg_res[1]);
    if (tcm >= 0) {
      const int nB = seg_res[8], nvB = seg_res[9];
      const int4 tr = P.scr_trace[static_cast<int64_t>(b) * (p.frames + 1) + tcm];
      const int n0 = tr.y, nv0 = tr.z;
      const int32_t* scr_tok = P.scr_tok + 2 * static_cast<int64_t>(b) * P.scr_cap;
      const int32_t* scr_frm = scr_tok + P.scr_cap;
      int32_t* out_tok = p.out_tokens + static_cast<int64_t>(b) * p.out_cap;
      int32_t* out_frm = p.out_frames + static_cast<int64_t>(b) * p.out_cap;
      for (int j = n0 + tid; j < nB && j < P.scr_cap; j += kThreadsF) {
        const int o = nA + j - n0;
        if (o < p.out_cap) { out_tok[o] = scr_tok[j]; out_frm[o] = scr_frm[j]; }
      }
      if (warp == 0) {
        // the score is the sum in visiting order: add pipeline 1's values one by one
        const float* vlog = P.scr_val + static_cast<int64_t>(b) * P.scr_cap;
        for (int i0 = nv0; i0 < nvB; i0 += 32) {
          const float v = i0 + lane < nvB ? vlog[i0 + lane] : 0.0f;
          const int m = min(32, nvB - i0);
          for (int j = 0; j < m; ++j) score = __fadd_rn(score, __shfl_sync(0xffffffffu, v, j));
        }
      }
      count = nA + nB - n0; s_fin = seg_res[10]; t_fin = seg_res[11];
    }
    if (tid == 0) {
      p.out_counts[b] = count; p.out_scores[b] = score; p.out_states[b] = s_fin;
      if (p.out_cursors) p.out_cursors[b] = t_fin;
    }
  }
  __syncthreads();
}

}  // namespace


namespace {
// scratch layout of the two-segment decode: tokens+frames, values, frame-start records
struct ScratchLayout { size_t tok, val, trace, total; };
ScratchLayout scratch_layout(int32_t n_streams, int32_t frames, int32_t S) {
  ScratchLayout l;
  const size_t cap = static_cast<size_t>(frames) * S, n = static_cast<size_t>(n_streams);
  size_t o = 0;
  l.tok = o; o += (n * 2 * cap * sizeof(int32_t) + 255) & ~static_cast<size_t>(255);
  l.val = o; o += (n * cap * sizeof(float) + 255) & ~static_cast<size_t>(255);
  l.trace = o; o += n * (static_cast<size_t>(frames) + 1) * sizeof(int4);
  l.total = o;
  return l;
}
}  // namespace

size_t tb_greedy_fast_scratch_bytes(int32_t n_streams, int32_t frames, int32_t S) {
  if (n_streams <= 0 || frames < kSegMinFrames || S <= 0) return 0;
  return scratch_layout(n_streams, frames, S).total;
}

// Returns TB_OK if the launch was made, 1 if this path does not cover the call (the caller then
// uses the general kernel), or an error code.
int tb_launch_greedy_fast(const TbDecodeParams& d, int32_t max_cache_bytes, int32_t max_states, int32_t all_resolved,
                          void* scratch, size_t scratch_bytes, cudaStream_t stream) {
  const int W = d.V + 1;
  if (d.dtype != TB_BF16 || d.persistent || d.n_dur != 0) return 1;
  if (d.sv != 1 || d.ss != W || d.st < static_cast<int64_t>(d.S) * W || d.sb < 0) return 1;
  if (d.S > kSMax || d.V > 256 * kNitMax || 2 * (d.V + 1) > (1 << TB_RS_TOK_BITS) || max_states >= (1 << (32 - TB_RS_TOK_BITS))) return 1;
  if (reinterpret_cast<uintptr_t>(d.logits) & 1) return 1;
  FastParams P;
  P.d = d;
  // 16 bytes past a multiple of 128: the decider's lanes (one slot each) then spread over the shared-memory banks
  P.slot_bytes = ((up16(d.S * W * 2 + 16) + 127) & ~127) + 16;
  P.tensor_lo = reinterpret_cast<const unsigned char*>(d.logits);
  const int64_t last = static_cast<int64_t>(d.n_streams - 1) * d.sb + static_cast<int64_t>(d.frames - 1) * d.st +
                       static_cast<int64_t>(d.S - 1) * d.ss + d.V;
  P.tensor_hi = P.tensor_lo + 2 * (last + 1);
  int dev = 0, max_smem = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) {
    cudaGetLastError();
    return TB_ERR_CUDA;
  }
  const int budget = max_smem - 1024;
  const int per_stage = P.slot_bytes + 16 + kSumStageBytes;
  const bool seg_ok = d.frames >= kSegMinFrames && scratch && (reinterpret_cast<uintptr_t>(scratch) & 15) == 0 &&
                      scratch_layout(d.n_streams, d.frames, d.S).total <= scratch_bytes;
  // Layouts in order of preference: the graphs' lists cached in shared memory with two segments per stream (each
  // half of the ring at least eight stages, the decider's window), cached with one segment, then not cached (lists read from the arena),
  // again with two segments or one.
  // A cache beyond 48 KB is only taken when no decider needs room to build or stage lists of its own.
  P.npipes = 1; P.scr_cap = 0; P.scr_tok = nullptr; P.scr_val = nullptr; P.scr_trace = nullptr;
  int nst = 0;
  for (int attempt = 0; attempt < 4 && nst == 0; ++attempt) {
    const bool want_cache = attempt < 2, want_seg = (attempt & 1) == 0;
    if (want_cache && !(max_cache_bytes > 0 && (max_cache_bytes <= 48 * 1024 || (all_resolved && max_cache_bytes <= 112 * 1024)))) continue;
    if (want_seg && !seg_ok) continue;
    P.cache_bytes = want_cache ? max_cache_bytes : 0;
    P.own_lists = (all_resolved && (P.cache_bytes > 0 || max_states == 0)) ? 0 : 1;
    const int np = want_seg ? 2 : 1;
    const int fixed = carve(0, P.slot_bytes, d.V, d.C, P.cache_bytes, np, P.own_lists).total;
    int n = (budget - fixed - 64) / per_stage;
    if (n > kStagesMax) n = kStagesMax;
    if (n < (np == 2 ? 16 : 9)) continue;     // a pipeline's part of the ring holds at least the decider's window
    nst = n; P.npipes = np;
  }
  if (nst == 0) return 1;
  if (P.npipes == 2) {
    const ScratchLayout l = scratch_layout(d.n_streams, d.frames, d.S);
    unsigned char* sb = static_cast<unsigned char*>(scratch);
    P.scr_cap = d.frames * d.S;
    P.scr_tok = reinterpret_cast<int32_t*>(sb + l.tok);
    P.scr_val = reinterpret_cast<float*>(sb + l.val);
    P.scr_trace = reinterpret_cast<int4*>(sb + l.trace);
  }
  if (nst < 9) return 1;   // the decider's window spans eight stages
  P.nst = nst;
  const Smem so = carve(nst, P.slot_bytes, d.V, d.C, P.cache_bytes, P.npipes, P.own_lists);
  if (so.total > budget) return 1;
  const int nit = (d.V + 255) / 256;
  void (*fn)(FastParams) = nit <= 1 ? k_greedy_fast<1, false> : nit <= 2 ? k_greedy_fast<2, false> : nit <= 4 ? k_greedy_fast<4, false> : k_greedy_fast<8, false>;
  // rows normalised inside the selection (log-softmax): the helpers also leave every row's normaliser
  if (d.normalize) fn = nit <= 1 ? k_greedy_fast<1, true> : nit <= 2 ? k_greedy_fast<2, true> : nit <= 4 ? k_greedy_fast<4, true> : k_greedy_fast<8, true>;
  if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem) != cudaSuccess) {
    cudaGetLastError();
    return 1;
  }
  fn<<<d.n_streams, kThreadsF, so.total, stream>>>(P);
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}
