// Segmented greedy RNNT decode for packed bf16 logits: every stream is cut into segments that are decoded at the
// same time by many small pipelines spread over all SMs, and stitched at the end.
//
// A pipeline is one decider warp plus a share of its block's helper warps.
//   helper warps : read rows straight from the tensor (one pass over HBM, 16 bytes per lane and load) and reduce
//                  each, independently of the graph state, to a 32-byte summary in a small shared-memory ring
//                  (see RowSummary);
//   decider warp : the sequential part -- walks the rows its segment's decode visits, resolves each from its summary
//                  plus the few tokens boosted by the current graph state, whose logits it gathers from the row in
//                  global memory (the row has just been read by a helper of the same pipeline, so the gather is
//                  served by L2), advances the graph state and the frame cursor and logs tokens and row values.
// Because no rows are kept in shared memory a pipeline needs about 3 KB of it, and a block holds several pipelines
// of one stream next to that stream's resolved lists (cached in shared memory once per block).
//
// Segments.  The decode from a given (frame start, graph state) is a function of those two alone.  Segment i > 0
// of a bound stream starts a few frames before its first frame f_i in the root state and, from f_i on, records at
// every frame start its graph state and how much it has logged.  Every segment keeps decoding past its nominal end
// until, at a frame start, its state equals the state the owner of that frame recorded there: from that point on
// the owner's log is this segment's continuation.  Segment 0 starts in the true state, so the chain
// segment 0 -> the segment it met -> the segment that one met -> ... is the sequential decode; segments that are
// not on the chain were speculation that did not pay.  Nothing ever waits for another block: a record that is not
// there yet just means the segment decodes on (in the worst case to the end of the stream).  Records carry a
// per-stream launch number, so a record of an earlier launch is never taken for one of this launch.
// The block that finishes last for a stream (an atomic counter) walks the chain, copies the tokens into the
// caller's arrays and adds the logged row values one by one in visiting order, so tokens, frames, final state and
// the fp32 score are those of the sequential decode bit for bit.
//
// Exactness of a row's selection: as in tb_greedy_fast.cu (summary winner accepted only with a margin that dominates
// all roundings, the state's own tokens always evaluated exactly, otherwise an exact rescan of the row).
//
// Every wait is bounded; a wait that runs out raises TB_STATUS_WAIT_TIMEOUT and makes all roles of the block leave.
#include "tb_fast_common.cuh"
#include "tb_launch.h"

namespace {

constexpr int kGMax = 4;            // pipelines (deciders) per block
constexpr int kRing = 32;           // frames of summaries a pipeline's ring holds (a power of two)
constexpr int kLead = 14;           // frames the helpers may claim ahead of the decider (claims race: up to a helper per warp more)
constexpr int kLeadOver = 9;        // the same once the segment is past its nominal end (the decider's window is eight frames)
constexpr int kWarm = 8;            // frames a segment decodes before the first frame it answers for
constexpr int kSegMinLen = 48;      // shortest nominal segment, in frames
constexpr int kSegCap = 32;         // most segments per stream
constexpr int kMaxThreadsS = 640;
constexpr int kGroupDeepS = 64;     // up to this many boosted tokens: eight rows per round, four lanes each
constexpr int kAllRowsDeepS = 64;   // all-rows mode in a state that just repeated itself: at most this many boosted tokens
constexpr uint32_t kSpinLimitS = 1u << 20;
constexpr int kRingBytes = kRing * kSumStageBytes;
constexpr int kRowBufs = 2;         // rows a helper warp keeps in flight (asynchronous copies into its own buffers)

struct SegRes {   // what a pipeline leaves for the stitch (32 bytes)
  int32_t n_tok, n_val;   // tokens / row values logged
  int32_t state, t_end;   // graph state and frame cursor where it stopped
  int32_t met;            // 1: stopped at frame start t_end because it met the record of that frame's owner
  int32_t failed;
  int32_t pad0, pad1;
};

struct SegParams {
  TbDecodeParams d;
  int32_t G, H, NB, nseg_max, cache_bytes;
  uint32_t spin_limit;                 // polls a bounded wait may take
  int32_t withhold_frame;              // self-test of the bounded waits: this frame is claimed but never summarised (-1: none)
  const unsigned char* tensor_lo;      // first / one-past-last byte of the logits tensor
  const unsigned char* tensor_hi;
  int32_t* log_tok;                    // [n_streams][log_stride] tokens, per segment region
  int32_t* log_frm;                    // [n_streams][log_stride] their frames
  float* log_val;                      // [n_streams][log_stride] value of every visited row, in order
  int64_t log_stride;
  int32_t seg_off[kSegCap + 1];        // region of segment i within a stream's log: [seg_off[i], seg_off[i + 1])
  unsigned long long* trace_st;        // [n_streams][frames + 1]: state | launch tag << 32 at a frame start
  int2* trace_aux;                     // [n_streams][frames + 1]: {tokens, values} its owner had logged there
  SegRes* seg_res;                     // [n_streams][nseg_max]
  uint32_t* done;                      // [n_streams] blocks of the stream that have finished (reset by the last one)
  uint32_t* epoch;                     // [n_streams] launches so far (bumped by the last block)
};

struct SmemS {
  int summ, cls16, tokcb, rootcw, rootdst, emit, misc, hops, rows, cache, total;
  int row_buf;   // bytes of one helper row buffer
};
__host__ __device__ inline int up16s(int x) { return (x + 15) & ~15; }
__host__ __device__ inline SmemS carve_s(int G, int H, int V, int C, int cache_bytes) {
  SmemS s;
  int o = 0;
  // a helper's row buffer holds the 16-byte aligned superset of a row (the row may start up to 14 bytes in) and at
  // least the whole passes the helper reads; 16 bytes more keep consecutive buffers on different banks
  const int nit = (V + 255) / 256;
  s.row_buf = (up16s(14 + 2 * (V + 1)) > nit * 512 ? up16s(14 + 2 * (V + 1)) : nit * 512) + 16;
  s.summ = o; o += G * kRingBytes;
  s.cls16 = o; o += up16s(2 * V);
  s.tokcb = o; o += up16s(4 * V);            // lambda * root-arc weight of every token (0 without a root arc)
  s.rootcw = o; o += up16s(4 * C);
  s.rootdst = o; o += up16s(4 * C);
  s.emit = o; o += G * 32 * 8;               // emitted (token, frame) pairs waiting for a coalesced store
  s.misc = o; o += 512;
  s.hops = o; o += kSegCap * 32;
  s.rows = o; o += (H + G) * kRowBufs * s.row_buf;   // every warp's rows in flight (helpers first, then the deciders)
  s.cache = o; o += up16s(cache_bytes);
  s.total = o;
  return s;
}

__device__ __forceinline__ uint32_t ldg_u16(const unsigned char* p) {
  uint16_t v;
  asm("ld.global.nc.u16 %0, [%1];" : "=h"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ void cp_async16(uint32_t dst_smem, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_smem), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ uint32_t lds_u32_volatile(uint32_t a) {
  uint32_t v;
  asm volatile("ld.volatile.shared.u32 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
  return v;
}

// Starts the copy of one row (its 16-byte aligned superset) from the tensor into a helper's buffer: 16 bytes per
// lane and copy, asynchronous, past L1.  A 16-byte piece that leaves the tensor [lo, hi) is assembled from the
// elements inside it (only the first and the last row of a tensor can need that).
__device__ __forceinline__ void fetch_row(unsigned char* buf, const unsigned char* rowp, int row_bytes,
                                          const unsigned char* lo, const unsigned char* hi, int lane) {
  const int off = static_cast<int>(reinterpret_cast<uintptr_t>(rowp) & 15);
  const unsigned char* a0 = rowp - off;
  const int nchunks = (off + row_bytes + 15) >> 4;
  const uint32_t buf_a = smem_u32(buf) + 16u * lane;
  const unsigned char* a = a0 + 16 * lane;
  if (a0 >= lo && a0 + 16 * nchunks <= hi) {
    // (a row of up to 2048 elements and its lead of up to 14 bytes are at most 257 pieces: nine per lane)
#pragma unroll
    for (int j = 0; j < 9; ++j)
      if (lane + 32 * j < nchunks) cp_async16(buf_a + 512u * j, a + 512 * j);
  } else {
    for (int c = lane; c < nchunks; c += 32) {
      const unsigned char* ac = a0 + 16 * c;
      if (ac >= lo && ac + 16 <= hi) {
        cp_async16(smem_u32(buf) + 16u * c, ac);
      } else {
        for (int e = 0; e < 8; ++e) {
          uint16_t x = 0xFF80u;
          if (ac + 2 * e >= lo && ac + 2 * e + 2 <= hi) x = *reinterpret_cast<const uint16_t*>(ac + 2 * e);
          *reinterpret_cast<uint16_t*>(buf + 16 * c + 2 * e) = x;
        }
      }
    }
  }
  cp_async_commit();
}

__device__ __forceinline__ uint2 ld_relaxed_u64(const unsigned long long* p) {
  uint2 v;
  asm volatile("ld.relaxed.gpu.global.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_relaxed_u64(unsigned long long* p, uint32_t lo, uint32_t hi) {
  asm volatile("st.relaxed.gpu.global.v2.u32 [%0], {%1, %2};" ::"l"(p), "r"(lo), "r"(hi) : "memory");
}

// The best of NE entries of a sorted list (entries first, first + step, ...; those at index >= n read as the
// never-selected sentinel) on the row at rowp: all entry loads are issued, then all gathers, then one comparison
// tree in which an entry replaces an earlier one only when strictly better (so the lowest token wins a tie).
// wv / wdt: the running best (value, entry word); seen: the summary's winner (2 * id in id1x2) is among the entries.
template <int NE>
__device__ __forceinline__ void eval_list(uint32_t laddr, int first, int step, int n, const unsigned char* rowp,
                                          uint32_t id1x2, uint32_t sent, float& wv, uint32_t& wdt, bool& seen) {
  uint32_t d[NE];
  float v[NE];
#pragma unroll
  for (int j = 0; j < NE; ++j) {
    const int i = first + j * step;
    uint2 e = make_uint2(sent, 0xFF800000u);
    if (i < n) e = lds_v2_nv(laddr + 8u * i);
    d[j] = e.x; v[j] = __uint_as_float(e.y);
  }
  uint32_t x[NE];
#pragma unroll
  for (int j = 0; j < NE; ++j) x[j] = ldg_u16(rowp + (d[j] & kTokMask));
#pragma unroll
  for (int j = 0; j < NE; ++j) {
    v[j] = __fadd_rn(bf16_bits_to_float(x[j]), v[j]);
    seen |= (d[j] & kTokMask) == id1x2;
  }
#pragma unroll
  for (int w = 1; w < NE; w <<= 1) {
#pragma unroll
    for (int j = 0; j + w < NE; j += 2 * w) {
      const bool take = v[j + w] > v[j];
      v[j] = take ? v[j + w] : v[j];
      d[j] = take ? d[j + w] : d[j];
    }
  }
  const bool bw = v[0] > wv;
  wv = bw ? v[0] : wv;
  wdt = bw ? d[0] : wdt;
}

// Entries first, first + step, ... of a sorted list of n entries, NE at a time.
template <int NE>
__device__ __forceinline__ void eval_list_all(uint32_t laddr, int first, int step, int n, const unsigned char* rowp,
                                              uint32_t id1x2, uint32_t sent, float& wv, uint32_t& wdt, bool& seen) {
  for (int f = first; f < n; f += NE * step) eval_list<NE>(laddr, f, step, n, rowp, id1x2, sent, wv, wdt, seen);
}

// One frame (S rows) reduced by a warp that is not a helper by trade: a decider whose own rows are not ready yet.
// Two buffers: the next row is on its way while the current one is reduced.
template <int NIT, bool NORM>
__device__ __noinline__ void summarize_frame(const HelperCtx h, unsigned char* bufs, int row_buf, const unsigned char* frame0,
                                             int row_bytes, int S, const unsigned char* lo, const unsigned char* hi,
                                             uint32_t out_a, uint32_t seq, int lane) {
  fetch_row(bufs, frame0, row_bytes, lo, hi, lane);
  for (int k = 0; k < S; ++k) {
    const unsigned char* rowp = frame0 + k * row_bytes;
    if (k + 1 < S) { fetch_row(bufs + ((k + 1) & 1) * row_buf, rowp + row_bytes, row_bytes, lo, hi, lane); cp_async_wait<1>(); }
    else cp_async_wait<0>();
    __syncwarp();
    summarize_row<NIT, NORM>(h, bufs + (k & 1) * row_buf, static_cast<int>(reinterpret_cast<uintptr_t>(rowp) & 15), out_a + k * 32, seq, lane,
                             out_a + kSMax * 32 + 4 * k);
  }
}

struct PipeInfo {   // one per pipeline of the block, in shared memory
  int32_t active, seg, pf0, f_first, f_next, is_last;
  int32_t pad0, pad1;
};

template <int NIT, bool NORM>
__global__ void __launch_bounds__(kMaxThreadsS, 1) k_greedy_seg(SegParams P) {
  extern __shared__ __align__(128) unsigned char dyn[];
  const TbDecodeParams& p = P.d;
  const int V = p.V, C = p.C, S = p.S, W = V + 1, G = P.G, H = P.H;
  const int nthreads = blockDim.x;
  const SmemS so = carve_s(G, H, V, C, P.cache_bytes);
  const uint32_t summ_a = smem_u32(dyn + so.summ);
  uint16_t* cls16 = reinterpret_cast<uint16_t*>(dyn + so.cls16);
  float* tokcb = reinterpret_cast<float*>(dyn + so.tokcb);
  float* rootcw = reinterpret_cast<float*>(dyn + so.rootcw);
  int32_t* rootdst = reinterpret_cast<int32_t*>(dyn + so.rootdst);
  volatile int* prog = reinterpret_cast<volatile int*>(dyn + so.misc);          // [kGMax] frame cursor of each decider; -1: the pipeline has stopped
  int* next_frame = reinterpret_cast<int*>(dyn + so.misc + 16);                 // [kGMax] first frame of the pipeline no helper has claimed yet
  volatile int* abort_f = reinterpret_cast<volatile int*>(dyn + so.misc + 96);  // a wait ran out somewhere in the block: everybody leaves
  float* root_stats = reinterpret_cast<float*>(dyn + so.misc + 32);             // beta_min, beta_max, R
  int* blk_vars = reinterpret_cast<int*>(dyn + so.misc + 48);                   // [0] this block stitches; stitch scalars
  PipeInfo* pinfo = reinterpret_cast<PipeInfo*>(dyn + so.misc + 128);           // [kGMax] (128 bytes)
  float* part = reinterpret_cast<float*>(dyn + so.misc + 256);                  // 3 floats per warp during set-up

  const int b = blockIdx.x / P.NB, sp = blockIdx.x - b * P.NB;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = nthreads >> 5;
  const TbSlotRec rec = p.slots[b];
  const bool bound = rec.n_states > 0;
  const float lam = bound ? rec.lambda : 0.0f;
  const unsigned char* blob = p.arena + rec.blob_off;
  int end = p.lengths ? p.lengths[b] : p.frames;
  end = max(0, min(end, p.frames));
  // segments of this stream: nseg pieces of L frames (the last one shorter)
  int nseg = min(P.nseg_max, max(1, end / kSegMinLen));
  const int L = max(1, (end + nseg - 1) / nseg);
  nseg = max(1, (end + L - 1) / L);
  const uint32_t tag = P.epoch[b] + 1u;
  unsigned long long* trace_st = P.trace_st + static_cast<int64_t>(b) * (p.frames + 1);
  int2* trace_aux = P.trace_aux + static_cast<int64_t>(b) * (p.frames + 1);
  SegRes* seg_res = P.seg_res + static_cast<int64_t>(b) * P.nseg_max;

  const bool usable = !bound || (rec.n_rsent >= 0 && P.cache_bytes >= rec.blob_bytes - rec.off_rsrec);
  if (!usable) {   // the launch was laid out without room for this graph's lists (the launcher prevents it)
    if (tid == 0) atomicOr(p.status, TB_STATUS_BAD_STATE);
    nseg = 0;
  }

  // ---- set-up: tables, root vectors, list cache ------------------------------------------------------------
  for (int v = tid; v < V; v += nthreads) cls16[v] = static_cast<uint16_t>(p.cls[v]);
  for (int c = tid; c < C; c += nthreads) { rootcw[c] = 0.0f; rootdst[c] = 0; }
  for (int i = tid; i < G * kRingBytes / 4; i += nthreads) reinterpret_cast<uint32_t*>(dyn + so.summ)[i] = 0u;   // no sequence word matches yet
  if (tid < kGMax) {
    const int g = tid, i = sp * G + g;
    PipeInfo pi;
    pi.seg = i;
    pi.active = g < G && i < nseg && end > 0;
    pi.f_first = i * L;
    pi.is_last = i == nseg - 1;
    pi.f_next = pi.is_last ? end : min(end, (i + 1) * L);
    pi.pf0 = max(0, pi.f_first - ((bound && i > 0) ? kWarm : 0));
    pi.pad0 = pi.pad1 = 0;
    pinfo[g] = pi;
    prog[g] = pi.active ? pi.pf0 : -1;
    next_frame[g] = pi.pf0;
  }
  if (tid == 0) { blk_vars[0] = 0; *abort_f = 0; }
  if (bound && usable) {
    // the lists the deciders read are the tail of the blob: one contiguous 16-byte aligned range
    const uint4* src = reinterpret_cast<const uint4*>(blob + rec.off_rsrec);
    uint4* dst = reinterpret_cast<uint4*>(dyn + so.cache);
    for (int i = tid; i < ((rec.blob_bytes - rec.off_rsrec) >> 4); i += nthreads) dst[i] = src[i];
  }
  __syncthreads();
  const GraphPtrs g0 = graph_of(p.arena, rec);
  {
    float bmin = 0.0f, bmax = 0.0f, R = 0.0f;
    if (bound) {
      const int e = g0.arc_begin[1];
      for (int a = g0.arc_begin[0] + tid; a < e; a += nthreads) {
        const int c = g0.arc_cls[a];
        const float wv = __fadd_rn(0.0f, g0.arc_w[a]);        // the walk's fl(acc + w) with acc = 0
        const float cb = __fmul_rn(lam, wv);
        rootcw[c] = wv; rootdst[c] = g0.arc_dst[a];
        bmin = fminf(bmin, cb); bmax = fmaxf(bmax, cb); R = fmaxf(R, fabsf(wv));
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      bmin = fminf(bmin, __shfl_xor_sync(0xffffffffu, bmin, off));
      bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, off));
      R = fmaxf(R, __shfl_xor_sync(0xffffffffu, R, off));
    }
    if (lane == 0) { part[3 * warp] = bmin; part[3 * warp + 1] = bmax; part[3 * warp + 2] = R; }
    __syncthreads();
    if (tid == 0) {
      for (int w2 = 1; w2 < nwarps; ++w2) {
        bmin = fminf(bmin, part[3 * w2]); bmax = fmaxf(bmax, part[3 * w2 + 1]); R = fmaxf(R, part[3 * w2 + 2]);
      }
      root_stats[0] = bmin; root_stats[1] = bmax; root_stats[2] = R;
    }
  }
  // (a class has a root arc exactly when its target is not the root)
  for (int v = tid; v < V; v += nthreads) { const int c = cls16[v]; tokcb[v] = rootdst[c] ? __fmul_rn(lam, rootcw[c]) : 0.0f; }
  __syncthreads();

  const unsigned char* base = reinterpret_cast<const unsigned char*>(p.logits) + 2 * static_cast<int64_t>(b) * p.sb;
  const int64_t fsb = 2 * p.st;                       // frame stride in bytes
  const int row_bytes = 2 * W;

  // Deciders sit on warps 0, 4, 8, 12: warps are spread over the SM's four schedulers by warp index, so all deciders
  // share one scheduler with each other only, and their dependent instruction chains do not queue behind helpers.
  const bool is_decider = (warp & 3) == 0 && (warp >> 2) < G;
  HelperCtx h;
  h.cls16 = cls16; h.tokcb = tokcb; h.rootcw = rootcw; h.rootdst = rootdst; h.V = V; h.nit = (V + 255) / 256;
  h.beta_min = root_stats[0]; h.beta_max = root_stats[1]; h.dbeta = __fsub_rn(root_stats[1], root_stats[0]);
  h.bmag_max = fabsf(lam) * ((bound ? rec.d_max : 0.0f) + root_stats[2]);
  if (!is_decider) {
    // ================================ helpers =====================================================
    // The rows of all pipelines of the block are dealt round-robin over the block's helpers: helper hw takes rows
    // hw, hw + H, ... of every pipeline (rows counted from the pipeline's first frame).  A pipeline whose ring is
    // full is skipped for now; one that has stopped is dropped, so its helpers' time goes to the others.
    const int hw = warp - min(G, (warp + 3) >> 2);      // index among the block's helper warps
    // Frames are claimed dynamically: a helper takes the next unclaimed frame of a pipeline (its home pipeline
    // first, then the others in turn) when the decider is not too far behind, and reduces the frame's S rows one
    // after the other.  A pipeline that has stopped is skipped, so its helpers' time goes to the others.  The warp
    // keeps two rows in flight: while it reduces one from its buffer, the next is on its way from HBM.
    unsigned char* bufs = dyn + so.rows + hw * kRowBufs * so.row_buf;
    const int home = hw % G;
    int cg = -1, cf = 0, ck = 0, cb = 0, coff = 0;      // the row in buffer cb: pipeline, frame, row in frame, byte offset
    uint32_t idle = 0;
    for (;;) {
      // ---- the row after the current one: the frame's next row, or the first row of a newly claimed frame
      int ng = -1, nf = 0, nk = 0;
      bool any_left = false;
      if (cg >= 0 && ck + 1 < S) { ng = cg; nf = cf; nk = ck + 1; }
      else {
        for (int j = 0; j < G && ng < 0; ++j) {
          int g = home + j; g -= g >= G ? G : 0;
          const int pr = prog[g];
          if (pr < 0) continue;
          const int seen = *reinterpret_cast<volatile int*>(next_frame + g);
          if (seen >= end) continue;
          any_left = true;
          const PipeInfo& pi = pinfo[g];
          if (seen - pr >= ((!pi.is_last && seen >= pi.f_next) ? kLeadOver : kLead)) continue;
          int f = 0;
          if (lane == 0) f = atomicAdd(next_frame + g, 1);
          f = __shfl_sync(0xffffffffu, f, 0);
          if (f < end) { ng = g; nf = f; nk = 0; }
        }
      }
      const int nb_ = cb ^ 1;
      int noff = 0;
      if (ng >= 0) {
        const unsigned char* rowp = base + static_cast<int64_t>(nf) * fsb + nk * row_bytes;
        noff = static_cast<int>(reinterpret_cast<uintptr_t>(rowp) & 15);
        fetch_row(bufs + nb_ * so.row_buf, rowp, row_bytes, P.tensor_lo, P.tensor_hi, lane);
      }
      if (cg >= 0) {
        // the current row has arrived when at most the newest copy group is still pending
        if (ng >= 0) cp_async_wait<1>(); else cp_async_wait<0>();
        __syncwarp();
        if (cf != P.withhold_frame)
        summarize_row<NIT, NORM>(h, bufs + cb * so.row_buf, coff,
                                 summ_a + cg * kRingBytes + (cf & (kRing - 1)) * kSumStageBytes + ck * 32,
                                 static_cast<uint32_t>(cf) + 1u, lane,
                                 summ_a + cg * kRingBytes + (cf & (kRing - 1)) * kSumStageBytes + kSMax * 32 + 4 * ck);
      }
      const bool had = cg >= 0;
      cg = ng; cf = nf; ck = nk; cb = nb_; coff = noff;
      if (ng >= 0 || had) { idle = 0; continue; }
      if (!any_left || *abort_f) break;
      if (++idle > (P.spin_limit >> 2)) {
        if (lane == 0) atomicOr(p.status, TB_STATUS_WAIT_TIMEOUT);
        *abort_f = 1;
        break;
      }
      __nanosleep(128);
    }
    cp_async_wait<0>();
  } else if (pinfo[warp >> 2].active) {
    // ================================ decider =====================================================
    // Works in rounds over a window of eight frames, as the decider of tb_greedy_fast.cu does: the warp is eight
    // groups of four lanes, group q stands for frame t + q.
    //   shared mode  : group q resolves one row under the current state -- group 0 the current row (t, k), group
    //                  q >= 1 row (t + q, 0); leading blank rows are consumed at once, the first row that selects a
    //                  token ends the round.
    //   all-rows mode: (no boosted tokens, or a state that just repeated itself) lane ql of group q resolves row
    //                  (t + q, ql); a round walks through tokens too while they leave the state unchanged.
    //   wide mode    : (many boosted tokens) all 32 lanes resolve the current row.
    const int pipe = warp >> 2;
    const PipeInfo pi = pinfo[pipe];
    const float R = root_stats[2];
    const uint32_t sring = summ_a + pipe * kRingBytes;
    const uint32_t cache_a = smem_u32(dyn + so.cache);
    const uint32_t rsent_cache_a = cache_a + static_cast<uint32_t>(rec.off_rsent - rec.off_rsrec);
    int2* emit_buf = reinterpret_cast<int2*>(dyn + so.emit + pipe * 256);
    const uint32_t sent = 2u * static_cast<uint32_t>(V);

    CurList Lc;
    Lc.addr = rsent_cache_a; Lc.n = 0; Lc.sorted = true; Lc.D = 0.0f; Lc.bmag = fabsf(lam) * R;

    const int q = lane >> 2, ql = lane & 3;
    constexpr int kWin = 8;
    const int f_next = pi.f_next;
    const bool is_last = pi.is_last != 0;
    const int rec_lo = pi.seg > 0 ? pi.f_first : INT32_MAX;        // frame starts this segment records: [rec_lo, f_next)
    int t = pi.pf0, k = 0, s = bound ? 0 : -1, n_out = 0, nv = 0;
    const int out_cap = P.seg_off[pi.seg + 1] - P.seg_off[pi.seg];
    int32_t* out_tok = P.log_tok + static_cast<int64_t>(b) * P.log_stride + P.seg_off[pi.seg];
    int32_t* out_frm = P.log_frm + static_cast<int64_t>(b) * P.log_stride + P.seg_off[pi.seg];
    float* vlog = P.log_val + static_cast<int64_t>(b) * P.log_stride + P.seg_off[pi.seg];
    int tc = -1;
        if (rec_lo == t && lane == 0) { trace_aux[t] = make_int2(0, 0); st_relaxed_u64(trace_st + t, static_cast<uint32_t>(s), tag); }
    const int max_rounds = p.frames * S + p.frames + 8;
    uint32_t spins = 0;
    bool failed = false, stable = false, no_allrows = false;

    // records frame start fs (reached with state st_, after n_tok tokens and n_val values) if it is this segment's
#define TB_TRACE_PUT(fs, st_, n_tok, n_val)                                                        \
    do { if ((fs) >= rec_lo && (fs) < f_next) {                                                    \
      trace_aux[(fs)] = make_int2((n_tok), (n_val));                                               \
      st_relaxed_u64(trace_st + (fs), static_cast<uint32_t>(st_), tag); } } while (0)

    for (int it = 0; t < end; ++it) {
      if (it >= max_rounds) { if (lane == 0) atomicOr(p.status, TB_STATUS_STEP_LIMIT); failed = true; break; }
      // ---- past the nominal end: has the owner of this frame start recorded the same state? ----------------
      if (k == 0 && t >= f_next && !is_last) {
        if (!bound) { tc = t; break; }                        // no graph state: the owner's decode from here is this one's
        const uint2 tr = ld_relaxed_u64(trace_st + t);
        if (tr.y == tag && static_cast<int>(tr.x) == s) { tc = t; break; }
      }
      // ---- nothing can happen before the current row is summarised: wait for it cheaply --------------------
      if (lds_u32_volatile(sring + (t & (kRing - 1)) * kSumStageBytes + k * 32u + 28u) != static_cast<uint32_t>(t) + 1u) {
        if (++spins > P.spin_limit || ((spins & 63u) == 0u && *abort_f)) {
          if (spins > P.spin_limit && lane == 0) atomicOr(p.status, TB_STATUS_WAIT_TIMEOUT);
          failed = true; break;
        }
        --it;                                               // a poll is not a round
        // Rather than sleep, do a helper's work: if the frame this decider waits for has been claimed already
        // (a helper is on it), take the next unclaimed frame of a pipeline of the block, this one's first.
        bool helped = false;
        for (int j = 0; j < G && !helped; ++j) {
          int g = pipe + j; g -= g >= G ? G : 0;
          const int pr = g == pipe ? t : prog[g];
          if (pr < 0) continue;
          const int seen = *reinterpret_cast<volatile int*>(next_frame + g);
          if (seen >= end) continue;
          const PipeInfo& pj = pinfo[g];
          if (seen - pr >= ((!pj.is_last && seen >= pj.f_next) ? kLeadOver : kLead)) continue;
          int f = 0;
          if (lane == 0) f = atomicAdd(next_frame + g, 1);
          f = __shfl_sync(0xffffffffu, f, 0);
          if (f >= end) continue;
          helped = true;
          if (f == P.withhold_frame) continue;
          summarize_frame<NIT, NORM>(h, dyn + so.rows + (H + pipe) * kRowBufs * so.row_buf, so.row_buf,
                               base + static_cast<int64_t>(f) * fsb, row_bytes, S, P.tensor_lo, P.tensor_hi,
                               summ_a + g * kRingBytes + (f & (kRing - 1)) * kSumStageBytes, static_cast<uint32_t>(f) + 1u, lane);
        }
        if (!helped) __nanosleep(32);
        continue;
      }
      const bool allrows = !no_allrows && (Lc.n == 0 || (stable && Lc.n <= kAllRowsDeepS));
      const bool wide = !allrows && Lc.n > kGroupDeepS;
      // ---- the usual round, without branches (see tb_greedy_fast.cu) ------------------------------------------
      if (bound && !allrows && !wide) {
      fast_again:
        const int rk = q == 0 ? k : 0;
        const int fq = t + q;
        const uint32_t sum_a = sring + (fq & (kRing - 1)) * kSumStageBytes + rk * 32u;
        const uint4 q1 = lds_v4_volatile(sum_a + 16u);
        const uint4 q0 = lds_v4_volatile(sum_a);
        const unsigned char* rowp = base + static_cast<int64_t>(min(fq, end - 1)) * fsb + rk * row_bytes;
        const bool ready = fq < end && q1.w == static_cast<uint32_t>(fq) + 1u;
        const float y1 = __uint_as_float(q0.x), y2b = __uint_as_float(q0.y), xb = __uint_as_float(q0.z), x1 = __uint_as_float(q0.w);
        // rows normalised: the row's normaliser comes off what the row adds to the score, after the selection
        const float lse = NORM ? lds_f32_volatile(sring + (fq & (kRing - 1)) * kSumStageBytes + kSMax * 32u + 4u * rk) : 0.0f;
        const uint32_t id1x2 = 2u * (q1.z & 0xFFFFu);
        // this lane's entries ql, ql + 4, ...: sorted by token, so a strict comparison keeps the lowest token
        float wv = -INFINITY;
        uint32_t wdt = sent;
        bool seen = false;
        if (Lc.n <= 16) eval_list<4>(Lc.addr, ql, 4, Lc.n, rowp, id1x2, sent, wv, wdt, seen);
        else eval_list_all<8>(Lc.addr, ql, 4, Lc.n, rowp, id1x2, sent, wv, wdt, seen);
        // the group's best: every lane fetches the other three lanes' results and reduces them itself.  Equal best
        // values in two lanes -- the lowest token would decide -- are left to the general code.
        bool tie;
        {
          const float o1 = __shfl_xor_sync(0xffffffffu, wv, 1), o2 = __shfl_xor_sync(0xffffffffu, wv, 2), o3 = __shfl_xor_sync(0xffffffffu, wv, 3);
          const uint32_t d1 = __shfl_xor_sync(0xffffffffu, wdt, 1), d2 = __shfl_xor_sync(0xffffffffu, wdt, 2), d3 = __shfl_xor_sync(0xffffffffu, wdt, 3);
          const unsigned seen_m = __ballot_sync(0xffffffffu, seen);
          const float hi1 = fmaxf(wv, o1), lo1 = fminf(wv, o1), hi2 = fmaxf(o2, o3), lo2 = fminf(o2, o3);
          const float gm = fmaxf(hi1, hi2), second = fmaxf(fminf(hi1, hi2), fmaxf(lo1, lo2));
          tie = second == gm;
          seen = ((seen_m >> (4 * q)) & 0xFu) != 0u;
          wdt = wv == gm ? wdt : (o1 == gm ? d1 : (o2 == gm ? d2 : d3));
          wv = gm;
        }
        const bool in_deep = seen;
        int wtok = static_cast<int>((wdt & kTokMask) >> 1);
        int wnext = static_cast<int>(wdt >> TB_RS_TOK_BITS);
        // the best plain token: exact when it clears the others by the margin, else bounded
        const bool plain_ok = !in_deep && ((q1.z & kSumGap) != 0 || s <= 0);
        const float nd = __fadd_rn(x1, __fmul_rn(lam, __fadd_rn(Lc.D, __uint_as_float(q1.x))));
        const int id1 = static_cast<int>(id1x2 >> 1);
        const float ub = (in_deep ? y2b : y1) + lam * Lc.D;
        const float tau = (fabsf(y1) + 4.0f * Lc.bmag) * 3.814697265625e-6f + 1e-30f;
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
        const float j_val = __shfl_sync(0xffffffffu, NORM ? __fsub_rn(wv, lse) : wv, jl);
        const float xbs = NORM ? __fsub_rn(xb, lse) : xb;
        const bool took = nb < kWin && j_ready;             // the row after the blanks selects a token
        const bool rare = (nb == 0 && !took) || (took && j_rescan) || (took && (j_next < 0 || j_next >= rec.n_states));
        if (!rare) {
          // ---- commit ----
          if (lane == 0 && took) emit_buf[n_out & 31] = make_int2(j_tok, t + nb);
          {
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
          // the values in visiting order, and the frame starts t + 1 .. t + adv this round reached
          if ((lane & 3) == 0 && q < nb && nv + q < out_cap) vlog[nv + q] = xbs;
          if (took && lane == 0 && nv + nb < out_cap) vlog[nv + nb] = j_val;
          if (lane < adv) TB_TRACE_PUT(t + lane + 1, lane >= nb ? tnext : s, n_out - ((took && lane < nb) ? 1 : 0), nv + lane + 1);
          nv += nb + (took ? 1 : 0);
          k = (took && !closes) ? k_row + 1 : 0;
          t += adv;
          stable = took ? tnext == s : stable;
          s = tnext;
          {
            const uint4 r4 = lds_v4(cache_a + 16u * static_cast<uint32_t>(max(s, 0)));   // the root's record is the empty list
            Lc.addr = rsent_cache_a + 8u * r4.x; Lc.n = static_cast<int>(r4.y);
            Lc.D = __uint_as_float(r4.z); Lc.bmag = __uint_as_float(r4.w);
          }
          if (lane == 0) prog[pipe] = t;
          spins = 0; no_allrows = false;
          // the next round is of the same kind more often than not: straight back, without the loop's bookkeeping
          if (Lc.n > 0 && Lc.n <= kGroupDeepS && !stable && t < end && it + 1 < max_rounds && (t < f_next || is_last)) { ++it; goto fast_again; }
          continue;
        }
      }
      // ---- the same for an all-rows round (root state, unbound stream, or a state that repeats itself): every
      // lane its own row, and the whole list of the state, if it has one
      if (allrows) {
        const int fq = t + q;
        const int rkq = min(ql, kSMax - 1);
        const uint32_t sum_a = sring + (fq & (kRing - 1)) * kSumStageBytes + rkq * 32u;
        const uint4 q1 = lds_v4_volatile(sum_a + 16u);
        const uint4 q0 = lds_v4_volatile(sum_a);
        const float xb = __uint_as_float(q0.z);
        const float lse = NORM ? lds_f32_volatile(sring + (fq & (kRing - 1)) * kSumStageBytes + kSMax * 32u + 4u * rkq) : 0.0f;
        // the plain winner: at the root (no list) it is the row's winner
        float wv = __fadd_rn(__uint_as_float(q0.w), __fmul_rn(lam, __fadd_rn(Lc.D, __uint_as_float(q1.x))));
        int wtok = static_cast<int>(q1.z & 0xFFFFu), wnext = bound ? static_cast<int>(q1.y) : -1;
        bool rescan = (q1.z & kSumOvf) != 0;
        if (Lc.n > 0) {
          const unsigned char* rowp = base + static_cast<int64_t>(min(fq, end - 1)) * fsb + min(rkq, S - 1) * row_bytes;
          const uint32_t id1x2 = 2u * (q1.z & 0xFFFFu);
          float lv = -INFINITY;
          uint32_t ld = sent;
          bool in_deep = false;
          eval_list_all<8>(Lc.addr, 0, 1, Lc.n, rowp, id1x2, sent, lv, ld, in_deep);
          const float y1 = __uint_as_float(q0.x), y2b = __uint_as_float(q0.y);
          const bool plain_ok = !in_deep && ((q1.z & kSumGap) != 0 || s <= 0);
          const float ub = (in_deep ? y2b : y1) + lam * Lc.D;
          const float tau = (fabsf(y1) + 4.0f * Lc.bmag) * 3.814697265625e-6f + 1e-30f;
          rescan = rescan || (!plain_ok && !(fmaxf(lv, xb) > ub + tau)) || (plain_ok && wv == lv);
          const bool take_plain = plain_ok && wv > lv;
          wv = take_plain ? wv : lv;
          wtok = take_plain ? wtok : static_cast<int>((ld & kTokMask) >> 1);
          wnext = take_plain ? wnext : static_cast<int>(ld >> TB_RS_TOK_BITS);
        }
        const bool ready = ql < S && (q > 0 || ql >= k) && fq < end && q1.w == static_cast<uint32_t>(fq) + 1u && !rescan;
        const unsigned ready_all = __ballot_sync(0xffffffffu, ready);
        const unsigned blank_all = __ballot_sync(0xffffffffu, ready && !(wv >= xb));
        const unsigned keep_all = __ballot_sync(0xffffffffu, wnext == s);
        // Which rows the decode visits follows from the blank / token pattern alone while the state stays what it
        // is: in a frame, row j is visited when rows 0 .. j-1 selected tokens (bit 4 q + j: row j of frame t + q).
        const unsigned m1 = 0x11111111u;
        const unsigned smask = S >= 4 ? 0xFFFFFFFFu : (m1 << S) - m1;
        const unsigned pre = (1u << k) - 1u;
        const unsigned tok_all = ready_all & ~blank_all;
        const unsigned tokx = tok_all | pre;
        const unsigned a0 = tokx & m1, a1 = (tokx >> 1) & m1, a2 = (tokx >> 2) & m1;
        const unsigned vis = (m1 | (a0 << 1) | ((a0 & a1) << 2) | ((a0 & a1 & a2) << 3)) & smask & ~pre;
        // the walk ends before a row that is not ready (or needs the rescan) and after a token that changes the state
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
          // frames closed: by a blank, or by a token in the frame's last row
          const unsigned cl = bm | (tm & (m1 << (S - 1)));
          const unsigned clf = (cl | (cl >> 1) | (cl >> 2) | (cl >> 3)) & m1;
          const int fcl = __popc(clf);
          const int pos = fcl < kWin ? __popc(((tm | (fcl == 0 ? pre : 0u)) >> (4 * (fcl & 7))) & 0xFu) : 0;
          const unsigned upto = 0xFFFFFFFFu >> (31 - lane);
          const bool mine_c = (cm >> lane) & 1u, mine_t = (tm >> lane) & 1u;
          const float val = NORM ? __fsub_rn(mine_t ? wv : xb, lse) : (mine_t ? wv : xb);
          {
            const int vi = nv + __popc(cm & upto) - 1;
            if (mine_c && vi < out_cap) vlog[vi] = val;
            if ((cl >> lane) & 1u)
              TB_TRACE_PUT(fq + 1, (last_tok && lane == pb) ? tnext : s, n_out + __popc(tm & upto), nv + __popc(cm & upto));
            nv += __popc(cm);
          }
          {
            // through the staging buffer; when these tokens fill the current block it goes out in between
            const int room = 32 - (n_out & 31), rank = __popc(tm & upto) - 1;
            if (mine_t && rank < room) emit_buf[(n_out + rank) & 31] = make_int2(wtok, fq);
            __syncwarp();
            const int2 e = emit_buf[lane];
            const int o = (n_out & ~31) + lane;
            if (nt >= room && o < out_cap) { out_tok[o] = e.x; out_frm[o] = e.y; }
            __syncwarp();
            if (mine_t && rank >= room) emit_buf[(n_out + rank) & 31] = make_int2(wtok, fq);
          }
          n_out += nt;
          k = pos;
          t += fcl;
          stable = last_tok ? false : stable;
          s = tnext;
          if (bound) {
            const uint4 r4 = lds_v4(cache_a + 16u * static_cast<uint32_t>(max(s, 0)));
            Lc.addr = rsent_cache_a + 8u * r4.x; Lc.n = static_cast<int>(r4.y);
            Lc.D = __uint_as_float(r4.z); Lc.bmag = __uint_as_float(r4.w);
          }
          if (lane == 0) prog[pipe] = t;
          spins = 0;
          continue;
        }
      }
      // ---- the general round: every mode, every case ---------------------------------------------------------
      const int rq = wide ? 0 : q;                          // window frame of this lane
      const int rk = allrows ? ql : (rq == 0 ? k : 0);      // row of that frame
      const int fq = t + rq;
      const uint32_t sum_a = sring + (fq & (kRing - 1)) * kSumStageBytes + min(rk, kSMax - 1) * 32u;
      // the half with the sequence word is read first: when it matches, the other half is complete
      const uint4 q1 = lds_v4_volatile(sum_a + 16u);
      const uint4 q0 = lds_v4_volatile(sum_a);
      const unsigned char* rowp = base + static_cast<int64_t>(min(fq, end - 1)) * fsb + min(rk, S - 1) * row_bytes;
      const bool in_row = rk < S && (rq > 0 || rk >= k);   // all-rows mode: rows before (t, k) are behind us
      const bool ready = in_row && fq < end && q1.w == static_cast<uint32_t>(fq) + 1u;
      const float y1 = __uint_as_float(q0.x), y2b = __uint_as_float(q0.y), xb = __uint_as_float(q0.z), x1 = __uint_as_float(q0.w);
      const float lse = NORM ? lds_f32_volatile(sring + (fq & (kRing - 1)) * kSumStageBytes + kSMax * 32u + 4u * min(rk, kSMax - 1)) : 0.0f;
      const float xbs = NORM ? __fsub_rn(xb, lse) : xb;
      const uint32_t id1x2 = 2u * (q1.z & 0xFFFFu);
      bool rescan = (q1.z & kSumOvf) != 0;
      // ---- the tokens the state's chain boosts: exact values; the lanes that share a row split the list
      float wv = -INFINITY;
      uint32_t wdt = sent;
      bool in_deep = false;
      {
        const int lstep = allrows ? 1 : (wide ? 32 : 4), l0 = allrows ? 0 : (wide ? lane : ql);
        eval_list_all<4>(Lc.addr, l0, lstep, Lc.n, rowp, id1x2, sent, wv, wdt, in_deep);
      }
      // combine over the lanes that share the row
      if (Lc.n > 0 && !allrows) {
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
        const float nd = __fadd_rn(x1, __fmul_rn(lam, __fadd_rn(Lc.D, __uint_as_float(q1.x))));
        const int id1 = static_cast<int>(id1x2 >> 1);
        if (plain_ok) {
          if (nd > wv || (nd == wv && id1 < wtok)) { wv = nd; wtok = id1; wnext = bound ? static_cast<int>(q1.y) : -1; }
        } else {
          const float ub = (in_deep ? y2b : y1) + lam * Lc.D;
          const float tau = (fabsf(y1) + 4.0f * Lc.bmag) * 3.814697265625e-6f + 1e-30f;
          if (!(fmaxf(wv, xb) > ub + tau)) rescan = true;
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
        const unsigned m1 = 0x11111111u;
        const unsigned smask = S >= 4 ? 0xFFFFFFFFu : (m1 << S) - m1;          // rows j < S of every frame
        const unsigned pre = (1u << k) - 1u;                                   // rows of frame t behind the cursor
        const unsigned tok_all = ready_all & ~blank_all;
        const unsigned tokx = tok_all | pre;
        const unsigned a0 = tokx & m1, a1 = (tokx >> 1) & m1, a2 = (tokx >> 2) & m1;
        const unsigned vis = (m1 | (a0 << 1) | ((a0 & a1) << 2) | ((a0 & a1 & a2) << 3)) & smask & ~pre;
        const unsigned bad = vis & (~ready_all | (tok_all & ~keep_all));
        const int pb = bad ? __ffs(bad) - 1 : 32;
        const bool last_tok = pb < 32 && ((tok_all >> pb) & 1u);                // that token is consumed too
        const unsigned cm = (vis & (pb < 32 ? (1u << pb) - 1u : 0xFFFFFFFFu)) | (last_tok ? 1u << pb : 0u);
        const unsigned tm = cm & tok_all, bm = cm & blank_all;
        progress = cm != 0u;
        if (last_tok) { tok = __shfl_sync(0xffffffffu, wtok, pb); tnext = __shfl_sync(0xffffffffu, wnext, pb); }
        const unsigned cl = bm | (tm & (m1 << (S - 1)));
        const unsigned clf = (cl | (cl >> 1) | (cl >> 2) | (cl >> 3)) & m1;
        const int fcl = __popc(clf);
        const int pos = fcl < kWin ? __popc(((tm | (fcl == 0 ? pre : 0u)) >> (4 * fcl)) & 0xFu) : 0;
        const unsigned upto = 0xFFFFFFFFu >> (31 - lane);                       // bits 0 .. lane
        const bool mine_c = (cm >> lane) & 1u, mine_t = (tm >> lane) & 1u;
        const float val = NORM ? __fsub_rn(mine_t ? wv : xb, lse) : (mine_t ? wv : xb);
        {
          const int vi = nv + __popc(cm & upto) - 1;
          if (mine_c && vi < out_cap) vlog[vi] = val;
          if ((cl >> lane) & 1u)
            TB_TRACE_PUT(fq + 1, (last_tok && lane == pb) ? tnext : s, n_out + __popc(tm & upto), nv + __popc(cm & upto));
          nv += __popc(cm);
        }
        // emitted tokens, in order, through the staging buffer (at most one block boundary is crossed)
        const int nt = __popc(tm);
        if (nt > 0) {
          const int room = 32 - (n_out & 31);
          const int rank = __popc(tm & upto) - 1;
          if (mine_t && rank < room) emit_buf[(n_out + rank) & 31] = make_int2(wtok, fq);
          if (nt >= room) {
            __syncwarp();
            const int2 e = emit_buf[lane];
            const int o = (n_out & ~31) + lane;
            if (o < out_cap) { out_tok[o] = e.x; out_frm[o] = e.y; }
            __syncwarp();
            if (mine_t && rank >= room) emit_buf[(n_out + rank) & 31] = make_int2(wtok, fq);
          }
          n_out += nt;
        }
        adv = fcl; k = pos;
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
        const bool j_ready = __shfl_sync(0xffffffffu, ready, jl);
        const bool j_rescan = __shfl_sync(0xffffffffu, rescan, jl);
        const int j_tok = __shfl_sync(0xffffffffu, wtok, jl);
        const float j_val = __shfl_sync(0xffffffffu, NORM ? __fsub_rn(wv, lse) : wv, jl);
        const float j_lse = NORM ? __shfl_sync(0xffffffffu, lse, jl) : 0.0f;
        const int j_next = __shfl_sync(0xffffffffu, wnext, jl);
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
            // exact evaluation of that row by the whole warp, straight from the tensor; whether a token is on the
            // state's list, and where, is found by bisection (the list is sorted by token)
            const int jf = min(t + nb, end - 1);
            const unsigned char* rrow = base + static_cast<int64_t>(jf) * fsb + k_row * row_bytes;
            ValId best{bf16_bits_to_float(ldg_u16(rrow + 2u * V)), V};
            int bn = s;
            for (int tk = lane; tk < V; tk += 32) {
              int lo = 0, hi = Lc.n;
              while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (((lds_v2(Lc.addr + 8u * mid).x & kTokMask) >> 1) < static_cast<uint32_t>(tk)) lo = mid + 1; else hi = mid;
              }
              float lbv; int nx;
              uint2 e = make_uint2(sent, 0u);
              if (lo < Lc.n) e = lds_v2(Lc.addr + 8u * lo);
              if (((e.x & kTokMask) >> 1) == static_cast<uint32_t>(tk)) { lbv = __uint_as_float(e.y); nx = static_cast<int>(e.x >> TB_RS_TOK_BITS); }
              else { const int c = cls16[tk]; lbv = __fmul_rn(lam, __fadd_rn(Lc.D, rootcw[c])); nx = rootdst[c]; }
              const float x = bf16_bits_to_float(ldg_u16(rrow + 2u * tk));
              const ValId c2{bound ? __fadd_rn(x, lbv) : x, tk};
              if (better(c2, best)) { best = c2; bn = bound ? nx : -1; }
            }
            const Pick pk = warp_pick(best, bn);
            tok = pk.win.i; tval = NORM ? __fsub_rn(pk.win.v, j_lse) : pk.win.v; tnext = pk.next;
            if (tok == V) ++adv;                              // blank after all: that frame is passed too
          }
          if (tok != V) {
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
        {
          // the values in visiting order, and the frame starts t + 1 .. t + adv this round reached
          if ((lane & 3) == 0 && q < nb && nv + q < out_cap) vlog[nv + q] = xbs;
          if (took && lane == 0 && nv + nb < out_cap) vlog[nv + nb] = tval;
          if (lane < adv) {
            const bool viatok = lane >= nb && tok != V;     // reached because the token closed its frame
            TB_TRACE_PUT(t + lane + 1, viatok ? tnext : s, n_out - ((tok != V && !viatok) ? 1 : 0), nv + lane + 1);
          }
          nv += nb + (took ? 1 : 0);
        }
        if (adv > 0 && (tok == V || k == S)) k = 0;
      }
      if (!progress) {                                      // the current row is not summarised yet: poll
        if (++spins > P.spin_limit || ((spins & 255u) == 0u && *abort_f)) {
          if (spins > P.spin_limit && lane == 0) atomicOr(p.status, TB_STATUS_WAIT_TIMEOUT);
          failed = true; break;
        }
        --it;                                               // a poll is not a round
        continue;
      }
      spins = 0;
      if (!allrows) no_allrows = false;
      t += adv;
      if (lane == 0) prog[pipe] = t;
      if (tok != V) stable = (tnext == s);                  // the last token left the state unchanged
      if (tok != V && bound && tnext != s) {
        s = tnext;
        if (s < 0 || s >= rec.n_states) { if (lane == 0) atomicOr(p.status, TB_STATUS_BAD_STATE); s = 0; }
        const uint4 r4 = lds_v4(cache_a + 16u * s);
        Lc.addr = rsent_cache_a + 8u * r4.x; Lc.n = static_cast<int>(r4.y);
        Lc.D = __uint_as_float(r4.z); Lc.bmag = __uint_as_float(r4.w);
      }
    }
#undef TB_TRACE_PUT
    if ((n_out & 31) != 0) {                  // the tokens still staged
      __syncwarp();
      const int2 e = emit_buf[lane];
      const int o = (n_out & ~31) + lane;
      if (lane < (n_out & 31) && o < out_cap) { out_tok[o] = e.x; out_frm[o] = e.y; }
    }
    if (failed || (tc < 0 && t < end)) {      // left early: let every role of the block stop
      failed = true;
      *abort_f = 1;
    }
    if (lane == 0) {
      prog[pipe] = -1;                        // this pipeline's rows are not needed any more
      SegRes r;
      r.n_tok = min(n_out, out_cap); r.n_val = min(nv, out_cap); r.state = s; r.t_end = tc >= 0 ? tc : t; r.met = tc >= 0 ? 1 : 0;
      r.failed = (failed || n_out > out_cap || nv > out_cap) ? 1 : 0; r.pad0 = r.pad1 = 0;
      if (r.failed && !failed) atomicOr(p.status, TB_STATUS_STEP_LIMIT);
      *reinterpret_cast<int4*>(&seg_res[pi.seg]) = make_int4(r.n_tok, r.n_val, r.state, r.t_end);
      *(reinterpret_cast<int4*>(&seg_res[pi.seg]) + 1) = make_int4(r.met, r.failed, 0, 0);
    }
  }

  // ---- the block that finishes last for its stream stitches the segments -------------------------------------
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const uint32_t old = atomicAdd(&P.done[b], 1u);
    blk_vars[0] = (old == static_cast<uint32_t>(P.NB) - 1u) ? 1 : 0;
  }
  __syncthreads();
  if (!blk_vars[0]) return;
  __threadfence();
  // (every pipeline has stopped: the row buffers are free and hold the stitch's working data)
  int4* hops = reinterpret_cast<int4*>(dyn + so.hops);   // per hop: {segment, first token, end token, output offset}, {first value, end value}
  int4* res_s = reinterpret_cast<int4*>(dyn + so.rows);  // the stream's segment results, fetched at once
  for (int i = tid; i < 2 * nseg; i += nthreads) res_s[i] = __ldcg(reinterpret_cast<const int4*>(seg_res) + i);
  __syncthreads();
  if (tid == 0) {
    int seg = 0, ptok = 0, pval = 0, n = 0, cnt = 0, fin_state = bound ? 0 : -1, fin_t = 0, bad = nseg == 0;
    for (int hop = 0; hop < nseg && !bad && end > 0; ++hop) {
      const int4 ra = res_s[2 * seg], rb = res_s[2 * seg + 1];
      if (rb.y || ra.x < ptok || ra.y < pval) { bad = 1; break; }
      hops[2 * cnt] = make_int4(seg, ptok, ra.x, n);
      hops[2 * cnt + 1] = make_int4(pval, ra.y, 0, 0);
      ++cnt;
      n += ra.x - ptok;
      fin_state = ra.z; fin_t = ra.w;
      if (!rb.x) break;                                   // decoded to the end of the stream
      const int tcm = ra.w;
      const int j = min(tcm / L, nseg - 1);               // the owner of frame start tcm
      if (j <= seg) { bad = 1; break; }
      const int2 aux = __ldcg(trace_aux + tcm);
      seg = j; ptok = aux.x; pval = aux.y;
      if (hop == nseg - 1) bad = 1;                       // a chain longer than the number of segments
    }
    if (bad && usable && end > 0) atomicOr(p.status, TB_STATUS_STEP_LIMIT);
    blk_vars[1] = cnt; blk_vars[2] = n; blk_vars[3] = fin_state; blk_vars[4] = fin_t;
  }
  __syncthreads();
  {
    const int cnt = blk_vars[1];
    int32_t* o_tok = p.out_tokens + static_cast<int64_t>(b) * p.out_cap;
    int32_t* o_frm = p.out_frames + static_cast<int64_t>(b) * p.out_cap;
    for (int hcur = 0; hcur < cnt; ++hcur) {
      const int4 ha = hops[2 * hcur];
      const int32_t* l_tok = P.log_tok + static_cast<int64_t>(b) * P.log_stride + P.seg_off[ha.x];
      const int32_t* l_frm = P.log_frm + static_cast<int64_t>(b) * P.log_stride + P.seg_off[ha.x];
      for (int j = ha.y + tid; j < ha.z; j += nthreads) {
        const int o = ha.w + j - ha.y;
        if (o < p.out_cap) { o_tok[o] = __ldcg(l_tok + j); o_frm[o] = __ldcg(l_frm + j); }
      }
    }
    // The score is the sum of the visited rows' values in visiting order: the chain's values are brought into
    // shared memory by all threads, a piece at a time, and added one by one by a single thread.
    float* vbuf = reinterpret_cast<float*>(dyn + so.rows + 2 * kSegCap * 16);
    const int vcap = ((G + H) * kRowBufs * so.row_buf - 2 * kSegCap * 16) / 4;
    float score = 0.0f;
    int hcur = 0, pos = cnt > 0 ? hops[1].x : 0;           // next value to fetch: hop and index in that hop's log
    while (hcur < cnt) {
      // this piece: up to vcap values starting at (hcur, pos); every thread walks the hops the same way
      int filled = 0, hc = hcur, ps = pos;
      while (hc < cnt && filled < vcap) {
        const int4 ha = hops[2 * hc], hb = hops[2 * hc + 1];
        const float* l_val = P.log_val + static_cast<int64_t>(b) * P.log_stride + P.seg_off[ha.x];
        const int take = min(hb.y - ps, vcap - filled);
        for (int j = tid; j < take; j += nthreads) vbuf[filled + j] = __ldcg(l_val + ps + j);
        filled += take; ps += take;
        if (ps >= hb.y) { ++hc; ps = hc < cnt ? hops[2 * hc + 1].x : 0; }
      }
      __syncthreads();
      if (tid == 0) {
        int i = 0;
        for (; i + 8 <= filled; i += 8) {
          const float4 a4 = *reinterpret_cast<const float4*>(vbuf + i), b4 = *reinterpret_cast<const float4*>(vbuf + i + 4);
          score = __fadd_rn(score, a4.x); score = __fadd_rn(score, a4.y); score = __fadd_rn(score, a4.z); score = __fadd_rn(score, a4.w);
          score = __fadd_rn(score, b4.x); score = __fadd_rn(score, b4.y); score = __fadd_rn(score, b4.z); score = __fadd_rn(score, b4.w);
        }
        for (; i < filled; ++i) score = __fadd_rn(score, vbuf[i]);
      }
      __syncthreads();
      hcur = hc; pos = ps;
    }
    if (tid == 0) {
      p.out_counts[b] = blk_vars[2]; p.out_scores[b] = score; p.out_states[b] = blk_vars[3];
      if (p.out_cursors) p.out_cursors[b] = blk_vars[4];
      P.done[b] = 0u;
      P.epoch[b] = tag;
    }
  }
}

struct SegLayout {
  size_t log_tok, log_frm, log_val, trace_st, trace_aux, seg_res, done, epoch, total;
  int64_t log_stride;
  int32_t seg_off[kSegCap + 1];
};
SegLayout seg_layout(int32_t n_streams, int32_t frames, int32_t S, int32_t nseg_max) {
  SegLayout l;
  int64_t o = 0;
  for (int i = 0; i <= kSegCap; ++i) {
    l.seg_off[i] = static_cast<int32_t>(o);
    if (i < nseg_max) {
      // segment i decodes at most the frames from its (warmed-up) start to the end of the stream
      const int64_t fr = (static_cast<int64_t>(frames) * (nseg_max - i) + nseg_max - 1) / nseg_max + kWarm + 1;
      o += ((fr < frames ? fr : frames) * S + 35) & ~static_cast<int64_t>(31);
    }
  }
  l.log_stride = o;
  const size_t n = static_cast<size_t>(n_streams);
  auto up = [](size_t x) { return (x + 255) & ~static_cast<size_t>(255); };
  size_t off = 0;
  l.log_tok = off; off += up(n * l.log_stride * 4);
  l.log_frm = off; off += up(n * l.log_stride * 4);
  l.log_val = off; off += up(n * l.log_stride * 4);
  l.trace_st = off; off += up(n * (static_cast<size_t>(frames) + 1) * 8);
  l.trace_aux = off; off += up(n * (static_cast<size_t>(frames) + 1) * 8);
  l.seg_res = off; off += up(n * nseg_max * sizeof(SegRes));
  l.done = off; off += up(n * 4);
  l.epoch = off; off += up(n * 4);
  l.total = off;
  return l;
}

}  // namespace

// How the segmented kernel would lay out a call: blocks per stream, pipelines and helpers per block.  Returns false
// when the call is outside what the kernel covers.
bool tb_greedy_seg_plan(const TbDecodeParams& d, int32_t max_cache_bytes, int32_t all_resolved, int32_t n_sm,
                        int32_t max_smem, TbSegPlan* plan) {
  const int W = d.V + 1;
  if (d.dtype != TB_BF16 || d.persistent || d.n_dur != 0) return false;
  if (d.sv != 1 || d.ss != W || d.st < static_cast<int64_t>(d.S) * W || d.sb < 0) return false;
  if (d.S > kSMax || d.V > 256 * kNitMax || 2 * (d.V + 1) > (1 << TB_RS_TOK_BITS)) return false;
  if (reinterpret_cast<uintptr_t>(d.logits) & 1) return false;
  if (!all_resolved || d.frames < 1 || d.n_streams < 1) return false;
  // blocks per SM by shared memory, then by threads (the register file holds 640 threads of this kernel)
  int G = 2, H = 8;                                         // (measured best on workload 2 among 2+4 .. 4+6)
  if (plan->force_G > 0) { G = plan->force_G; H = plan->force_H; }
  if (G < 1 || G > kGMax || H < 1 || (G + H) * 32 > kMaxThreadsS || G + H <= 4 * (G - 1)) return false;
  const int smem = carve_s(G, H, d.V, d.C, max_cache_bytes).total;
  if (smem > max_smem - 1024) return false;
  int per_sm = (max_smem - 1024) / (smem + 1024);
  const int by_threads = kMaxThreadsS / ((G + H) * 32);
  if (per_sm > by_threads) per_sm = by_threads;
  if (per_sm < 1) return false;
  const int64_t slots = static_cast<int64_t>(per_sm) * n_sm;
  int NB = static_cast<int>(slots / d.n_streams);
  // Cutting streams into segments pays when a batch leaves most SMs without a stream of their own: measured on
  // workload 2, 16 / 32 streams decode in 0.20 / 0.25 ms against 0.31 / 0.32 ms with one block per stream, 64
  // streams in the same time, 128 streams slower (0.54 against 0.34 ms).  Unless the caller asks for it, the
  // segmented kernel is therefore used only with at least five blocks per stream.
  if (plan->force_NB > 0) NB = plan->force_NB;
  else if (plan->force_G == 0 && NB < 5) return false;
  const int most = (d.frames / kSegMinLen + G - 1) / G;      // more blocks than that would have nothing to do
  if (NB > most) NB = most;
  if (NB * G > kSegCap) NB = kSegCap / G;
  if (NB < 1) NB = 1;
  plan->G = G; plan->H = H; plan->NB = NB; plan->smem = smem;
  return true;
}

size_t tb_greedy_seg_scratch_bytes(int32_t n_streams, int32_t frames, int32_t S, int32_t nseg_max) {
  return seg_layout(n_streams, frames, S, nseg_max).total;
}

// Launches the segmented decode.  scratch: device memory of at least tb_greedy_seg_scratch_bytes(...), zeroed once
// when it was allocated or when the call's shape (streams, frames, rows, segments) last changed; between launches of
// the same shape the kernel keeps it consistent by itself.
int tb_launch_greedy_seg(const TbDecodeParams& d, int32_t max_cache_bytes, const TbSegPlan& plan, void* scratch,
                         cudaStream_t stream) {
  SegParams P;
  P.d = d;
  P.G = plan.G; P.H = plan.H; P.NB = plan.NB; P.nseg_max = plan.NB * plan.G; P.cache_bytes = max_cache_bytes;
  P.spin_limit = plan.test_timeout ? 4096u : kSpinLimitS;
  P.withhold_frame = plan.test_timeout ? d.frames / 2 : -1;
  P.tensor_lo = reinterpret_cast<const unsigned char*>(d.logits);
  const int64_t last = static_cast<int64_t>(d.n_streams - 1) * d.sb + static_cast<int64_t>(d.frames - 1) * d.st +
                       static_cast<int64_t>(d.S - 1) * d.ss + d.V;
  P.tensor_hi = P.tensor_lo + 2 * (last + 1);
  const SegLayout l = seg_layout(d.n_streams, d.frames, d.S, P.nseg_max);
  unsigned char* sb = static_cast<unsigned char*>(scratch);
  P.log_tok = reinterpret_cast<int32_t*>(sb + l.log_tok);
  P.log_frm = reinterpret_cast<int32_t*>(sb + l.log_frm);
  P.log_val = reinterpret_cast<float*>(sb + l.log_val);
  P.log_stride = l.log_stride;
  for (int i = 0; i <= kSegCap; ++i) P.seg_off[i] = l.seg_off[i];
  P.trace_st = reinterpret_cast<unsigned long long*>(sb + l.trace_st);
  P.trace_aux = reinterpret_cast<int2*>(sb + l.trace_aux);
  P.seg_res = reinterpret_cast<SegRes*>(sb + l.seg_res);
  P.done = reinterpret_cast<uint32_t*>(sb + l.done);
  P.epoch = reinterpret_cast<uint32_t*>(sb + l.epoch);
  const int nit = (d.V + 255) / 256;
  void (*fn)(SegParams) = nit <= 1 ? k_greedy_seg<1, false> : nit <= 2 ? k_greedy_seg<2, false> : nit <= 4 ? k_greedy_seg<4, false> : k_greedy_seg<8, false>;
  // rows normalised inside the selection (log-softmax): the helpers also leave every row's normaliser
  if (d.normalize) fn = nit <= 1 ? k_greedy_seg<1, true> : nit <= 2 ? k_greedy_seg<2, true> : nit <= 4 ? k_greedy_seg<4, true> : k_greedy_seg<8, true>;
  if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, plan.smem) != cudaSuccess) {
    cudaGetLastError();
    return TB_ERR_CUDA;
  }
  fn<<<d.n_streams * plan.NB, (plan.G + plan.H) * 32, plan.smem, stream>>>(P);
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}

