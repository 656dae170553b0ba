// General decode kernels: one thread block per stream (or per stream's beam), any strides,
// any vocabulary up to TB_MAX_VOCAB, RNNT and TDT, offline and streaming.  Every row is
// evaluated exactly as the arithmetic contract in tb.h states.  These kernels are the
// reference device path; the pipelined greedy kernel in tb_greedy_fast.cu covers the packed
// layouts at streaming rate and falls back to this one otherwise.
#include <cfloat>

#include "tb_device.cuh"
#include "tb_launch.h"

namespace {

constexpr int kThreads = 256;
constexpr int kBeamList = 64;   // boosted tokens per hypothesis kept for the next-state lookup of the beam step

struct ChainSmem {
  int32_t state[TB_CHAIN_MAX];
  float acc[TB_CHAIN_MAX];
  int32_t len;
};

// Shared state of one block's sequential decode.
struct StepSmem {
  ValId red[kThreads / 32 + 1];
  ChainSmem chain;
  int32_t t, k, s, tok, go;
};

// Token view of the current graph state, for graphs that carry resolved lists (see TbRsRec):
// instead of walking the suffix chain into a class-indexed bonus vector, the state's finished list
// is scattered into two token-indexed arrays; a token that is not in the list ("plain") gets
// fl(lambda * fl(D + root arc weight of its class)) and the root arc's target.
struct TokView {
  float* rootcw;      // [C] root arc weight per class (0 if none)
  int32_t* rootdst;   // [C] root arc target per class (0 if none)
  float* tok_lb;      // [V] finished additive term of a listed token
  int32_t* tok_dst;   // [V] target state of a listed token, -1: not listed
  uint16_t* cur_tok;  // tokens of the list now scattered (to undo it)
  int32_t n;
  float D;
};
__host__ __device__ inline size_t tokview_bytes(int V, int C) {
  return static_cast<size_t>(C) * 8 + static_cast<size_t>(V) * 8 + ((static_cast<size_t>(V) * 2 + 8 + 15) & ~size_t(15));
}
// The beam kernels' auxiliary shared memory behind the candidate arrays: class vectors or the token view.
__host__ __device__ inline size_t beam_aux_bytes(int V, int C, int tokview) {
  size_t a = static_cast<size_t>(C) * 8;
  if (tokview && tokview_bytes(V, C) > a) a = tokview_bytes(V, C);
  return (a + 15) & ~size_t(15);
}
__device__ inline void tokview_init(TokView& tv, unsigned char* mem, int V, int C, const GraphPtrs& g) {
  tv.rootcw = reinterpret_cast<float*>(mem);
  tv.rootdst = reinterpret_cast<int32_t*>(mem + 4 * static_cast<size_t>(C));
  tv.tok_lb = reinterpret_cast<float*>(mem + 8 * static_cast<size_t>(C));
  tv.tok_dst = reinterpret_cast<int32_t*>(mem + 8 * static_cast<size_t>(C) + 4 * static_cast<size_t>(V));
  tv.cur_tok = reinterpret_cast<uint16_t*>(mem + 8 * static_cast<size_t>(C) + 8 * static_cast<size_t>(V));
  tv.n = 0; tv.D = 0.0f;
  for (int c = threadIdx.x; c < C; c += blockDim.x) { tv.rootcw[c] = 0.0f; tv.rootdst[c] = 0; }
  for (int v = threadIdx.x; v < V; v += blockDim.x) tv.tok_dst[v] = -1;
  __syncthreads();
  const int e = g.arc_begin[1];
  for (int a = g.arc_begin[0] + threadIdx.x; a < e; a += blockDim.x) {
    const int c = g.arc_cls[a];
    if (c >= 0 && c < C) { tv.rootcw[c] = __fadd_rn(0.0f, g.arc_w[a]); tv.rootdst[c] = g.arc_dst[a]; }
  }
  __syncthreads();
}
// The same tables, already filled by an earlier tokview_init of this block with the same arguments.
__device__ inline void tokview_attach(TokView& tv, unsigned char* mem, int V, int C) {
  tv.rootcw = reinterpret_cast<float*>(mem);
  tv.rootdst = reinterpret_cast<int32_t*>(mem + 4 * static_cast<size_t>(C));
  tv.tok_lb = reinterpret_cast<float*>(mem + 8 * static_cast<size_t>(C));
  tv.tok_dst = reinterpret_cast<int32_t*>(mem + 8 * static_cast<size_t>(C) + 4 * static_cast<size_t>(V));
  tv.cur_tok = reinterpret_cast<uint16_t*>(mem + 8 * static_cast<size_t>(C) + 8 * static_cast<size_t>(V));
  tv.n = 0; tv.D = 0.0f;
}
// Block-wide: replace the scattered list by that of state s (the root's list is empty, D = 0).
__device__ inline void tokview_enter(TokView& tv, const unsigned char* blob, const TbSlotRec& rec, int32_t s, int V,
                                     int32_t* status) {
  for (int i = threadIdx.x; i < tv.n; i += blockDim.x) {
    const int tk = tv.cur_tok[i];
    if (tk < V) tv.tok_dst[tk] = -1;
  }
  __syncthreads();
  if (s < 0 || s >= rec.n_states) { if (threadIdx.x == 0) atomicOr(status, TB_STATUS_BAD_STATE); s = 0; }
  const TbRsRec r = reinterpret_cast<const TbRsRec*>(blob + rec.off_rsrec)[s];
  const TbRsEnt* ent = reinterpret_cast<const TbRsEnt*>(blob + rec.off_rsent) + r.begin;
  const int n = min(r.count, V + 4);
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const TbRsEnt e = ent[i];
    const int tk = static_cast<int>((e.dst_tok & ((1u << TB_RS_TOK_BITS) - 1u)) >> 1);   // padding entries carry token V
    if (tk < V) { tv.tok_lb[tk] = e.lb; tv.tok_dst[tk] = static_cast<int32_t>(e.dst_tok >> TB_RS_TOK_BITS); }
    tv.cur_tok[i] = static_cast<uint16_t>(tk);
  }
  __syncthreads();
  tv.n = n; tv.D = r.D;
}

template <typename LT>
__global__ void __launch_bounds__(kThreads) k_decode_general(TbDecodeParams p, TbInlineBinds ib) {
  extern __shared__ __align__(16) unsigned char dyn[];
  float* bvec = reinterpret_cast<float*>(dyn);
  int32_t* nvec = reinterpret_cast<int32_t*>(dyn + sizeof(float) * p.C);
  __shared__ StepSmem sm;
  __shared__ float fred[kThreads / 32];

  const int b = blockIdx.x;
  TbSlotRec rec = p.slots[b];
  // A bind that travels with this launch (streaming chunks): the block of a re-bound slot brings the new graph's
  // image from page-locked host memory into its arena block itself, then stores the slot's new record; every other
  // block is on its way already.
  bool rebound = false;
  if (ib.n > 0) {
    int hit = -1;
#pragma unroll
    for (int i = 0; i < TB_INLINE_BINDS; ++i)
      if (i < ib.n && ib.slot[i] == b) hit = i;
    if (hit >= 0) {
      const unsigned char* src = nullptr;
      int32_t bytes = 0;
#pragma unroll
      for (int i = 0; i < TB_INLINE_BINDS; ++i)
        if (hit == i) { src = ib.src[i]; bytes = ib.bytes[i]; rec = ib.rec[i]; }
      rebound = true;
      const uint4* s16 = reinterpret_cast<const uint4*>(src);
      uint4* d16 = reinterpret_cast<uint4*>(ib.arena + rec.blob_off);
      const int n16 = (bytes + 15) >> 4;             // (both blocks are padded to the arena's granule)
      for (int j0 = 0; j0 < n16; j0 += 8 * kThreads) {
        uint4 v[8];                                    // eight loads per thread on their way across the bus at once
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int j = j0 + u * kThreads + threadIdx.x;
          if (j < n16) v[u] = s16[j];
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int j = j0 + u * kThreads + threadIdx.x;
          if (j < n16) d16[j] = v[u];
        }
      }
      __threadfence();
      __syncthreads();
      if (threadIdx.x == 0) ib.slots[b] = rec;
    }
  }
  const bool bound = rec.n_states > 0;
  const GraphPtrs g = graph_of(p.arena, rec);
  const unsigned char* blob = p.arena + rec.blob_off;
  const bool use_tv = bound && rec.n_rsent >= 0 && p.tokview;   // resolved lists: token view instead of a chain walk
  TokView tv;
  if (use_tv) tokview_init(tv, dyn, p.V, p.C, g);
  const LT* base = reinterpret_cast<const LT*>(p.logits) + static_cast<int64_t>(b) * p.sb;
  const int V = p.V;

  // where this call starts and ends for the stream
  int32_t t0 = 0, end, s, t, k, n_total = 0;
  float score;
  if (p.persistent) {
    TbSlotState st = p.sstate[b];
    if (rebound) { st.state = rec.n_states > 0 ? 0 : -1; st.t = 0; st.k = 0; st.score = 0.0f; st.n_emitted = 0; st.chunk_base = 0; }
    t0 = st.chunk_base; s = st.state; t = st.t; k = st.k; score = st.score; n_total = st.n_emitted;
    int32_t valid = p.lengths ? p.lengths[b] : INT32_MAX;
    end = min(t0 + p.frames, valid);
  } else {
    s = bound ? 0 : -1; t = 0; k = 0; score = 0.0f;
    int32_t len = p.lengths ? p.lengths[b] : p.frames;
    end = max(0, min(len, p.frames));
  }
  if (!bound) s = -1;
  int32_t n_out = 0;
  int32_t built_for = -2;  // state the bonus vector currently describes

  const int64_t max_steps = static_cast<int64_t>(p.frames) * p.S;
  for (int64_t it = 0; t < end; ++it) {
    if (it >= max_steps) {  // every step emits or closes a frame, so this cannot happen
      if (threadIdx.x == 0) atomicOr(p.status, TB_STATUS_STEP_LIMIT);
      break;
    }
    if (bound && built_for != s) {
      if (use_tv) tokview_enter(tv, blob, rec, s, V, p.status);
      else build_bonus(g, s, p.C, bvec, nvec, sm.chain.state, sm.chain.acc, &sm.chain.len, p.status);
      built_for = s;
    }
    const LT* row = base + static_cast<int64_t>(t - t0) * p.st + static_cast<int64_t>(k) * p.ss;
    float lse = 0.0f;
    if (p.normalize) {
      // log-softmax fused into the selection: L = m + log(sum_v exp(x_v - m)) over the row's V+1 entries, in
      // float with a fixed order of additions (per thread by index, then lanes, then warps), so that a launch
      // repeats bit for bit; every entry becomes x_v - L before its bonus is added
      float m = -INFINITY;
      for (int v = threadIdx.x; v <= V; v += kThreads) m = fmaxf(m, LogitLoad<LT>::at(row + static_cast<int64_t>(v) * p.sv));
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
      if ((threadIdx.x & 31) == 0) fred[threadIdx.x >> 5] = m;
      __syncthreads();
      m = fred[0];
      for (int w2 = 1; w2 < kThreads / 32; ++w2) m = fmaxf(m, fred[w2]);
      __syncthreads();
      float sum = 0.0f;
      for (int v = threadIdx.x; v <= V; v += kThreads) sum = __fadd_rn(sum, expf(__fsub_rn(LogitLoad<LT>::at(row + static_cast<int64_t>(v) * p.sv), m)));
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) sum = __fadd_rn(sum, __shfl_xor_sync(0xffffffffu, sum, off));
      if ((threadIdx.x & 31) == 0) fred[threadIdx.x >> 5] = sum;
      __syncthreads();
      sum = fred[0];
      for (int w2 = 1; w2 < kThreads / 32; ++w2) sum = __fadd_rn(sum, fred[w2]);
      __syncthreads();
      lse = m == -INFINITY ? 0.0f : __fadd_rn(m, logf(sum));
    }
    ValId best{-INFINITY, INT32_MAX};
    for (int v = threadIdx.x; v <= V; v += kThreads) {
      float x = LogitLoad<LT>::at(row + static_cast<int64_t>(v) * p.sv);
      if (p.normalize) x = __fsub_rn(x, lse);
      float val = x;
      if (bound && v < V) {
        if (use_tv) {
          const float lb = tv.tok_dst[v] >= 0 ? tv.tok_lb[v]
                                              : __fmul_rn(g.lambda, __fadd_rn(tv.D, tv.rootcw[__ldg(p.cls + v)]));
          val = __fadd_rn(x, lb);
        } else {
          val = __fadd_rn(x, __fmul_rn(g.lambda, bvec[__ldg(p.cls + v)]));
        }
      }
      ValId c{val, v};
      if (better(c, best)) best = c;
    }
    best = block_best(best, sm.red);
    // every thread now holds the same (value, token); all of them advance the same cursor
    const int tok = best.i;
    float add = best.v;
    int dur = 0;
    if (p.n_dur > 0) {
      float bd = 0.0f;
      for (int d = 0; d < p.n_dur; ++d) {
        float xd = LogitLoad<LT>::at(row + static_cast<int64_t>(V + 1 + d) * p.sv);
        if (d == 0 || xd > bd) { bd = xd; dur = d; }
      }
      add = __fadd_rn(add, bd);
    }
    score = __fadd_rn(score, add);
    if (tok == V) {
      t += (p.n_dur > 0) ? max(dur, 1) : 1;
      k = 0;
    } else {
      if (threadIdx.x == 0 && n_out < p.out_cap) {
        const int64_t o = static_cast<int64_t>(b) * p.out_cap + n_out;
        p.out_tokens[o] = tok;
        p.out_frames[o] = t;
        if (p.out_durs) p.out_durs[o] = dur;
      }
      ++n_out;
      if (bound) s = use_tv ? (tv.tok_dst[tok] >= 0 ? tv.tok_dst[tok] : tv.rootdst[__ldg(p.cls + tok)]) : nvec[__ldg(p.cls + tok)];
      if (p.n_dur > 0 && dur > 0) { t += dur; k = 0; }
      else { ++k; if (k == p.S) { ++t; k = 0; } }
    }
    __syncthreads();  // nvec / bvec are read above and may be rebuilt next
  }

  if (threadIdx.x == 0) {
    p.out_counts[b] = n_out;
    p.out_scores[b] = score;
    p.out_states[b] = s;
    if (p.out_cursors) p.out_cursors[b] = t;
    if (p.persistent) {
      TbSlotState st;
      st.state = s; st.t = t; st.k = k; st.score = score; st.n_emitted = n_total + n_out;
      st.chunk_base = t0 + p.frames; st.pad0 = 0; st.pad1 = 0;
      p.sstate[b] = st;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// beam step
// ---------------------------------------------------------------------------------------------

struct BeamKey {  // order: value descending, token key ascending, parent ascending
  float v;
  int32_t tkey, par;
};
// One beam expansion of the block's stream (the body of k_beam_step; k_beam_frames calls it once per row).
// The K largest of the keys ckey[first], ckey[first + stride], ... (those below n; 0 = no candidate) that this warp's
// lanes look at, R per lane: out_key[r] / out_idx[r] for r < K, best first (key 0, index -1 once nothing is left).
// Every lane keeps its keys sorted in registers, so a round is two warp-wide integer maxima over the lanes' heads;
// the lane that holds the winner finds its index again (one of its R places in the array) and moves up its other keys.
template <int R>
__device__ __forceinline__ void warp_top_keys(const unsigned long long* ckey, int n, int first, int stride, int K, int lane,
                                              unsigned long long* out_key, int32_t* out_idx) {
  unsigned long long ck[R];
#pragma unroll
  for (int j = 0; j < R; ++j) { const int i = first + stride * j; ck[j] = i < n ? ckey[i] : 0ull; }
  auto ce = [&](int a, int b) { const bool sw = ck[b] > ck[a]; const unsigned long long hi = sw ? ck[b] : ck[a], lo = sw ? ck[a] : ck[b]; ck[a] = hi; ck[b] = lo; };
  if (R == 2) { ce(0, 1); }
  if (R == 4) { ce(0, 1); ce(2, 3); ce(0, 2); ce(1, 3); ce(1, 2); }
  if (R == 8) {
    ce(0, 1); ce(2, 3); ce(4, 5); ce(6, 7); ce(0, 2); ce(1, 3); ce(4, 6); ce(5, 7); ce(1, 2); ce(5, 6);
    ce(0, 4); ce(1, 5); ce(2, 6); ce(3, 7); ce(2, 4); ce(3, 5); ce(1, 2); ce(3, 4); ce(5, 6);
  }
  for (int r = 0; r < K; ++r) {
    const unsigned long long a = ck[0];
    const uint32_t hi = static_cast<uint32_t>(a >> 32), lo = static_cast<uint32_t>(a);
    const uint32_t mh = __reduce_max_sync(0xffffffffu, hi);
    const uint32_t ml = __reduce_max_sync(0xffffffffu, hi == mh ? lo : 0u);
    const unsigned long long best = (static_cast<unsigned long long>(mh) << 32) | ml;
    if (best == 0ull) {
      if (lane == 0) { out_key[r] = 0ull; out_idx[r] = -1; }
    } else if (a == best) {
      int idx = -1;
#pragma unroll
      for (int j = 0; j < R; ++j) { const int i = first + stride * j; if (i < n && ckey[i] == best) idx = i; }
      out_key[r] = best; out_idx[r] = idx;
#pragma unroll
      for (int j = 0; j + 1 < R; ++j) ck[j] = ck[j + 1];
      ck[R - 1] = 0ull;
    }
  }
}

// threads of a beam block: more warps than the general kernel's hide the latencies of its short dependent phases; 17
// warps take a row of 1025 logits (vocabularies of about a thousand pieces) in two strides instead of three
constexpr int kBeamThreads = 544;
constexpr int kBeamPref = 5;   // elements of a shared row each thread may hold ahead of time (rows up to 5 * kBeamThreads wide)
// xpre / xpre_valid: this thread's elements of the stream's shared row, fetched ahead by the previous step of the same
// launch; next_row: where the next step's shared row starts (null: none), fetched while this step selects.
// What a beam block keeps in shared memory besides its candidate arrays: the stream's hypotheses from step to step,
// and the working set of a step.
constexpr int kTeamMaxK = 8;   // (= kFastMaxK, needed here already)
struct BeamShared {
  ChainSmem chain;
  // token-view path: per hypothesis a copy of its state's short list, to find the next state of a pick
  uint16_t hl_tok[TB_MAX_BEAM][kBeamList];
  int32_t hl_dst[TB_MAX_BEAM][kBeamList];
  int32_t hl_n[TB_MAX_BEAM];                                 // -1: list too long, walk the chain instead
  int32_t h_beg[TB_MAX_BEAM], h_cnt[TB_MAX_BEAM];
  float h_D[TB_MAX_BEAM];
  unsigned long long red64[2][kBeamThreads / 32];   // the warps' best keys, two copies used in turn by the selection rounds
  float h_score[TB_MAX_BEAM];
  int32_t h_state[TB_MAX_BEAM];
  uint8_t h_live[TB_MAX_BEAM];
  unsigned long long h_hash[TB_MAX_BEAM];   // identity of the hypothesis' token sequence
  int32_t h_len[TB_MAX_BEAM];
  BeamKey sel[TB_MAX_BEAM];
  int32_t sel_dst[TB_MAX_BEAM];      // compact path: the graph state a selected candidate leads to
  int32_t cp_n, cp_flag;             // compact path: candidates laid out; 0 = this step cannot take it
  int32_t cp_off[TB_MAX_BEAM + 1];   // compact path: where each hypothesis' listed candidates start
  int32_t rec_ready;                 // the hypotheses' list records in h_beg / h_cnt / h_D are those of their current states
  TbTopEnt ttop[2 * TB_MAX_BEAM + 9]; // this step's reduced row
  float root_wmax;                   // largest |root arc weight| of the stream's graph (filled with the root tables)
  int32_t fast_done;                 // narrow beams: steps the team has just taken
  // narrow beams, between the team's warps: the hypotheses a step works on, each worker's picks and bound term
  float f_sc[kTeamMaxK]; int32_t f_st[kTeamMaxK]; uint8_t f_lv[kTeamMaxK];
  unsigned long long f_key[kTeamMaxK][kTeamMaxK]; int32_t f_dst[kTeamMaxK][kTeamMaxK];
  float f_ub[kTeamMaxK];
  volatile int32_t f_cmd, f_fail;    // 1: the run ends here / a worker met a list it cannot take
};

template <typename LT>
__device__ __forceinline__ void beam_step_body(const TbBeamParams& p, BeamShared& sh, LT (&xpre)[kBeamPref], bool& xpre_valid,
                                               const LT* next_row, TbTopEnt& tpre, bool& tpre_valid,
                                               const TbTopEnt* next_top) {
  extern __shared__ __align__(16) unsigned char dyn[];
  const int V = p.V, K = p.K, W = V + 1;
  float* cand = reinterpret_cast<float*>(dyn);                         // [K, V+1]
  const int WW = (W + 31) >> 5;
  uint32_t* ovr = reinterpret_cast<uint32_t*>(dyn + ((static_cast<size_t>(K) * W * sizeof(float) + 15) & ~size_t(15)));   // [K, WW] bits: the value in cand is a boosted one
  unsigned char* aux = reinterpret_cast<unsigned char*>(ovr) + ((static_cast<size_t>(K) * WW * sizeof(uint32_t) + 15) & ~size_t(15));
  float* bvec = reinterpret_cast<float*>(aux);                         // [C]   (chain-walk path)
  int32_t* nvec = reinterpret_cast<int32_t*>(bvec + p.C);              // [C]
  ChainSmem& chain = sh.chain;
  auto& hl_tok = sh.hl_tok; auto& hl_dst = sh.hl_dst; auto& hl_n = sh.hl_n;
  auto& h_beg = sh.h_beg; auto& h_cnt = sh.h_cnt; auto& h_D = sh.h_D;
  auto& red64 = sh.red64;
  auto& h_score = sh.h_score; auto& h_state = sh.h_state; auto& h_live = sh.h_live; auto& h_hash = sh.h_hash; auto& h_len = sh.h_len;
  auto& sel = sh.sel; auto& sel_dst = sh.sel_dst;
  int32_t& cp_n = sh.cp_n; int32_t& cp_flag = sh.cp_flag;
  auto& cp_off = sh.cp_off;
  int32_t& rec_ready = sh.rec_ready;
  auto& ttop = sh.ttop;
  float& root_wmax = sh.root_wmax;

  const int b = blockIdx.x;
  const TbSlotRec rec = p.slots[b];
  const bool bound = rec.n_states > 0;
  const GraphPtrs g = graph_of(p.arena, rec);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned char* blob = p.arena + rec.blob_off;
  const bool use_tv = bound && rec.n_rsent >= 0 && p.tokview;
  // rows shared by the hypotheses of a stream (hyp_stride 0) depend on nothing that is loaded below: fetch this
  // thread's elements now, so that their latency overlaps the loads of the slot record, states and lists
  constexpr int kPref = kBeamPref;
  const bool pref = (use_tv || (!bound && p.top_row != nullptr)) && p.hyp_stride == 0 && W <= kPref * kBeamThreads;
  if (pref && !xpre_valid) {
    const LT* row0 = reinterpret_cast<const LT*>(p.logits) + static_cast<int64_t>(b) * p.stream_stride;
#pragma unroll
    for (int j = 0; j < kPref; ++j) {
      const int v = threadIdx.x + j * kBeamThreads;
      if (v < W) xpre[j] = LogitLoad<LT>::raw(row0 + v);
    }
  }
  TokView tv;
  if (use_tv) {
    if (p.tv_ready) tokview_attach(tv, aux, V, p.C);      // a later step of the same launch: the root tables are there
    else {
      tokview_init(tv, aux, V, p.C, g);
      if (warp == 0) {
        float r = 0.0f;
        for (int c = lane; c < p.C; c += 32) r = fmaxf(r, fabsf(tv.rootcw[c]));
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) r = fmaxf(r, __shfl_xor_sync(0xffffffffu, r, off));
        if (lane == 0) root_wmax = r;
      }
    }
  } else if (!p.tv_ready && threadIdx.x == 0) {
    root_wmax = 0.0f;
  }

  if (threadIdx.x < K) {
    if (p.tv_ready) {
      // a later step of the same launch: the previous step left its hypotheses in shared memory
      if (p.new_frame) h_live[threadIdx.x] = static_cast<uint8_t>(h_score[threadIdx.x] != -INFINITY);
    } else {
      const int64_t o = static_cast<int64_t>(b) * K + threadIdx.x;
      float sc = p.scores[o];
      h_score[threadIdx.x] = sc;
      h_state[threadIdx.x] = p.states[o];
      h_live[threadIdx.x] = p.new_frame ? static_cast<uint8_t>(sc != -INFINITY) : p.live[o];
      h_hash[threadIdx.x] = p.fresh ? 0ull : p.hash_in[o];
      h_len[threadIdx.x] = p.fresh ? 0 : p.len_in[o];
    }
  }
  __syncthreads();
  if (p.merge) {
    // hypotheses that have emitted the same token sequence are one transcript: the first in selection order (the
    // best) stays, the others become empty places before anything is expanded
    bool dup = false;
    if (threadIdx.x < K && h_score[threadIdx.x] != -INFINITY) {
      const int k = threadIdx.x;
      for (int j = 0; j < k; ++j)
        if (h_score[j] != -INFINITY && h_len[j] == h_len[k] && h_hash[j] == h_hash[k] && h_state[j] == h_state[k]) { dup = true; break; }
    }
    __syncthreads();
    if (dup) { h_score[threadIdx.x] = -INFINITY; h_state[threadIdx.x] = -1; h_live[threadIdx.x] = 0; }
    __syncthreads();
  }
  if (p.prune_delta >= 0.0f) {
    // still at the frame start: whatever scores below the best by more than the threshold becomes an empty place
    bool drop = false;
    if (threadIdx.x < K) {
      float best = -INFINITY;
      for (int j = 0; j < K; ++j) best = fmaxf(best, h_score[j]);
      const float sc = h_score[threadIdx.x];
      drop = sc != -INFINITY && sc < __fsub_rn(best, p.prune_delta);
    }
    __syncthreads();
    if (drop) { h_score[threadIdx.x] = -INFINITY; h_state[threadIdx.x] = -1; h_live[threadIdx.x] = 0; }
    __syncthreads();
  }

  auto make_key = [](float v, int tkey, int k) -> unsigned long long {
    const uint32_t u = __float_as_uint(v + 0.0f);             // -0 folded into +0: equal values, equal keys
    const uint32_t hi = u ^ ((u >> 31) ? 0xFFFFFFFFu : 0x80000000u);
    const uint32_t lo = 0xFFFFFFFFu - (static_cast<uint32_t>(tkey) * 32u + static_cast<uint32_t>(k));
    return (static_cast<unsigned long long>(hi) << 32) | lo;
  };
  // this thread's two best candidates, when the sweep below has already looked at all of them
  unsigned long long m1 = 0ull, m2 = 0ull;
  bool swept = false;
  auto offer = [&](unsigned long long kk) { if (kk > m1) { m2 = m1; m1 = kk; } else if (kk > m2) m2 = kk; };
  // ---- the compact path ---------------------------------------------------------------------------------
  // With the row reduced ahead of time to its top_m root-boosted tokens (k_beam_topm), a hypothesis' candidates are
  // its blank, the tokens its graph state lists (exact values from their entries) and the first tokens of that
  // short list which the state does not list (exact values from the list's logits): a few dozen per hypothesis
  // instead of vocab + 1.  Every token outside the list has y <= y_next, hence a value of at most
  // score + y_next + lambda * D plus roundings; the step is valid when the K-th selected candidate clears that
  // bound for every hypothesis by a margin that dominates the roundings.  Otherwise (or with a very long list)
  // the step is done again the long way below.
  bool compact_done = false;
  bool row_staged = false;      // the compact path put this step's row into shared memory and asked for the next one (in xpre)
  float* xrow_s = reinterpret_cast<float*>(aux + beam_aux_bytes(V, p.C, p.tokview));
  if (p.top_row != nullptr && p.hyp_stride == 0 && (use_tv || !bound) && p.top_m <= 2 * TB_MAX_BEAM + 8) {
    unsigned long long* ckey = reinterpret_cast<unsigned long long*>(cand);
    const int M = p.top_m;
    float* xrow = xrow_s;                                     // [W] this step's row, staged
    // the candidate arrays share the whole-row path's value array: keys, target states, then the warps' picks
    const int wsel_bytes = (kBeamThreads / 32) * TB_MAX_BEAM * 12;
    const int cap = (static_cast<int>(static_cast<size_t>(K) * W * sizeof(float)) - wsel_bytes - 16) / 12 & ~1;
    int32_t* cdst = reinterpret_cast<int32_t*>(ckey + cap);
    const LT* base = reinterpret_cast<const LT*>(p.logits) + static_cast<int64_t>(b) * p.stream_stride;
    const bool recs_at_hand = p.tv_ready && rec_ready;        // left by the previous step of this launch
    if (warp == 0) {
      // lane k: hypothesis k's list record (fetched now unless the previous step left it), then where its listed
      // candidates start in the candidate array: a prefix sum over the warp (K <= 32)
      const int k = lane;
      int cntk = 0;
      bool lv = false;
      if (k < K) {
        if (!recs_at_hand) {
          int32_t beg = 0;
          float Dk = 0.0f;
          if (bound && h_score[k] != -INFINITY) {
            int32_t st = h_state[k];
            if (st < 0 || st >= rec.n_states) { atomicOr(p.status, TB_STATUS_BAD_STATE); st = 0; }
            const TbRsRec r = reinterpret_cast<const TbRsRec*>(blob + rec.off_rsrec)[st];
            beg = r.begin; cntk = r.count; Dk = r.D;
          }
          h_beg[k] = beg; h_cnt[k] = cntk; h_D[k] = Dk;
        } else {
          cntk = h_cnt[k];
        }
        lv = h_score[k] != -INFINITY && h_live[k];
        hl_n[k] = !lv ? 0 : (cntk <= kBeamList ? cntk : -1);
      }
      const int c = lv ? cntk : 0;
      int incl = c;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += o;
      }
      if (k < K) cp_off[k] = incl - c;
      const int total = __shfl_sync(0xffffffffu, incl, 31);
      if (lane == 0) {
        cp_off[K] = total;
        cp_flag = total + K * (M + 1) <= cap ? 1 : 0;
        cp_n = total + K * (M + 1);
      }
    }
    for (int i = threadIdx.x; i < K * WW; i += kBeamThreads) ovr[i] = 0u;
    // the row and its reduced form, asked for during the previous step (or now), go to shared memory
    if (pref) {
#pragma unroll
      for (int j = 0; j < kPref; ++j) { const int v = threadIdx.x + j * kBeamThreads; if (v < W) xrow[v] = LogitLoad<LT>::widen(xpre[j]); }
    }
    if (threadIdx.x <= M) ttop[threadIdx.x] = tpre_valid ? tpre : p.top_row[threadIdx.x];
    __syncthreads();
    // the next step's row and reduced row are requested now: their trip overlaps the rest of this step
    row_staged = pref;
    xpre_valid = false;
    if (pref && next_row) {
#pragma unroll
      for (int j = 0; j < kPref; ++j) {
        const int v = threadIdx.x + j * kBeamThreads;
        if (v < W) xpre[j] = LogitLoad<LT>::raw(next_row + v);      // (the load alone: widened when it is used)
      }
      xpre_valid = true;
    }
    tpre_valid = false;
    if (next_top) { if (threadIdx.x <= M) tpre = next_top[threadIdx.x]; tpre_valid = true; }
    // (one warp doing a narrow beam's few dozen candidates by itself, with warp-wide synchronisation only, was
    // measured slower than the whole block; narrow beams are taken by a team of warps instead, see beam_fast_run)
    const int cth = static_cast<int>(threadIdx.x), cnt = kBeamThreads;
    {
      if (cp_flag) {
        const int n_listed = cp_off[K], n = cp_n;
        // the listed tokens of every hypothesis, all hypotheses at once: exact values; marked, so that the walk over
        // the reduced row leaves them out.  Candidate slots that stay unused hold key 0 (none).
        if (bound) {
          const TbRsEnt* ent = reinterpret_cast<const TbRsEnt*>(blob + rec.off_rsent);
          // (eight entries per thread are requested before the first is used: one trip to L2 for all of them)
          for (int q0 = cth; q0 < n_listed; q0 += 8 * cnt) {
            TbRsEnt e8[8];
            int k8[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int q = q0 + j * cnt;
              int k = 0;
              if (q < n_listed) {
                // the hypothesis whose listed candidates include place q: the last k with cp_off[k] <= q (bisection)
                int hi_k = K;
                while (hi_k - k > 1) { const int mid = (k + hi_k) >> 1; if (cp_off[mid] <= q) k = mid; else hi_k = mid; }
                e8[j] = ent[h_beg[k] + (q - cp_off[k])];
              }
              k8[j] = k;
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int q = q0 + j * cnt;
              if (q >= n_listed) continue;
              const int k = k8[j], i = q - cp_off[k];
              const TbRsEnt e = e8[j];
              const int tk = static_cast<int>((e.dst_tok & ((1u << TB_RS_TOK_BITS) - 1u)) >> 1);   // padding entries carry token V
              if (i < kBeamList) { hl_tok[k][i] = static_cast<uint16_t>(tk); hl_dst[k][i] = static_cast<int32_t>(e.dst_tok >> TB_RS_TOK_BITS); }
              unsigned long long key = 0ull;
              if (tk < V) {
                const float x = pref ? xrow[tk] : LogitLoad<LT>::at(base + tk);
                key = make_key(__fadd_rn(h_score[k], __fadd_rn(x, e.lb)), tk, k);
                atomicOr(&ovr[k * WW + (tk >> 5)], 1u << (tk & 31));
              }
              ckey[q] = key; cdst[q] = static_cast<int32_t>(e.dst_tok >> TB_RS_TOK_BITS);
            }
          }
        }
        __syncthreads();
        // blank, the first unlisted tokens of the reduced row, and the frozen hypotheses' carried candidates
        for (int pr = cth; pr < K * (M + 1); pr += cnt) {
          const int k = pr / (M + 1), j = pr - k * (M + 1);
          unsigned long long key = 0ull;
          int32_t dst = -1;
          if (h_score[k] != -INFINITY) {
            const TbTopEnt t = ttop[j];
            if (!h_live[k]) {
              if (j == M) { key = make_key(h_score[k], V + 1, k); dst = h_state[k]; }
            } else if (j == M) {
              key = make_key(__fadd_rn(h_score[k], t.x), V, k); dst = h_state[k];
            } else {
              const int tk = static_cast<int>(t.tok_cls & 0xFFFFu), cl = static_cast<int>(t.tok_cls >> 16);
              if (tk < V && !((ovr[k * WW + (tk >> 5)] >> (tk & 31)) & 1u)) {     // (tk >= V: the row has fewer tokens)
                const float val = bound ? __fadd_rn(t.x, __fmul_rn(g.lambda, __fadd_rn(h_D[k], tv.rootcw[cl]))) : t.x;
                key = make_key(__fadd_rn(h_score[k], val), tk, k);
                dst = bound ? tv.rootdst[cl] : -1;
              }
            }
          }
          ckey[n_listed + pr] = key; cdst[n_listed + pr] = dst;
        }
        __syncthreads();
        {
          // Selection (warp_top_keys).  A thread takes its candidates (indices thread, thread + block size, ...) into
          // registers once and keeps them sorted; a round is then two warp-wide integer maxima over the lanes' best.
          // Few candidates (narrow beams): warp 0 alone.  Many: every warp picks the K best of its candidates and
          // leaves them, best first, in shared memory; warp 0 then merges the warps' lists, one lane per list, the
          // head of each in a register.
          unsigned long long* wkey = reinterpret_cast<unsigned long long*>(cdst + cap);            // [warps][K] (key); behind the targets
          int32_t* widx = reinterpret_cast<int32_t*>(wkey + (kBeamThreads / 32) * TB_MAX_BEAM);   // [warps][K] where in ckey
          constexpr int kSelRegs = 8;
          constexpr int kRadixMinK = 9;       // beams at least this wide (wider than the teams of warps take) find their picks by radix selection
          const bool solo = n <= 32 * kSelRegs;
          auto put_sel = [&](int r, unsigned long long best, int idx) {
            const uint32_t mh = static_cast<uint32_t>(best >> 32);
            const uint32_t l2 = 0xFFFFFFFFu - static_cast<uint32_t>(best & 0xFFFFFFFFull);
            BeamKey c;
            c.v = __uint_as_float(mh ^ ((mh >> 31) ? 0x80000000u : 0xFFFFFFFFu));
            c.tkey = static_cast<int32_t>(l2 >> 5); c.par = static_cast<int32_t>(l2 & 31u);
            if (best == 0ull) c = BeamKey{-INFINITY, INT32_MAX, INT32_MAX};
            sel[r] = c; sel_dst[r] = best == 0ull ? -1 : cdst[idx];
          };
          if (solo) {
            if (warp == 0) {
              if (n <= 32 * 4) warp_top_keys<4>(ckey, n, lane, 32, K, lane, wkey, widx);
              else warp_top_keys<8>(ckey, n, lane, 32, K, lane, wkey, widx);
              __syncwarp();
              if (lane < K) put_sel(lane, wkey[lane], widx[lane]);
            }
          } else if (K >= kRadixMinK) {
            // Wide beams: K rounds at two levels cost more than finding the K-th largest key first.  The keys are 64-bit
            // numbers, all different; the K-th largest is found digit by digit (8 bits at a time, from the highest
            // digit in which the candidates differ) with a histogram in shared memory, the keys at or above it are
            // collected, and one warp orders them by counting, for each, the keys above it.
            int* hist = reinterpret_cast<int*>(wkey);                     // [256]
            int* ctl = hist + 256;                                        // digit, its count, rank left, collected
            unsigned long long* okey = reinterpret_cast<unsigned long long*>(ctl + 8);   // [K] the collected keys
            int32_t* oidx = reinterpret_cast<int32_t*>(okey + TB_MAX_BEAM);              // [K] where they sit in ckey
            uint32_t hmax = 0u, hmin = 0xFFFFFFFFu;
            for (int ii = threadIdx.x; ii < n; ii += kBeamThreads) {
              const unsigned long long kk = ckey[ii];
              if (kk != 0ull) { const uint32_t h = static_cast<uint32_t>(kk >> 32); hmax = max(hmax, h); hmin = min(hmin, h); }
            }
            hmax = __reduce_max_sync(0xffffffffu, hmax);
            hmin = __reduce_min_sync(0xffffffffu, hmin);
            if (lane == 0) { red64[0][warp] = hmax; red64[1][warp] = hmin; }
            if (threadIdx.x == 0) ctl[3] = 0;
            __syncthreads();
#pragma unroll
            for (int w2 = 0; w2 < kBeamThreads / 32; ++w2) {
              hmax = max(hmax, static_cast<uint32_t>(red64[0][w2])); hmin = min(hmin, static_cast<uint32_t>(red64[1][w2]));
            }
            unsigned long long t_low = 1ull;                               // keys at or above this are the picks
            if (hmax != 0u) {
              const uint32_t diff = hmax ^ hmin;
              int shift = diff == 0u ? 24 : 32 + ((31 - __clz(diff)) >> 3) * 8;
              unsigned long long prefix = shift + 8 >= 64 ? 0ull : ((static_cast<unsigned long long>(hmax) << 32) >> (shift + 8));
              int want = K;
              for (;;) {
                if (threadIdx.x < 256) hist[threadIdx.x] = 0;
                __syncthreads();
                for (int ii = threadIdx.x; ii < n; ii += kBeamThreads) {
                  const unsigned long long kk = ckey[ii];
                  if (kk != 0ull && (shift + 8 >= 64 || (kk >> (shift + 8)) == prefix)) atomicAdd(&hist[static_cast<int>((kk >> shift) & 255ull)], 1);
                }
                __syncthreads();
                if (warp == 0) {
                  // lane l looks at digits 255 - 8 l ... 248 - 8 l; the digit of the K-th key is the first at which
                  // the count of keys with that digit or a higher one reaches the rank wanted
                  int c[8], mine_total = 0;
#pragma unroll
                  for (int d = 0; d < 8; ++d) { c[d] = hist[255 - (8 * lane + d)]; mine_total += c[d]; }
                  int incl = mine_total;
#pragma unroll
                  for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += v; }
                  const int total = __shfl_sync(0xffffffffu, incl, 31);
                  const unsigned reach = __ballot_sync(0xffffffffu, incl >= want);
                  if (total < want) {
                    if (lane == 0) ctl[0] = -1;                           // fewer candidates than places: all of them
                  } else if (lane == __ffs(reach) - 1) {
                    int above = incl - mine_total, d = 0;
                    while (above + c[d] < want) { above += c[d]; ++d; }
                    ctl[0] = 255 - (8 * lane + d); ctl[1] = c[d]; ctl[2] = want - above;
                  }
                }
                __syncthreads();
                const int digit = ctl[0];
                if (digit < 0) break;
                const int cD = ctl[1];
                want = ctl[2];
                prefix = (prefix << 8) | static_cast<unsigned long long>(digit);
                if (want == cD || shift == 0) { t_low = prefix << shift; break; }
                shift -= 8;
              }
              for (int ii = threadIdx.x; ii < n; ii += kBeamThreads) {
                const unsigned long long kk = ckey[ii];
                if (kk != 0ull && kk >= t_low) {
                  const int pos = atomicAdd(&ctl[3], 1);
                  if (pos < TB_MAX_BEAM) { okey[pos] = kk; oidx[pos] = ii; }
                }
              }
            }
            __syncthreads();
            if (warp == 0) {
              const int cnt = min(ctl[3], K);
              if (lane < cnt) {
                const unsigned long long mine = okey[lane];
                int rank = 0;
                for (int j2 = 0; j2 < cnt; ++j2) rank += okey[j2] > mine ? 1 : 0;
                put_sel(rank, mine, oidx[lane]);
              } else if (lane < K) {
                put_sel(lane, 0ull, -1);
              }
            }
          } else {
            if (n <= kBeamThreads * 2) {
              warp_top_keys<2>(ckey, n, static_cast<int>(threadIdx.x), kBeamThreads, K, lane, wkey + warp * TB_MAX_BEAM, widx + warp * TB_MAX_BEAM);
            } else if (n <= kBeamThreads * 4) {
              warp_top_keys<4>(ckey, n, static_cast<int>(threadIdx.x), kBeamThreads, K, lane, wkey + warp * TB_MAX_BEAM, widx + warp * TB_MAX_BEAM);
            } else if (n <= kBeamThreads * 8) {
              warp_top_keys<8>(ckey, n, static_cast<int>(threadIdx.x), kBeamThreads, K, lane, wkey + warp * TB_MAX_BEAM, widx + warp * TB_MAX_BEAM);
            } else {
              // (more candidates than the registers take: rounds over the array in shared memory)
              unsigned long long lim = ~0ull;
              for (int r = 0; r < K; ++r) {
                unsigned long long a = 0ull;
                int ai = -1;
                for (int ii = threadIdx.x; ii < n; ii += kBeamThreads) { const unsigned long long kk = ckey[ii]; if (kk < lim && kk > a) { a = kk; ai = ii; } }
                const uint32_t hi = static_cast<uint32_t>(a >> 32), lo = static_cast<uint32_t>(a);
                const uint32_t mh = __reduce_max_sync(0xffffffffu, hi);
                const uint32_t ml = __reduce_max_sync(0xffffffffu, hi == mh ? lo : 0u);
                const unsigned long long best = (static_cast<unsigned long long>(mh) << 32) | ml;
                if (best != 0ull && a == best) { wkey[warp * TB_MAX_BEAM + r] = best; widx[warp * TB_MAX_BEAM + r] = ai; }
                if (best == 0ull && lane == 0) { wkey[warp * TB_MAX_BEAM + r] = 0ull; widx[warp * TB_MAX_BEAM + r] = -1; }
                lim = best;                                       // (0 once nothing is left: the later rounds find nothing either)
              }
            }
            __syncthreads();
            if (warp == 0) {
              // lane w walks warp w's list from its head, which it keeps in a register; a round takes the largest head
              int ptr = 0;
              unsigned long long hk = lane < kBeamThreads / 32 ? wkey[lane * TB_MAX_BEAM] : 0ull;
              for (int r = 0; r < K; ++r) {
                const uint32_t hi = static_cast<uint32_t>(hk >> 32), lo = static_cast<uint32_t>(hk);
                const uint32_t mh = __reduce_max_sync(0xffffffffu, hi);
                const uint32_t ml = __reduce_max_sync(0xffffffffu, hi == mh ? lo : 0u);
                const unsigned long long best = (static_cast<unsigned long long>(mh) << 32) | ml;
                if (best == 0ull) {
                  if (lane == 0) put_sel(r, 0ull, -1);
                } else if (hk == best) {
                  put_sel(r, best, widx[lane * TB_MAX_BEAM + ptr]);
                  ++ptr;
                  hk = ptr < K ? wkey[lane * TB_MAX_BEAM + ptr] : 0ull;
                }
              }
            }
          }
          if (warp == 0) {
            // does the K-th pick clear everything that was not looked at?  Lane k answers for hypothesis k.
            __syncwarp();
            const float y_next = ttop[M].y;
            bool okk = true;
            if (y_next != -INFINITY && lane < K && h_score[lane] != -INFINITY && h_live[lane]) {
              const int k = lane;
              const float c_k = sel[K - 1].par != INT32_MAX ? sel[K - 1].v : -INFINITY;
              const float lamD = bound ? g.lambda * h_D[k] : 0.0f;
              const float scale = fabsf(h_score[k]) + fabsf(y_next) + 2.0f * (bound ? fabsf(g.lambda) * (fabsf(h_D[k]) + root_wmax) : 0.0f);
              const float ub = (h_score[k] + y_next) + lamD + scale * 3.814697265625e-6f + 1e-30f;      // 2^-18 of the scale
              okk = c_k > ub;
            }
            const bool all_ok = __all_sync(0xffffffffu, okk);
            if (lane == 0) cp_flag = all_ok ? 1 : 0;
          }
        }
      }
    }
    __syncthreads();
    compact_done = cp_flag != 0;
  }
  if (threadIdx.x == 0) rec_ready = 0;      // (set again below, once the new hypotheses' records have been fetched)

  // all candidate values of the live hypotheses
  if (compact_done) {
    // (nothing to lay out)
  } else if (use_tv) {
    // every hypothesis at once: its state's record, then all plain values, then the listed tokens on top
    if (threadIdx.x < K) {
      const int k = threadIdx.x;
      int32_t st = h_state[k];
      if (st < 0 || st >= rec.n_states) { if (h_score[k] != -INFINITY && h_live[k]) atomicOr(p.status, TB_STATUS_BAD_STATE); st = 0; }
      const TbRsRec r = reinterpret_cast<const TbRsRec*>(blob + rec.off_rsrec)[st];
      h_beg[k] = r.begin; h_cnt[k] = r.count; h_D[k] = r.D;
      hl_n[k] = r.count <= kBeamList ? r.count : -1;
    }
    for (int i = threadIdx.x; i < K * WW; i += kBeamThreads) ovr[i] = 0u;
    __syncthreads();
    const LT* base = reinterpret_cast<const LT*>(p.logits) + static_cast<int64_t>(b) * p.stream_stride;
    // the boosted tokens of every hypothesis first: their values go to cand and are marked, so that the sweep over
    // all candidates below leaves them alone -- and sees every candidate's final value, which lets each thread
    // collect its best keys on the way instead of scanning cand again afterwards
    {
      const TbRsEnt* ent = reinterpret_cast<const TbRsEnt*>(blob + rec.off_rsent);
      for (int k = 0; k < K; ++k) {
        if (h_score[k] == -INFINITY || !h_live[k]) continue;
        for (int i = threadIdx.x; i < h_cnt[k]; i += kBeamThreads) {
          const TbRsEnt e = ent[h_beg[k] + i];
          const int tk = static_cast<int>((e.dst_tok & ((1u << TB_RS_TOK_BITS) - 1u)) >> 1);   // padding entries carry token V
          if (i < kBeamList) { hl_tok[k][i] = static_cast<uint16_t>(tk); hl_dst[k][i] = static_cast<int32_t>(e.dst_tok >> TB_RS_TOK_BITS); }
          if (tk < V) {
            const float x = LogitLoad<LT>::at(base + static_cast<int64_t>(k) * p.hyp_stride + tk);
            cand[static_cast<size_t>(k) * W + tk] = __fadd_rn(h_score[k], __fadd_rn(x, e.lb));
            atomicOr(&ovr[k * WW + (tk >> 5)], 1u << (tk & 31));
          }
        }
      }
    }
    __syncthreads();
    if (pref) {
      // the row sits in registers: every index below is a compile-time constant
#pragma unroll
      for (int j = 0; j < kPref; ++j) {
        const int v = threadIdx.x + j * kBeamThreads;
        if (v < W) {
          const float plain_w = v < V ? tv.rootcw[__ldg(p.cls + v)] : 0.0f;
          const float x = row_staged ? xrow_s[v] : LogitLoad<LT>::widen(xpre[j]);
          for (int k = 0; k < K; ++k) {
            if (h_score[k] == -INFINITY || !h_live[k]) continue;
            float c;
            if ((ovr[k * WW + (v >> 5)] >> (v & 31)) & 1u) {
              c = cand[static_cast<size_t>(k) * W + v];
            } else {
              const float val = v < V ? __fadd_rn(x, __fmul_rn(g.lambda, __fadd_rn(h_D[k], plain_w))) : x;
              c = __fadd_rn(h_score[k], val);
              cand[static_cast<size_t>(k) * W + v] = c;
            }
            offer(make_key(c, v, k));
          }
        }
      }
    } else {
      for (int v = threadIdx.x; v < W; v += kBeamThreads) {
        const float plain_w = v < V ? tv.rootcw[__ldg(p.cls + v)] : 0.0f;
        for (int k = 0; k < K; ++k) {
          if (h_score[k] == -INFINITY || !h_live[k]) continue;
          float c;
          if ((ovr[k * WW + (v >> 5)] >> (v & 31)) & 1u) {
            c = cand[static_cast<size_t>(k) * W + v];
          } else {
            const float x = LogitLoad<LT>::at(base + static_cast<int64_t>(k) * p.hyp_stride + v);
            const float val = v < V ? __fadd_rn(x, __fmul_rn(g.lambda, __fadd_rn(h_D[k], plain_w))) : x;
            c = __fadd_rn(h_score[k], val);
            cand[static_cast<size_t>(k) * W + v] = c;
          }
          offer(make_key(c, v, k));
        }
      }
    }
    // a frozen hypothesis is carried as one candidate (thread k offers it)
    if (threadIdx.x < K && h_score[threadIdx.x] != -INFINITY && !h_live[threadIdx.x]) offer(make_key(h_score[threadIdx.x], V + 1, threadIdx.x));
    swept = true;
    __syncthreads();
  } else {
    for (int k = 0; k < K; ++k) {
      if (h_score[k] == -INFINITY || !h_live[k]) continue;  // uniform across the block
      if (bound) build_bonus(g, h_state[k], p.C, bvec, nvec, chain.state, chain.acc, &chain.len, p.status);
      const LT* row = reinterpret_cast<const LT*>(p.logits) + static_cast<int64_t>(b) * p.stream_stride +
                      static_cast<int64_t>(k) * p.hyp_stride;
      const float sc = h_score[k];
      for (int v = threadIdx.x; v < W; v += kBeamThreads) {
        float x = LogitLoad<LT>::at(row + v);
        float val = (bound && v < V) ? __fadd_rn(x, __fmul_rn(g.lambda, bvec[__ldg(p.cls + v)])) : x;
        cand[static_cast<size_t>(k) * W + v] = __fadd_rn(sc, val);
      }
      __syncthreads();
    }
  }

  // K rounds of selection.  A candidate's place in the order (value descending, token key ascending,
  // parent ascending) is one 64-bit key: the order-preserving image of the value above the inverted
  // (token key, parent) pair; keys are distinct, 0 means "none".  Every thread keeps the best key among
  // its own candidates that has not been picked yet; after a round only the owner of the pick rescans.
  // best key below `limit` among this thread's candidates: tokens v = tid, tid + 256, ... of every live
  // hypothesis, plus (thread k) the carried candidate of a frozen hypothesis k
  // the row of the next step is requested now: its trip from HBM overlaps the selection rounds
  if (!compact_done && !row_staged) {
    xpre_valid = false;
    if (pref && next_row) {
#pragma unroll
      for (int j = 0; j < kPref; ++j) {
        const int v = threadIdx.x + j * kBeamThreads;
        if (v < W) xpre[j] = LogitLoad<LT>::raw(next_row + v);
      }
      xpre_valid = true;
    }
    tpre_valid = false;
    if (next_top) { if (threadIdx.x <= p.top_m) tpre = next_top[threadIdx.x]; tpre_valid = true; }
  }
  unsigned long long spare = 0ull;                            // this thread's second best key below the limit of its last scan
  bool have_spare = false;
  auto scan_mine = [&](unsigned long long limit) -> unsigned long long {
    unsigned long long m = 0ull, m2 = 0ull;
    for (int k = 0; k < K; ++k) {
      if (h_score[k] == -INFINITY) continue;
      if (!h_live[k]) {
        if (threadIdx.x == k) { const unsigned long long kk = make_key(h_score[k], V + 1, k); if (kk < limit) { if (kk > m) { m2 = m; m = kk; } else if (kk > m2) m2 = kk; } }
        continue;
      }
      const float* ck = cand + static_cast<size_t>(k) * W;
      for (int v = threadIdx.x; v < W; v += kBeamThreads) {
        const unsigned long long kk = make_key(ck[v], v, k);
        if (kk < limit) { if (kk > m) { m2 = m; m = kk; } else if (kk > m2) m2 = kk; }
      }
    }
    spare = m2; have_spare = true;
    return m;
  };
  unsigned long long mine = 0ull;
  if (compact_done) { /* picked already */ }
  else if (swept) { mine = m1; spare = m2; have_spare = true; }     // collected during the sweep
  else mine = scan_mine(~0ull);
  for (int r = 0; r < K && !compact_done; ++r) {
    // the warp's best key: the largest high word, then the largest low word among the lanes that have it
    const uint32_t hi = static_cast<uint32_t>(mine >> 32), lo = static_cast<uint32_t>(mine);
    const uint32_t mh = __reduce_max_sync(0xffffffffu, hi);
    const uint32_t ml = __reduce_max_sync(0xffffffffu, hi == mh ? lo : 0u);
    if (lane == 0) red64[r & 1][warp] = (static_cast<unsigned long long>(mh) << 32) | ml;
    __syncthreads();                     // (one barrier per round: the next round writes the other copy)
    unsigned long long best = red64[r & 1][0];
#pragma unroll
    for (int w2 = 1; w2 < kBeamThreads / 32; ++w2) { const unsigned long long o = red64[r & 1][w2]; if (o > best) best = o; }
    if (threadIdx.x == 0) {
      BeamKey c{-INFINITY, INT32_MAX, INT32_MAX};
      if (best != 0ull) {
        const uint32_t lo = 0xFFFFFFFFu - static_cast<uint32_t>(best & 0xFFFFFFFFull);
        c.tkey = static_cast<int32_t>(lo >> 5); c.par = static_cast<int32_t>(lo & 31u);
        c.v = c.tkey == V + 1 ? h_score[c.par] : cand[static_cast<size_t>(c.par) * W + c.tkey];
      }
      sel[r] = c;
    }
    if (best != 0ull && mine == best) {                          // this thread owned the pick: its next best
      if (have_spare) { mine = spare; have_spare = false; }
      else mine = scan_mine(best);
    }
  }
  __syncthreads();

  // new hypotheses, the hypothesis tree
  int32_t parent = -1, token = -1, state = -1;
  uint8_t lv = 0;
  float sc = -INFINITY;
  unsigned long long nh = 0ull;
  int32_t nl = 0;
  if (threadIdx.x < K) {
    const int r = threadIdx.x;
    const BeamKey c = sel[r];
    const int64_t o = static_cast<int64_t>(b) * K + r;
    if (c.par != INT32_MAX) {
      parent = c.par; sc = c.v;
      token = (c.tkey == V + 1) ? -1 : c.tkey;
      state = h_state[parent];
      if (token >= 0 && token != V) {
        if (compact_done) {
          state = sel_dst[r];
        } else if (use_tv && hl_n[parent] >= 0) {
          int nx = tv.rootdst[__ldg(p.cls + token)];          // a pick that the parent's list does not hold is a plain token
          for (int i = 0; i < hl_n[parent]; ++i)
            if (hl_tok[parent][i] == token) { nx = hl_dst[parent][i]; break; }
          state = nx;
        } else if (bound) {
          state = walk_next(g, state, __ldg(p.cls + token), p.status);
        }
        lv = h_live[parent];
      }
    }
    p.scores[o] = sc; p.states[o] = state; p.live[o] = lv;
    p.out_parent[o] = parent; p.out_token[o] = token;
    {
      if (parent >= 0) {
        nh = h_hash[parent]; nl = h_len[parent];
        if (token >= 0 && token != V) {          // one more token: a 64-bit mix of the sequence so far and the token
          nh = (nh ^ static_cast<unsigned long long>(token + 1)) * 0xff51afd7ed558ccdull;
          nh ^= nh >> 33;
          nh += 0x9e3779b97f4a7c15ull;
          ++nl;
        }
      }
      p.hash_out[o] = nh; p.len_out[o] = nl;
    }
    if (p.tree) {
      const int64_t at = p.tree_cap > 0 ? static_cast<int64_t>(b) * p.tree_cap + (p.step % p.tree_cap)
                                        : static_cast<int64_t>(p.step) * p.B + b;
      p.tree[at * K + r] = make_int2(parent, token);
    }
  }
  // the list record of every new hypothesis' state, for the next step's compact path: fetched now, so that its trip
  // to L2 is over when that step starts
  TbRsRec nrec{0, 0, 0.0f, 0.0f};
  int rec_ok = 1;
  if (threadIdx.x < K && p.top_row != nullptr && use_tv && sc != -INFINITY) {
    if (state >= 0 && state < rec.n_states) nrec = reinterpret_cast<const TbRsRec*>(blob + rec.off_rsrec)[state];
    else rec_ok = 0;                                        // (the next step reports it)
  }
  // ... and in shared memory, for the next step of a launch that runs several (read by every thread above: wait)
  const int all_ok = __syncthreads_and(rec_ok);
  if (threadIdx.x < K) {
    h_score[threadIdx.x] = sc; h_state[threadIdx.x] = state; h_live[threadIdx.x] = lv;
    h_hash[threadIdx.x] = nh; h_len[threadIdx.x] = nl;
    if (p.top_row != nullptr) { h_beg[threadIdx.x] = nrec.begin; h_cnt[threadIdx.x] = nrec.count; h_D[threadIdx.x] = nrec.D; }
  }
  if (threadIdx.x == 0) rec_ready = (p.top_row != nullptr && (use_tv || !bound) && all_ok) ? 1 : 0;
}

template <typename LT>
__global__ void __launch_bounds__(kBeamThreads) k_beam_step(TbBeamParams p) {
  LT xpre[kBeamPref] = {};
  bool xpre_valid = false;
  TbTopEnt tpre{0.0f, 0.0f, 0u};
  bool tpre_valid = false;
  __shared__ BeamShared sh;
  beam_step_body<LT>(p, sh, xpre, xpre_valid, static_cast<const LT*>(nullptr), tpre, tpre_valid, nullptr);
}


// ---- narrow beams: steps taken by a small team of warps ------------------------------------------------------------
// With K <= 8 and the rows reduced ahead of the steps, a step has a few dozen candidates, and the block-wide step body
// spends its time in block-wide barriers between short phases.  beam_fast_run lets K + 1 warps take such steps, one
// after the other, while the block's other warps wait: warp 0 coordinates (it holds the stream's hypotheses in
// registers, lane k: hypothesis k), warp k + 1 works for hypothesis k.  Per step
//   worker k     : the hypothesis' list record, its listed tokens (exact values; logits from the row, which arrives
//                  in shared memory by asynchronous copies the coordinator issues two steps ahead), blank, the first
//                  unlisted tokens of the reduced row or the carried hypothesis, every lane keeping the three best
//                  of those it sees in registers; the K best of them in K rounds of two warp-wide integer maxima;
//   barrier of the team (a named barrier, not the block's);
//   coordinator  : the K best of the workers' picks, the same bound check as the block-wide compact path, the new
//                  hypotheses, and, where the next step begins a frame, merging and pruning;
//   barrier of the team; then the workers go on while the coordinator writes the step's results to global memory
//                  and asks for the row after the next.
// A step the team cannot take (the bound not cleared, more than three picks due to one lane) is left untouched: the
// run ends before it, the hypotheses go back to shared memory, and the whole block does that step with
// beam_step_body.  Same arithmetic, same order of candidates, hence the same results bit for bit.
constexpr int kFastMaxK = 8;      // widest beam of the team's steps
constexpr int kFastMaxList = 2048; // longest list of boosted tokens a worker takes
constexpr int kFastRecCache = 48 << 10;   // shared memory for a copy of the stream's list records (graphs of up to 3072 states)

__device__ __forceinline__ unsigned long long beam_key(float v, int tkey, int k) {
  const uint32_t u = __float_as_uint(v + 0.0f);             // -0 folded into +0: equal values, equal keys
  const uint32_t hi = u ^ ((u >> 31) ? 0xFFFFFFFFu : 0x80000000u);
  const uint32_t lo = 0xFFFFFFFFu - (static_cast<uint32_t>(tkey) * 32u + static_cast<uint32_t>(k));
  return (static_cast<unsigned long long>(hi) << 32) | lo;
}
__device__ __forceinline__ float beam_key_value(unsigned long long key) {
  const uint32_t mh = static_cast<uint32_t>(key >> 32);
  return __uint_as_float(mh ^ ((mh >> 31) ? 0x80000000u : 0xFFFFFFFFu));
}
__device__ __forceinline__ unsigned long long shfl_u64(unsigned long long v, int src) {
  const uint32_t lo = __shfl_sync(0xffffffffu, static_cast<uint32_t>(v), src);
  const uint32_t hi = __shfl_sync(0xffffffffu, static_cast<uint32_t>(v >> 32), src);
  return (static_cast<unsigned long long>(hi) << 32) | lo;
}
__device__ __forceinline__ void beam_cp_async16(unsigned char* dst_smem, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(dst_smem))), "l"(src) : "memory");
}
__device__ __forceinline__ void beam_cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void beam_cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
template <typename LT> __device__ __forceinline__ float beam_smem_logit(const unsigned char* row, int idx);
template <> __device__ __forceinline__ float beam_smem_logit<uint16_t>(const unsigned char* row, int idx) {
  return __uint_as_float(static_cast<uint32_t>(*reinterpret_cast<const uint16_t*>(row + 2 * idx)) << 16);
}
template <> __device__ __forceinline__ float beam_smem_logit<float>(const unsigned char* row, int idx) {
  return *reinterpret_cast<const float*>(row + 4 * idx);
}
// Starts the copy of one row (its 16-byte aligned superset) into buf; a 16-byte piece that is not wholly inside the
// tensor [lo, hi) is assembled from the elements that are.
template <typename LT>
__device__ __forceinline__ void beam_fetch_row(unsigned char* buf, const LT* row, int W, const unsigned char* lo,
                                               const unsigned char* hi, int lane) {
  const unsigned char* rp = reinterpret_cast<const unsigned char*>(row);
  const int off = static_cast<int>(reinterpret_cast<uintptr_t>(rp) & 15);
  const unsigned char* a0 = rp - off;
  const int nchunks = (off + W * static_cast<int>(sizeof(LT)) + 15) >> 4;
  for (int c = lane; c < nchunks; c += 32) {
    const unsigned char* ac = a0 + 16 * c;
    if (ac >= lo && ac + 16 <= hi) {
      beam_cp_async16(buf + 16 * c, ac);
    } else {
      for (int e = 0; e < 16; e += static_cast<int>(sizeof(LT)))
        if (ac + e >= lo && ac + e + sizeof(LT) <= hi) *reinterpret_cast<LT*>(buf + 16 * c + e) = *reinterpret_cast<const LT*>(ac + e);
    }
  }
}
__host__ __device__ inline size_t beam_ring_bytes(int V, int elem) {   // two row buffers of the team steps
  const size_t one = ((static_cast<size_t>(V + 1) * elem + 16 + 15) & ~size_t(15)) + 16;
  return 2 * one + 16;
}

// Where the team keeps a copy of the stream's list records (16 bytes per graph state), behind the row buffers.
template <typename LT>
__device__ __forceinline__ TbRsRec* beam_rec_cache(const TbBeamParams& p, unsigned char* dyn) {
  const int W = p.V + 1, WW = (W + 31) >> 5;
  unsigned char* ovr = dyn + ((static_cast<size_t>(p.K) * W * sizeof(float) + 15) & ~size_t(15));
  unsigned char* aux = ovr + ((static_cast<size_t>(p.K) * WW * sizeof(uint32_t) + 15) & ~size_t(15));
  unsigned char* ring = aux + beam_aux_bytes(p.V, p.C, p.tokview) + static_cast<size_t>(W) * sizeof(float);
  ring += (16 - (reinterpret_cast<uintptr_t>(ring) & 15)) & 15;
  return reinterpret_cast<TbRsRec*>(ring + beam_ring_bytes(p.V, sizeof(LT)));
}
// Block-wide, once per launch: fills that copy if the stream's records fit.  Returns whether they do.
template <typename LT>
__device__ __forceinline__ bool beam_rec_cache_fill(const TbBeamParams& p, unsigned char* dyn) {
  const TbSlotRec& rec = p.slots[blockIdx.x];
  if (rec.n_states <= 0 || rec.n_rsent < 0 || static_cast<int64_t>(rec.n_states) * 16 > p.rec_cache_bytes) return false;
  const uint4* src = reinterpret_cast<const uint4*>(p.arena + rec.blob_off + rec.off_rsrec);
  uint4* dst = reinterpret_cast<uint4*>(beam_rec_cache<LT>(p, dyn));
  for (int i = threadIdx.x; i < rec.n_states; i += blockDim.x) dst[i] = src[i];
  return true;                                                  // (the barriers of the launch's first step come before any use)
}

__device__ __forceinline__ void beam_team_barrier(int n_threads) { asm volatile("bar.sync 1, %0;" ::"r"(n_threads) : "memory"); }

// Takes the steps sidx, sidx + 1, ... of the block's stream as long as it can; returns (on warp 0) how many it took.
// Called by warps 0 .. K; the hypotheses are read from and left in sh.h_*.  hashA / hashB, lenA / lenB: the two halves
// of the sequence records; step s writes half ((par0 + s) & 1 ? A : B).
template <typename LT>
__device__ __forceinline__ int beam_fast_run(const TbBeamParams& p, BeamShared& sh, unsigned char* dyn, int32_t sidx, const int32_t n_steps,
                                             const int32_t E, const int64_t frame_stride, const int64_t row_stride,
                                             const int32_t rows_per_stream, const int32_t step_base, unsigned long long* hashA,
                                             unsigned long long* hashB, int32_t* lenA, int32_t* lenB, const int32_t par0,
                                             const bool recs_cached) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int b = blockIdx.x, K = p.K, V = p.V, W = V + 1, M = p.top_m, WW = (W + 31) >> 5;
  const int team = 32 * (K + 1);
  const TbSlotRec rec = p.slots[b];
  const bool bound = rec.n_states > 0;
  const GraphPtrs g = graph_of(p.arena, rec);
  const unsigned char* blob = p.arena + rec.blob_off;
  uint32_t* ovr = reinterpret_cast<uint32_t*>(dyn + ((static_cast<size_t>(K) * W * sizeof(float) + 15) & ~size_t(15)));
  unsigned char* aux = reinterpret_cast<unsigned char*>(ovr) + ((static_cast<size_t>(K) * WW * sizeof(uint32_t) + 15) & ~size_t(15));
  unsigned char* ring = aux + beam_aux_bytes(V, p.C, p.tokview) + static_cast<size_t>(W) * sizeof(float);
  ring += (16 - (reinterpret_cast<uintptr_t>(ring) & 15)) & 15;
  const int row_buf = static_cast<int>((beam_ring_bytes(V, sizeof(LT)) - 16) / 2);
  const LT* stream_base = reinterpret_cast<const LT*>(p.logits) + static_cast<int64_t>(b) * p.stream_stride;
  auto row_of = [&](int s) -> const LT* {
    const int t = s / E, e = s - t * E;
    return stream_base + static_cast<int64_t>(t) * frame_stride + static_cast<int64_t>(e) * row_stride;
  };

  if (warp > 0) {
    // ================================ worker: hypothesis k ================================
    const int k = warp - 1;
    TokView tv;
    tokview_attach(tv, aux, V, p.C);
    const TbTopEnt* top0 = p.top_base + static_cast<int64_t>(b) * rows_per_stream * (M + 1);
    const TbRsRec* rsrec = recs_cached ? beam_rec_cache<LT>(p, dyn) : reinterpret_cast<const TbRsRec*>(blob + rec.off_rsrec);
    const TbRsEnt* ent = reinterpret_cast<const TbRsEnt*>(blob + rec.off_rsent);
    uint32_t* ovr_k = ovr + k * WW;
    TbTopEnt tnext{-INFINITY, -INFINITY, 0xFFFFu};
    if (lane <= M) tnext = top0[static_cast<int64_t>(sidx) * (M + 1) + lane];
    beam_team_barrier(team);                                   // the coordinator has set up the first step
    for (;; ++sidx) {
      if (sh.f_cmd != 0) break;
      const TbTopEnt tt = tnext;                               // (lane j: entry j of this step's reduced row, asked for a step ago)
      if (sidx + 1 < n_steps && lane <= M) tnext = top0[static_cast<int64_t>(sidx + 1) * (M + 1) + lane];
      const float sc1 = sh.f_sc[k];
      const int32_t st1 = sh.f_st[k];
      const bool lv1 = sh.f_lv[k] != 0;
      // a lane keeps the three best of the candidates it sees, best first (a step's K picks hardly ever include more
      // than three of one lane's; if they might, the step is left to the whole block)
      unsigned long long m0 = 0ull, m1 = 0ull, m2 = 0ull;
      int32_t e0 = -1, e1 = -1, e2 = -1;
      int n_seen = 0;
      auto offer = [&](unsigned long long kk, int32_t dd) {
        ++n_seen;
        if (kk > m0) { m2 = m1; e2 = e1; m1 = m0; e1 = e0; m0 = kk; e0 = dd; }
        else if (kk > m1) { m2 = m1; e2 = e1; m1 = kk; e1 = dd; }
        else if (kk > m2) { m2 = kk; e2 = dd; }
      };
      float D = 0.0f;
      if (sc1 != -INFINITY) {
        int32_t beg = 0, cnt = 0;
        if (bound) {
          int32_t sx = st1;
          if (sx < 0 || sx >= rec.n_states) { if (lane == 0) atomicOr(p.status, TB_STATUS_BAD_STATE); sx = 0; }
          const TbRsRec r = rsrec[sx];
          beg = r.begin; cnt = r.count; D = r.D;
        }
        const unsigned char* rowb = ring + (sidx & 1) * row_buf + (reinterpret_cast<uintptr_t>(row_of(sidx)) & 15);
        if (lv1) {
          if (cnt > kFastMaxList) { if (lane == 0) sh.f_fail = 1; cnt = 0; }
          for (int i = lane; i < WW; i += 32) ovr_k[i] = 0u;
          __syncwarp();
          // the listed tokens: exact values
          for (int i0 = 0; i0 < cnt; i0 += 32) {
            const int i = i0 + lane;
            if (i < cnt) {
              const TbRsEnt en = ent[beg + i];
              const int tk = static_cast<int>((en.dst_tok & ((1u << TB_RS_TOK_BITS) - 1u)) >> 1);   // padding entries carry token V
              if (tk < V) {
                const float x = beam_smem_logit<LT>(rowb, tk);
                offer(beam_key(__fadd_rn(sc1, __fadd_rn(x, en.lb)), tk, k), static_cast<int32_t>(en.dst_tok >> TB_RS_TOK_BITS));
                atomicOr(&ovr_k[tk >> 5], 1u << (tk & 31));
              }
            }
          }
          __syncwarp();
          // blank and the first unlisted tokens of the reduced row: lane j looks at its entry j
          if (lane == M) {
            offer(beam_key(__fadd_rn(sc1, tt.x), V, k), st1);
          } else if (lane < M) {
            const int tk = static_cast<int>(tt.tok_cls & 0xFFFFu), cl = static_cast<int>(tt.tok_cls >> 16);
            if (tk < V && !((ovr_k[tk >> 5] >> (tk & 31)) & 1u)) {     // (tk >= V: the row has fewer tokens)
              const float val = bound ? __fadd_rn(tt.x, __fmul_rn(g.lambda, __fadd_rn(D, tv.rootcw[cl]))) : tt.x;
              offer(beam_key(__fadd_rn(sc1, val), tk, k), bound ? tv.rootdst[cl] : -1);
            }
          }
        } else if (lane == M) {
          offer(beam_key(sc1, V + 1, k), st1);                             // a frozen hypothesis is carried
        }
      }
      // the K best of this hypothesis' candidates: lane r ends up with pick r
      unsigned long long mykey = 0ull;
      int32_t mydst = -1;
      int taken = 0;
      for (int r = 0; r < K; ++r) {
        const uint32_t hi = static_cast<uint32_t>(m0 >> 32), lo = static_cast<uint32_t>(m0);
        const uint32_t mh = __reduce_max_sync(0xffffffffu, hi);
        const uint32_t ml = __reduce_max_sync(0xffffffffu, hi == mh ? lo : 0u);
        const unsigned long long best = (static_cast<unsigned long long>(mh) << 32) | ml;
        if (best == 0ull) break;                                  // (uniform: nothing left; the later picks stay empty)
        const bool mine = m0 == best;
        const unsigned who = __ballot_sync(0xffffffffu, mine);
        const int32_t dsel = __shfl_sync(0xffffffffu, e0, __ffs(who) - 1);
        if (lane == r) { mykey = best; mydst = dsel; }
        if (mine) { m0 = m1; e0 = e1; m1 = m2; e1 = e2; m2 = 0ull; e2 = -1; ++taken; }
      }
      // a lane whose three kept candidates were all picked while it had seen more: a fourth might have been due
      if (__any_sync(0xffffffffu, taken == 3 && n_seen > 3) && lane == 0) sh.f_fail = 1;
      if (lane < K) { sh.f_key[k][lane] = mykey; sh.f_dst[k][lane] = mydst; }
      {
        // what the K-th pick of the step has to clear on behalf of this hypothesis (-inf: nothing)
        const float y_next = __shfl_sync(0xffffffffu, tt.y, M);
        if (lane == 0) {
          float ub = -INFINITY;
          if (y_next != -INFINITY && sc1 != -INFINITY && lv1) {
            const float lamD = bound ? g.lambda * D : 0.0f;
            const float scale = fabsf(sc1) + fabsf(y_next) + 2.0f * (bound ? fabsf(g.lambda) * (fabsf(D) + sh.root_wmax) : 0.0f);
            ub = (sc1 + y_next) + lamD + scale * 3.814697265625e-6f + 1e-30f;      // 2^-18 of the scale
          }
          sh.f_ub[k] = ub;
        }
      }
      beam_team_barrier(team);                                 // picks are in place
      beam_team_barrier(team);                                 // the coordinator has set up the next step (or ended the run)
    }
    return 0;
  }

  // ================================ coordinator ================================
  float sc = -INFINITY;
  int32_t st = -1, hl = 0;
  bool lv = false;
  unsigned long long hh = 0ull;
  if (lane < K) { sc = sh.h_score[lane]; st = sh.h_state[lane]; lv = sh.h_live[lane] != 0; hh = sh.h_hash[lane]; hl = sh.h_len[lane]; }
  // the working copy of the hypotheses for step s: after the frame start's liveness, merging and pruning
  float sc1 = sc;
  int32_t st1 = st;
  bool lv1 = lv;
  auto frame_start = [&](int s) {
    sc1 = sc; st1 = st; lv1 = lv;
    if (s % E != 0) return;
    lv1 = sc1 != -INFINITY;
    if (p.merge) {
      bool dup = false;
      for (int j = 0; j + 1 < K; ++j) {
        const float sj = __shfl_sync(0xffffffffu, sc, j);
        const int32_t lj = __shfl_sync(0xffffffffu, hl, j), stj = __shfl_sync(0xffffffffu, st, j);
        const unsigned long long hj = shfl_u64(hh, j);
        if (lane > j && lane < K && sc != -INFINITY && sj != -INFINITY && lj == hl && hj == hh && stj == st) dup = true;
      }
      if (dup) { sc1 = -INFINITY; st1 = -1; lv1 = false; }
    }
    if (p.prune_delta >= 0.0f) {
      float best = sc1;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, o));
      if (lane < K && sc1 != -INFINITY && sc1 < __fsub_rn(best, p.prune_delta)) { sc1 = -INFINITY; st1 = -1; lv1 = false; }
    }
  };
  auto publish = [&]() { if (lane < K) { sh.f_sc[lane] = sc1; sh.f_st[lane] = st1; sh.f_lv[lane] = lv1 ? 1 : 0; } };
  frame_start(sidx);
  publish();
  if (lane == 0) { sh.f_cmd = 0; sh.f_fail = 0; }
  beam_fetch_row<LT>(ring + (sidx & 1) * row_buf, row_of(sidx), W, p.tensor_lo, p.tensor_hi, lane);
  if (sidx + 1 < n_steps) beam_fetch_row<LT>(ring + ((sidx + 1) & 1) * row_buf, row_of(sidx + 1), W, p.tensor_lo, p.tensor_hi, lane);
  beam_cp_async_commit();
  beam_cp_async_wait<0>();
  __syncwarp();
  beam_team_barrier(team);
  int done = 0;
  for (;; ++sidx) {
    beam_team_barrier(team);                                   // the workers' picks are in place
    // ---- the K best of K * K picks: lane i looks at picks i and i + 32
    unsigned long long c0 = 0ull, c1 = 0ull;
    int32_t d0 = -1, d1 = -1;
    if (lane < K * K) { c0 = sh.f_key[lane / K][lane % K]; d0 = sh.f_dst[lane / K][lane % K]; }
    if (lane + 32 < K * K) { c1 = sh.f_key[(lane + 32) / K][(lane + 32) % K]; d1 = sh.f_dst[(lane + 32) / K][(lane + 32) % K]; }
    unsigned long long mykey = 0ull;
    int32_t mydst = -1;
    for (int r = 0; r < K; ++r) {
      const bool second = c1 > c0;
      const unsigned long long a = second ? c1 : c0;
      const uint32_t hi = static_cast<uint32_t>(a >> 32), lo = static_cast<uint32_t>(a);
      const uint32_t mh = __reduce_max_sync(0xffffffffu, hi);
      const uint32_t ml = __reduce_max_sync(0xffffffffu, hi == mh ? lo : 0u);
      const unsigned long long best = (static_cast<unsigned long long>(mh) << 32) | ml;
      if (best == 0ull) break;
      const bool mine = a == best;
      const unsigned who = __ballot_sync(0xffffffffu, mine);
      const int32_t dsel = __shfl_sync(0xffffffffu, second ? d1 : d0, __ffs(who) - 1);
      if (lane == r) { mykey = best; mydst = dsel; }
      if (mine) { if (second) c1 = 0ull; else c0 = 0ull; }
    }
    // ---- does the K-th pick clear everything that was not looked at?
    bool ok = sh.f_fail == 0;
    {
      const unsigned long long key_last = shfl_u64(mykey, K - 1);
      const float c_k = key_last != 0ull ? beam_key_value(key_last) : -INFINITY;
      bool okk = true;
      if (lane < K) { const float ub = sh.f_ub[lane]; okk = ub == -INFINITY || c_k > ub; }
      ok = ok && __all_sync(0xffffffffu, okk);
    }
    if (!ok) {
      if (lane == 0) sh.f_cmd = 1;
      __syncwarp();
      beam_team_barrier(team);
      break;
    }
    // ---- the new hypotheses
    int32_t parent = -1, token = -1, nstate = -1, nl = 0;
    bool nlv = false;
    float nsc = -INFINITY;
    unsigned long long nh = 0ull;
    {
      const uint32_t l2 = 0xFFFFFFFFu - static_cast<uint32_t>(mykey & 0xFFFFFFFFull);
      const int par_l = mykey != 0ull ? static_cast<int>(l2 & 31u) : 0;
      const int32_t pst = __shfl_sync(0xffffffffu, st1, par_l), pl = __shfl_sync(0xffffffffu, hl, par_l);
      const int plv = __shfl_sync(0xffffffffu, lv1 ? 1 : 0, par_l);
      const unsigned long long ph = shfl_u64(hh, par_l);
      if (lane < K && mykey != 0ull) {
        const int tkey = static_cast<int>(l2 >> 5);
        parent = par_l; nsc = beam_key_value(mykey);
        token = tkey == V + 1 ? -1 : tkey;
        nstate = pst;
        nh = ph; nl = pl;
        if (token >= 0 && token != V) {
          nstate = mydst; nlv = plv != 0;
          nh = (nh ^ static_cast<unsigned long long>(token + 1)) * 0xff51afd7ed558ccdull;
          nh ^= nh >> 33;
          nh += 0x9e3779b97f4a7c15ull;
          ++nl;
        }
      }
    }
    sc = nsc; st = nstate; lv = nlv; hh = nh; hl = nl;
    ++done;
    const bool last = sidx + 1 >= n_steps;
    if (!last) { frame_start(sidx + 1); publish(); }
    if (lane == 0 && last) sh.f_cmd = 1;
    beam_cp_async_wait<0>();                                   // the next step's row (asked for a step ago) is there
    __syncwarp();
    beam_team_barrier(team);                                   // the workers go on
    // ---- off the critical path: this step's results, the row after the next
    if (lane < K) {
      const int64_t o = static_cast<int64_t>(b) * K + lane;
      p.scores[o] = nsc; p.states[o] = nstate; p.live[o] = nlv ? 1 : 0;
      p.out_parent[o] = parent; p.out_token[o] = token;
      const bool odd = ((par0 + sidx) & 1) != 0;
      (odd ? hashA : hashB)[o] = nh; (odd ? lenA : lenB)[o] = nl;
      if (p.tree) {
        const int32_t step = step_base + sidx;
        const int64_t at = p.tree_cap > 0 ? static_cast<int64_t>(b) * p.tree_cap + (step % p.tree_cap)
                                          : static_cast<int64_t>(step) * p.B + b;
        p.tree[at * K + lane] = make_int2(parent, token);
      }
    }
    if (last) break;
    if (sidx + 2 < n_steps) beam_fetch_row<LT>(ring + (sidx & 1) * row_buf, row_of(sidx + 2), W, p.tensor_lo, p.tensor_hi, lane);
    beam_cp_async_commit();
  }
  beam_cp_async_wait<0>();
  if (lane < K) { sh.h_score[lane] = sc; sh.h_state[lane] = st; sh.h_live[lane] = lv ? 1 : 0; sh.h_hash[lane] = hh; sh.h_len[lane] = hl; }
  if (lane == 0) sh.rec_ready = 0;
  __syncwarp();
  return done;
}

// Whether the team's steps apply to this launch and this block's stream.
template <typename LT>
__device__ __forceinline__ bool beam_fast_applies(const TbBeamParams& p) {
  if (p.K > kFastMaxK || p.top_base == nullptr || p.tensor_lo == nullptr || p.top_m + 1 > 32) return false;
  const TbSlotRec& rec = p.slots[blockIdx.x];
  return rec.n_states <= 0 || (rec.n_rsent >= 0 && p.tokview);
}

// T frames of E rows in one launch: the block loops over the expansions of its stream; every hypothesis of the
// stream reads row (t, e).  What a step leaves in global memory (scores, states, liveness, sequence records) is read
// back in the next step by the thread that wrote it.
template <typename LT>
__global__ void __launch_bounds__(kBeamThreads) k_beam_frames(TbBeamParams p, int32_t T, int32_t E, int64_t frame_stride,
                                                          int64_t row_stride) {
  __shared__ BeamShared sh;
  LT xpre[kBeamPref] = {};
  bool xpre_valid = false;
  TbTopEnt tpre{0.0f, 0.0f, 0u};
  bool tpre_valid = false;
  const LT* stream_base = reinterpret_cast<const LT*>(p.logits) + static_cast<int64_t>(blockIdx.x) * p.stream_stride;
  extern __shared__ __align__(16) unsigned char dyn_all[];
  const bool fast = beam_fast_applies<LT>(p);
  const bool recs_cached = fast && beam_rec_cache_fill<LT>(p, dyn_all);
  int32_t skip = 0, backoff = 0;              // steps until the team tries again after a step it could not take
  for (int32_t sidx = 0; sidx < T * E; ++sidx) {
    if (fast && sidx > 0 && skip-- <= 0) {
      if (threadIdx.x < 32 * (p.K + 1)) {
        const int d = beam_fast_run<LT>(p, sh, dyn_all, sidx, T * E, E, frame_stride, row_stride, T * E, p.step,
                                        const_cast<unsigned long long*>(p.hash_in), p.hash_out, const_cast<int32_t*>(p.len_in), p.len_out, 0,
                                        recs_cached);
        if (threadIdx.x == 0) sh.fast_done = d;
      }
      __syncthreads();
      const int d = sh.fast_done;
      __syncthreads();                          // (read by everyone before a later run writes it again)
      sidx += d;
      backoff = d == 0 ? min(2 * backoff + 1, 32) : 0;
      skip = backoff;
      xpre_valid = false; tpre_valid = false;
      if (sidx >= T * E) break;
    }
    {
      const int32_t t = sidx / E, e = sidx - t * E;
      TbBeamParams q = p;
      q.logits = reinterpret_cast<const LT*>(p.logits) + static_cast<int64_t>(t) * frame_stride + static_cast<int64_t>(e) * row_stride;
      q.hyp_stride = 0;
      q.new_frame = e == 0 ? 1 : 0;
      q.merge = e == 0 ? p.merge : 0;
      q.prune_delta = e == 0 ? p.prune_delta : -1.0f;
      q.fresh = (p.fresh && sidx == 0) ? 1 : 0;
      q.tv_ready = sidx > 0 ? 1 : 0;
      q.step = p.step + sidx;
      q.top_row = p.top_base ? p.top_base + (static_cast<int64_t>(blockIdx.x) * T * E + sidx) * (p.top_m + 1) : nullptr;
      if (sidx & 1) { q.hash_in = p.hash_out; q.hash_out = const_cast<unsigned long long*>(p.hash_in); q.len_in = p.len_out; q.len_out = const_cast<int32_t*>(p.len_in); }
      const int32_t nt = e + 1 < E ? t : t + 1, ne = e + 1 < E ? e + 1 : 0;
      const LT* next_row = nt < T ? stream_base + static_cast<int64_t>(nt) * frame_stride + static_cast<int64_t>(ne) * row_stride : nullptr;
      const TbTopEnt* next_top = (nt < T && q.top_row) ? q.top_row + (p.top_m + 1) : nullptr;
      beam_step_body<LT>(q, sh, xpre, xpre_valid, next_row, tpre, tpre_valid, next_top);
      __syncthreads();
    }
  }
}

// Beam pre-pass: one warp per logit row, independent of every hypothesis.  With the rows of a stream shared by its
// hypotheses, the order of a row's tokens that no hypothesis' state boosts is, up to rounding, the order of their
// root-boosted values y -- so a step only needs the first few of them (see the compact path of beam_step_body).
constexpr int kTopWarps = 8;
template <typename LT>
__global__ void __launch_bounds__(kTopWarps * 32) k_beam_topm(const LT* logits, int32_t B, int32_t T, int32_t E, int32_t V, int32_t C,
                                                            int64_t stream_stride, int64_t frame_stride, int64_t row_stride,
                                                            const int32_t* n_frames, const TbSlotRec* slots, const unsigned char* arena,
                                                            const int32_t* cls, int32_t top_m, TbTopEnt* out) {
  extern __shared__ __align__(16) unsigned char dyn[];
  float* rootcw = reinterpret_cast<float*>(dyn);                                  // [C] root arc weight per class
  float* ybuf = reinterpret_cast<float*>(dyn) + C;                                // [kTopWarps][V]
  const int rows_per_stream = T * E, blocks_per_stream = (rows_per_stream + kTopWarps - 1) / kTopWarps;
  const int b = blockIdx.x / blocks_per_stream, r0 = (blockIdx.x - b * blocks_per_stream) * kTopWarps;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const TbSlotRec rec = slots[b];
  const bool bound = rec.n_states > 0;
  const GraphPtrs g = graph_of(arena, rec);
  for (int c = threadIdx.x; c < C; c += blockDim.x) rootcw[c] = 0.0f;
  __syncthreads();
  if (bound) {
    const int e = g.arc_begin[1];
    for (int a = g.arc_begin[0] + threadIdx.x; a < e; a += blockDim.x) {
      const int c = g.arc_cls[a];
      if (c >= 0 && c < C) rootcw[c] = __fadd_rn(0.0f, g.arc_w[a]);
    }
  }
  __syncthreads();
  const int r = r0 + warp;
  if (r >= rows_per_stream) return;
  const int t = r / E, e = r - t * E;
  if (n_frames && t >= n_frames[b]) return;
  const LT* row = logits + static_cast<int64_t>(b) * stream_stride + static_cast<int64_t>(t) * frame_stride + static_cast<int64_t>(e) * row_stride;
  TbTopEnt* o = out + (static_cast<int64_t>(b) * rows_per_stream + r) * (top_m + 1);
  float* y = ybuf + static_cast<size_t>(warp) * V;
  // y of every token; on the way every lane keeps the three best of its strip (value descending, token ascending:
  // the strip is walked in ascending token order, so a strict comparison keeps the lower token among equals)
  float v0 = -INFINITY, v1 = -INFINITY, v2 = -INFINITY;
  int i0 = INT32_MAX, i1 = INT32_MAX, i2 = INT32_MAX;
  int n_strip = 0;
#pragma unroll 4
  for (int v = lane; v < V; v += 32) {
    const float x = LogitLoad<LT>::at(row + v);
    const float yv = bound ? __fadd_rn(x, __fmul_rn(g.lambda, rootcw[__ldg(cls + v)])) : x;
    y[v] = yv;
    ++n_strip;
    if (yv > v0 || i0 == INT32_MAX) { v2 = v1; i2 = i1; v1 = v0; i1 = i0; v0 = yv; i0 = v; }
    else if (yv > v1 || i1 == INT32_MAX) { v2 = v1; i2 = i1; v1 = yv; i1 = v; }
    else if (yv > v2 || i2 == INT32_MAX) { v2 = yv; i2 = v; }
  }
  __syncwarp();
  int n_taken = 0;      // of this lane's strip
  // The rounds only note which token won and its y (the owner's registers hold both); the logit and the class of the
  // picks are looked up afterwards by all lanes at once, so that no round waits for a trip to memory.
  float* pick_y = reinterpret_cast<float*>(ybuf + static_cast<size_t>(kTopWarps) * V) + static_cast<size_t>(warp) * 2 * (top_m + 1);
  int32_t* pick_i = reinterpret_cast<int32_t*>(pick_y + (top_m + 1));
  for (int m = 0; m <= top_m; ++m) {
    // the warp's best: largest value, then lowest token
    const uint32_t u = __float_as_uint(v0 + 0.0f);
    const uint32_t key = i0 == INT32_MAX ? 0u : (u ^ ((u >> 31) ? 0xFFFFFFFFu : 0x80000000u));
    const uint32_t kmax = __reduce_max_sync(0xffffffffu, key);
    const uint32_t imin = __reduce_min_sync(0xffffffffu, (key == kmax && i0 != INT32_MAX) ? static_cast<uint32_t>(i0) : 0xFFFFFFFFu);
    const bool none = imin == 0xFFFFFFFFu;                    // fewer than m + 1 tokens in the row
    if (none) {
      if (lane == 0) { pick_y[m] = -INFINITY; pick_i[m] = -1; }
    } else if (static_cast<uint32_t>(i0) == imin) {
      pick_y[m] = v0; pick_i[m] = i0;
      if (m < top_m) {
        // the owner takes it out: its next best moves up; when the three it kept are used up and the strip holds
        // more, it looks through the strip again
        y[i0] = __int_as_float(0x7FC00000);                   // (a NaN: never greater than anything, never chosen again)
        ++n_taken;
        v0 = v1; i0 = i1; v1 = v2; i1 = i2; v2 = -INFINITY; i2 = INT32_MAX;
        if (i0 == INT32_MAX && n_taken < n_strip) {
          for (int v = lane; v < V; v += 32) {
            const float yv = y[v];
            if (yv == yv) {
              if (yv > v0 || i0 == INT32_MAX) { v2 = v1; i2 = i1; v1 = v0; i1 = i0; v0 = yv; i0 = v; }
              else if (yv > v1 || i1 == INT32_MAX) { v2 = v1; i2 = i1; v1 = yv; i1 = v; }
              else if (yv > v2 || i2 == INT32_MAX) { v2 = yv; i2 = v; }
            }
          }
        }
      }
    }
    __syncwarp();
  }
  for (int m = lane; m <= top_m; m += 32) {
    const int i = pick_i[m];
    TbTopEnt e;
    e.y = pick_y[m];
    if (m == top_m) { e.x = LogitLoad<LT>::at(row + V); e.tok_cls = 0u; }
    else if (i < 0) { e.x = -INFINITY; e.tok_cls = 0xFFFFu; }
    else { e.x = LogitLoad<LT>::at(row + i); e.tok_cls = static_cast<uint32_t>(i) | (static_cast<uint32_t>(__ldg(cls + i)) << 16); }
    o[m] = e;
  }
}

// A chunk of streaming beam decoding: slot by slot, n_frames[slot] frames (at most T) of E rows; each slot has its own
// position in its own tree ring and its own parity of the sequence-record halves, so that slots start, pause and end
// independently of each other (Sec. 2.3: hypotheses kept across chunks; Sec. 2.2 para. 4: slots re-bound in between).
template <typename LT>
__global__ void __launch_bounds__(kBeamThreads) k_beam_chunk(TbBeamParams p, int32_t T, int32_t E, int64_t frame_stride,
                                                         int64_t row_stride, const int32_t* n_frames, int32_t* slot_pos,
                                                         unsigned long long* hash, int32_t* len, size_t n_hyp) {
  __shared__ BeamShared sh;
  LT xpre[kBeamPref] = {};
  bool xpre_valid = false;
  TbTopEnt tpre{0.0f, 0.0f, 0u};
  bool tpre_valid = false;
  const int b = blockIdx.x;
  const int32_t nf = n_frames ? max(0, min(T, n_frames[b])) : T;
  const int32_t pos0 = slot_pos[b];
  const LT* stream_base = reinterpret_cast<const LT*>(p.logits) + static_cast<int64_t>(b) * p.stream_stride;
  extern __shared__ __align__(16) unsigned char dyn_all[];
  const bool fast = beam_fast_applies<LT>(p);
  const bool recs_cached = fast && beam_rec_cache_fill<LT>(p, dyn_all);
  int32_t skip = 0, backoff = 0;
  for (int32_t sidx = 0; sidx < nf * E; ++sidx) {
    if (fast && sidx > 0 && skip-- <= 0) {
      if (threadIdx.x < 32 * (p.K + 1)) {
        const int d = beam_fast_run<LT>(p, sh, dyn_all, sidx, nf * E, E, frame_stride, row_stride, T * E, pos0, hash, hash + n_hyp,
                                        len, len + n_hyp, pos0, recs_cached);
        if (threadIdx.x == 0) sh.fast_done = d;
      }
      __syncthreads();
      const int d = sh.fast_done;
      __syncthreads();
      sidx += d;
      backoff = d == 0 ? min(2 * backoff + 1, 32) : 0;
      skip = backoff;
      xpre_valid = false; tpre_valid = false;
      if (sidx >= nf * E) break;
    }
    {
      const int32_t t = sidx / E, e = sidx - t * E;
      TbBeamParams q = p;
      q.logits = reinterpret_cast<const LT*>(p.logits) + static_cast<int64_t>(t) * frame_stride + static_cast<int64_t>(e) * row_stride;
      q.hyp_stride = 0;
      q.new_frame = e == 0 ? 1 : 0;
      q.merge = e == 0 ? p.merge : 0;
      q.prune_delta = e == 0 ? p.prune_delta : -1.0f;
      q.fresh = 0;
      q.tv_ready = sidx > 0 ? 1 : 0;
      q.step = pos0 + sidx;
      q.top_row = p.top_base ? p.top_base + (static_cast<int64_t>(b) * T * E + sidx) * (p.top_m + 1) : nullptr;
      const size_t in = ((pos0 + sidx) & 1) ? n_hyp : 0, out = ((pos0 + sidx) & 1) ? 0 : n_hyp;
      q.hash_in = hash + in; q.hash_out = hash + out; q.len_in = len + in; q.len_out = len + out;
      const int32_t nt = e + 1 < E ? t : t + 1, ne = e + 1 < E ? e + 1 : 0;
      const LT* next_row = nt < nf ? stream_base + static_cast<int64_t>(nt) * frame_stride + static_cast<int64_t>(ne) * row_stride : nullptr;
      const TbTopEnt* next_top = (nt < nf && q.top_row) ? q.top_row + (p.top_m + 1) : nullptr;
      beam_step_body<LT>(q, sh, xpre, xpre_valid, next_row, tpre, tpre_valid, next_top);
      __syncthreads();
    }
  }
  if (threadIdx.x == 0) slot_pos[b] = pos0 + nf * E;
}

struct SlotList { int32_t slot[TB_BIND_PAIRS]; };
// A new utterance on some slots (or on all): position 0 in the slot's tree, every hypothesis' sequence empty.
// With `scores` given, the slots' rows of the caller's [n_slots, K] arrays are set up as well: hypothesis 0 with score 0
// in the root state (state -1 on an unbound slot), the others empty.
__global__ void k_beam_reset_slots(int32_t* slot_pos, unsigned long long* hash, int32_t* len, size_t n_hyp, int32_t max_beam,   // (max_beam: records per slot)
                                   int32_t n, SlotList sl, int32_t all_slots, const TbSlotRec* slots, int32_t K,
                                   float* scores, int32_t* states, uint8_t* live) {
  const int i = blockIdx.x;
  if (i >= n) return;
  const int slot = all_slots ? i : sl.slot[i];
  if (threadIdx.x == 0) slot_pos[slot] = 0;
  for (int k = threadIdx.x; k < max_beam; k += blockDim.x) {
    const size_t o = static_cast<size_t>(slot) * max_beam + k;
    hash[o] = 0ull; hash[n_hyp + o] = 0ull; len[o] = 0; len[n_hyp + o] = 0;
  }
  if (scores) {
    const bool bound = slots[slot].n_states > 0;
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
      const size_t o = static_cast<size_t>(slot) * K + k;
      scores[o] = k == 0 ? 0.0f : -INFINITY;
      states[o] = (k == 0 && bound) ? 0 : -1;
      live[o] = 0;
    }
  }
}

// The tokens of every hypothesis a slot holds, walked back through the slot's own ring to the start of its utterance.
// Backtrace of one stream's K hypotheses by one warp (lane k: hypothesis k).  The walk from the last step back to the
// first is a chain of dependent loads; the warp therefore brings the tree's nodes of 32 steps at a time into shared
// memory (coalesced, one trip) and the lanes follow their chains there.  The number of tokens of a hypothesis is its
// sequence record's length, so the tokens are written from the back in one walk; only where part of the utterance
// has left the ring (or no record is at hand) a first walk counts what is still there.
// RING: the stream's own ring of tree_cap steps at position slot_pos[slot] (streaming), sequence records in the half
// of len_base that the slot's last step wrote; else the batch-wide tree [n_steps, B, K] with the records at len_cur.
// sl / use_list: the slots to walk (output row i belongs to sl.slot[i]); else slot = block index.
constexpr int kBtSteps = 32;
constexpr int kBtBufs = 4;         // stages in flight: the copies of the next three are under way while one is walked
template <bool RING>
__global__ void __launch_bounds__(32) k_beam_backtrace_warp(const int2* tree, int32_t tree_cap, const int32_t* slot_pos, int32_t n_steps,
                                                           int32_t B, int32_t K, int32_t V, int32_t max_len, int32_t* out_tokens,
                                                           int32_t* out_lens, int32_t* status, const int32_t* len_base,
                                                           size_t n_hyp, const int32_t* len_cur, SlotList sl, int32_t use_list) {
  extern __shared__ __align__(16) int2 bt_stage[];           // [kBtBufs][kBtSteps][K]
  const int lane = threadIdx.x;
  const int b = use_list ? sl.slot[blockIdx.x] : blockIdx.x;
  const int32_t pos = RING ? slot_pos[b] : n_steps;
  const int32_t first = RING ? max(0, pos - tree_cap) : 0;
  const bool cut = RING && pos > tree_cap;
  if (cut && lane == 0) atomicOr(status, TB_STATUS_STEP_LIMIT);   // the utterance is longer than the ring: its start is gone
  const int64_t row = static_cast<int64_t>(blockIdx.x) * K + lane;
  const int32_t* lens = RING ? (pos > 0 ? len_base + (((pos - 1) & 1) ? 0 : n_hyp) : nullptr) : len_cur;
  const bool count_first = cut || (lens == nullptr && pos > 0);
  int32_t n = 0;
  if (!count_first && lane < K) {
    n = lens ? lens[static_cast<int64_t>(b) * K + lane] : 0;
    out_lens[row] = n;
  }
  // A stage is the nodes of up to kBtSteps consecutive steps, [step][K], brought in by asynchronous copies: 16 bytes
  // (two nodes) each when K is even (a step's K nodes are contiguous and then start on a 16-byte boundary), else 8.
  const bool wide = (K & 1) == 0 && (reinterpret_cast<uintptr_t>(tree) & 15) == 0;
  const int per_step = wide ? K >> 1 : K;                    // copies per step
  const uint32_t stage_a = static_cast<uint32_t>(__cvta_generic_to_shared(bt_stage));
  const int n_stages = (pos - first + kBtSteps - 1) / kBtSteps;
  const int ps_shift = (per_step & (per_step - 1)) == 0 ? 31 - __clz(per_step) : -1;   // copies per step a power of two: shifts
  auto fetch = [&](int sidx) {                               // stage sidx holds steps [lo, hi), hi = pos - sidx * kBtSteps
    if (sidx < n_stages) {
      const int32_t hi = pos - sidx * kBtSteps, lo = max(first, hi - kBtSteps), cnt = hi - lo;
      const uint32_t dst0 = stage_a + static_cast<uint32_t>(sidx % kBtBufs) * (kBtSteps * K * 8u);
      const int32_t r0 = RING ? lo % tree_cap : 0;           // ring position of the stage's first step
      const int2* base = RING ? tree + static_cast<int64_t>(b) * tree_cap * K : tree + static_cast<int64_t>(b) * K;
      const int64_t step_stride = RING ? K : static_cast<int64_t>(B) * K;
      const int total = cnt * per_step;
      for (int e = lane; e < total; e += 32) {
        const int j = ps_shift >= 0 ? e >> ps_shift : e / per_step;
        const int c = e - j * per_step;
        int32_t sj = RING ? r0 + j : lo + j;
        if (RING && sj >= tree_cap) sj -= tree_cap;
        const int2* src = base + sj * step_stride;
        if (wide) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst0 + (j * K + 2 * c) * 8u), "l"(src + 2 * c) : "memory");
        else asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst0 + (j * K + c) * 8u), "l"(src + c) : "memory");
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");      // (one group per call, empty beyond the last stage)
  };
  for (int pass = count_first ? 0 : 1; pass < 2; ++pass) {
    int32_t cur = lane < K ? lane : -1, at = n;
    for (int sidx = 0; sidx < kBtBufs - 1; ++sidx) fetch(sidx);
    for (int sidx = 0; sidx < n_stages; ++sidx) {
      fetch(sidx + kBtBufs - 1);
      asm volatile("cp.async.wait_group %0;" ::"n"(kBtBufs - 1) : "memory");
      __syncwarp();
      if (!__any_sync(0xffffffffu, cur >= 0 && (pass == 0 || at > 0))) break;
      const int32_t hi = pos - sidx * kBtSteps, lo = max(first, hi - kBtSteps), cnt = hi - lo;
      const int2* stg = bt_stage + static_cast<size_t>(sidx % kBtBufs) * (kBtSteps * K);
      for (int j = cnt - 1; j >= 0 && cur >= 0; --j) {
        const int2 e = stg[j * K + cur];
        if (e.y >= 0 && e.y != V) {
          if (pass == 0) ++n;
          else { --at; if (at >= 0 && at < max_len) out_tokens[row * max_len + at] = e.y; }
        }
        cur = e.x;
      }
      __syncwarp();
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    __syncwarp();
    if (pass == 0 && lane < K) out_lens[row] = n;
  }
}

__global__ void k_publish_slot(TbSlotRec* slots, TbSlotState* sstate, int32_t slot, TbSlotRec rec) {
  if (threadIdx.x == 0) {
    slots[slot] = rec;
    TbSlotState st;
    st.state = rec.n_states > 0 ? 0 : -1; st.t = 0; st.k = 0; st.score = 0.0f; st.n_emitted = 0;
    st.chunk_base = 0; st.pad0 = 0; st.pad1 = 0;
    sstate[slot] = st;
  }
}

template <typename F>
int set_smem(F* fn, size_t bytes) {
  // (the default limit of 48 KB counts the kernel's static shared memory too -- up to 16 KB here -- so the opt-in
  //  starts well below it)
  if (bytes > 24 * 1024) {
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes)) != cudaSuccess) {
      cudaGetLastError();
      return TB_ERR_INVALID_ARG;
    }
  }
  return TB_OK;
}

}  // namespace

int tb_launch_decode_general(const TbDecodeParams& p_in, cudaStream_t stream, const TbInlineBinds* binds) {
  TbDecodeParams p = p_in;
  TbInlineBinds ib;
  if (binds) ib = *binds; else ib.n = 0;
  if (ib.n < 0 || ib.n > TB_INLINE_BINDS || (ib.n > 0 && (!p.persistent || !ib.arena || !ib.slots))) return TB_ERR_INVALID_ARG;
  size_t smem = static_cast<size_t>(p.C) * (sizeof(float) + sizeof(int32_t));
  // graphs with resolved lists exist only for vocabularies whose token view fits comfortably
  p.tokview = 2 * (p.V + 1) <= (1 << TB_RS_TOK_BITS) ? 1 : 0;
  if (p.tokview && tokview_bytes(p.V, p.C) > smem) smem = tokview_bytes(p.V, p.C);
  int rc;
  if (p.dtype == TB_BF16) {
    if ((rc = set_smem(k_decode_general<uint16_t>, smem)) != TB_OK) return rc;
    k_decode_general<uint16_t><<<p.n_streams, kThreads, smem, stream>>>(p, ib);
  } else {
    if ((rc = set_smem(k_decode_general<float>, smem)) != TB_OK) return rc;
    k_decode_general<float><<<p.n_streams, kThreads, smem, stream>>>(p, ib);
  }
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}

int tb_launch_beam_step(const TbBeamParams& p_in, cudaStream_t stream) {
  TbBeamParams p = p_in;
  p.tokview = 2 * (p.V + 1) <= (1 << TB_RS_TOK_BITS) ? 1 : 0;
  const size_t aux = beam_aux_bytes(p.V, p.C, p.tokview) + static_cast<size_t>(p.V + 1) * sizeof(float);   // + the staged row
  const size_t smem = ((static_cast<size_t>(p.K) * (p.V + 1) * sizeof(float) + 15) & ~size_t(15)) +
                      ((static_cast<size_t>(p.K) * ((p.V + 1 + 31) >> 5) * sizeof(uint32_t) + 15) & ~size_t(15)) + aux;
  if (smem > 200 * 1024) return TB_ERR_INVALID_ARG;
  int rc;
  if (p.dtype == TB_BF16) {
    if ((rc = set_smem(k_beam_step<uint16_t>, smem)) != TB_OK) return rc;
    k_beam_step<uint16_t><<<p.B, kBeamThreads, smem, stream>>>(p);
  } else {
    if ((rc = set_smem(k_beam_step<float>, smem)) != TB_OK) return rc;
    k_beam_step<float><<<p.B, kBeamThreads, smem, stream>>>(p);
  }
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}

// The team steps of narrow beams (beam_fast_run) read rows through two buffers behind the block's other shared
// memory and need the extent of the logits tensor; without either (a wide beam, odd strides) they stay off.
static void beam_fast_setup(TbBeamParams* p, int32_t T, int32_t E, int64_t frame_stride, int64_t row_stride, size_t* smem) {
  p->tensor_lo = nullptr; p->tensor_hi = nullptr; p->rec_cache_bytes = 0;
  if (p->K > kFastMaxK || !p->top_base || p->stream_stride < 0 || frame_stride < 0 || row_stride < 0) return;
  const size_t elem = p->dtype == TB_BF16 ? 2 : 4;
  const size_t more = beam_ring_bytes(p->V, static_cast<int>(elem)) + 16;
  if (*smem + more > 200 * 1024) return;
  *smem += more;
  p->rec_cache_bytes = 0;
  if (*smem + kFastRecCache <= 200 * 1024) { p->rec_cache_bytes = kFastRecCache; *smem += kFastRecCache; }
  const int64_t last = static_cast<int64_t>(p->B - 1) * p->stream_stride + static_cast<int64_t>(T - 1) * frame_stride +
                       static_cast<int64_t>(E - 1) * row_stride + p->V;
  p->tensor_lo = static_cast<const unsigned char*>(p->logits);
  p->tensor_hi = p->tensor_lo + static_cast<size_t>(last + 1) * elem;
}

int tb_launch_beam_frames(const TbBeamParams& p_in, int32_t T, int32_t E, int64_t frame_stride, int64_t row_stride,
                          cudaStream_t stream) {
  TbBeamParams p = p_in;
  p.tokview = 2 * (p.V + 1) <= (1 << TB_RS_TOK_BITS) ? 1 : 0;
  const size_t aux = beam_aux_bytes(p.V, p.C, p.tokview) + static_cast<size_t>(p.V + 1) * sizeof(float);   // + the staged row
  size_t smem = ((static_cast<size_t>(p.K) * (p.V + 1) * sizeof(float) + 15) & ~size_t(15)) +
                ((static_cast<size_t>(p.K) * ((p.V + 1 + 31) >> 5) * sizeof(uint32_t) + 15) & ~size_t(15)) + aux;
  beam_fast_setup(&p, T, E, frame_stride, row_stride, &smem);
  if (smem > 200 * 1024) return TB_ERR_INVALID_ARG;
  int rc;
  if (p.dtype == TB_BF16) {
    if ((rc = set_smem(k_beam_frames<uint16_t>, smem)) != TB_OK) return rc;
    k_beam_frames<uint16_t><<<p.B, kBeamThreads, smem, stream>>>(p, T, E, frame_stride, row_stride);
  } else {
    if ((rc = set_smem(k_beam_frames<float>, smem)) != TB_OK) return rc;
    k_beam_frames<float><<<p.B, kBeamThreads, smem, stream>>>(p, T, E, frame_stride, row_stride);
  }
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}

int tb_launch_beam_backtrace(const int2* tree, int32_t n_steps, int32_t B, int32_t K, int32_t V, int32_t max_len,
                             int32_t* out_tokens, int32_t* out_lens, const int32_t* len_cur, cudaStream_t stream) {
  SlotList none;
  for (int i = 0; i < TB_BIND_PAIRS; ++i) none.slot[i] = 0;
  k_beam_backtrace_warp<false><<<B, 32, kBtBufs * kBtSteps * K * sizeof(int2), stream>>>(tree, 0, nullptr, n_steps, B, K, V, max_len, out_tokens,
                                                                              out_lens, nullptr, nullptr, 0, len_cur, none, 0);
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}

// End of stream: every hypothesis that stops in a graph state is charged that state's final weight,
// score' = fl(score + fl(lambda * final(state))).  Unbound slots, state -1 and empty places (-inf) stay as they are.
__global__ void k_final_weights(const TbSlotRec* slots, const unsigned char* arena, int32_t B, int32_t K, float* scores,
                                const int32_t* states, int32_t* status) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= B * K) return;
  const TbSlotRec rec = slots[i / K];
  const int32_t s = states[i];
  if (rec.n_states <= 0 || s < 0) return;
  if (s >= rec.n_states) { atomicOr(status, TB_STATUS_BAD_STATE); return; }
  const float fin = reinterpret_cast<const float*>(arena + rec.blob_off + rec.off_final)[s];
  const float sc = scores[i];
  if (sc == -INFINITY) return;
  scores[i] = __fadd_rn(sc, __fmul_rn(rec.lambda, fin));
}

int tb_launch_final_weights(const TbSlotRec* slots, const unsigned char* arena, int32_t B, int32_t K, float* scores,
                            const int32_t* states, int32_t* status, cudaStream_t stream) {
  const int n = B * K;
  k_final_weights<<<(n + 127) / 128, 128, 0, stream>>>(slots, arena, B, K, scores, states, status);
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}

__global__ void k_publish_model(TbSlotRec* model_recs, int32_t model_id, TbSlotRec rec) {
  if (threadIdx.x == 0) model_recs[model_id] = rec;
}

struct BindPairs { int32_t slot[TB_BIND_PAIRS]; int32_t model[TB_BIND_PAIRS]; };
__global__ void k_bind_models(TbSlotRec* slots, TbSlotState* sstate, const TbSlotRec* model_recs, int32_t n, BindPairs pr) {
  const int i = threadIdx.x;
  if (i >= n) return;
  TbSlotRec rec;
  if (pr.model[i] >= 0) rec = model_recs[pr.model[i]];
  else memset(&rec, 0, sizeof rec);
  slots[pr.slot[i]] = rec;
  TbSlotState st;
  st.state = rec.n_states > 0 ? 0 : -1; st.t = 0; st.k = 0; st.score = 0.0f; st.n_emitted = 0;
  st.chunk_base = 0; st.pad0 = 0; st.pad1 = 0;
  sstate[pr.slot[i]] = st;
}

int tb_launch_publish_model(TbSlotRec* model_recs, int32_t model_id, const TbSlotRec& rec, cudaStream_t stream) {
  k_publish_model<<<1, 32, 0, stream>>>(model_recs, model_id, rec);
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}

int tb_launch_bind_models(TbSlotRec* slots, TbSlotState* sstate, const TbSlotRec* model_recs, int32_t n,
                          const int32_t* slot_of, const int32_t* model_of, cudaStream_t stream) {
  if (n < 1 || n > TB_BIND_PAIRS) return TB_ERR_INVALID_ARG;
  BindPairs pr;
  for (int i = 0; i < TB_BIND_PAIRS; ++i) { pr.slot[i] = i < n ? slot_of[i] : 0; pr.model[i] = i < n ? model_of[i] : -1; }
  k_bind_models<<<1, TB_BIND_PAIRS, 0, stream>>>(slots, sstate, model_recs, n, pr);
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}

int tb_launch_publish_slot(TbSlotRec* slots, TbSlotState* sstate, int32_t slot, const TbSlotRec& rec,
                           cudaStream_t stream) {
  k_publish_slot<<<1, 32, 0, stream>>>(slots, sstate, slot, rec);
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}

namespace {
// Many slots published at once: the records and their slot indices were copied to the device with the graphs.
__global__ void k_publish_slots(TbSlotRec* slots, TbSlotState* sstate, int32_t n, const TbSlotRec* recs, const int32_t* slot_of) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const TbSlotRec rec = recs[i];
  slots[slot_of[i]] = rec;
  TbSlotState st;
  st.state = rec.n_states > 0 ? 0 : -1; st.t = 0; st.k = 0; st.score = 0.0f; st.n_emitted = 0;
  st.chunk_base = 0; st.pad0 = 0; st.pad1 = 0;
  sstate[slot_of[i]] = st;
}

// Binds carried out by one launch (see TbInlineBinds): block i brings the image of bind i from page-locked host
// memory, read in place, into its arena block, then stores the slot's record and starts the slot's stream afresh.
constexpr int kPullThreads = 512;
__global__ void __launch_bounds__(kPullThreads) k_pull_binds(TbInlineBinds ib, TbSlotState* sstate) {
  const int i = blockIdx.x;
  const unsigned char* src = nullptr;
  int32_t bytes = 0, slot = -1;
  TbSlotRec rec;
#pragma unroll
  for (int j = 0; j < TB_INLINE_BINDS; ++j)
    if (i == j) { src = ib.src[j]; bytes = ib.bytes[j]; slot = ib.slot[j]; rec = ib.rec[j]; }
  if (i >= ib.n || slot < 0) return;
  const uint4* s16 = reinterpret_cast<const uint4*>(src);
  uint4* d16 = reinterpret_cast<uint4*>(ib.arena + rec.blob_off);
  const int n16 = (bytes + 15) >> 4;               // (both blocks are padded to the arena's granule)
  for (int j0 = 0; j0 < n16; j0 += 8 * kPullThreads) {
    uint4 v[8];                                      // eight loads per thread on their way across the bus at once
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int j = j0 + u * kPullThreads + threadIdx.x;
      if (j < n16) v[u] = s16[j];
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int j = j0 + u * kPullThreads + threadIdx.x;
      if (j < n16) d16[j] = v[u];
    }
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    ib.slots[slot] = rec;
    TbSlotState st;
    st.state = rec.n_states > 0 ? 0 : -1; st.t = 0; st.k = 0; st.score = 0.0f; st.n_emitted = 0;
    st.chunk_base = 0; st.pad0 = 0; st.pad1 = 0;
    sstate[slot] = st;
  }
}

__global__ void k_final_weights_slots(const TbSlotRec* slots, const unsigned char* arena, int32_t n, SlotList sl, int32_t K,
                                      float* scores, const int32_t* states, int32_t* status) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n * K) return;
  const int slot = sl.slot[i / K];
  const int64_t o = static_cast<int64_t>(slot) * K + i % K;
  const TbSlotRec rec = slots[slot];
  const float sc = scores[o];
  const int32_t st = states[o];
  if (rec.n_states <= 0 || st < 0 || sc == -INFINITY) return;
  if (st >= rec.n_states) { atomicOr(status, TB_STATUS_BAD_STATE); return; }
  const float fw = reinterpret_cast<const float*>(arena + rec.blob_off + rec.off_final)[st];
  scores[o] = __fadd_rn(sc, __fmul_rn(rec.lambda, fw));
}
}  // namespace

int tb_launch_beam_chunk(const TbBeamParams& p_in, int32_t T, int32_t E, int64_t frame_stride, int64_t row_stride,
                         const int32_t* n_frames, int32_t* slot_pos, unsigned long long* hash, int32_t* len, size_t n_hyp,
                         cudaStream_t stream) {
  TbBeamParams p = p_in;
  p.tokview = 2 * (p.V + 1) <= (1 << TB_RS_TOK_BITS) ? 1 : 0;
  const size_t aux = beam_aux_bytes(p.V, p.C, p.tokview) + static_cast<size_t>(p.V + 1) * sizeof(float);   // + the staged row
  size_t smem = ((static_cast<size_t>(p.K) * (p.V + 1) * sizeof(float) + 15) & ~size_t(15)) +
                ((static_cast<size_t>(p.K) * ((p.V + 1 + 31) >> 5) * sizeof(uint32_t) + 15) & ~size_t(15)) + aux;
  beam_fast_setup(&p, T, E, frame_stride, row_stride, &smem);
  if (smem > 200 * 1024) return TB_ERR_INVALID_ARG;
  int rc;
  if (p.dtype == TB_BF16) {
    if ((rc = set_smem(k_beam_chunk<uint16_t>, smem)) != TB_OK) return rc;
    k_beam_chunk<uint16_t><<<p.B, kBeamThreads, smem, stream>>>(p, T, E, frame_stride, row_stride, n_frames, slot_pos, hash, len, n_hyp);
  } else {
    if ((rc = set_smem(k_beam_chunk<float>, smem)) != TB_OK) return rc;
    k_beam_chunk<float><<<p.B, kBeamThreads, smem, stream>>>(p, T, E, frame_stride, row_stride, n_frames, slot_pos, hash, len, n_hyp);
  }
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}

int tb_launch_beam_reset_slots(int32_t* slot_pos, unsigned long long* hash, int32_t* len, size_t n_hyp, int32_t max_beam,
                               int32_t n, const int32_t* slots, int32_t all_slots, const TbSlotRec* slot_recs, int32_t K,
                               float* scores, int32_t* states, uint8_t* live, cudaStream_t stream) {
  if (n < 1 || (!all_slots && n > TB_BIND_PAIRS)) return TB_ERR_INVALID_ARG;
  SlotList sl;
  for (int i = 0; i < TB_BIND_PAIRS; ++i) sl.slot[i] = (!all_slots && i < n) ? slots[i] : 0;
  k_beam_reset_slots<<<n, 32, 0, stream>>>(slot_pos, hash, len, n_hyp, max_beam, n, sl, all_slots, slot_recs, K, scores, states, live);
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}

int tb_launch_beam_backtrace_slots(const int2* tree, int32_t tree_cap, const int32_t* slot_pos, int32_t n_slots, int32_t K,
                                   int32_t V, int32_t max_len, int32_t* out_tokens, int32_t* out_lens, int32_t* status,
                                   const int32_t* len_base, size_t n_hyp, const int32_t* slot_list, cudaStream_t stream) {
  // slot_list (host, n_slots entries, at most TB_BIND_PAIRS): the slots to walk; null: slots 0 .. n_slots-1
  if (slot_list && n_slots > TB_BIND_PAIRS) return TB_ERR_INVALID_ARG;
  SlotList sl;
  for (int i = 0; i < TB_BIND_PAIRS; ++i) sl.slot[i] = (slot_list && i < n_slots) ? slot_list[i] : 0;
  k_beam_backtrace_warp<true><<<n_slots, 32, kBtBufs * kBtSteps * K * sizeof(int2), stream>>>(tree, tree_cap, slot_pos, 0, n_slots, K, V, max_len,
                                                                                   out_tokens, out_lens, status, len_base, n_hyp, nullptr,
                                                                                   sl, slot_list ? 1 : 0);
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}

int tb_launch_final_weights_slots(const TbSlotRec* slots, const unsigned char* arena, int32_t n, const int32_t* slot_list,
                                  int32_t K, float* scores, const int32_t* states, int32_t* status, cudaStream_t stream) {
  if (n < 1 || n > TB_BIND_PAIRS) return TB_ERR_INVALID_ARG;
  SlotList sl;
  for (int i = 0; i < TB_BIND_PAIRS; ++i) sl.slot[i] = i < n ? slot_list[i] : 0;
  const int total = n * K;
  k_final_weights_slots<<<(total + 127) / 128, 128, 0, stream>>>(slots, arena, n, sl, K, scores, states, status);
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}

int tb_launch_publish_slots(TbSlotRec* slots, TbSlotState* sstate, int32_t n, const TbSlotRec* recs, const int32_t* slot_of,
                            cudaStream_t stream) {
  if (n < 1) return TB_ERR_INVALID_ARG;
  k_publish_slots<<<(n + 63) / 64, 64, 0, stream>>>(slots, sstate, n, recs, slot_of);
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}

int tb_launch_pull_binds(const TbInlineBinds& ib, TbSlotState* sstate, cudaStream_t stream) {
  if (ib.n < 1 || ib.n > TB_INLINE_BINDS || !ib.arena || !ib.slots || !sstate) return TB_ERR_INVALID_ARG;
  k_pull_binds<<<ib.n, kPullThreads, 0, stream>>>(ib, sstate);
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}

int tb_launch_beam_topm(const void* logits, int dtype, int32_t B, int32_t T, int32_t E, int32_t V, int32_t C,
                        int64_t stream_stride, int64_t frame_stride, int64_t row_stride, const int32_t* n_frames,
                        const TbSlotRec* slots, const unsigned char* arena, const int32_t* cls, int32_t top_m,
                        TbTopEnt* out, cudaStream_t stream) {
  // root weights per class, every warp's y values, every warp's picks (value and token, top_m + 1 each)
  const size_t smem = (static_cast<size_t>(C) + static_cast<size_t>(kTopWarps) * V + static_cast<size_t>(kTopWarps) * 2 * (top_m + 1)) * sizeof(float);
  const int blocks = B * ((T * E + kTopWarps - 1) / kTopWarps);
  int rc;
  if (dtype == TB_BF16) {
    if ((rc = set_smem(k_beam_topm<uint16_t>, smem)) != TB_OK) return rc;
    k_beam_topm<uint16_t><<<blocks, kTopWarps * 32, smem, stream>>>(static_cast<const uint16_t*>(logits), B, T, E, V, C, stream_stride,
                                                                  frame_stride, row_stride, n_frames, slots, arena, cls, top_m, out);
  } else {
    if ((rc = set_smem(k_beam_topm<float>, smem)) != TB_OK) return rc;
    k_beam_topm<float><<<blocks, kTopWarps * 32, smem, stream>>>(static_cast<const float*>(logits), B, T, E, V, C, stream_stride,
                                                               frame_stride, row_stride, n_frames, slots, arena, cls, top_m, out);
  }
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}
