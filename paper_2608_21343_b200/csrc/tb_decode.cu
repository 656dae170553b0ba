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

template <typename LT>
__global__ void __launch_bounds__(kThreads) k_decode_general(TbDecodeParams p) {
  extern __shared__ __align__(16) unsigned char dyn[];
  float* bvec = reinterpret_cast<float*>(dyn);
  int32_t* nvec = reinterpret_cast<int32_t*>(dyn + sizeof(float) * p.C);
  __shared__ StepSmem sm;

  const int b = blockIdx.x;
  const TbSlotRec rec = p.slots[b];
  const bool bound = rec.n_states > 0;
  const GraphPtrs g = graph_of(p.arena, rec);
  const LT* base = reinterpret_cast<const LT*>(p.logits) + static_cast<int64_t>(b) * p.sb;
  const int V = p.V;

  // where this call starts and ends for the stream
  int32_t t0 = 0, end, s, t, k, n_total = 0;
  float score;
  if (p.persistent) {
    const TbSlotState st = p.sstate[b];
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
      build_bonus(g, s, p.C, bvec, nvec, sm.chain.state, sm.chain.acc, &sm.chain.len, p.status);
      built_for = s;
    }
    const LT* row = base + static_cast<int64_t>(t - t0) * p.st + static_cast<int64_t>(k) * p.ss;
    ValId best{-INFINITY, INT32_MAX};
    for (int v = threadIdx.x; v <= V; v += kThreads) {
      float x = LogitLoad<LT>::at(row + static_cast<int64_t>(v) * p.sv);
      float val = (bound && v < V) ? __fadd_rn(x, __fmul_rn(g.lambda, bvec[__ldg(p.cls + v)])) : x;
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
      if (bound) s = nvec[__ldg(p.cls + tok)];
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
__device__ __forceinline__ bool before(const BeamKey& a, const BeamKey& b) {
  return a.v > b.v || (a.v == b.v && (a.tkey < b.tkey || (a.tkey == b.tkey && a.par < b.par)));
}
__device__ __forceinline__ BeamKey warp_first(BeamKey x) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    BeamKey y;
    y.v = __shfl_xor_sync(0xffffffffu, x.v, off);
    y.tkey = __shfl_xor_sync(0xffffffffu, x.tkey, off);
    y.par = __shfl_xor_sync(0xffffffffu, x.par, off);
    if (before(y, x)) x = y;
  }
  return x;
}

template <typename LT>
__global__ void __launch_bounds__(kThreads) k_beam_step(TbBeamParams p) {
  extern __shared__ __align__(16) unsigned char dyn[];
  const int V = p.V, K = p.K, W = V + 1;
  float* cand = reinterpret_cast<float*>(dyn);                         // [K, V+1]
  float* bvec = cand + static_cast<size_t>(K) * W;                     // [C]
  int32_t* nvec = reinterpret_cast<int32_t*>(bvec + p.C);              // [C]
  __shared__ ChainSmem chain;
  __shared__ BeamKey red[kThreads / 32 + 1];
  __shared__ float h_score[TB_MAX_BEAM];
  __shared__ int32_t h_state[TB_MAX_BEAM];
  __shared__ uint8_t h_live[TB_MAX_BEAM];
  __shared__ BeamKey sel[TB_MAX_BEAM];

  const int b = blockIdx.x;
  const TbSlotRec rec = p.slots[b];
  const bool bound = rec.n_states > 0;
  const GraphPtrs g = graph_of(p.arena, rec);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  if (threadIdx.x < K) {
    const int64_t o = static_cast<int64_t>(b) * K + threadIdx.x;
    float sc = p.scores[o];
    h_score[threadIdx.x] = sc;
    h_state[threadIdx.x] = p.states[o];
    h_live[threadIdx.x] = p.new_frame ? static_cast<uint8_t>(sc != -INFINITY) : p.live[o];
  }
  __syncthreads();

  // all candidate values of the live hypotheses
  for (int k = 0; k < K; ++k) {
    if (h_score[k] == -INFINITY || !h_live[k]) continue;  // uniform across the block
    if (bound) build_bonus(g, h_state[k], p.C, bvec, nvec, chain.state, chain.acc, &chain.len, p.status);
    const LT* row = reinterpret_cast<const LT*>(p.logits) + static_cast<int64_t>(b) * p.stream_stride +
                    static_cast<int64_t>(k) * p.hyp_stride;
    const float sc = h_score[k];
    for (int v = threadIdx.x; v < W; v += kThreads) {
      float x = LogitLoad<LT>::at(row + v);
      float val = (bound && v < V) ? __fadd_rn(x, __fmul_rn(g.lambda, bvec[__ldg(p.cls + v)])) : x;
      cand[static_cast<size_t>(k) * W + v] = __fadd_rn(sc, val);
    }
    __syncthreads();
  }

  // K rounds: the first candidate, in order, that comes strictly after the previous pick
  BeamKey prev{INFINITY, -2, -2};
  const BeamKey none{-INFINITY, INT32_MAX, INT32_MAX};
  for (int r = 0; r < K; ++r) {
    BeamKey best = none;
    for (int k = 0; k < K; ++k) {
      if (h_score[k] == -INFINITY) continue;
      if (!h_live[k]) {
        if (threadIdx.x == 0) {
          BeamKey c{h_score[k], V + 1, k};
          if (before(prev, c) && before(c, best)) best = c;
        }
        continue;
      }
      for (int v = threadIdx.x; v < W; v += kThreads) {
        BeamKey c{cand[static_cast<size_t>(k) * W + v], v, k};
        if (before(prev, c) && before(c, best)) best = c;
      }
    }
    best = warp_first(best);
    if (lane == 0) red[warp] = best;
    __syncthreads();
    if (warp == 0) {
      BeamKey y = lane < kThreads / 32 ? red[lane] : none;
      y = warp_first(y);
      if (lane == 0) red[kThreads / 32] = y;
    }
    __syncthreads();
    best = red[kThreads / 32];
    if (threadIdx.x == 0) sel[r] = best;
    prev = best;           // once `none` is reached every later round yields `none` again
    __syncthreads();
  }

  // new hypotheses, the hypothesis tree
  if (threadIdx.x < K) {
    const int r = threadIdx.x;
    const BeamKey c = sel[r];
    const int64_t o = static_cast<int64_t>(b) * K + r;
    int32_t parent = -1, token = -1, state = -1;
    uint8_t lv = 0;
    float sc = -INFINITY;
    if (c.par != INT32_MAX) {
      parent = c.par; sc = c.v;
      token = (c.tkey == V + 1) ? -1 : c.tkey;
      state = h_state[parent];
      if (token >= 0 && token != V) {
        if (bound) state = walk_next(g, state, __ldg(p.cls + token), p.status);
        lv = h_live[parent];
      }
    }
    p.scores[o] = sc; p.states[o] = state; p.live[o] = lv;
    p.out_parent[o] = parent; p.out_token[o] = token;
    if (p.tree) p.tree[(static_cast<int64_t>(p.step) * p.B + b) * K + r] = make_int2(parent, token);
  }
}

__global__ void k_beam_backtrace(const int2* tree, int32_t n_steps, int32_t B, int32_t K, int32_t V,
                                 int32_t max_len, int32_t* out_tokens, int32_t* out_lens) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= B * K) return;
  const int b = idx / K;
  // pass 1: length; pass 2: fill from the back
  int32_t n = 0;
  for (int pass = 0; pass < 2; ++pass) {
    int32_t slot = idx % K, pos = n;
    for (int32_t st = n_steps - 1; st >= 0 && slot >= 0; --st) {
      const int2 e = tree[(static_cast<int64_t>(st) * B + b) * K + slot];
      if (e.y >= 0 && e.y != V) {
        if (pass == 0) ++n;
        else { --pos; if (pos < max_len) out_tokens[static_cast<int64_t>(idx) * max_len + pos] = e.y; }
      }
      slot = e.x;
    }
    if (pass == 0) out_lens[idx] = n;
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
  if (bytes > 48 * 1024) {
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes)) != cudaSuccess) {
      cudaGetLastError();
      return TB_ERR_INVALID_ARG;
    }
  }
  return TB_OK;
}

}  // namespace

int tb_launch_decode_general(const TbDecodeParams& p, cudaStream_t stream) {
  const size_t smem = static_cast<size_t>(p.C) * (sizeof(float) + sizeof(int32_t));
  int rc;
  if (p.dtype == TB_BF16) {
    if ((rc = set_smem(k_decode_general<uint16_t>, smem)) != TB_OK) return rc;
    k_decode_general<uint16_t><<<p.n_streams, kThreads, smem, stream>>>(p);
  } else {
    if ((rc = set_smem(k_decode_general<float>, smem)) != TB_OK) return rc;
    k_decode_general<float><<<p.n_streams, kThreads, smem, stream>>>(p);
  }
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}

int tb_launch_beam_step(const TbBeamParams& p, cudaStream_t stream) {
  const size_t smem = static_cast<size_t>(p.K) * (p.V + 1) * sizeof(float) +
                      static_cast<size_t>(p.C) * (sizeof(float) + sizeof(int32_t));
  if (smem > 200 * 1024) return TB_ERR_INVALID_ARG;
  int rc;
  if (p.dtype == TB_BF16) {
    if ((rc = set_smem(k_beam_step<uint16_t>, smem)) != TB_OK) return rc;
    k_beam_step<uint16_t><<<p.B, kThreads, smem, stream>>>(p);
  } else {
    if ((rc = set_smem(k_beam_step<float>, smem)) != TB_OK) return rc;
    k_beam_step<float><<<p.B, kThreads, smem, stream>>>(p);
  }
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}

int tb_launch_beam_backtrace(const int2* tree, int32_t n_steps, int32_t B, int32_t K, int32_t V, int32_t max_len,
                             int32_t* out_tokens, int32_t* out_lens, cudaStream_t stream) {
  const int n = B * K;
  k_beam_backtrace<<<(n + 127) / 128, 128, 0, stream>>>(tree, n_steps, B, K, V, max_len, out_tokens, out_lens);
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}

int tb_launch_publish_slot(TbSlotRec* slots, TbSlotState* sstate, int32_t slot, const TbSlotRec& rec,
                           cudaStream_t stream) {
  k_publish_slot<<<1, 32, 0, stream>>>(slots, sstate, slot, rec);
  return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}
