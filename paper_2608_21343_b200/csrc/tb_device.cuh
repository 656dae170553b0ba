// Device-side building blocks shared by the decode kernels: graph access through the slot
// offset table, the suffix-link walk, ordered (value, id) reductions.
#ifndef TB_DEVICE_CUH_
#define TB_DEVICE_CUH_

#include <cuda_runtime.h>

#include <cstdint>

#include "tb_internal.h"

#define TB_CHAIN_MAX 257  // a walk visits at most max_depth + 1 <= 256 states

struct GraphPtrs {
  const int32_t* arc_begin;
  const int32_t* fail;
  const float* bw;
  const int32_t* arc_cls;
  const float* arc_w;
  const int32_t* arc_dst;
  int32_t n_states, n_arcs, max_depth;
  float lambda;
};

// The slot's record selects the stream's graph: per-slot offsets into the arena give the graph's arrays (Sec. 2.2 para. 3).
__device__ __forceinline__ GraphPtrs graph_of(const unsigned char* arena, const TbSlotRec& r) {
  GraphPtrs g;
  const unsigned char* blob = arena + r.blob_off;
  g.arc_begin = reinterpret_cast<const int32_t*>(blob + r.off_arc_begin);
  g.fail = reinterpret_cast<const int32_t*>(blob + r.off_fail);
  g.bw = reinterpret_cast<const float*>(blob + r.off_bw);
  g.arc_cls = reinterpret_cast<const int32_t*>(blob + r.off_arc_cls);
  g.arc_w = reinterpret_cast<const float*>(blob + r.off_arc_w);
  g.arc_dst = reinterpret_cast<const int32_t*>(blob + r.off_arc_dst);
  g.n_states = r.n_states; g.n_arcs = r.n_arcs; g.max_depth = r.max_depth; g.lambda = r.lambda;
  return g;
}

template <typename LT> struct LogitLoad;
template <> struct LogitLoad<float> {
  static __device__ __forceinline__ float at(const float* p) { return __ldg(p); }
  // the load alone (nothing waits for it until the value is widened), and the widening
  static __device__ __forceinline__ float raw(const float* p) { return __ldg(p); }
  static __device__ __forceinline__ float widen(float r) { return r; }
};
template <> struct LogitLoad<uint16_t> {  // bf16 bits, widened exactly
  static __device__ __forceinline__ float at(const uint16_t* p) {
    return __uint_as_float(static_cast<uint32_t>(__ldg(p)) << 16);
  }
  static __device__ __forceinline__ uint16_t raw(const uint16_t* p) { return __ldg(p); }
  static __device__ __forceinline__ float widen(uint16_t r) { return __uint_as_float(static_cast<uint32_t>(r) << 16); }
};

// Index of the arc of state u labelled with class c, or -1 (arcs are sorted by class).
__device__ __forceinline__ int32_t find_arc(const GraphPtrs& g, int32_t u, int32_t c) {
  int32_t lo = g.arc_begin[u], hi = g.arc_begin[u + 1];
  while (lo < hi) {
    int32_t mid = (lo + hi) >> 1;
    int32_t cm = g.arc_cls[mid];
    if (cm < c) lo = mid + 1; else hi = mid;
  }
  return (lo < g.arc_begin[u + 1] && g.arc_cls[lo] == c) ? lo : -1;
}

// Suffix-link walk for one (state, class): the next state.  The bonus is not needed by the
// callers of this function (they evaluate whole rows through the bonus vector).
__device__ inline int32_t walk_next(const GraphPtrs& g, int32_t s, int32_t c, int32_t* status) {
  int32_t u = s;
  for (int32_t it = 0; it <= g.max_depth + 1; ++it) {
    int32_t a = find_arc(g, u, c);
    if (a >= 0) return g.arc_dst[a];
    if (u == 0) return 0;
    u = g.fail[u];
  }
  atomicOr(status, TB_STATUS_WALK_TOO_DEEP);
  return 0;
}

// (value, id) ordered "larger value first, then smaller id".
struct ValId {
  float v;
  int32_t i;
};
__device__ __forceinline__ bool better(const ValId& a, const ValId& b) {
  return a.v > b.v || (a.v == b.v && a.i < b.i);
}
__device__ __forceinline__ ValId warp_best(ValId x) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    ValId y;
    y.v = __shfl_xor_sync(0xffffffffu, x.v, off);
    y.i = __shfl_xor_sync(0xffffffffu, x.i, off);
    if (better(y, x)) x = y;
  }
  return x;
}

// Block-wide best; every thread gets the result.  `scratch` holds one ValId per warp plus one.
__device__ __forceinline__ ValId block_best(ValId x, ValId* scratch) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
  x = warp_best(x);
  __syncthreads();  // scratch may still be read from the previous use
  if (lane == 0) scratch[warp] = x;
  __syncthreads();
  if (warp == 0) {
    ValId y = lane < nwarps ? scratch[lane] : ValId{-INFINITY, INT32_MAX};
    y = warp_best(y);
    if (lane == 0) scratch[nwarps] = y;
  }
  __syncthreads();
  return scratch[nwarps];
}

// Dense bonus / next-state vectors over classes for state s (what the scoring kernel of
// Sec. 2.2 para. 3 hands the decoder per batch item; here kept in shared memory, indexed by class).
// The chain s, fail(s), ... root is walked once; acc_j is the sum of the suffix-link weights
// crossed before chain state j (float adds in walk order).  Classes are then filled from the
// root end of the chain toward s, so the state closest to s wins.
__device__ inline void build_bonus(const GraphPtrs& g, int32_t s, int32_t C, float* bvec, int32_t* nvec,
                                   int32_t* ch_state, float* ch_acc, int32_t* ch_len, int32_t* status) {
  if (threadIdx.x == 0) {
    int32_t m = 0, u = s;
    float acc = 0.0f;
    if (u < 0 || u >= g.n_states) { atomicOr(status, TB_STATUS_BAD_STATE); u = 0; }
    for (;;) {
      ch_state[m] = u; ch_acc[m] = acc; ++m;
      if (u == 0) break;
      if (m > g.max_depth + 1 || m >= TB_CHAIN_MAX - 1) {  // cannot happen for a well-formed graph
        atomicOr(status, TB_STATUS_WALK_TOO_DEEP);
        ch_state[m] = 0; ch_acc[m] = acc; ++m;
        break;
      }
      acc = __fadd_rn(acc, g.bw[u]);
      u = g.fail[u];
    }
    *ch_len = m;
  }
  __syncthreads();
  const int32_t m = *ch_len;
  const float dflt = ch_acc[m - 1];
  for (int32_t c = threadIdx.x; c < C; c += blockDim.x) { bvec[c] = dflt; nvec[c] = 0; }
  for (int32_t j = m - 1; j >= 0; --j) {
    __syncthreads();
    const int32_t u = ch_state[j];
    const float acc = ch_acc[j];
    const int32_t e = g.arc_begin[u + 1];
    for (int32_t a = g.arc_begin[u] + threadIdx.x; a < e; a += blockDim.x) {
      const int32_t c = g.arc_cls[a];
      if (c >= 0 && c < C) { bvec[c] = __fadd_rn(acc, g.arc_w[a]); nvec[c] = g.arc_dst[a]; }
    }
  }
  __syncthreads();
}

#endif  // TB_DEVICE_CUH_
