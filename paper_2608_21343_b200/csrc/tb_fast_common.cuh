// Device code shared by the two pipelined greedy kernels (tb_greedy_fast.cu, tb_greedy_seg.cu): the row summary a
// helper warp leaves for a decider, the helper itself (one row of packed bf16 logits -> summary), the view of the
// current graph state's boosted-token list, and small shared-memory / packing primitives.
#ifndef TB_FAST_COMMON_CUH_
#define TB_FAST_COMMON_CUH_

#include <cuda_bf16.h>

#include "tb_device.cuh"

namespace {

constexpr int kSMax = 4;        // rows per frame the ring bookkeeping is sized for
constexpr int kNitMax = 8;      // 256 tokens per pass iteration: V <= 2048 (kernel instantiated for 1, 2, 4, 8)

// What a helper leaves for the decider about one row (32 bytes, read as two 16-byte loads).
struct RowSummary {
  float y1;          // best root-boosted token value of the row (ties: lowest id)
  float y2b;         // upper bound on the root-boosted value of every other token
  float xb;          // blank logit
  float x1;          // raw logit of the best token
  float rootcw1;     // root arc weight of the best token's class (0 if none)
  int32_t rootdst1;  // root arc target of the best token's class (0 if none)
  uint32_t packed;   // id1 | overflow << 16 | gap_ok << 17  (gap_ok: y1 clears y2b by the rounding margin of any state)
  uint32_t seq;      // frame number + 1: written last; the decider takes the summary as valid when it matches
};
constexpr uint32_t kSumOvf = 1u << 16, kSumGap = 1u << 17;
// Summaries of one ring stage are kSMax * 32 bytes; stages are spaced 16 bytes further apart so that the
// decider's lanes (one stage each) read their 16-byte halves from distinct shared-memory banks.  A decode that
// normalises its rows keeps the stage's kSMax normalisers (floats) in those 16 bytes.
constexpr int kSumStageBytes = kSMax * 32 + 16;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }
__device__ __forceinline__ float row_at(const unsigned char* rowp, int idx) {
  return bf16_bits_to_float(*reinterpret_cast<const uint16_t*>(rowp + 2 * idx));
}
__device__ __forceinline__ __nv_bfloat162 as_bf162(uint32_t w) {
  __nv_bfloat162 r;
  *reinterpret_cast<uint32_t*>(&r) = w;
  return r;
}
// Order-preserving map float -> uint32 (-0 is folded into +0 first, so equal floats get equal keys).
__device__ __forceinline__ uint32_t fkey(float v) {
  const uint32_t u = __float_as_uint(v + 0.0f);
  return u ^ ((u >> 31) ? 0xFFFFFFFFu : 0x80000000u);
}
__device__ __forceinline__ float fkey_inv(uint32_t k) {
  return __uint_as_float(k ^ ((k >> 31) ? 0x80000000u : 0xFFFFFFFFu));
}

// Shared-memory accesses by 32-bit shared address (keeps the decider's address arithmetic short).
__device__ __forceinline__ uint32_t lds_u16(uint32_t a) {
  uint16_t v;
  asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ uint2 lds_v2(uint32_t a) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
  return v;
}
__device__ __forceinline__ uint4 lds_v4(uint32_t a) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
  return v;
}
// The same loads as plain asm (not volatile): for the list cache and for rows of a held ring slot, which do not
// change while the decider reads them, so that the compiler may schedule them freely.
__device__ __forceinline__ uint32_t lds_u16_nv(uint32_t a) {
  uint16_t v;
  asm("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ uint2 lds_v2_nv(uint32_t a) {
  uint2 v;
  asm("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
  return v;
}
__device__ __forceinline__ uint4 lds_v4_volatile(uint32_t a) {
  uint4 v;
  asm volatile("ld.volatile.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a) : "memory");
  return v;
}
__device__ __forceinline__ float lds_f32_volatile(uint32_t a) {
  float v;
  asm volatile("ld.volatile.shared.f32 %0, [%1];" : "=f"(v) : "r"(a) : "memory");
  return v;
}
__device__ __forceinline__ float exp2f_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void sts_v4_volatile(uint32_t a, uint4 v) {
  asm volatile("st.volatile.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// ---- helper: one row -> summary ----------------------------------------------------------------
struct HelperCtx {
  const uint16_t* cls16;
  const float* tokcb;
  const float* rootcw;
  const int32_t* rootdst;
  float beta_min, beta_max, dbeta;
  float bmag_max;   // bound on |lambda| * (|D(s)| + largest root weight) over all states s
  int V, nit;
};

// One row as a helper warp holds it: lane l has the 16-byte blocks l, l + 32, ... of the 16-byte aligned superset of
// the row (words w), and one of the at most seven tokens that follow the last full pass (tail_bits).
template <int NIT>
struct RowRegs {
  uint32_t w[4 * NIT];
  uint32_t tail_bits;
};

// Loads a row.  `slot + off_bytes` is the row's first element; the blocks are read from the aligned address below it.
// lo / hi: when not null, the first and one-past-last byte that may be read (the tensor); a block that leaves this
// range is assembled from the elements inside it, the rest reads as -inf.  Without them every block must be readable.
template <int NIT>
__device__ __forceinline__ void load_row(const HelperCtx& h, const unsigned char* slot, int off_bytes, int lane,
                                         const unsigned char* lo, const unsigned char* hi, RowRegs<NIT>& r) {
  const int p = (off_bytes & 15) >> 1;
  const unsigned char* a0 = slot + (off_bytes & ~15);
  const uint4* blk = reinterpret_cast<const uint4*>(a0);
  const unsigned char* rowp = slot + off_bytes;
  const uint32_t NEG2 = 0xFF80FF80u;                      // two bf16 -inf
  const bool guard = lo != nullptr && (a0 < lo || a0 + h.nit * 512 > hi);      // the same for the whole warp
#pragma unroll
  for (int j = 0; j < NIT; ++j) {
    if (j < h.nit) {
      if (!guard) {
        const uint4 q = blk[j * 32 + lane];
        r.w[4 * j] = q.x; r.w[4 * j + 1] = q.y; r.w[4 * j + 2] = q.z; r.w[4 * j + 3] = q.w;
      } else {
        const unsigned char* a = a0 + 16 * (j * 32 + lane);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          uint32_t lo16 = 0xFF80u, hi16 = 0xFF80u;
          if (a + 4 * e >= lo && a + 4 * e + 2 <= hi) lo16 = *reinterpret_cast<const uint16_t*>(a + 4 * e);
          if (a + 4 * e + 2 >= lo && a + 4 * e + 4 <= hi) hi16 = *reinterpret_cast<const uint16_t*>(a + 4 * e + 2);
          r.w[4 * j + e] = lo16 | (hi16 << 16);
        }
      }
    } else {
      r.w[4 * j] = r.w[4 * j + 1] = r.w[4 * j + 2] = r.w[4 * j + 3] = NEG2;
    }
  }
  // tokens after the last full pass (at most 7): one element per lane
  const int tail_idx = h.nit * 256 - p + lane;
  r.tail_bits = 0xFF80u;
  if (tail_idx < h.V && tail_idx >= 0) r.tail_bits = *reinterpret_cast<const uint16_t*>(rowp + 2 * tail_idx);
}

// Row in registers -> summary at shared address out_a (see RowSummary).  rowp: the row's first element (the few exact
// candidate values are re-read from there), p: elements of the first 16-byte block that precede the row.
// NORM: the row's log-softmax normaliser L = M + log(sum_v exp(x_v - M)) over its V + 1 entries (M: their maximum)
// is computed as well, in float with a fixed order of additions, and stored at shared address lse_a before the
// summary's sequence word (0 for a row without a finite entry).
template <int NIT, bool NORM = false>
__device__ __forceinline__ void finish_row(const HelperCtx& h, RowRegs<NIT>& r, const unsigned char* rowp, int p,
                                           uint32_t out_a, uint32_t seq, int lane, uint32_t lse_a = 0u) {
  const int V = h.V;
  uint32_t (&w)[4 * NIT] = r.w;
  // What the 16-byte blocks hold beyond this row's tokens is masked to -inf: the p elements before the row in
  // the first block (lane 0 only), and everything from element V on when the passes reach that far.
  if (p > 0 && lane == 0) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (2 * e < p) w[e] = (w[e] & 0xFFFF0000u) | 0xFF80u;
      if (2 * e + 1 < p) w[e] = (w[e] & 0x0000FFFFu) | 0xFF800000u;
    }
  }
  if (V + p < h.nit * 256) {
#pragma unroll
    for (int j = 0; j < NIT; ++j) {
      const int idx0 = (j * 32 + lane) * 8 - p;             // token id of the block's first element
      if (j < h.nit && idx0 + 8 > V) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int i0 = idx0 + 2 * e;
          if (i0 >= V) w[4 * j + e] = (w[4 * j + e] & 0xFFFF0000u) | 0xFF80u;
          if (i0 + 1 >= V) w[4 * j + e] = (w[4 * j + e] & 0x0000FFFFu) | 0xFF800000u;
        }
      }
    }
  }
  const int tail_idx = h.nit * 256 - p + lane;
  const bool tail_ok = tail_idx < V && tail_idx >= 0;
  const uint32_t tail_bits = r.tail_bits;

  // pass 1: raw maximum of the row's token logits (tree of packed maxima, then across the warp)
  __nv_bfloat162 mm[4 * NIT];
#pragma unroll
  for (int i = 0; i < 4 * NIT; ++i) mm[i] = as_bf162(w[i]);
#pragma unroll
  for (int n = 2 * NIT; n >= 1; n >>= 1) {
#pragma unroll
    for (int i = 0; i < n; ++i) mm[i] = __hmax2(mm[i], mm[i + n]);
  }
  const __nv_bfloat162 m2 = __hmax2(mm[0], as_bf162(tail_bits | 0xFF800000u));
  __nv_bfloat16 m = __hmax(__low2bfloat16(m2), __high2bfloat16(m2));
  {
    // order-preserving integer image of a bf16, so that one warp-wide integer max does the reduction
    const uint32_t u = __bfloat16_as_ushort(m);
    const uint32_t key = (u & 0x8000u) ? (0xFFFFu ^ u) : (u | 0x8000u);
    const uint32_t kmax = __reduce_max_sync(0xffffffffu, key);
    const uint32_t ub = (kmax & 0x8000u) ? (kmax ^ 0x8000u) : (0xFFFFu ^ kmax);
    m = __ushort_as_bfloat16(static_cast<unsigned short>(ub));
  }
  const float mf = __bfloat162float(m);
  float lse = 0.0f;
  if constexpr (NORM) {
    // sum_v 2^(x_v * log2(e) - c) with c = fl(M * log2(e)): one fused multiply-add and one exponential per entry; what
    // the rounding of c scales the sum by (2^(c - M * log2(e)), the same for every entry) is taken off the logarithm
    const float xbl = row_at(rowp, V);
    const float M = fmaxf(mf, xbl);
    const float kL2e = 1.4426950408889634f;
    const float c = __fmul_rn(M, kL2e), nc = -c;
    float acc0 = 0.0f, acc1 = 0.0f;
#pragma unroll
    for (int i = 0; i < 4 * NIT; ++i) {
      acc0 = __fadd_rn(acc0, exp2f_approx(__fmaf_rn(__uint_as_float(w[i] << 16), kL2e, nc)));
      acc1 = __fadd_rn(acc1, exp2f_approx(__fmaf_rn(__uint_as_float(w[i] & 0xFFFF0000u), kL2e, nc)));
    }
    float acc = __fadd_rn(acc0, acc1);
    if (tail_ok) acc = __fadd_rn(acc, exp2f_approx(__fmaf_rn(bf16_bits_to_float(tail_bits), kL2e, nc)));
    if (lane == 0) acc = __fadd_rn(acc, exp2f_approx(__fmaf_rn(xbl, kL2e, nc)));
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc = __fadd_rn(acc, __shfl_xor_sync(0xffffffffu, acc, off));
    const float c_lo = __fmaf_rn(M, kL2e, nc);                       // M * log2(e) - c, exactly
    lse = (M == -INFINITY) ? 0.0f : __fadd_rn(M, __fsub_rn(logf(acc), __fmul_rn(c_lo, 0.6931471805599453f)));
  }
  // Every token whose root-boosted value can reach that of the raw maximum has x >= m - dbeta;
  // gamma keeps a strict margin over all roundings.  thr is rounded down.
  const float gamma = (fabsf(mf) + fabsf(h.beta_max) + fabsf(h.beta_min)) * 0.0009765625f + 1e-30f;
  const float thr_f = __fsub_rn(__fsub_rn(mf, h.dbeta), gamma);
  const __nv_bfloat16 thr = __float2bfloat16_rd(thr_f);
  const __nv_bfloat162 thr2 = __halves2bfloat162(thr, thr);

  // pass 2: one bit per element of this lane that reaches the threshold (bit i + 16 h: word i, half h)
  uint32_t hits = 0;
#pragma unroll
  for (int i = 0; i < 4 * NIT; ++i) {
    const uint32_t mk = __hge2_mask(as_bf162(w[i]), thr2);          // 0xFFFF per half that passes
    if (4 * NIT <= 16) hits |= mk & (0x00010001u << i);
    else if (mk) hits |= 1u << (i & 31);                             // NIT = 8: one bit per word, both halves re-tested below
  }
  // exact root-boosted values of this lane's candidates: best (value, lowest id) and runner-up value
  ValId b{-INFINITY, INT32_MAX};
  float sec = -INFINITY;
  while (hits) {
    const int bit = __ffs(hits) - 1;
    hits &= hits - 1u;
    if (4 * NIT <= 16) {
      const int i = bit & 15;
      const int idx = ((i >> 2) * 32 + lane) * 8 + (i & 3) * 2 + (bit >> 4) - p;
      if (idx >= 0 && idx < V) {                            // masked elements pass only a threshold of -inf
        const ValId c{__fadd_rn(row_at(rowp, idx), h.tokcb[idx]), idx};
        if (better(c, b)) { sec = fmaxf(sec, b.v); b = c; } else { sec = fmaxf(sec, c.v); }
      }
    } else {
      const int i = bit;
      const int idx0 = ((i >> 2) * 32 + lane) * 8 + (i & 3) * 2 - p;
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int idx = idx0 + hh;
        if (idx >= 0 && idx < V) {
          const float x = row_at(rowp, idx);
          if (x >= __bfloat162float(thr)) {
            const ValId c{__fadd_rn(x, h.tokcb[idx]), idx};
            if (better(c, b)) { sec = fmaxf(sec, b.v); b = c; } else { sec = fmaxf(sec, c.v); }
          }
        }
      }
    }
  }
  if (tail_ok && __hge(__ushort_as_bfloat16(static_cast<unsigned short>(tail_bits)), thr)) {
    const ValId c{__fadd_rn(bf16_bits_to_float(tail_bits), h.tokcb[tail_idx]), tail_idx};
    if (better(c, b)) { sec = fmaxf(sec, b.v); b = c; } else { sec = fmaxf(sec, c.v); }
  }
  // across the warp: best (value, lowest id) and the runner-up value
  const uint32_t key = fkey(b.v);
  const uint32_t kmax = __reduce_max_sync(0xffffffffu, key);
  const int idmin = static_cast<int>(__reduce_min_sync(0xffffffffu, key == kmax ? static_cast<uint32_t>(b.i) : 0x7FFFFFFFu));
  const bool mine = (key == kmax) && (b.i == idmin);
  const uint32_t k2 = __reduce_max_sync(0xffffffffu, fkey(mine ? sec : b.v));
  const bool ovf = idmin >= V;   // no candidate at all (cannot happen with finite logits)
  if (mine || (ovf && lane == 0)) {
    // tokens that are not candidates have x < thr, hence root-boosted value <= fl(thr + beta_max)
    const float ncb = __fadd_rn(__bfloat162float(thr), h.beta_max);
    const int id1 = ovf ? 0 : b.i;
    const int cl1 = h.cls16[id1];
    RowSummary r;
    r.y1 = b.v; r.y2b = fmaxf(fkey_inv(k2), ncb); r.xb = row_at(rowp, V); r.x1 = row_at(rowp, id1);
    r.rootcw1 = h.rootcw[cl1]; r.rootdst1 = h.rootdst[cl1];
    // same margin as the decider's, with the largest scale any state can have
    const float tau = (fabsf(r.y1) + 4.0f * h.bmag_max) * 1.9073486328125e-6f + 1e-30f;
    r.packed = static_cast<uint32_t>(id1) | (ovf ? kSumOvf : 0u) | ((r.y1 - r.y2b > tau) ? kSumGap : 0u);
    r.seq = seq;
    if (!ovf || lane == 0) {
      if constexpr (NORM) asm volatile("st.volatile.shared.f32 [%0], %1;" ::"r"(lse_a), "f"(lse) : "memory");
      // first half, fence, then the half that carries the sequence word
      sts_v4_volatile(out_a, make_uint4(__float_as_uint(r.y1), __float_as_uint(r.y2b), __float_as_uint(r.xb), __float_as_uint(r.x1)));
      __threadfence_block();
      sts_v4_volatile(out_a + 16u, make_uint4(__float_as_uint(r.rootcw1), static_cast<uint32_t>(r.rootdst1), r.packed, r.seq));
    }
  }
  __syncwarp();
}

// Both steps at once, for a row that sits in shared memory (every block readable).
template <int NIT, bool NORM = false>
__device__ __forceinline__ void summarize_row(const HelperCtx& h, const unsigned char* slot, int off_bytes,
                                              uint32_t out_a, uint32_t seq, int lane, uint32_t lse_a = 0u) {
  RowRegs<NIT> r;
  load_row<NIT>(h, slot, off_bytes, lane, nullptr, nullptr, r);
  finish_row<NIT, NORM>(h, r, slot + off_bytes, (off_bytes & 15) >> 1, out_a, seq, lane, lse_a);
}

// The tokens boosted by the non-root part of the suffix chain of the current state, as 8-byte
// entries {target state << 11 | token, lb} with lb = fl(lambda * fl(acc + w)).  Either a slice of
// the graph's resolved lists cached in shared memory (sorted by token id), or a list assembled in
// `lbuf`: copied from the resolved lists in the arena, or built by walking the chain (unsorted).
struct CurList {
  uint32_t addr;   // shared address of the first entry
  int n;
  bool sorted;
  float D, bmag;
};
constexpr uint32_t kTokMask = (1u << TB_RS_TOK_BITS) - 1u;   // low bits of an entry: 2 * token

struct Pick {
  ValId win;
  int next;
};

// Warp-wide best of per-lane (value, id, next): two integer reductions and a shuffle.
__device__ __forceinline__ Pick warp_pick(ValId v, int next) {
  const uint32_t key = fkey(v.v);
  const uint32_t kmax = __reduce_max_sync(0xffffffffu, key);
  const uint32_t idmin = __reduce_min_sync(0xffffffffu, key == kmax ? static_cast<uint32_t>(v.i) : 0xFFFFFFFFu);
  const unsigned who = __ballot_sync(0xffffffffu, key == kmax && static_cast<uint32_t>(v.i) == idmin);
  const int src = __ffs(who) - 1;
  Pick p;
  p.win.v = __shfl_sync(0xffffffffu, v.v, src);
  p.win.i = static_cast<int>(idmin);
  p.next = __shfl_sync(0xffffffffu, next, src);
  return p;
}

}  // namespace

#endif  // TB_FAST_COMMON_CUH_
