/*
 * tb_oracle.c -- CPU oracle for per-stream phrase boosting inside Transducer decoding.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the method
 * computes.  Nothing in the product (the CUDA library and its Python binding) includes,
 * links, imports or calls it; only the tests, the smoke check and the benchmark's
 * CPU-baseline leg do.  It shares no code, table or helper with the CUDA path.
 *
 * What it follows (paper sections):
 *   - Sec. 2.1 para. 1: a phrase list is a tree over tokenised phrases with suffix links;
 *     every matched token earns a shallow-fusion bonus.
 *   - Sec. 2.1 para. 2: case-insensitive matching by parallel arcs for the case variants
 *     of a symbol.  Here a token -> case-class map says which tokens are variants of one
 *     another; the tree is built over classes, so one arc stands for all its siblings.
 *   - Sec. 2.1 para. 6 (text above Eq. 1): states carry a cumulative score potential and
 *     an arc scores "destination potential minus source potential".  With one token per
 *     arc the Eq. 1 split is the trivial one (m_k = 1, Delta = w_k).
 *   - Sec. 2.2 para. 2: the compiled acceptor is a set of arc arrays (label, target state,
 *     weight) and state arrays (outgoing-arc range, suffix-link target, suffix-link weight,
 *     final weight).
 *   - Sec. 2.2 para. 3: model id -1 (here: a NULL graph) gives zero bonus and no valid next
 *     state (-1), so the stream decodes exactly as an unboosted one.
 *   - Sec. 2.3 and Sec. 3.4: greedy (label-looping) and beam decoding of Transducers, and
 *     streaming with state carried across chunk boundaries.  The paper only cites these
 *     decoders; the rules used here are spelled out at each function.
 *
 * Readings where the paper is silent are marked "READING" below.
 *
 * Parity pins: every function here is pinned by tests that do not use this file's own
 * formulas (brute-force substring matching, explicit case expansion, exhaustive beam
 * enumeration, library argmax).  Not pinned beyond reduced cases ("parity unpinned"):
 * beam decoding with K smaller than the number of alignments on large inputs, TDT with
 * durations that vary from row to row (pinned by a hand-worked case and by the reductions
 * "all durations 0 = the RNNT rule" and "all durations d = the unit case on every d-th
 * frame"), and the stream-churn schedule.  The order of equal beam candidates (value, token, parent) has a
 * hand-worked pin of its own; the normalised decode (orc_row_lse, orc_greedy_rnnt_lsm) is pinned against a
 * library log-sum-exp, closed forms, exact shifts of whole rows and the un-normalised decode.
 *
 * Arithmetic: potentials in double, each stored value rounded once to float; every
 * run-time sum is a float add in the order written, compiled with -ffp-contract=off so
 * that "x + lambda*bonus" is a rounded multiply followed by a rounded add.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_OK 0
#define ORC_ERR_INVALID_ARG (-1)
#define ORC_ERR_OOM (-2)

#define ORC_BF16 0
#define ORC_F32 1

typedef struct {
  int32_t n_states, n_arcs, n_classes, vocab, max_depth;
  float lambda;
  int32_t *state_arc_begin; /* [n_states+1] */
  int32_t *arc_class;       /* [n_arcs], ascending inside a state */
  int32_t *arc_dst;         /* [n_arcs] */
  float *arc_w;             /* [n_arcs] */
  int32_t *state_fail;      /* [n_states] */
  float *state_bw;          /* [n_states] suffix-link weight */
  float *state_final;       /* [n_states] */
  uint8_t *state_depth;     /* [n_states] */
  int32_t *case_class;      /* [vocab] */
} orc_graph;

/* ------------------------------------------------------------------------------------ */
/* Graph build (Sec. 2.1 para. 1-2, Sec. 2.1 para. 6, Sec. 2.2 para. 2).                  */
/* ------------------------------------------------------------------------------------ */

typedef struct {
  int32_t parent, cls, depth;
  int32_t first_child, next_sibling; /* unsorted child list */
  double wt;                         /* token weight of the arc entering this node */
  int is_end;                        /* a phrase ends here */
} trie_node;

static int32_t trie_child(const trie_node *n, int32_t u, int32_t c) {
  for (int32_t k = n[u].first_child; k >= 0; k = n[k].next_sibling)
    if (n[k].cls == c) return k;
  return -1;
}

typedef struct { int32_t cls, node; } child_ref;
static int cmp_child(const void *a, const void *b) {
  int32_t x = ((const child_ref *)a)->cls, y = ((const child_ref *)b)->cls;
  return (x > y) - (x < y);
}

void orc_graph_free(orc_graph *g) {
  if (!g) return;
  free(g->state_arc_begin); free(g->arc_class); free(g->arc_dst); free(g->arc_w);
  free(g->state_fail); free(g->state_bw); free(g->state_final); free(g->state_depth);
  free(g->case_class); free(g);
}

/*
 * phrase_tokens [sum of lengths], phrase_offsets [n_phrases+1], token_weights (NULL = 1.0)
 * one per phrase token, case_class [vocab] (NULL = identity: every token its own class).
 *
 * READING (potentials): the paper defines an arc score as a difference of potentials but
 * not what becomes of the credit once a phrase is complete.  Here credit for a partial
 * match is "on loan" (taken back through the suffix link if the match breaks) and is
 * "banked" for good when a phrase ends:
 *   loan(root) = 0;  loan(n) = is_end(n) ? 0 : loan(parent(n)) + wt(n)
 *   bank(n)    = is_end(n) ? loan(parent(n)) + wt(n) : 0
 *   out(n)     = bank(n) + out(fail(n)),  out(root) = 0   (all phrases completed on arrival)
 *   arc_w(u->d) = loan(d) - loan(u) + out(d)
 *   bw(u)       = loan(fail(u)) - loan(u),  bw(root) = 0
 *   final(u)    = -loan(u)
 * READING (shared prefixes, duplicates): a node's weight is the largest weight any phrase
 * gives that position; phrases equal after case folding are one phrase.
 * READING (numbering): states are numbered breadth-first from root = 0, the children of a
 * node in ascending class order, so two correct compilers emit identical arrays.
 */
int orc_graph_build(const int32_t *phrase_tokens, const int64_t *phrase_offsets, int32_t n_phrases,
                    const float *token_weights, const int32_t *case_class, int32_t vocab,
                    float lambda, orc_graph **out) {
  if (!out || vocab <= 0 || n_phrases < 0 || (n_phrases > 0 && (!phrase_tokens || !phrase_offsets)))
    return ORC_ERR_INVALID_ARG;
  if (!(lambda == lambda) || isinf(lambda)) return ORC_ERR_INVALID_ARG;
  *out = NULL;
  int32_t n_classes = 0;
  if (case_class) {
    for (int32_t v = 0; v < vocab; ++v) {
      if (case_class[v] < 0) return ORC_ERR_INVALID_ARG;
      if (case_class[v] + 1 > n_classes) n_classes = case_class[v] + 1;
    }
  } else {
    n_classes = vocab;
  }
  int64_t total = n_phrases > 0 ? phrase_offsets[n_phrases] : 0;
  if (n_phrases > 0 && phrase_offsets[0] != 0) return ORC_ERR_INVALID_ARG;
  for (int32_t p = 0; p < n_phrases; ++p)
    if (phrase_offsets[p + 1] < phrase_offsets[p]) return ORC_ERR_INVALID_ARG;
  for (int64_t i = 0; i < total; ++i) {
    if (phrase_tokens[i] < 0 || phrase_tokens[i] >= vocab) return ORC_ERR_INVALID_ARG;
    if (token_weights) {
      float w = token_weights[i];
      if (!(w == w) || isinf(w) || w < 0.0f) return ORC_ERR_INVALID_ARG;
    }
  }

  /* 1-2. tree over class sequences */
  int64_t cap = total + 1;
  trie_node *n = (trie_node *)malloc((size_t)cap * sizeof(trie_node));
  if (!n) return ORC_ERR_OOM;
  int32_t N = 1;
  n[0].parent = -1; n[0].cls = -1; n[0].depth = 0; n[0].first_child = -1;
  n[0].next_sibling = -1; n[0].wt = 0.0; n[0].is_end = 0;
  int32_t max_depth = 0;
  for (int32_t p = 0; p < n_phrases; ++p) {
    int64_t b = phrase_offsets[p], e = phrase_offsets[p + 1];
    if (e == b) continue; /* empty phrase: skipped */
    if (e - b > 255) { free(n); return ORC_ERR_INVALID_ARG; } /* depth is stored in a byte */
    int32_t u = 0;
    for (int64_t i = b; i < e; ++i) {
      int32_t tok = phrase_tokens[i];
      int32_t c = case_class ? case_class[tok] : tok;
      double w = token_weights ? (double)token_weights[i] : 1.0;
      int32_t k = trie_child(n, u, c);
      if (k < 0) {
        k = N++;
        n[k].parent = u; n[k].cls = c; n[k].depth = n[u].depth + 1; n[k].first_child = -1;
        n[k].next_sibling = n[u].first_child; n[u].first_child = k;
        n[k].wt = w; n[k].is_end = 0;
        if (n[k].depth > max_depth) max_depth = n[k].depth;
      } else if (w > n[k].wt) {
        n[k].wt = w;
      }
      u = k;
    }
    n[u].is_end = 1;
  }

  /* 3. canonical numbering: breadth-first, children by ascending class */
  int32_t *order = (int32_t *)malloc((size_t)N * sizeof(int32_t));   /* new id -> old node */
  int32_t *newid = (int32_t *)malloc((size_t)N * sizeof(int32_t));   /* old node -> new id */
  child_ref *tmp = (child_ref *)malloc((size_t)(n_classes > 0 ? n_classes : 1) * sizeof(child_ref));
  orc_graph *g = (orc_graph *)calloc(1, sizeof(orc_graph));
  if (!order || !newid || !tmp || !g) { free(n); free(order); free(newid); free(tmp); free(g); return ORC_ERR_OOM; }
  int32_t A = N - 1;
  g->n_states = N; g->n_arcs = A; g->n_classes = n_classes; g->vocab = vocab;
  g->max_depth = max_depth; g->lambda = lambda;
  g->state_arc_begin = (int32_t *)calloc((size_t)N + 1, sizeof(int32_t));
  g->arc_class = (int32_t *)calloc((size_t)(A > 0 ? A : 1), sizeof(int32_t));
  g->arc_dst = (int32_t *)calloc((size_t)(A > 0 ? A : 1), sizeof(int32_t));
  g->arc_w = (float *)calloc((size_t)(A > 0 ? A : 1), sizeof(float));
  g->state_fail = (int32_t *)calloc((size_t)N, sizeof(int32_t));
  g->state_bw = (float *)calloc((size_t)N, sizeof(float));
  g->state_final = (float *)calloc((size_t)N, sizeof(float));
  g->state_depth = (uint8_t *)calloc((size_t)N, 1);
  g->case_class = (int32_t *)malloc((size_t)vocab * sizeof(int32_t));
  double *loan = (double *)calloc((size_t)N, sizeof(double));
  double *bank = (double *)calloc((size_t)N, sizeof(double));
  double *outp = (double *)calloc((size_t)N, sizeof(double));
  if (!g->state_arc_begin || !g->arc_class || !g->arc_dst || !g->arc_w || !g->state_fail ||
      !g->state_bw || !g->state_final || !g->state_depth || !g->case_class || !loan || !bank || !outp) {
    free(n); free(order); free(newid); free(tmp); free(loan); free(bank); free(outp);
    orc_graph_free(g); return ORC_ERR_OOM;
  }
  for (int32_t v = 0; v < vocab; ++v) g->case_class[v] = case_class ? case_class[v] : v;

  int32_t head = 0, tail = 0, arc = 0;
  order[tail] = 0; newid[0] = 0; tail++;
  while (head < tail) {
    int32_t id = head, u = order[head++];
    int32_t nc = 0;
    for (int32_t k = n[u].first_child; k >= 0; k = n[k].next_sibling) { tmp[nc].cls = n[k].cls; tmp[nc].node = k; nc++; }
    qsort(tmp, (size_t)nc, sizeof(child_ref), cmp_child);
    g->state_arc_begin[id] = arc;
    for (int32_t j = 0; j < nc; ++j) {
      newid[tmp[j].node] = tail; order[tail] = tmp[j].node;
      g->arc_class[arc] = tmp[j].cls; g->arc_dst[arc] = tail;
      arc++; tail++;
    }
  }
  g->state_arc_begin[N] = arc;

  /* 4. suffix links: fail(n) = longest proper suffix of path(n) that is a tree path.
   * Processed in id order (breadth-first), so fail(parent) is ready when n is reached. */
  for (int32_t id = 1; id < N; ++id) {
    int32_t u = order[id], p = n[u].parent, c = n[u].cls;
    int32_t f = 0;
    if (p != 0) {
      int32_t q = order[g->state_fail[newid[p]]]; /* old node of fail(parent) */
      for (;;) {
        int32_t k = trie_child(n, q, c);
        if (k >= 0) { f = newid[k]; break; }
        if (q == 0) { f = 0; break; }
        q = order[g->state_fail[newid[q]]];
      }
    }
    g->state_fail[id] = f;
  }

  /* 5. potentials in double (id order: parent and fail have smaller ids) */
  for (int32_t id = 1; id < N; ++id) {
    int32_t u = order[id];
    int32_t pid = newid[n[u].parent];
    double through = loan[pid] + n[u].wt;
    if (n[u].is_end) { loan[id] = 0.0; bank[id] = through; } else { loan[id] = through; bank[id] = 0.0; }
    outp[id] = bank[id] + outp[g->state_fail[id]];
  }

  /* 6. stored values, each rounded once from double */
  for (int32_t id = 0; id < N; ++id) {
    int32_t u = order[id];
    g->state_depth[id] = (uint8_t)n[u].depth;
    g->state_final[id] = (float)(-loan[id]);
    g->state_bw[id] = id == 0 ? 0.0f : (float)(loan[g->state_fail[id]] - loan[id]);
    for (int32_t a = g->state_arc_begin[id]; a < g->state_arc_begin[id + 1]; ++a) {
      int32_t d = g->arc_dst[a];
      g->arc_w[a] = (float)(loan[d] - loan[id] + outp[d]);
    }
  }
  free(n); free(order); free(newid); free(tmp); free(loan); free(bank); free(outp);
  *out = g;
  return ORC_OK;
}

/* Copies the struct of pointers so that a caller can read the arrays. */
void orc_graph_get(const orc_graph *g, orc_graph *view) { *view = *g; }

/* ------------------------------------------------------------------------------------ */
/* One boosting step (Sec. 2.2 para. 3: "suffix-link traversal").                        */
/* ------------------------------------------------------------------------------------ */

static int32_t find_arc(const orc_graph *g, int32_t u, int32_t c) {
  for (int32_t a = g->state_arc_begin[u]; a < g->state_arc_begin[u + 1]; ++a)
    if (g->arc_class[a] == c) return a;
  return -1;
}

/*
 * Non-blank token v in state s: walk the suffix links from s; the first state with an arc
 * on v's class ends the walk.  bonus = suffix-link weights crossed + that arc's weight;
 * next = the arc's target.  No arc anywhere: bonus = the crossed weights, next = root.
 * READING: a token the list does not know costs nothing beyond the refunded loan.
 * A NULL graph (model id -1) gives bonus 0 and next state -1.
 */
void orc_step(const orc_graph *g, int32_t s, int32_t v, float *bonus, int32_t *next) {
  if (!g) { *bonus = 0.0f; *next = -1; return; }
  int32_t c = g->case_class[v];
  float acc = 0.0f;
  int32_t u = s;
  for (;;) {
    int32_t a = find_arc(g, u, c);
    if (a >= 0) { *bonus = acc + g->arc_w[a]; *next = g->arc_dst[a]; return; }
    if (u == 0) { *bonus = acc; *next = 0; return; }
    acc = acc + g->state_bw[u];
    u = g->state_fail[u];
  }
}

/*
 * End of stream (Sec. 2.2 para. 2 lists a final weight per state): a hypothesis that stops in
 * state s is charged that state's final weight, score' = score + lambda * final(s), a rounded
 * multiply and a rounded add like every other bonus.  final(s) = -loan(s): what a partial match
 * had been lent is returned, so that a finished hypothesis keeps the bonus of the phrases it
 * completed and nothing else.  READING: the paper names the tensor only; this is the one use
 * that makes its value (the loan, negated) meaningful.  A NULL graph or state -1 changes nothing.
 */
float orc_apply_final_weight(const orc_graph *g, int32_t s, float score) {
  if (!g || s < 0) return score;
  float lam_f = g->lambda * g->state_final[s];
  return score + lam_f;
}

/* ------------------------------------------------------------------------------------ */
/* Logit access and the boosted value of one candidate.                                  */
/* ------------------------------------------------------------------------------------ */

static float logit_at(const void *base, int dtype, int64_t idx) {
  if (dtype == ORC_F32) return ((const float *)base)[idx];
  uint32_t bits = (uint32_t)((const uint16_t *)base)[idx] << 16; /* bf16 -> float is exact */
  float f;
  memcpy(&f, &bits, sizeof f);
  return f;
}

/*
 * val(v) = x[v] + lambda * bonus(s, v) for a non-blank token of a bound stream: one rounded
 * multiply, then one rounded add.  Blank (id V) and unbound streams use x itself
 * (READING: blank earns nothing and leaves the state alone).
 */
static float boosted(const orc_graph *g, int32_t s, int32_t v, int32_t V, float x, int32_t *next) {
  if (!g) { *next = -1; return x; }
  if (v == V) { *next = s; return x; }
  float b;
  orc_step(g, s, v, &b, next);
  float lam_b = g->lambda * b;
  return x + lam_b;
}

/* argmax over one row's V+1 candidates; ties go to the lowest token id (READING). */
static int32_t select_row(const orc_graph *g, int32_t s, const void *logits, int dtype, int64_t row,
                          int64_t stride_v, int32_t V, float *best_val, int32_t *best_next) {
  int32_t best = -1, nx = -1;
  float bv = 0.0f;
  for (int32_t v = 0; v <= V; ++v) {
    int32_t nv;
    float val = boosted(g, s, v, V, logit_at(logits, dtype, row + v * stride_v), &nv);
    if (best < 0 || val > bv) { best = v; bv = val; nx = nv; }
  }
  *best_val = bv; *best_next = nx;
  return best;
}

/* ------------------------------------------------------------------------------------ */
/* Greedy RNNT for one stream (Sec. 3.4: greedy label-looping decoding).                  */
/* ------------------------------------------------------------------------------------ */

/*
 * logits: [T, S, V+1] with element strides {stride_t, stride_s, stride_v}; row k of frame t is
 * the joint output after k symbols were emitted in that frame.  Rules (READING: the paper
 * cites the decoder only): start at t = 0, k = 0; pick the argmax of the boosted row; blank
 * closes the frame; a non-blank token is emitted at frame t, advances the graph state and
 * moves to row k+1; after S symbols the frame closes by force, adding nothing to the score.
 * Returns the number of emitted tokens.
 */
int64_t orc_greedy_rnnt(const orc_graph *g, const void *logits, int dtype, int32_t T, int32_t S,
                        int32_t V, const int64_t *strides, int32_t len, int32_t *out_tokens,
                        int32_t *out_frames, float *out_score, int32_t *out_state) {
  int32_t s = g ? 0 : -1, t = 0, k = 0;
  float score = 0.0f;
  int64_t n = 0;
  if (len > T) len = T;
  while (t < len) {
    int64_t row = (int64_t)t * strides[0] + (int64_t)k * strides[1];
    float val; int32_t nx;
    int32_t tok = select_row(g, s, logits, dtype, row, strides[2], V, &val, &nx);
    score = score + val;
    if (tok == V) { t++; k = 0; }
    else {
      out_tokens[n] = tok; out_frames[n] = t; n++;
      s = nx; k++;
      if (k == S) { t++; k = 0; }
    }
  }
  *out_score = score; *out_state = s;
  return n;
}

/* ------------------------------------------------------------------------------------ */
/* Greedy RNNT on normalised scores: log-softmax fused into the selection                  */
/* (Sec. 2.2 para. 3 speaks of one fused scoring operation; READING: the paper does not say  */
/* whether the joint output is normalised before the bonus is added -- this variant does it). */
/* ------------------------------------------------------------------------------------ */

/* log sum exp of the V+1 entries of one row, in double: L = m + log(sum_v exp(x_v - m)), m = max_v x_v. */
double orc_row_lse(const void *logits, int dtype, int64_t row, int64_t stride_v, int32_t V) {
  double m = -INFINITY;
  for (int32_t v = 0; v <= V; ++v) {
    double x = (double)logit_at(logits, dtype, row + v * stride_v);
    if (x > m) m = x;
  }
  if (m == -INFINITY) return -INFINITY;
  double sum = 0.0;
  for (int32_t v = 0; v <= V; ++v) sum += exp((double)logit_at(logits, dtype, row + v * stride_v) - m);
  return m + log(sum);
}

/*
 * As orc_greedy_rnnt, on val(v) = (x_v - L(row)) + lambda * bonus(s, v), everything after the float bonus
 * term in double: the bonus term is the float product fl(lambda * bonus) of the un-normalised decode, the
 * normalised logit x_v - L and the sum are double, the score is a double sum.  L is the same for every entry of
 * a row, so in exact arithmetic the selected tokens are those of the un-normalised decode and the score is lower
 * by the sum of L over the visited rows.
 *
 * follow_tokens / follow_frames (n_follow >= 0): another decoder's output to be checked against this one.  At
 * every visited row the other decoder's action there (its next token if that token's frame is the current frame,
 * else blank) is compared with this decoder's choice; where they differ and the two values are closer than eps
 * the other decoder's action is taken (and counted in *n_followed), so that one near-tie does not make the rest
 * of the stream incomparable; where they differ by eps or more the decode stops and *first_mismatch receives the
 * index of the visited row (else -1).  n_follow < 0: a free decode.
 */
int64_t orc_greedy_rnnt_lsm(const orc_graph *g, const void *logits, int dtype, int32_t T, int32_t S, int32_t V,
                            const int64_t *strides, int32_t len, const int32_t *follow_tokens,
                            const int32_t *follow_frames, int64_t n_follow, double eps, int32_t *out_tokens,
                            int32_t *out_frames, double *out_score, int32_t *out_state, int64_t *n_followed,
                            int64_t *first_mismatch, int64_t *rows_visited) {
  int32_t s = g ? 0 : -1, t = 0, k = 0;
  double score = 0.0;
  int64_t n = 0, rows = 0, followed = 0;
  if (first_mismatch) *first_mismatch = -1;
  if (len > T) len = T;
  while (t < len) {
    int64_t row = (int64_t)t * strides[0] + (int64_t)k * strides[1];
    double L = orc_row_lse(logits, dtype, row, strides[2], V);
    int32_t best = -1, best_next = -1;
    double bv = 0.0;
    for (int32_t v = 0; v <= V; ++v) {
      float x = logit_at(logits, dtype, row + v * strides[2]);
      int32_t nv;
      float lam_b = boosted(g, s, v, V, 0.0f, &nv);          /* fl(0 + fl(lambda * bonus)): the float bonus term alone */
      double val = ((double)x - L) + (double)lam_b;
      if (best < 0 || val > bv) { best = v; bv = val; best_next = nv; }
    }
    int32_t tok = best, nx = best_next;
    double val = bv;
    if (n_follow >= 0) {
      int32_t want = (n < n_follow && follow_frames[n] == t) ? follow_tokens[n] : V;
      if (want < 0 || want > V) want = V;
      if (want != best) {
        float xw = logit_at(logits, dtype, row + want * strides[2]);
        int32_t nw;
        float lam_w = boosted(g, s, want, V, 0.0f, &nw);
        double vw = ((double)xw - L) + (double)lam_w;
        if (bv - vw < eps) { tok = want; nx = nw; val = vw; followed++; }
        else { if (first_mismatch) *first_mismatch = rows; break; }
      }
    }
    rows++;
    score += val;
    if (tok == V) { t++; k = 0; }
    else {
      out_tokens[n] = tok; out_frames[n] = t; n++;
      s = nx; k++;
      if (k == S) { t++; k = 0; }
    }
  }
  *out_score = score; *out_state = s;
  if (n_followed) *n_followed = followed;
  if (rows_visited) *rows_visited = rows;
  return n;
}

/* ------------------------------------------------------------------------------------ */
/* Streaming greedy, RNNT or TDT, one slot, one chunk (Sec. 2.3: state kept across chunks) */
/* ------------------------------------------------------------------------------------ */

typedef struct {
  int32_t state;  /* graph state, -1 when unbound */
  int32_t t;      /* global frame cursor */
  int32_t k;      /* symbols already emitted in frame t */
  float score;
  int32_t n_emitted;
} orc_stream_state;

/*
 * logits: [chunk, S, V+1+n_dur]; the chunk covers global frames [t0, t0+chunk); frames at or
 * beyond valid_frames (the stream's total length so far) are not decoded.  n_dur = 0: the
 * RNNT rules above.  n_dur > 0 (TDT; READING, the paper only cites it): the row carries
 * n_dur duration logits after the V+1 token logits, for durations 0..n_dur-1; the duration
 * is their argmax (lowest index on ties); score += val[token] + x_dur[duration];
 * blank: t += max(duration, 1), k = 0; non-blank: emit, advance the state, then
 * duration > 0 ? (t += duration, k = 0) : (k++, and k == S closes the frame).
 * A cursor beyond the chunk end is carried to the next chunk.  Returns tokens emitted.
 */
int64_t orc_stream_chunk(const orc_graph *g, const void *logits, int dtype, int32_t chunk, int32_t S,
                         int32_t V, int32_t n_dur, const int64_t *strides, int32_t t0,
                         int32_t valid_frames, orc_stream_state *st, int32_t *out_tokens,
                         int32_t *out_frames, int32_t *out_durs) {
  int64_t n = 0;
  int32_t end = t0 + chunk;
  if (valid_frames < end) end = valid_frames;
  while (st->t < end) {
    int64_t row = (int64_t)(st->t - t0) * strides[0] + (int64_t)st->k * strides[1];
    float val; int32_t nx;
    int32_t tok = select_row(g, st->state, logits, dtype, row, strides[2], V, &val, &nx);
    int32_t dur = 0;
    if (n_dur > 0) {
      float bd = 0.0f;
      for (int32_t d = 0; d < n_dur; ++d) {
        float xd = logit_at(logits, dtype, row + (int64_t)(V + 1 + d) * strides[2]);
        if (d == 0 || xd > bd) { bd = xd; dur = d; }
      }
      st->score = st->score + (val + bd);
    } else {
      st->score = st->score + val;
    }
    if (tok == V) {
      int32_t adv = n_dur > 0 ? (dur > 1 ? dur : 1) : 1;
      st->t += adv; st->k = 0;
    } else {
      out_tokens[n] = tok; out_frames[n] = st->t; if (out_durs) out_durs[n] = dur; n++;
      st->n_emitted++;
      st->state = nx;
      if (n_dur > 0 && dur > 0) { st->t += dur; st->k = 0; }
      else { st->k++; if (st->k == S) { st->t++; st->k = 0; } }
    }
  }
  return n;
}

/* ------------------------------------------------------------------------------------ */
/* Beam step and the frame-synchronous driver (Sec. 2.3, Sec. 3.4: beam search).          */
/* ------------------------------------------------------------------------------------ */

/*
 * One expansion for one stream.  In: K hypotheses {score (-inf = empty slot), state, live}.
 * rows[k] is the element offset of hypothesis k's logit row.  Candidates: every live,
 * non-empty k with every token v in 0..V scores fl(score_k + val_k(v)) (val first, then the
 * add); every frozen non-empty k is carried as one candidate with its score and token -1.
 * The K best are taken in the order (score descending, token key ascending with the carried
 * candidate's key = V+1, parent ascending) (READING).  Out slot j: parent, token, score;
 * state = token non-blank ? next(state_parent, token) : state_parent;
 * live = live_parent and token non-blank and token carried != -1.  Unfilled slots: score -inf,
 * parent -1, token -1, state -1, live 0.
 */
void orc_beam_step(const orc_graph *g, const void *logits, int dtype, const int64_t *rows,
                   int64_t stride_v, int32_t K, int32_t V, float *scores, int32_t *states,
                   uint8_t *live, int32_t *out_parent, int32_t *out_token) {
  float *ns = (float *)malloc((size_t)K * sizeof(float));
  int32_t *nst = (int32_t *)malloc((size_t)K * sizeof(int32_t));
  uint8_t *nl = (uint8_t *)malloc((size_t)K);
  int32_t *key = (int32_t *)malloc((size_t)K * sizeof(int32_t));
  int32_t filled = 0;
  /* selection by insertion into a sorted list of at most K entries */
  for (int32_t k = 0; k < K; ++k) {
    if (scores[k] == -INFINITY) continue;
    int32_t v_lo = live[k] ? 0 : -1, v_hi = live[k] ? V : -1;
    for (int32_t v = v_lo; v <= v_hi; ++v) {
      float cand; int32_t nx; int32_t tkey;
      if (v < 0) { cand = scores[k]; nx = states[k]; tkey = V + 1; }
      else {
        float val = boosted(g, states[k], v, V, logit_at(logits, dtype, rows[k] + v * stride_v), &nx);
        cand = scores[k] + val; tkey = v;
      }
      /* position: first slot j such that the candidate comes strictly before entry j */
      int32_t pos = filled;
      for (int32_t j = 0; j < filled; ++j) {
        int before = cand > ns[j] || (cand == ns[j] && (tkey < key[j] || (tkey == key[j] && k < out_parent[j])));
        if (before) { pos = j; break; }
      }
      if (pos >= K) continue;
      int32_t last = filled < K ? filled : K - 1;
      for (int32_t j = last; j > pos; --j) {
        ns[j] = ns[j - 1]; nst[j] = nst[j - 1]; nl[j] = nl[j - 1]; key[j] = key[j - 1];
        out_parent[j] = out_parent[j - 1]; out_token[j] = out_token[j - 1];
      }
      ns[pos] = cand; nst[pos] = nx; key[pos] = tkey; out_parent[pos] = k; out_token[pos] = v;
      nl[pos] = (uint8_t)(v >= 0 && v != V && live[k]);
      if (filled < K) filled++;
    }
  }
  for (int32_t j = 0; j < K; ++j) {
    if (j < filled) { scores[j] = ns[j]; states[j] = nst[j]; live[j] = nl[j]; }
    else { scores[j] = -INFINITY; states[j] = -1; live[j] = 0; out_parent[j] = -1; out_token[j] = -1; }
  }
  free(ns); free(nst); free(nl); free(key);
}

/*
 * Frame-synchronous driver (READING: the paper's beam algorithm is cited, not described):
 * logits [T, E, V+1]; hypothesis 0 starts as {0, root, live}, the rest empty; at each frame
 * every non-empty hypothesis becomes live, then E steps follow, all hypotheses reading row
 * (t, e); after row E-1 the frame closes by force.  Every step appends K (parent, token)
 * pairs to tree [T*E, K, 2].  Results per final slot j: token sequence (backtrace, carried
 * candidates skipped, blanks dropped) in out_tokens[j*max_len ...], its length, score, state.
 */
/*
 * merge != 0 (Sec. 2.3: stored hypotheses are anchors for continuing, merging and pruning): at the start of
 * every frame, hypotheses that have emitted the same token sequence are one transcript reached by different
 * alignments; the best of them (the first in selection order) is kept, the others become empty places.
 * READING: merging happens where the hypotheses are in the same situation -- all live, at a frame start -- so
 * that equal sequences have equal futures and keeping the best loses nothing (the result is, per token
 * sequence, the best alignment, as long as the beam is wide enough).
 * prune_delta >= 0 (Sec. 2.3: ... and pruning): after the merge, still at the frame start, every hypothesis
 * whose score is below (best score - prune_delta), one rounded subtraction, becomes an empty place.
 * READING: the paper names pruning only; a threshold relative to the best hypothesis is the usual rule.
 * A negative prune_delta switches it off.
 */
int orc_beam_decode_opts(const orc_graph *g, const void *logits, int dtype, int32_t T, int32_t E, int32_t V,
                         const int64_t *strides, int32_t K, int32_t max_len, int32_t merge, float prune_delta,
                         int32_t *out_tokens, int32_t *out_lens, float *out_scores, int32_t *out_states,
                         int32_t *tree) {
  float *scores = (float *)malloc((size_t)K * sizeof(float));
  int32_t *states = (int32_t *)malloc((size_t)K * sizeof(int32_t));
  uint8_t *live = (uint8_t *)malloc((size_t)K);
  int64_t *rows = (int64_t *)malloc((size_t)K * sizeof(int64_t));
  int32_t *par = (int32_t *)malloc((size_t)K * sizeof(int32_t));
  int32_t *tok = (int32_t *)malloc((size_t)K * sizeof(int32_t));
  int32_t *rev = (int32_t *)malloc((size_t)T * E * sizeof(int32_t) + 4);
  for (int32_t k = 0; k < K; ++k) { scores[k] = -INFINITY; states[k] = -1; live[k] = 0; }
  scores[0] = 0.0f; states[0] = g ? 0 : -1; live[0] = 1;
  int64_t step = 0;
  /* the token sequence of every hypothesis, kept explicitly for the merge */
  const int64_t cap = (int64_t)T * E + 1;
  int32_t *seq = (int32_t *)malloc((size_t)K * cap * sizeof(int32_t));
  int32_t *seq2 = (int32_t *)malloc((size_t)K * cap * sizeof(int32_t));
  int32_t *len = (int32_t *)calloc((size_t)K, sizeof(int32_t));
  int32_t *len2 = (int32_t *)calloc((size_t)K, sizeof(int32_t));
  for (int32_t t = 0; t < T; ++t) {
    if (merge) {
      for (int32_t k = 1; k < K; ++k) {
        if (scores[k] == -INFINITY) continue;
        for (int32_t j = 0; j < k; ++j) {
          if (scores[j] == -INFINITY || len[j] != len[k]) continue;
          if (memcmp(seq + j * cap, seq + k * cap, (size_t)len[k] * sizeof(int32_t)) != 0) continue;
          scores[k] = -INFINITY; states[k] = -1; live[k] = 0;
          break;
        }
      }
    }
    if (prune_delta >= 0.0f) {
      float best = -INFINITY;
      for (int32_t k = 0; k < K; ++k) if (scores[k] > best) best = scores[k];
      float floor_ = best - prune_delta;
      for (int32_t k = 0; k < K; ++k)
        if (scores[k] != -INFINITY && scores[k] < floor_) { scores[k] = -INFINITY; states[k] = -1; live[k] = 0; }
    }
    for (int32_t k = 0; k < K; ++k) live[k] = (uint8_t)(scores[k] != -INFINITY);
    for (int32_t e = 0; e < E; ++e, ++step) {
      for (int32_t k = 0; k < K; ++k) rows[k] = (int64_t)t * strides[0] + (int64_t)e * strides[1];
      orc_beam_step(g, logits, dtype, rows, strides[2], K, V, scores, states, live, par, tok);
      for (int32_t k = 0; k < K; ++k) { tree[(step * K + k) * 2] = par[k]; tree[(step * K + k) * 2 + 1] = tok[k]; }
      for (int32_t k = 0; k < K; ++k) {
        len2[k] = 0;
        if (par[k] < 0) continue;
        memcpy(seq2 + k * cap, seq + par[k] * cap, (size_t)len[par[k]] * sizeof(int32_t));
        len2[k] = len[par[k]];
        if (tok[k] >= 0 && tok[k] != V) seq2[k * cap + len2[k]++] = tok[k];
      }
      { int32_t *sw = seq; seq = seq2; seq2 = sw; sw = len; len = len2; len2 = sw; }
    }
  }
  free(seq); free(seq2); free(len); free(len2);
  for (int32_t j = 0; j < K; ++j) {
    out_scores[j] = scores[j]; out_states[j] = states[j];
    int32_t n = 0, slot = j;
    if (scores[j] != -INFINITY) {
      for (int64_t st = step - 1; st >= 0 && slot >= 0; --st) {
        int32_t p = tree[(st * K + slot) * 2], tk = tree[(st * K + slot) * 2 + 1];
        if (tk >= 0 && tk != V) rev[n++] = tk;
        slot = p;
      }
    }
    int32_t m = n < max_len ? n : max_len;
    for (int32_t i = 0; i < m; ++i) out_tokens[(int64_t)j * max_len + i] = rev[n - 1 - i];
    out_lens[j] = n;
  }
  free(scores); free(states); free(live); free(rows); free(par); free(tok); free(rev);
  return ORC_OK;
}

int orc_beam_decode(const orc_graph *g, const void *logits, int dtype, int32_t T, int32_t E, int32_t V,
                    const int64_t *strides, int32_t K, int32_t max_len, int32_t *out_tokens,
                    int32_t *out_lens, float *out_scores, int32_t *out_states, int32_t *tree) {
  return orc_beam_decode_opts(g, logits, dtype, T, E, V, strides, K, max_len, 0, -1.0f, out_tokens, out_lens,
                              out_scores, out_states, tree);
}
