"""Pins for the CPU oracle: each test checks the oracle against something that is not the oracle --
a hand-derived worked example, brute-force substring matching, explicit case expansion, numpy's
argmax, exhaustive enumeration of alignments -- so that a dropped term, a wrong sign or index or a
transposed operand in the oracle fails at least one of them.  None of these tests needs a GPU.

The brute-force definitions used here (no tree, no suffix links):
  * a phrase list is a set of class sequences; wt(prefix) is the largest weight any phrase gives
    that position;
  * loan(q), q a phrase prefix: the weights of q's positions after its longest prefix (q included)
    that is a complete phrase;  bank(p), p a phrase: the weights after its longest *proper* prefix
    that is a complete phrase;
  * G(h) = sum over every occurrence of a phrase as a (class-wise) substring of h of bank(p),
    plus loan of the longest suffix of h that is a phrase prefix.
The method's per-token bonus must be G(h.v) - G(h) and its state that longest suffix
(Sec. 2.1: every matched token is rewarded, arc score = potential difference).
"""
import itertools
import os

import numpy as np
import pytest

from oracle import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------------------------------------
# brute-force definitions
# ---------------------------------------------------------------------------------------------

class Brute:
    def __init__(self, phrases, case_class=None, weights=None):
        fold = (lambda t: t) if case_class is None else (lambda t: int(case_class[t]))
        self.fold = fold
        self.ends = set()
        self.wt = {}
        for i, p in enumerate(phrases):
            if not p:
                continue
            cp = tuple(fold(t) for t in p)
            self.ends.add(cp)
            for j in range(len(cp)):
                w = 1.0 if weights is None else float(weights[i][j])
                self.wt[cp[:j + 1]] = max(self.wt.get(cp[:j + 1], 0.0), w)
        self.maxlen = max((len(p) for p in self.ends), default=0)

    def _since_last_end(self, q, proper):
        last = 0
        top = len(q) - 1 if proper else len(q)
        for j in range(1, top + 1):
            if q[:j] in self.ends:
                last = j
        return sum(self.wt[q[:j + 1]] for j in range(last, len(q)))

    def loan(self, q):
        return self._since_last_end(q, proper=False) if q else 0.0

    def bank(self, p):
        return self._since_last_end(p, proper=True)

    def state_path(self, h):
        """Longest suffix of h (class sequence) that is a phrase prefix."""
        for L in range(min(len(h), self.maxlen), 0, -1):
            if tuple(h[-L:]) in self.wt:
                return tuple(h[-L:])
        return ()

    def G(self, toks):
        h = tuple(self.fold(t) for t in toks)
        total = 0.0
        for i in range(1, len(h) + 1):
            for L in range(1, min(i, self.maxlen) + 1):
                if h[i - L:i] in self.ends:
                    total += self.bank(h[i - L:i])
        return total + self.loan(self.state_path(h))


def state_paths(g):
    """Class path of every state, rebuilt from the arrays alone."""
    paths = {0: ()}
    for s in range(g.n_states):
        for a in range(g.state_arc_begin[s], g.state_arc_begin[s + 1]):
            paths[int(g.arc_dst[a])] = paths[s] + (int(g.arc_class[a]),)
    return paths


def random_list(rng, V, n, maxlen, dyadic_weights=False):
    phrases = [[int(t) for t in rng.integers(0, V, size=rng.integers(1, maxlen + 1))] for _ in range(n)]
    weights = None
    if dyadic_weights:
        weights = [[float(rng.choice([0.5, 1.0, 1.5, 2.0])) for _ in p] for p in phrases]
    return phrases, weights


# ---------------------------------------------------------------------------------------------
# worked example, derived by hand
# ---------------------------------------------------------------------------------------------

def _read_golden(name):
    rows, steps = {}, []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            if key == "step":
                steps.append([float(v) for v in vals])
            else:
                rows[key] = [float(v) for v in vals]
    return rows, steps


def test_hand_derived_example():
    rows, steps = _read_golden("worked_example_nested.txt")
    g = O.Graph([[0, 1], [0, 1, 2, 3], [1, 2]], vocab=4)
    assert g.n_states == rows["n_states"][0] and g.n_arcs == rows["n_arcs"][0]
    assert g.max_depth == rows["max_depth"][0]
    for key in ("state_arc_begin", "arc_class", "arc_dst", "arc_w", "state_fail", "state_bw",
                "state_final", "state_depth"):
        assert list(map(float, getattr(g, key))) == rows[key], key
    for s, v, bonus, nxt in steps:
        assert g.step(int(s), int(v)) == (bonus, int(nxt))


# ---------------------------------------------------------------------------------------------
# P1: the walk equals direct substring matching, for every history
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("seed", range(24))
def test_walk_equals_substring_matching(seed):
    rng = np.random.default_rng(seed)
    V = int(rng.integers(2, 6))
    depth = 6 if V <= 3 else 5
    phrases, weights = random_list(rng, V, int(rng.integers(1, 7)), 4, dyadic_weights=seed % 2 == 1)
    g = O.Graph(phrases, V, weights=weights)
    br = Brute(phrases, None, weights)
    paths = state_paths(g)
    assert len(paths) == g.n_states

    def rec(h, s, Gh):
        assert paths[s] == br.state_path(h)
        if len(h) == depth:
            return
        for v in range(V):
            b, nx = g.step(s, v)
            Gn = br.G(h + (v,))
            assert b == Gn - Gh, (h, v, b, Gn - Gh)   # dyadic weights: exact
            rec(h + (v,), nx, Gn)

    rec((), 0, 0.0)


def test_walk_equals_substring_matching_long_random_histories():
    rng = np.random.default_rng(99)
    V = 12
    phrases, weights = random_list(rng, V, 6, 4, dyadic_weights=True)
    phrases += [phrases[0] + phrases[1], phrases[2][-1:] + phrases[3]]      # nested / overlapping
    weights += [weights[0] + weights[1], weights[2][-1:] + weights[3]]
    g = O.Graph(phrases, V, weights=weights)
    br = Brute(phrases, None, weights)
    paths = state_paths(g)
    pool = sorted({t for p in phrases for t in p})
    for _ in range(400):
        h, s, Gh = (), 0, 0.0
        for _ in range(14):
            v = int(rng.choice(pool)) if rng.random() < 0.8 else int(rng.integers(0, V))
            b, nx = g.step(s, v)
            Gn = br.G(h + (v,))
            assert b == Gn - Gh
            h, s, Gh = h + (v,), nx, Gn
            assert paths[s] == br.state_path(h)


# ---------------------------------------------------------------------------------------------
# P2: case-insensitive graph == explicit case expansion (Sec. 2.1 para. 2)
# ---------------------------------------------------------------------------------------------

def _sibling_vocab(n3, neutral):
    cc = np.array([c for c in range(n3) for _ in range(3)] + [n3 + i for i in range(neutral)], dtype=np.int32)
    sib = {c: [3 * c, 3 * c + 1, 3 * c + 2] for c in range(n3)}
    sib.update({n3 + i: [3 * n3 + i] for i in range(neutral)})
    return cc, sib


@pytest.mark.parametrize("seed", range(8))
def test_case_insensitive_equals_full_expansion(seed):
    rng = np.random.default_rng(100 + seed)
    cc, sib = _sibling_vocab(3, 2)
    V = len(cc)
    phrases, weights = random_list(rng, V, 4, 3, dyadic_weights=True)
    gi = O.Graph(phrases, V, case_class=cc, weights=weights)
    exp_p, exp_w = [], []
    for p, w in zip(phrases, weights):
        for combo in itertools.product(*[sib[int(cc[t])] for t in p]):
            exp_p.append(list(combo))
            exp_w.append(w)
    gx = O.Graph(exp_p, V, weights=exp_w)           # case-sensitive: every token its own class
    pi, px = state_paths(gi), state_paths(gx)
    for _ in range(300):
        si = sx = 0
        for _ in range(8):
            v = int(rng.integers(0, V))
            bi, si = gi.step(si, v)
            bx, sx = gx.step(sx, v)
            assert bi == bx
            assert pi[si] == tuple(int(cc[t]) for t in px[sx])


def test_lower_upper_title_expansion_agrees_on_single_casings():
    rng = np.random.default_rng(7)
    cc, sib = _sibling_vocab(4, 2)
    V = len(cc)
    lower = [[3 * int(c) for c in rng.integers(0, 4, size=rng.integers(1, 4))] for _ in range(5)]
    gi = O.Graph(lower, V, case_class=cc)
    three = []
    for p in lower:
        three += [p, [t + 1 for t in p], [p[0] + 2] + p[1:]]
    g3 = O.Graph(three, V)
    for casing in (0, 1):
        for _ in range(200):
            si = s3 = 0
            for _ in range(8):
                v = 3 * int(rng.integers(0, 4)) + casing if rng.random() < 0.85 else 12 + int(rng.integers(0, 2))
                bi, si = gi.step(si, v)
                b3, s3 = g3.step(s3, v)
                assert bi == b3
    # a Title rendering between neutral tokens earns the same as the lower-case one
    for p in lower:
        for render in (p, [p[0] + 2] + p[1:]):
            tot_i = tot_3 = 0.0
            si = s3 = 0
            for v in [12] + render + [13]:
                bi, si = gi.step(si, v)
                b3, s3 = g3.step(s3, v)
                tot_i += bi
                tot_3 += b3
            assert tot_i == tot_3


def test_every_casing_earns_the_same_total():
    """Sec. 2.1 (end of the paragraph after Eq. 1): every accepted spelling gets the same bonus."""
    rng = np.random.default_rng(11)
    cc, sib = _sibling_vocab(5, 1)
    V = len(cc)
    phrases = [[3 * int(c) for c in rng.integers(0, 5, size=L)] for L in (1, 2, 3, 4, 4)]
    weights = [[float(rng.choice([0.5, 1.0, 2.0])) for _ in p] for p in phrases]
    g = O.Graph(phrases, V, case_class=cc, weights=weights)
    br = Brute(phrases, cc, weights)
    for p in phrases:
        totals = []
        for combo in itertools.product(range(3), repeat=len(p)):
            s, tot = 0, 0.0
            for t, j in zip(p, combo):
                b, s = g.step(s, t + j)
                tot += b
            totals.append(tot)
        assert len(set(totals)) == 1
        assert totals[0] == br.G(p)


# ---------------------------------------------------------------------------------------------
# P8: structure of the compiled arrays
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("seed", range(6))
def test_csr_invariants(seed):
    rng = np.random.default_rng(200 + seed)
    V = 30
    cc = (np.arange(V) // 2).astype(np.int32)
    phrases, weights = random_list(rng, V, 40, 5, dyadic_weights=True)
    phrases.append([])                                   # empty phrases are skipped
    weights.append([])
    g = O.Graph(phrases, V, case_class=cc, weights=weights)
    assert g.n_arcs == g.n_states - 1
    assert np.array_equal(g.arc_dst, np.arange(1, g.n_states))        # breadth-first numbering of a tree
    assert g.state_arc_begin[0] == 0 and g.state_arc_begin[-1] == g.n_arcs
    for s in range(g.n_states):
        cls = g.arc_class[g.state_arc_begin[s]:g.state_arc_begin[s + 1]]
        assert np.all(np.diff(cls) > 0)
        if s:
            assert g.state_depth[g.state_fail[s]] < g.state_depth[s]
    assert g.max_depth == g.state_depth.max()
    paths = state_paths(g)
    br = Brute(phrases, cc, weights)
    for s in range(g.n_states):
        # suffix link = longest proper suffix of the path that is a tree path
        assert paths[int(g.state_fail[s])] == (br.state_path(paths[s][1:]) if s else ())
        # back-off weights down the whole chain return the loan; the final weight does the same
        u, acc = s, 0.0
        while u:
            acc += float(g.state_bw[u])
            u = int(g.state_fail[u])
        assert acc == -br.loan(paths[s]) == float(g.state_final[s])
        # with non-negative weights no arc on the chain is worth less than missing everything
        for v in range(V):
            b, _ = g.step(s, v)
            assert b >= acc


def test_build_rejects_bad_input():
    with pytest.raises(ValueError):
        O.Graph([[0, 5]], vocab=4)
    with pytest.raises(ValueError):
        O.Graph([[0, 1]], vocab=4, weights=[[1.0, -0.5]])
    with pytest.raises(ValueError):
        O.Graph([[0, 1]], vocab=4, weights=[[1.0, float("nan")]])
    with pytest.raises(ValueError):
        O.Graph([[0, 1]], vocab=4, case_class=np.array([0, -1, 1, 1], dtype=np.int32))
    g = O.Graph([], vocab=4)                              # empty list: root only
    assert g.n_states == 1 and g.step(0, 2) == (0.0, 0)


# ---------------------------------------------------------------------------------------------
# greedy decoding
# ---------------------------------------------------------------------------------------------

def dyadic_logits(rng, shape, blank_bias=0.0, q=64):
    """float32 logits on a grid of 1/q: sums along any alignment are exact in float32."""
    x = rng.integers(-4 * q, 4 * q + 1, size=shape).astype(np.float32) / np.float32(q)
    x[..., -1] += np.float32(blank_bias)
    return x


def numpy_greedy(logits):
    """Unboosted greedy RNNT with numpy's argmax (first maximum = lowest id)."""
    T, S, _ = logits.shape
    V = logits.shape[2] - 1
    t = k = 0
    toks, frs, score = [], [], np.float32(0)
    while t < T:
        tok = int(np.argmax(logits[t, k]))
        score = np.float32(score + logits[t, k, tok])
        if tok == V:
            t, k = t + 1, 0
        else:
            toks.append(tok)
            frs.append(t)
            k += 1
            if k == S:
                t, k = t + 1, 0
    return toks, frs, score


def test_unbound_empty_and_zero_lambda_reduce_to_argmax():
    """Sec. 2.2 para. 3: model id -1 decodes exactly as an unboosted stream."""
    rng = np.random.default_rng(5)
    V = 40
    x = rng.standard_normal((60, 3, V + 1)).astype(np.float32)
    x[:, :, V] += 1.5
    x[3, 0, 7] = x[3, 0, 9] = x[3, 0].max() + 1          # exact ties go to the lowest id
    x[5, 1, V] = x[5, 1, 2] = x[5, 1].max() + 1          # a tie with blank goes to the token
    toks, frs, score = numpy_greedy(x)
    phrases, _ = random_list(rng, V, 10, 3)
    for graph in (None, O.Graph([], V), O.Graph(phrases, V, lam=0.0)):
        r = O.greedy_rnnt(graph, x)
        assert list(r["tokens"]) == toks and list(r["frames"]) == frs
        assert r["score"] == score
    assert O.greedy_rnnt(None, x)["state"] == -1
    assert O.null_step(3) == (0.0, -1)
    # bf16 storage: the same decode on the exactly up-converted values
    from paper_2608_21343_b200.workloads import f32_to_bf16_bits, bf16_bits_to_f32
    xb = f32_to_bf16_bits(x)
    toks_b, frs_b, score_b = numpy_greedy(bf16_bits_to_f32(xb))
    r = O.greedy_rnnt(None, xb)
    assert list(r["tokens"]) == toks_b and list(r["frames"]) == frs_b and r["score"] == score_b
    # strided view and a shorter length
    big = np.zeros((60, 3, V + 9), dtype=np.float32)
    big[:, :, 4:V + 5] = x
    r = O.greedy_rnnt(None, big[:, :, 4:V + 5], length=31)
    toks31, frs31, score31 = numpy_greedy(x[:31])
    assert list(r["tokens"]) == toks31 and r["score"] == score31


@pytest.mark.parametrize("seed", range(6))
def test_greedy_score_bookkeeping(seed):
    """P5: boosted score - raw logits along the chosen alignment = lambda * G(history)."""
    rng = np.random.default_rng(300 + seed)
    V = 9
    cc = (np.arange(V) // 2).astype(np.int32)
    lam = [1.0, 0.5, 2.0][seed % 3]
    phrases, weights = random_list(rng, V, 5, 3, dyadic_weights=True)
    g = O.Graph(phrases, V, case_class=cc, weights=weights, lam=lam)
    br = Brute(phrases, cc, weights)
    x = dyadic_logits(rng, (40, 3, V + 1), blank_bias=0.5)
    r = O.greedy_rnnt(g, x)
    # replay the alignment: every choice must be the argmax of raw + lambda * (G difference)
    t = k = 0
    h, raw, i = (), 0.0, 0
    while t < 40:
        Gh = br.G(h)
        vals = [float(x[t, k, v]) + lam * (br.G(h + (v,)) - Gh) for v in range(V)] + [float(x[t, k, V])]
        tok = int(np.argmax(vals))
        raw += float(x[t, k, tok])
        if tok == V:
            t, k = t + 1, 0
        else:
            assert r["tokens"][i] == tok and r["frames"][i] == t
            i += 1
            h += (tok,)
            k += 1
            if k == 3:
                t, k = t + 1, 0
    assert i == len(r["tokens"])
    assert float(r["score"]) == raw + lam * br.G(h)
    assert state_paths(g)[r["state"]] == br.state_path(tuple(int(cc[v]) for v in h))


# ---------------------------------------------------------------------------------------------
# beam
# ---------------------------------------------------------------------------------------------

def _alignments(x, E, V):
    """Every alignment of a [T, E, V+1] tensor as (score terms, token history)."""
    T = x.shape[0]
    per_frame = []
    for t in range(T):
        opts = []

        def rec(e, toks, raw):
            if e == E:
                opts.append((toks, raw))
                return
            opts.append((toks, raw + [float(x[t, e, V])]))
            for v in range(V):
                rec(e + 1, toks + [v], raw + [float(x[t, e, v])])

        rec(0, [], [])
        per_frame.append(opts)
    for combo in itertools.product(*per_frame):
        yield [v for toks, _ in combo for v in toks], sum(sum(raw) for _, raw in combo)


@pytest.mark.parametrize("seed", range(4))
def test_beam_equals_exhaustive_enumeration(seed):
    """P11: with room for every alignment the beam is the sorted list of all of them."""
    rng = np.random.default_rng(400 + seed)
    V, T, E = 3, 3, 2
    phrases = [[0, 1], [1], [2, 0, 1]][: 2 + seed % 2]
    g = O.Graph(phrases, V)
    br = Brute(phrases)
    x = dyadic_logits(rng, (T, E, V + 1), q=1 << 16)       # fine grid: ties are unlikely
    allal = [(raw + br.G(h), tuple(h)) for h, raw in _alignments(x, E, V)]
    K = len(allal)
    assert K == 13 ** 3
    r = O.beam_decode(g, x, K)
    got = [(float(r["scores"][k]), tuple(int(v) for v in r["tokens"][k])) for k in range(K)]
    assert sorted(got, key=lambda p: (-p[0], p[1])) == sorted(allal, key=lambda p: (-p[0], p[1]))
    assert all(got[i][0] >= got[i + 1][0] for i in range(K - 1))   # slots come out best first
    paths = state_paths(g)
    for k in range(K):
        assert paths[int(r["states"][k])] == br.state_path(got[k][1])
    # a narrow beam: each survivor's score is still the brute-force score of its own history,
    # and no survivor beats the true optimum
    best = max(s for s, _ in allal)
    r4 = O.beam_decode(g, x, 4)
    for k in range(4):
        hist = tuple(int(v) for v in r4["tokens"][k])
        assert (float(r4["scores"][k]), hist) in set(allal)
        assert float(r4["scores"][k]) <= best


@pytest.mark.parametrize("seed", range(4))
def test_beam_of_one_is_greedy(seed):
    """P10: K = 1 with E = S rows per frame is greedy decoding."""
    rng = np.random.default_rng(500 + seed)
    V = 12
    cc = (np.arange(V) // 3).astype(np.int32)
    phrases, weights = random_list(rng, V, 6, 3, dyadic_weights=True)
    g = O.Graph(phrases, V, case_class=cc, weights=weights)
    x = dyadic_logits(rng, (50, 3, V + 1), blank_bias=0.75)
    x[4, 0, 2] = x[4, 0, 5] = 6.0                                # a tie
    rg = O.greedy_rnnt(g, x)
    rb = O.beam_decode(g, x, 1)
    assert list(rb["tokens"][0]) == list(rg["tokens"])
    assert rb["scores"][0] == rg["score"] and rb["states"][0] == rg["state"]


def test_beam_step_order_and_carry():
    """Ordering (score, then token id, then parent), frozen hypotheses carried, empty slots."""
    V = 3
    g = O.Graph([[0]], V)
    rows = np.zeros((3, V + 1), dtype=np.float32)
    rows[0] = [1.0, 2.0, 0.0, 2.0]          # live: token 0 gets +1 -> 2.0, ties with token 1 and blank
    rows[1] = [9.0, 9.0, 9.0, 9.0]          # frozen: its row must not be read
    scores = np.array([0.0, 2.0, -np.inf], dtype=np.float32)
    states = np.array([0, 0, -1], dtype=np.int32)
    live = np.array([1, 0, 0], dtype=np.uint8)
    par, tok = O.beam_step(g, rows, scores, states, live)
    # candidates worth 2.0: (k0,tok0) (k0,tok1) (k0,blank=3) (k1 carried, key 4)
    assert list(par) == [0, 0, 0] and list(tok) == [0, 1, 3]
    assert list(scores) == [2.0, 2.0, 2.0] and list(states) == [1, 0, 0] and list(live) == [1, 1, 0]
    scores = np.array([-np.inf, 1.0, -np.inf], dtype=np.float32)
    states = np.array([-1, 0, -1], dtype=np.int32)
    live = np.array([0, 0, 0], dtype=np.uint8)
    par, tok = O.beam_step(g, rows, scores, states, live)
    assert list(par) == [1, -1, -1] and list(tok) == [-1, -1, -1]
    assert scores[0] == 1.0 and np.isneginf(scores[1]) and list(states) == [0, -1, -1]


def test_beam_step_equal_candidates_go_to_the_lower_parent():
    """Hand-worked step for the last clause of the order (score, token id, parent): two live hypotheses with
    equal scores and equal graph states read the same row, so every (token) candidate exists twice with the same
    value; each pair must come out lower parent first.  A third hypothesis with a lower score whose row lifts one
    of its candidates to the same value joins such a pair as the highest parent."""
    V = 3
    g = O.Graph([[0]], V)                                   # token 0 earns +1 at the root
    row = np.array([0.0, 0.5, -4.0, 0.5], dtype=np.float32)  # values at the root: 1.0, 0.5, -4.0, blank 0.5
    rows = np.stack([row, row, row, row])
    scores = np.array([0.0, -np.inf, 0.0, -np.inf], dtype=np.float32)   # hypotheses 0 and 2, slot 1 and 3 empty
    states = np.array([0, -1, 0, -1], dtype=np.int32)
    live = np.array([1, 0, 1, 0], dtype=np.uint8)
    par, tok = O.beam_step(g, rows, scores, states, live)
    # 1.0: (0, tok 0) (2, tok 0);  0.5: (0, tok 1) (2, tok 1), then the blanks (0, 3) (2, 3) which no longer fit
    assert list(tok) == [0, 0, 1, 1] and list(par) == [0, 2, 0, 2]
    assert list(scores) == [1.0, 1.0, 0.5, 0.5] and list(states) == [1, 1, 0, 0] and list(live) == [1, 1, 1, 1]
    # three parents in one tie: hypothesis 1 scores 0.25 less and its own row offers token 0 at 0.25 more
    rows = np.stack([row, row + np.float32(0.25), row, row])
    scores = np.array([0.0, -0.25, 0.0, -np.inf], dtype=np.float32)
    states = np.array([0, 0, 0, -1], dtype=np.int32)
    live = np.array([1, 1, 1, 0], dtype=np.uint8)
    par, tok = O.beam_step(g, rows, scores, states, live)
    assert list(tok) == [0, 0, 0, 1] and list(par) == [0, 1, 2, 0]
    assert list(scores) == [1.0, 1.0, 1.0, 0.5]
    # frozen hypotheses with equal scores are carried in parent order as well (their key is the same, V + 1)
    scores = np.array([2.0, 2.0, 2.0, -np.inf], dtype=np.float32)
    states = np.array([0, 1, 0, -1], dtype=np.int32)
    live = np.array([0, 0, 0, 0], dtype=np.uint8)
    par, tok = O.beam_step(g, rows, scores, states, live)
    assert list(par) == [0, 1, 2, -1] and list(tok) == [-1, -1, -1, -1] and list(states) == [0, 1, 0, -1]


# ---------------------------------------------------------------------------------------------
# TDT and streaming
# ---------------------------------------------------------------------------------------------

def test_tdt_with_unit_durations_is_one_symbol_per_frame():
    """P12: durations rigged to 1 -> per-frame argmax of the first row plus the walk."""
    rng = np.random.default_rng(8)
    V, D, T = 10, 5, 40
    phrases, _ = random_list(rng, V, 5, 3)
    g = O.Graph(phrases, V)
    x = dyadic_logits(rng, (T, 3, V + 1 + D))
    x[:, :, V + 1:] = 0.0
    x[:, :, V + 2] = 1.0                                         # duration index 1 always wins
    st = O.StreamState(0, 0, 0, 0.0, 0)
    r = O.stream_chunk(g, x, D, 0, T, st)
    s, toks, frs, score = 0, [], [], 0.0
    for t in range(T):
        vals = [float(x[t, 0, v]) + g.step(s, v)[0] for v in range(V)] + [float(x[t, 0, V])]
        tok = int(np.argmax(vals))
        score += vals[tok] + 1.0
        if tok != V:
            toks.append(tok)
            frs.append(t)
            s = g.step(s, tok)[1]
    assert list(r["tokens"]) == toks and list(r["frames"]) == frs and set(r["durs"]) <= {1}
    assert st.state == s and st.t == T and float(st.score) == score


def test_tdt_duration_rules():
    V, D = 2, 5
    x = np.zeros((12, 2, V + 1 + D), dtype=np.float32)

    def row(t, k, tok, dur, tie_dur=None):
        x[t, k, tok] = 5.0
        x[t, k, V + 1 + dur] = 2.0
        if tie_dur is not None:
            x[t, k, V + 1 + tie_dur] = 2.0

    row(0, 0, 0, 0)           # token 0, duration 0: stay in frame 0, next row
    row(0, 1, 1, 0)           # token 1, duration 0, second symbol: frame closes by force
    row(1, 0, V, 0)           # blank with duration 0 still advances one frame
    row(2, 0, 1, 3, tie_dur=4)   # token 1, durations 3 and 4 tie -> 3: jump to frame 5
    row(5, 0, V, 4)           # blank, duration 4 -> frame 9
    row(9, 0, 0, 2)           # token at 9, duration 2 -> frame 11
    row(11, 0, V, 4)          # blank: cursor carried beyond the end (15)
    st = O.StreamState(-1, 0, 0, 0.0, 0)
    r = O.stream_chunk(None, x, D, 0, 12, st)
    assert list(r["tokens"]) == [0, 1, 1, 0] and list(r["frames"]) == [0, 0, 2, 9]
    assert list(r["durs"]) == [0, 0, 3, 2]
    assert st.t == 15 and st.k == 0 and st.state == -1 and st.n_emitted == 4
    assert float(st.score) == 7 * 7.0


@pytest.mark.parametrize("n_dur", [0, 5])
def test_chunked_equals_unchunked(n_dur):
    """P13 (Sec. 2.3: state is kept across chunk boundaries)."""
    rng = np.random.default_rng(9 + n_dur)
    V, T = 15, 67
    cc = (np.arange(V) // 3).astype(np.int32)
    phrases, weights = random_list(rng, V, 8, 4, dyadic_weights=True)
    g = O.Graph(phrases, V, case_class=cc, weights=weights)
    x = dyadic_logits(rng, (T, 3, V + 1 + n_dur), blank_bias=0.0)
    x[:, :, V] += 0.5
    valid = 61
    whole = O.StreamState(0, 0, 0, 0.0, 0)
    ref = O.stream_chunk(g, x, n_dur, 0, valid, whole)
    if n_dur == 0:
        rg = O.greedy_rnnt(g, x, length=valid)
        assert list(rg["tokens"]) == list(ref["tokens"]) and list(rg["frames"]) == list(ref["frames"])
        assert rg["score"] == np.float32(whole.score) and rg["state"] == whole.state
    for chunk in (1, 8, 13):
        st = O.StreamState(0, 0, 0, 0.0, 0)
        toks, frs, durs = [], [], []
        for t0 in range(0, T, chunk):
            part = np.ascontiguousarray(x[t0:t0 + chunk])
            r = O.stream_chunk(g, part, n_dur, t0, valid, st)
            toks += list(r["tokens"]); frs += list(r["frames"]); durs += list(r["durs"])
        assert toks == list(ref["tokens"]) and frs == list(ref["frames"]) and durs == list(ref["durs"])
        assert (st.state, st.t, st.k, st.n_emitted) == (whole.state, whole.t, whole.k, whole.n_emitted)
        assert st.score == whole.score


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_tdt_with_zero_durations_is_the_rnnt_rule(seed):
    """Durations rigged to 0 on every row: a token stays in its frame and moves to the next row, blank still
    advances one frame, the S-th symbol closes the frame -- the label-looping RNNT rule, which is pinned on its own.
    The duration logit that wins is 0, so even the scores agree bit for bit."""
    rng = np.random.default_rng(40 + seed)
    V, D, T, S = 12, 5, 50, 3
    phrases, weights = random_list(rng, V, 6, 3, dyadic_weights=True)
    g = O.Graph(phrases, V, weights=weights)
    x = dyadic_logits(rng, (T, S, V + 1 + D), blank_bias=0.5)
    x[:, :, V + 1:] = -1.0
    x[:, :, V + 1] = 0.0
    st = O.StreamState(0, 0, 0, 0.0, 0)
    r = O.stream_chunk(g, x, D, 0, T, st)
    ref = O.greedy_rnnt(g, np.ascontiguousarray(x[:, :, :V + 1]))
    assert list(r["tokens"]) == list(ref["tokens"]) and list(r["frames"]) == list(ref["frames"])
    assert set(r["durs"]) <= {0} and st.state == ref["state"] and st.t == T
    assert np.float32(st.score) == ref["score"]


@pytest.mark.parametrize("d", [2, 3, 4])
def test_tdt_with_constant_durations_is_the_unit_case_on_every_dth_frame(d):
    """Durations rigged to d on every row: only rows (0, 0), (d, 0), (2d, 0), ... are visited, each once -- the
    unit-duration decode (pinned above against a per-frame argmax) of the tensor that keeps every d-th frame."""
    rng = np.random.default_rng(50 + d)
    V, D, T, S = 10, 5, 61, 2
    phrases, _ = random_list(rng, V, 5, 3)
    g = O.Graph(phrases, V)
    x = dyadic_logits(rng, (T, S, V + 1 + D))
    x[:, :, V + 1:] = 0.0
    x[:, :, V + 1 + d] = 1.0
    st = O.StreamState(0, 0, 0, 0.0, 0)
    r = O.stream_chunk(g, x, D, 0, T, st)
    y = np.ascontiguousarray(x[::d])
    y[:, :, V + 1:] = 0.0
    y[:, :, V + 2] = 1.0                                         # the same rows, duration 1
    Ty = y.shape[0]
    st1 = O.StreamState(0, 0, 0, 0.0, 0)
    r1 = O.stream_chunk(g, y, D, 0, Ty, st1)
    assert list(r["tokens"]) == list(r1["tokens"]) and list(r["frames"]) == [d * f for f in r1["frames"]]
    assert set(r["durs"]) <= {d} and st.state == st1.state and st.score == st1.score
    assert st.t == d * Ty and st.n_emitted == st1.n_emitted


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_final_weight_leaves_exactly_the_completed_phrases(seed):
    """After the end-of-stream charge the bonus a history has collected is the sum over the phrase occurrences
    that were completed in it, found by plain substring matching (no automaton): the loan of an unfinished
    match is gone.  Dyadic weights make every sum exact."""
    rng = np.random.default_rng(70 + seed)
    V = 6
    phrases, weights = random_list(rng, V, 8, 4, dyadic_weights=True)
    merged = {}
    for p, wts in zip(phrases, weights):                       # duplicates: element-wise largest weight
        if len(p):
            merged[tuple(p)] = [max(a, b) for a, b in zip(merged.get(tuple(p), [0.0] * len(p)), wts)]
    # weight of the node reached by a prefix = largest weight any phrase through it gives that position
    node_w = {}
    for p, wts in merged.items():
        for i in range(len(p)):
            node_w[p[:i + 1]] = max(node_w.get(p[:i + 1], 0.0), wts[i])
    ends = sorted(merged, key=len)

    def completed_value(p):
        # what completing p banks: the node weights since the last phrase end strictly inside p
        last = max([len(q) for q in ends if len(q) < len(p) and p[:len(q)] == q], default=0)
        return sum(node_w[p[:i + 1]] for i in range(last, len(p)))
    g = O.Graph(phrases, V, weights=weights, lam=2.0)
    for _ in range(200):
        h = [int(t) for t in rng.integers(0, V, size=int(rng.integers(0, 14)))]
        s, total = 0, 0.0
        for t in h:
            b, s = g.step(s, t)
            total += 2.0 * float(b)
        total = float(O.apply_final_weight(g, s, total))
        want = 0.0
        for p in merged:
            for i in range(len(h) - len(p) + 1):
                if tuple(h[i:i + len(p)]) == p:
                    want += 2.0 * completed_value(p)
        assert total == want, (h, total, want)
    assert float(O.apply_final_weight(None, -1, 3.5)) == 3.5 and float(O.apply_final_weight(g, -1, 3.5)) == 3.5


@pytest.mark.parametrize("seed", range(4))
def test_beam_with_merging_keeps_the_best_alignment_of_every_sequence(seed):
    """With room for everything, merging equal token sequences at frame starts leaves, for every distinct
    token sequence, exactly its best alignment (found by exhaustive enumeration), in score order."""
    rng = np.random.default_rng(600 + seed)
    V, T, E = 3, 3, 2
    phrases = [[0, 1], [1], [2, 0, 1]][: 2 + seed % 2]
    g = O.Graph(phrases, V)
    br = Brute(phrases)
    x = dyadic_logits(rng, (T, E, V + 1), q=1 << 16)
    best = {}
    for h, raw in _alignments(x, E, V):
        sc = raw + br.G(h)
        best[tuple(h)] = max(best.get(tuple(h), -np.inf), sc)
    K = 13 ** 3
    r = O.beam_decode(g, x, K, merge=True)
    got = [(float(r["scores"][k]), tuple(int(v) for v in r["tokens"][k])) for k in range(K) if np.isfinite(r["scores"][k])]
    # merging happens at frame starts, so the alignments of the last frame are still all there: reduce them
    final = {}
    for sc, h in got:
        final[h] = max(final.get(h, -np.inf), sc)
    assert final == best
    # and before the last frame nothing is double: the number of survivors is what the last frame can make of
    # the distinct sequences alive at its start
    r2 = O.beam_decode(g, x[:T - 1], K, merge=True)
    alive = [tuple(int(v) for v in r2["tokens"][k]) for k in range(K) if np.isfinite(r2["scores"][k])]
    n_start = len(set(alive))
    assert len(got) == 13 * n_start
    # without merging the same run keeps every alignment
    r0 = O.beam_decode(g, x, K)
    assert int(np.isfinite(r0["scores"]).sum()) == K > len(got)


@pytest.mark.parametrize("seed", range(3))
def test_beam_pruning_reductions_and_brute_force(seed):
    """Pruning at frame starts against what does not use the beam code: a threshold of infinity changes nothing;
    a threshold of 0 with one row per frame leaves one hypothesis per frame, i.e. the beam of one (greedy);
    and with room for everything the survivors are the alignments whose prefixes, frame by frame, stayed
    within the threshold of the best surviving prefix (set recursion over exhaustive enumeration)."""
    rng = np.random.default_rng(700 + seed)
    V, T, E = 3, 3, 2
    phrases = [[0, 1], [1], [2, 0, 1]][: 2 + seed % 2]
    g = O.Graph(phrases, V)
    br = Brute(phrases)
    x = dyadic_logits(rng, (T, E, V + 1), q=1 << 16)
    K = 13 ** 3
    r_inf = O.beam_decode(g, x, K, prune_delta=float("inf"))
    r_off = O.beam_decode(g, x, K)
    assert np.array_equal(r_inf["tree"], r_off["tree"]) and np.array_equal(r_inf["scores"], r_off["scores"])
    x1 = np.ascontiguousarray(x[:, :1])                         # one row per frame: every step starts a frame
    r0 = O.beam_decode(g, x1, 5, prune_delta=0.0)
    r1 = O.beam_decode(g, x1, 1)
    assert list(r0["tokens"][0]) == list(r1["tokens"][0]) and r0["scores"][0] == r1["scores"][0]
    # brute force: per frame, extend every surviving history by every alignment of that frame, then prune
    delta = 1.5
    per_frame = []
    for t in range(T):
        opts = []

        def rec(e, toks, raw):
            if e == E:
                opts.append((toks, raw)); return
            opts.append((toks, raw + [float(x[t, e, V])]))
            for v in range(V):
                rec(e + 1, toks + [v], raw + [float(x[t, e, v])])
        rec(0, [], [])
        per_frame.append(opts)
    alive = [((), 0.0)]                                         # (history, raw logit sum); the bonus comes from Brute
    for t in range(T):
        total = [(h, raw + br.G(list(h))) for h, raw in alive]
        best = max(s for _, s in total)
        alive = [(h, raw) for (h, raw), (_, s) in zip(alive, total) if s >= best - delta]
        alive = [(h + tuple(toks), raw + sum(rw)) for h, raw in alive for toks, rw in per_frame[t]]
    want = sorted(((raw + br.G(list(h)), h) for h, raw in alive), key=lambda p: (-p[0], p[1]))
    r = O.beam_decode(g, x, K, prune_delta=delta)
    got = [(float(r["scores"][k]), tuple(int(v) for v in r["tokens"][k])) for k in range(K) if np.isfinite(r["scores"][k])]
    assert sorted(got, key=lambda p: (-p[0], p[1])) == want
    assert 0 < len(got) < K
