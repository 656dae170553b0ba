"""Pins of the oracle's variative, case-insensitive compile (Sec. 2.1 para. 4-7, Eq. 1) against things that
are not its own formulas: the C tree compiler (itself pinned by brute-force substring matching) on
single-character vocabularies, closed forms of Eq. 1, a hand-worked two-letter list, and the invariance
the section states: every spelling of a phrase, in any casing and segmentation, earns the same total."""
import math

import numpy as np
import pytest

from oracle import oracle as orc
from oracle import variative as var
from paper_2608_21343_b200 import workloads as W


def _single_char_vocab(letters):
    out = []
    for i in range(letters):
        out += [bytes([97 + i]), bytes([65 + i])]
    return out


def _arrays_equal(a, g):
    for k in ("state_arc_begin", "arc_class", "arc_dst", "state_fail", "state_depth", "case_class"):
        assert np.array_equal(a[k], getattr(g, k)), k
    for k in ("arc_w", "state_bw", "state_final"):
        assert np.array_equal(a[k].view(np.uint32), getattr(g, k).view(np.uint32)), k


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_single_character_vocabulary_reduces_to_the_tree_compiler(seed):
    # every piece one character: m_k = 1, Eq. 1 gives the whole score to that character, arcs never skip
    rng = np.random.default_rng(seed)
    letters = 5
    pieces = _single_char_vocab(letters)
    phrases = [bytes(int(x) + 97 for x in rng.integers(0, letters, size=int(rng.integers(1, 6)))) for _ in range(12)]
    wts = [float(rng.choice([0.5, 1.0, 1.5, 2.0])) for _ in phrases]
    a = var.build(phrases, pieces, weights=wts, tau=1.3, lam=1.0)
    cc, _ = var.piece_classes(pieces)
    tok = [[2 * (b - 97) for b in p] for p in phrases]
    g = orc.Graph(tok, len(pieces), case_class=cc, weights=[[w] * len(p) for w, p in zip(wts, phrases)], lam=1.0)
    assert a["n_states"] == g.n_states and a["n_arcs"] == g.n_arcs
    _arrays_equal(a, g)


def test_eq1_closed_forms():
    for m in (1, 2, 3, 7):
        u = var.eq1_split(2.0, m, 0.0)
        assert np.allclose(u, [2.0 / m] * m, rtol=1e-15)                       # tau = 0: uniform
        for tau in (0.5, 1.0, 2.0):
            d = var.eq1_split(1.5, m, tau)
            assert abs(sum(d) - 1.5) < 1e-12                                      # the shares add up to w_k
            assert all(d[i] < d[i + 1] for i in range(m - 1))                     # growing towards the end
            for i in range(m - 1):                                                # ratio of neighbours
                assert math.isclose(d[i + 1] / d[i], math.exp((i + 2) ** tau - (i + 1) ** tau), rel_tol=1e-12)
    d = var.eq1_split(1.0, 4, 6.0)
    assert d[-1] > 1.0 - 1e-12                                                    # large tau: all at the end
    assert math.isclose(var.eq1_split(1.0, 2, 1.0)[0], 1.0 / (1.0 + math.e), rel_tol=1e-15)


def test_hand_worked_two_letter_list():
    # list {"ab"}, pieces a A b B ab: backbone "ab" (m = 2); tau = 0 halves the score
    pieces = [b"a", b"A", b"b", b"B", b"ab"]
    a = var.build([b"ab"], pieces, tau=0.0)
    assert a["n_states"] == 3 and list(a["case_class"]) == [0, 0, 1, 1, 2]
    assert list(a["state_arc_begin"]) == [0, 2, 3, 3]
    assert list(a["arc_class"]) == [0, 2, 1] and list(a["arc_dst"]) == [1, 2, 2]
    assert list(a["arc_w"]) == [0.5, 1.0, 0.5]             # a: half on loan; ab: the whole phrase; b after a: the rest
    assert list(a["state_fail"]) == [0, 0, 0]
    assert list(a["state_bw"]) == [0.0, -0.5, 0.0]         # leaving "a" unfinished returns the loan
    assert list(a["state_final"]) == [0.0, -0.5, 0.0]
    # tau = 1: shares 1 / (1 + e) and e / (1 + e)
    b = var.build([b"ab"], pieces, tau=1.0)
    assert np.allclose(b["arc_w"], [1 / (1 + math.e), 1.0, math.e / (1 + math.e)], rtol=1e-7)


def test_backbone_is_longest_match_first():
    cls = {b"a": 0, b"b": 1, b"ab": 2, b"abb": 3, b"c": 4}
    assert var.greedy_backbone(b"abbc", cls, 3) == [3, 1]
    assert var.greedy_backbone(b"abab", cls, 3) == [2, 2]
    assert var.greedy_backbone(b"bca", cls, 3) == [1, 1, 1]
    with pytest.raises(ValueError):
        var.greedy_backbone(b"abz", cls, 3)


def _walk(g, toks, s=0):
    total = 0.0
    for t in toks:
        b, s = g.step(s, t)
        total += float(b)
    return total, s


@pytest.mark.parametrize("seed", [0, 1, 2, 3, 4])
def test_every_spelling_of_a_phrase_earns_the_same(seed):
    pieces = W.make_piece_vocab(seed, letters=6, merged=40, max_len=3)
    phrases = W.draw_string_phrases(seed, pieces, 30, 1, 4)
    tau = [0.0, 0.5, 1.0, 2.0, 1.0][seed]
    g = orc.GraphFromArrays(var.build(phrases, pieces, tau=tau))
    ids = {p: t for t, p in reversed(list(enumerate(pieces)))}
    rng = np.random.default_rng(seed)
    for ph in phrases:
        chars = [ids[bytes([b])] for b in ph]
        ref_total, ref_state = _walk(g, chars)                 # character by character, lower case
        for _ in range(8):
            toks = W.random_spelling(rng, ph, pieces)
            total, state = _walk(g, toks)
            assert state == ref_state
            assert abs(total - ref_total) < 1e-5
    # ... and from inside other matches too: a random prefix first, then the phrase
    for _ in range(50):
        pre = phrases[int(rng.integers(len(phrases)))]
        ph = phrases[int(rng.integers(len(phrases)))]
        cut = int(rng.integers(0, len(pre) + 1))
        head = [ids[bytes([b])] for b in pre[:cut]]
        t0, s0 = _walk(g, head)
        ref_total, ref_state = _walk(g, [ids[bytes([b])] for b in ph], s0)
        total, state = _walk(g, W.random_spelling(rng, ph, pieces), s0)
        # (a merged piece is retried whole from the suffix states, so the two may differ when the walk
        #  leaves the tree in mid-piece; they must agree whenever the characters stay on one path)
        if _stays_on_path(g, s0, [ids[bytes([b])] for b in ph]):
            assert state == ref_state and abs(total - ref_total) < 1e-5


def _stays_on_path(g, s, chars):
    for t in chars:
        c = g.case_class[t]
        arcs = range(g.state_arc_begin[s], g.state_arc_begin[s + 1])
        nxt = [g.arc_dst[a] for a in arcs if g.arc_class[a] == c]
        if not nxt:
            return False
        s = nxt[0]
    return True


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_single_character_arcs_equal_the_tree_compiler_on_eq1_shares(seed):
    # the same character tree given to the C tree compiler with Eq. 1's shares as per-character weights:
    # the states coincide, and so must every single-character arc, suffix link and suffix-link weight;
    # a merged arc equals the sum of the single-character arcs it spans
    pieces = W.make_piece_vocab(seed, letters=5, merged=25, max_len=3)
    phrases = W.draw_string_phrases(seed, pieces, 20, 1, 3)
    tau = 0.7
    a = var.build(phrases, pieces, tau=tau)
    cls = {c: i for i, c in enumerate(var.piece_classes(pieces)[1])}
    longest = max(len(c) for c in cls)
    letters = sorted({b for p in phrases for b in p})
    tok = [[letters.index(b) for b in p] for p in phrases]
    wts = [[d for m in var.greedy_backbone(p, cls, longest) for d in var.eq1_split(1.0, m, tau)] for p in phrases]
    t = orc.Graph(tok, len(letters), weights=wts)
    assert t.n_states == a["n_states"]
    assert np.array_equal(t.state_fail, a["state_fail"]) and np.array_equal(t.state_depth, a["state_depth"])
    assert np.allclose(t.state_bw, a["state_bw"], rtol=0, atol=1e-6)
    single = {}
    for u in range(t.n_states):
        for x in range(t.state_arc_begin[u], t.state_arc_begin[u + 1]):
            single[(u, letters[t.arc_class[x]])] = (t.arc_dst[x], float(t.arc_w[x]))
    spell = var.piece_classes(pieces)[1]
    for u in range(a["n_states"]):
        for x in range(a["state_arc_begin"][u], a["state_arc_begin"][u + 1]):
            s, total = u, 0.0
            for b in spell[a["arc_class"][x]]:
                s, w = single[(s, b)]
                total += w
            assert s == a["arc_dst"][x]
            assert abs(total - float(a["arc_w"][x])) < 1e-5
