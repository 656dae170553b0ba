"""Oracle front end: variative, case-insensitive compile of phrase lists over a piece vocabulary.

TEST INFRASTRUCTURE ONLY: imported by the tests (and by nothing in the product).  Plain Python,
potentials in double precision, every stored value rounded once to float32.  It produces the same
arrays as the C oracle's own tree compiler (arc label / target / weight, per state the arc range,
suffix link, suffix-link weight, final weight), so the C oracle's decoders run on its graphs
unchanged.

What it follows (paper sections):
  - Sec. 2.1 para. 4: a phrase is turned into a chain of its characters; every vocabulary piece
    whose spelling covers a contiguous stretch of the chain is an arc over that stretch (single
    characters and merged pieces alike).
  - Sec. 2.1 para. 5: for case-insensitive boosting the chain is lower-cased and a piece is an arc
    wherever its lower-cased spelling matches; the result is not a tree (arcs of different lengths
    converge) but is acyclic apart from the suffix links.
  - Sec. 2.1 para. 6-7 and Eq. 1: states carry a cumulative potential and an arc scores the
    difference of the potentials of its ends; the potentials come from the greedy tokenisation of
    the lower-cased phrase: token k with score w_k and m_k characters gives character i of it the
    share w_k * exp((i+1)^tau) / sum_j exp((j+1)^tau).

READINGS (the paper does not fix these):
  - lower-casing is that of the ASCII letters; pieces with the same lower-cased spelling form one
    class and share their arcs;
  - the "greedy tokenisation" is longest-match-first over the lower-cased spellings in the
    vocabulary (any deterministic tokeniser can serve as the scoring backbone);
  - phrases that share a prefix share its states; a state's share is the largest any of them gives it;
  - suffix links, the loan / bank split of the potential and the suffix-link weights are those of
    the tree compiler, taken over the character chain: a phrase counts as completed whenever the
    emitted characters reach its end, also in the middle of a merged piece, so an arc's weight is
    the sum of the single-character arc weights along its stretch.  Every segmentation of the same
    characters therefore earns the same total.

Pins (tests/test_oracle_variative_pins.py): with a vocabulary of single characters the arrays equal
those of the C tree compiler; Eq. 1 closed forms (tau = 0 uniform, shares sum to w_k, growing with
i); all segmentations of a spelling, in any casing, collect the same bonus and end in the same
state as the character-by-character path.
"""
from __future__ import annotations

import math

import numpy as np


def canonical(piece: bytes) -> bytes:
    """Lower-cased spelling (ASCII letters)."""
    return bytes(b + 32 if 65 <= b <= 90 else b for b in piece)


def piece_classes(pieces):
    """(case_class[V], spellings): one class per distinct lower-cased spelling, numbered in order of the
    lowest token id that has it."""
    ids, cc = {}, []
    for p in pieces:
        c = canonical(p)
        if len(c) == 0:
            raise ValueError("empty piece")
        if c not in ids:
            ids[c] = len(ids)
        cc.append(ids[c])
    spell = [None] * len(ids)
    for c, i in ids.items():
        spell[i] = c
    return np.array(cc, dtype=np.int32), spell


def greedy_backbone(canon: bytes, class_of: dict, longest: int):
    """Lengths m_k of the greedy (longest match first) segmentation of a lower-cased phrase."""
    out, i = [], 0
    while i < len(canon):
        for m in range(min(longest, len(canon) - i), 0, -1):
            if canon[i:i + m] in class_of:
                out.append(m)
                i += m
                break
        else:
            raise ValueError("a character of the phrase has no piece")
    return out


def eq1_split(w: float, m: int, tau: float):
    """Eq. 1: the shares of a token's score over its m characters (exponents shifted by the largest one,
    which leaves the quotient as it is and keeps exp in range)."""
    top = float(m) ** tau
    e = [math.exp(float(i + 1) ** tau - top) for i in range(m)]
    z = 0.0
    for x in e:
        z = z + x
    return [w * x / z for x in e]


def build(phrases, pieces, weights=None, tau: float = 1.0, lam: float = 1.0) -> dict:
    """Compile phrases (byte strings, any casing) over the piece vocabulary (byte strings).
    tau and the weights are taken at float32 precision (what a caller of the library can pass)."""
    tau = float(np.float32(tau))
    case_class, spell = piece_classes(pieces)
    class_of = {c: i for i, c in enumerate(spell)}
    longest = max(len(c) for c in spell)
    # ---- character tree (Sec. 2.1 para. 4-5), node weights from Eq. 1 -------------------------
    child = [dict()]
    par, dep, wt, end = [-1], [0], [0.0], [False]
    for pi, ph in enumerate(phrases):
        canon = canonical(ph)
        if len(canon) == 0:
            continue
        if len(canon) > 255:
            raise ValueError("phrase longer than 255 characters")
        w = 1.0 if weights is None else float(np.float32(weights[pi]))
        shares = [d for m in greedy_backbone(canon, class_of, longest) for d in eq1_split(w, m, tau)]
        u = 0
        for i, b in enumerate(canon):
            v = child[u].get(b)
            if v is None:
                v = len(child)
                child[u][b] = v
                child.append(dict()); par.append(u); dep.append(dep[u] + 1); wt.append(0.0); end.append(False)
            wt[v] = max(wt[v], shares[i])
            u = v
        end[u] = True
    # ---- canonical numbering: breadth first, children in ascending character order -------------
    order = [0]
    for u in order:
        for b in sorted(child[u]):
            order.append(child[u][b])
    new = {old: i for i, old in enumerate(order)}
    n = len(order)
    kids = [{b: new[v] for b, v in child[old].items()} for old in order]
    parent = [new[par[old]] if par[old] >= 0 else -1 for old in order]
    depth = [dep[old] for old in order]
    wgt = [wt[old] for old in order]
    is_end = [end[old] for old in order]
    byte_in = [0] * n
    for u in range(n):
        for b, v in kids[u].items():
            byte_in[v] = b
    # ---- suffix links over the characters --------------------------------------------------------
    fail = [0] * n
    for v in range(1, n):
        u = parent[v]
        if u == 0:
            continue
        f = fail[u]
        while True:
            if byte_in[v] in kids[f]:
                fail[v] = kids[f][byte_in[v]]
                break
            if f == 0:
                break
            f = fail[f]
    # ---- potentials: on loan since the last completed phrase / banked on arrival -----------------
    loan, out = [0.0] * n, [0.0] * n
    for v in range(1, n):
        through = loan[parent[v]] + wgt[v]
        loan[v] = 0.0 if is_end[v] else through
        out[v] = (through if is_end[v] else 0.0) + out[fail[v]]
    # ---- arcs: every class whose spelling continues the state's path ------------------------------
    arc_begin, arc_class, arc_dst, arc_w = [0], [], [], []
    for u in range(n):
        found = []
        stack = [(u, b"", 0.0)]
        while stack:
            x, path, banked = stack.pop()
            for b, v in kids[x].items():
                p2 = path + bytes([b])
                got = banked + out[v]
                if p2 in class_of:
                    found.append((class_of[p2], v, loan[v] - loan[u] + got))
                if len(p2) < longest:
                    stack.append((v, p2, got))
        found.sort()
        for c, v, w in found:
            arc_class.append(c); arc_dst.append(v); arc_w.append(np.float32(w))
        arc_begin.append(len(arc_class))
    return dict(
        n_states=n, n_arcs=len(arc_class), n_classes=len(spell), vocab=len(pieces), max_depth=max(depth), lam=lam,
        state_arc_begin=np.array(arc_begin, dtype=np.int32), arc_class=np.array(arc_class, dtype=np.int32),
        arc_dst=np.array(arc_dst, dtype=np.int32), arc_w=np.array(arc_w, dtype=np.float32),
        state_fail=np.array(fail, dtype=np.int32),
        state_bw=np.array([np.float32(loan[fail[u]] - loan[u]) if u else np.float32(0.0) for u in range(n)], dtype=np.float32),
        state_final=np.array([np.float32(-loan[u]) for u in range(n)], dtype=np.float32),
        state_depth=np.array(depth, dtype=np.uint8), case_class=case_class)
