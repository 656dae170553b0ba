"""Pins of the oracle's normalised (log-softmax) greedy decode, against what the mathematics fixes and against
library routines it does not itself call: the normaliser against scipy's logsumexp, the probabilities summing to
one, invariance under a per-row shift, the selected tokens being those of the un-normalised decode (the normaliser
is the same for every entry of a row), the score being the un-normalised row values minus the normalisers, and the
behaviour of the follow mode that the GPU comparison relies on."""
import numpy as np
import pytest
from scipy.special import logsumexp

from oracle import oracle as O
from paper_2608_21343_b200 import workloads as W


def _case(seed, V=40, T=60, S=3, n_phrases=12, grid=None):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((T, S, V + 1)).astype(np.float32)
    x[..., V] += 1.5
    if grid:
        x = (np.round(x * grid) / grid).astype(np.float32)
    cc = (np.arange(V) // 2).astype(np.int32)
    phrases = [[int(t) for t in rng.integers(0, V, size=rng.integers(1, 5))] for _ in range(n_phrases)]
    return x, O.Graph(phrases, V, case_class=cc), phrases


def _visited_rows(tokens, frames, T, S):
    """(t, k, emitted token or None for blank) of every row a greedy decode with this output visits."""
    rows, n = [], 0
    for t in range(T):
        k = 0
        while k < S and n < len(tokens) and frames[n] == t:
            rows.append((t, k, int(tokens[n])))
            n += 1
            k += 1
        if k < S:
            rows.append((t, k, None))
    return rows


@pytest.mark.parametrize("seed", range(4))
def test_normaliser_is_logsumexp_and_probabilities_sum_to_one(seed):
    x, _, _ = _case(seed, V=200)
    for t in (0, 7, 31):
        row = x[t, 1]
        L = O.row_lse(row)
        assert abs(L - logsumexp(row.astype(np.float64))) < 1e-12
        assert abs(np.exp(row.astype(np.float64) - L).sum() - 1.0) < 1e-12
        assert abs(O.row_lse(W.f32_to_bf16_bits(row)) - logsumexp(W.bf16_bits_to_f32(W.f32_to_bf16_bits(row)).astype(np.float64))) < 1e-12
    # closed forms: n equal entries -> x + log n; one dominant entry -> that entry
    assert abs(O.row_lse(np.full(8, 2.5, dtype=np.float32)) - (2.5 + np.log(8.0))) < 1e-14
    assert abs(O.row_lse(np.array([50.0, -50.0, -60.0], dtype=np.float32)) - 50.0) < 1e-12
    assert abs(O.row_lse(np.array([-1e4, -1e4 + 1.0], dtype=np.float32)) - (-1e4 + 1.0 + np.log1p(np.exp(-1.0)))) < 1e-9


@pytest.mark.parametrize("seed", range(4))
def test_tokens_are_those_of_the_unnormalised_decode_and_the_score_is_lower_by_the_normalisers(seed):
    x, g, _ = _case(seed)
    plain = O.greedy_rnnt(g, x)
    lsm = O.greedy_rnnt_lsm(g, x)
    assert np.array_equal(plain["tokens"], lsm["tokens"]) and np.array_equal(plain["frames"], lsm["frames"])
    assert plain["state"] == lsm["state"]
    # the score, rebuilt row by row from the un-normalised pieces: x[token] + lambda * bonus - logsumexp(row)
    total, s = 0.0, 0
    rows = _visited_rows(lsm["tokens"], lsm["frames"], x.shape[0], x.shape[1])
    assert lsm["rows"] == len(rows)
    for t, k, tok in rows:
        L = logsumexp(x[t, k].astype(np.float64))
        if tok is None:
            total += float(x[t, k, -1]) - L
        else:
            bonus, s2 = g.step(s, tok)
            total += float(x[t, k, tok]) - L + float(np.float32(g.lam) * np.float32(bonus))
            s = s2
    assert abs(lsm["score"] - total) < 1e-9 * max(1, len(rows))
    assert s == lsm["state"]


@pytest.mark.parametrize("seed", range(3))
def test_a_shift_of_every_row_changes_nothing(seed):
    """Adding a constant to all entries of a row leaves the normalised values alone (logits on a grid of 1/64 and
    shifts that are multiples of 1/4, so that the shifted logits are exact floats)."""
    x, g, _ = _case(10 + seed, grid=64)
    rng = np.random.default_rng(seed)
    shift = (rng.integers(-40, 41, size=x.shape[:2]) / 4.0).astype(np.float32)
    y = (x + shift[..., None]).astype(np.float32)
    assert np.array_equal((y - shift[..., None]).astype(np.float32), x)       # the shift is exact
    a, b = O.greedy_rnnt_lsm(g, x), O.greedy_rnnt_lsm(g, y)
    assert np.array_equal(a["tokens"], b["tokens"]) and np.array_equal(a["frames"], b["frames"]) and a["state"] == b["state"]
    assert abs(a["score"] - b["score"]) < 1e-9 * a["rows"]
    assert abs(O.row_lse(y[3, 0]) - (O.row_lse(x[3, 0]) + float(shift[3, 0]))) < 1e-12


def test_unbound_decode_is_argmax_with_normalised_score():
    x, _, _ = _case(5)
    r = O.greedy_rnnt_lsm(None, x)
    p = O.greedy_rnnt(None, x)
    assert np.array_equal(r["tokens"], p["tokens"]) and r["state"] == -1
    rows = _visited_rows(r["tokens"], r["frames"], x.shape[0], x.shape[1])
    want = sum(float(x[t, k, -1 if tok is None else tok]) - logsumexp(x[t, k].astype(np.float64)) for t, k, tok in rows)
    assert abs(r["score"] - want) < 1e-9 * len(rows)


def test_follow_mode():
    x, g, _ = _case(7)
    free = O.greedy_rnnt_lsm(g, x)
    # following its own output: nothing to follow, nothing changes
    same = O.greedy_rnnt_lsm(g, x, follow=(free["tokens"], free["frames"]), eps=1e-6)
    assert same["followed"] == 0 and same["first_mismatch"] == -1 and same["score"] == free["score"]
    assert np.array_equal(same["tokens"], free["tokens"])
    # an exact tie between two tokens in the first visited row: the free decode takes the lower id, a decoder that
    # took the higher one is followed (gap 0 < eps), and the rest of the stream continues from ITS graph state
    y = x.copy()
    y[0, 0, :] = -5.0
    y[0, 0, 20] = y[0, 0, 21] = 4.0                      # tokens 20 and 21 are case variants: the same bonus in every state
    a = O.greedy_rnnt_lsm(g, y)
    assert a["tokens"][0] == 20
    other_first = O.greedy_rnnt_lsm(g, y, follow=(np.array([21]), np.array([0])), eps=1e-6)
    assert other_first["first_mismatch"] != 0            # row 0 itself is accepted (what follows has nothing to follow)
    assert other_first["followed"] >= 1 and other_first["tokens"][0] == 21
    # a choice that is worse by far more than eps is a mismatch at that visited row
    bad_tok = int(np.argmin(y[0, 0, :-1]))
    bad = O.greedy_rnnt_lsm(g, y, follow=(np.array([bad_tok]), np.array([0])), eps=1e-6)
    assert bad["first_mismatch"] == 0
    # deviating later: the index of the visited row is reported
    toks, frs = free["tokens"].copy(), free["frames"].copy()
    j = len(toks) // 2
    toks[j] = (toks[j] + 7) % 40
    dev = O.greedy_rnnt_lsm(g, x, follow=(toks, frs), eps=1e-9)
    rows = _visited_rows(free["tokens"], free["frames"], x.shape[0], x.shape[1])
    want_row = [i for i, (t, k, tok) in enumerate(rows) if tok is not None][j]
    assert dev["first_mismatch"] == want_row
