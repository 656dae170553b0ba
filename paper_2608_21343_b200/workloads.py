"""Seeded synthetic inputs for the five decode workloads.

This module only *makes inputs*: vocabularies with case siblings, phrase lists, logit tensors
with planted phrases, and the stream-churn schedule of the streaming workload.  It contains
none of the boosting method's arithmetic (no graph, no bonus, no selection) and is the one
module that both the CUDA path's tests/benchmark and the CPU oracle's tests read, so that both
sides consume the same bits.  Everything is derived from ``numpy.random.default_rng`` streams
keyed by (workload seed, stream index); nothing is read from disk.

The shapes follow the paper's production setting (Sec. 3.3-3.4 and Table 3: 128 concurrent
streams, per-stream lists of target phrases plus distractors, cased model output against
uncased lists); the logits are synthetic stand-ins for a joint network's output.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Optional

import numpy as np

BLANK_BIAS = 3.0


# ----------------------------------------------------------------------------------------------
# dtype helpers (storage formats only)
# ----------------------------------------------------------------------------------------------

def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_dtype(a: np.ndarray, dtype: str) -> np.ndarray:
    """float32 array whose values are representable in ``dtype`` ('bf16' or 'f32')."""
    if dtype == "f32":
        return np.ascontiguousarray(a, dtype=np.float32)
    return bf16_bits_to_f32(f32_to_bf16_bits(a))


def to_storage(a: np.ndarray, dtype: str) -> np.ndarray:
    """float32 values -> the array handed to a decoder: float32, or uint16 holding bf16 bits."""
    return np.ascontiguousarray(a, dtype=np.float32) if dtype == "f32" else f32_to_bf16_bits(a)


# ----------------------------------------------------------------------------------------------
# vocabulary with case siblings
# ----------------------------------------------------------------------------------------------

@dataclass
class Vocab:
    """V non-blank tokens (blank id = V).  The first 3*n3 ids are n3 case classes with three
    siblings each (3c = lower, 3c+1 = UPPER, 3c+2 = Title); the rest are case-neutral tokens,
    one class each."""
    V: int
    n3: int
    n_classes: int
    case_class: np.ndarray  # int32 [V]

    def token_of(self, cls: int, sibling: int = 0) -> int:
        if cls < self.n3:
            return 3 * cls + sibling
        return 3 * self.n3 + (cls - self.n3)

    def recase(self, tok: int, sibling: int) -> int:
        c = int(self.case_class[tok])
        return self.token_of(c, sibling) if c < self.n3 else tok


def make_vocab(V: int) -> Vocab:
    n3 = (80 * V) // 256
    neutral = V - 3 * n3
    cc = np.empty(V, dtype=np.int32)
    cc[: 3 * n3] = np.repeat(np.arange(n3, dtype=np.int32), 3)
    cc[3 * n3:] = n3 + np.arange(neutral, dtype=np.int32)
    return Vocab(V=V, n3=n3, n_classes=n3 + neutral, case_class=cc)


# ----------------------------------------------------------------------------------------------
# workload descriptions
# ----------------------------------------------------------------------------------------------

@dataclass
class Workload:
    name: str
    cid: int                 # 1..5
    seed: int
    B: int                   # streams (slots for the streaming workload)
    T: int                   # frames per stream (upper bound of lengths for streaming)
    S: int                   # rows (max symbols / expansions) per frame
    V: int
    dtype: str               # 'bf16' or 'f32'
    n_phrases: int
    len_lo: int
    len_hi: int
    token_draw: str          # 'uniform' over tokens or 'zipf' over classes
    n_plants: int
    K: int = 1               # beams
    n_dur: int = 0           # TDT duration logits
    chunk: int = 0           # streaming chunk (frames)
    n_shared: int = 0        # distractor phrases shared by all streams
    near_miss_frac: float = 0.0
    recase_mode: str = "random"   # 'half' (workload 1) or 'random'
    T_lo: int = 0            # streaming: stream length ~ U[T_lo, T]
    n_phrases_lo: int = 0    # streaming: list size ~ U[n_phrases_lo, n_phrases]
    lam: float = 1.0
    vocab: Vocab = field(default=None, repr=False)

    @property
    def row_width(self) -> int:
        return self.V + 1 + self.n_dur


def get_workload(cid: int, **over) -> Workload:
    """The five workloads; keyword overrides give the scaled-down cases the tests use."""
    base = {
        1: Workload("tiny_greedy_rnnt", 1, 0, B=4, T=100, S=3, V=256, dtype="f32", n_phrases=10, len_lo=1,
                    len_hi=4, token_draw="uniform", n_plants=10, recase_mode="half"),
        2: Workload("batched_greedy_rnnt", 2, 2000, B=128, T=750, S=3, V=1024, dtype="bf16", n_phrases=100,
                    len_lo=1, len_hi=6, token_draw="zipf", n_plants=20),
        3: Workload("large_lists_greedy_rnnt", 3, 3000, B=64, T=750, S=3, V=1024, dtype="bf16", n_phrases=1000,
                    len_lo=3, len_hi=10, token_draw="zipf", n_plants=50, n_shared=4000, near_miss_frac=1.0 / 3),
        4: Workload("beam_rnnt", 4, 4000, B=32, T=500, S=2, V=1024, dtype="bf16", n_phrases=300, len_lo=1,
                    len_hi=6, token_draw="zipf", n_plants=20, K=4),
        5: Workload("streaming_tdt_churn", 5, 5000, B=512, T=1500, S=3, V=1024, dtype="bf16", n_phrases=500,
                    len_lo=1, len_hi=6, token_draw="zipf", n_plants=0, n_dur=5, chunk=8, T_lo=200,
                    n_phrases_lo=50),
    }[cid]
    w = replace(base, **over)
    w.vocab = make_vocab(w.V)
    return w


# ----------------------------------------------------------------------------------------------
# phrases
# ----------------------------------------------------------------------------------------------

def _rng(w: Workload, *key) -> np.random.Generator:
    return np.random.default_rng(np.random.SeedSequence([w.seed, *[int(k) for k in key]]))


def _zipf_table(w: Workload):
    """Class probabilities ~ 1/rank^1.1 with the ranks scattered over class ids by a permutation
    that is fixed per workload."""
    C = w.vocab.n_classes
    p = 1.0 / np.arange(1, C + 1, dtype=np.float64) ** 1.1
    p /= p.sum()
    perm = _rng(w, 777).permutation(C)
    return perm, np.cumsum(p)


def draw_phrases(w: Workload, rng: np.random.Generator, n: int, len_lo=None, len_hi=None) -> List[List[int]]:
    """n phrases as token lists.  'zipf': classes ~ Zipf(1.1), listed with their lower-case
    sibling (user lists are usually unformatted); 'uniform': tokens uniform over the vocabulary."""
    len_lo = w.len_lo if len_lo is None else len_lo
    len_hi = w.len_hi if len_hi is None else len_hi
    lens = rng.integers(len_lo, len_hi + 1, size=n)
    total = int(lens.sum())
    if w.token_draw == "uniform":
        toks = rng.integers(0, w.V, size=total)
    else:
        perm, cdf = _zipf_table(w)
        ranks = np.searchsorted(cdf, rng.random(total), side="right").clip(0, len(cdf) - 1)
        cls = perm[ranks]
        v = w.vocab
        toks = np.where(cls < v.n3, 3 * cls, 3 * v.n3 + (cls - v.n3))
    out, pos = [], 0
    for L in lens:
        out.append([int(t) for t in toks[pos:pos + L]])
        pos += L
    return out


def stream_phrases(w: Workload, b: int) -> List[List[int]]:
    """The phrase list of stream b: its own phrases first, then the shared distractors."""
    rng = _rng(w, 1, b)
    n_local = w.n_phrases
    if w.n_phrases_lo:
        n_local = int(rng.integers(w.n_phrases_lo, w.n_phrases + 1))
    local = draw_phrases(w, rng, n_local)
    if w.n_shared:
        local = local + draw_phrases(w, _rng(w, 2), w.n_shared)
    return local


# ----------------------------------------------------------------------------------------------
# logits with planted phrases
# ----------------------------------------------------------------------------------------------

def _render(w: Workload, phrase: List[int], mode: int) -> List[int]:
    """mode 0: as listed; 1: UPPER; 2: Title on the first token, lower after; 3: every token
    moved to its next sibling (a casing different from the listed one)."""
    v = w.vocab
    if mode == 0:
        return list(phrase)
    if mode == 1:
        return [v.recase(t, 1) for t in phrase]
    if mode == 2:
        return [v.recase(t, 2 if i == 0 else 0) for i, t in enumerate(phrase)]
    out = []
    for t in phrase:
        c = int(v.case_class[t])
        out.append(v.token_of(c, (t - 3 * c + 1) % 3) if c < v.n3 else t)
    return out


def _plant_tokens(x: np.ndarray, w: Workload, toks: List[int], t0: int, rng: np.random.Generator):
    """Write one rendered phrase into rows (t0+j, 0): the token's logit becomes
    (largest other token logit of that row, blank included) - m with m ~ U[0, 1.5]; the blank of
    row (t0+j, 1) gets a further +3 so that the frame normally closes after one symbol."""
    W1 = w.V + 1
    for j, tok in enumerate(toks):
        t = t0 + j
        if t >= x.shape[0]:
            break
        row = x[t, 0, :W1]
        others = np.delete(row, tok)
        m = np.float32(rng.uniform(0.0, 1.5))
        row[tok] = round_to_dtype(np.array([others.max() - m], dtype=np.float32), w.dtype)[0]
        if w.S > 1:
            x[t, 1, w.V] = round_to_dtype(np.array([x[t, 1, w.V] + BLANK_BIAS], dtype=np.float32), w.dtype)[0]


def stream_logits_f32(w: Workload, b: int, phrases: Optional[List[List[int]]] = None,
                      T: Optional[int] = None) -> np.ndarray:
    """float32 array [T, S, V+1+n_dur] holding values representable in the workload's dtype."""
    rng = _rng(w, 3, b)
    T = w.T if T is None else T
    x = rng.standard_normal((T, w.S, w.row_width), dtype=np.float32)
    x[:, :, w.V] += np.float32(BLANK_BIAS)
    x = round_to_dtype(x, w.dtype)
    n_plants = w.n_plants
    if n_plants <= 0 or T < n_plants:
        return x
    phrases = stream_phrases(w, b) if phrases is None else phrases
    n_own = len(phrases) - w.n_shared
    prng = _rng(w, 4, b)
    seg = T // n_plants
    prefixes = None
    for i in range(n_plants):
        if w.recase_mode == "half":
            p = phrases[i % n_own]
            mode = 3 if (i % 2) else 0
        else:
            p = phrases[int(prng.integers(0, n_own))]
            mode = int(prng.integers(0, 3))
        toks = _render(w, p, mode)
        if w.near_miss_frac > 0 and prng.random() < w.near_miss_frac and len(toks) > 1:
            # keep 1-3 leading tokens, then a token whose class continues no listed phrase here
            if prefixes is None:
                cc = w.vocab.case_class
                prefixes = {tuple(int(cc[t]) for t in q[:n]) for q in phrases for n in range(1, len(q) + 1)}
            keep = int(prng.integers(1, min(3, len(toks) - 1) + 1))
            head = tuple(int(w.vocab.case_class[t]) for t in toks[:keep])
            for _ in range(64):
                c = int(prng.integers(0, w.vocab.n_classes))
                if head + (c,) not in prefixes:
                    toks = toks[:keep] + [w.vocab.token_of(c, 0)]
                    break
        t0 = i * seg + int(prng.integers(0, max(1, seg - len(toks))))
        _plant_tokens(x, w, toks, t0, prng)
    return x


def stream_length(w: Workload, b: int) -> int:
    if w.T_lo:
        return int(_rng(w, 5, b).integers(w.T_lo, w.T + 1))
    return w.T


def stream_inputs(w: Workload, b: int) -> dict:
    """Everything stream b needs: phrases, logits in storage format [len, S, W], its length."""
    phrases = stream_phrases(w, b)
    L = stream_length(w, b)
    x = stream_logits_f32(w, b, phrases, T=L)
    return dict(phrases=phrases, logits=to_storage(x, w.dtype), length=L)


def batch_inputs(w: Workload, streams=None) -> dict:
    """Stacked inputs for the offline workloads (1-4): logits [B, T, S, V+1] in storage format
    and one phrase list per stream."""
    streams = list(range(w.B)) if streams is None else list(streams)
    np_dt = np.float32 if w.dtype == "f32" else np.uint16
    logits = np.empty((len(streams), w.T, w.S, w.row_width), dtype=np_dt)
    phrases = []
    for i, b in enumerate(streams):
        d = stream_inputs(w, b)
        logits[i] = d["logits"]
        phrases.append(d["phrases"])
    return dict(logits=logits, phrases=phrases, streams=streams)


# ----------------------------------------------------------------------------------------------
# streaming workload with stream churn
# ----------------------------------------------------------------------------------------------

class ChurnSchedule:
    """Feeds the streaming workload chunk by chunk.

    Slot i starts with stream i.  A slot whose stream has no frames left after a chunk is
    refilled, before the next chunk, with the next unused stream id (slots visited in ascending
    order) and that stream's own phrase list; the new stream starts at frame 0 of the next chunk.
    ``next_chunk`` returns the chunk tensor [slots, chunk, S, W] in storage format, the per-slot
    total stream lengths, and the list of (slot, stream id, phrases) binds that must be applied
    before this chunk is decoded."""

    def __init__(self, w: Workload, workers: int = 0):
        """workers > 0: the inputs of the streams that come next are generated ahead of time on that many
        threads (every stream has its own generator, so the bits do not depend on it)."""
        assert w.chunk > 0
        self.w = w
        self._pool = None
        self._ahead = {}
        if workers > 0:
            from concurrent.futures import ThreadPoolExecutor
            self._pool = ThreadPoolExecutor(max_workers=workers)
            self._n_ahead = 4 * workers
        self.next_stream = w.B
        self.stream_of = list(range(w.B))
        self.offset = [0] * w.B        # frames of the current stream already served
        self.data = [None] * w.B
        self.pending = list(range(w.B))
        np_dt = np.float32 if w.dtype == "f32" else np.uint16
        self.zero_chunk = np.zeros((w.chunk, w.S, w.row_width), dtype=np_dt)

    def _inputs(self, stream_id: int) -> dict:
        if self._pool is None:
            return stream_inputs(self.w, stream_id)
        # stream ids are handed out in ascending order: keep the next few in flight
        hi = max(stream_id + 1, min(self.next_stream, stream_id + 1) + self._n_ahead)
        if stream_id < self.w.B:
            hi = max(hi, self.w.B)          # the first chunk asks for all slots' streams at once
        for sid in range(stream_id, hi):
            if sid not in self._ahead:
                self._ahead[sid] = self._pool.submit(stream_inputs, self.w, sid)
        return self._ahead.pop(stream_id).result()

    def close(self):
        if self._pool is not None:
            for f in self._ahead.values():
                f.cancel()
            self._pool.shutdown(wait=True)
            self._pool = None
            self._ahead = {}

    def next_chunk(self):
        w = self.w
        binds = []
        for slot in self.pending:
            d = self._inputs(self.stream_of[slot])
            self.data[slot] = d
            self.offset[slot] = 0
            binds.append((slot, self.stream_of[slot], d["phrases"]))
        self.pending = []
        chunk = np.empty((w.B, w.chunk, w.S, w.row_width), dtype=self.zero_chunk.dtype)
        lengths = np.empty(w.B, dtype=np.int32)
        for slot in range(w.B):
            d, off = self.data[slot], self.offset[slot]
            part = d["logits"][off:off + w.chunk]
            chunk[slot, :part.shape[0]] = part
            if part.shape[0] < w.chunk:
                chunk[slot, part.shape[0]:] = self.zero_chunk[part.shape[0]:]
            lengths[slot] = d["length"]
            self.offset[slot] = off + w.chunk
            if self.offset[slot] >= d["length"]:
                self.stream_of[slot] = self.next_stream
                self.next_stream += 1
                self.pending.append(slot)
        return chunk, lengths, binds


# ----------------------------------------------------------------------------------------------
# piece vocabularies and phrases as strings (inputs of the variative compile; Sec. 2.1 para. 4-5)
# ----------------------------------------------------------------------------------------------

def make_piece_vocab(seed: int, letters: int = 12, merged: int = 200, max_len: int = 4) -> List[bytes]:
    """A synthetic piece vocabulary (stand-in for a SentencePiece model's): every letter as a piece of its own
    in both cases (a, A, b, B, ...), then ``merged`` distinct lower-case pieces of 2..max_len letters; about
    half of them also have a Title-case piece and a quarter an UPPER-case one -- a vocabulary does not hold
    every case variant of every piece."""
    rng = np.random.default_rng([seed, 77001])
    out: List[bytes] = []
    for i in range(letters):
        out.append(bytes([97 + i]))
        out.append(bytes([65 + i]))
    seen = set()
    merged = min(merged, sum(letters ** n for n in range(2, max_len + 1)))   # no more than there are
    while len(seen) < merged:
        n = int(rng.integers(2, max_len + 1))
        seen.add(bytes(int(x) + 97 for x in rng.integers(0, letters, size=n)))
    for p in sorted(seen):
        out.append(p)
        r = rng.random()
        if r < 0.5:
            out.append(bytes([p[0] - 32]) + p[1:])
        if r < 0.25:
            out.append(bytes(b - 32 for b in p))
    return out


def draw_string_phrases(seed: int, pieces: List[bytes], n: int, len_lo: int = 1, len_hi: int = 4) -> List[bytes]:
    """``n`` phrases, each the concatenation of len_lo..len_hi pieces drawn from the lower-case pieces (so that
    merged pieces occur inside phrases), given in lower case as user lists usually are."""
    rng = np.random.default_rng([seed, 77002])
    lower = [p for p in pieces if p == p.lower()]
    out = []
    for _ in range(n):
        k = int(rng.integers(len_lo, len_hi + 1))
        out.append(b"".join(lower[int(i)] for i in rng.integers(0, len(lower), size=k)))
    return out


def random_spelling(rng: np.random.Generator, phrase: bytes, pieces: List[bytes], casing: Optional[int] = None) -> List[int]:
    """Token ids of one way the model could emit ``phrase``: a casing (0 lower, 1 UPPER, 2 Title, 3 random per
    letter; drawn if None) and a random segmentation of that spelling into pieces the vocabulary holds."""
    ids = {}
    for t, p in enumerate(pieces):
        ids.setdefault(p, t)
    longest = max(len(p) for p in pieces)
    mode = int(rng.integers(0, 4)) if casing is None else casing
    low = phrase.lower()
    if mode == 0:
        s = low
    elif mode == 1:
        s = low.upper()
    elif mode == 2:
        s = low[:1].upper() + low[1:]
    else:
        s = bytes((b - 32 if (97 <= b <= 122 and rng.random() < 0.5) else b) for b in low)
    toks, i = [], 0
    while i < len(s):
        cand = [m for m in range(1, min(longest, len(s) - i) + 1) if s[i:i + m] in ids]
        m = cand[int(rng.integers(0, len(cand)))]
        toks.append(ids[s[i:i + m]])
        i += m
    return toks


@dataclass
class _RowShape:
    V: int
    S: int
    dtype: str


def variative_stream_logits(seed: int, b: int, pieces: List[bytes], phrases: List[bytes], T: int, S: int = 3,
                            dtype: str = "bf16", n_plants: int = 20) -> np.ndarray:
    """Logits [T, S, V+1] in storage format for stream ``b`` of a variative-list decode: the same recipe as the
    token-list workloads (N(0,1) token logits, blank +3), with ``n_plants`` phrases planted as random spellings
    (casing and segmentation drawn per plant), one piece per frame."""
    shp = _RowShape(V=len(pieces), S=S, dtype=dtype)
    rng = np.random.default_rng([seed, 77003, b])
    x = rng.standard_normal((T, S, shp.V + 1), dtype=np.float32)
    x[:, :, shp.V] += np.float32(BLANK_BIAS)
    x = round_to_dtype(x, dtype)
    if n_plants > 0 and len(phrases) > 0 and T >= n_plants:
        seg = T // n_plants
        for i in range(n_plants):
            toks = random_spelling(rng, phrases[int(rng.integers(0, len(phrases)))], pieces)
            t0 = i * seg + int(rng.integers(0, max(1, seg - len(toks))))
            _plant_tokens(x, shp, toks, t0, rng)
    return to_storage(x, dtype)
