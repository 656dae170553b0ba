"""ctypes wrapper around the CPU oracle in ``tb_oracle.c``.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the benchmark's
CPU-baseline leg.  The CUDA library and its binding never import this module, and this module
never imports them.  It holds no arithmetic of its own: every number comes out of the C file,
which is compiled with ``-O2 -ffp-contract=off`` so that a multiply and an add stay two
rounded operations.
"""
from __future__ import annotations

import ctypes as C
import hashlib
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tb_oracle.c")
_LIB = os.path.join(_HERE, "libtb_oracle.so")
_STAMP = _LIB + ".srchash"

BF16 = 0
F32 = 1


def _src_hash() -> str:
    with open(_SRC, "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or older than its source."""
    h = _src_hash()
    if not force and os.path.exists(_LIB) and os.path.exists(_STAMP):
        with open(_STAMP) as f:
            if f.read().strip() == h:
                return _LIB
    cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-Wall", "-Wextra",
           "-o", _LIB, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    with open(_STAMP, "w") as f:
        f.write(h)
    return _LIB


class _GraphStruct(C.Structure):
    _fields_ = [
        ("n_states", C.c_int32), ("n_arcs", C.c_int32), ("n_classes", C.c_int32),
        ("vocab", C.c_int32), ("max_depth", C.c_int32), ("lambda_", C.c_float),
        ("state_arc_begin", C.POINTER(C.c_int32)), ("arc_class", C.POINTER(C.c_int32)),
        ("arc_dst", C.POINTER(C.c_int32)), ("arc_w", C.POINTER(C.c_float)),
        ("state_fail", C.POINTER(C.c_int32)), ("state_bw", C.POINTER(C.c_float)),
        ("state_final", C.POINTER(C.c_float)), ("state_depth", C.POINTER(C.c_uint8)),
        ("case_class", C.POINTER(C.c_int32)),
    ]


class StreamState(C.Structure):
    """Per-slot state carried across chunks by ``stream_chunk``."""
    _fields_ = [("state", C.c_int32), ("t", C.c_int32), ("k", C.c_int32),
                ("score", C.c_float), ("n_emitted", C.c_int32)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_graph_build.restype = C.c_int
        _lib.orc_graph_build.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                         C.c_int32, C.c_float, C.POINTER(C.c_void_p)]
        _lib.orc_graph_free.restype = None
        _lib.orc_graph_free.argtypes = [C.c_void_p]
        _lib.orc_graph_get.restype = None
        _lib.orc_graph_get.argtypes = [C.c_void_p, C.POINTER(_GraphStruct)]
        _lib.orc_step.restype = None
        _lib.orc_step.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.POINTER(C.c_float), C.POINTER(C.c_int32)]
        _lib.orc_apply_final_weight.restype = C.c_float
        _lib.orc_apply_final_weight.argtypes = [C.c_void_p, C.c_int32, C.c_float]
        _lib.orc_greedy_rnnt.restype = C.c_int64
        _lib.orc_greedy_rnnt.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int32, C.c_int32, C.c_int32,
                                         C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                         C.POINTER(C.c_float), C.POINTER(C.c_int32)]
        _lib.orc_row_lse.restype = C.c_double
        _lib.orc_row_lse.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int32]
        _lib.orc_greedy_rnnt_lsm.restype = C.c_int64
        _lib.orc_greedy_rnnt_lsm.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                                             C.c_int32, C.c_void_p, C.c_void_p, C.c_int64, C.c_double, C.c_void_p, C.c_void_p,
                                             C.POINTER(C.c_double), C.POINTER(C.c_int32), C.POINTER(C.c_int64),
                                             C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        _lib.orc_stream_chunk.restype = C.c_int64
        _lib.orc_stream_chunk.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int32, C.c_int32, C.c_int32,
                                          C.c_int32, C.c_void_p, C.c_int32, C.c_int32,
                                          C.POINTER(StreamState), C.c_void_p, C.c_void_p, C.c_void_p]
        _lib.orc_beam_step.restype = None
        _lib.orc_beam_step.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_int64, C.c_int32,
                                       C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib.orc_beam_decode_opts.restype = C.c_int
        _lib.orc_beam_decode_opts.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int32, C.c_int32, C.c_int32,
                                              C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_float, C.c_void_p,
                                              C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib.orc_beam_decode.restype = C.c_int
        _lib.orc_beam_decode.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int32, C.c_int32, C.c_int32,
                                         C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.c_void_p, C.c_void_p]
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16  # raw bf16 bit patterns
    raise TypeError("logits must be float32 or uint16 (bf16 bits)")


def flatten_phrases(phrases, weights=None):
    """List of token lists -> (tokens int32, offsets int64, weights float32 or None)."""
    offs = np.zeros(len(phrases) + 1, dtype=np.int64)
    for i, p in enumerate(phrases):
        offs[i + 1] = offs[i] + len(p)
    toks = np.array([t for p in phrases for t in p], dtype=np.int32)
    w = None
    if weights is not None:
        w = np.array([x for p in weights for x in p], dtype=np.float32)
        assert w.shape == toks.shape
    return toks, offs, w


class Graph:
    """One compiled boosting graph (the oracle's own compiler)."""

    def __init__(self, phrases, vocab, case_class=None, weights=None, lam=1.0):
        toks, offs, w = flatten_phrases(phrases, weights)
        self._cc = None if case_class is None else np.ascontiguousarray(case_class, dtype=np.int32)
        h = C.c_void_p()
        rc = lib().orc_graph_build(_ptr(toks), _ptr(offs), len(phrases), _ptr(w), _ptr(self._cc),
                                   vocab, float(lam), C.byref(h))
        if rc != 0:
            raise ValueError(f"orc_graph_build failed with code {rc}")
        self.handle = h
        s = _GraphStruct()
        lib().orc_graph_get(h, C.byref(s))
        self.n_states, self.n_arcs, self.n_classes = s.n_states, s.n_arcs, s.n_classes
        self.vocab, self.max_depth, self.lam = s.vocab, s.max_depth, s.lambda_
        n, a = s.n_states, s.n_arcs

        def arr(p, cnt, dt):
            if cnt == 0:
                return np.zeros(0, dtype=dt)
            return np.ctypeslib.as_array(p, shape=(cnt,)).astype(dt, copy=True)

        self.state_arc_begin = arr(s.state_arc_begin, n + 1, np.int32)
        self.arc_class = arr(s.arc_class, a, np.int32)
        self.arc_dst = arr(s.arc_dst, a, np.int32)
        self.arc_w = arr(s.arc_w, a, np.float32)
        self.state_fail = arr(s.state_fail, n, np.int32)
        self.state_bw = arr(s.state_bw, n, np.float32)
        self.state_final = arr(s.state_final, n, np.float32)
        self.state_depth = arr(s.state_depth, n, np.uint8)
        self.case_class = arr(s.case_class, s.vocab, np.int32)

    def __del__(self):
        h = getattr(self, "handle", None)
        if h and lib is not None:          # at interpreter shutdown module globals may already be gone
            lib().orc_graph_free(h)
            self.handle = None

    def step(self, s: int, v: int):
        """(bonus, next_state) for non-blank token v in state s."""
        b = C.c_float()
        nx = C.c_int32()
        lib().orc_step(self.handle, s, v, C.byref(b), C.byref(nx))
        return b.value, nx.value


class GraphFromArrays(Graph):
    """A graph given as its arrays (built by another front end of the oracle, e.g. ``variative.py``); the decode
    functions of the C file read it through the same structure as a graph the C file built itself."""

    def __init__(self, a: dict):
        self.n_states, self.n_arcs, self.n_classes = int(a["n_states"]), int(a["n_arcs"]), int(a["n_classes"])
        self.vocab, self.max_depth, self.lam = int(a["vocab"]), int(a["max_depth"]), float(a["lam"])
        self.state_arc_begin = np.ascontiguousarray(a["state_arc_begin"], dtype=np.int32)
        self.arc_class = np.ascontiguousarray(a["arc_class"], dtype=np.int32)
        self.arc_dst = np.ascontiguousarray(a["arc_dst"], dtype=np.int32)
        self.arc_w = np.ascontiguousarray(a["arc_w"], dtype=np.float32)
        self.state_fail = np.ascontiguousarray(a["state_fail"], dtype=np.int32)
        self.state_bw = np.ascontiguousarray(a["state_bw"], dtype=np.float32)
        self.state_final = np.ascontiguousarray(a["state_final"], dtype=np.float32)
        self.state_depth = np.ascontiguousarray(a["state_depth"], dtype=np.uint8)
        self.case_class = np.ascontiguousarray(a["case_class"], dtype=np.int32)
        assert self.state_arc_begin.shape == (self.n_states + 1,) and self.arc_class.shape == (self.n_arcs,)
        s = _GraphStruct()
        s.n_states, s.n_arcs, s.n_classes = self.n_states, self.n_arcs, self.n_classes
        s.vocab, s.max_depth, s.lambda_ = self.vocab, self.max_depth, self.lam

        def p(x, t):
            return x.ctypes.data_as(C.POINTER(t))

        s.state_arc_begin = p(self.state_arc_begin, C.c_int32); s.arc_class = p(self.arc_class, C.c_int32)
        s.arc_dst = p(self.arc_dst, C.c_int32); s.arc_w = p(self.arc_w, C.c_float)
        s.state_fail = p(self.state_fail, C.c_int32); s.state_bw = p(self.state_bw, C.c_float)
        s.state_final = p(self.state_final, C.c_float); s.state_depth = p(self.state_depth, C.c_uint8)
        s.case_class = p(self.case_class, C.c_int32)
        self._struct = s                       # the arrays above stay alive with this object
        self.handle = C.cast(C.pointer(s), C.c_void_p)

    def __del__(self):                         # nothing of this graph was allocated by the C file
        self.handle = None


def apply_final_weight(graph, state: int, score) -> np.float32:
    """score + lambda * final(state): the end-of-stream charge of a hypothesis that stops in ``state``."""
    return np.float32(lib().orc_apply_final_weight(graph.handle if graph is not None else None, int(state), float(score)))


def null_step(v: int):
    b = C.c_float()
    nx = C.c_int32()
    lib().orc_step(None, -1, v, C.byref(b), C.byref(nx))
    return b.value, nx.value


def _strides3(a: np.ndarray):
    assert a.ndim == 3
    es = a.dtype.itemsize
    return np.array([a.strides[0] // es, a.strides[1] // es, a.strides[2] // es], dtype=np.int64)


def greedy_rnnt(graph, logits: np.ndarray, length=None):
    """Greedy RNNT over one stream.  logits [T, S, V+1] float32 or uint16 (bf16 bits).

    Returns dict(tokens, frames, score, state)."""
    T, S, V1 = logits.shape
    length = T if length is None else int(length)
    toks = np.zeros(T * S, dtype=np.int32)
    frs = np.zeros(T * S, dtype=np.int32)
    score = C.c_float()
    state = C.c_int32()
    st = _strides3(logits)
    n = lib().orc_greedy_rnnt(graph.handle if graph is not None else None, _ptr(logits), _dtype_code(logits),
                              T, S, V1 - 1, _ptr(st), length, _ptr(toks), _ptr(frs),
                              C.byref(score), C.byref(state))
    return dict(tokens=toks[:n].copy(), frames=frs[:n].copy(), score=np.float32(score.value), state=state.value)


def row_lse(row: np.ndarray) -> float:
    """log sum exp of one row [V+1] (float32 or bf16 bits), in double."""
    row = np.ascontiguousarray(row)
    return float(lib().orc_row_lse(_ptr(row), _dtype_code(row), 0, 1, row.shape[0] - 1))


def greedy_rnnt_lsm(graph, logits: np.ndarray, length=None, follow=None, eps: float = 0.0):
    """Greedy RNNT on log-softmax scores (double).  follow = (tokens, frames) of another decoder: its choices are
    taken wherever they are within eps of this decoder's (counted in ``followed``); a larger difference stops the
    decode (``first_mismatch`` = index of the visited row, else -1).

    Returns dict(tokens, frames, score (float64), state, followed, first_mismatch, rows)."""
    T, S, V1 = logits.shape
    length = T if length is None else int(length)
    toks = np.zeros(T * S, dtype=np.int32)
    frs = np.zeros(T * S, dtype=np.int32)
    score = C.c_double()
    state = C.c_int32()
    nf, mm, rows = C.c_int64(), C.c_int64(), C.c_int64()
    st = _strides3(logits)
    if follow is None:
        ft = ff = None
        n_follow = -1
    else:
        ft = np.ascontiguousarray(follow[0], dtype=np.int32)
        ff = np.ascontiguousarray(follow[1], dtype=np.int32)
        n_follow = len(ft)
    n = lib().orc_greedy_rnnt_lsm(graph.handle if graph is not None else None, _ptr(logits), _dtype_code(logits), T, S,
                                  V1 - 1, _ptr(st), length, _ptr(ft), _ptr(ff), n_follow, float(eps), _ptr(toks), _ptr(frs),
                                  C.byref(score), C.byref(state), C.byref(nf), C.byref(mm), C.byref(rows))
    return dict(tokens=toks[:n].copy(), frames=frs[:n].copy(), score=score.value, state=state.value,
                followed=nf.value, first_mismatch=mm.value, rows=rows.value)


def stream_chunk(graph, logits: np.ndarray, n_dur: int, t0: int, valid_frames: int, st: StreamState):
    """One chunk for one slot.  logits [chunk, S, V+1+n_dur].  Updates ``st`` in place."""
    chunk, S, W = logits.shape
    V = W - 1 - n_dur
    cap = chunk * S
    toks = np.zeros(cap, dtype=np.int32)
    frs = np.zeros(cap, dtype=np.int32)
    durs = np.zeros(cap, dtype=np.int32)
    sd = _strides3(logits)
    n = lib().orc_stream_chunk(graph.handle if graph is not None else None, _ptr(logits), _dtype_code(logits),
                               chunk, S, V, n_dur, _ptr(sd), t0, valid_frames, C.byref(st),
                               _ptr(toks), _ptr(frs), _ptr(durs))
    return dict(tokens=toks[:n].copy(), frames=frs[:n].copy(), durs=durs[:n].copy())


def beam_step(graph, rows_logits: np.ndarray, scores, states, live):
    """One beam expansion for one stream.  rows_logits [K, V+1] (row k belongs to hypothesis k).

    scores/states/live are updated in place (float32 / int32 / uint8 arrays of length K).
    Returns (parent, token) int32 arrays."""
    K, V1 = rows_logits.shape
    es = rows_logits.dtype.itemsize
    rows = np.array([k * (rows_logits.strides[0] // es) for k in range(K)], dtype=np.int64)
    par = np.zeros(K, dtype=np.int32)
    tok = np.zeros(K, dtype=np.int32)
    assert scores.dtype == np.float32 and states.dtype == np.int32 and live.dtype == np.uint8
    lib().orc_beam_step(graph.handle if graph is not None else None, _ptr(rows_logits), _dtype_code(rows_logits),
                        _ptr(rows), rows_logits.strides[1] // es, K, V1 - 1, _ptr(scores), _ptr(states),
                        _ptr(live), _ptr(par), _ptr(tok))
    return par, tok


def beam_decode(graph, logits: np.ndarray, K: int, max_len=None, merge: bool = False, prune_delta: float = -1.0):
    """Frame-synchronous beam decode of one stream.  logits [T, E, V+1].
    merge: hypotheses with equal token sequences are merged at every frame start (the best is kept).
    prune_delta >= 0: at every frame start hypotheses scoring below best - prune_delta are dropped.

    Returns dict(tokens=list of K arrays, lens, scores, states, tree [T*E, K, 2])."""
    T, E, V1 = logits.shape
    max_len = T * E if max_len is None else max_len
    out_tokens = np.zeros((K, max_len), dtype=np.int32)
    lens = np.zeros(K, dtype=np.int32)
    scores = np.zeros(K, dtype=np.float32)
    states = np.zeros(K, dtype=np.int32)
    tree = np.zeros((T * E, K, 2), dtype=np.int32)
    st = _strides3(logits)
    rc = lib().orc_beam_decode_opts(graph.handle if graph is not None else None, _ptr(logits), _dtype_code(logits),
                                    T, E, V1 - 1, _ptr(st), K, max_len, 1 if merge else 0, float(prune_delta),
                                    _ptr(out_tokens), _ptr(lens), _ptr(scores), _ptr(states), _ptr(tree))
    assert rc == 0
    return dict(tokens=[out_tokens[k, :min(lens[k], max_len)].copy() for k in range(K)], lens=lens,
                scores=scores, states=states, tree=tree)
