"""Python side of the C-ABI library ``libtb.so``: the same calls with the same names, taking
torch tensors for device memory and numpy arrays for host memory.  Argument marshalling only --
every step of the decode path runs in the library's CUDA kernels.  There is no CPU fallback: if
the library cannot be loaded, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("TB_LIB_PATH") or os.path.join(_HERE, "libtb.so")

if not os.path.exists(LIB_PATH):
    raise RuntimeError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2608_21343_b200.build` "
        "(or __graft_entry__.build()); this package has no fallback path")
_lib = C.CDLL(LIB_PATH)

TB_OK = 0
TB_ERR_INVALID_ARG, TB_ERR_OOM, TB_ERR_CUDA, TB_ERR_ARENA_FULL, TB_ERR_BAD_SLOT, TB_ERR_DEVICE_STATUS = -1, -2, -3, -4, -5, -6
TB_ERR_IO = -7
TB_FRAME_SAME, TB_FRAME_NEW, TB_FRAME_NEW_MERGE = 0, 1, 2
TB_BF16, TB_F32 = 0, 1
TB_COMPILE_PAGEABLE = 1


class TbError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {tb_strerror(code)} ({code})")


class _GraphView(C.Structure):
    _fields_ = [
        ("n_states", C.c_int32), ("n_arcs", C.c_int32), ("n_classes", C.c_int32), ("vocab", C.c_int32),
        ("max_depth", C.c_int32), ("lambda_", C.c_float),
        ("state_arc_begin", C.POINTER(C.c_int32)), ("arc_class", C.POINTER(C.c_int32)),
        ("arc_dst", C.POINTER(C.c_int32)), ("arc_w", C.POINTER(C.c_float)),
        ("state_fail", C.POINTER(C.c_int32)), ("state_bw", C.POINTER(C.c_float)),
        ("state_final", C.POINTER(C.c_float)), ("state_depth", C.POINTER(C.c_uint8)),
        ("case_class", C.POINTER(C.c_int32)),
    ]


_vp, _i32, _i64 = C.c_void_p, C.c_int32, C.c_int64
_SIGS = {
    "tb_strerror": (C.c_char_p, [C.c_int]),
    "tb_graph_compile": (C.c_int, [_vp, _vp, _i32, _vp, _vp, _i32, C.c_float, C.c_uint32, C.POINTER(_vp)]),
    "tb_piece_classes": (C.c_int, [_vp, _vp, _i32, _vp, C.POINTER(_i32)]),
    "tb_graph_compile_variative": (C.c_int, [_vp, _vp, _i32, _vp, _vp, _vp, _i32, C.c_float, C.c_float, C.c_uint32,
                                             C.POINTER(_vp)]),
    "tb_graph_view_get": (C.c_int, [_vp, C.POINTER(_GraphView)]),
    "tb_graph_free": (None, [_vp]),
    "tb_graph_save": (C.c_int, [_vp, C.c_char_p]),
    "tb_graph_load": (C.c_int, [C.c_char_p, C.POINTER(_vp)]),
    "tb_cache_create": (C.c_int, [C.c_size_t, C.POINTER(_vp)]),
    "tb_cache_destroy": (None, [_vp]),
    "tb_cache_compile": (C.c_int, [_vp, _vp, _vp, _i32, _vp, _vp, _i32, C.c_float, C.c_uint32, C.POINTER(_vp),
                                   C.POINTER(_i32)]),
    "tb_cache_compile_variative": (C.c_int, [_vp, _vp, _vp, _i32, _vp, _vp, _vp, _i32, C.c_float, C.c_float, C.c_uint32,
                                             C.POINTER(_vp), C.POINTER(_i32)]),
    "tb_cache_stats": (C.c_int, [_vp, C.POINTER(_i64), C.POINTER(_i64), C.POINTER(_i64), C.POINTER(C.c_size_t),
                                 C.POINTER(_i64)]),
    "tb_batch_register_model": (C.c_int, [_vp, _vp, C.POINTER(_i32), _vp]),
    "tb_batch_bind_model": (C.c_int, [_vp, _i32, _i32, _vp]),
    "tb_batch_unregister_model": (C.c_int, [_vp, _i32]),
    "tb_batch_bind_models": (C.c_int, [_vp, _i32, _vp, _vp, _vp]),
    "tb_batch_create": (C.c_int, [_i32, _vp, _i32, _i32, _i32, C.c_size_t, C.c_int, C.POINTER(_vp)]),
    "tb_batch_destroy": (None, [_vp]),
    "tb_batch_bind_stream": (C.c_int, [_vp, _i32, _vp, _vp]),
    "tb_batch_bind_streams": (C.c_int, [_vp, _i32, _vp, _vp, _vp]),
    "tb_batch_status": (C.c_int, [_vp, C.POINTER(_i32), _vp]),
    "tb_batch_set_flags": (C.c_int, [_vp, C.c_uint32]),
    "tb_batch_set_greedy_plan": (C.c_int, [_vp, _i32, _i32, _i32]),
    "tb_batch_last_greedy_kernel": (C.c_int, [_vp, C.POINTER(_i32), C.POINTER(_i32), C.POINTER(_i32)]),
    "tb_batch_bind_counts": (C.c_int, [_vp, C.POINTER(_i64), C.POINTER(_i64)]),
    "tb_greedy_decode": (C.c_int, [_vp, _vp, C.c_int, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "tb_stream_chunk": (C.c_int, [_vp, _vp, C.c_int, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp,
                                  _vp, _vp, _vp]),
    "tb_stream_chunk_binds": (C.c_int, [_vp, _i32, _vp, _vp, _vp, C.c_int, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp,
                                        _vp, _vp, _vp, _vp, _vp]),
    "tb_beam_reset": (C.c_int, [_vp]),
    "tb_beam_step": (C.c_int, [_vp, _vp, C.c_int, _i32, _i32, _i64, _i64, _i32, _vp, _vp, _vp, _vp, _vp, _vp]),
    "tb_beam_backtrace": (C.c_int, [_vp, _i32, _i32, _i32, _vp, _vp, _vp]),
    "tb_beam_frames": (C.c_int, [_vp, _vp, C.c_int, _i32, _i32, _i32, _i32, _i64, _i64, _i64, _i32, _vp, _vp, _vp, _vp, _vp,
                                 _vp]),
    "tb_apply_final_weights": (C.c_int, [_vp, _i32, _i32, _vp, _vp, _vp]),
    "tb_beam_reset_slots": (C.c_int, [_vp, _i32, _vp, _vp]),
    "tb_beam_start_slots": (C.c_int, [_vp, _i32, _vp, _i32, _vp, _vp, _vp, _vp]),
    "tb_beam_chunk": (C.c_int, [_vp, _vp, C.c_int, _i32, _i32, _i32, _i32, _i64, _i64, _i64, _i32, _vp, _vp, _vp, _vp, _vp,
                                _vp, _vp]),
    "tb_beam_backtrace_slots": (C.c_int, [_vp, _i32, _i32, _i32, _vp, _vp, _vp]),
    "tb_beam_backtrace_slot_list": (C.c_int, [_vp, _i32, _vp, _i32, _i32, _vp, _vp, _vp]),
    "tb_apply_final_weights_slots": (C.c_int, [_vp, _i32, _vp, _i32, _vp, _vp, _vp]),
    "tb_batch_set_beam_prune": (C.c_int, [_vp, C.c_float]),
    "tb_greedy_decode_noalloc": (C.c_int, [C.c_int, _vp, C.c_int, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp,
                                           _vp, _vp, _vp]),
}
for _name, (_res, _args) in _SIGS.items():
    _fn = getattr(_lib, _name)       # AttributeError here = the library lacks a declared symbol
    _fn.restype, _fn.argtypes = _res, _args

EXPORTED = tuple(_SIGS)


def tb_strerror(code: int) -> str:
    return _lib.tb_strerror(code).decode()


def _check(code: int, where: str):
    if code != TB_OK:
        raise TbError(code, where)


def _host(a, dtype):
    return None if a is None else np.ascontiguousarray(a, dtype=dtype)


def _hp(a):
    # (the address from the array interface: numpy's .ctypes helper object costs several microseconds per call)
    if a is None or isinstance(a, C.Array):        # (a ctypes array is passed as it is)
        return a
    return _vp(a.__array_interface__["data"][0])


def _slots(slots):
    """A short list of slot indices as (n, host int32 array for the call)."""
    if isinstance(slots, (list, tuple)):         # (the usual case: no numpy array is built for a handful of indices)
        n = len(slots)
        return n, ((_i32 * n)(*slots) if n else None)
    a = _host(slots, np.int32)
    return len(a), _hp(a)


def _dp(t):
    # (an address as a plain int: ctypes converts it for a pointer argument; whatever is not a CUDA tensor is refused
    # here, before its address could reach a kernel)
    if t is None:
        return None
    if not t.is_cuda:
        raise TypeError("expected a CUDA tensor")
    return t.data_ptr()


_raw_current_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream(stream):
    if stream is None:
        if _raw_current_stream is not None:       # the current stream's handle without building a Stream object
            return _raw_current_stream(torch.cuda.current_device())
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def _logit_dtype(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return TB_BF16
    if t.dtype == torch.float32:
        return TB_F32
    raise TypeError("logits must be bfloat16 or float32")


class Graph:
    """A compiled boosting graph (host object)."""

    def __init__(self, handle):
        self.handle = handle

    def view(self) -> dict:
        v = _GraphView()
        _check(_lib.tb_graph_view_get(self.handle, C.byref(v)), "tb_graph_view_get")
        n, a = v.n_states, v.n_arcs

        def arr(p, cnt, dt):
            return np.ctypeslib.as_array(p, shape=(cnt,)).astype(dt, copy=True) if cnt else np.zeros(0, dtype=dt)

        return dict(
            n_states=n, n_arcs=a, n_classes=v.n_classes, vocab=v.vocab, max_depth=v.max_depth, lam=v.lambda_,
            state_arc_begin=arr(v.state_arc_begin, n + 1, np.int32), arc_class=arr(v.arc_class, a, np.int32),
            arc_dst=arr(v.arc_dst, a, np.int32), arc_w=arr(v.arc_w, a, np.float32),
            state_fail=arr(v.state_fail, n, np.int32), state_bw=arr(v.state_bw, n, np.float32),
            state_final=arr(v.state_final, n, np.float32), state_depth=arr(v.state_depth, n, np.uint8),
            case_class=arr(v.case_class, v.vocab, np.int32))

    def free(self):
        if self.handle and _lib is not None:
            _lib.tb_graph_free(self.handle)
            self.handle = None

    def __del__(self):
        self.free()


def tb_graph_compile(phrases, vocab: int, case_class=None, token_weights=None, lam: float = 1.0, flags: int = 0) -> Graph:
    """phrases: list of token lists, or a (tokens, offsets) pair of arrays."""
    if isinstance(phrases, tuple):
        toks, offs = _host(phrases[0], np.int32), _host(phrases[1], np.int64)
        n = len(offs) - 1
        w = _host(token_weights, np.float32)
    else:
        n = len(phrases)
        offs = np.zeros(n + 1, dtype=np.int64)
        if n:
            offs[1:] = np.cumsum([len(p) for p in phrases])
        toks = np.array([t for p in phrases for t in p], dtype=np.int32)
        w = None if token_weights is None else np.array([x for p in token_weights for x in p], dtype=np.float32)
    cc = _host(case_class, np.int32)
    h = _vp()
    _check(_lib.tb_graph_compile(_hp(toks), _hp(offs), n, _hp(w), _hp(cc), vocab, float(lam), flags, C.byref(h)),
           "tb_graph_compile")
    return Graph(h)


def _flatten_phrases(phrases, token_weights):
    if isinstance(phrases, tuple):
        toks, offs = _host(phrases[0], np.int32), _host(phrases[1], np.int64)
        return toks, offs, len(offs) - 1, _host(token_weights, np.float32)
    n = len(phrases)
    offs = np.zeros(n + 1, dtype=np.int64)
    if n:
        offs[1:] = np.cumsum([len(p) for p in phrases])
    toks = np.array([t for p in phrases for t in p], dtype=np.int32)
    w = None if token_weights is None else np.array([x for p in token_weights for x in p], dtype=np.float32)
    return toks, offs, n, w


def tb_graph_save(graph: Graph, path: str):
    _check(_lib.tb_graph_save(graph.handle, os.fsencode(path)), "tb_graph_save")


def tb_graph_load(path: str) -> Graph:
    h = _vp()
    _check(_lib.tb_graph_load(os.fsencode(path), C.byref(h)), "tb_graph_load")
    return Graph(h)


class Cache:
    """Compiled graphs kept in host memory (tb_cache)."""

    def __init__(self, handle):
        self.handle = handle

    def stats(self) -> dict:
        h, m, e, n = _i64(), _i64(), _i64(), _i64()
        used = C.c_size_t()
        _check(_lib.tb_cache_stats(self.handle, C.byref(h), C.byref(m), C.byref(e), C.byref(used), C.byref(n)),
               "tb_cache_stats")
        return dict(hits=h.value, misses=m.value, evictions=e.value, bytes_used=used.value, entries=n.value)

    def destroy(self):
        if self.handle and _lib is not None:
            _lib.tb_cache_destroy(self.handle)
            self.handle = None

    def __del__(self):
        self.destroy()


def tb_cache_create(capacity_bytes: int) -> Cache:
    h = _vp()
    _check(_lib.tb_cache_create(capacity_bytes, C.byref(h)), "tb_cache_create")
    return Cache(h)


def tb_cache_compile(cache: Cache, phrases, vocab: int, case_class=None, token_weights=None, lam: float = 1.0,
                     flags: int = 0):
    """Returns (graph, hit)."""
    toks, offs, n, w = _flatten_phrases(phrases, token_weights)
    cc = _host(case_class, np.int32)
    h, hit = _vp(), _i32()
    _check(_lib.tb_cache_compile(cache.handle, _hp(toks), _hp(offs), n, _hp(w), _hp(cc), vocab, float(lam), flags,
                                 C.byref(h), C.byref(hit)), "tb_cache_compile")
    return Graph(h), bool(hit.value)


def tb_cache_compile_variative(cache: Cache, phrases, pieces, phrase_weights=None, tau: float = 1.0, lam: float = 1.0,
                               flags: int = 0):
    """Returns (graph, hit).  ``pieces`` may be the (bytes, offsets) pair made once by ``_flat_bytes``."""
    pf, po = _flat_bytes(phrases)
    vf, vo = pieces if isinstance(pieces, tuple) else _flat_bytes(pieces)
    w = _host(phrase_weights, np.float32)
    h, hit = _vp(), _i32()
    _check(_lib.tb_cache_compile_variative(cache.handle, _hp(pf), _hp(po), len(phrases), _hp(w), _hp(vf), _hp(vo),
                                           len(vo) - 1, float(tau), float(lam), flags, C.byref(h), C.byref(hit)),
           "tb_cache_compile_variative")
    return Graph(h), bool(hit.value)


def tb_batch_register_model(batch, graph: Graph, stream=None) -> int:
    mid = _i32()
    _check(_lib.tb_batch_register_model(batch.handle, graph.handle, C.byref(mid), _stream(stream)),
           "tb_batch_register_model")
    return mid.value


def tb_batch_bind_model(batch, slot: int, model_id: int, stream=None):
    _check(_lib.tb_batch_bind_model(batch.handle, slot, model_id, _stream(stream)), "tb_batch_bind_model")


def tb_batch_bind_models(batch, slots, model_ids, stream=None):
    sl, ids = _host(slots, np.int32), _host(model_ids, np.int32)
    assert sl.shape == ids.shape
    _check(_lib.tb_batch_bind_models(batch.handle, len(sl), _hp(sl), _hp(ids), _stream(stream)), "tb_batch_bind_models")


def tb_batch_unregister_model(batch, model_id: int):
    _check(_lib.tb_batch_unregister_model(batch.handle, model_id), "tb_batch_unregister_model")


def _flat_bytes(items):
    """List of byte strings -> (bytes uint8, offsets int64)."""
    offs = np.zeros(len(items) + 1, dtype=np.int64)
    if len(items):
        offs[1:] = np.cumsum([len(x) for x in items])
    flat = np.frombuffer(b"".join(items), dtype=np.uint8).copy() if offs[-1] else np.zeros(0, dtype=np.uint8)
    return flat, offs


def tb_piece_classes(pieces):
    """pieces: list of byte strings (the vocabulary's spellings).  Returns (case_class int32 [V], n_classes)."""
    flat, offs = _flat_bytes(pieces)
    cc = np.zeros(len(pieces), dtype=np.int32)
    n = _i32()
    _check(_lib.tb_piece_classes(_hp(flat), _hp(offs), len(pieces), _hp(cc), C.byref(n)), "tb_piece_classes")
    return cc, n.value


def tb_graph_compile_variative(phrases, pieces, phrase_weights=None, tau: float = 1.0, lam: float = 1.0,
                               flags: int = 0) -> Graph:
    """phrases, pieces: lists of byte strings (phrases in any casing)."""
    pf, po = _flat_bytes(phrases)
    vf, vo = _flat_bytes(pieces)
    w = _host(phrase_weights, np.float32)
    h = _vp()
    _check(_lib.tb_graph_compile_variative(_hp(pf), _hp(po), len(phrases), _hp(w), _hp(vf), _hp(vo), len(pieces),
                                           float(tau), float(lam), flags, C.byref(h)), "tb_graph_compile_variative")
    return Graph(h)


class Batch:
    """Device arena + slot table + per-slot decode state."""

    def __init__(self, handle, vocab, n_slots, max_beam, device):
        self.handle, self.vocab, self.n_slots, self.max_beam, self.device = handle, vocab, n_slots, max_beam, device

    def destroy(self):
        if self.handle and _lib is not None:
            _lib.tb_batch_destroy(self.handle)
            self.handle = None

    def __del__(self):
        self.destroy()


def tb_batch_create(vocab: int, case_class, n_slots: int, max_beam: int = 1, max_tree_steps: int = 0,
                    arena_bytes: int = 64 << 20, device: int = 0) -> Batch:
    cc = _host(case_class, np.int32)
    h = _vp()
    _check(_lib.tb_batch_create(vocab, _hp(cc), n_slots, max_beam, max_tree_steps, arena_bytes, device, C.byref(h)),
           "tb_batch_create")
    return Batch(h, vocab, n_slots, max_beam, device)


def tb_batch_destroy(batch: Batch):
    batch.destroy()


def tb_batch_bind_stream(batch: Batch, slot: int, graph, stream=None):
    _check(_lib.tb_batch_bind_stream(batch.handle, slot, None if graph is None else graph.handle, _stream(stream)),
           "tb_batch_bind_stream")


TB_STATUS_WALK_TOO_DEEP, TB_STATUS_BAD_STATE, TB_STATUS_STEP_LIMIT, TB_STATUS_WAIT_TIMEOUT = 1, 2, 4, 8
TB_FLAG_GENERAL_KERNELS = 1
TB_FLAG_ONE_BLOCK_PER_STREAM = 2
TB_FLAG_TEST_WAIT_TIMEOUT = 4
TB_FLAG_LOG_SOFTMAX = 8
TB_FLAG_BEAM_WHOLE_ROWS = 16
TB_FLAG_COPIED_BINDS = 32
TB_KERNEL_GENERAL, TB_KERNEL_PIPELINED, TB_KERNEL_SEGMENTED = 1, 2, 3


def tb_batch_bind_streams(batch: Batch, slots, graphs, stream=None):
    """Bind graphs[i] (None: unbind) to slots[i], all in one copy and one launch."""
    n = len(graphs)
    assert len(slots) == n
    if n == 0:
        return
    sl = (_i32 * n)(*[int(x) for x in slots])
    arr = (_vp * n)(*[None if g is None else g.handle for g in graphs])
    _check(_lib.tb_batch_bind_streams(batch.handle, n, sl, arr, _stream(stream)), "tb_batch_bind_streams")


def tb_batch_set_flags(batch: Batch, flags: int):
    _check(_lib.tb_batch_set_flags(batch.handle, flags), "tb_batch_set_flags")


def tb_batch_set_greedy_plan(batch: Batch, deciders_per_block: int = 0, helpers_per_block: int = 0,
                             blocks_per_stream: int = 0):
    _check(_lib.tb_batch_set_greedy_plan(batch.handle, deciders_per_block, helpers_per_block, blocks_per_stream),
           "tb_batch_set_greedy_plan")


def tb_batch_last_greedy_kernel(batch: Batch) -> dict:
    k, nb, g = _i32(0), _i32(0), _i32(0)
    _check(_lib.tb_batch_last_greedy_kernel(batch.handle, C.byref(k), C.byref(nb), C.byref(g)),
           "tb_batch_last_greedy_kernel")
    return dict(kernel=k.value, blocks_per_stream=nb.value, deciders_per_block=g.value)


def tb_batch_bind_counts(batch: Batch) -> dict:
    """Binds of tb_stream_chunk_binds so far: carried out inside the chunk's launch / ahead of it."""
    pulled, copied = _i64(0), _i64(0)
    _check(_lib.tb_batch_bind_counts(batch.handle, C.byref(pulled), C.byref(copied)), "tb_batch_bind_counts")
    return dict(pulled=pulled.value, copied=copied.value)


def tb_batch_status(batch: Batch, stream=None) -> int:
    st = _i32(0)
    rc = _lib.tb_batch_status(batch.handle, C.byref(st), _stream(stream))
    if rc not in (TB_OK, TB_ERR_DEVICE_STATUS):
        raise TbError(rc, "tb_batch_status")
    return st.value


def _strides4(t: torch.Tensor):
    assert t.dim() == 4
    return (_i64 * 4)(*t.stride())


def tb_greedy_decode(batch: Batch, logits: torch.Tensor, lengths=None, out=None, stream=None) -> dict:
    """logits [B, T, S, vocab+1] on the batch's device.  Returns device tensors."""
    B, T, S, W = logits.shape
    if W != batch.vocab + 1:
        raise ValueError("last dimension must be vocab + 1")
    dev = logits.device
    if out is None:
        out = dict(tokens=torch.empty((B, T * S), dtype=torch.int32, device=dev),
                   frames=torch.empty((B, T * S), dtype=torch.int32, device=dev),
                   counts=torch.empty(B, dtype=torch.int32, device=dev),
                   scores=torch.empty(B, dtype=torch.float32, device=dev),
                   states=torch.empty(B, dtype=torch.int32, device=dev))
    st = _strides4(logits)
    _check(_lib.tb_greedy_decode(batch.handle, _dp(logits), _logit_dtype(logits), B, T, S, _hp(st), _dp(lengths),
                                 _dp(out["tokens"]), _dp(out["frames"]), _dp(out["counts"]), _dp(out["scores"]),
                                 _dp(out["states"]), _stream(stream)), "tb_greedy_decode")
    return out


def tb_stream_chunk(batch: Batch, logits: torch.Tensor, n_dur: int, valid_frames: torch.Tensor, out=None,
                    stream=None) -> dict:
    """logits [n_slots, chunk, S, vocab+1+n_dur].  Returns device tensors."""
    n, chunk, S, W = logits.shape
    if W != batch.vocab + 1 + n_dur:
        raise ValueError("last dimension must be vocab + 1 + n_dur")
    dev = logits.device
    if out is None:
        out = dict(tokens=torch.empty((n, chunk * S), dtype=torch.int32, device=dev),
                   frames=torch.empty((n, chunk * S), dtype=torch.int32, device=dev),
                   durs=torch.empty((n, chunk * S), dtype=torch.int32, device=dev),
                   counts=torch.empty(n, dtype=torch.int32, device=dev),
                   scores=torch.empty(n, dtype=torch.float32, device=dev),
                   states=torch.empty(n, dtype=torch.int32, device=dev),
                   cursors=torch.empty(n, dtype=torch.int32, device=dev))
    st = _strides4(logits)
    _check(_lib.tb_stream_chunk(batch.handle, _dp(logits), _logit_dtype(logits), n, chunk, S, n_dur, _hp(st),
                                _dp(valid_frames), _dp(out["tokens"]), _dp(out["frames"]), _dp(out.get("durs")),
                                _dp(out["counts"]), _dp(out["scores"]), _dp(out["states"]), _dp(out.get("cursors")),
                                _stream(stream)), "tb_stream_chunk")
    return out


def tb_stream_chunk_binds(batch: Batch, slots, graphs, logits: torch.Tensor, n_dur: int, valid_frames: torch.Tensor,
                          out=None, stream=None) -> dict:
    """tb_batch_bind_streams(batch, slots, graphs) followed by tb_stream_chunk(batch, logits, ...), in one call."""
    n, chunk, S, W = logits.shape
    if W != batch.vocab + 1 + n_dur:
        raise ValueError("last dimension must be vocab + 1 + n_dur")
    nb = len(graphs)
    assert len(slots) == nb
    dev = logits.device
    if out is None:
        out = dict(tokens=torch.empty((n, chunk * S), dtype=torch.int32, device=dev),
                   frames=torch.empty((n, chunk * S), dtype=torch.int32, device=dev),
                   durs=torch.empty((n, chunk * S), dtype=torch.int32, device=dev),
                   counts=torch.empty(n, dtype=torch.int32, device=dev),
                   scores=torch.empty(n, dtype=torch.float32, device=dev),
                   states=torch.empty(n, dtype=torch.int32, device=dev),
                   cursors=torch.empty(n, dtype=torch.int32, device=dev))
    sl = (_i32 * nb)(*[int(x) for x in slots]) if nb else None
    arr = (_vp * nb)(*[None if g is None else g.handle for g in graphs]) if nb else None
    _check(_lib.tb_stream_chunk_binds(batch.handle, nb, sl, arr, _dp(logits), _logit_dtype(logits), n, chunk, S, n_dur,
                                      _strides4(logits), _dp(valid_frames), _dp(out["tokens"]), _dp(out["frames"]),
                                      _dp(out.get("durs")), _dp(out["counts"]), _dp(out["scores"]), _dp(out["states"]),
                                      _dp(out.get("cursors")), _stream(stream)), "tb_stream_chunk_binds")
    return out


def tb_beam_reset(batch: Batch):
    _check(_lib.tb_beam_reset(batch.handle), "tb_beam_reset")


def tb_beam_step(batch: Batch, logits: torch.Tensor, stream_stride: int, hyp_stride: int, new_frame,
                 scores: torch.Tensor, states: torch.Tensor, live: torch.Tensor, out_parent: torch.Tensor,
                 out_token: torch.Tensor, stream=None, offset: int = 0):
    """logits: any tensor; hypothesis k of stream i reads vocab+1 contiguous elements at element
    offset ``offset + i*stream_stride + k*hyp_stride``.  scores/states/live [B, K] are updated in place.
    new_frame: False / True, or one of TB_FRAME_SAME / TB_FRAME_NEW / TB_FRAME_NEW_MERGE."""
    B, K = scores.shape
    ptr = _vp(logits.data_ptr() + offset * logits.element_size())
    _check(_lib.tb_beam_step(batch.handle, ptr, _logit_dtype(logits), B, K, stream_stride, hyp_stride,
                             int(new_frame), _dp(scores), _dp(states), _dp(live), _dp(out_parent),
                             _dp(out_token), _stream(stream)), "tb_beam_step")


def tb_beam_frames(batch: Batch, logits: torch.Tensor, merge: bool, scores: torch.Tensor, states: torch.Tensor,
                   live: torch.Tensor, out_parent: torch.Tensor, out_token: torch.Tensor, stream=None):
    """logits [B, T, E, V+1] (any strides with a contiguous last dimension): T frames of E expansions in one launch."""
    B, K = scores.shape
    assert logits.dim() == 4 and logits.shape[0] == B and logits.stride(3) == 1
    sb, st, se, _ = logits.stride()
    _check(_lib.tb_beam_frames(batch.handle, _dp(logits), _logit_dtype(logits), B, K, logits.shape[1], logits.shape[2],
                               sb, st, se, 1 if merge else 0, _dp(scores), _dp(states), _dp(live), _dp(out_parent),
                               _dp(out_token), _stream(stream)), "tb_beam_frames")


def tb_beam_reset_slots(batch: Batch, slots=None, stream=None):
    """A new utterance on ``slots`` (None: on every slot) for streaming beam decoding."""
    if slots is None:
        _check(_lib.tb_beam_reset_slots(batch.handle, 0, None, _stream(stream)), "tb_beam_reset_slots")
        return
    n, sl = _slots(slots)
    if n:
        _check(_lib.tb_beam_reset_slots(batch.handle, n, sl, _stream(stream)), "tb_beam_reset_slots")


def tb_beam_start_slots(batch: Batch, slots, scores: torch.Tensor, states: torch.Tensor, live: torch.Tensor, stream=None):
    """tb_beam_reset_slots that also sets up the slots' rows of scores / states / live [n_slots, K] (None: every slot)."""
    n, sl = (0, None) if slots is None else _slots(slots)
    if slots is not None and n == 0:
        return
    _check(_lib.tb_beam_start_slots(batch.handle, n, sl, scores.shape[1], _dp(scores),
                                    _dp(states), _dp(live), _stream(stream)), "tb_beam_start_slots")


def tb_beam_chunk(batch: Batch, logits: torch.Tensor, merge: bool, n_frames, scores: torch.Tensor, states: torch.Tensor,
                  live: torch.Tensor, out_parent: torch.Tensor, out_token: torch.Tensor, stream=None):
    """logits [n_slots, chunk, E, vocab+1]; n_frames: device int32 [n_slots] (frames of this chunk each slot decodes)."""
    B, T, E, W = logits.shape
    K = scores.shape[1]
    sb, st, se, sv = logits.stride()
    assert sv == 1 and W == batch.vocab + 1
    _check(_lib.tb_beam_chunk(batch.handle, _dp(logits), _logit_dtype(logits), B, K, T, E, sb, st, se, 1 if merge else 0,
                              _dp(n_frames), _dp(scores), _dp(states), _dp(live), _dp(out_parent), _dp(out_token),
                              _stream(stream)), "tb_beam_chunk")


def tb_beam_backtrace_slots(batch: Batch, n_slots: int, K: int, max_len: int, stream=None, out=None):
    """out: (tokens int32 [n_slots, K, max_len], lens int32 [n_slots, K]) to write into instead of new tensors."""
    dev = torch.device("cuda", batch.device)
    if out is not None:
        toks, lens = out
        if tuple(toks.shape) != (n_slots, K, max_len) or tuple(lens.shape) != (n_slots, K) or toks.dtype != torch.int32 \
                or lens.dtype != torch.int32 or not toks.is_contiguous() or not lens.is_contiguous():
            raise ValueError("out must be contiguous int32 tensors [n_slots, K, max_len] and [n_slots, K]")
    else:
        toks = torch.zeros((n_slots, K, max_len), dtype=torch.int32, device=dev)
        lens = torch.zeros((n_slots, K), dtype=torch.int32, device=dev)
    _check(_lib.tb_beam_backtrace_slots(batch.handle, n_slots, K, max_len, _dp(toks), _dp(lens), _stream(stream)),
           "tb_beam_backtrace_slots")
    return toks, lens


def tb_beam_backtrace_slot_list(batch: Batch, slots, K: int, max_len: int, stream=None, out=None):
    """Transcripts of the slots in ``slots`` only: (tokens int32 [n, K, max_len], lens int32 [n, K]); ``out``: tensors of
    at least that many rows to write into (their first n rows are used)."""
    n = len(slots)
    dev = torch.device("cuda", batch.device)
    if out is not None:
        toks, lens = out
        if toks.dim() != 3 or toks.shape[0] < n or tuple(toks.shape[1:]) != (K, max_len) or lens.shape[0] < n or lens.shape[1] != K \
                or toks.dtype != torch.int32 or lens.dtype != torch.int32 or not toks.is_contiguous() or not lens.is_contiguous():
            raise ValueError("out must be contiguous int32 tensors [>= n, K, max_len] and [>= n, K]")
    else:
        toks = torch.zeros((n, K, max_len), dtype=torch.int32, device=dev)
        lens = torch.zeros((n, K), dtype=torch.int32, device=dev)
    if n:
        sl = (_i32 * n)(*[int(x) for x in slots])
        _check(_lib.tb_beam_backtrace_slot_list(batch.handle, n, sl, K, max_len, _dp(toks), _dp(lens), _stream(stream)),
               "tb_beam_backtrace_slot_list")
    return toks[:n], lens[:n]


def tb_apply_final_weights_slots(batch: Batch, slots, scores: torch.Tensor, states: torch.Tensor, stream=None):
    n, sl = _slots(slots)
    if n:
        _check(_lib.tb_apply_final_weights_slots(batch.handle, n, sl, scores.shape[1], _dp(scores), _dp(states),
                                                 _stream(stream)), "tb_apply_final_weights_slots")


def tb_batch_set_beam_prune(batch: Batch, delta: float):
    _check(_lib.tb_batch_set_beam_prune(batch.handle, float(delta)), "tb_batch_set_beam_prune")


def tb_apply_final_weights(batch: Batch, scores: torch.Tensor, states: torch.Tensor, stream=None):
    """scores float32 [B] or [B, K], states int32 of the same shape (device, contiguous); scores updated in place."""
    assert scores.dtype == torch.float32 and states.dtype == torch.int32 and scores.shape == states.shape
    assert scores.is_contiguous() and states.is_contiguous()
    B = scores.shape[0]
    K = 1 if scores.dim() == 1 else scores.shape[1]
    _check(_lib.tb_apply_final_weights(batch.handle, B, K, _dp(scores), _dp(states), _stream(stream)),
           "tb_apply_final_weights")
    return scores


def tb_beam_backtrace(batch: Batch, B: int, K: int, max_len: int, stream=None):
    dev = torch.device("cuda", batch.device)
    toks = torch.zeros((B, K, max_len), dtype=torch.int32, device=dev)
    lens = torch.zeros((B, K), dtype=torch.int32, device=dev)
    _check(_lib.tb_beam_backtrace(batch.handle, B, K, max_len, _dp(toks), _dp(lens), _stream(stream)),
           "tb_beam_backtrace")
    return toks, lens


TB_NOALLOC_MAX_STREAMS = 256


def tb_greedy_decode_noalloc(logits: torch.Tensor, out: dict, lengths=None, stream=None) -> dict:
    """Unboosted greedy decode for callers that must not allocate device memory at decode time
    (a server with a fixed, pre-divided memory budget; a thread that cannot afford the device-wide
    synchronisation of cudaMalloc).  The library's own working memory is a fixed array inside the
    library, so the caller brings every buffer: ``out`` must hold preallocated device tensors
    ``tokens`` / ``frames`` [B, T*S], ``counts`` / ``states`` [B] (int32), ``scores`` [B] (float32) and
    optionally ``status`` [1] (int32).  Calls that overlap on one GPU race on the shared array."""
    B, T, S, W = logits.shape
    _check_noalloc_buffers(logits, out, lengths)
    st = _strides4(logits)
    device = logits.device.index if logits.device.index is not None else torch.cuda.current_device()
    _check(_lib.tb_greedy_decode_noalloc(device, _dp(logits), _logit_dtype(logits), B, T, S, W - 1,
                                         _hp(st), _dp(lengths), _dp(out["tokens"]), _dp(out["frames"]),
                                         _dp(out["counts"]), _dp(out["scores"]), _dp(out["states"]),
                                         _dp(out.get("status")), _stream(stream)), "tb_greedy_decode_noalloc")
    return out


def _check_noalloc_buffers(logits: torch.Tensor, out: dict, lengths):
    """The caller brings every output buffer of tb_greedy_decode_noalloc, and the kernel writes them without
    knowing their sizes: a buffer that is too short, of another type, strided, or on another device is refused
    here, before anything is launched.  Sizes and types are checked first (they need no GPU), devices last."""
    B, T, S, _ = logits.shape
    need = {"tokens": (torch.int32, B * T * S), "frames": (torch.int32, B * T * S), "counts": (torch.int32, B),
            "states": (torch.int32, B), "scores": (torch.float32, B)}
    if out.get("status") is not None:
        need["status"] = (torch.int32, 1)
    tensors = []
    for name, (dt, n) in need.items():
        t = out.get(name)
        if not isinstance(t, torch.Tensor):
            raise ValueError(f"tb_greedy_decode_noalloc: out[{name!r}] must be a preallocated tensor")
        if t.dtype != dt:
            raise ValueError(f"tb_greedy_decode_noalloc: out[{name!r}] must be {dt}, got {t.dtype}")
        if not t.is_contiguous():
            raise ValueError(f"tb_greedy_decode_noalloc: out[{name!r}] must be contiguous")
        if t.numel() < n:
            raise ValueError(f"tb_greedy_decode_noalloc: out[{name!r}] holds {t.numel()} elements, {n} are written")
        tensors.append((name, t))
    if lengths is not None:
        if lengths.dtype != torch.int32 or not lengths.is_contiguous() or lengths.numel() < B:
            raise ValueError("tb_greedy_decode_noalloc: lengths must be a contiguous int32 tensor of at least B elements")
        tensors.append(("lengths", lengths))
    if not logits.is_cuda:
        raise ValueError("tb_greedy_decode_noalloc: logits must be on a CUDA device")
    for name, t in tensors:
        if t.device != logits.device:
            raise ValueError(f"tb_greedy_decode_noalloc: {name} is on {t.device}, the logits are on {logits.device}")
