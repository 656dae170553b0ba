"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, and its graph compiler emits arrays identical to the oracle's compiler (both
use the breadth-first canonical numbering, so equality is element for element)."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import oracle as O
from paper_2608_21343_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
ARRAYS = ("state_arc_begin", "arc_class", "arc_dst", "arc_w", "state_fail", "state_bw", "state_final",
          "state_depth", "case_class")


def declared_functions():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"\b(tb_[a-z_0-9]+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_symbol(tb):
    lib = ctypes.CDLL(tb.LIB_PATH)
    names = declared_functions()
    assert len(names) >= 13
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(tb.EXPORTED)
    assert tb.tb_strerror(0) == "ok" and "arena" in tb.tb_strerror(tb.TB_ERR_ARENA_FULL)


def assert_same_graph(tb, phrases, V, cc, weights=None, lam=1.0):
    go = O.Graph(phrases, V, case_class=cc, weights=weights, lam=lam)
    gl = tb.tb_graph_compile(phrases, V, case_class=cc, token_weights=weights, lam=lam).view()
    for k in ("n_states", "n_arcs", "n_classes", "vocab", "max_depth"):
        assert gl[k] == getattr(go, k), k
    assert gl["lam"] == go.lam
    for k in ARRAYS:
        a, b = gl[k], getattr(go, k)
        assert a.dtype == b.dtype and a.shape == b.shape and a.tobytes() == b.tobytes(), k
    return go


@pytest.mark.parametrize("seed", range(10))
def test_compiler_matches_oracle_random_lists(tb, seed):
    rng = np.random.default_rng(seed)
    V = int(rng.integers(3, 40))
    cc = None if seed % 3 == 0 else rng.integers(0, max(1, V // 2), size=V).astype(np.int32)
    n = int(rng.integers(0, 60))
    phrases = [[int(t) for t in rng.integers(0, V, size=rng.integers(0, 7))] for _ in range(n)]
    weights = None
    if seed % 2:
        weights = [[float(rng.choice([0.25, 0.5, 1.0, 1.3, 2.0])) for _ in p] for p in phrases]
    assert_same_graph(tb, phrases, V, cc, weights, lam=[1.0, 0.5, 2.0][seed % 3])


def test_compiler_matches_oracle_on_workload_lists(tb):
    for cid, b in ((1, 0), (1, 3), (2, 5), (4, 1), (5, 7)):
        w = W.get_workload(cid)
        g = assert_same_graph(tb, W.stream_phrases(w, b), w.V, w.vocab.case_class)
        assert g.n_states > 10
    w = W.get_workload(3)
    g = assert_same_graph(tb, W.stream_phrases(w, 2), w.V, w.vocab.case_class)
    assert 15000 < g.n_states < 40000          # "about 20-30k states and arcs per stream"


def test_compile_error_codes(tb):
    def code(*a, **k):
        with pytest.raises(tb.TbError) as e:
            tb.tb_graph_compile(*a, **k)
        return e.value.code
    assert code([[0, 9]], 4) == tb.TB_ERR_INVALID_ARG
    assert code([[0, -1]], 4) == tb.TB_ERR_INVALID_ARG
    assert code([[0, 1]], 4, token_weights=[[1.0, -1.0]]) == tb.TB_ERR_INVALID_ARG
    assert code([[0, 1]], 4, token_weights=[[1.0, float("inf")]]) == tb.TB_ERR_INVALID_ARG
    assert code([[0, 1]], 4, case_class=[0, -2, 1, 1]) == tb.TB_ERR_INVALID_ARG
    assert code([[0, 1]], 4, lam=float("nan")) == tb.TB_ERR_INVALID_ARG
    assert code([[0, 1]], 0) == tb.TB_ERR_INVALID_ARG
    assert code([[0, 1]], 100000) == tb.TB_ERR_INVALID_ARG
    assert code([[0] * 300], 4) == tb.TB_ERR_INVALID_ARG
    assert code([[0, 1]], 4, flags=2) == tb.TB_ERR_INVALID_ARG
    tb.tb_graph_compile([[0, 1]], 4, flags=tb.TB_COMPILE_PAGEABLE)       # the one flag there is
    g = tb.tb_graph_compile([], 4).view()
    assert g["n_states"] == 1 and g["n_arcs"] == 0


# ---- variative, case-insensitive compile (Sec. 2.1 para. 4-7, Eq. 1) -------------------------------------

def assert_same_variative_graph(tb, phrases, pieces, weights=None, tau=1.0, lam=1.0):
    from oracle import variative as var
    a = var.build(phrases, pieces, weights=weights, tau=tau, lam=lam)
    gl = tb.tb_graph_compile_variative(phrases, pieces, phrase_weights=weights, tau=tau, lam=lam).view()
    for k in ("n_states", "n_arcs", "n_classes", "vocab", "max_depth"):
        assert gl[k] == a[k], k
    for k in ARRAYS:
        assert gl[k].dtype == a[k].dtype and gl[k].shape == a[k].shape and gl[k].tobytes() == a[k].tobytes(), k
    return a


@pytest.mark.parametrize("seed", range(8))
def test_variative_compiler_matches_oracle(tb, seed):
    rng = np.random.default_rng(seed)
    pieces = W.make_piece_vocab(seed, letters=int(rng.integers(3, 12)), merged=int(rng.integers(0, 80)),
                                max_len=int(rng.integers(2, 6)))
    phrases = W.draw_string_phrases(seed, pieces, int(rng.integers(0, 90)), 1, 5)
    if seed % 2:                                         # user lists in mixed casing, duplicates, an empty phrase
        phrases = [p.upper() if i % 3 == 0 else p.title() if i % 3 == 1 else p for i, p in enumerate(phrases)]
        phrases += phrases[:3] + [b""]
    weights = None if seed % 3 == 0 else [float(rng.uniform(0.0, 2.5)) for _ in phrases]
    a = assert_same_variative_graph(tb, phrases, pieces, weights, tau=float(rng.uniform(0.0, 3.0)),
                                    lam=[1.0, 0.5, 2.0][seed % 3])
    cc, n = tb.tb_piece_classes(pieces)
    assert np.array_equal(cc, a["case_class"]) and n == a["n_classes"]


def test_variative_compiler_on_a_production_sized_list(tb):
    # 300 phrases over a 1024-piece vocabulary, the size of the per-stream lists of the decode workloads
    pieces = W.make_piece_vocab(11, letters=26, merged=560, max_len=5)[:1024]
    phrases = W.draw_string_phrases(11, pieces, 300, 1, 6)
    a = assert_same_variative_graph(tb, phrases, pieces, tau=1.0)
    assert a["n_states"] > 1000 and a["n_arcs"] > a["n_states"]          # not a tree: arcs converge


def test_variative_compile_error_codes(tb):
    pieces = [b"a", b"A", b"b", b"ab"]

    def code(*a, **k):
        with pytest.raises(tb.TbError) as e:
            tb.tb_graph_compile_variative(*a, **k)
        return e.value.code
    assert code([b"abc"], pieces) == tb.TB_ERR_INVALID_ARG                   # 'c' has no piece
    assert code([b"ab"], pieces, tau=-1.0) == tb.TB_ERR_INVALID_ARG
    assert code([b"ab"], pieces, tau=float("nan")) == tb.TB_ERR_INVALID_ARG
    assert code([b"ab"], pieces, lam=float("inf")) == tb.TB_ERR_INVALID_ARG
    assert code([b"ab"], pieces, phrase_weights=[-1.0]) == tb.TB_ERR_INVALID_ARG
    assert code([b"a" * 256], pieces) == tb.TB_ERR_INVALID_ARG
    assert code([b"ab"], pieces + [b""]) == tb.TB_ERR_INVALID_ARG             # an empty piece
    assert code([b"ab"], pieces + [b"a" * 33]) == tb.TB_ERR_INVALID_ARG       # a piece longer than TB_MAX_PIECE_LEN
    assert code([b"ab"], pieces, flags=2) == tb.TB_ERR_INVALID_ARG
    g = tb.tb_graph_compile_variative([], pieces).view()
    assert g["n_states"] == 1 and g["n_arcs"] == 0
    g = tb.tb_graph_compile_variative([b"AB"], pieces, tau=0.0).view()      # the hand-worked list, given in upper case
    assert list(g["arc_class"]) == [0, 2, 1] and list(g["arc_w"]) == [0.5, 1.0, 0.5]


# ---- model lifecycle off the device: disk and memory levels (Sec. 2.2 para. 5) ---------------------------

def _same_view(a, b):
    for k in a:
        if isinstance(a[k], np.ndarray):
            assert a[k].dtype == b[k].dtype and a[k].tobytes() == b[k].tobytes(), k
        else:
            assert a[k] == b[k], k


def test_graph_save_load_round_trip(tb, tmp_path):
    w = W.get_workload(2)
    for i, g in enumerate([tb.tb_graph_compile(W.stream_phrases(w, 3), w.V, case_class=w.vocab.case_class, lam=0.5),
                           tb.tb_graph_compile([], 7),
                           tb.tb_graph_compile_variative([b"hello", b"help"], [bytes([c]) for c in b"helopHELOP"] + [b"he", b"He", b"llo"])]):
        path = str(tmp_path / f"g{i}.tbg")
        tb.tb_graph_save(g, path)
        _same_view(g.view(), tb.tb_graph_load(path).view())


def test_graph_load_refuses_damaged_files(tb, tmp_path):
    w = W.get_workload(1)
    g = tb.tb_graph_compile(W.stream_phrases(w, 0), w.V, case_class=w.vocab.case_class)
    path = str(tmp_path / "g.tbg")
    tb.tb_graph_save(g, path)
    raw = open(path, "rb").read()

    def code(data):
        p = str(tmp_path / "bad.tbg")
        open(p, "wb").write(data)
        with pytest.raises(tb.TbError) as e:
            tb.tb_graph_load(p)
        return e.value.code
    assert code(raw[:-1]) == tb.TB_ERR_INVALID_ARG                       # cut short
    assert code(raw + b"\0") == tb.TB_ERR_INVALID_ARG                    # longer than it says
    assert code(b"XXXX" + raw[4:]) == tb.TB_ERR_INVALID_ARG              # not such a file
    assert code(raw[:40]) == tb.TB_ERR_IO                                # not even a header
    for pos in (8, len(raw) // 2, len(raw) - 3):                          # one altered byte: header field, payload
        b = bytearray(raw)
        b[pos] ^= 0x40
        assert code(bytes(b)) == tb.TB_ERR_INVALID_ARG
    with pytest.raises(tb.TbError) as e:
        tb.tb_graph_load(str(tmp_path / "missing.tbg"))
    assert e.value.code == tb.TB_ERR_IO

    # a file whose checksum is right but whose tables point outside themselves is refused as well
    HDR, HASH_AT = 112, 104

    def checksum(data):
        h, m = 1469598103934665603, (1 << 64) - 1
        i = 0
        while i + 8 <= len(data):
            h = ((h ^ int.from_bytes(data[i:i + 8], "little")) * 1099511628211) & m
            h ^= h >> 29
            i += 8
        for c in data[i:]:
            h = ((h ^ c) * 1099511628211) & m
        return h

    def resealed(b):
        b = bytearray(b)
        b[HASH_AT:HASH_AT + 8] = bytes(8)
        b[HASH_AT:HASH_AT + 8] = checksum(bytes(b)).to_bytes(8, "little")
        return bytes(b)
    assert resealed(raw) == raw                                           # the checksum as this test computes it
    hv = g.view()
    N, A = hv["n_states"], hv["n_arcs"]
    field = {"n_states": 8, "max_depth": 24, "off_arc_begin": 40, "off_strec": 64, "off_tokent": 68, "n_tokent": 72,
             "off_rsrec": 76, "off_rsent": 80, "n_rsent": 84}

    def with_i32(at, value):
        b = bytearray(raw)
        b[at:at + 4] = int(value).to_bytes(4, "little", signed=True)
        return resealed(b)
    n_tokent = int.from_bytes(raw[72:76], "little")
    blob_bytes = int.from_bytes(raw[96:104], "little")
    bad = [with_i32(field["max_depth"], 4096),                            # deeper than any phrase may be
           with_i32(field["off_strec"], (blob_bytes - 16) & ~15),          # a section that runs off the end of the blob
           with_i32(field["n_tokent"], n_tokent + (1 << 20)),
           with_i32(field["n_rsent"], 1 << 17),
           with_i32(HDR + 4 * (N + 1) + 4 * A, N),                        # first arc target: one past the last state
           with_i32(HDR + 4 * (N + 1) + 4 * A, -1),
           with_i32(HDR + 4 * (N + 1) + 3 * 4 * A + 4, N + 7),            # suffix link of state 1
           with_i32(HDR + 4, 1 << 30)]                                          # arc ranges that go backwards
    for data in bad:
        assert code(data) == tb.TB_ERR_INVALID_ARG
    # the same in the device copy of a table: suffix link of state 1 inside the blob
    blob_at = len(raw) - blob_bytes
    off_fail = int.from_bytes(raw[44:48], "little")
    assert code(with_i32(blob_at + off_fail + 4, N)) == tb.TB_ERR_INVALID_ARG
    off_rsent = int.from_bytes(raw[80:84], "little")
    n_rsent = int.from_bytes(raw[84:88], "little", signed=True)
    assert n_rsent > 0
    ent = int.from_bytes(raw[blob_at + off_rsent:blob_at + off_rsent + 4], "little")
    assert code(with_i32(blob_at + off_rsent, (ent & 0xfff) | ((N + 3) << 12))) == tb.TB_ERR_INVALID_ARG
    with pytest.raises(tb.TbError) as e:
        tb.tb_graph_save(g, str(tmp_path / "no_such_dir" / "g.tbg"))
    assert e.value.code == tb.TB_ERR_IO


def test_cache_returns_what_the_compiler_returns(tb):
    w = W.get_workload(2)
    cc = w.vocab.case_class
    cache = tb.tb_cache_create(1 << 20)
    lists = [W.stream_phrases(w, b) for b in range(6)]
    first = []
    for p in lists:
        g, hit = tb.tb_cache_compile(cache, p, w.V, case_class=cc)
        assert not hit
        _same_view(g.view(), tb.tb_graph_compile(p, w.V, case_class=cc).view())
        first.append(g)
    for p, g0 in zip(lists, first):
        g, hit = tb.tb_cache_compile(cache, p, w.V, case_class=cc)
        assert hit and g.handle.value == g0.handle.value               # the very same compiled graph
    # anything the compiler reads is part of the key
    assert not tb.tb_cache_compile(cache, lists[0], w.V, case_class=cc, lam=0.5)[1]
    assert not tb.tb_cache_compile(cache, lists[0], w.V, case_class=None)[1]
    assert not tb.tb_cache_compile(cache, lists[0], w.V, case_class=cc, token_weights=[[1.0] * len(p) for p in lists[0]])[1]
    assert not tb.tb_cache_compile(cache, lists[0][:-1], w.V, case_class=cc)[1]
    assert not tb.tb_cache_compile(cache, lists[0][:-2] + [lists[0][-2] + lists[0][-1]], w.V, case_class=cc)[1]   # same tokens, other phrase boundaries
    st = cache.stats()
    assert st["hits"] == 6 and st["misses"] == 11 and st["entries"] == 11 and st["evictions"] == 0
    # errors pass through, nothing is kept for them
    with pytest.raises(tb.TbError):
        tb.tb_cache_compile(cache, [[0, w.V + 5]], w.V, case_class=cc)
    assert cache.stats()["entries"] == 11
    # a graph handed out stays valid when the cache goes away
    cache.destroy()
    assert first[2].view()["n_states"] > 10


def test_cache_drops_least_recently_used(tb):
    w = W.get_workload(2)
    cc = w.vocab.case_class
    lists = [W.stream_phrases(w, b) for b in range(5)]
    probe = tb.tb_cache_create(1 << 24)
    tb.tb_cache_compile(probe, lists[0], w.V, case_class=cc)
    one = probe.stats()["bytes_used"]
    cache = tb.tb_cache_create(int(3.5 * one))                           # room for three such graphs
    for p in lists[:3]:
        tb.tb_cache_compile(cache, p, w.V, case_class=cc)
    assert tb.tb_cache_compile(cache, lists[0], w.V, case_class=cc)[1]   # 0 is now the most recent
    tb.tb_cache_compile(cache, lists[3], w.V, case_class=cc)             # drops 1, the least recent
    assert cache.stats()["evictions"] >= 1
    assert tb.tb_cache_compile(cache, lists[0], w.V, case_class=cc)[1]
    assert not tb.tb_cache_compile(cache, lists[1], w.V, case_class=cc)[1]
    tiny = tb.tb_cache_create(64)                                        # too small for any graph: compiles, keeps nothing
    g, hit = tb.tb_cache_compile(tiny, lists[0], w.V, case_class=cc)
    assert not hit and g.view()["n_states"] > 10 and tiny.stats()["entries"] == 0


def test_cache_is_safe_from_several_threads(tb):
    import threading
    w = W.get_workload(2)
    cc = w.vocab.case_class
    lists = [W.stream_phrases(w, b) for b in range(8)]
    want = [tb.tb_graph_compile(p, w.V, case_class=cc).view()["n_states"] for p in lists]
    cache = tb.tb_cache_create(1 << 22)
    errors = []

    def work(tid):
        try:
            for r in range(30):
                i = (tid + r) % len(lists)
                g, _ = tb.tb_cache_compile(cache, lists[i], w.V, case_class=cc)
                assert g.view()["n_states"] == want[i]
        except Exception as e:              # noqa: BLE001
            errors.append(e)
    threads = [threading.Thread(target=work, args=(t,)) for t in range(8)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors
    st = cache.stats()
    assert st["hits"] + st["misses"] == 240 and st["entries"] == 8


def test_cache_of_variative_lists(tb):
    pieces = W.make_piece_vocab(3, letters=10, merged=60, max_len=4)
    lists = [W.draw_string_phrases(30 + b, pieces, 40, 1, 4) for b in range(4)]
    cache = tb.tb_cache_create(1 << 22)
    first = []
    for p in lists:
        g, hit = tb.tb_cache_compile_variative(cache, p, pieces, tau=1.5)
        assert not hit
        _same_view(g.view(), tb.tb_graph_compile_variative(p, pieces, tau=1.5).view())
        first.append(g)
    for p, g0 in zip(lists, first):
        g, hit = tb.tb_cache_compile_variative(cache, p, pieces, tau=1.5)
        assert hit and g.handle.value == g0.handle.value
    assert not tb.tb_cache_compile_variative(cache, lists[0], pieces, tau=0.5)[1]                    # tau is part of the key
    assert not tb.tb_cache_compile_variative(cache, lists[0], pieces, tau=1.5, lam=2.0)[1]
    assert not tb.tb_cache_compile_variative(cache, lists[0], pieces, tau=1.5, phrase_weights=[1.0] * 40)[1]
    assert not tb.tb_cache_compile_variative(cache, lists[0], pieces[:-1] + [b"zz"], tau=1.5)[1]     # so is the vocabulary
    assert not tb.tb_cache_compile_variative(cache, [p.upper() for p in lists[0]], pieces, tau=1.5)[1]   # the text as given
    with pytest.raises(tb.TbError):
        tb.tb_cache_compile_variative(cache, [b"\\x01"], pieces)
    st = cache.stats()
    assert st["hits"] == 4 and st["entries"] == 9
    # token lists and text lists live side by side
    w = W.get_workload(1)
    assert not tb.tb_cache_compile(cache, W.stream_phrases(w, 0), w.V, case_class=w.vocab.case_class)[1]
    assert tb.tb_cache_compile(cache, W.stream_phrases(w, 0), w.V, case_class=w.vocab.case_class)[1]


def test_noalloc_binding_refuses_bad_buffers_before_any_launch(tb):
    """tb_greedy_decode_noalloc writes into buffers the caller brings; the binding refuses a buffer that is too
    short, of the wrong type or strided without touching a GPU (sizes and types are checked before devices)."""
    import torch
    B, T, S, V = 3, 5, 2, 8
    logits = torch.zeros((B, T, S, V + 1), dtype=torch.float32)

    def bufs():
        return dict(tokens=torch.zeros((B, T * S), dtype=torch.int32), frames=torch.zeros((B, T * S), dtype=torch.int32),
                    counts=torch.zeros(B, dtype=torch.int32), states=torch.zeros(B, dtype=torch.int32),
                    scores=torch.zeros(B, dtype=torch.float32), status=torch.zeros(1, dtype=torch.int32))

    o = bufs(); o["tokens"] = torch.zeros((B, T * S - 1), dtype=torch.int32)
    with pytest.raises(ValueError, match="tokens.*elements"):
        tb.tb_greedy_decode_noalloc(logits, o)
    o = bufs(); o["scores"] = torch.zeros(B, dtype=torch.float64)
    with pytest.raises(ValueError, match="scores.*float32"):
        tb.tb_greedy_decode_noalloc(logits, o)
    o = bufs(); o["frames"] = torch.zeros((B, 2 * T * S), dtype=torch.int32)[:, ::2]
    with pytest.raises(ValueError, match="frames.*contiguous"):
        tb.tb_greedy_decode_noalloc(logits, o)
    o = bufs(); del o["counts"]
    with pytest.raises(ValueError, match="counts"):
        tb.tb_greedy_decode_noalloc(logits, o)
    with pytest.raises(ValueError, match="lengths"):
        tb.tb_greedy_decode_noalloc(logits, bufs(), lengths=torch.zeros(B - 1, dtype=torch.int32))
    with pytest.raises(ValueError, match="CUDA"):           # everything else in order: the logits are not on a GPU
        tb.tb_greedy_decode_noalloc(logits, bufs())
