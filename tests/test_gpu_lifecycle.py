"""GPU checks of the model lifecycle (Sec. 2.2 para. 4-5): models registered with the decoder ahead of a
session and bound to slots by id, graphs that went through a file, graphs from the host-memory cache -- every
way of getting a list onto the device must decode exactly like compiling and binding it, i.e. like the oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2608_21343_b200 import workloads as W
from helpers import check_greedy, oracle_graph, to_device, to_host

pytestmark = pytest.mark.gpu


def _decode_and_check(tb, w, batch, data, lists, what):
    out = to_host(tb.tb_greedy_decode(batch, to_device(data["logits"])))
    assert tb.tb_batch_status(batch) == 0
    for i, p in enumerate(lists):
        check_greedy(out, i, O.greedy_rnnt(oracle_graph(w, p), data["logits"][i]), what)


def test_registered_models_decode_like_bound_graphs(tb):
    w = W.get_workload(2, B=6, T=200)
    data = W.batch_inputs(w)
    cc = w.vocab.case_class
    graphs = [tb.tb_graph_compile(p, w.V, case_class=cc) for p in data["phrases"]]
    batch = tb.tb_batch_create(w.V, cc, w.B, arena_bytes=4 << 20)
    ids = [tb.tb_batch_register_model(batch, g) for g in graphs]
    assert sorted(ids) == list(range(w.B))
    for i, m in enumerate(ids):
        tb.tb_batch_bind_model(batch, i, m)
    _decode_and_check(tb, w, batch, data, data["phrases"], "registered")
    # several slots on one model, one slot unbound by id -1, one bound the ordinary way
    plan = [ids[2], ids[2], -1, ids[0], ids[2], None]
    lists = [data["phrases"][2], data["phrases"][2], None, data["phrases"][0], data["phrases"][2], data["phrases"][5]]
    for i, m in enumerate(plan):
        if m is None:
            tb.tb_batch_bind_stream(batch, i, graphs[5])
        else:
            tb.tb_batch_bind_model(batch, i, m)
    _decode_and_check(tb, w, batch, data, lists, "shared model")
    # a model in use cannot be dropped; one that is not can, and its id is handed out again
    with pytest.raises(tb.TbError) as e:
        tb.tb_batch_unregister_model(batch, ids[2])
    assert e.value.code == tb.TB_ERR_INVALID_ARG
    tb.tb_batch_unregister_model(batch, ids[4])
    with pytest.raises(tb.TbError):
        tb.tb_batch_bind_model(batch, 0, ids[4])
    with pytest.raises(tb.TbError):
        tb.tb_batch_unregister_model(batch, ids[4])
    assert tb.tb_batch_register_model(batch, graphs[1]) == ids[4]
    with pytest.raises(tb.TbError) as e:
        tb.tb_batch_bind_model(batch, 99, ids[0])
    assert e.value.code == tb.TB_ERR_BAD_SLOT
    with pytest.raises(tb.TbError):
        tb.tb_batch_bind_model(batch, 0, 12345)
    # moving every slot off a model frees it for removal
    for i in range(w.B):
        tb.tb_batch_bind_model(batch, i, -1)
    for m in set(ids):
        tb.tb_batch_unregister_model(batch, m)
    _decode_and_check(tb, w, batch, data, [None] * w.B, "all unbound")


def test_registration_does_not_leak_arena_space(tb):
    w = W.get_workload(2, B=2, T=130)
    data = W.batch_inputs(w)
    cc = w.vocab.case_class
    g = tb.tb_graph_compile(data["phrases"][0], w.V, case_class=cc)
    batch = tb.tb_batch_create(w.V, cc, 2, arena_bytes=256 << 10)       # room for a few such graphs only
    for r in range(200):
        m = tb.tb_batch_register_model(batch, g)
        tb.tb_batch_bind_model(batch, r % 2, m)
        tb.tb_batch_bind_model(batch, r % 2, -1)
        tb.tb_batch_unregister_model(batch, m)
    held = []
    with pytest.raises(tb.TbError) as e:                                 # and the arena does fill up when models are kept
        for _ in range(100):
            held.append(tb.tb_batch_register_model(batch, g))
    assert e.value.code == tb.TB_ERR_ARENA_FULL and len(held) >= 2
    tb.tb_batch_bind_model(batch, 0, held[0])
    tb.tb_batch_bind_stream(batch, 1, None)
    _decode_and_check(tb, w, batch, data, [data["phrases"][0], None], "after churn")


def test_graphs_from_file_and_from_the_cache_decode_the_same(tb, tmp_path):
    w = W.get_workload(2, B=4, T=150)
    data = W.batch_inputs(w)
    cc = w.vocab.case_class
    cache = tb.tb_cache_create(8 << 20)
    batch = tb.tb_batch_create(w.V, cc, w.B, arena_bytes=4 << 20)
    for i, p in enumerate(data["phrases"]):
        if i % 2:
            path = str(tmp_path / f"list{i}.tbg")
            tb.tb_graph_save(tb.tb_graph_compile(p, w.V, case_class=cc), path)
            g = tb.tb_graph_load(path)
        else:
            tb.tb_cache_compile(cache, p, w.V, case_class=cc)
            g, hit = tb.tb_cache_compile(cache, p, w.V, case_class=cc)
            assert hit
        tb.tb_batch_bind_stream(batch, i, g)
        g.free()                      # the caller's handle may go at once: a copy in flight keeps what it reads
        if i == 2:
            cache.destroy()           # ... and so may the cache that pinned the graph
            cache = tb.tb_cache_create(8 << 20)
    cache.destroy()
    _decode_and_check(tb, w, batch, data, data["phrases"], "file / cache")


def test_streaming_with_registered_models(tb):
    # chunked decoding of slots bound by id equals the offline decode of the same streams
    w = W.get_workload(2, B=3, T=64)
    data = W.batch_inputs(w)
    cc = w.vocab.case_class
    batch = tb.tb_batch_create(w.V, cc, w.B, arena_bytes=2 << 20)
    for i, p in enumerate(data["phrases"]):
        tb.tb_batch_bind_model(batch, i, tb.tb_batch_register_model(batch, tb.tb_graph_compile(p, w.V, case_class=cc)))
    logits = to_device(data["logits"])
    toks = [[] for _ in range(w.B)]
    valid = torch.full((w.B,), w.T, dtype=torch.int32, device="cuda:0")
    for c in range(w.T // 8):
        out = to_host(tb.tb_stream_chunk(batch, logits[:, 8 * c:8 * c + 8].contiguous(), 0, valid))
        for i in range(w.B):
            toks[i] += list(out["tokens"][i, :out["counts"][i]])
    for i, p in enumerate(data["phrases"]):
        ref = O.greedy_rnnt(oracle_graph(w, p), data["logits"][i])
        assert toks[i] == list(ref["tokens"])


def test_final_weights_after_greedy_and_beam(tb):
    # greedy: the charge on out_scores / out_states equals the oracle's; beam: on the [B, K] arrays, empty places kept
    w = W.get_workload(2, B=5, T=140)
    data = W.batch_inputs(w)
    cc = w.vocab.case_class
    lists = list(data["phrases"])
    lists[3] = None
    batch = tb.tb_batch_create(w.V, cc, w.B, arena_bytes=4 << 20, max_beam=4)
    for i, p in enumerate(lists):
        tb.tb_batch_bind_stream(batch, i, None if p is None else tb.tb_graph_compile(p, w.V, case_class=cc, lam=0.5))
    out = tb.tb_greedy_decode(batch, to_device(data["logits"]))
    before = out["scores"].clone()
    tb.tb_apply_final_weights(batch, out["scores"], out["states"])
    torch.cuda.synchronize()
    changed = 0
    for i, p in enumerate(lists):
        g = oracle_graph(w, p, lam=0.5)
        want = O.apply_final_weight(g, int(out["states"][i]), float(before[i]))
        assert np.float32(out["scores"][i].item()) == want
        changed += float(before[i]) != float(want)
    assert float(out["scores"][3]) == float(before[3])
    # every state of one graph, as a [1, K] call per group of four states
    g = oracle_graph(w, lists[0], lam=0.5)
    n = g.n_states
    states = torch.arange(0, 4 * (n // 4), dtype=torch.int32, device="cuda:0").reshape(-1, 4)
    for r in range(0, states.shape[0], 97):
        sc = torch.tensor([[1.5, float("-inf"), -2.25, 0.0]], device="cuda:0")
        st = states[r:r + 1].contiguous()
        tb.tb_apply_final_weights(batch, sc, st)
        torch.cuda.synchronize()
        for k in range(4):
            if k == 1:
                assert float(sc[0, k]) == float("-inf")
            else:
                assert np.float32(sc[0, k].item()) == O.apply_final_weight(g, int(st[0, k]), [1.5, 0, -2.25, 0.0][k])
    assert tb.tb_batch_status(batch) == 0
    bad = torch.tensor([[10 ** 6]], dtype=torch.int32, device="cuda:0")
    tb.tb_apply_final_weights(batch, torch.zeros((1, 1), device="cuda:0"), bad)
    assert tb.tb_batch_status(batch) == 2            # TB_STATUS_BAD_STATE: a state outside the graph is reported, not used
    assert tb.tb_batch_status(batch) == 0            # (reading the word clears it)


def test_error_codes_of_the_beam_and_lifecycle_calls(tb):
    w = W.get_workload(1, B=2, T=4, S=2, V=8, n_plants=0)
    data = W.batch_inputs(w)
    cc = w.vocab.case_class
    K = 4
    batch = tb.tb_batch_create(w.V, cc, 2, arena_bytes=1 << 20, max_beam=K, max_tree_steps=6)
    logits = to_device(data["logits"])
    dev = logits.device
    scores = torch.full((2, K), float("-inf"), device=dev); scores[:, 0] = 0
    states = torch.full((2, K), -1, dtype=torch.int32, device=dev)
    live = torch.zeros((2, K), dtype=torch.uint8, device=dev)
    par = torch.empty((2, K), dtype=torch.int32, device=dev); tok = torch.empty_like(par)

    def code(fn, *a, **k):
        with pytest.raises(tb.TbError) as e:
            fn(*a, **k)
        return e.value.code
    tb.tb_beam_reset(batch)
    assert code(tb.tb_beam_frames, batch, logits, False, scores, states, live, par, tok) == tb.TB_ERR_INVALID_ARG   # 8 steps, room for 6
    tb.tb_beam_frames(batch, logits[:, :3], False, scores, states, live, par, tok)                                    # 6 steps fit
    assert code(tb.tb_beam_frames, batch, logits[:, 3:], False, scores, states, live, par, tok) == tb.TB_ERR_INVALID_ARG
    wide = torch.zeros((2, 8), device=dev)
    assert code(tb.tb_beam_frames, batch, logits[:, :1], False, wide, torch.zeros((2, 8), dtype=torch.int32, device=dev),
                torch.zeros((2, 8), dtype=torch.uint8, device=dev), torch.zeros((2, 8), dtype=torch.int32, device=dev),
                torch.zeros((2, 8), dtype=torch.int32, device=dev)) == tb.TB_ERR_INVALID_ARG                          # K above max_beam
    tb.tb_beam_reset(batch)
    assert code(tb.tb_beam_step, batch, logits, logits.stride(0), 0, 3, scores, states, live, par, tok) == tb.TB_ERR_INVALID_ARG   # no such frame flag
    three = torch.zeros((3, 1), device=dev)
    assert code(tb.tb_apply_final_weights, batch, three, torch.zeros((3, 1), dtype=torch.int32, device=dev)) == tb.TB_ERR_INVALID_ARG   # more streams than slots
    other = tb.tb_graph_compile([[1, 2]], w.V + 1)
    assert code(tb.tb_batch_register_model, batch, other) == tb.TB_ERR_INVALID_ARG                                    # another vocabulary
    assert tb.tb_batch_status(batch) == 0


def test_binding_many_registered_models_at_once(tb):
    w = W.get_workload(2, B=6, T=150)
    data = W.batch_inputs(w)
    cc = w.vocab.case_class
    n_slots = 300                                       # more than one launch's worth of pairs
    batch = tb.tb_batch_create(w.V, cc, n_slots, arena_bytes=4 << 20)
    ids = [tb.tb_batch_register_model(batch, tb.tb_graph_compile(p, w.V, case_class=cc)) for p in data["phrases"]]
    slots = list(range(n_slots))
    models = [ids[i % 6] if i % 7 else -1 for i in range(n_slots)]
    tb.tb_batch_bind_models(batch, slots, models)
    lists = [None if models[i] < 0 else data["phrases"][models[i]] for i in range(6)]
    _decode_and_check(tb, w, batch, data, lists, "bound at once")
    # the last slots too: decode them through a strided view of the same logits
    tb.tb_batch_bind_models(batch, [5, 0, 299], [ids[0], -1, ids[3]])
    lists[5], lists[0] = data["phrases"][0], None
    _decode_and_check(tb, w, batch, data, lists, "re-bound at once")

    def code(*a):
        with pytest.raises(tb.TbError) as e:
            tb.tb_batch_bind_models(batch, *a)
        return e.value.code
    assert code([0, 1, 0], [ids[0], ids[1], ids[2]]) == tb.TB_ERR_INVALID_ARG      # a slot twice
    assert code([0, 300], [ids[0], ids[1]]) == tb.TB_ERR_BAD_SLOT
    assert code([0, 1], [ids[0], 77]) == tb.TB_ERR_INVALID_ARG
    _decode_and_check(tb, w, batch, data, lists, "nothing changed by refused calls")
    with pytest.raises(tb.TbError):
        tb.tb_batch_unregister_model(batch, ids[3])                               # slot 299 still uses it
    tb.tb_batch_bind_models(batch, [], [])


def test_binding_forty_streams_in_one_call(tb):
    """tb_batch_bind_streams with more graphs than one binding launch carries (several launches of sixteen, each block
    reading one image from page-locked memory in place), some of them on the heap (copied), some slots unbound."""
    w = W.get_workload(2, B=40, T=60, n_phrases=30, n_plants=4)
    data = W.batch_inputs(w)
    logits = to_device(data["logits"])
    batch = tb.tb_batch_create(w.V, w.vocab.case_class, w.B, arena_bytes=8 << 20)
    lists = list(data["phrases"])
    lists[7] = lists[23] = None
    graphs = [None if p is None else tb.tb_graph_compile(p, w.V, case_class=w.vocab.case_class,
                                                         flags=tb.TB_COMPILE_PAGEABLE if i in (18, 33) else 0) for i, p in enumerate(lists)]
    tb.tb_batch_bind_streams(batch, list(range(w.B)), graphs)
    del graphs                                           # (the library holds what it still reads)
    out = to_host(tb.tb_greedy_decode(batch, logits))
    assert tb.tb_batch_status(batch) == 0
    for i in range(w.B):
        check_greedy(out, i, O.greedy_rnnt(oracle_graph(w, lists[i]), data["logits"][i]), "forty at once")
    assert out["states"][7] == -1 and out["states"][23] == -1


def test_binding_many_streams_at_once(tb):
    """tb_batch_bind_streams: several slots get new lists (or lose theirs) in one copy and one launch; the result is
    what the same binds one by one give, other slots are untouched, and a small arena falls back to single binds."""
    w = W.get_workload(2, B=8, T=100, n_phrases=40, n_plants=6)
    data = W.batch_inputs(w)
    logits = to_device(data["logits"])
    batch = tb.tb_batch_create(w.V, w.vocab.case_class, w.B, arena_bytes=4 << 20)
    graphs = [tb.tb_graph_compile(p, w.V, case_class=w.vocab.case_class) for p in data["phrases"]]
    tb.tb_batch_bind_streams(batch, list(range(w.B)), graphs)
    out = to_host(tb.tb_greedy_decode(batch, logits))
    for i in range(w.B):
        check_greedy(out, i, O.greedy_rnnt(oracle_graph(w, data["phrases"][i]), data["logits"][i]), "all at once")
    # a second round: three slots swap lists, one is unbound, the rest stay
    other = [W.stream_phrases(w, 50 + i) for i in range(3)]
    tb.tb_batch_bind_streams(batch, [6, 1, 4, 2], [tb.tb_graph_compile(p, w.V, case_class=w.vocab.case_class) for p in other] + [None])
    lists = list(data["phrases"])
    lists[6], lists[1], lists[4], lists[2] = other[0], other[1], other[2], None
    out = to_host(tb.tb_greedy_decode(batch, logits))
    for i in range(w.B):
        check_greedy(out, i, O.greedy_rnnt(oracle_graph(w, lists[i]), data["logits"][i]), "second round")
    assert out["states"][2] == -1
    # streaming state is reset by the bind, as with a single bind
    valid = torch.full((w.B,), w.T, dtype=torch.int32, device="cuda:0")
    tb.tb_stream_chunk(batch, logits[:, :8], 0, valid)
    tb.tb_batch_bind_streams(batch, [0, 3], [graphs[0], graphs[3]])
    ch = to_host(tb.tb_stream_chunk(batch, logits[:, :8], 0, valid))
    assert ch["cursors"][0] == 8 and ch["cursors"][3] == 8 and ch["cursors"][1] == 16
    # binds and chunk in one call: the same as the two calls
    tb.tb_batch_bind_streams(batch, [0, 3], [graphs[0], graphs[3]])
    want = to_host(tb.tb_stream_chunk(batch, logits[:, :8], 0, valid))
    got = to_host(tb.tb_stream_chunk_binds(batch, [0, 3], [graphs[0], graphs[3]], logits[:, :8], 0, valid))
    for i in (0, 3):
        n = int(want["counts"][i])
        assert int(got["counts"][i]) == n and np.array_equal(got["tokens"][i, :n], want["tokens"][i, :n])
        assert got["scores"][i] == want["scores"][i] and got["states"][i] == want["states"][i] and got["cursors"][i] == 8
    assert got["cursors"][1] == want["cursors"][1] + 8                    # the other slots went on
    more = to_host(tb.tb_stream_chunk_binds(batch, [], [], logits[:, 8:16], 0, valid))      # no binds: a plain chunk
    assert more["cursors"][0] == 16
    assert tb.tb_batch_bind_counts(batch) == dict(pulled=2, copied=0)     # the two binds rode on the chunk's launch
    # a graph on the heap cannot be read by the kernel in place: the group goes ahead of the launch; a slot that is
    # unbound in the same call as another is bound: carried out by the launch; and the result is the same every way
    heap = tb.tb_graph_compile(data["phrases"][5], w.V, case_class=w.vocab.case_class, flags=tb.TB_COMPILE_PAGEABLE)
    a_ = to_host(tb.tb_stream_chunk_binds(batch, [5, 6], [heap, None], logits[:, :8], 0, valid))
    assert tb.tb_batch_bind_counts(batch) == dict(pulled=2, copied=2)
    b_ = to_host(tb.tb_stream_chunk_binds(batch, [5, 6], [graphs[5], None], logits[:, :8], 0, valid))
    assert tb.tb_batch_bind_counts(batch) == dict(pulled=4, copied=2)
    ref5 = O.stream_chunk(oracle_graph(w, data["phrases"][5]), data["logits"][5][:8], 0, 0, w.T, O.StreamState(0, 0, 0, 0.0, 0))
    ref6 = O.stream_chunk(None, data["logits"][6][:8], 0, 0, w.T, O.StreamState(-1, 0, 0, 0.0, 0))
    for got_ in (a_, b_):
        for i, ref in ((5, ref5), (6, ref6)):
            n = int(got_["counts"][i])
            assert n == len(ref["tokens"]) and np.array_equal(got_["tokens"][i, :n], ref["tokens"]) and got_["cursors"][i] == 8
        assert got_["states"][6] == -1 and a_["scores"][5] == b_["scores"][5]
    # a chunk that is refused binds nothing
    with pytest.raises(tb.TbError):
        tb.tb_stream_chunk_binds(batch, [7], [graphs[0]], logits[:, :8], 0, None)        # no frame counts: the chunk is refused
    assert tb.tb_batch_bind_counts(batch) == dict(pulled=4, copied=2)
    # slots beyond the chunk's are bound ahead of the launch
    tb.tb_stream_chunk_binds(batch, [7], [graphs[7]], logits[:4, :8], 0, valid[:4])
    assert tb.tb_batch_bind_counts(batch) == dict(pulled=4, copied=3)
    assert tb.tb_batch_status(batch) == 0
    # errors: checked before anything changes
    with pytest.raises(tb.TbError) as e:
        tb.tb_stream_chunk_binds(batch, [0, 0], [graphs[0], graphs[1]], logits[:, :8], 0, valid)
    assert e.value.code == tb.TB_ERR_INVALID_ARG
    with pytest.raises(tb.TbError) as e:
        tb.tb_batch_bind_streams(batch, [0, 0], [graphs[0], graphs[1]])
    assert e.value.code == tb.TB_ERR_INVALID_ARG
    with pytest.raises(tb.TbError) as e:
        tb.tb_batch_bind_streams(batch, [0, w.B], [graphs[0], graphs[1]])
    assert e.value.code == tb.TB_ERR_BAD_SLOT
    # many rounds into a small arena: space is handed back, and when no contiguous block fits the group the binds
    # still succeed one by one
    small = tb.tb_batch_create(w.V, w.vocab.case_class, w.B, arena_bytes=360 << 10)
    for r in range(12):
        sl = [(r + j) % w.B for j in range(4)]
        tb.tb_batch_bind_streams(small, sl, [graphs[(r + 2 * j) % w.B] for j in range(4)])
    tb.tb_batch_bind_streams(small, list(range(w.B)), [None] * w.B)
    tb.tb_batch_bind_streams(small, [0, 1, 2, 3, 4], graphs[:5])
    out = to_host(tb.tb_greedy_decode(small, logits))
    for i in range(5):
        check_greedy(out, i, O.greedy_rnnt(oracle_graph(w, data["phrases"][i]), data["logits"][i]), "small arena")
    assert tb.tb_batch_status(batch) == 0 and tb.tb_batch_status(small) == 0


def test_graph_images_in_page_locked_memory_and_on_the_heap(tb):
    """Once a batch exists, compiled and loaded graphs keep their device image in the library's pool of page-locked
    memory and binds copy from there; TB_COMPILE_PAGEABLE keeps an image on the heap, and binds stage it.  Both kinds,
    mixed in one group and one by one, must decode the same; images are released and their room is reused; more
    images than one piece of the pool holds spill into further pieces."""
    w = W.get_workload(2, B=8, T=100, n_phrases=40, n_plants=6)
    data = W.batch_inputs(w)
    logits = to_device(data["logits"])
    batch = tb.tb_batch_create(w.V, w.vocab.case_class, w.B, arena_bytes=8 << 20)
    refs = [O.greedy_rnnt(oracle_graph(w, data["phrases"][i]), data["logits"][i]) for i in range(w.B)]

    def graphs(kind):
        return [tb.tb_graph_compile(p, w.V, case_class=w.vocab.case_class,
                                    flags=tb.TB_COMPILE_PAGEABLE if (kind == "heap" or (kind == "mixed" and i % 3 == 1)) else 0)
                for i, p in enumerate(data["phrases"])]
    for kind in ("pool", "heap", "mixed"):
        for grouped in (True, False):
            gs = graphs(kind)
            tb.tb_batch_bind_streams(batch, list(range(w.B)), [None] * w.B)
            if grouped:
                tb.tb_batch_bind_streams(batch, list(range(w.B)), gs)
            else:
                for i, g in enumerate(gs):
                    tb.tb_batch_bind_stream(batch, i, g)
            del gs                                           # the copies in flight hold the graphs they read
            out = to_host(tb.tb_greedy_decode(batch, logits))
            for i in range(w.B):
                check_greedy(out, i, refs[i], f"{kind}, grouped={grouped}")
    # a long series of lists of different sizes, kept alive in a window: images come and go, room is reused, and the
    # total (about 60 MB alive at the peak) needs more than one 32 MB piece
    wl = W.get_workload(5, B=4)
    big = tb.tb_batch_create(wl.V, wl.vocab.case_class, 4, arena_bytes=16 << 20)
    alive = []
    for r in range(700):
        g = tb.tb_graph_compile(W.stream_phrases(wl, r % 97), wl.V, case_class=wl.vocab.case_class)
        alive.append(g)
        if len(alive) > 450:
            del alive[:200]
        if r % 50 == 49:
            tb.tb_batch_bind_streams(big, [0, 1, 2, 3], alive[-4:])
    torch.cuda.synchronize()
    assert tb.tb_batch_status(big) == 0
    # what was bound last decodes as its list says (no image was overwritten by a later one)
    lists = [W.stream_phrases(wl, r % 97) for r in range(696, 700)]
    x = np.stack([np.ascontiguousarray(W.stream_inputs(wl, i)["logits"][:60, :, : wl.V + 1]) for i in range(4)])
    out = to_host(tb.tb_greedy_decode(big, to_device(x)))
    for i in range(4):
        check_greedy(out, i, O.greedy_rnnt(oracle_graph(wl, lists[i]), x[i]), "after many images")
