"""GPU parity for tb_beam_step / tb_beam_backtrace and tb_stream_chunk against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2608_21343_b200 import workloads as W
from helpers import SCORE_TOL, make_batch, oracle_graph, to_device, to_host

pytestmark = pytest.mark.gpu


def run_beam(tb, w, data, K, phrase_lists=None, batch=None, merge=False, prune_delta=None):
    """Frame-synchronous driver: E = w.S rows per frame shared by all hypotheses of a stream.
    (batch: one made by the caller, with slot i bound unless phrase_lists[i] is None)"""
    phrase_lists = data["phrases"] if phrase_lists is None else phrase_lists
    B, T, E, Wd = data["logits"].shape
    if batch is None:
        batch, _ = make_batch(tb, w, phrase_lists, max_beam=K, max_tree_steps=T * E)
    if prune_delta is not None:
        tb.tb_batch_set_beam_prune(batch, prune_delta)
    logits = to_device(data["logits"])
    dev = logits.device
    scores = torch.full((B, K), float("-inf"), device=dev)
    scores[:, 0] = 0.0
    states = torch.full((B, K), -1, dtype=torch.int32, device=dev)
    states[:, 0] = torch.tensor([0 if p is not None else -1 for p in phrase_lists], dtype=torch.int32, device=dev)
    live = torch.zeros((B, K), dtype=torch.uint8, device=dev)
    par = torch.empty((B, K), dtype=torch.int32, device=dev)
    tok = torch.empty((B, K), dtype=torch.int32, device=dev)
    tb.tb_beam_reset(batch)
    tree = []
    sb, st, se, _ = logits.stride()
    for t in range(T):
        for e in range(E):
            frame = (tb.TB_FRAME_NEW_MERGE if merge else tb.TB_FRAME_NEW) if e == 0 else tb.TB_FRAME_SAME
            tb.tb_beam_step(batch, logits, sb, 0, frame, scores, states, live, par, tok, offset=t * st + e * se)
            tree.append(torch.stack([par, tok], dim=-1).clone())
    toks, lens = tb.tb_beam_backtrace(batch, B, K, T * E)
    assert tb.tb_batch_status(batch) == 0
    torch.cuda.synchronize()
    return dict(scores=scores.cpu().numpy(), states=states.cpu().numpy(), live=live.cpu().numpy(),
                tree=torch.stack(tree, dim=1).cpu().numpy(), tokens=toks.cpu().numpy(), lens=lens.cpu().numpy())


def compare_beam(w, data, out, K, streams, phrase_lists=None, merge=False):
    phrase_lists = data["phrases"] if phrase_lists is None else phrase_lists
    for i in streams:
        ref = O.beam_decode(oracle_graph(w, phrase_lists[i]), data["logits"][i], K, merge=merge)
        assert np.array_equal(out["tree"][i], ref["tree"]), f"stream {i}: (parent, token) tree"
        assert np.array_equal(out["states"][i], ref["states"]), f"stream {i}: states"
        assert np.array_equal(out["lens"][i], ref["lens"]), f"stream {i}: lengths"
        for k in range(K):
            assert np.array_equal(out["tokens"][i, k, :ref["lens"][k]], ref["tokens"][k]), f"stream {i} hyp {k}"
        fin = np.isfinite(ref["scores"])
        assert np.array_equal(np.isfinite(out["scores"][i]), fin)
        assert np.all(np.abs(out["scores"][i][fin] - ref["scores"][fin]) <= SCORE_TOL), f"stream {i}: scores"


def test_workload4_beam_reduced(tb):
    w = W.get_workload(4, B=5, T=60, n_plants=6)
    data = W.batch_inputs(w)
    lists = list(data["phrases"])
    lists[2] = None
    out = run_beam(tb, w, data, w.K, lists)
    compare_beam(w, data, out, w.K, range(w.B), lists)


def _competing_alignments(w, seed):
    """Logits on which alignments of the same short transcript compete for the beam: a token costs about 2 against
    blank in the first row of a frame, the second row closes the frame, noise of 0.3 decides the rest."""
    rng = np.random.default_rng(seed)
    x = (rng.standard_normal((w.B, w.T, w.S, w.V + 1)) * 0.3).astype(np.float32)
    x[:, :, 0, w.V] += 2.0
    x[:, :, 1:, :w.V] -= 2.0
    return x


@pytest.mark.parametrize("K", [8, 32])
def test_beam_with_merging_of_equal_sequences(tb, K):
    w = W.get_workload(1, B=4, T=12, S=2, V=8, n_plants=0)
    data = W.batch_inputs(w)
    data["logits"] = _competing_alignments(w, 5)
    lists = [None, data["phrases"][1], None, data["phrases"][3]]
    batch, _ = make_batch(tb, w, lists, lam=0.125, max_beam=K, max_tree_steps=w.T * w.S)
    out = run_beam(tb, w, data, K, lists, batch=batch, merge=True)
    changed = 0
    for i in range(w.B):
        g = oracle_graph(w, lists[i], lam=0.125)
        ref = O.beam_decode(g, data["logits"][i], K, merge=True)
        assert np.array_equal(out["tree"][i], ref["tree"]), f"stream {i}: (parent, token) tree"
        assert np.array_equal(out["states"][i], ref["states"]) and np.array_equal(out["lens"][i], ref["lens"])
        for k in range(K):
            assert np.array_equal(out["tokens"][i, k, :ref["lens"][k]], ref["tokens"][k])
        fin = np.isfinite(ref["scores"])
        assert np.array_equal(np.isfinite(out["scores"][i]), fin)
        assert np.all(np.abs(out["scores"][i][fin] - ref["scores"][fin]) <= SCORE_TOL)
        changed += not np.array_equal(ref["tree"], O.beam_decode(g, data["logits"][i], K)["tree"])
    assert changed >= 3                       # on these inputs merging does change what the beam holds


@pytest.mark.parametrize("delta,merge", [(0.5, False), (1.5, True), (0.0, True), (float("inf"), False)])
def test_beam_with_pruning(tb, delta, merge):
    w = W.get_workload(1, B=4, T=12, S=2, V=8, n_plants=0)
    data = W.batch_inputs(w)
    data["logits"] = _competing_alignments(w, 7)
    lists = [None, data["phrases"][1], None, data["phrases"][3]]
    K = 16
    batch, _ = make_batch(tb, w, lists, lam=0.125, max_beam=K, max_tree_steps=w.T * w.S)
    out = run_beam(tb, w, data, K, lists, batch=batch, merge=merge, prune_delta=delta)
    changed = 0
    for i in range(w.B):
        g = oracle_graph(w, lists[i], lam=0.125)
        ref = O.beam_decode(g, data["logits"][i], K, merge=merge, prune_delta=delta)
        assert np.array_equal(out["tree"][i], ref["tree"]), f"stream {i}: (parent, token) tree"
        assert np.array_equal(out["states"][i], ref["states"]) and np.array_equal(out["lens"][i], ref["lens"])
        fin = np.isfinite(ref["scores"])
        assert np.array_equal(np.isfinite(out["scores"][i]), fin)
        assert np.all(np.abs(out["scores"][i][fin] - ref["scores"][fin]) <= SCORE_TOL)
        changed += not np.array_equal(ref["tree"], O.beam_decode(g, data["logits"][i], K, merge=merge)["tree"])
    assert (changed >= 2) == (delta < 10)     # a finite threshold bites on these inputs, an infinite one never
    tb.tb_batch_set_beam_prune(batch, -1.0)
    with pytest.raises(tb.TbError):
        tb.tb_batch_set_beam_prune(batch, float("nan"))


def test_beam_merging_is_off_unless_asked_for(tb):
    w = W.get_workload(1, B=2, T=10, S=2, V=8, n_plants=0)
    data = W.batch_inputs(w)
    data["logits"] = _competing_alignments(w, 6)
    out = run_beam(tb, w, data, 16, [None, None])
    compare_beam(w, data, out, 16, range(w.B), [None, None])


@pytest.mark.parametrize("K", [1, 2, 7])
def test_beam_other_widths_fp32(tb, K):
    w = W.get_workload(1, B=3, T=25, S=2)
    data = W.batch_inputs(w)
    out = run_beam(tb, w, data, K)
    compare_beam(w, data, out, K, range(w.B))
    if K == 1:       # a beam of one is greedy decoding
        for i in range(w.B):
            ref = O.greedy_rnnt(oracle_graph(w, data["phrases"][i]), data["logits"][i])
            n = len(ref["tokens"])
            assert out["lens"][i, 0] == n and np.array_equal(out["tokens"][i, 0, :n], ref["tokens"])


def test_beam_step_frozen_and_empty(tb):
    """One step by hand: ordering of equal scores, a frozen hypothesis carried, empty places."""
    w = W.get_workload(1, B=1, T=1)
    batch, _ = make_batch(tb, w, [[[0]]], max_beam=3)
    V = w.V
    rows = torch.full((1, 3, V + 1), -5.0, device="cuda:0")
    rows[0, 0, 0] = 1.0           # +1 bonus for class 0 -> 2.0
    rows[0, 0, 4] = 2.0
    rows[0, 0, V] = 2.0
    rows[0, 1, :] = 9.0           # frozen hypothesis: its row must not be read
    scores = torch.tensor([[0.0, 2.0, float("-inf")]], device="cuda:0")
    states = torch.tensor([[0, 0, -1]], dtype=torch.int32, device="cuda:0")
    live = torch.tensor([[1, 0, 0]], dtype=torch.uint8, device="cuda:0")
    par = torch.empty((1, 3), dtype=torch.int32, device="cuda:0")
    tok = torch.empty((1, 3), dtype=torch.int32, device="cuda:0")
    tb.tb_beam_step(batch, rows, 3 * (V + 1), V + 1, False, scores, states, live, par, tok)
    torch.cuda.synchronize()
    assert par.tolist() == [[0, 0, 0]] and tok.tolist() == [[0, 4, V]]
    assert scores.tolist() == [[2.0, 2.0, 2.0]] and states.tolist() == [[1, 0, 0]] and live.tolist() == [[1, 1, 0]]
    ref_scores = np.array([0.0, 2.0, -np.inf], dtype=np.float32)
    ref_states = np.array([0, 0, -1], dtype=np.int32)
    ref_live = np.array([1, 0, 0], dtype=np.uint8)
    rp, rt = O.beam_step(O.Graph([[0]], V, case_class=w.vocab.case_class), rows[0].cpu().numpy(), ref_scores, ref_states, ref_live)
    assert rp.tolist() == [0, 0, 0] and rt.tolist() == [0, 4, V]


def run_stream(tb, w, n_chunks, weights_lam=None, in_chunk=False, flags=0, counts=None):
    """Streaming decode with stream churn on both sides; compares after every chunk.  in_chunk: the new streams'
    binds travel with the chunk call (tb_stream_chunk_binds) instead of one tb_batch_bind_stream each."""
    sched_gpu = W.ChurnSchedule(w)
    batch = tb.tb_batch_create(w.V, w.vocab.case_class, w.B, arena_bytes=8 << 20)
    tb.tb_batch_set_flags(batch, flags)
    slots = [dict(graph=None, st=None, t0=0) for _ in range(w.B)]
    n_binds = 0
    for c in range(n_chunks):
        chunk, lengths, binds = sched_gpu.next_chunk()
        new = []
        for slot, stream_id, phrases in binds:
            g = tb.tb_graph_compile(phrases, w.V, case_class=w.vocab.case_class)
            if in_chunk:
                new.append((slot, g))
            else:
                tb.tb_batch_bind_stream(batch, slot, g)
            og = oracle_graph(w, phrases)
            slots[slot] = dict(graph=og, st=O.StreamState(0, 0, 0, 0.0, 0), t0=0)
            n_binds += 1
        if in_chunk:
            out = to_host(tb.tb_stream_chunk_binds(batch, [sl for sl, _ in new], [g for _, g in new], to_device(chunk), w.n_dur,
                                                   torch.from_numpy(lengths).to("cuda:0")))
            del new                                   # (the library holds the graphs for as long as it reads them)
        else:
            out = to_host(tb.tb_stream_chunk(batch, to_device(chunk), w.n_dur,
                                             torch.from_numpy(lengths).to("cuda:0")))
        for i in range(w.B):
            sl = slots[i]
            ref = O.stream_chunk(sl["graph"], chunk[i], w.n_dur, sl["t0"], int(lengths[i]), sl["st"])
            sl["t0"] += w.chunk
            n = int(out["counts"][i])
            assert n == len(ref["tokens"]), (c, i)
            assert np.array_equal(out["tokens"][i, :n], ref["tokens"]), (c, i)
            assert np.array_equal(out["frames"][i, :n], ref["frames"]), (c, i)
            assert np.array_equal(out["durs"][i, :n], ref["durs"]), (c, i)
            assert out["states"][i] == sl["st"].state and out["cursors"][i] == sl["st"].t, (c, i)
            assert abs(float(out["scores"][i]) - float(sl["st"].score)) <= SCORE_TOL, (c, i)
    assert tb.tb_batch_status(batch) == 0
    if counts is not None:
        counts.update(tb.tb_batch_bind_counts(batch))
    return n_binds


def test_workload5_streaming_tdt_with_churn_reduced(tb):
    w = W.get_workload(5, B=12, T=90, T_lo=20, n_phrases=60, n_phrases_lo=10)
    n_binds = run_stream(tb, w, n_chunks=30)
    assert n_binds > 2 * w.B          # slots were refilled while others kept running


def test_streaming_binds_carried_out_by_the_chunk_launch(tb):
    """tb_stream_chunk_binds: the first chunk's twenty binds exceed what a launch carries and go ahead of it; the
    refills afterwards (a few per chunk) are carried out by the chunk's own launch -- the re-bound slot's block reads
    the image from host memory -- and the decode is the oracle's, chunk by chunk, as with single binds."""
    w = W.get_workload(5, B=20, T=90, T_lo=20, n_phrases=60, n_phrases_lo=10)
    counts = {}
    n_binds = run_stream(tb, w, n_chunks=40, in_chunk=True, counts=counts)
    assert counts["copied"] == w.B and counts["pulled"] == n_binds - w.B and counts["pulled"] > w.B
    # the same with the switch that keeps every bind ahead of the launch
    counts = {}
    n_binds = run_stream(tb, w, n_chunks=12, in_chunk=True, flags=tb.TB_FLAG_COPIED_BINDS, counts=counts)
    assert counts["pulled"] == 0 and counts["copied"] == n_binds


def test_streaming_rnnt_chunked_equals_offline(tb):
    """Sec. 2.3: state carried across chunk boundaries -- chunks of 8 frames give the offline result."""
    w = W.get_workload(2, B=4, T=64, n_phrases=50, n_plants=6)
    data = W.batch_inputs(w)
    batch, _ = make_batch(tb, w, data["phrases"])
    logits = to_device(data["logits"])
    off = to_host(tb.tb_greedy_decode(batch, logits))
    valid = torch.full((w.B,), w.T, dtype=torch.int32, device="cuda:0")
    toks = [[] for _ in range(w.B)]
    for c in range(0, w.T, 8):
        out = to_host(tb.tb_stream_chunk(batch, logits[:, c:c + 8], 0, valid))
        for i in range(w.B):
            toks[i] += list(zip(out["tokens"][i, :out["counts"][i]], out["frames"][i, :out["counts"][i]]))
    for i in range(w.B):
        n = int(off["counts"][i])
        assert toks[i] == list(zip(off["tokens"][i, :n], off["frames"][i, :n]))
        assert out["states"][i] == off["states"][i] and out["scores"][i] == off["scores"][i]
        assert out["cursors"][i] == w.T


def run_beam_frames(tb, w, data, K, phrase_lists, batch, merge=False, chunks=(None,)):
    """The same decode through tb_beam_frames: the whole utterance in one launch, or chunk by chunk."""
    B, T, E, Wd = data["logits"].shape
    logits = to_device(data["logits"])
    dev = logits.device
    scores = torch.full((B, K), float("-inf"), device=dev)
    scores[:, 0] = 0.0
    states = torch.full((B, K), -1, dtype=torch.int32, device=dev)
    states[:, 0] = torch.tensor([0 if p is not None else -1 for p in phrase_lists], dtype=torch.int32, device=dev)
    live = torch.zeros((B, K), dtype=torch.uint8, device=dev)
    par = torch.empty((B, K), dtype=torch.int32, device=dev)
    tok = torch.empty((B, K), dtype=torch.int32, device=dev)
    tb.tb_beam_reset(batch)
    t0 = 0
    for n in chunks:
        n = T - t0 if n is None else n
        tb.tb_beam_frames(batch, logits[:, t0:t0 + n], merge, scores, states, live, par, tok)
        t0 += n
    assert t0 == T
    toks, lens = tb.tb_beam_backtrace(batch, B, K, T * E)
    assert tb.tb_batch_status(batch) == 0
    torch.cuda.synchronize()
    return dict(scores=scores.cpu().numpy(), states=states.cpu().numpy(), tokens=toks.cpu().numpy(), lens=lens.cpu().numpy(),
                last=torch.stack([par, tok], dim=-1).cpu().numpy())


@pytest.mark.parametrize("merge,chunks", [(False, (None,)), (True, (None,)), (True, (5, 1, 6)), (False, (1,) * 12)])
def test_beam_frames_in_one_launch_equals_the_steps(tb, merge, chunks):
    w = W.get_workload(1, B=4, T=12, S=2, V=8, n_plants=0)
    data = W.batch_inputs(w)
    data["logits"] = _competing_alignments(w, 8)
    lists = [None, data["phrases"][1], None, data["phrases"][3]]
    K = 16
    batch, _ = make_batch(tb, w, lists, lam=0.125, max_beam=K, max_tree_steps=w.T * w.S)
    tb.tb_batch_set_beam_prune(batch, 3.0)
    out = run_beam_frames(tb, w, data, K, lists, batch, merge=merge, chunks=chunks)
    for i in range(w.B):
        ref = O.beam_decode(oracle_graph(w, lists[i], lam=0.125), data["logits"][i], K, merge=merge, prune_delta=3.0)
        assert np.array_equal(out["states"][i], ref["states"]) and np.array_equal(out["lens"][i], ref["lens"])
        assert np.array_equal(out["last"][i], ref["tree"][-1])
        for k in range(K):
            assert np.array_equal(out["tokens"][i, k, :ref["lens"][k]], ref["tokens"][k])
        fin = np.isfinite(ref["scores"])
        assert np.array_equal(np.isfinite(out["scores"][i]), fin)
        assert np.all(np.abs(out["scores"][i][fin] - ref["scores"][fin]) <= SCORE_TOL)


def test_beam_frames_on_workload4_reduced(tb):
    w = W.get_workload(4, B=5, T=60, n_plants=6)
    data = W.batch_inputs(w)
    lists = list(data["phrases"])
    lists[2] = None
    batch, _ = make_batch(tb, w, lists, max_beam=w.K, max_tree_steps=w.T * w.S)
    out = run_beam_frames(tb, w, data, w.K, lists, batch, chunks=(8,) * 7 + (4,))
    for i in range(w.B):
        ref = O.beam_decode(oracle_graph(w, lists[i]), data["logits"][i], w.K)
        assert np.array_equal(out["states"][i], ref["states"]) and np.array_equal(out["lens"][i], ref["lens"])
        for k in range(w.K):
            assert np.array_equal(out["tokens"][i, k, :ref["lens"][k]], ref["tokens"][k])
        fin = np.isfinite(ref["scores"])
        assert np.all(np.abs(out["scores"][i][fin] - ref["scores"][fin]) <= SCORE_TOL)


@pytest.mark.parametrize("K", [8, 10, 12, 32])
def test_beam_widths_whose_shared_memory_straddles_the_default_limit(tb, K):
    # V = 1024: K * (V + 1) floats plus the tables is 33-49 KB of dynamic shared memory, which together with the
    # kernel's static 16 KB crosses the 48 KB a launch may use without opting in
    w = W.get_workload(4, B=2, T=12, n_plants=2)
    data = W.batch_inputs(w)
    out = run_beam(tb, w, data, K)
    compare_beam(w, data, out, K, range(w.B))
    batch, _ = make_batch(tb, w, data["phrases"], max_beam=K, max_tree_steps=w.T * w.S)
    fr = run_beam_frames(tb, w, data, K, data["phrases"], batch)
    assert np.array_equal(fr["tokens"], out["tokens"]) and np.array_equal(fr["scores"], out["scores"])


@pytest.mark.parametrize("K", [4, 16])
def test_beam_frames_when_the_reduced_rows_do_not_suffice(tb, K):
    """tb_beam_frames reduces every row to its few best tokens ahead of the steps and redoes a step on the whole row
    when those cannot be shown to hold the K best candidates.  Flat rows (all tokens equal, or equal but for a few)
    force that second path at almost every step; rows with a clear order in between take the short one.  Both,
    with and without the pre-pass, against the oracle."""
    w = W.get_workload(4, B=4, T=30, V=256, n_phrases=30, n_plants=3)
    data = W.batch_inputs(w)
    x = W.bf16_bits_to_f32(data["logits"])
    x[:, 0::3, :, :w.V] = 0.0                                         # every token the same
    x[:, 1::3, :, :w.V] = np.round(x[:, 1::3, :, :w.V])               # a handful of distinct values
    x[:, :, :, w.V] = 0.25                                            # blank close to the tokens: tokens do get emitted
    data["logits"] = W.f32_to_bf16_bits(x)
    lists = [data["phrases"][0], None, data["phrases"][2], data["phrases"][3]]
    refs = [O.beam_decode(oracle_graph(w, lists[i]), data["logits"][i], K, merge=True) for i in range(w.B)]
    for flags in (0, tb.TB_FLAG_BEAM_WHOLE_ROWS):
        batch, _ = make_batch(tb, w, lists, max_beam=K, max_tree_steps=w.T * w.S)
        tb.tb_batch_set_flags(batch, flags)
        out = run_beam_frames(tb, w, data, K, lists, batch, merge=True, chunks=(7, 23))
        for i in range(w.B):
            ref = refs[i]
            assert np.array_equal(out["states"][i], ref["states"]) and np.array_equal(out["lens"][i], ref["lens"]), (flags, i)
            assert np.array_equal(out["last"][i], ref["tree"][-1]), (flags, i)
            for k in range(K):
                assert np.array_equal(out["tokens"][i, k, :ref["lens"][k]], ref["tokens"][k]), (flags, i, k)
            fin = np.isfinite(ref["scores"])
            assert np.array_equal(np.isfinite(out["scores"][i]), fin)
            assert np.all(np.abs(out["scores"][i][fin] - ref["scores"][fin]) <= SCORE_TOL), (flags, i)


@pytest.mark.parametrize("block", range(4))
def test_beam_frames_random_configurations(tb, block):
    """Random small configurations of tb_beam_frames against the oracle: beams of 1 to 32 (narrow ones are decoded by a
    team of warps, wide ones by the whole block), vocabularies of 4 to 1024, 1-3 expansions per frame, fp32 and bf16,
    bound and unbound streams, with and without merging and pruning, each decode cut into random chunks."""
    for seed in range(30 * block, 30 * block + 30):
        rng = np.random.default_rng(41000 + seed)
        V = int(rng.choice([4, 8, 30, 200, 1024]))
        B, T, E = int(rng.integers(1, 5)), int(rng.integers(2, 40)), int(rng.integers(1, 4))
        K = int(rng.choice([1, 2, 3, 4, 5, 8, 16, 32]))
        f32 = bool(rng.integers(0, 2))
        cc = (np.arange(V) // int(rng.integers(1, 4))).astype(np.int32)
        lists = [None if rng.random() < 0.3 else
                 [[int(t) for t in rng.integers(0, V, size=rng.integers(1, 5))] for _ in range(int(rng.integers(1, 12)))]
                 for _ in range(B)]
        lam = float(rng.choice([0.125, 0.5, 1.0]))
        x = (rng.standard_normal((B, T, E, V + 1)) * float(rng.choice([0.05, 0.3, 1.0]))).astype(np.float32)
        x[:, :, 0, V] += 2.0
        if E > 1:
            x[:, :, 1:, :V] -= 2.0
        x = W.round_to_dtype(x, "f32" if f32 else "bf16")
        xs = x if f32 else W.to_storage(x, "bf16")
        merge = bool(rng.integers(0, 4) != 0)
        delta = float(rng.choice([0.5, 2.0, 8.0])) if rng.random() < 0.5 else None
        batch = tb.tb_batch_create(V, cc, B, arena_bytes=8 << 20, max_beam=K, max_tree_steps=T * E)
        if delta is not None:
            tb.tb_batch_set_beam_prune(batch, delta)
        for i, p in enumerate(lists):
            tb.tb_batch_bind_stream(batch, i, None if p is None else tb.tb_graph_compile(p, V, case_class=cc, lam=lam))
        t = to_device(xs)
        dev = t.device
        scores = torch.full((B, K), float("-inf"), device=dev)
        scores[:, 0] = 0.0
        states = torch.full((B, K), -1, dtype=torch.int32, device=dev)
        states[:, 0] = torch.tensor([0 if p is not None else -1 for p in lists], dtype=torch.int32, device=dev)
        live = torch.zeros((B, K), dtype=torch.uint8, device=dev)
        par = torch.empty((B, K), dtype=torch.int32, device=dev)
        tok = torch.empty((B, K), dtype=torch.int32, device=dev)
        tb.tb_beam_reset(batch)
        t0 = 0
        while t0 < T:
            n = int(rng.integers(1, T - t0 + 1))
            tb.tb_beam_frames(batch, t[:, t0:t0 + n], merge, scores, states, live, par, tok)
            t0 += n
        toks, lens = tb.tb_beam_backtrace(batch, B, K, T * E)
        torch.cuda.synchronize()
        assert tb.tb_batch_status(batch) == 0, seed
        sc, stt, toks, lens = scores.cpu().numpy(), states.cpu().numpy(), toks.cpu().numpy(), lens.cpu().numpy()
        last = torch.stack([par, tok], dim=-1).cpu().numpy()
        for i in range(B):
            g = None if lists[i] is None else O.Graph(lists[i], V, case_class=cc, lam=lam)
            ref = O.beam_decode(g, xs[i], K, merge=merge, prune_delta=-1.0 if delta is None else delta)
            fin = np.isfinite(ref["scores"])
            what = (seed, i, dict(V=V, T=T, E=E, K=K, f32=f32, merge=merge, delta=delta))
            assert np.array_equal(stt[i], ref["states"]) and np.array_equal(lens[i], ref["lens"]), what
            assert np.array_equal(last[i], ref["tree"][-1]), what
            assert np.array_equal(np.isfinite(sc[i]), fin) and np.all(np.abs(sc[i][fin] - ref["scores"][fin]) <= SCORE_TOL), what
            for k in range(K):
                assert np.array_equal(toks[i, k, :ref["lens"][k]], ref["tokens"][k]), what
        batch.destroy()
