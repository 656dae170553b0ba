"""GPU parity at the full size of all five workloads, every stream checked against the CPU oracle.

The other GPU test files hold the reduced and the edge cases; this one runs each workload in the shape and launch
configuration the benchmark times and compares every stream (every slot and every chunk for the streaming workload)
with the oracle: tokens, frames, durations, parents and graph states bit-exact, scores within 1e-4 absolute.  The
oracle decodes one stream per call; the calls are spread over a thread pool (the C code runs without the
interpreter lock)."""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2608_21343_b200 import workloads as W
from helpers import SCORE_TOL, check_greedy, make_batch, oracle_graph, to_device, to_host
from test_gpu_beam_stream import run_beam, run_beam_frames

pytestmark = pytest.mark.gpu

WORKERS = max(2, min(16, os.cpu_count() or 2))


def pool_map(fn, items):
    with ThreadPoolExecutor(max_workers=WORKERS) as ex:
        return list(ex.map(fn, items))


def batch_inputs_parallel(w):
    """W.batch_inputs with the streams generated on several threads (same bits: one generator per stream)."""
    parts = pool_map(lambda b: W.stream_inputs(w, b), range(w.B))
    logits = np.stack([d["logits"] for d in parts])
    return dict(logits=logits, phrases=[d["phrases"] for d in parts], streams=list(range(w.B)))


def oracle_greedy_all(w, data, lists):
    return pool_map(lambda i: O.greedy_rnnt(oracle_graph(w, lists[i]), data["logits"][i]), range(len(lists)))


def test_workload2_full_size_every_stream(tb):
    w = W.get_workload(2)
    data = batch_inputs_parallel(w)
    batch, _ = make_batch(tb, w, data["phrases"])
    logits = to_device(data["logits"])
    out = to_host(tb.tb_greedy_decode(batch, logits))
    assert tb.tb_batch_status(batch) == 0
    # the configuration the benchmark times must run on a pipelined kernel: a silent fall-back to the general one
    # would keep every comparison below green and cost an order of magnitude
    assert tb.tb_batch_last_greedy_kernel(batch)["kernel"] in (tb.TB_KERNEL_PIPELINED, tb.TB_KERNEL_SEGMENTED)
    refs = oracle_greedy_all(w, data, data["phrases"])
    for i, ref in enumerate(refs):
        check_greedy(out, i, ref, "w2")
    # the same batch through the segmented kernel (two blocks per stream, as many as fit a B200 at 128 streams)
    tb.tb_batch_set_greedy_plan(batch, 2, 8, 2)
    out = to_host(tb.tb_greedy_decode(batch, logits))
    assert tb.tb_batch_last_greedy_kernel(batch)["kernel"] == tb.TB_KERNEL_SEGMENTED
    for i, ref in enumerate(refs):
        check_greedy(out, i, ref, "w2 segmented")
    tb.tb_batch_set_greedy_plan(batch, 0, 0, 0)
    # the unboosted decode of the same tensor (what the benchmark's overhead figure is measured against)
    for i in range(w.B):
        tb.tb_batch_bind_stream(batch, i, None)
    out0 = to_host(tb.tb_greedy_decode(batch, logits))
    assert tb.tb_batch_status(batch) == 0
    for i, ref in enumerate(oracle_greedy_all(w, data, [None] * w.B)):
        check_greedy(out0, i, ref, "w2-unboosted")
    assert (out0["states"] == -1).all()


def test_workload3_full_size_every_stream(tb):
    """64 streams, each with its own graph of about 24.7 k states (1000 own + 4000 shared phrases) in the arena."""
    w = W.get_workload(3)
    data = batch_inputs_parallel(w)
    batch, graphs = make_batch(tb, w, data["phrases"])
    n_states = [g.view()["n_states"] for g in graphs]
    assert min(n_states) > 20000
    out = to_host(tb.tb_greedy_decode(batch, to_device(data["logits"])))
    assert tb.tb_batch_status(batch) == 0
    for i, ref in enumerate(oracle_greedy_all(w, data, data["phrases"])):
        check_greedy(out, i, ref, "w3")


def _check_beam_stream(out, i, ref, K, tree=True):
    if tree:
        assert np.array_equal(out["tree"][i], ref["tree"]), f"stream {i}: (parent, token) tree"
    else:
        assert np.array_equal(out["last"][i], ref["tree"][-1]), f"stream {i}: last (parent, token) step"
    assert np.array_equal(out["states"][i], ref["states"]), f"stream {i}: states"
    assert np.array_equal(out["lens"][i], ref["lens"]), f"stream {i}: lengths"
    for k in range(K):
        assert np.array_equal(out["tokens"][i, k, :ref["lens"][k]], ref["tokens"][k]), f"stream {i} hyp {k}"
    fin = np.isfinite(ref["scores"])
    assert np.array_equal(np.isfinite(out["scores"][i]), fin)
    assert np.all(np.abs(out["scores"][i][fin] - ref["scores"][fin]) <= SCORE_TOL), f"stream {i}: scores"


def test_workload4_full_size_every_stream_both_entry_points(tb):
    w = W.get_workload(4)
    data = batch_inputs_parallel(w)
    refs = pool_map(lambda i: O.beam_decode(oracle_graph(w, data["phrases"][i]), data["logits"][i], w.K), range(w.B))
    out = run_beam(tb, w, data, w.K)                                  # tb_beam_step, one expansion per call
    for i in range(w.B):
        _check_beam_stream(out, i, refs[i], w.K)
    batch, _ = make_batch(tb, w, data["phrases"], max_beam=w.K, max_tree_steps=w.T * w.S)
    fr = run_beam_frames(tb, w, data, w.K, data["phrases"], batch)     # tb_beam_frames, the utterance in one launch
    for i in range(w.B):
        _check_beam_stream(fr, i, refs[i], w.K, tree=False)


def test_workload5_full_size_with_churn(tb):
    """512 slots, chunks of 8 frames, TDT with 5 duration logits, lists of 50-500 phrases, stream lengths
    200-1500 frames: 160 chunks, so that the shortest streams end and their slots are refilled (from chunk 25 on)
    while the others keep decoding.  Every slot is compared with the oracle after every chunk."""
    w = W.get_workload(5)
    n_chunks = 160
    sched = W.ChurnSchedule(w, workers=WORKERS)
    batch = tb.tb_batch_create(w.V, w.vocab.case_class, w.B, arena_bytes=256 << 20)   # the size the benchmark gives this workload
    slots = [None] * w.B
    t0 = np.zeros(w.B, dtype=np.int64)
    n_binds = n_refills = n_tokens = 0
    try:
        with ThreadPoolExecutor(max_workers=WORKERS) as ex:
            for c in range(n_chunks):
                chunk, lengths, binds = sched.next_chunk()
                graphs = list(ex.map(lambda b: tb.tb_graph_compile(b[2], w.V, case_class=w.vocab.case_class), binds))
                ographs = list(ex.map(lambda b: oracle_graph(w, b[2]), binds))
                for (slot, _sid, _phr), g, og in zip(binds, graphs, ographs):
                    if c % 2:
                        tb.tb_batch_bind_stream(batch, slot, g)
                    slots[slot] = dict(graph=og, st=O.StreamState(0, 0, 0, 0.0, 0))
                    t0[slot] = 0
                    n_binds += 1
                    n_refills += c > 0
                if c % 2:
                    out = to_host(tb.tb_stream_chunk(batch, to_device(chunk), w.n_dur, torch.from_numpy(lengths).to("cuda:0")))
                else:
                    # every other chunk brings its binds along (the first one all 512, ahead of the launch; refills of up
                    # to eight slots inside the launch)
                    out = to_host(tb.tb_stream_chunk_binds(batch, [bd[0] for bd in binds], graphs, to_device(chunk), w.n_dur,
                                                           torch.from_numpy(lengths).to("cuda:0")))

                def one(i):
                    sl = slots[i]
                    return O.stream_chunk(sl["graph"], chunk[i], w.n_dur, int(t0[i]), int(lengths[i]), sl["st"])

                refs = list(ex.map(one, range(w.B)))
                for i, ref in enumerate(refs):
                    n = int(out["counts"][i])
                    assert n == len(ref["tokens"]), (c, i)
                    assert np.array_equal(out["tokens"][i, :n], ref["tokens"]), (c, i)
                    assert np.array_equal(out["frames"][i, :n], ref["frames"]), (c, i)
                    assert np.array_equal(out["durs"][i, :n], ref["durs"]), (c, i)
                    st = slots[i]["st"]
                    assert out["states"][i] == st.state and out["cursors"][i] == st.t, (c, i)
                    assert abs(float(out["scores"][i]) - float(st.score)) <= SCORE_TOL, (c, i)
                    n_tokens += n
                t0 += w.chunk
    finally:
        sched.close()
    assert tb.tb_batch_status(batch) == 0
    assert n_binds == w.B + n_refills and n_refills > 300 and n_tokens > 100000
    counts = tb.tb_batch_bind_counts(batch)
    assert counts["pulled"] > 100 and counts["copied"] >= w.B      # both ways of tb_stream_chunk_binds were taken


def _coarse(x):
    """Logits on a grid of 0.5: exact ties between tokens, and between hypotheses, at almost every step."""
    return (np.round(x * 2) / 2).astype(x.dtype)


@pytest.mark.parametrize("K,merge", [(4, False), (4, True), (32, False), (32, True)])
def test_beam_on_coarse_grid_logits_ties_between_parents(tb, K, merge):
    """With rows shared by the hypotheses of a stream and logits on a coarse grid, candidates from different
    parents tie in score and token all the time: the order (score, token id, parent) decides the tree."""
    w = W.get_workload(4, B=4, T=40, V=64, n_phrases=12, n_plants=4)
    data = W.batch_inputs(w)
    data["logits"] = W.to_storage(_coarse(W.bf16_bits_to_f32(data["logits"])), w.dtype)
    lists = [data["phrases"][0], None, data["phrases"][2], []]
    out = run_beam(tb, w, data, K, lists, merge=merge)
    refs = [O.beam_decode(oracle_graph(w, lists[i]), data["logits"][i], K, merge=merge) for i in range(w.B)]
    for i in range(w.B):
        _check_beam_stream(out, i, refs[i], K)
    # how often the last clause of the order decides: drive the oracle's step by hand (no merging) on two streams and
    # count the steps whose new beam holds two places equal in score and token
    ties = 0
    for i in (0, 1):
        g = oracle_graph(w, lists[i])
        sc = np.full(K, -np.inf, dtype=np.float32); sc[0] = 0.0
        st = np.full(K, -1, dtype=np.int32); st[0] = 0 if g is not None else -1
        lv = np.zeros(K, dtype=np.uint8)
        for t in range(w.T):
            lv[:] = np.isfinite(sc)
            for e in range(w.S):
                rows = np.broadcast_to(data["logits"][i, t, e], (K, w.V + 1)).copy()
                _par, tk = O.beam_step(g, rows, sc, st, lv)
                pairs = [(float(a), int(b)) for a, b in zip(sc, tk) if np.isfinite(a)]
                ties += len(set(pairs)) < len(pairs)
    assert ties > 20
    batch, _ = make_batch(tb, w, lists, max_beam=K, max_tree_steps=w.T * w.S)
    fr = run_beam_frames(tb, w, data, K, lists, batch, merge=merge, chunks=(8,) * 5)
    for i in range(w.B):
        _check_beam_stream(fr, i, refs[i], K, tree=False)


def test_beam_step_equal_candidates_go_to_the_lower_parent(tb):
    """The hand-worked step of the oracle's pin, on the GPU: hypotheses 0 and 2 are equal in score and state and
    read the same row; every pair of equal candidates comes out lower parent first."""
    w = W.get_workload(1, B=1, T=1)
    V = w.V
    batch, _ = make_batch(tb, w, [[[0]]], max_beam=4)
    dev = "cuda:0"
    row = torch.full((V + 1,), -9.0, device=dev)
    row[0], row[5], row[V] = 0.0, 0.5, 0.5            # values at the root: token 0 -> 1.0, token 5 -> 0.5, blank 0.5
    rows = row.repeat(1, 1).contiguous()
    scores = torch.tensor([[0.0, float("-inf"), 0.0, float("-inf")]], device=dev)
    states = torch.tensor([[0, -1, 0, -1]], dtype=torch.int32, device=dev)
    live = torch.tensor([[1, 0, 1, 0]], dtype=torch.uint8, device=dev)
    par = torch.empty((1, 4), dtype=torch.int32, device=dev)
    tok = torch.empty((1, 4), dtype=torch.int32, device=dev)
    tb.tb_beam_step(batch, rows, V + 1, 0, False, scores, states, live, par, tok)      # hyp stride 0: one shared row
    torch.cuda.synchronize()
    assert tok.tolist() == [[0, 0, 5, 5]] and par.tolist() == [[0, 2, 0, 2]]
    assert scores.tolist() == [[1.0, 1.0, 0.5, 0.5]] and states.tolist() == [[1, 1, 0, 0]]
    # the same inputs through the oracle
    rs = np.array([0.0, -np.inf, 0.0, -np.inf], dtype=np.float32)
    rst = np.array([0, -1, 0, -1], dtype=np.int32)
    rl = np.array([1, 0, 1, 0], dtype=np.uint8)
    rp, rt = O.beam_step(O.Graph([[0]], V, case_class=w.vocab.case_class),
                         np.broadcast_to(row.cpu().numpy(), (4, V + 1)).copy(), rs, rst, rl)
    assert rp.tolist() == [0, 2, 0, 2] and rt.tolist() == [0, 0, 5, 5]
