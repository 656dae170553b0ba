"""GPU parity of decoding with variative, case-insensitive graphs (Sec. 2.1 para. 4-7, Eq. 1): the graphs come
from tb_graph_compile_variative, the expected results from the oracle's own variative compile and decoders, on
the same seeded inputs (a synthetic piece vocabulary, phrases as text, logits with phrases planted in random
casings and segmentations)."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from oracle import variative as var
from paper_2608_21343_b200 import workloads as W
from helpers import SCORE_TOL, check_greedy, to_device, to_host
from test_gpu_beam_stream import run_beam

pytestmark = pytest.mark.gpu


def make_variative_batch(tb, pieces, lists, tau, lam=1.0, **kw):
    cc, _ = tb.tb_piece_classes(pieces)
    graphs = [None if p is None else tb.tb_graph_compile_variative(p, pieces, tau=tau, lam=lam) for p in lists]
    total = sum(512 * (g.view()["n_states"] + g.view()["n_arcs"]) + 8192 for g in graphs if g is not None)
    batch = tb.tb_batch_create(len(pieces), cc, len(lists), arena_bytes=max(1 << 20, total), **kw)
    for i, g in enumerate(graphs):
        tb.tb_batch_bind_stream(batch, i, g)
    return batch


def oracle_graphs(pieces, lists, tau, lam=1.0):
    return [None if p is None else O.GraphFromArrays(var.build(p, pieces, tau=tau, lam=lam)) for p in lists]


@pytest.mark.parametrize("seed,tau,general", [(0, 1.0, False), (1, 0.0, False), (2, 2.5, False), (3, 0.5, True)])
def test_greedy_decode_with_variative_graphs(tb, seed, tau, general):
    # 1031 pieces (every letter in both cases + merged pieces with some case variants), 100 phrases per stream,
    # streams long enough for the two-segment decode; one stream unbound
    pieces = W.make_piece_vocab(seed, letters=26, merged=560, max_len=5)
    B, T, S = 6, 300, 3
    lists = [W.draw_string_phrases(100 * seed + b, pieces, 100, 1, 4) for b in range(B)]
    lists[4] = None
    x = np.stack([W.variative_stream_logits(seed, b, pieces, lists[b] or lists[0], T, S) for b in range(B)])
    batch = make_variative_batch(tb, pieces, lists, tau)
    if general:
        tb.tb_batch_set_flags(batch, tb.TB_FLAG_GENERAL_KERNELS)
    lengths = torch.tensor([T, T - 7, T, 131, T, 60], dtype=torch.int32, device="cuda:0")
    out = to_host(tb.tb_greedy_decode(batch, to_device(x), lengths=lengths))
    assert tb.tb_batch_status(batch) == 0
    boosted_differs = 0
    for b, g in enumerate(oracle_graphs(pieces, lists, tau)):
        L = int(lengths[b])
        ref = O.greedy_rnnt(g, x[b], L)
        check_greedy(out, b, ref, "variative")
        if g is not None:
            boosted_differs += len(ref["tokens"]) != len(O.greedy_rnnt(None, x[b], L)["tokens"])
    assert boosted_differs >= 3          # the lists change what is decoded


def test_greedy_decode_variative_fp32_small(tb):
    pieces = W.make_piece_vocab(9, letters=8, merged=40, max_len=3)
    B, T, S = 3, 50, 2
    lists = [W.draw_string_phrases(b, pieces, 15, 1, 3) for b in range(B)]
    x = np.stack([W.variative_stream_logits(9, b, pieces, lists[b], T, S, dtype="f32", n_plants=5) for b in range(B)])
    batch = make_variative_batch(tb, pieces, lists, tau=1.0, lam=0.5)
    out = to_host(tb.tb_greedy_decode(batch, to_device(x)))
    for b, g in enumerate(oracle_graphs(pieces, lists, 1.0, lam=0.5)):
        check_greedy(out, b, O.greedy_rnnt(g, x[b]), "variative f32")


def test_beam_decode_with_variative_graphs(tb):
    pieces = W.make_piece_vocab(4, letters=26, merged=560, max_len=5)
    B, T, E, K = 4, 40, 2, 4
    lists = [W.draw_string_phrases(40 + b, pieces, 100, 1, 4) for b in range(B)]
    lists[1] = None
    x = np.stack([W.variative_stream_logits(4, b, pieces, lists[b] or lists[0], T, E, n_plants=5) for b in range(B)])
    batch = make_variative_batch(tb, pieces, lists, tau=1.0, max_beam=K, max_tree_steps=T * E)
    out = run_beam(tb, None, dict(logits=x, phrases=lists), K, lists, batch=batch)
    for i, g in enumerate(oracle_graphs(pieces, lists, 1.0)):
        ref = O.beam_decode(g, x[i], K)
        assert np.array_equal(out["tree"][i], ref["tree"]), f"stream {i}: (parent, token) tree"
        assert np.array_equal(out["states"][i], ref["states"]), f"stream {i}: states"
        assert np.array_equal(out["lens"][i], ref["lens"])
        for k in range(K):
            assert np.array_equal(out["tokens"][i, k, :ref["lens"][k]], ref["tokens"][k])
        fin = np.isfinite(ref["scores"])
        assert np.all(np.abs(out["scores"][i][fin] - ref["scores"][fin]) <= SCORE_TOL)


@pytest.mark.parametrize("n_phrases,letters,merged", [(400, 26, 560), (30, 8, 40), (200, 12, 300)])
def test_greedy_decode_variative_list_sizes(tb, n_phrases, letters, merged):
    # from lists whose resolved per-state lists fit the kernel's shared-memory cache with room to spare, over
    # ones that take most of it (shorter ring), to lists read from the arena
    pieces = W.make_piece_vocab(21, letters=letters, merged=merged, max_len=4)
    B, T, S = 4, 260, 3
    lists = [W.draw_string_phrases(700 + b, pieces, n_phrases, 1, 5) for b in range(B)]
    x = np.stack([W.variative_stream_logits(21, b, pieces, lists[b], T, S, n_plants=15) for b in range(B)])
    batch = make_variative_batch(tb, pieces, lists, tau=1.5)
    out = to_host(tb.tb_greedy_decode(batch, to_device(x)))
    assert tb.tb_batch_status(batch) == 0
    for b, g in enumerate(oracle_graphs(pieces, lists, 1.5)):
        check_greedy(out, b, O.greedy_rnnt(g, x[b]), f"variative {n_phrases} phrases")


def test_variative_full_size_sampled_streams(tb):
    # the configuration bench.py --workload 6 times (128 streams of 750 frames, lists cached in shared memory with
    # the short ring), checked on sampled streams
    B, T, S = 128, 750, 3
    pieces = W.make_piece_vocab(6, letters=26, merged=560, max_len=5)
    lists = [W.draw_string_phrases(6000 + b, pieces, 100, 1, 4) for b in range(B)]
    x = np.stack([W.variative_stream_logits(6, b, pieces, lists[b], T, S) for b in range(B)])
    batch = make_variative_batch(tb, pieces, lists, tau=1.0)
    out = to_host(tb.tb_greedy_decode(batch, to_device(x)))
    assert tb.tb_batch_status(batch) == 0
    for b in (0, 41, 94, 127):
        g = O.GraphFromArrays(var.build(lists[b], pieces, tau=1.0))
        check_greedy(out, b, O.greedy_rnnt(g, x[b]), "variative full size")
