"""GPU parity for streaming beam decoding (tb_beam_reset_slots / tb_beam_chunk / tb_beam_backtrace_slots /
tb_apply_final_weights_slots) against the CPU oracle: streams of different lengths come and go on their slots
(Sec. 2.2 para. 4), every slot keeps its hypotheses -- tree, scores, graph states -- from chunk to chunk (Sec. 2.3),
equal transcripts are merged and the beam is pruned at frame starts, and a finished stream is charged its final
weights.  The oracle decodes each stream on its own, whole, with the same options."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2608_21343_b200 import workloads as W
from helpers import SCORE_TOL, oracle_graph, to_device

pytestmark = pytest.mark.gpu


def run_streaming_beam(tb, w, K, n_chunks, merge, prune_delta, check_partial=False, max_beam=None):
    """Chunks of w.chunk frames over w.B slots with stream churn; returns the number of streams checked."""
    E = w.S
    sched = W.ChurnSchedule(w)
    batch = tb.tb_batch_create(w.V, w.vocab.case_class, w.B, max_beam=max_beam or K, max_tree_steps=w.T * E, arena_bytes=32 << 20)
    if prune_delta is not None:
        tb.tb_batch_set_beam_prune(batch, prune_delta)
    dev = torch.device("cuda:0")
    scores = torch.full((w.B, K), float("-inf"), device=dev)
    states = torch.full((w.B, K), -1, dtype=torch.int32, device=dev)
    live = torch.zeros((w.B, K), dtype=torch.uint8, device=dev)
    par = torch.empty((w.B, K), dtype=torch.int32, device=dev)
    tok = torch.empty((w.B, K), dtype=torch.int32, device=dev)
    tb.tb_beam_reset_slots(batch)                        # a new session: every slot at the start of an utterance
    slot = [None] * w.B
    served = np.zeros(w.B, dtype=np.int64)
    checked = 0
    for c in range(n_chunks):
        chunk, lengths, binds = sched.next_chunk()
        new = []
        for s, _sid, phrases in binds:
            g = tb.tb_graph_compile(phrases, w.V, case_class=w.vocab.case_class)
            tb.tb_batch_bind_stream(batch, s, g)
            slot[s] = dict(phrases=phrases, logits=sched.data[s]["logits"], length=int(sched.data[s]["length"]))
            served[s] = 0
            new.append(s)
        if new and c % 2 == 0:
            # the caller sets up the new slots' rows itself ...
            idx = torch.tensor(new, device=dev)
            scores[idx] = float("-inf")
            scores[idx, 0] = 0.0
            states[idx] = -1
            states[idx, 0] = 0
            live[idx] = 0
            tb.tb_beam_reset_slots(batch, new)
        elif new:
            # ... or lets the library do it in the same launch (garbage first, to see that every entry is written)
            idx = torch.tensor(new, device=dev)
            scores[idx] = 123.0
            states[idx] = 7
            live[idx] = 1
            tb.tb_beam_start_slots(batch, new, scores, states, live)
        left = np.clip(np.array([slot[s]["length"] for s in range(w.B)]) - served, 0, w.chunk).astype(np.int32)
        tb.tb_beam_chunk(batch, to_device(chunk), merge, torch.from_numpy(left).to(dev), scores, states, live, par, tok)
        served += left
        ended = [s for s in range(w.B) if left[s] > 0 and served[s] >= slot[s]["length"]]
        if check_partial and c % 3 == 1:
            # the running result of a stream in mid-utterance: the oracle on the frames decoded so far
            s = int(np.argmax(served * (served < np.array([slot[i]["length"] for i in range(w.B)]))))
            toks, lens = tb.tb_beam_backtrace_slots(batch, w.B, K, w.T * E)
            ref = O.beam_decode(oracle_graph(w, slot[s]["phrases"]), slot[s]["logits"][:served[s]], K, merge=merge,
                                prune_delta=-1.0 if prune_delta is None else prune_delta)
            assert np.array_equal(lens[s].cpu().numpy(), ref["lens"]), (c, s)
            assert np.array_equal(states[s].cpu().numpy(), ref["states"]), (c, s)
        if ended:
            tb.tb_apply_final_weights_slots(batch, ended, scores, states)
            toks, lens = tb.tb_beam_backtrace_slots(batch, w.B, K, w.T * E)
            some_t, some_l = tb.tb_beam_backtrace_slot_list(batch, ended, K, w.T * E)      # ... and of the ended slots only
            torch.cuda.synchronize()
            h_tok, h_len, h_sc, h_st = toks.cpu().numpy(), lens.cpu().numpy(), scores.cpu().numpy(), states.cpu().numpy()
            for i, s in enumerate(ended):
                assert np.array_equal(some_l[i].cpu().numpy(), h_len[s]) and np.array_equal(some_t[i].cpu().numpy(), h_tok[s]), (c, s)
            for s in ended:
                g = oracle_graph(w, slot[s]["phrases"])
                ref = O.beam_decode(g, slot[s]["logits"][:slot[s]["length"]], K, merge=merge,
                                    prune_delta=-1.0 if prune_delta is None else prune_delta)
                assert np.array_equal(h_len[s], ref["lens"]), (c, s, "lengths")
                assert np.array_equal(h_st[s], ref["states"]), (c, s, "states")
                for k in range(K):
                    assert np.array_equal(h_tok[s, k, :ref["lens"][k]], ref["tokens"][k]), (c, s, k)
                    if np.isfinite(ref["scores"][k]):
                        want = O.apply_final_weight(g, int(ref["states"][k]), ref["scores"][k])
                        assert abs(float(h_sc[s, k]) - float(want)) <= SCORE_TOL, (c, s, k, "score")
                    else:
                        assert not np.isfinite(h_sc[s, k])
                checked += 1
    assert tb.tb_batch_status(batch) == 0
    return checked


@pytest.mark.parametrize("K,merge,prune", [(4, True, 8.0), (32, True, 8.0), (4, False, None), (32, False, 2.0)])
def test_streaming_beam_with_churn(tb, K, merge, prune):
    """The streaming workload's shape in small: 10 slots, chunks of 8 frames, 2 expansions per frame, streams of
    20-70 frames that end in the middle of chunks, lists of 10-60 phrases compiled and bound as streams arrive."""
    w = W.get_workload(5, B=10, T=70, T_lo=20, S=2, n_dur=0, n_phrases=60, n_phrases_lo=10)
    n = run_streaming_beam(tb, w, K, n_chunks=24, merge=merge, prune_delta=prune, check_partial=True)
    assert n >= 2 * w.B                                     # every slot saw several streams


def test_streaming_beam_narrower_than_the_batch_allows(tb):
    """A session may use a beam narrower than the batch was created for: the per-slot records (tree ring, sequence
    hashes and lengths) are then laid out at the session's width, also when single slots restart."""
    w = W.get_workload(5, B=6, T=50, T_lo=15, S=2, n_dur=0, n_phrases=40, n_phrases_lo=10)
    n = run_streaming_beam(tb, w, 3, n_chunks=20, merge=True, prune_delta=6.0, check_partial=True, max_beam=8)
    assert n >= w.B


def test_streaming_beam_refuses_to_mix_with_the_batch_wide_tree(tb):
    w = W.get_workload(5, B=3, T=16, T_lo=16, S=2, n_dur=0, n_phrases=10, n_phrases_lo=10)
    batch = tb.tb_batch_create(w.V, w.vocab.case_class, w.B, max_beam=4, max_tree_steps=64, arena_bytes=1 << 20)
    dev = torch.device("cuda:0")
    logits = torch.zeros((w.B, 8, 2, w.V + 1), dtype=torch.bfloat16, device=dev)
    scores = torch.zeros((w.B, 4), device=dev)
    states = torch.full((w.B, 4), -1, dtype=torch.int32, device=dev)
    live = torch.zeros((w.B, 4), dtype=torch.uint8, device=dev)
    par = torch.empty((w.B, 4), dtype=torch.int32, device=dev)
    tok = torch.empty((w.B, 4), dtype=torch.int32, device=dev)
    tb.tb_beam_reset_slots(batch)
    tb.tb_beam_chunk(batch, logits, False, None, scores, states, live, par, tok)
    with pytest.raises(tb.TbError):                        # a batch-wide step in the middle of a streaming session
        tb.tb_beam_frames(batch, logits, False, scores, states, live, par, tok)
    with pytest.raises(tb.TbError):                        # another beam width in the same session
        tb.tb_beam_chunk(batch, logits, False, None, scores[:, :2].contiguous(), states[:, :2].contiguous(),
                         live[:, :2].contiguous(), par[:, :2].contiguous(), tok[:, :2].contiguous())
    with pytest.raises(tb.TbError):
        tb.tb_beam_reset_slots(batch, [w.B])
    tb.tb_beam_reset(batch)                                # ends the session
    tb.tb_beam_frames(batch, logits, False, scores, states, live, par, tok)
    with pytest.raises(tb.TbError):                        # and the other way round
        tb.tb_beam_chunk(batch, logits, False, None, scores, states, live, par, tok)
    torch.cuda.synchronize()


def test_an_utterance_longer_than_the_tree_ring_is_reported(tb):
    """A slot's hypothesis tree is a ring of max_tree_steps steps.  An utterance that outgrows it keeps decoding
    correctly (scores, states); its backtrace raises TB_STATUS_STEP_LIMIT and yields the tokens still in the ring: the
    tail of each transcript."""
    w = W.get_workload(5, B=2, T=24, T_lo=24, S=2, n_dur=0, n_phrases=30, n_phrases_lo=30)
    K, E, cap = 4, 2, 12
    dev = torch.device("cuda:0")
    batch = tb.tb_batch_create(w.V, w.vocab.case_class, w.B, max_beam=K, max_tree_steps=cap, arena_bytes=4 << 20)
    data = [W.stream_inputs(w, i) for i in range(w.B)]
    for i, d in enumerate(data):
        tb.tb_batch_bind_stream(batch, i, tb.tb_graph_compile(d["phrases"], w.V, case_class=w.vocab.case_class))
    scores = torch.empty((w.B, K), device=dev)
    states = torch.empty((w.B, K), dtype=torch.int32, device=dev)
    live = torch.empty((w.B, K), dtype=torch.uint8, device=dev)
    par = torch.empty((w.B, K), dtype=torch.int32, device=dev)
    tok = torch.empty((w.B, K), dtype=torch.int32, device=dev)
    tb.tb_beam_start_slots(batch, None, scores, states, live)
    x = np.stack([d["logits"][:24] for d in data])                      # [2, 24, E, V + 1]
    for c in range(3):                                                  # three chunks of 8 frames = 48 steps per slot
        tb.tb_beam_chunk(batch, to_device(np.ascontiguousarray(x[:, 8 * c:8 * c + 8])), False, None, scores, states, live, par, tok)
    toks, lens = tb.tb_beam_backtrace_slots(batch, w.B, K, 64)
    torch.cuda.synchronize()
    status = tb.tb_batch_status(batch)
    assert status & tb.TB_STATUS_STEP_LIMIT, status
    toks, lens = toks.cpu().numpy(), lens.cpu().numpy()
    for i in range(w.B):
        ref = O.beam_decode(oracle_graph(w, data[i]["phrases"]), x[i], K, merge=False, prune_delta=-1.0)
        assert np.array_equal(states[i].cpu().numpy(), ref["states"])
        assert np.allclose(scores[i].cpu().numpy(), ref["scores"], atol=SCORE_TOL)
        for k in range(K):
            n = int(lens[i, k])
            assert n <= ref["lens"][k]
            assert np.array_equal(toks[i, k, :n], ref["tokens"][k][ref["lens"][k] - n:ref["lens"][k]]), (i, k)
        assert lens[i].max() <= cap
