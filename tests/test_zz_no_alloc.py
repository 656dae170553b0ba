"""The no-allocation entry point against the ordinary one.

tb_greedy_decode_noalloc exists for callers that are not allowed to allocate device memory when they
decode (a server that divided its memory budget up front, or a thread that cannot take the device-wide
synchronisation of cudaMalloc): it keeps the kernel's working memory in a fixed array inside the library and
decodes every stream as unbound.  Its results must equal those of tb_greedy_decode on a batch whose slots
are all unbound, and those of the CPU oracle decoding without a graph -- tokens, frames, counts and states
exactly, scores within the tolerance of the other parity tests -- on two calls in a row (the second call meets
the array as the first one left it).

This file is collected last on purpose: if it fails, a run that stops at the first failure has already run
every other test.  It passes alone in a fresh process as well as after the others.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2608_21343_b200 import workloads as W
from helpers import SCORE_TOL, check_greedy, to_device

pytestmark = pytest.mark.gpu


def _out(B, T, S, dev):
    return dict(tokens=torch.full((B, T * S), -7, dtype=torch.int32, device=dev),
                frames=torch.full((B, T * S), -7, dtype=torch.int32, device=dev),
                counts=torch.full((B,), -7, dtype=torch.int32, device=dev),
                scores=torch.full((B,), float("nan"), dtype=torch.float32, device=dev),
                states=torch.full((B,), -7, dtype=torch.int32, device=dev),
                status=torch.full((1,), -7, dtype=torch.int32, device=dev))


def _same(a, b):
    torch.cuda.synchronize()
    n = a["counts"].cpu().numpy()
    assert np.array_equal(n, b["counts"].cpu().numpy())
    assert np.array_equal(a["states"].cpu().numpy(), b["states"].cpu().numpy())
    ta, tb_, fa, fb = (x.cpu().numpy() for x in (a["tokens"], b["tokens"], a["frames"], b["frames"]))
    for i in range(len(n)):
        assert np.array_equal(ta[i, :n[i]], tb_[i, :n[i]]) and np.array_equal(fa[i, :n[i]], fb[i, :n[i]])
    assert np.all(np.abs(a["scores"].cpu().numpy() - b["scores"].cpu().numpy()) <= SCORE_TOL)


def test_noalloc_matches_unbound_decode_twice(tb):
    dev = torch.device("cuda:0")
    cases = [W.get_workload(2, B=6, T=90, n_plants=4), W.get_workload(1, B=3, T=40)]   # bf16, then fp32
    for w in cases:
        data = W.batch_inputs(w)
        logits = to_device(data["logits"])
        batch = tb.tb_batch_create(w.V, w.vocab.case_class, w.B, arena_bytes=1 << 16)    # every slot unbound
        ref = tb.tb_greedy_decode(batch, logits)
        for call in range(2):
            # the second call runs on the other stream half so that the array's old contents differ
            lg = logits if call == 0 else logits.flip(0).contiguous()
            rf = ref if call == 0 else tb.tb_greedy_decode(batch, lg)
            out = tb.tb_greedy_decode_noalloc(lg, _out(w.B, w.T, w.S, dev))
            _same(out, rf)
            assert int(out["status"].item()) == 0 and (out["states"] == -1).all()
            # and against the oracle, stream by stream (no graph: the unboosted decode)
            host = {k: v.cpu().numpy() for k, v in out.items()}
            lg_host = data["logits"] if call == 0 else data["logits"][::-1]
            for i in range(w.B):
                check_greedy(host, i, O.greedy_rnnt(None, np.ascontiguousarray(lg_host[i])), "noalloc")
    # a length vector and a strided view, still without a batch
    w = cases[0]
    data = W.batch_inputs(w)
    big = torch.zeros((w.B, w.T, w.S, w.V + 9), dtype=torch.bfloat16, device=dev)
    big[..., 3:w.V + 4] = to_device(data["logits"])
    view = big[..., 3:w.V + 4]
    lengths = torch.tensor([90, 0, 17, 1, 89, 45], dtype=torch.int32, device=dev)
    batch = tb.tb_batch_create(w.V, w.vocab.case_class, w.B, arena_bytes=1 << 16)
    out = tb.tb_greedy_decode_noalloc(view, _out(w.B, w.T, w.S, dev), lengths=lengths)
    _same(out, tb.tb_greedy_decode(batch, view, lengths=lengths))
    host = {k: v.cpu().numpy() for k, v in out.items()}
    for i in range(w.B):
        check_greedy(host, i, O.greedy_rnnt(None, data["logits"][i], int(lengths[i])), "noalloc-lengths")


def test_noalloc_rejects_sizes_beyond_its_array(tb):
    dev = torch.device("cuda:0")
    B = tb.TB_NOALLOC_MAX_STREAMS + 1
    logits = torch.zeros((B, 1, 1, 9), dtype=torch.float32, device=dev)
    with pytest.raises(tb.TbError) as e:
        tb.tb_greedy_decode_noalloc(logits, _out(B, 1, 1, dev))
    assert e.value.code == tb.TB_ERR_INVALID_ARG
