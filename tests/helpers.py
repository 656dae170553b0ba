"""Shared helpers of the GPU parity tests: run one workload through the C-ABI library and
through the oracle on the same seeded inputs."""
import numpy as np
import torch

from oracle import oracle as O

SCORE_TOL = 1e-4   # absolute, float32 scores (the tolerance the benchmark spec states for scores)


def to_device(logits_np: np.ndarray, device="cuda:0") -> torch.Tensor:
    t = torch.from_numpy(logits_np)
    if logits_np.dtype == np.uint16:
        t = t.view(torch.bfloat16)
    return t.to(device)


def make_batch(tb, w, phrase_lists, n_slots=None, weights=None, lam=None, arena_bytes=None, **kw):
    """Compile one graph per stream and bind graph i to slot i (None = leave unbound)."""
    n_slots = len(phrase_lists) if n_slots is None else n_slots
    graphs = []
    total = 0
    for i, p in enumerate(phrase_lists):
        if p is None:
            graphs.append(None)
            continue
        g = tb.tb_graph_compile(p, w.V, case_class=w.vocab.case_class,
                                token_weights=None if weights is None else weights[i],
                                lam=w.lam if lam is None else lam)
        graphs.append(g)
        v = g.view()
        total += 512 * (v["n_states"] + v["n_arcs"]) + 8192
    batch = tb.tb_batch_create(w.V, w.vocab.case_class, n_slots, arena_bytes=arena_bytes or max(1 << 20, total), **kw)
    for i, g in enumerate(graphs):
        tb.tb_batch_bind_stream(batch, i, g)
    return batch, graphs


def oracle_graph(w, phrases, weights=None, lam=None):
    if phrases is None:
        return None
    return O.Graph(phrases, w.V, case_class=w.vocab.case_class, weights=weights, lam=w.lam if lam is None else lam)


def check_greedy(out, i, ref, what=""):
    n = int(out["counts"][i])
    assert n == len(ref["tokens"]), f"{what} stream {i}: count {n} vs {len(ref['tokens'])}"
    assert np.array_equal(out["tokens"][i, :n], ref["tokens"]), f"{what} stream {i}: tokens"
    assert np.array_equal(out["frames"][i, :n], ref["frames"]), f"{what} stream {i}: frames"
    assert int(out["states"][i]) == ref["state"], f"{what} stream {i}: state"
    assert abs(float(out["scores"][i]) - float(ref["score"])) <= SCORE_TOL, f"{what} stream {i}: score"


def to_host(out: dict) -> dict:
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}
