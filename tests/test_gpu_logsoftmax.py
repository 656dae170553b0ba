"""GPU parity of the fused log-softmax selection (TB_FLAG_LOG_SOFTMAX) against the oracle's normalised decode.

The oracle normalises in double, the kernel in float, so the two may choose differently where two candidates are
closer than the float roundings involved.  The comparison therefore lets the oracle follow the kernel's choice
where -- and only where -- the kernel's candidate is within EPS of the oracle's best, counts those places, and
treats any larger difference as an error; scores are compared within a bound derived from the float arithmetic.

EPS: a candidate's value is fl(fl(x - L) + lb); the error of L is common to all candidates of a row and does not
change their order, the two roundings are at most half an ulp of a value below 16 each, i.e. 2 * 2^-21 together per
candidate and twice that between two candidates: 4e-6 covers it.
Score bound per visited row: |L_float - L_double| (float exp / sum / log of about a thousand terms: below 2e-6), the
two roundings above (1e-6), and half an ulp of the running score for the float accumulation."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2608_21343_b200 import workloads as W
from helpers import make_batch, oracle_graph, to_device, to_host

pytestmark = pytest.mark.gpu

EPS = 4e-6


def compare(out, i, g, logits_i, length=None):
    n = int(out["counts"][i])
    ref = O.greedy_rnnt_lsm(g, logits_i, length, follow=(out["tokens"][i, :n], out["frames"][i, :n]), eps=EPS)
    assert ref["first_mismatch"] == -1, f"stream {i}: the kernel's choice at visited row {ref['first_mismatch']} is off by more than {EPS}"
    assert len(ref["tokens"]) == n and np.array_equal(ref["tokens"], out["tokens"][i, :n]), f"stream {i}: tokens"
    assert np.array_equal(ref["frames"], out["frames"][i, :n]), f"stream {i}: frames"
    assert int(out["states"][i]) == ref["state"], f"stream {i}: state"
    bound = ref["rows"] * (3e-6 + 0.5 * float(np.spacing(np.float32(max(1.0, abs(ref["score"]))))))
    assert abs(float(out["scores"][i]) - ref["score"]) <= bound, f"stream {i}: score {out['scores'][i]} vs {ref['score']} (bound {bound})"
    return ref["followed"], ref["rows"]


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_normalised_greedy_decode(tb, dtype):
    w = W.get_workload(2, B=10, T=200, dtype=dtype, n_phrases=60, n_plants=10)
    data = W.batch_inputs(w)
    lists = list(data["phrases"])
    lists[4] = None
    batch, _ = make_batch(tb, w, lists)
    tb.tb_batch_set_flags(batch, tb.TB_FLAG_LOG_SOFTMAX)
    lengths = [200, 199, 1, 0, 200, 150, 200, 200, 77, 200]
    out = to_host(tb.tb_greedy_decode(batch, to_device(data["logits"]), lengths=torch.tensor(lengths, dtype=torch.int32, device="cuda:0")))
    assert tb.tb_batch_status(batch) == 0
    # packed bf16 rows: a pipelined kernel (its helpers leave every row's normaliser, and the selection takes it off
    # the selected value; ten streams: the segmented one); anything else: the general kernel, which normalises every
    # entry before the bonus
    assert tb.tb_batch_last_greedy_kernel(batch)["kernel"] == (tb.TB_KERNEL_SEGMENTED if dtype == "bf16" else tb.TB_KERNEL_GENERAL)
    followed = rows = 0
    for i in range(w.B):
        f, r = compare(out, i, oracle_graph(w, lists[i]), data["logits"][i], lengths[i])
        followed += f
        rows += r
    assert followed <= 0.02 * rows                     # near-ties are the exception (they are counted, not ignored)
    if dtype == "bf16":
        # the same decode on the general kernel meets the same bar, and differs from the pipelined one by roundings only
        tb.tb_batch_set_flags(batch, tb.TB_FLAG_LOG_SOFTMAX | tb.TB_FLAG_GENERAL_KERNELS)
        gen = to_host(tb.tb_greedy_decode(batch, to_device(data["logits"]), lengths=torch.tensor(lengths, dtype=torch.int32, device="cuda:0")))
        assert tb.tb_batch_last_greedy_kernel(batch)["kernel"] == tb.TB_KERNEL_GENERAL
        for i in range(w.B):
            compare(gen, i, oracle_graph(w, lists[i]), data["logits"][i], lengths[i])
        assert np.allclose(gen["scores"], out["scores"], rtol=0, atol=2e-3)
    # in exact arithmetic the tokens are those of the un-normalised decode: on these inputs almost every stream agrees
    tb.tb_batch_set_flags(batch, 0)
    plain = to_host(tb.tb_greedy_decode(batch, to_device(data["logits"]), lengths=torch.tensor(lengths, dtype=torch.int32, device="cuda:0")))
    same = sum(int(plain["counts"][i]) == int(out["counts"][i]) and
               np.array_equal(plain["tokens"][i, :plain["counts"][i]], out["tokens"][i, :out["counts"][i]]) for i in range(w.B))
    assert same >= w.B - 3
    assert np.all(out["scores"][[0, 1, 4, 5]] < plain["scores"][[0, 1, 4, 5]])      # log-probabilities are negative


def test_normalised_streaming_chunks_equal_the_offline_decode(tb):
    w = W.get_workload(2, B=4, T=64, n_phrases=40, n_plants=5)
    data = W.batch_inputs(w)
    batch, _ = make_batch(tb, w, data["phrases"])
    # (streaming chunks run on the general kernel; so does the offline decode they are compared with bit for bit)
    tb.tb_batch_set_flags(batch, tb.TB_FLAG_LOG_SOFTMAX | tb.TB_FLAG_GENERAL_KERNELS)
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
        compare(off, i, oracle_graph(w, data["phrases"][i]), data["logits"][i])
    # duration logits have no normalisation defined here: refused
    tdt = torch.zeros((w.B, 8, w.S, w.V + 6), dtype=torch.bfloat16, device="cuda:0")
    with pytest.raises(tb.TbError):
        tb.tb_stream_chunk(batch, tdt, 5, valid)


@pytest.mark.parametrize("wl,B,T,one_block", [(2, 16, 750, False), (2, 16, 750, True), (2, 3, 100, False), (2, 3, 100, True),
                                               (3, 3, 300, True)])
def test_normalised_decode_on_the_pipelined_kernels(tb, wl, B, T, one_block):
    """The benchmark's workload (and a short case, and large lists that the decider walks in the arena) with rows
    normalised, on the segmented kernel and on the one-block-per-stream kernel with one and two segments: bound and
    unbound slots, ragged lengths; every stream against the oracle's normalised decode."""
    w = W.get_workload(wl, B=B, T=T)
    data = W.batch_inputs(w)
    lists = list(data["phrases"])
    lists[1] = None
    batch, _ = make_batch(tb, w, lists)
    base = tb.TB_FLAG_ONE_BLOCK_PER_STREAM if one_block else 0
    tb.tb_batch_set_flags(batch, base | tb.TB_FLAG_LOG_SOFTMAX)
    lengths = np.full(B, T, dtype=np.int32)
    lengths[2] = T - 37
    out = to_host(tb.tb_greedy_decode(batch, to_device(data["logits"]), lengths=torch.from_numpy(lengths).to("cuda:0")))
    assert tb.tb_batch_status(batch) == 0
    ran = tb.tb_batch_last_greedy_kernel(batch)["kernel"]
    assert ran == (tb.TB_KERNEL_PIPELINED if one_block else tb.TB_KERNEL_SEGMENTED)   # (large lists: always one block per stream)
    followed = rows = 0
    for i in range(B):
        f, r = compare(out, i, oracle_graph(w, lists[i]), data["logits"][i], int(lengths[i]))
        followed += f
        rows += r
    assert followed <= 0.02 * rows
    # the tokens are those of the un-normalised decode (the normaliser is taken off after the selection)
    tb.tb_batch_set_flags(batch, base)
    plain = to_host(tb.tb_greedy_decode(batch, to_device(data["logits"]), lengths=torch.from_numpy(lengths).to("cuda:0")))
    assert tb.tb_batch_last_greedy_kernel(batch)["kernel"] == ran
    assert np.array_equal(plain["counts"], out["counts"]) and np.array_equal(plain["states"], out["states"])
    for i in range(B):
        assert np.array_equal(plain["tokens"][i, :plain["counts"][i]], out["tokens"][i, :out["counts"][i]])
