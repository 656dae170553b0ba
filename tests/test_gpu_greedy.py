"""GPU parity, greedy RNNT (tb_greedy_decode) against the CPU oracle on the same seeded inputs:
tokens, frames and graph states bit-exact, scores within 1e-4 absolute."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2608_21343_b200 import workloads as W
from helpers import SCORE_TOL, check_greedy, make_batch, oracle_graph, to_device, to_host

pytestmark = pytest.mark.gpu


def run_and_compare(tb, w, data, lengths=None, phrase_lists=None, weights=None, lam=None, what=""):
    phrase_lists = data["phrases"] if phrase_lists is None else phrase_lists
    batch, _ = make_batch(tb, w, phrase_lists, weights=weights, lam=lam)
    logits = to_device(data["logits"])
    dl = None if lengths is None else torch.tensor(lengths, dtype=torch.int32, device="cuda:0")
    out = to_host(tb.tb_greedy_decode(batch, logits, lengths=dl))
    assert tb.tb_batch_status(batch) == 0
    for i, p in enumerate(phrase_lists):
        g = oracle_graph(w, p, None if weights is None else weights[i], lam)
        ref = O.greedy_rnnt(g, data["logits"][i], None if lengths is None else lengths[i])
        check_greedy(out, i, ref, what)
    return out, batch


def test_workload1_tiny_greedy_full(tb):
    w = W.get_workload(1)
    data = W.batch_inputs(w)
    out, _ = run_and_compare(tb, w, data, what="w1")
    assert out["counts"].min() > 5
    # per-stream independence (Sec. 2.2 para. 3): each stream alone gives the same result
    for i in range(w.B):
        batch1, _ = make_batch(tb, w, [data["phrases"][i]])
        solo = to_host(tb.tb_greedy_decode(batch1, to_device(data["logits"][i:i + 1])))
        n = int(out["counts"][i])
        assert int(solo["counts"][0]) == n
        assert np.array_equal(solo["tokens"][0, :n], out["tokens"][i, :n])
        assert np.array_equal(solo["frames"][0, :n], out["frames"][i, :n])
        assert solo["states"][0] == out["states"][i] and solo["scores"][0] == out["scores"][i]


def test_workload2_reduced_and_unbound_mix(tb):
    w = W.get_workload(2, B=12, T=160)
    data = W.batch_inputs(w)
    lists = list(data["phrases"])
    lists[3] = None            # model id -1
    lists[7] = []              # an empty list: root only
    out, _ = run_and_compare(tb, w, data, phrase_lists=lists, what="w2r")
    assert out["states"][3] == -1


def test_workload3_large_lists(tb):
    w = W.get_workload(3, B=3, T=300)
    data = W.batch_inputs(w)
    out, _ = run_and_compare(tb, w, data, what="w3")


@pytest.mark.parametrize("lam", [0.5, 2.0, 0.0])
def test_weighted_lists_and_lambda(tb, lam):
    w = W.get_workload(2, B=5, T=120, n_phrases=40)
    data = W.batch_inputs(w)
    rng = np.random.default_rng(1)
    weights = [[[float(rng.choice([0.5, 1.0, 1.5, 2.0])) for _ in p] for p in lst] for lst in data["phrases"]]
    run_and_compare(tb, w, data, weights=weights, lam=lam, what=f"lam{lam}")


def test_lengths_strides_and_edges(tb):
    w = W.get_workload(1, B=5, T=40)
    data = W.batch_inputs(w)
    lengths = [40, 0, 1, 17, 39]
    run_and_compare(tb, w, data, lengths=lengths, what="lengths")
    # non-contiguous logits: rows padded to 272 elements, streams reversed in memory
    batch, _ = make_batch(tb, w, data["phrases"])
    big = torch.zeros((w.B, w.T, w.S, 272), dtype=torch.float32, device="cuda:0")
    big[..., 5:5 + w.V + 1] = to_device(data["logits"])
    view = big[..., 5:5 + w.V + 1]
    assert not view.is_contiguous()
    out = to_host(tb.tb_greedy_decode(batch, view))
    for i in range(w.B):
        check_greedy(out, i, O.greedy_rnnt(oracle_graph(w, data["phrases"][i]), data["logits"][i]), "strided")
    # S = 1 and T = 1
    for T, S in ((1, 3), (9, 1)):
        w2 = W.get_workload(1, B=2, T=T, S=S, n_plants=0)
        d2 = W.batch_inputs(w2)
        run_and_compare(tb, w2, d2, what=f"T{T}S{S}")


def test_exact_ties_go_to_lowest_id(tb):
    w = W.get_workload(1, B=2, T=30, n_plants=0)
    data = W.batch_inputs(w)
    x = data["logits"]
    x[:, ::2, 0, :] = np.round(x[:, ::2, 0, :] * 2) / 2           # coarse grid: many exact ties
    x[0, 1, 0, 10] = x[0, 1, 0, 200] = x[0, 1, 0, w.V] = 9.0      # token tie that also ties with blank
    run_and_compare(tb, w, data, what="ties")


def test_rebind_one_slot_leaves_others_alone(tb):
    """Sec. 2.2 para. 4: lists are swapped while other streams keep theirs."""
    w = W.get_workload(2, B=6, T=100)
    data = W.batch_inputs(w)
    batch, graphs = make_batch(tb, w, data["phrases"], arena_bytes=1 << 20)
    logits = to_device(data["logits"])
    before = to_host(tb.tb_greedy_decode(batch, logits))
    other = W.stream_phrases(w, 77)
    g_new = tb.tb_graph_compile(other, w.V, case_class=w.vocab.case_class)
    tb.tb_batch_bind_stream(batch, 2, g_new)
    g_new.free()                                   # bind copied what it needs
    tb.tb_batch_bind_stream(batch, 4, None)
    after = to_host(tb.tb_greedy_decode(batch, logits))
    for i in (0, 1, 3, 5):
        for k in before:
            assert np.array_equal(before[k][i], after[k][i]), (i, k)
    check_greedy(after, 2, O.greedy_rnnt(oracle_graph(w, other), data["logits"][2]), "rebound")
    check_greedy(after, 4, O.greedy_rnnt(None, data["logits"][4]), "unbound")
    # churn the arena: many swaps into a small arena must keep working (free list reuse)
    for r in range(40):
        g = tb.tb_graph_compile(W.stream_phrases(w, 100 + r), w.V, case_class=w.vocab.case_class)
        tb.tb_batch_bind_stream(batch, r % w.B, g)
    final = to_host(tb.tb_greedy_decode(batch, logits))
    for i in range(w.B):
        r = max(r for r in range(40) if r % w.B == i)
        check_greedy(final, i, O.greedy_rnnt(oracle_graph(w, W.stream_phrases(w, 100 + r)), data["logits"][i]), "churn")


def test_error_codes(tb):
    w = W.get_workload(1, B=2, T=8)
    data = W.batch_inputs(w)
    batch, graphs = make_batch(tb, w, data["phrases"], arena_bytes=8192)

    def code(fn, *a, **k):
        with pytest.raises(tb.TbError) as e:
            fn(*a, **k)
        return e.value.code
    assert code(tb.tb_batch_bind_stream, batch, 2, graphs[0]) == tb.TB_ERR_BAD_SLOT
    assert code(tb.tb_batch_bind_stream, batch, -1, graphs[0]) == tb.TB_ERR_BAD_SLOT
    other_vocab = tb.tb_graph_compile([[1, 2]], w.V - 1)
    assert code(tb.tb_batch_bind_stream, batch, 0, other_vocab) == tb.TB_ERR_INVALID_ARG
    other_map = tb.tb_graph_compile([[1, 2]], w.V)          # identity class map
    assert code(tb.tb_batch_bind_stream, batch, 0, other_map) == tb.TB_ERR_INVALID_ARG
    big = tb.tb_graph_compile(W.stream_phrases(W.get_workload(1, n_phrases=400), 0), w.V, case_class=w.vocab.case_class)
    logits = to_device(data["logits"])
    before = to_host(tb.tb_greedy_decode(batch, logits))
    assert code(tb.tb_batch_bind_stream, batch, 0, big) == tb.TB_ERR_ARENA_FULL
    after = to_host(tb.tb_greedy_decode(batch, logits))       # a failed bind changes nothing
    for k in before:
        assert np.array_equal(before[k], after[k])
    three = torch.zeros((3, 8, 3, w.V + 1), device="cuda:0")
    assert code(tb.tb_greedy_decode, batch, three) == tb.TB_ERR_INVALID_ARG   # B > n_slots
    assert code(tb.tb_batch_create, 0, None, 1) == tb.TB_ERR_INVALID_ARG
    assert code(tb.tb_batch_create, 8, None, 1, max_beam=99) == tb.TB_ERR_INVALID_ARG


# ---------------------------------------------------------------------------------------------
# the pipelined kernel (packed bf16) against the oracle and against the general kernel
# ---------------------------------------------------------------------------------------------

SEG_PLANS = [(2, 8, 0), (1, 3, 1), (3, 7, 2), (4, 9, 3)]    # deciders, helpers per block; blocks per stream (0: automatic)


def both_kernels(tb, w, data, phrase_lists=None, weights=None, lam=None, lengths=None, logits=None, what="", plans=SEG_PLANS,
                 expect_fast=None):
    """Every kernel tb_greedy_decode can take -- the segmented one under several plans, the one-block-per-stream
    pipelined one, the general one -- against the oracle, stream by stream; all must agree bit for bit."""
    phrase_lists = data["phrases"] if phrase_lists is None else phrase_lists
    batch, _ = make_batch(tb, w, phrase_lists, weights=weights, lam=lam)
    logits = to_device(data["logits"]) if logits is None else logits
    dl = None if lengths is None else torch.tensor(lengths, dtype=torch.int32, device="cuda:0")
    refs = []
    for i, p in enumerate(phrase_lists):
        g = oracle_graph(w, p, None if weights is None else weights[i], lam)
        refs.append(O.greedy_rnnt(g, data["logits"][i], None if lengths is None else lengths[i]))
    outs = {}
    for plan in plans:
        tb.tb_batch_set_greedy_plan(batch, *plan)
        outs[f"segmented{plan}"] = to_host(tb.tb_greedy_decode(batch, logits, lengths=dl))
        outs[f"segmented{plan} again"] = to_host(tb.tb_greedy_decode(batch, logits, lengths=dl))   # what the first launch left must not matter
        if expect_fast is not None:
            assert (tb.tb_batch_last_greedy_kernel(batch)["kernel"] == tb.TB_KERNEL_SEGMENTED) == expect_fast, plan
    tb.tb_batch_set_greedy_plan(batch, 0, 0, 0)
    tb.tb_batch_set_flags(batch, tb.TB_FLAG_ONE_BLOCK_PER_STREAM)
    fast = outs["pipelined"] = to_host(tb.tb_greedy_decode(batch, logits, lengths=dl))
    if expect_fast is not None:
        assert (tb.tb_batch_last_greedy_kernel(batch)["kernel"] == tb.TB_KERNEL_PIPELINED) == expect_fast
    tb.tb_batch_set_flags(batch, tb.TB_FLAG_GENERAL_KERNELS)
    outs["general"] = to_host(tb.tb_greedy_decode(batch, logits, lengths=dl))
    assert tb.tb_batch_last_greedy_kernel(batch)["kernel"] == tb.TB_KERNEL_GENERAL
    tb.tb_batch_set_flags(batch, 0)
    assert tb.tb_batch_status(batch) == 0
    for name, out in outs.items():
        for i, ref in enumerate(refs):
            check_greedy(out, i, ref, f"{what} {name}")
            assert out["scores"][i] == fast["scores"][i], (name, i)
    return fast


def decode_every_way(tb, batch, logits, lengths, seed=0):
    """Outputs of tb_greedy_decode on one batch under the default choice of kernel, a forced segmented plan (where the
    call fits the segmented kernel; otherwise the library falls back by itself), the one-block-per-stream pipelined
    kernel and the general kernel."""
    outs = {"default": to_host(tb.tb_greedy_decode(batch, logits, lengths=lengths))}
    tb.tb_batch_set_greedy_plan(batch, *SEG_PLANS[seed % len(SEG_PLANS)])
    outs["segmented"] = to_host(tb.tb_greedy_decode(batch, logits, lengths=lengths))
    tb.tb_batch_set_greedy_plan(batch, 0, 0, 0)
    tb.tb_batch_set_flags(batch, tb.TB_FLAG_ONE_BLOCK_PER_STREAM)
    outs["pipelined"] = to_host(tb.tb_greedy_decode(batch, logits, lengths=lengths))
    tb.tb_batch_set_flags(batch, tb.TB_FLAG_GENERAL_KERNELS)
    outs["general"] = to_host(tb.tb_greedy_decode(batch, logits, lengths=lengths))
    tb.tb_batch_set_flags(batch, 0)
    assert tb.tb_batch_status(batch) == 0
    return outs


@pytest.mark.parametrize("V,S,T", [(1024, 3, 150), (300, 4, 70), (256, 1, 90), (2048, 2, 40), (700, 3, 33)])
def test_pipelined_kernel_shapes(tb, V, S, T):
    w = W.get_workload(2, B=7, T=T, S=S, V=V, n_phrases=60, n_plants=8)
    data = W.batch_inputs(w)
    lists = list(data["phrases"])
    lists[1] = None
    lists[4] = []
    lengths = [T, T - 1, 0, 1, T // 2, T, 3]
    both_kernels(tb, w, data, phrase_lists=lists, lengths=lengths, what=f"V{V}S{S}", expect_fast=V <= 2047)


@pytest.mark.parametrize("lam", [0.5, 2.0, -1.0])
def test_pipelined_kernel_weights_and_ties(tb, lam):
    """Coarse logits (many exact ties), mixed weights, lambda of either sign: the exact rescan path."""
    w = W.get_workload(2, B=6, T=120, n_phrases=80, n_plants=10)
    data = W.batch_inputs(w)
    x = W.bf16_bits_to_f32(data["logits"])
    x[:, ::3] = np.round(x[:, ::3] * 4) / 4
    data["logits"] = W.f32_to_bf16_bits(x)
    rng = np.random.default_rng(3)
    weights = [[[float(rng.choice([0.5, 1.0, 1.5, 2.0])) for _ in p] for p in lst] for lst in data["phrases"]]
    both_kernels(tb, w, data, weights=weights, lam=lam, what=f"ties lam{lam}")


def test_pipelined_kernel_unaligned_and_padded_frames(tb):
    w = W.get_workload(2, B=4, T=50, n_phrases=40, n_plants=5)
    data = W.batch_inputs(w)
    Wd = w.V + 1
    for shift, pad in ((1, 0), (3, 0), (0, 7), (5, 64)):
        flat = torch.zeros(shift + w.B * w.T * (w.S * Wd + pad) + 8, dtype=torch.bfloat16, device="cuda:0")
        view = flat[shift:shift + w.B * w.T * (w.S * Wd + pad)].view(w.B, w.T, w.S * Wd + pad)[:, :, :w.S * Wd]
        view = view.reshape(w.B, w.T, w.S, Wd) if pad == 0 else view.unflatten(2, (w.S, Wd))
        view.copy_(to_device(data["logits"]))
        assert view.data_ptr() % 16 == (flat.data_ptr() + 2 * shift) % 16
        both_kernels(tb, w, data, logits=view, what=f"shift{shift}pad{pad}")
    # the last stream's last frame ends exactly at the end of the allocation's tensor
    exact = to_device(data["logits"]).clone()
    both_kernels(tb, w, data, logits=exact, what="exact end")


def test_pipelined_kernel_large_lists_not_cached(tb):
    """Graphs too large for the shared-memory cache are walked in the arena (workload 3 lists)."""
    w = W.get_workload(3, B=2, T=150)
    data = W.batch_inputs(w)
    both_kernels(tb, w, data, what="w3")


@pytest.mark.parametrize("V,S", [(5, 3), (17, 2), (33, 4)])
def test_pipelined_kernel_tiny_vocabularies(tb, V, S):
    """Rows far shorter than one 16-byte-block pass of the helpers."""
    rng = np.random.default_rng(V)
    B, T = 5, 60
    cc = (np.arange(V) // 2).astype(np.int32)
    x = rng.standard_normal((B, T, S, V + 1)).astype(np.float32)
    x[..., V] += 0.5
    xb = W.f32_to_bf16_bits(x)
    lists = [[[int(t) for t in rng.integers(0, V, size=rng.integers(1, 4))] for _ in range(6)] for _ in range(B)]
    lists[2] = None
    batch = tb.tb_batch_create(V, cc, B + 2, arena_bytes=1 << 20)          # more slots than streams
    for i, p in enumerate(lists):
        tb.tb_batch_bind_stream(batch, i, None if p is None else tb.tb_graph_compile(p, V, case_class=cc))
    lengths = torch.tensor([T, T + 50, 7, 0, T - 1], dtype=torch.int32, device="cuda:0")   # T + 50 is clamped to T
    out = to_host(tb.tb_greedy_decode(batch, to_device(xb), lengths=lengths))
    assert tb.tb_batch_status(batch) == 0
    for i, p in enumerate(lists):
        g = None if p is None else O.Graph(p, V, case_class=cc)
        check_greedy(out, i, O.greedy_rnnt(g, xb[i], min(int(lengths[i]), T)), f"V{V}")


@pytest.mark.parametrize("seed", range(10))
def test_pipelined_kernel_random_configurations(tb, seed):
    """Random shapes, class maps, list sizes, weights, lambda, lengths and base offsets: both kernels
    against the oracle."""
    rng = np.random.default_rng(1000 + seed)
    V = int(rng.choice([9, 40, 255, 256, 257, 511, 1023, 1500, 2046]))
    S = int(rng.integers(1, 5))
    B, T = int(rng.integers(1, 7)), int(rng.integers(1, 70))
    n_cls = int(rng.integers(1, V + 1))
    cc = rng.integers(0, n_cls, size=V).astype(np.int32)
    lam = float(rng.choice([1.0, 0.5, 2.0, -0.5]))
    x = rng.standard_normal((B, T, S, V + 1)).astype(np.float32) * float(rng.choice([0.3, 1.0, 3.0]))
    x[..., V] += float(rng.choice([0.0, 1.0, 3.0]))
    if seed % 3 == 0:
        x = np.round(x * 2) / 2                                   # coarse grid: exact ties everywhere
    xb = W.f32_to_bf16_bits(x)
    lists, weights = [], []
    hot = rng.integers(0, V, size=max(2, V // 20))                # a small pool makes phrases chain and repeat
    for b in range(B):
        n = int(rng.integers(0, 60))
        ph = [[int(t) for t in rng.choice(hot, size=rng.integers(1, 6))] for _ in range(n)]
        lists.append(None if (b == 1 and B > 1) else ph)
        weights.append([[float(rng.choice([0.5, 1.0, 1.5, 2.0])) for _ in p] for p in ph])
    batch = tb.tb_batch_create(V, cc, B, arena_bytes=8 << 20)
    for i, p in enumerate(lists):
        if p is not None:
            tb.tb_batch_bind_stream(batch, i, tb.tb_graph_compile(p, V, case_class=cc, token_weights=weights[i], lam=lam))
    shift = int(rng.integers(0, 9))
    flat = torch.zeros(shift + xb.size + 8, dtype=torch.bfloat16, device="cuda:0")
    view = flat[shift:shift + xb.size].view(B, T, S, V + 1)
    view.copy_(to_device(xb))
    lens = rng.integers(0, T + 1, size=B).astype(np.int32)
    dl = torch.from_numpy(lens).to("cuda:0")
    outs = decode_every_way(tb, batch, view, dl, seed)
    for i, p in enumerate(lists):
        g = None if p is None else O.Graph(p, V, case_class=cc, weights=weights[i], lam=lam)
        ref = O.greedy_rnnt(g, xb[i], int(lens[i]))
        for name, out in outs.items():
            check_greedy(out, i, ref, f"seed{seed} {name} V{V} S{S}")


# ---------------------------------------------------------------------------------------------
# streams long enough to be decoded as two segments that are merged at the end
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("V,S,T", [(1024, 3, 128), (1024, 3, 129), (1024, 3, 193), (300, 4, 260), (256, 1, 500), (700, 2, 333)])
def test_two_segment_decode_shapes(tb, V, S, T):
    """Lengths on both sides of the two-segment threshold in one batch, an unbound slot and an empty list."""
    w = W.get_workload(2, B=8, T=T, S=S, V=V, n_phrases=60, n_plants=12)
    data = W.batch_inputs(w)
    lists = list(data["phrases"])
    lists[1] = None
    lists[4] = []
    lengths = [T, T, 127, 128, T, T - 1, 0, 200 if T >= 200 else T]
    both_kernels(tb, w, data, phrase_lists=lists, lengths=lengths, what=f"two segments V{V}S{S}T{T}")


@pytest.mark.parametrize("seed", range(6))
def test_two_segment_decode_slow_to_meet(tb, seed):
    """Heavy boosts over a small pool of tokens keep the decode inside phrases, so the segment that starts in the
    root state takes long to fall in with the true one (or never does); coarse logits add exact ties."""
    rng = np.random.default_rng(7000 + seed)
    V, S = int(rng.choice([64, 257, 1024])), int(rng.integers(1, 4))
    B, T = 5, int(rng.integers(128, 420))
    cc = rng.integers(0, max(1, V // 2), size=V).astype(np.int32)
    lam = float(rng.choice([1.0, 3.0, -2.0]))
    x = rng.standard_normal((B, T, S, V + 1)).astype(np.float32) * float(rng.choice([0.5, 1.0]))
    x[..., V] += float(rng.choice([0.5, 2.0]))
    if seed % 2 == 0:
        x = np.round(x * 2) / 2
    xb = W.f32_to_bf16_bits(x)
    hot = rng.integers(0, V, size=6)
    lists, weights = [], []
    for b in range(B):
        ph = [[int(t) for t in rng.choice(hot, size=rng.integers(2, 9))] for _ in range(int(rng.integers(5, 80)))]
        lists.append(ph)
        weights.append([[float(rng.choice([0.5, 1.0, 2.0, 4.0])) for _ in p] for p in ph])
    batch = tb.tb_batch_create(V, cc, B, arena_bytes=16 << 20)
    for i, p in enumerate(lists):
        tb.tb_batch_bind_stream(batch, i, tb.tb_graph_compile(p, V, case_class=cc, token_weights=weights[i], lam=lam))
    lens = np.array([T, T - 3, 128, T, 250 if T >= 250 else T], dtype=np.int32)
    dl = torch.from_numpy(lens).to("cuda:0")
    outs = decode_every_way(tb, batch, to_device(xb), dl, seed)
    for i, p in enumerate(lists):
        ref = O.greedy_rnnt(O.Graph(p, V, case_class=cc, weights=weights[i], lam=lam), xb[i], int(lens[i]))
        for name, out in outs.items():
            check_greedy(out, i, ref, f"seed {seed} {name}")
            assert out["scores"][i] == outs["general"]["scores"][i]


def test_two_segment_decode_repeats_and_rebinding(tb):
    """The same batch decoded again after a slot changed its list, and twice in a row: the scratch memory of the
    second segment carries nothing over."""
    w = W.get_workload(2, B=6, T=300, n_phrases=50, n_plants=15)
    data = W.batch_inputs(w)
    batch, _ = make_batch(tb, w, data["phrases"], arena_bytes=8 << 20)
    logits = to_device(data["logits"])
    first = to_host(tb.tb_greedy_decode(batch, logits))
    again = to_host(tb.tb_greedy_decode(batch, logits))
    for k in first:
        assert np.array_equal(first[k], again[k]), k
    other = W.stream_phrases(w, 17)
    tb.tb_batch_bind_stream(batch, 2, tb.tb_graph_compile(other, w.V, case_class=w.vocab.case_class))
    out = to_host(tb.tb_greedy_decode(batch, logits))
    assert tb.tb_batch_status(batch) == 0
    for i in range(w.B):
        p = other if i == 2 else data["phrases"][i]
        check_greedy(out, i, O.greedy_rnnt(oracle_graph(w, p), data["logits"][i]), "after rebinding")


@pytest.mark.parametrize("block", range(4))
def test_pipelined_kernel_soak_against_oracle(tb, block):
    """Ten random configurations per case, lengths on both sides of the two-segment threshold, any alignment:
    tokens, frames, states and the float32 score bit for bit as the oracle's."""
    for seed in range(10 * block, 10 * block + 10):
        rng = np.random.default_rng(50000 + seed)
        V = int(rng.choice([9, 64, 255, 256, 257, 511, 1023, 1024, 1500, 2046]))
        S = int(rng.integers(1, 5))
        B = int(rng.integers(1, 6))
        T = int(rng.choice([rng.integers(1, 128), rng.integers(128, 300), rng.integers(300, 700)]))
        cc = rng.integers(0, int(rng.integers(1, V + 1)), size=V).astype(np.int32)
        lam = float(rng.choice([1.0, 0.5, 2.0, 3.0, -0.5]))
        x = rng.standard_normal((B, T, S, V + 1)).astype(np.float32) * float(rng.choice([0.3, 1.0, 3.0]))
        x[..., V] += float(rng.choice([0.0, 1.0, 3.0]))
        if seed % 3 == 0:
            x = np.round(x * 2) / 2
        xb = W.f32_to_bf16_bits(x)
        hot = rng.integers(0, V, size=max(2, int(rng.choice([4, V // 20 + 2, V // 4 + 2]))))
        lists, weights = [], []
        for b in range(B):
            ph = [[int(t) for t in rng.choice(hot, size=rng.integers(1, 7))] for _ in range(int(rng.integers(0, 120)))]
            lists.append(None if (b == 1 and B > 1 and seed % 2) else ph)
            weights.append([[float(rng.choice([0.5, 1.0, 1.5, 2.0])) for _ in p] for p in ph])
        batch = tb.tb_batch_create(V, cc, B, arena_bytes=32 << 20)
        for i, p in enumerate(lists):
            if p is not None:
                tb.tb_batch_bind_stream(batch, i, tb.tb_graph_compile(p, V, case_class=cc, token_weights=weights[i], lam=lam))
        shift = int(rng.integers(0, 9))
        flat = torch.zeros(shift + xb.size + 8, dtype=torch.bfloat16, device="cuda:0")
        view = flat[shift:shift + xb.size].view(B, T, S, V + 1)
        view.copy_(to_device(xb))
        lens = rng.integers(max(0, T - 40), T + 1, size=B).astype(np.int32)
        outs = decode_every_way(tb, batch, view, torch.from_numpy(lens).to("cuda:0"), seed)
        for i, p in enumerate(lists):
            g = None if p is None else O.Graph(p, V, case_class=cc, weights=weights[i], lam=lam)
            ref = O.greedy_rnnt(g, xb[i], int(lens[i]))
            for name, out in outs.items():
                check_greedy(out, i, ref, f"seed {seed} {name}")
                assert float(out["scores"][i]) == float(ref["score"]), f"seed {seed} stream {i} {name}: score bits"


def test_greedy_decode_in_a_cuda_graph(tb):
    """One decode captured into a CUDA graph and replayed twice gives the outputs of the direct call -- both when
    an earlier call has sized the batch's scratch memory and when the batch's first decode happens under capture
    (nothing is allocated there; the streams are then decoded whole)."""
    w = W.get_workload(2, B=6, T=300, n_phrases=50, n_plants=15)
    data = W.batch_inputs(w)
    logits = to_device(data["logits"])
    refs = [O.greedy_rnnt(oracle_graph(w, data["phrases"][i]), data["logits"][i]) for i in range(w.B)]
    for warm in (True, False):
        batch, _ = make_batch(tb, w, data["phrases"], arena_bytes=8 << 20)
        n = w.T * w.S
        out = dict(tokens=torch.zeros((w.B, n), dtype=torch.int32, device="cuda:0"),
                   frames=torch.zeros((w.B, n), dtype=torch.int32, device="cuda:0"),
                   counts=torch.zeros(w.B, dtype=torch.int32, device="cuda:0"),
                   scores=torch.zeros(w.B, dtype=torch.float32, device="cuda:0"),
                   states=torch.zeros(w.B, dtype=torch.int32, device="cuda:0"))
        if warm:
            tb.tb_greedy_decode(batch, logits, out=out)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            tb.tb_greedy_decode(batch, logits, out=out, stream=torch.cuda.current_stream())
        for _ in range(2):
            for v in out.values():
                v.zero_()
            graph.replay()
            host = to_host(out)
            for i in range(w.B):
                check_greedy(host, i, refs[i], f"graph replay, warm={warm}")
        assert tb.tb_batch_status(batch) == 0


@pytest.mark.parametrize("seed", range(3))
def test_pipelined_kernel_masked_logits(tb, seed):
    """Token logits of -inf (masked tokens), whole rows with every token masked: the decode picks blank there and
    stays bit-exact with the oracle."""
    rng = np.random.default_rng(8000 + seed)
    V, S, B, T = int(rng.choice([257, 1024])), int(rng.integers(2, 4)), 4, int(rng.choice([90, 260]))
    cc = (np.arange(V) // 3).astype(np.int32)
    x = rng.standard_normal((B, T, S, V + 1)).astype(np.float32)
    x[..., V] += 2.0
    m = rng.random(x.shape) < 0.15
    m[..., V] = False
    x[m] = -np.inf
    x[:, ::7, :, :V] = -np.inf
    xb = W.f32_to_bf16_bits(x)
    hot = rng.integers(0, V, size=12)
    lists = [[[int(t) for t in rng.choice(hot, size=rng.integers(1, 6))] for _ in range(40)] for _ in range(B)]
    batch = tb.tb_batch_create(V, cc, B, arena_bytes=8 << 20)
    for i, p in enumerate(lists):
        tb.tb_batch_bind_stream(batch, i, tb.tb_graph_compile(p, V, case_class=cc))
    outs = decode_every_way(tb, batch, to_device(xb), None, seed)
    for i, p in enumerate(lists):
        ref = O.greedy_rnnt(O.Graph(p, V, case_class=cc), xb[i])
        for name, out in outs.items():
            check_greedy(out, i, ref, f"masked seed {seed} {name}")
            assert float(out["scores"][i]) == float(ref["score"]) or (np.isinf(ref["score"]) and np.isinf(out["scores"][i]))


# ---------------------------------------------------------------------------------------------
# the segmented kernel: cut points, streams whose segments never meet, choice of kernel, reuse of its scratch memory
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("T", [47, 48, 49, 95, 96, 97, 143, 145, 191, 193, 400])
def test_segmented_decode_cut_points(tb, T):
    """Lengths on both sides of every multiple of the shortest segment (48 frames), so that the number of segments
    and their cut points change from stream to stream within one launch."""
    w = W.get_workload(2, B=7, T=T, n_phrases=60, n_plants=max(1, T // 25))
    data = W.batch_inputs(w)
    lists = list(data["phrases"])
    lists[3] = None
    lengths = [T, T - 1, max(0, T - 47), T, max(0, T - 48), max(0, T - 49), 1]
    both_kernels(tb, w, data, phrase_lists=lists, lengths=lengths, what=f"cut points T{T}", expect_fast=True)


def test_segmented_decode_segments_that_never_meet(tb):
    """A list with a phrase that repeats one class makes the graph state loop on itself: the decode stays in that
    state for most of the stream, a segment that starts in the root state hardly ever reaches it, and the first
    segment ends up decoding almost everything (with another list on the same logits as a control)."""
    w = W.get_workload(2, B=4, T=600, n_phrases=30, n_plants=0)
    data = W.batch_inputs(w)
    c = 5                                                     # class 5: tokens 15, 16, 17
    loop = [[15] * 6, [15, 15], [15, 40, 41]]
    lists = [loop + data["phrases"][0], data["phrases"][1], loop, None]
    x = W.bf16_bits_to_f32(data["logits"])
    x[:, :, :, 15:18] += 1.0                                  # the class is frequent enough to enter the loop, not to stay without it
    data["logits"] = W.f32_to_bf16_bits(x)
    fast = both_kernels(tb, w, data, phrase_lists=lists, what="never meet", expect_fast=True)
    assert fast["counts"][0] > 2 * fast["counts"][1] and fast["counts"][2] > 2 * fast["counts"][3]


def test_choice_of_greedy_kernel(tb):
    """Which kernel a call gets: few streams -> segmented (many blocks per stream); a full batch -> one block per
    stream; fp32 or a padded token stride -> general.  A silent fall-back would cost a factor, so it is observable."""
    w = W.get_workload(2, B=8, T=200, n_phrases=40, n_plants=5)
    data = W.batch_inputs(w)
    batch, _ = make_batch(tb, w, data["phrases"])
    logits = to_device(data["logits"])
    tb.tb_greedy_decode(batch, logits)
    k = tb.tb_batch_last_greedy_kernel(batch)
    assert k["kernel"] == tb.TB_KERNEL_SEGMENTED and k["blocks_per_stream"] * k["deciders_per_block"] >= 2
    big = W.get_workload(2, B=128, T=60, n_phrases=20, n_plants=2)
    dbig = W.batch_inputs(big)
    bbatch, _ = make_batch(tb, big, dbig["phrases"])
    tb.tb_greedy_decode(bbatch, to_device(dbig["logits"]))
    assert tb.tb_batch_last_greedy_kernel(bbatch)["kernel"] == tb.TB_KERNEL_PIPELINED
    tb.tb_greedy_decode(batch, logits.float())
    assert tb.tb_batch_last_greedy_kernel(batch)["kernel"] == tb.TB_KERNEL_GENERAL
    with pytest.raises(tb.TbError):
        tb.tb_batch_set_greedy_plan(batch, 5, 4, 0)
    with pytest.raises(tb.TbError):
        tb.tb_batch_set_greedy_plan(batch, 2, 0, 0)


def test_segmented_decode_reuses_its_scratch_memory(tb):
    """Launches of different shapes on one batch (more streams, longer streams, another plan) and back: the working
    memory is laid out anew each time and nothing of an earlier launch is taken for a record of this one."""
    w = W.get_workload(2, B=6, T=300, n_phrases=50, n_plants=10)
    data = W.batch_inputs(w)
    batch, _ = make_batch(tb, w, data["phrases"])
    logits = to_device(data["logits"])
    refs = [O.greedy_rnnt(oracle_graph(w, data["phrases"][i]), data["logits"][i]) for i in range(w.B)]
    refs150 = [O.greedy_rnnt(oracle_graph(w, data["phrases"][i]), data["logits"][i, :150]) for i in range(w.B)]
    for plan, nb, T in [((2, 8, 3), 6, 300), ((2, 8, 3), 3, 300), ((3, 7, 2), 6, 150), ((2, 8, 3), 6, 300), ((1, 3, 4), 6, 300),
                        ((2, 8, 3), 6, 300)]:
        tb.tb_batch_set_greedy_plan(batch, *plan)
        for _ in range(3):
            out = to_host(tb.tb_greedy_decode(batch, logits[:nb, :T]))
            assert tb.tb_batch_last_greedy_kernel(batch)["kernel"] == tb.TB_KERNEL_SEGMENTED
            for i in range(nb):
                check_greedy(out, i, (refs if T == 300 else refs150)[i], f"plan {plan} nb {nb} T {T}")
    assert tb.tb_batch_status(batch) == 0


def test_segmented_decode_in_a_cuda_graph(tb):
    """The segmented decode captured once and replayed: every replay starts from what the previous one left in the
    working memory (launch numbers advance on the device), with other logits in the same buffer each time."""
    w = W.get_workload(2, B=5, T=260, n_phrases=50, n_plants=10)
    data = W.batch_inputs(w)
    batch, _ = make_batch(tb, w, data["phrases"])
    tb.tb_batch_set_greedy_plan(batch, 2, 8, 3)
    logits = to_device(data["logits"]).clone()
    out = tb.tb_greedy_decode(batch, logits)                  # allocates the working memory (not allowed while capturing)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        tb.tb_greedy_decode(batch, logits, out=out, stream=torch.cuda.current_stream())
    assert tb.tb_batch_last_greedy_kernel(batch)["kernel"] == tb.TB_KERNEL_SEGMENTED
    for shift in (0, 1, 2):
        rolled = np.roll(data["logits"], shift, axis=0)        # stream i now carries the logits of stream i - shift
        logits.copy_(to_device(rolled))
        for v in out.values():
            v.zero_()
        graph.replay()
        host = to_host(out)
        for i in range(w.B):
            check_greedy(host, i, O.greedy_rnnt(oracle_graph(w, data["phrases"][i]), rolled[i]), f"replay, shift {shift}")
    assert tb.tb_batch_status(batch) == 0


def test_a_bounded_wait_that_runs_out(tb):
    """The kernels wait for each other's results with a limit on every wait.  The self-test flag makes one wait run
    out on purpose (a frame's summaries are withheld, the limit is a few thousand polls): the call returns, the status
    word carries TB_STATUS_WAIT_TIMEOUT, and the next ordinary decode on the same batch is bit-exact again."""
    w = W.get_workload(2, B=6, T=200, n_phrases=40, n_plants=6)
    data = W.batch_inputs(w)
    batch, _ = make_batch(tb, w, data["phrases"])
    logits = to_device(data["logits"])
    refs = [O.greedy_rnnt(oracle_graph(w, data["phrases"][i]), data["logits"][i]) for i in range(w.B)]
    tb.tb_batch_set_flags(batch, tb.TB_FLAG_TEST_WAIT_TIMEOUT)
    tb.tb_greedy_decode(batch, logits)
    torch.cuda.synchronize()                                  # the launch ends by itself
    status = tb.tb_batch_status(batch)
    assert status & tb.TB_STATUS_WAIT_TIMEOUT, status
    assert tb.tb_batch_status(batch) == 0                     # reading the status clears it
    tb.tb_batch_set_flags(batch, 0)
    for _ in range(2):
        out = to_host(tb.tb_greedy_decode(batch, logits))
        assert tb.tb_batch_last_greedy_kernel(batch)["kernel"] == tb.TB_KERNEL_SEGMENTED
        for i in range(w.B):
            check_greedy(out, i, refs[i], "after the timeout")
    assert tb.tb_batch_status(batch) == 0
