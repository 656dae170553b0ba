#!/usr/bin/env python
"""Benchmark of the boosted greedy decode hot path (workload 2: B=128 streams, T=750 frames,
S=3 rows per frame, V=1024 + blank, bf16 logits, 100 phrases per stream).

One "step" is one pass of the whole hot path over one batch: tb_greedy_decode over all streams
(boost + select + advance for every visited row, device-resident loop).  Graph compile and bind
happen once before the timed region (decoder-level registration in the paper's Table 3 terms).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  With N > 1 (under torchrun) every rank decodes its own batch of 128
independent streams (weak scaling, no collective on the data path; the only collective is the
timing barrier / max).

Side measurements, one JSON line each (not the headline): --workload 3 large lists, 4 beam decoding (step by
step, under graph replay, and all expansions in one launch), 5 streaming TDT chunks with stream churn, 6 variative
case-insensitive lists compiled from text, 7 model lifecycle sweep (cache: none / disk / memory / decoder).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2608_21343_b200 import workloads as W  # noqa: E402

METRIC = "boosted_greedy_decode_frames_per_s_B128"
UNIT = "frames/s"
# DRAM read + write bytes per logits row of k_greedy_fast, from an ncu capture of one 32-stream launch
# (155.53 MB read + 3.83 MB written for 72000 rows: each stream's second segment re-reads 16 warm-up frames, and
# what it emits goes through scratch memory); the kernel runs one block per stream, so traffic scales with the
# stream count.  Captured with the command recorded in profiles/greedy_fast_small_case_B32_counters.md
# (`python bench.py --streams 32 --steps 2 --warmup 3 --no-extras --one-block-per-stream` under
# `ncu --clock-control none -k regex:k_greedy_fast -s 4 -c 1 ...`) on the kernel as of the commit that made it a
# template over "rows normalised or not" (the plain instance; the earlier captures read 2233 and 2237); to be
# re-captured whenever tb_greedy_fast.cu or tb_fast_common.cuh changes.
NCU_DRAM_BYTES_PER_ROW = 2213.0


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "25"], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm = [float(r[0]) for r in self.rows if len(r) >= 6 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 6 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({names[i] for r in self.rows if len(r) >= 6 for i in range(4) if r[2 + i] == "Active"})
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def rows_visited(counts: np.ndarray, frames: np.ndarray, T: int, S: int) -> int:
    """Rows the decode loop read: per frame, the emitted tokens plus the closing blank row (no
    blank row when the frame closed by force after S tokens)."""
    total = 0
    for i in range(len(counts)):
        per = np.bincount(frames[i, :counts[i]], minlength=T)
        total += int(per.sum() + (per < S).sum())
    return total


def run_reference(args, w):
    """The oracle as it stands on the host cores, on a bounded sample of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle as orc
    n_sample = 8
    streams = [W.stream_inputs(w, b) for b in range(n_sample)]
    graphs = [orc.Graph(d["phrases"], w.V, case_class=w.vocab.case_class) for d in streams]

    def step():
        for d, g in zip(streams, graphs):
            orc.greedy_rnnt(g, d["logits"])
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / args.steps
    val = n_sample * w.T / dt
    sample = f"{n_sample} of {w.B} streams per step, full length T={w.T}"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "T": w.T, "S": w.S, "V": w.V, "logits": w.dtype, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def side_measurement(args):
    """Workloads 3-5 on one GPU: one JSON line each, with that workload's own metric (not the headline)."""
    import torch
    from paper_2608_21343_b200 import binding as tb
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)

    def timed(fn, n, warm):
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(n):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / n

    if args.workload == 3:
        w = W.get_workload(3, **({"B": args.streams} if args.streams else {}))
        data = W.batch_inputs(w)
        t0 = time.perf_counter()
        graphs = [tb.tb_graph_compile(p, w.V, case_class=w.vocab.case_class) for p in data["phrases"]]
        compile_ms = (time.perf_counter() - t0) * 1e3 / w.B
        batch = tb.tb_batch_create(w.V, w.vocab.case_class, w.B, arena_bytes=int(4.5e6) * w.B + (1 << 20))
        for i, g in enumerate(graphs):
            tb.tb_batch_bind_stream(batch, i, g)
        logits = torch.from_numpy(data["logits"]).view(torch.bfloat16).to(dev)
        out = tb.tb_greedy_decode(batch, logits)
        ms = timed(lambda: tb.tb_greedy_decode(batch, logits, out=out), args.steps, args.warmup)
        assert tb.tb_batch_status(batch) == 0
        print(json.dumps({"metric": "boosted_greedy_decode_frames_per_s_large_lists", "value": w.B * w.T / (ms * 1e-3),
                          "unit": UNIT, "ms_per_step": ms, "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
                          "config": {"workload": w.name, "B": w.B, "T": w.T, "states_per_graph": graphs[0].view()["n_states"]},
                          "graph_compile_ms_per_list": compile_ms, "data": "synthetic"}))
    elif args.workload == 6:
        # variative, case-insensitive lists (Sec. 2.1, Eq. 1) at workload 2's shape: phrases as text over a synthetic
        # piece vocabulary, compiled per stream; spellings planted in random casings and segmentations
        B, T, S = (args.streams or 128), (args.frames or 750), 3
        pieces = W.make_piece_vocab(6, letters=26, merged=560, max_len=5)
        lists = [W.draw_string_phrases(6000 + b, pieces, 100, 1, 4) for b in range(B)]
        x = np.stack([W.variative_stream_logits(6, b, pieces, lists[b], T, S) for b in range(B)])
        cc, n_cls = tb.tb_piece_classes(pieces)
        t0 = time.perf_counter()
        graphs = [tb.tb_graph_compile_variative(p, pieces, tau=1.0) for p in lists]
        compile_ms = (time.perf_counter() - t0) * 1e3 / B
        v0 = graphs[0].view()
        batch = tb.tb_batch_create(len(pieces), cc, B, arena_bytes=(1 << 20) * B + (1 << 20))
        for i, g in enumerate(graphs):
            tb.tb_batch_bind_stream(batch, i, g)
        logits = torch.from_numpy(x).view(torch.bfloat16).to(dev)
        out = tb.tb_greedy_decode(batch, logits)
        ms = timed(lambda: tb.tb_greedy_decode(batch, logits, out=out), args.steps, args.warmup)
        assert tb.tb_batch_status(batch) == 0
        plain = tb.tb_batch_create(len(pieces), cc, B, arena_bytes=1 << 20)
        out0 = tb.tb_greedy_decode(plain, logits)
        ms0 = timed(lambda: tb.tb_greedy_decode(plain, logits, out=out0), args.steps, args.warmup)
        print(json.dumps({"metric": "boosted_greedy_decode_frames_per_s_variative_lists", "value": B * T / (ms * 1e-3),
                          "unit": UNIT, "ms_per_step": ms, "unboosted_ms_per_step": ms0, "n_gpus": 1, "steps": args.steps,
                          "warmup": args.warmup,
                          "config": {"workload": "variative_greedy_rnnt", "B": B, "T": T, "S": S, "V": len(pieces),
                                     "classes": n_cls, "phrases_per_stream": 100, "tau": 1.0,
                                     "states_per_graph": v0["n_states"], "arcs_per_graph": v0["n_arcs"]},
                          "graph_compile_ms_per_list": compile_ms,
                          "graph_compile_phrases_per_s": 100.0 / (compile_ms * 1e-3),
                          "tokens_emitted": int(out["counts"].sum().item()), "data": "synthetic"}))
    elif args.workload == 4:
        w = W.get_workload(4)
        data = W.batch_inputs(w)
        B, T, E, _ = data["logits"].shape
        K = w.K
        batch = tb.tb_batch_create(w.V, w.vocab.case_class, B, max_beam=K, max_tree_steps=T * E, arena_bytes=64 << 20)
        for i, p in enumerate(data["phrases"]):
            tb.tb_batch_bind_stream(batch, i, tb.tb_graph_compile(p, w.V, case_class=w.vocab.case_class))
        logits = torch.from_numpy(data["logits"]).view(torch.bfloat16).to(dev)
        sb, st, se, _ = logits.stride()
        scores = torch.empty((B, K), device=dev)
        states = torch.empty((B, K), dtype=torch.int32, device=dev)
        live = torch.zeros((B, K), dtype=torch.uint8, device=dev)
        par = torch.empty((B, K), dtype=torch.int32, device=dev)
        tok = torch.empty_like(par)

        def run():
            scores.fill_(float("-inf")); scores[:, 0] = 0.0
            states.fill_(-1); states[:, 0] = 0
            tb.tb_beam_reset(batch)
            for t in range(T):
                for e in range(E):
                    tb.tb_beam_step(batch, logits, sb, 0, e == 0, scores, states, live, par, tok, offset=t * st + e * se)
        ms = timed(run, max(2, args.steps // 5), 1)
        # the same T*E steps captured once in a CUDA graph and replayed: no host work per step
        graph_ms = None
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                run()
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            cg = torch.cuda.CUDAGraph()
            with torch.cuda.graph(cg):
                run()
            graph_ms = timed(cg.replay, max(2, args.steps // 5), 1)
        except Exception as exc:  # noqa: BLE001
            graph_ms = f"capture failed: {exc}"
        # ... and the whole utterance in one launch (each stream's block loops over its expansions)
        l4 = logits.view(B, T, E, -1)

        def run_fused():
            scores.fill_(float("-inf")); scores[:, 0] = 0.0
            states.fill_(-1); states[:, 0] = 0
            tb.tb_beam_reset(batch)
            tb.tb_beam_frames(batch, l4, False, scores, states, live, par, tok)
        fused_ms = timed(run_fused, max(2, args.steps // 5), 1)
        assert tb.tb_batch_status(batch) == 0
        print(json.dumps({"metric": "beam_decode_frames_per_s_K4_B32", "value": B * T / (ms * 1e-3), "unit": UNIT,
                          "ms_per_decode": ms, "us_per_beam_step": ms * 1e3 / (T * E), "n_gpus": 1,
                          "cuda_graph_ms_per_decode": graph_ms, "one_launch_ms_per_decode": fused_ms,
                          "one_launch_frames_per_s": B * T / (fused_ms * 1e-3),
                          "config": {"workload": w.name, "B": B, "K": K, "T": T, "E": E,
                                     "note": "one tb_beam_step call per expansion, driven from the host"}, "data": "synthetic"}))
    elif args.workload == 5:
        w = W.get_workload(5, **({"B": args.streams} if args.streams else {}))
        sched = W.ChurnSchedule(w)                       # (inputs drawn by this thread: worker threads would compete with the timed calls for the interpreter)
        batch = tb.tb_batch_create(w.V, w.vocab.case_class, w.B, arena_bytes=256 << 20)
        n_chunks, lat, binds, t_compile = 40 + 10 * args.steps, [], 0, 0.0
        host_us = []
        ev5 = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
        ev5[0].record(); ev5[1].record(); torch.cuda.synchronize()
        bufs = []
        outs = None
        for c in range(n_chunks):
            chunk, lengths, bl = sched.next_chunk()
            t0 = time.perf_counter()
            gs = [(sl, tb.tb_graph_compile(p, w.V, case_class=w.vocab.case_class)) for sl, _, p in bl]
            t_compile += time.perf_counter() - t0
            dl = torch.from_numpy(chunk).view(torch.bfloat16).to(dev)      # a fresh buffer per chunk: nothing stays in L2
            dv = torch.from_numpy(lengths).to(dev)
            bufs = (bufs + [dl])[-8:]
            torch.cuda.synchronize()
            a, b = ev5                                     # (one pair of events for all chunks: every chunk ends with a synchronize)
            th = time.perf_counter()
            a.record()
            if args.single_binds:
                for sl, g in gs:
                    tb.tb_batch_bind_stream(batch, sl, g)
                outs = tb.tb_stream_chunk(batch, dl, w.n_dur, dv, out=outs)      # the result tensors are allocated once
            else:
                # the new streams' binds (one copy, one launch) and the chunk in one call
                outs = tb.tb_stream_chunk_binds(batch, [sl for sl, _ in gs], [g for _, g in gs], dl, w.n_dur, dv, out=outs)
            b.record()
            host_us.append((time.perf_counter() - th) * 1e6)
            torch.cuda.synchronize()
            lat.append(a.elapsed_time(b))
            binds += len(bl)
        lat = np.array(lat[10:])
        # The same, with the chunks' logits already on the device when the loop starts (as when the joint network
        # produced them there) and nothing but the library calls between two chunks: the schedule goes on, the next
        # chunks are staged first -- every chunk its own buffer, used once, so nothing of it is in L2 --, then timed.
        staged = []
        for c in range(min(96, max(16, n_chunks // 8))):
            chunk, lengths, bl = sched.next_chunk()
            gs = [(sl, tb.tb_graph_compile(p, w.V, case_class=w.vocab.case_class)) for sl, _, p in bl]
            staged.append(([sl for sl, _ in gs], [g for _, g in gs], torch.from_numpy(chunk).view(torch.bfloat16).to(dev),
                           torch.from_numpy(lengths).to(dev)))
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        res_lat, res_binds = [], 0
        for sl_, g_, dl, dv in staged:
            a.record()
            outs = tb.tb_stream_chunk_binds(batch, sl_, g_, dl, w.n_dur, dv, out=outs)
            b.record()
            torch.cuda.synchronize()
            res_lat.append(a.elapsed_time(b))
            res_binds += len(sl_)
        res_lat = np.array(res_lat[4:])
        assert tb.tb_batch_status(batch) == 0
        print(json.dumps({"metric": "streaming_tdt_chunk_latency_ms", "p50": float(np.percentile(lat, 50)),
                          "p99": float(np.percentile(lat, 99)), "unit": "ms", "higher_is_better": False, "n_gpus": 1,
                          "inputs_resident": {"p50": float(np.percentile(res_lat, 50)), "p99": float(np.percentile(res_lat, 99)),
                                              "chunks": len(res_lat), "binds_per_chunk": res_binds / max(1, len(staged)),
                                              "note": "chunk logits staged on the device before the loop, one buffer per chunk; binds and chunk call timed as above"},
                          "config": {"workload": w.name, "slots": w.B, "chunk_frames": w.chunk, "chunks": len(lat),
                                     "binds_in_timed_region": True, "rebinds": binds - w.B,
                                     "binds": "one by one" if args.single_binds else "tb_stream_chunk_binds (up to 16 binds per chunk carried out by the chunk's own launch, larger groups by copies and a launch ahead of it)",
                                     "bind_counts": tb.tb_batch_bind_counts(batch)},
                          "frames_per_s_at_p50": w.B * w.chunk / (float(np.percentile(lat, 50)) * 1e-3),
                          "host_issue_us_p50": float(np.percentile(np.array(host_us[10:]), 50)),
                          "graph_compile_ms_per_list": 1e3 * t_compile / max(1, binds),
                          "data": "synthetic"}))

    elif args.workload == 8:
        # Streaming beam search (Sec. 2.3; Sec. 3.4 uses beam 32): the streaming workload's churn without duration
        # logits, 2 expansions per frame, chunks of 8 frames through tb_beam_chunk; equal transcripts merged and the
        # beam pruned at frame starts; a finished stream gets its final weights and a backtrace, a new one is compiled
        # and bound.  Timed per chunk with the binds and the finishing calls inside the timed region.
        rows = []
        for K in (4, 32):
            w = W.get_workload(5, B=args.streams or 128, S=2, n_dur=0)
            E = w.S
            sched = W.ChurnSchedule(w)
            batch = tb.tb_batch_create(w.V, w.vocab.case_class, w.B, max_beam=K, max_tree_steps=w.T * E, arena_bytes=256 << 20)
            tb.tb_batch_set_beam_prune(batch, 10.0)
            scores = torch.full((w.B, K), float("-inf"), device=dev)
            states = torch.full((w.B, K), -1, dtype=torch.int32, device=dev)
            live = torch.zeros((w.B, K), dtype=torch.uint8, device=dev)
            par = torch.empty((w.B, K), dtype=torch.int32, device=dev)
            tok = torch.empty((w.B, K), dtype=torch.int32, device=dev)
            bt = (torch.zeros((w.B, K, 256), dtype=torch.int32, device=dev), torch.zeros((w.B, K), dtype=torch.int32, device=dev))
            tb.tb_beam_reset_slots(batch)
            served = np.zeros(w.B, dtype=np.int64)
            total = np.zeros(w.B, dtype=np.int64)
            n_chunks, lat, kern, n_done, frames = 30 + 2 * args.steps, [], [], 0, 0
            bufs = []
            ev8 = tuple(torch.cuda.Event(enable_timing=True) for _ in range(4))
            for e_ in ev8:
                e_.record()
            torch.cuda.synchronize()
            for c in range(n_chunks):
                chunk, lengths, bl = sched.next_chunk()
                gs = [(sl, tb.tb_graph_compile(p, w.V, case_class=w.vocab.case_class)) for sl, _, p in bl]
                for sl, _, _ in bl:
                    served[sl] = 0
                total[:] = lengths
                left = np.clip(total - served, 0, w.chunk).astype(np.int32)
                dl = torch.from_numpy(chunk).view(torch.bfloat16).to(dev)   # a fresh buffer per chunk: nothing stays in L2
                dn = torch.from_numpy(left).to(dev)
                bufs = (bufs + [dl])[-8:]
                new = [sl for sl, _ in gs]
                torch.cuda.synchronize()
                a, m0, m1, b = ev8                          # (one set of events for all chunks: every chunk ends with a synchronize)
                a.record()
                tb.tb_batch_bind_streams(batch, new, [g for _, g in gs])
                tb.tb_beam_start_slots(batch, new, scores, states, live)     # the new slots' beams, set up by the library
                m0.record()
                tb.tb_beam_chunk(batch, dl, True, dn, scores, states, live, par, tok)
                m1.record()
                served += left
                ended = [sl for sl in range(w.B) if left[sl] > 0 and served[sl] >= total[sl]]
                if ended:
                    tb.tb_apply_final_weights_slots(batch, ended, scores, states)
                    tb.tb_beam_backtrace_slot_list(batch, ended, K, 256, out=bt)    # the transcripts of the streams that ended
                b.record()
                torch.cuda.synchronize()
                lat.append(a.elapsed_time(b)); kern.append(m0.elapsed_time(m1))
                n_done += len(ended); frames += int(left.sum())
            assert tb.tb_batch_status(batch) == 0
            # the same with the chunks' logits on the device before the loop starts (one buffer per chunk, used once) and
            # nothing but the library calls between two chunks
            staged = []
            for c in range(min(96, max(16, n_chunks // 4))):
                chunk, lengths, bl = sched.next_chunk()
                gs = [(sl, tb.tb_graph_compile(p, w.V, case_class=w.vocab.case_class)) for sl, _, p in bl]
                for sl, _, _ in bl:
                    served[sl] = 0
                total[:] = lengths
                left = np.clip(total - served, 0, w.chunk).astype(np.int32)
                served += left
                ended = [sl for sl in range(w.B) if left[sl] > 0 and served[sl] >= total[sl]]
                staged.append(([sl for sl, _ in gs], [g for _, g in gs], torch.from_numpy(chunk).view(torch.bfloat16).to(dev),
                               torch.from_numpy(left).to(dev), ended))
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            res_lat = []
            for new, g_, dl, dn, ended in staged:
                a.record()
                tb.tb_batch_bind_streams(batch, new, g_)
                tb.tb_beam_start_slots(batch, new, scores, states, live)
                tb.tb_beam_chunk(batch, dl, True, dn, scores, states, live, par, tok)
                if ended:
                    tb.tb_apply_final_weights_slots(batch, ended, scores, states)
                    tb.tb_beam_backtrace_slot_list(batch, ended, K, 256, out=bt)
                b.record()
                torch.cuda.synchronize()
                res_lat.append(a.elapsed_time(b))
            res_lat = np.array(res_lat[4:])
            assert tb.tb_batch_status(batch) == 0
            sched.close()
            lat, kern = np.array(lat[10:]), np.array(kern[10:])
            rows.append({"K": K, "p50_ms": float(np.percentile(lat, 50)), "p99_ms": float(np.percentile(lat, 99)),
                         "inputs_resident": {"p50_ms": float(np.percentile(res_lat, 50)), "p99_ms": float(np.percentile(res_lat, 99)),
                                             "chunks": int(len(res_lat))},
                         "chunk_kernel_p50_ms": float(np.percentile(kern, 50)),
                         "frames_per_s_at_p50": w.B * w.chunk / (float(np.percentile(lat, 50)) * 1e-3),
                         "chunks": int(len(lat)), "streams_finished": n_done})
        print(json.dumps({"metric": "streaming_beam_chunk_latency_ms", "unit": "ms", "higher_is_better": False, "n_gpus": 1,
                          "rows": rows, "config": {"workload": "streaming_beam_churn", "slots": w.B, "chunk_frames": w.chunk,
                                                   "expansions_per_frame": E, "merge": True, "prune_delta": 10.0,
                                                   "binds_and_finishing_in_timed_region": True}, "data": "synthetic"}))

    elif args.workload == 7:
        # Model lifecycle sweep in the manner of the paper's speed table (128 streams; cache: none / disk / memory /
        # decoder): the streaming workload's churn with 128 slots, the same schedule for every mode; the timed region of
        # a chunk is host wall clock from "the new streams' lists are known" to "the chunk is decoded".
        import tempfile
        w = W.get_workload(5, B=args.streams or 128)
        cc = w.vocab.case_class
        sched = W.ChurnSchedule(w)
        n_chunks = 30 + max(args.steps, 100)
        plan = [sched.next_chunk() for _ in range(n_chunks)]
        def flat(p):                                     # the lists as arrays, as a server would hold them
            offs = np.zeros(len(p) + 1, dtype=np.int64)
            offs[1:] = np.cumsum([len(x) for x in p])
            return (np.array([t for x in p for t in x], dtype=np.int32), offs)
        plan = [(c, l, [(sl, sid, flat(p)) for sl, sid, p in bl]) for c, l, bl in plan]
        lists = {sid: p for _, _, bl in plan for _, sid, p in bl}
        tmp = tempfile.mkdtemp(prefix="tb_lists_")
        rows = []
        for mode in ("none", "disk", "memory", "decoder"):
            batch = tb.tb_batch_create(w.V, cc, w.B, arena_bytes=1 << 30)
            cache, model_of = None, {}
            if mode == "disk":
                for sid, p in lists.items():
                    tb.tb_graph_save(tb.tb_graph_compile(p, w.V, case_class=cc), os.path.join(tmp, "%d.tbg" % sid))
            elif mode == "memory":
                cache = tb.tb_cache_create(1 << 30)
                for p in lists.values():
                    tb.tb_cache_compile(cache, p, w.V, case_class=cc)
            elif mode == "decoder":
                for sid, p in lists.items():
                    model_of[sid] = tb.tb_batch_register_model(batch, tb.tb_graph_compile(p, w.V, case_class=cc))
            torch.cuda.synchronize()
            lat, binds = [], 0
            for chunk, lengths, bl in plan:
                dl = torch.from_numpy(chunk).view(torch.bfloat16).to(dev)
                dv = torch.from_numpy(lengths).to(dev)
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                for sl, sid, p in bl:
                    if mode == "none":
                        tb.tb_batch_bind_stream(batch, sl, tb.tb_graph_compile(p, w.V, case_class=cc))
                    elif mode == "disk":
                        tb.tb_batch_bind_stream(batch, sl, tb.tb_graph_load(os.path.join(tmp, "%d.tbg" % sid)))
                    elif mode == "memory":
                        tb.tb_batch_bind_stream(batch, sl, tb.tb_cache_compile(cache, p, w.V, case_class=cc)[0])
                    else:
                        break
                if mode == "decoder" and bl:
                    tb.tb_batch_bind_models(batch, [sl for sl, _, _ in bl], [model_of[sid] for _, sid, _ in bl])
                tb.tb_stream_chunk(batch, dl, w.n_dur, dv)
                torch.cuda.synchronize()
                lat.append((time.perf_counter() - t0) * 1e3)
                binds += len(bl)
            assert tb.tb_batch_status(batch) == 0
            steady = np.array(lat[30:])                      # the first chunks bind every slot at once
            nb = sum(len(bl) for _, _, bl in plan[30:])
            rows.append({"cache": mode, "ms_per_chunk_mean": float(steady.mean()), "ms_per_chunk_p50": float(np.percentile(steady, 50)),
                         "ms_per_chunk_p99": float(np.percentile(steady, 99)),
                         "frames_per_s": w.B * w.chunk * len(steady) / (float(steady.sum()) * 1e-3),
                         "binds_per_chunk": nb / len(steady)})
            batch.destroy()
        # the same four levels around the offline decode of workload 2: every one of the 128 streams brings its own list
        w2 = W.get_workload(2)
        d2 = W.batch_inputs(w2)
        cc2 = w2.vocab.case_class
        l2 = torch.from_numpy(d2["logits"]).view(torch.bfloat16).to(dev)
        flat2 = [flat(p) for p in d2["phrases"]]
        rows2 = []
        for mode in ("none", "disk", "memory", "decoder"):
            batch = tb.tb_batch_create(w2.V, cc2, w2.B, arena_bytes=64 << 20)
            cache, ids = None, []
            if mode == "disk":
                for i, p in enumerate(flat2):
                    tb.tb_graph_save(tb.tb_graph_compile(p, w2.V, case_class=cc2), os.path.join(tmp, "w2_%d.tbg" % i))
            elif mode == "memory":
                cache = tb.tb_cache_create(1 << 30)
                for p in flat2:
                    tb.tb_cache_compile(cache, p, w2.V, case_class=cc2)
            elif mode == "decoder":
                ids = [tb.tb_batch_register_model(batch, tb.tb_graph_compile(p, w2.V, case_class=cc2)) for p in flat2]
            out2 = tb.tb_greedy_decode(batch, l2)
            torch.cuda.synchronize()
            ts = []
            all_slots = np.arange(w2.B, dtype=np.int32)
            slot_list = list(range(w2.B))
            for _ in range(max(5, args.steps // 20)):
                t0 = time.perf_counter()
                if mode == "none":
                    gl = [tb.tb_graph_compile(p, w2.V, case_class=cc2) for p in flat2]
                elif mode == "disk":
                    gl = [tb.tb_graph_load(os.path.join(tmp, "w2_%d.tbg" % i)) for i in range(len(flat2))]
                elif mode == "memory":
                    gl = [tb.tb_cache_compile(cache, p, w2.V, case_class=cc2)[0] for p in flat2]
                if mode == "decoder":
                    tb.tb_batch_bind_models(batch, all_slots, ids)
                else:
                    tb.tb_batch_bind_streams(batch, slot_list, gl)      # all 128 in one call
                    gl = None
                tb.tb_greedy_decode(batch, l2, out=out2)
                torch.cuda.synchronize()
                ts.append((time.perf_counter() - t0) * 1e3)
            assert tb.tb_batch_status(batch) == 0
            rows2.append({"cache": mode, "ms_per_batch": float(np.median(ts)), "frames_per_s": w2.B * w2.T / (float(np.median(ts)) * 1e-3)})
            batch.destroy()
        for r in rows2:
            r["vs_decoder_level"] = r["frames_per_s"] / rows2[-1]["frames_per_s"]
        print(json.dumps({"metric": "model_lifecycle_sweep_offline_greedy", "unit": UNIT, "n_gpus": 1, "rows": rows2,
                          "config": {"workload": w2.name, "B": w2.B, "T": w2.T, "phrases_per_stream": 100,
                                     "timed": "host wall clock per batch: obtain and bind all 128 streams' graphs, decode, synchronise"},
                          "data": "synthetic"}))
        base = rows[-1]["frames_per_s"]
        for r in rows:
            r["vs_decoder_level"] = r["frames_per_s"] / base
        print(json.dumps({"metric": "model_lifecycle_sweep_streaming_tdt", "unit": UNIT, "n_gpus": 1, "rows": rows,
                          "config": {"workload": w.name + " (128 slots)", "slots": w.B, "chunk_frames": w.chunk,
                                     "chunks": n_chunks - 30, "lists": len(lists),
                                     "timed": "host wall clock per chunk: obtain the new streams' graphs, bind, decode the chunk, synchronise"},
                          "data": "synthetic"}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--streams", type=int, default=0, help="override B (profiling captures use a small case)")
    ap.add_argument("--frames", type=int, default=0, help="override T (profiling captures use a small case)")
    ap.add_argument("--single-binds", action="store_true", help="workload 5: bind new streams one by one instead of in one call")
    ap.add_argument("--no-extras", action="store_true", help="skip unboosted / e2e / cpu legs (profiling)")
    ap.add_argument("--one-block-per-stream", action="store_true",
                    help="never the segmented kernel (small-case captures of k_greedy_fast: fewer streams would otherwise select it)")
    ap.add_argument("--log-softmax", action="store_true",
                    help="the timed decode normalises every visited row (TB_FLAG_LOG_SOFTMAX): a side measurement and profiling captures, not the headline")
    ap.add_argument("--workload", type=int, default=2, choices=[2, 3, 4, 5, 6, 7, 8],
                    help="2 = the headline (default); 3 large lists, 4 beam, 5 streaming TDT with churn, 6 variative lists, 7 model lifecycle sweep: side measurements")
    args = ap.parse_args()
    if args.workload != 2:
        side_measurement(args)
        return
    args.warmup = max(args.warmup, 3)
    over = {}
    if args.streams:
        over["B"] = args.streams
    if args.frames:
        over["T"] = args.frames
    w = W.get_workload(2, **over)
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    from paper_2608_21343_b200 import binding as tb

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    from paper_2608_21343_b200 import sharding

    # ---- inputs: this rank's own 128 streams (stream ids offset by rank), graphs compiled and bound
    streams = sharding.rank_streams(rank, w.B)
    data = W.batch_inputs(w, streams)
    host_logits = torch.from_numpy(data["logits"]).view(torch.bfloat16).pin_memory()
    logits = host_logits.to(dev, non_blocking=True)
    batch = tb.tb_batch_create(w.V, w.vocab.case_class, w.B, arena_bytes=32 << 20, device=local_rank)
    t_c = time.perf_counter()
    graphs = [tb.tb_graph_compile(p, w.V, case_class=w.vocab.case_class) for p in data["phrases"]]
    compile_s = time.perf_counter() - t_c
    for i, g in enumerate(graphs):
        tb.tb_batch_bind_stream(batch, i, g)
    plain = tb.tb_batch_create(w.V, w.vocab.case_class, w.B, arena_bytes=1 << 20, device=local_rank)  # all unbound
    main_flags = (tb.TB_FLAG_ONE_BLOCK_PER_STREAM if args.one_block_per_stream else 0) | (tb.TB_FLAG_LOG_SOFTMAX if args.log_softmax else 0)
    if main_flags:
        tb.tb_batch_set_flags(batch, main_flags)
        tb.tb_batch_set_flags(plain, main_flags)
    out = tb.tb_greedy_decode(batch, logits)
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()
    ran = tb.tb_batch_last_greedy_kernel(batch)       # which kernel the library chose for this shape
    kernel_name = {tb.TB_KERNEL_PIPELINED: "k_greedy_fast", tb.TB_KERNEL_SEGMENTED: "k_greedy_seg",
                   tb.TB_KERNEL_GENERAL: "k_decode_general"}[ran["kernel"]]
    fast = ran["kernel"] == tb.TB_KERNEL_PIPELINED

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, warmup, per_launch=False):
        for _ in range(warmup):
            fn()
        barrier()
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        evs[0].record(stream)
        for i in range(steps):
            fn()
            evs[i + 1].record(stream)
        barrier()
        total_ms = evs[0].elapsed_time(evs[-1])
        each = [evs[i].elapsed_time(evs[i + 1]) for i in range(steps)]
        return total_ms, each

    # clocks are sampled from before the warm-up until the timed steps end (the GPU is busy throughout;
    # the timed region alone can be shorter than one nvidia-smi sampling period)
    sampler = ClockSampler(local_rank)
    sampler.start()

    def keep_busy(until, limit_s):
        # untimed decodes, the same load as the timed ones, until the sampler has delivered enough lines
        t_end = time.perf_counter() + limit_s
        while not until() and time.perf_counter() < t_end:
            for _ in range(20):
                tb.tb_greedy_decode(batch, logits, out=out)
            torch.cuda.synchronize()
    keep_busy(lambda: len(sampler.rows) >= 1, 5.0)          # nvidia-smi takes a moment to come up
    n_before = len(sampler.rows)
    timed(lambda: tb.tb_greedy_decode(batch, logits, out=out), max(50, args.steps), args.warmup)
    total_ms, each_ms = timed(lambda: tb.tb_greedy_decode(batch, logits, out=out), args.steps, args.warmup)
    keep_busy(lambda: len(sampler.rows) - n_before >= 6, 3.0)   # the timed region can be shorter than a sampling period
    clocks = sampler.stop()
    assert tb.tb_batch_status(batch) == 0, "a kernel recorded a violated bound"
    job = sharding.job_throughput(w.B * w.T, total_ms / args.steps, device=dev)   # max over ranks of the time
    ms, value = job["ms"], job["value"]

    counts = out["counts"].cpu().numpy()
    frames = out["frames"].cpu().numpy()
    visited = rows_visited(counts, frames, w.T, w.S)
    row_bytes = 2 * (w.V + 1)
    peak, peak_kind = load_peaks()
    kern_ms = float(np.mean(each_ms))            # one kernel launch per step: launch-to-launch time on the stream
    achieved = visited * row_bytes / (kern_ms * 1e-3) / 1e9
    streamed = w.B * w.T * w.S * row_bytes / (kern_ms * 1e-3) / 1e9
    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "T": w.T, "S": w.S, "V": w.V, "logits": w.dtype,
                   "phrases_per_stream": w.n_phrases, "log_softmax": bool(args.log_softmax), "l2": "inputs (590 MB per step) larger than L2, no flush",
                   "parallelism": f"replicas x{world}, streams partitioned, no collective"},
        "gpu_launches": args.steps * 1,
        "clocks": clocks,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": NCU_DRAM_BYTES_PER_ROW * w.B * w.T * w.S if fast else None,
                     "traffic_note": "ncu dram read+write of a 32-stream launch scaled by streams" if fast else "captured for k_greedy_fast only",
                     "peak_kind": f"of {peak_kind}",
                     "kernel": f"{kernel_name} (one launch per decode; {ran['blocks_per_stream']} block(s) per stream)",
                     "rows_visited": visited, "bytes_per_row": row_bytes,
                     "all_rows_GBs": streamed, "all_rows_frac": streamed / peak,
                     "measured_GBs": NCU_DRAM_BYTES_PER_ROW * w.B * w.T * w.S / (kern_ms * 1e-3) / 1e9 if fast else None,
                     "measured_frac": NCU_DRAM_BYTES_PER_ROW * w.B * w.T * w.S / (kern_ms * 1e-3) / 1e9 / peak if fast else None,
                     "frac_of_nominal_8000": achieved / 8000.0},
        "ms_per_step_median": float(np.median(each_ms)), "ms_per_step_min": float(np.min(each_ms)),
        "ns_per_visited_row_per_stream": kern_ms * 1e6 / (visited / w.B),
        "rows_visited_per_frame": visited / (w.B * w.T),
        "tokens_emitted": int(counts.sum()),
        "graph_compile_ms_per_list": compile_s * 1e3 / w.B,
        "graph_compile_phrases_per_s": w.B * w.n_phrases / compile_s,
    }

    if rank == 0:
        # unboosted: the same call with every slot unbound
        out0 = tb.tb_greedy_decode(plain, logits)
        p_ms, _ = timed(lambda: tb.tb_greedy_decode(plain, logits, out=out0), args.steps, args.warmup)
        p_ms /= args.steps
        result["unboosted"] = {"ms_per_step": p_ms, "frames_per_s": w.B * w.T / (p_ms * 1e-3),
                               "boosted_overhead_pct": 100.0 * (total_ms / args.steps / p_ms - 1.0),
                               # an unboosted decode streams every row once: the whole tensor over the launch time
                               "all_rows_GBs": logits.numel() * logits.element_size() / (p_ms * 1e-3) / 1e9,
                               "all_rows_frac_of_measured_peak": logits.numel() * logits.element_size() / (p_ms * 1e-3) / 1e9 / result["roofline"]["peak"]}
    if not args.no_extras and rank == 0 and w.B >= 64:
        # the same streams in smaller batches (the first 16 / 32 of them): with most SMs free, tb_greedy_decode cuts
        # every stream into segments decoded by several blocks at once (k_greedy_seg); reported beside the headline,
        # not part of it
        small = {}
        for nb_ in (16, 32):
            sb_ = tb.tb_batch_create(w.V, w.vocab.case_class, nb_, arena_bytes=16 << 20, device=local_rank)
            for i in range(nb_):
                tb.tb_batch_bind_stream(sb_, i, graphs[i])
            lg_ = logits[:nb_]
            o_ = tb.tb_greedy_decode(sb_, lg_)
            ran_ = tb.tb_batch_last_greedy_kernel(sb_)
            ms_, _ = timed(lambda: tb.tb_greedy_decode(sb_, lg_, out=o_), max(20, args.steps // 4), args.warmup)
            ms_ /= max(20, args.steps // 4)
            same_ = all(int(o_["counts"][i]) == int(counts[i]) for i in range(nb_))      # (the same decode as in the full batch)
            small[str(nb_)] = {"ms_per_step": ms_, "frames_per_s": nb_ * w.T / (ms_ * 1e-3), "blocks_per_stream": ran_["blocks_per_stream"],
                               "kernel": {tb.TB_KERNEL_PIPELINED: "k_greedy_fast", tb.TB_KERNEL_SEGMENTED: "k_greedy_seg",
                                          tb.TB_KERNEL_GENERAL: "k_decode_general"}[ran_["kernel"]],
                               "same_token_counts_as_in_full_batch": bool(same_)}
            sb_.destroy()
        result["smaller_batches"] = small
    if not args.no_extras and rank == 0 and not args.log_softmax:
        # the same decode with every row log-softmax normalised inside the selection (TB_FLAG_LOG_SOFTMAX): the
        # helpers also leave each row's normaliser; reported beside the headline, not part of it
        base_flags = tb.TB_FLAG_ONE_BLOCK_PER_STREAM if args.one_block_per_stream else 0
        tb.tb_batch_set_flags(batch, base_flags | tb.TB_FLAG_LOG_SOFTMAX)
        on_ = tb.tb_greedy_decode(batch, logits)
        ran_ = tb.tb_batch_last_greedy_kernel(batch)
        n_ms, _ = timed(lambda: tb.tb_greedy_decode(batch, logits, out=on_), max(20, args.steps // 4), args.warmup)
        n_ms /= max(20, args.steps // 4)
        valid_ = torch.arange(out["tokens"].shape[1], device=dev)[None, :] < out["counts"][:, None]
        result["log_softmax"] = {"ms_per_step": n_ms, "frames_per_s": w.B * w.T / (n_ms * 1e-3),
                                 "kernel": {tb.TB_KERNEL_PIPELINED: "k_greedy_fast", tb.TB_KERNEL_SEGMENTED: "k_greedy_seg",
                                            tb.TB_KERNEL_GENERAL: "k_decode_general"}[ran_["kernel"]],
                                 "same_tokens_as_unnormalised": bool(torch.equal(on_["counts"], out["counts"]) and torch.equal(
                                     torch.where(valid_, on_["tokens"], 0), torch.where(valid_, out["tokens"], 0)))}
        tb.tb_batch_set_flags(batch, base_flags)
    if not args.no_extras and rank == 0:
        # end to end through the public call with host buffers: H2D of the logits, decode, D2H of results
        dl = torch.empty_like(logits)
        host_out = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in out.items()}

        def e2e_step():
            dl.copy_(host_logits, non_blocking=True)
            o = tb.tb_greedy_decode(batch, dl, out=out)
            for k in host_out:
                host_out[k].copy_(o[k], non_blocking=True)
            torch.cuda.synchronize()
        n_e2e = max(3, min(args.steps, 5))
        for _ in range(2):
            e2e_step()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            e2e_step()
        e_s = (time.perf_counter() - t0) / n_e2e
        result["e2e"] = {"value": w.B * w.T / e_s, "unit": UNIT,
                         "h2d_bytes_per_step": host_logits.numel() * 2,
                         "d2h_bytes_per_step": int(sum(v.numel() * v.element_size() for v in host_out.values())),
                         "ms_per_step": e_s * 1e3, "steps": n_e2e}
        # the oracle on this machine's host cores, one thread, on a bounded sample
        from oracle import oracle as orc
        n_cpu, passes = w.B, 3
        ograph = [orc.Graph(data["phrases"][i], w.V, case_class=w.vocab.case_class) for i in range(n_cpu)]
        t0 = time.perf_counter()
        for _ in range(passes):
            for i in range(n_cpu):
                orc.greedy_rnnt(ograph[i], data["logits"][i])
        c_s = time.perf_counter() - t0
        result["cpu_baseline"] = {"value": passes * n_cpu * w.T / c_s, "unit": UNIT, "cores": 1, "kind": "oracle",
                                  "sample": f"all {n_cpu} streams, full length, {passes} passes ({c_s:.1f} s)"}
        # the same oracle calls, one stream per call, spread over the machine's cores by a thread pool (the C
        # oracle runs outside the interpreter lock): context for what a multi-core host would reach
        from concurrent.futures import ThreadPoolExecutor
        n_thr = max(1, min(os.cpu_count() or 1, n_cpu))
        t0 = time.perf_counter()
        with ThreadPoolExecutor(n_thr) as pool:
            for _ in range(passes):
                list(pool.map(lambda i: orc.greedy_rnnt(ograph[i], data["logits"][i]), range(n_cpu)))
        m_s = time.perf_counter() - t0
        result["cpu_baseline_all_cores"] = {"value": passes * n_cpu * w.T / m_s, "unit": UNIT, "cores": n_thr,
                                            "kind": "oracle, one stream per call over a thread pool",
                                            "sample": f"all {n_cpu} streams, full length, {passes} passes ({m_s:.1f} s)"}
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(result))


if __name__ == "__main__":
    main()
