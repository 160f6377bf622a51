#!/usr/bin/env python
"""Benchmark of the SwiftPrune pruning pass on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload llama2-7b] [--batch-seqs 16]

A step is one pass of the whole hot path over one synthetic model: for every block and every
distinct layer input, the calibration statistics are accumulated over all calibration tokens
(sp_calib_accumulate in batches), finalised, and every layer reading that input is selected
and written back (sp_select_nm / sp_select_unstructured).  The metric is pruned weights per
second (all linear-layer weights of the model / step time).  With N > 1 ranks (torchrun) every
rank prunes its own model of the same shape (independent problems, no data-path collective):
weak scaling; the value is the total over ranks divided by the slowest rank's time.

--impl reference times the CPU oracle (the plain restatement of the paper's algorithm) on the
host cores on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "pruned_weights_per_sec"
UNIT = "weights/s"
# fused select + write-back: 2 B read + 2 B write per weight + 1 bit of mask
SELECT_BYTES_PER_WEIGHT = 4.125
CALIB_BYTES_PER_ELEMENT = 2.0


# DRAM bytes (read + write) per launch from ncu captures of the kernels as committed
# (summarised under profiles/), for the launch shapes of the default configuration
# (32768-token calibration batches; selection launches per block or grouped per layer input).
# Keys: calibration -> d_in; selection -> (total rows of the launch, d_in), or
# ("block", workload) for one launch over all layers of a block.  Shapes that were
# not captured, and kernels changed since, report null.
NCU_CALIB_TRAFFIC = {4096: 272.0e6, 11008: 725.0e6}
NCU_SELECT_TRAFFIC = {
    "select_nm_stream_kernel": {("block", "llama2-7b"): 782.4e6,
                                (12288, 4096): 154.9e6, (4096, 4096): 33.6e6,
                                (22016, 4096): 314.6e6, (4096, 11008): 127.7e6},
    "ewma_pair_scan_kernel": {("block", "llama3-8b"): 845.2e6,
                              (6144, 4096): 54.2e6, (4096, 4096): 33.6e6,
                              (28672, 4096): 426.1e6, (4096, 14336): 184.8e6},
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2-7b")
    ap.add_argument("--select-launch", default="auto", choices=["auto", "block", "input", "layer"],
                    help="selection calls of the pass: one per block, one per layer input "
                         "(grouped), or one per layer; auto = block")
    ap.add_argument("--calib-launch", default="auto", choices=["auto", "input", "shared"],
                    help="accumulate launches: one per layer input and batch, or shared by the "
                         "inputs of a block (sp_calib_accumulate_multi); auto = shared when a "
                         "batch of the widest input is at most 64 MiB")
    ap.add_argument("--batch-seqs", type=int, default=16,
                    help="calibration sequences per sp_calib_accumulate call")
    ap.add_argument("--e2e-steps", type=int, default=1)
    ap.add_argument("--blocks", type=int, default=0,
                    help="profiling aid: prune only the first BLOCKS blocks (0 = the whole model)")
    ap.add_argument("--seqs", type=int, default=0,
                    help="profiling aid: calibration sequences (0 = the workload's own number); "
                         "keeps the resident activations to a few GB for an ncu capture")
    ap.add_argument("--mode-index", type=int, default=0,
                    help="which of the workload's sparsities / N:M patterns to run")
    ap.add_argument("--graph", action="store_true",
                    help="replay the whole-model pass as one CUDA graph in the timed region "
                         "(for launch-bound small models)")
    ap.add_argument("--split", default="models", choices=["models", "blocks", "tokens"],
                    help="with N > 1 ranks: every rank prunes its own model (weak scaling, the "
                         "default), or the ranks share ONE model by blocks (no exchange) or by "
                         "calibration tokens and rows (one small all-reduce per layer input)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--ewma-blocks", type=int, default=6,
                    help="blocks of LLaMA-3-8B-shaped layers the EWMA selection kernel is timed "
                         "on, alone, after the step (0 = skip)")
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_uuid: str | None):
        self.samples = []
        self.proc = None
        self.uuid = gpu_uuid

    def start(self):
        cmd = ["nvidia-smi", "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
               "-lms", "100"]
        if self.uuid:
            cmd += ["-i", self.uuid]
        try:
            self.proc = subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.DEVNULL,
                                         text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            parts = [p.strip() for p in s.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def mode_args(w):
    if w.mode == "nm":
        return [tuple(p) for p in w.patterns]
    return list(w.sparsities)


# ---------------------------------------------------------------------------- CPU oracle legs

def oracle_sample(w, threads: int):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload: the selection of
    every layer of block 0 at full size, and the calibration statistics of block 0's four
    inputs over a subset of the sequences (scaled to all sequences).  Returns a dict with the
    extrapolated weights/s for one whole-model pass."""
    import torch
    from oracle import swiftprune_oracle as so
    from paper_2501_16376_b200 import synth

    odt = so.F16 if w.dtype == "f16" else so.BF16
    sample_seqs = max(1, min(w.n_seqs, 2))
    t_calib = 0.0
    stats = {}
    for name, d_in in w.input_widths().items():
        X = synth.gen_activations(w, 0, name, d_in, 0, sample_seqs, "cpu")
        Xb = synth.bits_of(X)
        st = so.new_stats(d_in)
        t0 = time.perf_counter()
        so.colsq_accumulate(st, Xb, odt, threads=threads)
        t_calib += time.perf_counter() - t0
        stats[name] = st
    t_calib_full = t_calib * (w.n_seqs / sample_seqs)
    arg = mode_args(w)[0]
    t_select = 0.0
    weights = 0
    for layer in w.layers:
        W = synth.bits_of(synth.gen_weight(w, 0, layer, "cpu"))
        t0 = time.perf_counter()
        if w.mode == "nm":
            so.select_nm(W, odt, stats[layer.input], arg[0], arg[1], threads=threads)
        else:
            so.select_unstructured(W, odt, stats[layer.input], arg, threads=threads)
        t_select += time.perf_counter() - t0
        weights += layer.d_out * layer.d_in
    t_block = t_calib_full + t_select
    return {
        "value": weights / t_block,
        "unit": UNIT,
        "cores": threads,
        "kind": "oracle",
        "sample": ("block 0 of %d: selection of all %d layers at full size (%.2f s) + statistics "
                   "of its %d inputs over %d of %d sequences (%.2f s, scaled x%d)"
                   % (w.blocks, len(w.layers), t_select, len(stats), sample_seqs, w.n_seqs,
                      t_calib, w.n_seqs // sample_seqs)),
        "block_seconds": t_block,
        "whole_model_seconds": t_block * w.blocks,
    }


def reference_arm(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from oracle import swiftprune_oracle as so
    from paper_2501_16376_b200 import synth
    w = synth.WORKLOADS[args.workload]
    threads = so.max_threads()
    so.build()
    for _ in range(min(args.warmup, 1)):
        oracle_sample(synth.scaled(w, blocks=1, n_seqs=2, seq_len=64, shrink=8), threads)
    t0 = time.perf_counter()
    results = [oracle_sample(w, threads) for _ in range(max(1, args.steps))]
    wall = time.perf_counter() - t0
    best = max(results, key=lambda r: r["value"])
    mean_block = sum(r["block_seconds"] for r in results) / len(results)
    value = w.weights_per_block() / mean_block
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": args.gpus, "steps": len(results), "warmup": min(args.warmup, 1),
        # what was run and timed: one bounded sample per step (wall time incl. input generation)
        "ms_per_step": wall / len(results) * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "mode": w.mode, "mode_arg": str(mode_args(w)[0]),
                   "note": "CPU oracle on host cores; a step is a bounded sample of the workload, "
                           "not a whole-model pass"},
        "extrapolated": {
            "what": "value = weights of one block / oracle seconds for one block, where the "
                    "statistics were timed on a subset of the sequences and scaled up",
            "oracle_seconds_per_block": mean_block,
            "whole_model_seconds": mean_block * w.blocks,
            "sample": best["sample"],
        },
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": best["sample"]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ---------------------------------------------------------------------------- GPU arm

# DRAM bytes per launch of the EWMA selection kernel (ncu, see profiles/): (rows, d_in) -> bytes
NCU_EWMA_TRAFFIC = NCU_SELECT_TRAFFIC["ewma_pair_scan_kernel"]


def ewma_block(device, peak, peak_kind, blocks=4):
    """The paper's own selection rule (Algorithm 1, EWMA running threshold) timed alone on the
    LLaMA-3-8B-shaped layers (bf16, unstructured 50 %): every launch group of a block (q/k/v;
    o; gate/up; down) back to back over `blocks` blocks' distinct weights, outputs and masks
    (more than L2 per group), statistics in place; and every layer on its own the same way."""
    import torch
    from paper_2501_16376_b200 import binding as sp
    from paper_2501_16376_b200 import pipeline, synth

    w0 = synth.WORKLOADS["llama3-8b"]
    w = synth.Workload(**{**w0.__dict__, "blocks": blocks, "n_seqs": 2})
    mb = pipeline.allocate_model(w, device)
    for name in w.input_widths():
        pipeline.calibrate_input(mb.ctxs[name], mb.acts[name], 4096)
        mb.ctxs[name].sp_score(None)
    torch.cuda.synchronize()
    sparsity = w.sparsities[0]

    def timed(fn, reps=3):
        # the launches of all blocks replayed as one CUDA graph: the host's enqueue rate (tens of
        # microseconds per call from Python) would otherwise set the pace of 10-50 us kernels
        for b in range(blocks):
            fn(b)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for b in range(blocks):
                fn(b)
        graph.replay()
        torch.cuda.synchronize()
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        best = None
        for _ in range(reps):
            t0.record()
            graph.replay()
            t1.record()
            torch.cuda.synchronize()
            ms = t0.elapsed_time(t1) / blocks
            best = ms if best is None else min(best, ms)
        return best

    def entry(label, rows, d_in, ms, launches):
        gbs = SELECT_BYTES_PER_WEIGHT * rows * d_in / (ms * 1e-3) / 1e9
        return {"launch": label, "rows": rows, "d_in": d_in, "kernel_launches": launches,
                "avg_ms": ms, "achieved": gbs, "frac": gbs / peak, "frac_of_8TBs": gbs / 8000.0,
                "traffic": NCU_EWMA_TRAFFIC.get((rows, d_in))}

    groups, singles = [], []
    total_bytes = total_ms = 0.0
    for name, d_in in w.input_widths().items():
        idx = [li for li, l in enumerate(w.layers) if l.input == name]
        ctx = mb.ctxs[name]
        rows = sum(w.layers[li].d_out for li in idx)

        def run_group(b, idx=idx, ctx=ctx):
            if len(idx) > 1:
                ctx.sp_select_unstructured_group([mb.weights[b][li] for li in idx], sparsity,
                                                 masks=[mb.masks[b][li] for li in idx],
                                                 W_outs=[mb.outputs[b][li] for li in idx])
            else:
                li = idx[0]
                ctx.sp_select_unstructured(mb.weights[b][li], sparsity, mask=mb.masks[b][li],
                                           W_out=mb.outputs[b][li])
        ms = timed(run_group)
        groups.append(entry("+".join(w.layers[li].name for li in idx), rows, d_in, ms, 1))
        total_bytes += SELECT_BYTES_PER_WEIGHT * rows * d_in
        total_ms += ms
        if len(idx) > 1:
            for li in idx:
                def run_one(b, li=li, ctx=ctx):
                    ctx.sp_select_unstructured(mb.weights[b][li], sparsity, mask=mb.masks[b][li],
                                               W_out=mb.outputs[b][li])
                singles.append(entry(w.layers[li].name, w.layers[li].d_out, d_in,
                                     timed(run_one), 1))
    # all seven layers of a block in ONE launch (sp_select_unstructured_multi): what the pass uses
    block_ms = timed(lambda b: pipeline.select_block(mb, b, sparsity))
    mb.close()
    del mb
    torch.cuda.empty_cache()
    gbs = total_bytes / (block_ms * 1e-3) / 1e9
    grouped_gbs = total_bytes / (total_ms * 1e-3) / 1e9
    return {
        "kernel": "ewma_pair_scan_kernel", "workload": "llama3-8b layer shapes, bf16, "
        "unstructured %.0f %%, default mode (drift gate on)" % (sparsity * 100),
        "bound": "hbm", "unit": "GB/s", "peak": peak, "peak_kind": peak_kind,
        "achieved": gbs, "frac": gbs / peak, "frac_of_8TBs": gbs / 8000.0,
        "ms_per_block": block_ms, "blocks_timed": blocks, "kernel_launches_per_block": 1,
        "traffic": NCU_EWMA_TRAFFIC.get(("block", "llama3-8b")),
        "one_launch_per_layer_input": {"ms_per_block": total_ms, "achieved": grouped_gbs,
                                       "frac": grouped_gbs / peak,
                                       "frac_of_8TBs": grouped_gbs / 8000.0,
                                       "per_launch": groups},
        "single_layer_calls": singles,
        "note": "selection launches only: the calls of %d blocks on distinct buffers replayed as "
                "one CUDA graph, CUDA events around the replay, best of 3; achieved = 4.125 B per "
                "weight / time; the headline figure is one launch per block (all seven layers, "
                "each with its own input's statistics), the breakdown below it one launch per "
                "layer input and one per layer" % blocks,
    }

def gpu_arm(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library has no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    from paper_2501_16376_b200 import binding as sp
    from paper_2501_16376_b200 import pipeline, synth
    from paper_2501_16376_b200 import sharding

    w = synth.WORKLOADS[args.workload]
    if args.blocks > 0:
        w = synth.Workload(**{**w.__dict__, "blocks": min(args.blocks, w.blocks)})
    if args.seqs > 0:
        w = synth.Workload(**{**w.__dict__, "n_seqs": min(args.seqs, w.n_seqs)})
    arg = mode_args(w)[args.mode_index]
    batch_tokens = args.batch_seqs * w.seq_len
    # weak scaling: rank r prunes its own model (seed offset r); with --split blocks / tokens
    # all ranks hold the same model and share its work
    shared = args.split != "models"
    mb = pipeline.allocate_model(
        w, device, model_seed_offset=0 if shared else sharding.unit_of_rank(rank, world))
    torch.cuda.synchronize()

    select_launch = args.select_launch
    if select_launch == "auto":
        select_launch = "block"
    if select_launch != "block" and shared:
        raise SystemExit("--split passes make one selection call per block")
    how = {"grouped": select_launch != "layer", "per_block": select_launch == "block"}
    if args.calib_launch != "auto":
        if args.calib_launch == "shared" and select_launch != "block":
            raise SystemExit("--calib-launch shared needs --select-launch block")
        how["multi_calib"] = args.calib_launch == "shared"

    def one_pass():
        if shared:
            return pipeline.prune_model_split(mb, arg, batch_tokens, rank, world, args.split)
        return pipeline.prune_model(mb, arg, batch_tokens, **how)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        one_pass()
    barrier()

    uuid = None
    try:
        uuid = "GPU-" + str(torch.cuda.get_device_properties(device).uuid)
    except Exception:
        pass
    sampler = ClockSampler(uuid)
    sampler.start()

    phase_events = []
    graph = None
    if args.graph and shared:
        raise SystemExit("--graph replays the single-model pass; it cannot be combined with --split")
    if args.graph:
        graph, counts = pipeline.capture_model_graph(mb, arg, batch_tokens, **how)
        for _ in range(3):
            graph.replay()
    launches_before = sp.sp_launch_count()
    start = torch.cuda.Event(enable_timing=True)
    stop = torch.cuda.Event(enable_timing=True)
    barrier()
    start.record()
    if graph is not None:
        for _ in range(args.steps):
            graph.replay()
    else:
        counts = None
        for _ in range(args.steps):
            counts = one_pass()
    stop.record()
    barrier()
    clocks = sampler.stop()
    elapsed_ms = start.elapsed_time(stop)
    if graph is not None:
        launches = sum(counts.values()) * args.steps
    else:
        launches = sp.sp_launch_count() - launches_before
    # The per-phase breakdown and the per-kernel rates come from instrumented passes after the
    # timed region: the event records between phases would otherwise sit inside it (they keep a
    # kernel from overlapping the tail of its predecessor).
    for _ in range(args.steps):
        pipeline.prune_model(mb, arg, batch_tokens, phase_events, **how)
    torch.cuda.synchronize()

    elapsed_ms = sharding.max_over_ranks(elapsed_ms, world, device)
    total_weights = w.total_weights() * (1 if shared else world)
    value = total_weights * args.steps / (elapsed_ms * 1e-3)

    calib_ms = sum(a.elapsed_time(b) for k, a, b, _ in phase_events if k == "calib")
    select_ms = sum(a.elapsed_time(b) for k, a, b, _ in phase_events if k == "select")
    final_ms = sum(a.elapsed_time(b) for k, a, b, _ in phase_events if k == "finalize")
    x_elements = sum(u for k, _, _, u in phase_events if k == "calib")
    sel_weights = sum(u for k, _, _, u in phase_events if k == "select")
    calib_launches = counts["calib"] * args.steps
    select_launches = counts["select"] * args.steps
    peak, peak_kind = measured_peaks()
    calib_gbs = CALIB_BYTES_PER_ELEMENT * x_elements / (calib_ms * 1e-3) / 1e9
    select_gbs = SELECT_BYTES_PER_WEIGHT * sel_weights / (select_ms * 1e-3) / 1e9
    calib_traffic = None
    widths = list(w.input_widths().values())
    if batch_tokens == 32768 and w.tokens % batch_tokens == 0 and \
            all(d in NCU_CALIB_TRAFFIC for d in widths):
        calib_traffic = sum(NCU_CALIB_TRAFFIC[d] for d in widths) / len(widths)
    sel_kernel = "select_nm_stream_kernel" if w.mode == "nm" else "ewma_pair_scan_kernel"
    sel_traffic = None
    table = NCU_SELECT_TRAFFIC[sel_kernel]
    if select_launch == "block":     # one launch per block
        if w.mode != "nm" or arg == (2, 4):
            sel_traffic = table.get(("block", w.name))
    elif select_launch == "input":   # one grouped launch per layer input: (total rows, d_in)
        shapes = []
        for name, d_in in w.input_widths().items():
            shapes.append((sum(l.d_out for l in w.layers if l.input == name), d_in))
        if all(sh in table for sh in shapes) and (w.mode != "nm" or arg == (2, 4)):
            sel_traffic = sum(table[sh] for sh in shapes) / len(shapes)
    roofline = {
        "kernel": "calib_accumulate_kernel", "bound": "hbm", "achieved": calib_gbs, "peak": peak,
        "peak_kind": peak_kind, "unit": "GB/s", "frac": calib_gbs / peak,
        "frac_of_8TBs": calib_gbs / 8000.0, "traffic": calib_traffic,
        "avg_launch_ms": calib_ms / calib_launches,
        "bytes_per_launch": CALIB_BYTES_PER_ELEMENT * x_elements / calib_launches,
        "note": "from instrumented passes run after the timed region; events bracket the "
                "back-to-back accumulate launches of one layer input; the peak is a measured "
                "read+write copy rate, which a read-only kernel can exceed (frac > 1): "
                "frac_of_8TBs is the fraction of the nominal HBM bandwidth",
    }
    roofline_select = {
        "kernel": sel_kernel,
        "bound": "hbm", "achieved": select_gbs, "peak": peak, "peak_kind": peak_kind,
        "unit": "GB/s", "frac": select_gbs / peak, "frac_of_8TBs": select_gbs / 8000.0,
        "traffic": sel_traffic, "avg_launch_ms": select_ms / select_launches,
        "bytes_per_launch": SELECT_BYTES_PER_WEIGHT * sel_weights / select_launches,
        "weights_per_sec": sel_weights / (select_ms * 1e-3),
        "select_launch": select_launch,
        "note": "from instrumented passes run after the timed region; events bracket the "
                "selection launch(es) of one %s; ncu traffic counts DRAM bytes while the "
                "kernel runs (part of the output is still in L2 when it ends)" % (
                    "block" if select_launch == "block" else "layer input"),
    }

    # The same select kernel timed alone on the largest layer shape: one launch per block over
    # every block's own weights / outputs (distinct buffers, far more than L2), statistics in
    # place, the sequence replayed as one CUDA graph so that the host's enqueue rate does not
    # set the pace.
    li = max(range(len(w.layers)), key=lambda i: w.layers[i].d_out * w.layers[i].d_in)
    big = w.layers[li]
    if w.blocks * big.d_out * big.d_in * 4 > 256e6:
        ctx_big = mb.ctxs[big.input]

        def big_layer_launches():
            for b in range(w.blocks):
                pipeline.select_layer(ctx_big, w, mb.weights[b][li], mb.masks[b][li],
                                      mb.outputs[b][li], arg)
        big_layer_launches()
        torch.cuda.synchronize()
        alone_graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(alone_graph):
            big_layer_launches()
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        alone_ms = None
        for rep in range(3):   # the first repetition warms up
            t0.record()
            alone_graph.replay()
            t1.record()
            torch.cuda.synchronize()
            if rep:
                ms = t0.elapsed_time(t1) / w.blocks
                alone_ms = ms if alone_ms is None else min(alone_ms, ms)
        del alone_graph
        alone_gbs = SELECT_BYTES_PER_WEIGHT * big.d_out * big.d_in / (alone_ms * 1e-3) / 1e9
        roofline_select["alone"] = {
            "layer": "%dx%d" % (big.d_out, big.d_in), "launches": w.blocks,
            "avg_launch_ms": alone_ms, "achieved": alone_gbs, "frac": alone_gbs / peak,
            "frac_of_8TBs": alone_gbs / 8000.0,
            "note": "select launches of this one layer only, back to back over all blocks as one "
                    "CUDA graph (no calibration traffic in between, so the SM clock is not held "
                    "down by the power cap)",
        }

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": elapsed_ms / args.steps,
        "higher_is_better": True, "scaling": "strong" if shared else "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "weights_dtype": w.dtype, "mode": w.mode,
                   "mode_arg": str(arg), "blocks": w.blocks, "total_weights": w.total_weights(),
                   "calib_tokens": w.tokens, "batch_tokens": batch_tokens,
                   "l2": "inputs larger than L2: weights, masks and outputs are touched once per "
                         "step; the activation buffers of block 0 (%.1f GB) are re-read for "
                         "every block, with at least %.1f GB of other traffic between two "
                         "reads of the same buffer" % (
                             sum(x.numel() * 2 for x in mb.acts.values()) / 1e9,
                             min(x.numel() * 2 for x in mb.acts.values()) / 1e9),
                   "launch": "cuda graph replay" if graph is not None else "stream launches",
                   "calib_launch": ("one per layer input and batch" if counts["calib"] ==
                                    w.blocks * len(w.input_widths()) * -(-w.tokens // batch_tokens)
                                    or shared else "shared by the inputs of a block"),
                   "calib_flags": "SP_CALIB_X_COMPLETE (the activations are resident and complete "
                                  "long before the step starts)",
                   "parallelism": ("single GPU" if world == 1 else
                                   "independent models per rank" if not shared else
                                   "one model, blocks split over ranks (no exchange)"
                                   if args.split == "blocks" else
                                   "one model, calibration tokens and rows split over ranks "
                                   "(one all-reduce of d_in + 1 doubles per layer input)")},
        "whole_model_prune_s": {"calib": calib_ms / args.steps * 1e-3,
                                "finalize": final_ms / args.steps * 1e-3,
                                "select_apply": select_ms / args.steps * 1e-3,
                                "total": elapsed_ms / args.steps * 1e-3},
        "phase_note": "calib / finalize / select_apply are event brackets from instrumented passes "
                      "run after the timed region (the brackets stop kernels from overlapping "
                      "their predecessors' tails); total is the timed region",
        "roofline": roofline, "roofline_select": roofline_select,
        "ewma": (ewma_block(device, peak, peak_kind, args.ewma_blocks)
                 if args.ewma_blocks > 0 and world == 1 else None),
        "clocks": clocks, "gpu_launches": int(launches),
    }

    # End to end: the same pass with every input and output in pinned HOST memory, through the
    # library's host-buffer entry points (copies inside the timed region).
    if args.e2e_steps > 0:
        hb = pipeline.allocate_host(mb, batch_tokens)
        pipeline.prune_model_host(
            pipeline.ModelBuffers(synth.Workload(**{**w.__dict__, "blocks": 1}), device,
                                  mb.weights, mb.outputs, mb.masks, mb.acts, mb.ctxs),
            hb, arg)                                           # warm-up: one block
        barrier()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.e2e_steps):
            h2d, d2h = pipeline.prune_model_host(mb, hb, arg)
        e1.record()
        barrier()
        e2e_ms = sharding.max_over_ranks(e0.elapsed_time(e1), world, device)
        line["e2e"] = {"value": total_weights * args.e2e_steps / (e2e_ms * 1e-3), "unit": UNIT,
                       "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                       "ms_per_step": e2e_ms / args.e2e_steps, "steps": args.e2e_steps,
                       "note": "host buffers are pinned; one calibration batch and one block's "
                               "weights are the host-side source for every batch / block"}
        del hb

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import swiftprune_oracle as so
        cb = oracle_sample(w, so.max_threads())
        line["cpu_baseline"] = {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")}
        line["cpu_baseline"]["whole_model_seconds"] = cb["whole_model_seconds"]
        one = oracle_sample(w, 1)                  # the same sample on a single thread
        line["cpu_baseline"]["single_thread_value"] = one["value"]
        line["cpu_baseline"]["single_thread_whole_model_seconds"] = one["whole_model_seconds"]

    mb.close()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line))
    return 0


def main():
    args = parse_args()
    if args.impl == "reference":
        return reference_arm(args)
    return gpu_arm(args)


if __name__ == "__main__":
    sys.exit(main())
