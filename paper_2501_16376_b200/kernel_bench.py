"""Stand-alone timing of single library calls on one layer shape.

    python -m paper_2501_16376_b200.kernel_bench --call ewma --shape 14336x4096 --dtype bf16
    python -m paper_2501_16376_b200.kernel_bench --call nm --nm 2:4 --shape 11008x4096
    python -m paper_2501_16376_b200.kernel_bench --call calib --shape 32768x4096

The call is repeated over distinct weight / output / mask buffers whose total size exceeds the
L2 cache (so every launch reads from and writes to HBM), the sequence is replayed as one CUDA
graph (the host's enqueue rate does not set the pace) and timed with CUDA events.  One JSON line
per run: microseconds per call, algorithmic GB/s (4.125 B per weight for the fused selections,
3.125 B for the compressed 2:4 form, 2 B per activation element for the statistics), and the
fraction of the measured copy rate when MEASURED_PEAKS.json is present.

Calls: ewma (default mode, drift gate on) | ewma-frozen | ewma-literal | ewma-literal-scan |
ewma-x2 | nm |
compressed24 | calib | search (24 counting passes) | block (all layers of one block of
--workload in one call: sp_select_nm_multi / sp_select_unstructured_multi; --shape is ignored).
--few N limits the number of buffers (for a profiler capture that should see only a handful of
launches).
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import torch

from . import binding as sp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"])
    except Exception:
        return None


def run(call: str, rows: int, cols: int, dtype, nm=(2, 4), reps: int = 5, few: int = 0,
        calib_tokens: int = 4096, stats_scale: float = 0.0):
    dev = torch.device("cuda", torch.cuda.current_device())
    g = torch.Generator(device=dev)
    g.manual_seed(1)
    if call == "calib":
        # rows = tokens per call here; several distinct batches
        nbuf = few or max(3, int(600e6 // (rows * cols * 2)) + 1)
        Xs = [torch.randn(rows, cols, device=dev, generator=g).to(dtype) for _ in range(nbuf)]
        ctx = sp.Context(cols)

        def one(i):
            ctx.sp_calib_accumulate(Xs[i], x_complete=True)
        bytes_per_call = rows * cols * 2.0
    else:
        nbuf = few or max(3, int(600e6 // (rows * cols * 2)) + 1)
        Ws = [(torch.randn(rows, cols, device=dev, generator=g) * 0.02).to(dtype) for _ in range(nbuf)]
        outs = [torch.empty_like(w) for w in Ws]
        masks = [torch.empty(rows, (cols + 31) // 32, dtype=torch.int32, device=dev) for _ in Ws]
        ctx = sp.Context(cols)
        X = torch.randn(calib_tokens, cols, device=dev, generator=g).to(dtype)
        ctx.sp_calib_accumulate(X)
        if stats_scale > 0.0:
            gen = torch.Generator().manual_seed(2)
            ctx.sp_set_stats((1.0 + torch.rand(cols, generator=gen, dtype=torch.float64))
                             * stats_scale, calib_tokens)
        ctx.sp_score(None)
        bytes_per_call = rows * cols * 4.125
        if call.startswith("ewma"):
            mode = {"ewma": sp.SP_S_GATED, "ewma-frozen": sp.SP_S_FROZEN,
                    "ewma-literal": sp.SP_S_LITERAL_W2, "ewma-x2": sp.SP_S_READING_X2,
                    "ewma-literal-scan": sp.SP_S_LITERAL_SCAN}[call]
            prm = sp.EwmaParams(0.125, 0.125, 0.5, mode)

            def one(i):
                ctx.sp_select_unstructured(Ws[i], params=prm, mask=masks[i], W_out=outs[i])
        elif call == "nm":
            def one(i):
                ctx.sp_select_nm(Ws[i], nm[0], nm[1], mask=masks[i], W_out=outs[i])
        elif call == "compressed24":
            vals = [torch.empty(rows, cols // 2, dtype=dtype, device=dev) for _ in Ws]
            metas = [torch.zeros(rows, (cols + 31) // 32, dtype=torch.int32, device=dev) for _ in Ws]
            bytes_per_call = rows * cols * 3.125

            def one(i):
                ctx.sp_select_24_compressed(Ws[i], vals[i], metas[i])
        elif call == "search":
            bytes_per_call = rows * cols * 2.0 * 24

            def one(i):
                ctx.sp_search_la(Ws[i], 0.55, iterations=24)
        else:
            raise SystemExit("unknown call " + call)

    for i in range(nbuf):
        one(i)
    torch.cuda.synchronize()
    if call == "search":            # synchronises inside: cannot be captured; time it plainly
        graph = None
    else:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for i in range(nbuf):
                one(i)
        graph.replay()
        torch.cuda.synchronize()
    best = None
    for _ in range(reps):
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        if graph is not None:
            graph.replay()
        else:
            for i in range(nbuf):
                one(i)
        e1.record()
        torch.cuda.synchronize()
        t = e0.elapsed_time(e1) / nbuf
        best = t if best is None else min(best, t)
    ctx.close()
    gbs = bytes_per_call / (best * 1e-3) / 1e9
    peak = _peak()
    return {"call": call, "rows": rows, "cols": cols, "dtype": str(dtype).replace("torch.", ""),
            "nm": "%d:%d" % nm if call == "nm" else None, "buffers": nbuf,
            "us_per_call": best * 1e3, "algorithmic_GBs": gbs,
            "frac_of_measured_copy_rate": gbs / peak if peak else None,
            "frac_of_8TBs": gbs / 8000.0}


def run_block(workload: str, blocks: int = 6, reps: int = 5):
    """One selection call per block of a synthetic model (every layer with the statistics of the
    input it reads), over `blocks` blocks' distinct buffers, replayed as one CUDA graph."""
    from . import pipeline, synth
    dev = torch.device("cuda", torch.cuda.current_device())
    w0 = synth.WORKLOADS[workload]
    w = synth.Workload(**{**w0.__dict__, "blocks": blocks, "n_seqs": 2})
    mb = pipeline.allocate_model(w, dev)
    for name in w.input_widths():
        pipeline.calibrate_input(mb.ctxs[name], mb.acts[name], 4096)
        mb.ctxs[name].sp_score(None)
    arg = w.patterns[0] if w.mode == "nm" else w.sparsities[0]

    def all_blocks():
        for b in range(blocks):
            pipeline.select_block(mb, b, arg)
    all_blocks()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        all_blocks()
    graph.replay()
    torch.cuda.synchronize()
    best = None
    for _ in range(reps):
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        graph.replay()
        e1.record()
        torch.cuda.synchronize()
        t = e0.elapsed_time(e1) / blocks
        best = t if best is None else min(best, t)
    mb.close()
    weights = sum(l.d_out * l.d_in for l in w.layers)
    gbs = weights * 4.125 / (best * 1e-3) / 1e9
    peak = _peak()
    return {"call": "block", "workload": workload, "mode": w.mode, "mode_arg": str(arg),
            "weights_per_block": weights, "blocks": blocks, "us_per_call": best * 1e3,
            "algorithmic_GBs": gbs, "frac_of_measured_copy_rate": gbs / peak if peak else None,
            "frac_of_8TBs": gbs / 8000.0}


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawTextHelpFormatter)
    ap.add_argument("--call", default="ewma")
    ap.add_argument("--shape", action="append", default=None, help="ROWSxCOLS (repeatable)")
    ap.add_argument("--dtype", default="bf16", choices=["f16", "bf16"])
    ap.add_argument("--nm", default="2:4")
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--few", type=int, default=0)
    ap.add_argument("--stats-scale", type=float, default=0.0,
                    help="replace the calibration statistics by uniform(1,2) * SCALE per channel "
                         "(e.g. 1e-3: S small enough for Algorithm 1's S update to matter)")
    ap.add_argument("--workload", default="llama2-7b", help="model shape for --call block")
    args = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise SystemExit("kernel_bench needs a CUDA device")
    if args.call == "block":
        print(json.dumps(run_block(args.workload, args.few or 6, args.reps)), flush=True)
        return 0
    dtype = torch.float16 if args.dtype == "f16" else torch.bfloat16
    nm = tuple(int(v) for v in args.nm.split(":"))
    for shape in args.shape or ["4096x4096"]:
        rows, cols = (int(v) for v in shape.lower().split("x"))
        print(json.dumps(run(args.call, rows, cols, dtype, nm, args.reps, args.few,
                             stats_scale=args.stats_scale)), flush=True)
    return 0


if __name__ == "__main__":
    sys.exit(main())
