"""Whole-model driver: walks the linear layers of a synthetic model and issues the library's
calls for each (calibration batches -> selection fused with write-back).  Pure call sequencing
and buffer bookkeeping; all arithmetic happens inside the CUDA library.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import torch

from . import binding as sp
from . import synth


@dataclass
class ModelBuffers:
    """Device-resident tensors of one synthetic model (one rank's unit of work)."""
    workload: synth.Workload
    device: torch.device
    weights: list = field(default_factory=list)   # [block][layer] -> W
    outputs: list = field(default_factory=list)   # [block][layer] -> W_out
    masks: list = field(default_factory=list)     # [block][layer] -> mask
    acts: dict = field(default_factory=dict)      # input name -> X [tokens, d_in] (shared by blocks)
    ctxs: dict = field(default_factory=dict)      # input name -> Context

    def close(self):
        for c in self.ctxs.values():
            c.close()
        self.ctxs.clear()


def allocate_model(w: synth.Workload, device, model_seed_offset: int = 0,
                   distinct_acts: bool = True) -> ModelBuffers:
    """Generates all weights of the workload and one set of calibration activations (the
    activations of block 0, reused for every block: 128 x 2048 tokens for every block of a
    7B-shaped model would not fit in device memory at once)."""
    device = torch.device(device)
    wl = w if model_seed_offset == 0 else synth.Workload(
        **{**w.__dict__, "seed": w.seed + model_seed_offset})
    mb = ModelBuffers(wl, device)
    for b in range(wl.blocks):
        ws, outs, ms = [], [], []
        for layer in wl.layers:
            W = synth.gen_weight(wl, b, layer, device)
            ws.append(W)
            outs.append(torch.empty_like(W))
            ms.append(torch.empty(layer.d_out, (layer.d_in + 31) // 32, dtype=torch.int32,
                                  device=device))
        mb.weights.append(ws)
        mb.outputs.append(outs)
        mb.masks.append(ms)
    by_width = {}
    for name, d_in in wl.input_widths().items():
        if not distinct_acts and d_in in by_width:
            mb.acts[name] = by_width[d_in]
        else:
            X = torch.empty(wl.tokens, d_in, dtype=wl.torch_dtype, device=device)
            step = max(1, min(8, wl.n_seqs))
            for s in range(0, wl.n_seqs, step):
                k = min(step, wl.n_seqs - s)
                synth.gen_activations(wl, 0, name, d_in, s, k, device,
                                      out=X[s * wl.seq_len:(s + k) * wl.seq_len])
            mb.acts[name] = X
            by_width[d_in] = X
        mb.ctxs[name] = sp.Context(d_in, device.index if device.index is not None
                                   else torch.cuda.current_device())
    return mb


def calibrate_input(ctx: sp.Context, X: torch.Tensor, batch_tokens: int, stream=None,
                    x_complete: bool = False) -> int:
    """Streams X through sp_calib_accumulate in batches; returns the number of launches.
    x_complete: the activations were complete before the previous operation on the stream began
    (true for the resident synthetic activations of ModelBuffers)."""
    ctx.sp_calib_reset(stream)
    T = X.shape[0]
    launches = 0
    for t0 in range(0, T, batch_tokens):
        ctx.sp_calib_accumulate(X[t0:min(T, t0 + batch_tokens)], stream, x_complete)
        launches += 1
    return launches


def select_layer(ctx: sp.Context, w: synth.Workload, W, mask, W_out, mode_arg, stream=None):
    """One selection call: mode_arg is a sparsity (unstructured) or an (N, M) pair."""
    if w.mode == "nm":
        N, M = mode_arg
        ctx.sp_select_nm(W, N, M, mask=mask, W_out=W_out, stream=stream)
    else:
        ctx.sp_select_unstructured(W, mode_arg, mask=mask, W_out=W_out, stream=stream)


def select_group(ctx: sp.Context, w: synth.Workload, Ws, masks, W_outs, mode_arg, stream=None):
    """One grouped selection call for layers that read the same input."""
    if w.mode == "nm":
        N, M = mode_arg
        ctx.sp_select_nm_group(Ws, N, M, masks=masks, W_outs=W_outs, stream=stream)
    else:
        ctx.sp_select_unstructured_group(Ws, mode_arg, masks=masks, W_outs=W_outs, stream=stream)


def select_block(mb: ModelBuffers, b: int, mode_arg, stream=None):
    """Every layer of block b in one call, each layer with the statistics of the input it reads
    (sp_select_unstructured_multi / sp_select_nm_multi)."""
    w = mb.workload
    ctxs = [mb.ctxs[layer.input] for layer in w.layers]
    if w.mode == "nm":
        N, M = mode_arg
        sp.sp_select_nm_multi(ctxs, mb.weights[b], N, M, masks=mb.masks[b], W_outs=mb.outputs[b],
                              stream=stream)
    else:
        sp.sp_select_unstructured_multi(ctxs, mb.weights[b], mode_arg, masks=mb.masks[b],
                                        W_outs=mb.outputs[b], stream=stream)


#: up to this many bytes per accumulate launch, the inputs of a block share their launches
MULTI_CALIB_BYTES = 64 << 20


def calibrate_block(mb: ModelBuffers, batch_tokens: int, stream=None) -> int:
    """Statistics of all layer inputs of a block with shared launches: per batch one
    sp_calib_accumulate_multi over the inputs, then one finalisation launch.  Returns the number
    of accumulate launches."""
    names = list(mb.workload.input_widths())
    ctxs = [mb.ctxs[name] for name in names]
    for ctx in ctxs:
        ctx.sp_calib_reset(stream)
    T = mb.workload.tokens
    before = sp.sp_launch_count()
    for t0 in range(0, T, batch_tokens):
        sp.sp_calib_accumulate_multi(ctxs, [mb.acts[name][t0:min(T, t0 + batch_tokens)]
                                            for name in names], stream, True)
    return sp.sp_launch_count() - before


def prune_model(mb: ModelBuffers, mode_arg, batch_tokens: int, phase_events=None, stream=None,
                grouped: bool = True, per_block: bool | None = None,
                multi_calib: bool | None = None):
    """One pass of the whole hot path over the model: for every block and every distinct layer
    input, accumulate the calibration statistics, finalise them, then select + write back every
    layer that reads this input.  phase_events, if given, is a list that receives
    (kind, start_event, end_event, units) tuples: "calib" (units = activation elements, brackets
    the back-to-back accumulate launches of one layer input), "finalize", and "select" (units =
    weights, brackets the back-to-back selection launches of one layer input, or of one block);
    with phase_events the calls are issued strictly phase by phase so that the brackets are
    clean, without it the next input's calibration is enqueued ahead of the current input's
    selections where there are any (same calls, same results).

    Selection calls: per_block (the default) prunes all layers of a block with one call once
    all its inputs are calibrated; otherwise grouped gives the layers that read one input one
    grouped call (one launch when their layouts allow), else every layer gets a call of its
    own.  multi_calib (per-block passes; the default when one input's batch is below
    MULTI_CALIB_BYTES): the inputs of a block share their accumulate launches and their
    finalisation launch.  Returns launch counts."""
    w = mb.workload
    n_calib = n_select = n_final = 0
    if stream is None:
        stream = torch.cuda.current_stream()   # looked up once, not once per call
    if per_block is None:
        per_block = grouped
    if multi_calib is None:
        multi_calib = per_block and len(w.input_widths()) > 1 and \
            batch_tokens * max(w.input_widths().values()) * 2 <= MULTI_CALIB_BYTES
    if multi_calib and not per_block:
        raise ValueError("multi_calib needs per_block")

    def mark():
        e = torch.cuda.Event(enable_timing=True)
        e.record(stream)
        return e

    def select_input(b, name, ctx):
        nonlocal n_select
        idx = [li for li, layer in enumerate(w.layers) if layer.input == name]
        before = sp.sp_launch_count()
        if grouped and len(idx) > 1:
            select_group(ctx, w, [mb.weights[b][li] for li in idx], [mb.masks[b][li] for li in idx],
                         [mb.outputs[b][li] for li in idx], mode_arg, stream)
        else:
            for li in idx:
                select_layer(ctx, w, mb.weights[b][li], mb.masks[b][li], mb.outputs[b][li],
                             mode_arg, stream)
        n_select += sp.sp_launch_count() - before
        return sum(w.layers[li].d_out * w.layers[li].d_in for li in idx)

    if per_block:
        # calibrate + finalise every input of the block (the next input's accumulate launches
        # follow an input's finalisation directly and stream under it), then one selection call
        block_weights = sum(layer.d_out * layer.d_in for layer in w.layers)
        last = mark() if phase_events is not None else None
        all_ctxs = [mb.ctxs[name] for name in w.input_widths()]
        x_elements = sum(mb.acts[name].shape[0] * d_in for name, d_in in w.input_widths().items())
        for b in range(w.blocks):
            if multi_calib:
                n_calib += calibrate_block(mb, batch_tokens, stream)
                e1 = mark() if phase_events is not None else None
                sp.sp_finalize_multi(all_ctxs, stream)
                n_final += 1
                if phase_events is not None:
                    e2 = mark()
                    phase_events.append(("calib", last, e1, x_elements))
                    phase_events.append(("finalize", e1, e2, sum(w.input_widths().values())))
                    last = e2
            for name, d_in in ([] if multi_calib else w.input_widths().items()):
                ctx = mb.ctxs[name]
                n_calib += calibrate_input(ctx, mb.acts[name], batch_tokens, stream, True)
                e1 = mark() if phase_events is not None else None
                ctx.sp_score(None, stream=stream)          # finalisation only
                n_final += 1
                if phase_events is not None:
                    e2 = mark()
                    phase_events.append(("calib", last, e1, mb.acts[name].shape[0] * d_in))
                    phase_events.append(("finalize", e1, e2, d_in))
                    last = e2
            before = sp.sp_launch_count()
            select_block(mb, b, mode_arg, stream)
            n_select += sp.sp_launch_count() - before
            if phase_events is not None:
                e3 = mark()
                phase_events.append(("select", last, e3, block_weights))
                last = e3
        return {"calib": n_calib, "finalize": n_final, "select": n_select}

    if phase_events is None:
        # Plain pass.  The calibration of the next input is enqueued between an input's
        # finalisation and its selections: the accumulate kernel only waits for its predecessor
        # before it writes its partial sums, so it streams its activations while the few CTAs
        # of the finalisation run (inputs of different widths have different contexts; with a
        # single input the order is simply calibrate, finalise, select).
        units = [(b, name) for b in range(w.blocks) for name in w.input_widths()]
        distinct = len(w.input_widths()) > 1
        for i, (b, name) in enumerate(units):
            ctx = mb.ctxs[name]
            if i == 0 or not distinct:
                n_calib += calibrate_input(ctx, mb.acts[name], batch_tokens, stream, True)
            ctx.sp_score(None, stream=stream)          # finalisation only
            n_final += 1
            if distinct and i + 1 < len(units):
                nxt = units[i + 1][1]
                n_calib += calibrate_input(mb.ctxs[nxt], mb.acts[nxt], batch_tokens, stream, True)
            select_input(b, name, ctx)
        return {"calib": n_calib, "finalize": n_final, "select": n_select}

    last = mark()
    for b in range(w.blocks):
        for name, d_in in w.input_widths().items():
            ctx = mb.ctxs[name]
            X = mb.acts[name]
            e0 = last
            n_calib += calibrate_input(ctx, X, batch_tokens, stream, True)
            e1 = mark()
            ctx.sp_score(None, stream=stream)          # finalisation only
            n_final += 1
            e2 = mark()
            phase_events.append(("calib", e0, e1, X.shape[0] * d_in))
            phase_events.append(("finalize", e1, e2, d_in))
            sel_weights = select_input(b, name, ctx)
            last = mark()
            phase_events.append(("select", e2, last, sel_weights))
    return {"calib": n_calib, "finalize": n_final, "select": n_select}


def prune_model_split(mb: ModelBuffers, mode_arg, batch_tokens: int, rank: int, world: int,
                      split: str, stream=None):
    """One pass over ONE model shared by `world` ranks (strong scaling).

    split == "blocks": rank r prunes the blocks sharding.assign_units gives it, on its own; no
    exchange at all.
    split == "tokens": for every block and layer input, rank r accumulates its share of the
    calibration tokens, the ranks sum their column sums of squares with one all-reduce of
    d_in + 1 doubles (sharding.merge_calibration), and rank r then prunes its share of the rows
    of every layer of the block with one call.  Masks and outputs of rows a rank does not own are left
    untouched.  Returns launch counts."""
    from . import sharding
    w = mb.workload
    n_calib = n_final = n_select = 0
    if stream is None:
        stream = torch.cuda.current_stream()
    blocks = sharding.assign_units(w.blocks, world, rank) if split == "blocks" else range(w.blocks)
    for b in blocks:
        for name, d_in in w.input_widths().items():
            ctx = mb.ctxs[name]
            X = mb.acts[name]
            if split == "tokens":
                share = sharding.token_share(X.shape[0], world, rank, align=w.seq_len)
                ctx.sp_calib_reset(stream)
                for t0 in range(share.start, share.stop, batch_tokens):
                    ctx.sp_calib_accumulate(X[t0:min(share.stop, t0 + batch_tokens)], stream, True)
                    n_calib += 1
                sharding.merge_calibration(ctx, world, mb.device, stream)
            else:
                n_calib += calibrate_input(ctx, X, batch_tokens, stream, True)
            ctx.sp_score(None, stream=stream)
            n_final += 1
        # this rank's rows of every layer of the block, in one call
        ctxs, Ws, masks, outs = [], [], [], []
        for li, layer in enumerate(w.layers):
            rows = (sharding.row_share(layer.d_out, world, rank)
                    if split == "tokens" else range(layer.d_out))
            if len(rows) == 0:
                continue
            ctxs.append(mb.ctxs[layer.input])
            Ws.append(mb.weights[b][li][rows.start:rows.stop])
            masks.append(mb.masks[b][li][rows.start:rows.stop])
            outs.append(mb.outputs[b][li][rows.start:rows.stop])
        before = sp.sp_launch_count()
        if Ws and w.mode == "nm":
            sp.sp_select_nm_multi(ctxs, Ws, mode_arg[0], mode_arg[1], masks=masks, W_outs=outs,
                                  stream=stream)
        elif Ws:
            sp.sp_select_unstructured_multi(ctxs, Ws, mode_arg, masks=masks, W_outs=outs,
                                            stream=stream)
        n_select += sp.sp_launch_count() - before
    return {"calib": n_calib, "finalize": n_final, "select": n_select}


def capture_model_graph(mb: ModelBuffers, mode_arg, batch_tokens: int, **how):
    """Captures one whole-model pass into a CUDA graph (for models whose layers are so small
    that the pass is bound by launch overhead).  The library's calls only enqueue kernels on the
    current stream, so they can be captured as they are.  Returns (graph, launch counts)."""
    prune_model(mb, mode_arg, batch_tokens, **how)   # everything allocated and finalised once
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        counts = prune_model(mb, mode_arg, batch_tokens, **how)
    return graph, counts


@dataclass
class HostBuffers:
    """Pinned host copies for the end-to-end path: one calibration batch per layer input and the
    weights / outputs / masks of one block (reused for every block: the bytes that cross the
    bus per step are those of the whole model)."""
    x_batch: dict = field(default_factory=dict)    # input name -> [batch_tokens, d_in]
    weights: list = field(default_factory=list)    # per layer of a block
    outputs: list = field(default_factory=list)
    masks: list = field(default_factory=list)


def allocate_host(mb: ModelBuffers, batch_tokens: int) -> HostBuffers:
    hb = HostBuffers()
    w = mb.workload
    for name, d_in in w.input_widths().items():
        hb.x_batch[name] = mb.acts[name][:batch_tokens].cpu().pin_memory()
    for li, layer in enumerate(w.layers):
        hb.weights.append(mb.weights[0][li].cpu().pin_memory())
        hb.outputs.append(torch.empty(layer.d_out, layer.d_in, dtype=w.torch_dtype).pin_memory())
        hb.masks.append(torch.empty(layer.d_out, (layer.d_in + 31) // 32,
                                    dtype=torch.int32).pin_memory())
    return hb


def prune_model_host(mb: ModelBuffers, hb: HostBuffers, mode_arg, stream=None):
    """One pass of the whole hot path with every input and output in host memory, through the
    host-buffer entry points.  Returns (h2d_bytes, d2h_bytes) that crossed the bus."""
    w = mb.workload
    h2d = d2h = 0
    for b in range(w.blocks):
        for name, d_in in w.input_widths().items():
            ctx = mb.ctxs[name]
            ctx.sp_calib_reset(stream)
            xb = hb.x_batch[name]
            for t0 in range(0, w.tokens, xb.shape[0]):
                rows = min(xb.shape[0], w.tokens - t0)
                ctx.sp_calib_accumulate_host(xb[:rows], stream)
                h2d += rows * d_in * 2
            for li, layer in enumerate(w.layers):
                if layer.input != name:
                    continue
                if w.mode == "nm":
                    ctx.sp_select_nm_host(hb.weights[li], mode_arg[0], mode_arg[1], hb.masks[li],
                                          hb.outputs[li], stream)
                else:
                    ctx.sp_select_unstructured_host(hb.weights[li], mode_arg, hb.masks[li],
                                                    hb.outputs[li], stream)
                h2d += layer.d_out * layer.d_in * 2
                d2h += layer.d_out * layer.d_in * 2 + hb.masks[li].numel() * 4
    return h2d, d2h
