"""GPU parity at the full layer sizes of the five synthetic workloads, in the launch configuration
the benchmark times (same calibration batch size; one selection call per block).

For the first and the last block of every model-shaped workload, every row of every layer is
selected on the GPU and by the oracle and compared entry by entry.  The statistics of the first
block are accumulated over ALL calibration tokens on both sides (the last block's over two
batches: its purpose is a second, different set of weights and statistics).  Selections are
compared with the library's own statistics handed to the oracle, which isolates the selection
from the 1e-7 differences of the column sums: N:M masks must then be bit-identical, EWMA masks
may differ only inside the 1e-5 band around the oracle's threshold, in at most 1e-6 of the
entries of a workload; pruned weights must be bit-identical wherever the masks agree.
"""
import numpy as np
import pytest
import torch

from oracle import swiftprune_oracle as so
from paper_2501_16376_b200 import synth
from tests import parity as P

pytestmark = pytest.mark.gpu

BATCH_SEQS = 16          # sequences per sp_calib_accumulate call, as in bench.py
LAST_BLOCK_BATCHES = 2   # calibration batches used for the last block


@pytest.fixture(scope="module")
def sp():
    from paper_2501_16376_b200 import binding
    return binding


def _calibrate(sp, w, block, name, d_in, all_tokens):
    """Statistics of one layer input on the GPU and, from the same bits, by the oracle."""
    ctx = sp.Context(d_in)
    st = so.new_stats(d_in)
    seqs = min(BATCH_SEQS, w.n_seqs)
    batches = w.n_seqs // seqs if all_tokens else max(1, min(LAST_BLOCK_BATCHES, w.n_seqs // seqs))
    for b in range(batches):
        X = synth.gen_activations(w, block, name, d_in, b * seqs, seqs, "cuda")
        ctx.sp_calib_accumulate(X)
        so.colsq_accumulate(st, P.bits(X), P.odtype(X), threads=so.max_threads())
        del X
    colsq, S, factor, ntok = ctx.sp_get_stats()
    assert ntok == st.n_tokens == batches * seqs * w.seq_len
    assert P.rel_err(colsq.numpy(), st.colsq) <= P.SCORE_RTOL
    assert abs(S - st.S) <= P.SCORE_RTOL * st.S
    assert P.rel_err(factor.numpy(), st.channel_factor32()) <= P.SCORE_RTOL
    return ctx, so.Stats(colsq.numpy().copy(), ntok)


def _compare_layer(W, mask, out, sel, n, nm):
    """Entry-by-entry comparison of one layer; returns (flips, entries, achieved sparsity)."""
    got = so.unpack_mask(P.mask_np(mask), n)
    want = sel.keep_bool(n)
    diff = got != want
    flips = int(diff.sum())
    if nm is not None:
        assert flips == 0, "N:M mask differs in %d entries" % flips
        assert (got.reshape(got.shape[0], n // nm[1], nm[1]).sum(-1) == nm[0]).all()
    else:
        assert got[:, 0].all()                                   # column 0 survives
        if flips:
            L = sel.L[diff].astype(np.float64)
            thr = sel.thr[diff].astype(np.float64)
            band = np.abs(L - thr) <= P.BAND_RTOL * np.maximum(np.abs(L), np.abs(thr))
            assert band.all(), "mask differs outside the threshold band"
    words = P.mask_np(mask)
    if n % 32:
        assert (words[:, -1] >> np.uint32(n % 32)).max(initial=0) == 0
    out_bits = P.bits(out)
    w_bits = P.bits(W)
    assert np.array_equal(out_bits, np.where(got, w_bits, 0))    # kept exact, pruned +0
    if flips:
        assert np.array_equal(out_bits[~diff], sel.W_out[~diff])
    else:
        assert np.array_equal(out_bits, sel.W_out)
    return flips, diff.size, 1.0 - float(got.mean())


def _run_workload(sp, name, modes):
    w = synth.WORKLOADS[name]
    threads = so.max_threads()
    flips = entries = 0
    report = []
    for block in sorted({0, w.blocks - 1}):
        ctxs = {}
        try:
            for input_name, d_in in w.input_widths().items():
                ctxs[input_name] = _calibrate(sp, w, block, input_name, d_in, all_tokens=block == 0)
            # one call per block over all its layers, as bench.py's pass makes it
            Ws = [synth.gen_weight(w, block, l, "cuda") for l in w.layers]
            owners = [ctxs[l.input][0] for l in w.layers]
            for mode in modes:
                nm = mode if isinstance(mode, tuple) else None
                if nm is not None:
                    masks, outs = sp.sp_select_nm_multi(owners, Ws, nm[0], nm[1])
                else:
                    masks, outs = sp.sp_select_unstructured_multi(owners, Ws, mode)
                for layer, W, mask, out in zip(w.layers, Ws, masks, outs):
                    st = ctxs[layer.input][1]
                    if nm is not None:
                        sel = so.select_nm(P.bits(W), P.odtype(W), st, nm[0], nm[1], threads=threads)
                    else:
                        sel = so.select_unstructured(P.bits(W), P.odtype(W), st, mode,
                                                     want_trace=True, threads=threads)
                    f, e, achieved = _compare_layer(W, mask, out, sel, layer.d_in, nm)
                    flips += f
                    entries += e
                    report.append((block, layer.name, mode, round(achieved, 4)))
                    del sel
                del masks, outs
            del Ws
        finally:
            for ctx, _ in ctxs.values():
                ctx.close()
    P.FLIP_TALLY["flips"] += flips
    P.FLIP_TALLY["entries"] += entries
    P.FLIP_TALLY["cases"] += 1
    print(name, "flips", flips, "of", entries, "entries")
    assert flips <= P.FLIP_FRACTION * entries, "%d flips in %d entries" % (flips, entries)
    return report


def test_single_layer_512_every_entry(sp):
    w = synth.WORKLOADS["single-512"]
    layer = w.layers[0]
    W = synth.gen_weight(w, 0, layer, "cuda")
    X = synth.gen_activations(w, 0, layer.input, layer.d_in, 0, w.n_seqs, "cuda")
    with sp.Context(layer.d_in) as ctx:
        ctx.sp_calib_accumulate(X)
        mask, out = ctx.sp_select_unstructured(W, 0.5)
    st = P.oracle_stats([X], layer.d_in)          # the oracle's own statistics: the full path
    sel = so.select_unstructured(P.bits(W), so.F16, st, 0.5, want_trace=True)
    flips = P.check_selection(mask, out, W, sel, P.ewma_allowed_flips(sel))
    assert flips <= 1
    achieved = 1.0 - sel.keep_bool(layer.d_in).mean()
    assert 0.45 < achieved < 0.60


def test_pythia_410m_layers(sp):
    _run_workload(sp, "pythia-410m", [0.5])


def test_llama2_7b_layers_2_4(sp):
    _run_workload(sp, "llama2-7b", [(2, 4)])


def test_llama3_8b_layers_sparsity_sweep(sp):
    report = _run_workload(sp, "llama3-8b", [0.5, 0.6, 0.7, 0.8])
    # the rule only approximates the nominal ratio; it must at least be monotone in it
    by_layer = {}
    for block, layer, mode, achieved in report:
        by_layer.setdefault((block, layer), []).append(achieved)
    for vals in by_layer.values():
        assert vals == sorted(vals)


def test_llama2_13b_layers_2_4_and_4_8(sp):
    _run_workload(sp, "llama2-13b", [(2, 4), (4, 8)])


def test_repeated_nm_pruning_is_idempotent(sp):
    # the repeated-prune loop: pruning the already pruned matrix again changes nothing
    w = synth.WORKLOADS["llama2-13b"]
    layer = w.layers[0]
    W = synth.gen_weight(w, 0, layer, "cuda")
    X = synth.gen_activations(w, 0, layer.input, layer.d_in, 0, 2, "cuda")
    with sp.Context(layer.d_in) as ctx:
        ctx.sp_calib_accumulate(X)
        for N, M in ((2, 4), (4, 8)):
            mask, out = ctx.sp_select_nm(W, N, M)
            for _ in range(3):
                mask2, out2 = ctx.sp_select_nm(out, N, M)
                assert torch.equal(mask, mask2)
                assert torch.equal(out.view(torch.int16), out2.view(torch.int16))
