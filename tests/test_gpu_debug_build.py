"""The debug build of the library (index checks compiled in: an out-of-range store is skipped
and recorded, nothing traps) run over ragged, strided, grouped and multi-context cases in a
process of its own:
it must record no violation and give the release build's results."""
import json
import os
import subprocess
import sys

import pytest
import torch

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_SCRIPT = r"""
import json, sys, hashlib
import torch
sys.path.insert(0, %r)
from paper_2501_16376_b200 import binding as sp

def digest(*tensors):
    h = hashlib.sha256()
    for t in tensors:
        h.update(t.detach().cpu().contiguous().view(torch.uint8).numpy().tobytes())
    return h.hexdigest()

g = torch.Generator(device="cuda").manual_seed(3)
out = {}
kept = {}
for n, R, dtype in ((520, 77, torch.float16), (1536, 130, torch.bfloat16), (8704, 9, torch.float16)):
    W = (torch.randn(R, n, device="cuda", generator=g) * 0.02).to(dtype)
    X = torch.randn(700, n, device="cuda", generator=g).to(dtype)
    with sp.Context(n) as ctx:
        ctx.sp_calib_accumulate(X[:300])
        ctx.sp_calib_accumulate(X[300:])
        m1, o1 = ctx.sp_select_unstructured(W, 0.5)
        m2, o2 = ctx.sp_select_nm(W, 2, 4)
        ms, os_ = ctx.sp_select_unstructured_group([W[:40], W[40:]], 0.6)
        mn, on = ctx.sp_select_nm_group([W[:40], W[40:]], 4, 8)
        m3, o3 = ctx.sp_select_unstructured(W, params=sp.EwmaParams(0.125, 0.125, 0.5, sp.SP_S_LITERAL_W2))
        m4, o4 = ctx.sp_select_unstructured(W, params=sp.EwmaParams(0.125, 0.125, 0.5, sp.SP_S_LITERAL_SCAN))
        colsq = ctx.sp_get_stats()[0]
    out[str(n)] = digest(m1, o1, m2, o2, *ms, *os_, *mn, *on, m3, o3, m4, o4, colsq)
    if dtype == torch.float16:
        kept[n] = (W, X)
# matrices that read different inputs, in one call each
ctxs = {n: sp.Context(n) for n in kept}
for n, (W, X) in kept.items():
    ctxs[n].sp_calib_accumulate(X)
owners = [ctxs[n] for n in kept] + [ctxs[520]]
Ws = [kept[n][0] for n in kept] + [kept[520][0][:33]]
mu, ou = sp.sp_select_unstructured_multi(owners, Ws, 0.5)
mm, om = sp.sp_select_nm_multi(owners, Ws, 2, 4)
out["multi"] = digest(*mu, *ou, *mm, *om)
for c in ctxs.values():
    c.close()
out["debug_status"] = list(sp.sp_debug_status())
print(json.dumps(out))
"""


def _run(library):
    env = dict(os.environ)
    if library:
        env["SWIFTPRUNE_LIBRARY"] = library
    else:
        env.pop("SWIFTPRUNE_LIBRARY", None)
    proc = subprocess.run([sys.executable, "-c", _SCRIPT % ROOT], env=env, capture_output=True,
                          text=True, timeout=600)
    assert proc.returncode == 0, proc.stderr[-2000:]
    return json.loads(proc.stdout.strip().splitlines()[-1])


def test_debug_build_records_no_violation_and_matches_the_release_build():
    from paper_2501_16376_b200 import build
    debug_lib = build.build(debug=True)
    release = _run(None)
    debug = _run(debug_lib)
    assert release.pop("debug_status")[0] == -1          # no checks compiled into the release build
    status = debug.pop("debug_status")
    assert status[0] == 0, "index check failed: code %d index %d limit %d" % tuple(status[1:])
    assert debug == release
