"""The debug build of the library (-DVARCO_DEBUG: device-side index checks that record a code and skip the
access, host-side validation of the plan image, guard blocks behind the workspace segments) on the tiny cases:
results equal the release build's contract and no check fires.  Runs in a child process, because a process
holds one copy of the library."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import numpy as np, torch, sys
sys.path.insert(0, %(root)r)
sys.path.insert(0, %(tests)r)
import oracle
from paper_2406_17611_b200 import binding as vb, synth
from helpers import LayerCase, close, dev_weights, host64, to_device_rows, to_host_rows, TOL
assert vb.varco_debug_status() == (True, 0)
orc = oracle.Oracle()
for name, scale, layer, ratio in [("c1", 0.2, 0, (4, 1)), ("c1", 0.2, 1, (1, 1)), ("c2r", 0.01, 1, (16, 1)),
                                  ("c3", 0.002, 1, (1, 1)), ("c3", 0.002, 2, (64, 1)), ("c3", 0.002, 2, (4, 1)), ("c3", 0.002, 0, (1, 0)),
                                  ("c4", 0.01, 0, (8, 1))]:
    case = LayerCase(orc, synth.make_workload(name, scale))
    wl, dt = case.wl, case.dtype
    Ws, Wn, b = wl.layer_weights(layer)
    F_in, F_out = wl.widths[layer], wl.widths[layer + 1]
    relu = layer < len(wl.widths) - 2
    X = synth.normal_features(wl.n, F_in, 3, wl.bf16)
    Xd = to_device_rows(X, case.perm, dt)
    key = (5, 1, layer)
    Y, Agg, hb = vb.varco_layer_fwd(case.plan, Xd, dev_weights(Ws, dt), dev_weights(Wn, dt),
                                    dev_weights(b, torch.float32), relu, ratio, key, case.ws, F_in=F_in)
    assert vb.varco_workspace_status(case.ws) == 0          # bounded waits fine, guard blocks intact
    Yr, Aggr, hbr = case.g.layer_fwd(X, Ws, Wn, b, relu, ratio, key, elem_bytes=case.es)
    assert hb == hbr and close(to_host_rows(Y, case.perm, F_out), Yr, TOL[dt])
    dY = np.random.default_rng(1).standard_normal((wl.n, F_out)).astype(np.float32)
    dY = synth.bf16_round(dY) if wl.bf16 else dY
    Yd = to_device_rows(Yr.astype(np.float32), case.perm, dt)
    dX, dWs, dWn, db, _ = vb.varco_layer_bwd(case.plan, Xd, Yd, Agg, dev_weights(Ws, dt), dev_weights(Wn, dt),
                                             to_device_rows(dY, case.perm, dt), relu, ratio, key, case.ws, F_in=F_in)
    assert vb.varco_workspace_status(case.ws) == 0
    rX = case.g.layer_bwd(X, to_host_rows(Yd, case.perm, F_out), Ws, Wn, dY, relu, ratio, key, elem_bytes=case.es)[0]
    assert close(to_host_rows(dX, case.perm, F_in), rX, TOL[dt])
    assert vb.varco_debug_status() == (True, 0)            # no index check fired
    case.plan.close()
# a guard block that something wrote into is reported (bit 30), without touching anything else
case = LayerCase(orc, synth.make_workload("c1", 0.2))
wl = case.wl
Ws, Wn, b = wl.layer_weights(0)
Xd = to_device_rows(synth.normal_features(wl.n, 64, 3, False), case.perm, torch.float32)
vb.varco_layer_fwd(case.plan, Xd, None, dev_weights(Wn, torch.float32), dev_weights(b, torch.float32), True, (1, 1),
                   (5, 1, 0), case.ws, F_in=64)
assert vb.varco_workspace_status(case.ws) == 0
base = (256 - case.ws.data_ptr() %% 256) %% 256
table = case.ws[base + 64:base + 64 + 72].cpu().numpy().view(np.uint64)
assert 1 <= int(table[0]) <= 8
case.ws[base + int(table[1]) + 5] = 0                      # one byte of the first guard block
assert vb.varco_workspace_status(case.ws) == 1 << 30
print("debug build ok")
"""


def test_tiny_cases_under_the_debug_build_are_clean():
    from paper_2406_17611_b200 import build as vbuild
    lib = vbuild.build(debug=True)
    env = dict(os.environ, VARCO_LIBRARY=lib)
    code = CHILD % {"root": ROOT, "tests": os.path.join(ROOT, "tests")}
    r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and "debug build ok" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]
