"""Full-size parity: the products-shaped workload (2.45M nodes, ~123M stored entries, 16 partitions,
bf16) in the launch configuration the benchmark times.  The oracle cannot run whole layers at this
size in test time, so outputs are checked on sampled rows that it computes one by one from the
definitions, integer artefacts are compared exactly, and the weight gradient (a reduction over all
rows) is checked entry-wise against an fp64 recomputation from the device's own operands."""
import numpy as np
import pytest
import torch

from paper_2406_17611_b200 import binding as vb
from paper_2406_17611_b200 import synth

from helpers import dev_weights, rel_err

pytestmark = pytest.mark.gpu

SEED = 2406


@pytest.fixture(scope="module")
def big(orc):
    wl = synth.make_workload("c3", 1.0)
    plan = vb.Plan(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv).upload()
    g = orc.graph(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv)
    perm = plan.perm()
    inv = np.empty_like(perm)
    inv[perm] = np.arange(perm.shape[0])
    ws = plan.workspace(256, 256, vb.BF16)
    return dict(wl=wl, plan=plan, g=g, perm=perm, inv=inv, ws=ws)


def test_partition_artefacts_bit_exact(big):
    plan, g, wl = big["plan"], big["g"], big["wl"]
    assert plan.H_total == g.H_total and plan.cross_entries == g.cross_entries
    assert np.array_equal(plan.counts(), g.counts())
    assert np.array_equal(big["perm"], g.perm())
    for p, q in [(0, 1), (7, 3), (15, 0), (9, 9)]:
        assert np.array_equal(plan.halo(p, q), g.halo(p, q))
    # byte counts of every epoch of the 100-epoch schedule follow the closed form
    for e in range(100):
        r = vb.varco_schedule_linear(e, 100)
        for F in (100, 256):
            k = vb.varco_kept(F, r)
            assert k == min(F, max(1, -(-F * r[1] // r[0])))


def sample_rows(big, count):
    wl = big["wl"]
    deg = np.diff(wl.row_ptr)
    rng = np.random.default_rng(5)
    rows = set(rng.integers(0, wl.n, size=count).tolist())
    rows.add(int(np.argmax(deg)))                      # the largest hub
    rows.update(np.nonzero(deg == 0)[0][:2].tolist())  # isolated nodes
    rows.update(np.argsort(deg)[-3:].tolist())
    return np.asarray(sorted(rows), dtype=np.int64)


@pytest.mark.parametrize("layer,ratio", [(1, (1, 1)), (1, (4, 1)), (1, (385, 4)), (2, (1, 1)), (2, (64, 1)),
                                         (2, (8, 1))])
def test_layer_on_sampled_rows(orc, big, layer, ratio):
    """Layer 1 (256 -> 256, ReLU) and the output layer (256 -> 47, linear: the narrow backward, whose slot
    gradients come from the kept-entry product at 64:1 and from the product + selection at 8:1)."""
    wl, plan, g, perm, inv, ws = (big[k] for k in ("wl", "plan", "g", "perm", "inv", "ws"))
    F_in, F_out = wl.widths[layer], wl.widths[layer + 1]
    relu = layer < len(wl.widths) - 2
    dt = torch.bfloat16
    Ws, Wn, b = wl.layer_weights(layer)
    X = synth.normal_features(wl.n, F_in, SEED + 1, True)            # original order, bf16-representable
    Xd = torch.from_numpy(X[perm]).to(dt).cuda()
    key = (SEED, 7, layer)
    Y, Agg, hb = vb.varco_layer_fwd(plan, Xd, dev_weights(Ws, dt), dev_weights(Wn, dt),
                                    dev_weights(b, torch.float32), relu, ratio, key, ws, F_in=F_in)
    assert vb.varco_workspace_status(ws) == 0
    k = orc.kept(F_in, ratio)
    assert hb == g.H_total * k * 2
    rows = sample_rows(big, 48)
    X64 = X.astype(np.float64)
    Yr, Aggr = g.layer_fwd_rows(rows, X64, Ws, Wn, b, relu, ratio, key)
    got_Y = Y[torch.from_numpy(inv[rows]).cuda()][:, :F_out].double().cpu().numpy()
    got_A = Agg[torch.from_numpy(inv[rows]).cuda()].double().cpu().numpy()
    assert rel_err(got_A, Aggr) <= 2e-2
    assert rel_err(got_Y, Yr) <= 2e-2

    # backward on sampled rows; Y fed to both sides is the device's own forward output (its ReLU
    # mask is then the same decision on both sides), dY is seeded
    dY = synth.bf16_round(np.random.default_rng(11).standard_normal((wl.n, F_out)).astype(np.float32))
    dYd = torch.zeros_like(Y)
    dYd[:, :F_out] = torch.from_numpy(dY[perm]).to(dt).cuda()
    dX, dWs, dWn, db, hb2 = vb.varco_layer_bwd(plan, Xd, Y, Agg, dev_weights(Ws, dt), dev_weights(Wn, dt), dYd, relu,
                                               ratio, key, ws, F_in=F_in)
    assert vb.varco_workspace_status(ws) == 0 and hb2 == hb
    Yh = np.empty((wl.n, F_out), dtype=np.float32)
    Yh[perm] = Y[:, :F_out].float().cpu().numpy()
    rX = g.layer_dx_rows(rows[:24], Yh, Ws, Wn, dY, relu, ratio, key)
    got_dX = dX[torch.from_numpy(inv[rows[:24]]).cuda()].double().cpu().numpy()
    assert rel_err(got_dX, rX) <= 2e-2
    # weight gradients: entries recomputed in fp64 from the device's Agg / X and the masked dY
    dZ = dYd.double() * (Y > 0).double() if relu else dYd.double()
    for (a, o) in [(0, 0), (17, 200 % F_out), (255, F_out - 1), (100, 3)]:
        want_n = float((Agg[:, a].double() * dZ[:, o]).sum().item())
        want_s = float((Xd[:, a].double() * dZ[:, o]).sum().item())
        scale_n = float((Agg[:, a].double().abs() * dZ[:, o].abs()).sum().item())
        scale_s = float((Xd[:, a].double().abs() * dZ[:, o].abs()).sum().item())
        assert abs(float(dWn[a, o]) - want_n) <= 1e-4 * scale_n
        assert abs(float(dWs[a, o]) - want_s) <= 1e-4 * scale_s
    assert abs(float(db[5]) - float(dZ[:, 5].sum().item())) <= 1e-4 * float(dZ[:, 5].abs().sum().item())


def test_compress_samples_bit_exact(orc, big):
    wl, plan, g, perm = big["wl"], big["plan"], big["g"], big["perm"]
    F, ratio, key = 100, (16, 1), (SEED, 3, 0)
    X = wl.features()
    Xd = torch.zeros((wl.n, 104), dtype=torch.bfloat16)
    Xd[:, :F] = torch.from_numpy(X[perm]).to(torch.bfloat16)
    Xd = Xd.cuda()
    packed, nbytes = vb.varco_compress(plan, Xd, F, ratio, key)
    k = orc.kept(F, ratio)
    assert nbytes == g.H_total * k * 2
    cnt = g.counts()
    base = np.concatenate([[0], np.cumsum(cnt.reshape(-1))])
    rng = np.random.default_rng(2)
    for _ in range(40):
        p, q = rng.integers(0, 16, size=2)
        if p == q or cnt[p, q] == 0:
            continue
        ids = g.halo(int(p), int(q))
        r = int(rng.integers(0, len(ids)))
        j = int(ids[r])
        idx = orc.wire_positions(*key, j, F, k)
        got = packed[base[p * 16 + q] + r].float().cpu().numpy()
        assert np.array_equal(got, X[j, idx])
