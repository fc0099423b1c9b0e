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

from helpers import close, dev_weights, rel_err

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


# ------------------------------------------------------------------------------------------ the other configs
def test_sbm_random_split_every_row(orc):
    """The 100,000-node SBM with the random 8-way split (fp32) at its full size: the oracle runs whole layers
    here, so every row of every layer is compared, forward and backward, at full communication and at 4:1."""
    wl = synth.make_workload("c2r", 1.0)
    plan = vb.Plan(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv).upload()
    g = orc.graph(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv)
    perm = plan.perm()
    assert plan.H_total == g.H_total and np.array_equal(plan.counts(), g.counts())
    ws = plan.workspace(256, 256, vb.F32)
    dt = torch.float32
    L = len(wl.widths) - 1
    for ratio in [(1, 1), (4, 1)]:
        X = wl.features().astype(np.float32)
        for layer in range(L):
            F_in, F_out = wl.widths[layer], wl.widths[layer + 1]
            relu = layer < L - 1
            Ws, Wn, b = wl.layer_weights(layer)
            key = (SEED, 1, layer)
            Xd = torch.from_numpy(X[perm]).cuda()
            Y, Agg, hb = vb.varco_layer_fwd(plan, Xd, dev_weights(Ws, dt), dev_weights(Wn, dt),
                                            dev_weights(b, dt), relu, ratio, key, ws, F_in=F_in)
            Yr, Aggr, hbr = g.layer_fwd(X, Ws, Wn, b, relu, ratio, key, elem_bytes=4)
            assert hb == hbr == g.H_total * orc.kept(F_in, ratio) * 4
            gotY = np.empty_like(Yr)
            gotY[perm] = Y[:, :F_out].double().cpu().numpy()
            gotA = np.empty_like(Aggr)
            gotA[perm] = Agg[:, :F_in].double().cpu().numpy()
            assert close(gotA, Aggr, 1e-5) and close(gotY, Yr, 1e-5)
            dY = np.random.default_rng(layer).standard_normal((wl.n, F_out)).astype(np.float32)
            Yd = torch.from_numpy(Yr.astype(np.float32)[perm]).cuda()
            dX, dWs, dWn, db, hb2 = vb.varco_layer_bwd(plan, Xd, Yd, Agg, dev_weights(Ws, dt), dev_weights(Wn, dt),
                                                       torch.from_numpy(dY[perm]).cuda(), relu, ratio, key, ws,
                                                       F_in=F_in)
            rX, rWs, rWn, rb, _ = g.layer_bwd(X, Yr.astype(np.float32), Ws, Wn, dY, relu, ratio, key, elem_bytes=4)
            got = np.empty_like(rX)
            got[perm] = dX[:, :F_in].double().cpu().numpy()
            assert hb2 == hb and close(got, rX, 1e-5)
            assert close(dWn.double().cpu().numpy(), rWn, 1e-5) and close(dWs.double().cpu().numpy(), rWs, 1e-5)
            assert rel_err(db.double().cpu().numpy(), rb) <= 1e-5
            X = Yr.astype(np.float32)      # the next layer's input: the oracle's own output, on both sides
    plan.close()


def test_dense_neighbourhood_config_on_sampled_rows(orc):
    """The 233,000-node dense-neighbourhood graph (mean degree 490, random 8-way split, GCN 602-256-41, bf16)
    at its full size: sampled rows including the widest hub, both layers, full communication and 16:1."""
    wl = synth.make_workload("c4", 1.0)
    plan = vb.Plan(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv).upload()
    g = orc.graph(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv)
    perm = plan.perm()
    inv = np.empty_like(perm)
    inv[perm] = np.arange(perm.shape[0])
    assert plan.H_total == g.H_total and plan.cross_entries == g.cross_entries
    assert np.array_equal(plan.counts(), g.counts())
    ws = plan.workspace(602, 256, vb.BF16)
    dt = torch.bfloat16
    deg = np.diff(wl.row_ptr)
    rng = np.random.default_rng(3)
    rows = np.unique(np.concatenate([rng.integers(0, wl.n, size=20), [int(np.argmax(deg)), int(np.argmin(deg))]]))
    for layer, ratio in [(0, (1, 1)), (0, (16, 1)), (1, (1, 1)), (1, (16, 1))]:
        F_in, F_out = wl.widths[layer], wl.widths[layer + 1]
        relu = layer == 0
        Ws, Wn, b = wl.layer_weights(layer)
        X = synth.normal_features(wl.n, F_in, SEED + layer, True)
        ld = (F_in + 7) // 8 * 8
        Xd = torch.zeros((wl.n, ld), dtype=dt)
        Xd[:, :F_in] = torch.from_numpy(X[perm]).to(dt)
        Xd = Xd.cuda()
        key = (SEED, 4, layer)
        Y, Agg, hb = vb.varco_layer_fwd(plan, Xd, None, dev_weights(Wn, dt), dev_weights(b, torch.float32), relu,
                                        ratio, key, ws, F_in=F_in)
        assert vb.varco_workspace_status(ws) == 0
        assert hb == g.H_total * orc.kept(F_in, ratio) * 2
        Yr, Aggr = g.layer_fwd_rows(rows, X.astype(np.float64), None, Wn, b, relu, ratio, key)
        sel = torch.from_numpy(inv[rows]).cuda()
        assert close(Agg[sel][:, :F_in].double().cpu().numpy(), Aggr, 2e-2)
        assert close(Y[sel][:, :F_out].double().cpu().numpy(), Yr, 2e-2)
        dY = synth.bf16_round(np.random.default_rng(11).standard_normal((wl.n, F_out)).astype(np.float32))
        dYd = torch.zeros_like(Y)
        dYd[:, :F_out] = torch.from_numpy(dY[perm]).to(dt).cuda()
        dX, _, dWn, db, hb2 = vb.varco_layer_bwd(plan, Xd, Y, Agg, None, dev_weights(Wn, dt), dYd, relu, ratio, key,
                                                 ws, F_in=F_in)
        assert vb.varco_workspace_status(ws) == 0 and hb2 == hb
        Yh = np.empty((wl.n, F_out), dtype=np.float32)
        Yh[perm] = Y[:, :F_out].float().cpu().numpy()
        few = rows[:8]
        rX = g.layer_dx_rows(few, Yh, None, Wn, dY, relu, ratio, key)
        got = dX[torch.from_numpy(inv[few]).cuda()][:, :F_in].double().cpu().numpy()
        assert close(got, rX, 2e-2)
    plan.close()


@pytest.mark.parametrize("epoch", [0, 1, 19, 20])
def test_four_layer_model_at_schedule_points(orc, big, epoch):
    """The rate-sweep configuration (4-layer SAGE 100-256-256-256-47 on the 2.45M-node graph) at epochs
    0, 1, 19 and 20 of the 100-epoch schedule (slope 5: ratios 128, 121.65, 7.35 and 1): the four layers chained
    on the device, each checked on sampled rows against the oracle fed the same layer input, forward and
    input gradient, with the halo bytes of the epoch against the closed form."""
    wl, plan, g, perm, inv, ws = (big[k] for k in ("wl", "plan", "g", "perm", "inv", "ws"))
    widths = [100, 256, 256, 256, 47]
    L = 4
    dt = torch.bfloat16
    ratio = vb.varco_schedule_linear(epoch, 100, 5)
    assert ratio == orc.schedule_linear(epoch, 100, 5)
    rows = sample_rows(big, 24)
    sel = torch.from_numpy(inv[rows]).cuda()
    weights = []
    for l in range(L):
        s = SEED + 50 + 10 * l
        weights.append((synth.glorot_uniform(widths[l], widths[l + 1], s, True),
                        synth.glorot_uniform(widths[l], widths[l + 1], s + 1, True),
                        (0.1 * np.random.default_rng(s + 2).standard_normal(widths[l + 1])).astype(np.float32)))
    X = wl.features()
    Xd = torch.zeros((wl.n, 104), dtype=dt)
    Xd[:, :100] = torch.from_numpy(X[perm]).to(dt)
    acts, aggs = [Xd.cuda()], []
    total_bytes = 0
    for l in range(L):
        Ws, Wn, b = weights[l]
        F_in, F_out = widths[l], widths[l + 1]
        key = (SEED, epoch, l)
        Y, Agg, hb = vb.varco_layer_fwd(plan, acts[l], dev_weights(Ws, dt), dev_weights(Wn, dt),
                                        dev_weights(b, torch.float32), l < L - 1, ratio, key, ws, F_in=F_in)
        assert vb.varco_workspace_status(ws) == 0
        total_bytes += hb
        Xh = np.empty((wl.n, F_in))
        Xh[perm] = acts[l][:, :F_in].double().cpu().numpy()       # this layer's input as the device holds it
        Yr, Aggr = g.layer_fwd_rows(rows, Xh, Ws, Wn, b, l < L - 1, ratio, key)
        assert close(Agg[sel][:, :F_in].double().cpu().numpy(), Aggr, 2e-2)
        assert close(Y[sel][:, :F_out].double().cpu().numpy(), Yr, 2e-2)
        acts.append(Y)
        aggs.append(Agg)
        del Xh
    ks = [orc.kept(F, ratio) for F in widths[:-1]]
    assert ks == {0: [1, 2, 2, 2], 1: [1, 3, 3, 3], 19: [14, 35, 35, 35], 20: [100, 256, 256, 256]}[epoch]
    assert total_bytes == g.H_total * sum(ks) * 2
    # backward chain: the gradient of every layer feeds the layer below; sampled input-gradient rows
    dY = synth.bf16_round(np.random.default_rng(13).standard_normal((wl.n, 47)).astype(np.float32))
    grad = torch.zeros_like(acts[L])
    grad[:, :47] = torch.from_numpy(dY[perm]).to(dt).cuda()
    few = rows[:10]
    fsel = torch.from_numpy(inv[few]).cuda()
    back_bytes = 0
    for l in reversed(range(L)):
        Ws, Wn, b = weights[l]
        F_in, F_out = widths[l], widths[l + 1]
        key = (SEED, epoch, l)
        dX, dWs, dWn, db, hb = vb.varco_layer_bwd(plan, acts[l], acts[l + 1], aggs[l], dev_weights(Ws, dt),
                                                  dev_weights(Wn, dt), grad, l < L - 1, ratio, key, ws, F_in=F_in)
        assert vb.varco_workspace_status(ws) == 0
        back_bytes += hb
        Yh = np.empty((wl.n, F_out), dtype=np.float32)
        Yh[perm] = acts[l + 1][:, :F_out].float().cpu().numpy()
        gh = np.empty((wl.n, F_out), dtype=np.float32)
        gh[perm] = grad[:, :F_out].float().cpu().numpy()
        rX = g.layer_dx_rows(few, Yh, Ws, Wn, gh, l < L - 1, ratio, key)
        assert close(dX[fsel][:, :F_in].double().cpu().numpy(), rX, 2e-2)
        grad = dX
    assert back_bytes == total_bytes
