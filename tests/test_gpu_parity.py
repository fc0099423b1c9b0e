"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Integer artefacts and moved values bit-exact; activations and gradients within
1e-5 (fp32) / 2e-2 (bf16), norm-wise relative."""
import numpy as np
import pytest
import torch

from paper_2406_17611_b200 import binding as vb
from paper_2406_17611_b200 import synth

from helpers import TOL, LayerCase, close, dev_weights, host64, rel_err, to_device_rows, to_host_rows

pytestmark = pytest.mark.gpu

SEED = 77


@pytest.fixture(scope="module")
def cases(orc):
    cache = {}

    def get(name, scale):
        key = (name, scale)
        if key not in cache:
            cache[key] = LayerCase(orc, synth.make_workload(name, scale))
        return cache[key]
    return get


def send_order_slots(case):
    """slot (receive order) -> position in send order, from the oracle's halo sets."""
    g, P = case.g, case.wl.parts
    cnt = g.counts()
    send_base = np.zeros((P, P), dtype=np.int64)
    s = 0
    for p in range(P):
        for q in range(P):
            send_base[p, q] = s
            s += cnt[p, q]
    pos = []
    for q in range(P):
        for p in range(P):
            pos.extend(range(send_base[p, q], send_base[p, q] + cnt[p, q]))
    return np.asarray(pos, dtype=np.int64)


@pytest.mark.parametrize("name,scale,F", [("c1", 1.0, 64), ("c1", 1.0, 8), ("c2r", 0.05, 128), ("c3", 0.004, 100),
                                          ("c3", 0.004, 256), ("c4", 0.02, 602), ("c2", 0.05, 47)])
@pytest.mark.parametrize("ratio", [(1, 1), (4, 1), (385, 4), (128, 1), (1, 0)])
def test_compress_decompress_bit_exact(orc, cases, name, scale, F, ratio):
    case = cases(name, scale)
    X = synth.normal_features(case.wl.n, F, SEED, case.wl.bf16)
    Xd = to_device_rows(X, case.perm, case.dtype)
    key = (SEED, 3, 1)
    packed, nbytes = vb.varco_compress(case.plan, Xd, F, ratio, key)
    ref_packed, sent = case.g.compress(X, ratio, key)
    k = orc.kept(F, ratio)
    assert nbytes == sent * case.es == case.g.H_total * k * case.es
    assert np.array_equal(packed.to(torch.float64).cpu().numpy(), ref_packed)
    halo = vb.varco_decompress(case.plan, packed, F, ratio, key)
    ref_halo = case.g.decompress(ref_packed, F, ratio, key)
    assert np.array_equal(halo[:, :F].to(torch.float64).cpu().numpy(), ref_halo)
    assert (halo[:, :F] != 0).sum().item() <= case.g.H_total * k


def layer_io(case, layer, seed):
    wl = case.wl
    Ws, Wn, b = wl.layer_weights(layer)
    F_in, F_out = wl.widths[layer], wl.widths[layer + 1]
    X = synth.normal_features(wl.n, F_in, seed, wl.bf16)
    relu = layer < len(wl.widths) - 2
    return X, Ws, Wn, b, F_in, F_out, relu


CONFIG_LAYERS = [("c1", 1.0, 0), ("c1", 1.0, 1), ("c2", 0.05, 0), ("c2r", 0.05, 1), ("c2", 0.05, 2),
                 ("c3", 0.004, 0), ("c3", 0.004, 1), ("c3", 0.004, 2), ("c4", 0.02, 0), ("c4", 0.02, 1)]


@pytest.mark.parametrize("name,scale,layer", CONFIG_LAYERS)
@pytest.mark.parametrize("ratio", [(1, 1), (4, 1), (16, 1), (1935, 20), (1, 0)])
def test_layer_forward_and_backward(orc, cases, name, scale, layer, ratio):
    """Every layer of every configuration at full communication, fixed ratios, a scheduled fractional ratio and
    the "no communication" setting (ratio with denominator 0: k = 0, bytes 0)."""
    case = cases(name, scale)
    wl, dt = case.wl, case.dtype
    X, Ws, Wn, b, F_in, F_out, relu = layer_io(case, layer, SEED + layer)
    key = (SEED, 2, layer)
    Xd = to_device_rows(X, case.perm, dt)
    Wsd, Wnd, bd = dev_weights(Ws, dt), dev_weights(Wn, dt), dev_weights(b, torch.float32)
    Y, Agg, hb = vb.varco_layer_fwd(case.plan, Xd, Wsd, Wnd, bd, relu, ratio, key, case.ws, F_in=F_in)
    Yr, Aggr, hbr = case.g.layer_fwd(X, Ws, Wn, b, relu, ratio, key, elem_bytes=case.es)
    assert hb == hbr == case.g.H_total * orc.kept(F_in, ratio) * case.es
    assert vb.varco_workspace_status(case.ws) == 0
    tol = TOL[dt]
    assert close(to_host_rows(Agg, case.perm, F_in), Aggr, tol)
    assert close(to_host_rows(Y, case.perm, F_out), Yr, tol)

    # backward: both sides get the same Y (the oracle's, in the layer's dtype) so that the ReLU
    # mask is the same decision on both sides
    rng = np.random.default_rng(SEED + 5)
    dY = rng.standard_normal((wl.n, F_out)).astype(np.float32)
    if wl.bf16:
        dY = synth.bf16_round(dY)
    Yd = to_device_rows(Yr.astype(np.float32), case.perm, dt)
    Y_shared = to_host_rows(Yd, case.perm, F_out)
    dYd = to_device_rows(dY, case.perm, dt)
    dX, dWs, dWn, db, hb2 = vb.varco_layer_bwd(case.plan, Xd, Yd, Agg, Wsd, Wnd, dYd, relu, ratio, key, case.ws,
                                               F_in=F_in)
    rX, rWs, rWn, rb, hb2r = case.g.layer_bwd(X, Y_shared, Ws, Wn, dY, relu, ratio, key, elem_bytes=case.es)
    assert hb2 == hb2r == hb
    assert vb.varco_workspace_status(case.ws) == 0
    assert close(to_host_rows(dX, case.perm, F_in), rX, tol)
    assert close(host64(dWn), rWn, tol)
    assert rel_err(host64(db), rb) <= tol
    if wl.conv == "sage":
        assert close(host64(dWs), rWs, tol)


@pytest.mark.parametrize("name,scale,layer", [("c1", 1.0, 0), ("c3", 0.004, 1), ("c3", 0.004, 2), ("c4", 0.02, 0)])
@pytest.mark.parametrize("ratio", [(4, 3), (2, 1), (9, 1)])
def test_layer_forward_mild_and_mid_ratios(orc, cases, name, scale, layer, ratio):
    """Ratios between the cases above: three quarters of a row kept (packed rows wider than two chunks per lane:
    the slot-by-slot decompression), half, and a ninth (kept columns on the way back for the wide rows)."""
    case = cases(name, scale)
    wl, dt = case.wl, case.dtype
    X, Ws, Wn, b, F_in, F_out, relu = layer_io(case, layer, SEED + 3 * layer)
    key = (SEED + 1, 5, layer)
    Xd = to_device_rows(X, case.perm, dt)
    Wsd, Wnd, bd = dev_weights(Ws, dt), dev_weights(Wn, dt), dev_weights(b, torch.float32)
    Y, Agg, hb = vb.varco_layer_fwd(case.plan, Xd, Wsd, Wnd, bd, relu, ratio, key, case.ws, F_in=F_in)
    Yr, Aggr, hbr = case.g.layer_fwd(X, Ws, Wn, b, relu, ratio, key, elem_bytes=case.es)
    assert hb == hbr
    tol = TOL[dt]
    assert rel_err(to_host_rows(Agg, case.perm, F_in), Aggr) <= tol
    assert rel_err(to_host_rows(Y, case.perm, F_out), Yr) <= tol
    rng = np.random.default_rng(SEED + 9)
    dY = rng.standard_normal((wl.n, F_out)).astype(np.float32)
    if wl.bf16:
        dY = synth.bf16_round(dY)
    Yd = to_device_rows(Yr.astype(np.float32), case.perm, dt)
    dX, dWs, dWn, db, hb2 = vb.varco_layer_bwd(case.plan, Xd, Yd, Agg, Wsd, Wnd, to_device_rows(dY, case.perm, dt),
                                               relu, ratio, key, case.ws, F_in=F_in)
    rX, rWs, rWn, rb, _ = case.g.layer_bwd(X, to_host_rows(Yd, case.perm, F_out), Ws, Wn, dY, relu, ratio, key,
                                           elem_bytes=case.es)
    assert hb2 == hb and vb.varco_workspace_status(case.ws) == 0
    assert rel_err(to_host_rows(dX, case.perm, F_in), rX) <= tol
    assert rel_err(host64(dWn), rWn) <= tol and rel_err(host64(db), rb) <= tol


def test_tiny_config_two_layer_epochs(orc, cases):
    """Config 1 end to end: 2-layer GCN over the scheduled epochs 0, 3, 4 (k = 1, 2, 64) and at
    full communication; each layer's input is the previous layer's device output."""
    case = cases("c1", 1.0)
    wl, dt = case.wl, case.dtype
    X0 = wl.features()
    total = 0
    for epoch, ratio in [(0, orc.schedule_linear(0, 20)), (3, orc.schedule_linear(3, 20)),
                         (4, orc.schedule_linear(4, 20)), (19, (1, 1))]:
        Xd = to_device_rows(X0, case.perm, dt)
        Xh = X0.astype(np.float64)
        for layer in range(2):
            Ws, Wn, b = wl.layer_weights(layer)
            relu = layer == 0
            key = (SEED, epoch, layer)
            Y, Agg, hb = vb.varco_layer_fwd(case.plan, Xd, None, dev_weights(Wn, dt), dev_weights(b, torch.float32),
                                            relu, ratio, key, case.ws, F_in=wl.widths[layer])
            Yr, _, hbr = case.g.layer_fwd(Xh, None, Wn, b, relu, ratio, key, elem_bytes=4)
            assert hb == hbr
            total += hb
            assert rel_err(to_host_rows(Y, case.perm, wl.widths[layer + 1]), Yr) <= 1e-5
            Xd, Xh = Y, Yr
    k = [orc.kept(64, orc.schedule_linear(e, 20)) for e in (0, 3, 4)] + [64]
    assert total == 2 * 4 * case.g.H_total * sum(k)


def test_degenerate_graphs(orc):
    """No edges at all, a single partition (no halo), isolated nodes, one node per partition."""
    n, F_in, F_out = 37, 12, 5
    rng = np.random.default_rng(0)
    X = rng.standard_normal((n, F_in)).astype(np.float32)
    Wn = rng.standard_normal((F_in, F_out)).astype(np.float32)
    Ws = rng.standard_normal((F_in, F_out)).astype(np.float32)
    b = rng.standard_normal(F_out).astype(np.float32)
    empty = (np.zeros(n + 1, dtype=np.int64), np.zeros(0, dtype=np.int32))
    ring_u = np.arange(n - 5, dtype=np.int64)
    ring = synth._csr_from_pairs(n, ring_u, (ring_u + 1) % (n - 5))        # last 5 nodes isolated
    for (rp, col), P, part in [(empty, 3, np.arange(n) % 3), (ring, 1, np.zeros(n)), (ring, n, np.arange(n)),
                               (ring, 4, np.arange(n) % 4)]:
        for conv in ("gcn", "sage"):
            part = np.asarray(part, dtype=np.int32)
            plan = vb.Plan(rp, col, part, P, conv).upload()
            g = orc.graph(rp, col, part, P, conv)
            perm = plan.perm()
            ws = plan.workspace(F_in, F_out, vb.F32)
            Xd = to_device_rows(X, perm, torch.float32)
            W_self = Ws if conv == "sage" else None
            ratio, key = (3, 1), (1, 2, 3)
            Y, Agg, hb = vb.varco_layer_fwd(plan, Xd, dev_weights(W_self, torch.float32),
                                            dev_weights(Wn, torch.float32), dev_weights(b, torch.float32), True,
                                            ratio, key, ws, F_in=F_in)
            Yr, Aggr, hbr = g.layer_fwd(X, W_self, Wn, b, True, ratio, key)
            assert hb == hbr
            assert rel_err(to_host_rows(Y, perm, F_out), Yr) <= 1e-5
            dY = rng.standard_normal((n, F_out)).astype(np.float32)
            Yd = to_device_rows(Yr.astype(np.float32), perm, torch.float32)
            dX, dWs, dWn, db, _ = vb.varco_layer_bwd(plan, Xd, Yd, Agg, dev_weights(W_self, torch.float32),
                                                     dev_weights(Wn, torch.float32),
                                                     to_device_rows(dY, perm, torch.float32), True, ratio, key, ws,
                                                     F_in=F_in)
            rX, rWs, rWn, rb, _ = g.layer_bwd(X, to_host_rows(Yd, perm, F_out), W_self, Wn, dY, True, ratio, key)
            assert rel_err(to_host_rows(dX, perm, F_in), rX) <= 1e-5
            assert rel_err(host64(dWn), rWn) <= 1e-5 and rel_err(host64(db), rb) <= 1e-5
            plan.close()


@pytest.mark.parametrize("bf16,F_in,F_out", [(False, 64, 32), (True, 256, 64), (True, 100, 47)])
def test_hub_rows(orc, bf16, F_in, F_out):
    """Rows and sources with thousands of entries take the CTA-per-row path of the aggregation."""
    n, P = 6000, 4
    rng = np.random.default_rng(3)
    hubs = np.repeat(np.arange(3, dtype=np.int64), n - 3)
    others = np.tile(np.arange(3, n, dtype=np.int64), 3)
    ring = np.arange(n, dtype=np.int64)
    rp, col = synth._csr_from_pairs(n, np.concatenate([hubs, ring]), np.concatenate([others, (ring + 1) % n]))
    part = synth.partition_random_equal(n, P, 5)
    dt = torch.bfloat16 if bf16 else torch.float32
    X = synth.normal_features(n, F_in, 1, bf16)
    Wn = synth.glorot_uniform(F_in, F_out, 2, bf16)
    Ws = synth.glorot_uniform(F_in, F_out, 3, bf16)
    b = (0.1 * rng.standard_normal(F_out)).astype(np.float32)
    dY = rng.standard_normal((n, F_out)).astype(np.float32)
    dY = synth.bf16_round(dY) if bf16 else dY
    plan = vb.Plan(rp, col, part, P, "sage").upload()
    g = orc.graph(rp, col, part, P, "sage")
    perm = plan.perm()
    ws = plan.workspace(F_in, F_out, vb.BF16 if bf16 else vb.F32)
    Xd = to_device_rows(X, perm, dt)
    for ratio in [(1, 1), (4, 1), (32, 1)]:   # full, dense-compressed, sparse-halo paths
        key = (9, 1, 0)
        Y, Agg, _ = vb.varco_layer_fwd(plan, Xd, dev_weights(Ws, dt), dev_weights(Wn, dt),
                                       dev_weights(b, torch.float32), True, ratio, key, ws, F_in=F_in)
        Yr, Aggr, _ = g.layer_fwd(X, Ws, Wn, b, True, ratio, key)
        assert rel_err(to_host_rows(Agg, perm, F_in), Aggr) <= TOL[dt]
        assert rel_err(to_host_rows(Y, perm, F_out), Yr) <= TOL[dt]
        Yd = to_device_rows(Yr.astype(np.float32), perm, dt)
        dX, dWs, dWn, db, _ = vb.varco_layer_bwd(plan, Xd, Yd, Agg, dev_weights(Ws, dt), dev_weights(Wn, dt),
                                                 to_device_rows(dY, perm, dt), True, ratio, key, ws, F_in=F_in)
        rX, rWs, rWn, rb, _ = g.layer_bwd(X, to_host_rows(Yd, perm, F_out), Ws, Wn, dY, True, ratio, key)
        assert vb.varco_workspace_status(ws) == 0
        assert rel_err(to_host_rows(dX, perm, F_in), rX) <= TOL[dt]
        assert rel_err(host64(dWn), rWn) <= TOL[dt] and rel_err(host64(dWs), rWs) <= TOL[dt]
    plan.close()


@pytest.mark.parametrize("bf16,F_in,F_out,conv", [(True, 256, 64, "sage"), (True, 602, 48, "gcn"), (False, 64, 32, "sage")])
def test_feature_panels_on_dense_graph(orc, bf16, F_in, F_out, conv):
    """Dense neighbourhoods (about 120 entries per row, every source row reused ~30 times): with a tiny L2
    budget the forward aggregation runs in its finest feature panels; results must not change."""
    n, P = 1500, 4
    rp, col = synth.erdos_renyi(n, 120.0, 21)
    part = synth.partition_random_equal(n, P, 22)
    dt = torch.bfloat16 if bf16 else torch.float32
    rng = np.random.default_rng(5)
    X = synth.normal_features(n, F_in, 1, bf16)
    Wn = synth.glorot_uniform(F_in, F_out, 2, bf16)
    Ws = synth.glorot_uniform(F_in, F_out, 3, bf16) if conv == "sage" else None
    b = (0.1 * rng.standard_normal(F_out)).astype(np.float32)
    plan = vb.Plan(rp, col, part, P, conv).upload()
    plan.set_l2_budget(1024)
    g = orc.graph(rp, col, part, P, conv)
    perm = plan.perm()
    ws = plan.workspace(F_in, F_out, vb.BF16 if bf16 else vb.F32)
    Xd = to_device_rows(X, perm, dt)
    for ratio in [(1, 1), (4, 1)]:
        key = (3, 1, 0)
        Y, Agg, hb = vb.varco_layer_fwd(plan, Xd, dev_weights(Ws, dt), dev_weights(Wn, dt),
                                        dev_weights(b, torch.float32), True, ratio, key, ws, F_in=F_in)
        Yr, Aggr, hbr = g.layer_fwd(X, Ws, Wn, b, True, ratio, key, elem_bytes=2 if bf16 else 4)
        assert hb == hbr and vb.varco_workspace_status(ws) == 0
        assert rel_err(to_host_rows(Agg, perm, F_in), Aggr) <= TOL[dt]
        assert rel_err(to_host_rows(Y, perm, F_out), Yr) <= TOL[dt]
    plan.close()


def test_backward_is_reproducible(cases):
    """The ordered (atomic-free) gradient accumulation gives bit-identical results run to run."""
    case = cases("c2r", 0.05)
    wl, dt = case.wl, case.dtype
    X, Ws, Wn, b, F_in, F_out, relu = layer_io(case, 1, SEED)
    Xd = to_device_rows(X, case.perm, dt)
    Wsd, Wnd, bd = dev_weights(Ws, dt), dev_weights(Wn, dt), dev_weights(b, torch.float32)
    key, ratio = (SEED, 1, 1), (4, 1)
    Y, Agg, _ = vb.varco_layer_fwd(case.plan, Xd, Wsd, Wnd, bd, relu, ratio, key, case.ws, F_in=F_in)
    dYd = torch.randn_like(Y)
    outs = []
    for _ in range(2):
        dX, dWs, dWn, db, _ = vb.varco_layer_bwd(case.plan, Xd, Y, Agg, Wsd, Wnd, dYd, relu, ratio, key, case.ws,
                                                 F_in=F_in)
        outs.append((dX.clone(), dWs.clone(), dWn.clone(), db.clone()))
    for a, c in zip(*outs):
        assert torch.equal(a, c)
