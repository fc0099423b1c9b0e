"""Pins for the oracle's partition sets, compressor and partitioned layer.

Everything the oracle computes is checked here against something other than
itself: dense-matrix brute force (NumPy) on tiny graphs, PyTorch autograd,
the centralized layer at full communication, finite differences, and the
byte-count formula of the paper's efficiency section.
"""
import numpy as np
import pytest

from oracle import dense
from paper_2406_17611_b200 import synth

KEY = (1234, 3, 1)


def tiny_graph(n, m, seed):
    rng = np.random.default_rng(seed)
    u = rng.integers(0, n, size=m)
    v = rng.integers(0, n, size=m)
    return synth._csr_from_pairs(n, u.astype(np.int64), v.astype(np.int64))


def masks_for(orc, n, F, k, key):
    M = np.zeros((n, F))
    for j in range(n):
        M[j, orc.perm_indices(key[0], key[1], key[2], j, F, k)] = 1.0
    return M


def weights(F_in, F_out, sage, seed):
    rng = np.random.default_rng(seed)
    Wn = rng.standard_normal((F_in, F_out)) * 0.3
    Ws = rng.standard_normal((F_in, F_out)) * 0.3 if sage else None
    b = rng.standard_normal(F_out) * 0.1
    return Ws, Wn, b


# ------------------------------------------------------------------ partition / halo sets
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_halo_sets_match_brute_force(orc, seed):
    n, P = 10, 3
    rp, col = tiny_graph(n, 14, seed)
    part = np.random.default_rng(seed).integers(0, P, size=n).astype(np.int32)
    g = orc.graph(rp, col, part, P, "sage")
    A = np.zeros((n, n), dtype=bool)
    for i in range(n):
        A[i, col[rp[i]:rp[i + 1]]] = True
    total = 0
    for p in range(P):
        for q in range(P):
            want = [j for j in range(n) if p != q and part[j] == p and any(A[i, j] and part[i] == q for i in range(n))]
            assert g.halo(p, q).tolist() == want
            total += len(want)
    assert g.H_total == total
    cross = sum(1 for i in range(n) for j in range(n) if A[i, j] and part[i] != part[j])
    assert g.cross_entries == cross and g.self_entries == A.sum() - cross
    perm = g.perm()
    assert perm.tolist() == sorted(range(n), key=lambda i: (part[i], i))


# ------------------------------------------------------------------ compressor
def test_decompress_of_compress_is_the_masked_row_bit_exact(orc):
    wl = synth.make_workload("c1", scale=0.1)
    g = orc.graph(wl.row_ptr, wl.col, wl.part, wl.parts, "gcn")
    F = 64
    X = synth.normal_features(wl.n, F, 5).astype(np.float64)
    for ratio in [(1, 1), (4, 1), (385, 4), (128, 1)]:
        k = orc.kept(F, ratio)
        packed, sent = g.compress(X, ratio, KEY)
        assert packed.shape == (g.H_total, k) and sent == g.H_total * k
        Xh = g.decompress(packed, F, ratio, KEY)
        # walk the receive order (destination, owner, id) and compare with M_j (.) x_j
        slot = 0
        pos = {}
        s = 0
        for p in range(wl.parts):
            for q in range(wl.parts):
                pos[(p, q)] = s
                s += len(g.halo(p, q))
        for q in range(wl.parts):
            for p in range(wl.parts):
                for r, j in enumerate(g.halo(p, q)):
                    idx = orc.wire_positions(*KEY, int(j), F, k)
                    if k < F:       # kept positions: the first k images of the keyed permutation
                        assert np.array_equal(idx, orc.perm_indices(*KEY, int(j), F, k))
                    else:           # full communication: the row as it is
                        assert np.array_equal(idx, np.arange(F))
                    assert np.array_equal(packed[pos[(p, q)] + r], X[j, idx])
                    want = np.zeros(F)
                    want[idx] = X[j, idx]
                    assert np.array_equal(Xh[slot], want)
                    assert np.count_nonzero(Xh[slot]) == k
                    slot += 1
        if k == F:
            assert slot == 0 or np.array_equal(np.sort(Xh, axis=1), np.sort(X[[j for q in range(wl.parts)
                                               for p in range(wl.parts) for j in g.halo(p, q)]], axis=1))


# ------------------------------------------------------------------ brute force on <= 10 nodes
@pytest.mark.parametrize("conv", ["gcn", "sage"])
@pytest.mark.parametrize("seed", [0, 1, 2, 3])
@pytest.mark.parametrize("ratio", [(1, 1), (2, 1), (8, 3), (128, 1)])
def test_layer_matches_dense_brute_force(orc, conv, seed, ratio):
    n, P, F_in, F_out = 10 - seed % 2, 3, 8, 5
    rp, col = tiny_graph(n, 16, seed)
    part = np.random.default_rng(seed + 7).integers(0, P, size=n).astype(np.int32)
    rng = np.random.default_rng(seed + 11)
    X = rng.standard_normal((n, F_in))
    Ws, Wn, b = weights(F_in, F_out, conv == "sage", seed)
    relu = seed % 2 == 0
    g = orc.graph(rp, col, part, P, conv)
    k = orc.kept(F_in, ratio)
    M = masks_for(orc, n, F_in, k, KEY)
    S = dense.dense_operator(rp, col, conv)
    Yd, Aggd = dense.layer_dense(S, part, X, M, Ws, Wn, b, relu)
    Y, Agg, hb = g.layer_fwd(X, Ws, Wn, b, relu, ratio, KEY, elem_bytes=4)
    assert np.allclose(Agg, Aggd, rtol=0, atol=1e-12)
    assert np.allclose(Y, Yd, rtol=0, atol=1e-12)
    assert hb == g.H_total * k * 4
    # single-row evaluation agrees too
    Yr, Aggr = g.layer_fwd_rows(np.arange(n), X, Ws, Wn, b, relu, ratio, KEY)
    assert np.allclose(Yr, Yd, atol=1e-12) and np.allclose(Aggr, Aggd, atol=1e-12)
    # gradients against autograd of the dense formulation
    dY = rng.standard_normal((n, F_out))
    gX, gWs, gWn, gb = dense.layer_dense_grads(S, part, X, M, Ws, Wn, b, relu, dY)
    dX, dWs, dWn, db, hb2 = g.layer_bwd(X, Y, Ws, Wn, dY, relu, ratio, KEY, elem_bytes=2)
    assert np.allclose(dX, gX, atol=1e-12)
    assert np.allclose(dWn, gWn, atol=1e-12)
    assert np.allclose(db, gb, atol=1e-12)
    if conv == "sage":
        assert np.allclose(dWs, gWs, atol=1e-12)
    assert hb2 == g.H_total * k * 2
    dXr = g.layer_dx_rows(np.arange(n), Y, Ws, Wn, dY, relu, ratio, KEY)
    assert np.allclose(dXr, gX, atol=1e-12)


# ------------------------------------------------------------------ full communication == centralized
@pytest.mark.parametrize("conv", ["gcn", "sage"])
def test_full_communication_equals_centralized_layer(orc, conv):
    wl = synth.make_workload("c1", scale=0.15)
    n, F_in, F_out = wl.n, 16, 12
    rng = np.random.default_rng(3)
    X = rng.standard_normal((n, F_in))
    Ws, Wn, b = weights(F_in, F_out, conv == "sage", 4)
    S = dense.dense_operator(wl.row_ptr, wl.col, conv)
    ones = np.ones((n, F_in))
    one_part = np.zeros(n, dtype=np.int32)
    Yc, Aggc = dense.layer_dense(S, one_part, X, ones, Ws, Wn, b, True)     # unpartitioned
    g = orc.graph(wl.row_ptr, wl.col, wl.part, wl.parts, conv)
    Y, Agg, hb = g.layer_fwd(X, Ws, Wn, b, True, (1, 1), KEY)
    assert np.allclose(Y, Yc, atol=1e-12) and np.allclose(Agg, Aggc, atol=1e-12)
    dY = rng.standard_normal((n, F_out))
    gX, gWs, gWn, gb = dense.layer_dense_grads(S, one_part, X, ones, Ws, Wn, b, True, dY)
    dX, dWs, dWn, db, _ = g.layer_bwd(X, Y, Ws, Wn, dY, True, (1, 1), KEY)
    assert np.allclose(dX, gX, atol=1e-11) and np.allclose(dWn, gWn, atol=1e-10) and np.allclose(db, gb, atol=1e-11)
    # and a compressed run is NOT the centralized one (the pin can fail)
    Y4, _, hb4 = g.layer_fwd(X, Ws, Wn, b, True, (4, 1), KEY)
    assert not np.allclose(Y4, Yc, atol=1e-3)
    assert hb4 * 4 == hb


# ------------------------------------------------------------------ finite differences, masks held fixed
def test_backward_matches_central_finite_differences(orc):
    n, P, F_in, F_out = 9, 3, 6, 4
    rp, col = tiny_graph(n, 15, 5)
    part = (np.arange(n) % P).astype(np.int32)
    rng = np.random.default_rng(8)
    X = rng.standard_normal((n, F_in))
    Ws, Wn, b = weights(F_in, F_out, True, 9)
    dY = rng.standard_normal((n, F_out))
    g = orc.graph(rp, col, part, P, "sage")
    ratio = (3, 1)
    # identity activation so that finite differences never straddle a ReLU kink
    loss = lambda X_, Ws_, Wn_, b_: float(np.sum(g.layer_fwd(X_, Ws_, Wn_, b_, False, ratio, KEY)[0] * dY))
    Y = g.layer_fwd(X, Ws, Wn, b, False, ratio, KEY)[0]
    dX, dWs, dWn, db, _ = g.layer_bwd(X, Y, Ws, Wn, dY, False, ratio, KEY)
    eps = 1e-6

    def fd(arr, which):
        out = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            a1, a2 = arr.copy(), arr.copy()
            a1[idx] += eps
            a2[idx] -= eps
            args1 = [X, Ws, Wn, b]
            args2 = [X, Ws, Wn, b]
            args1[which], args2[which] = a1, a2
            out[idx] = (loss(*args1) - loss(*args2)) / (2 * eps)
        return out
    assert np.allclose(fd(X, 0), dX, atol=1e-6)
    assert np.allclose(fd(Ws, 1), dWs, atol=1e-6)
    assert np.allclose(fd(Wn, 2), dWn, atol=1e-6)
    assert np.allclose(fd(b, 3), db, atol=1e-6)


def test_adjoint_identity_of_the_partitioned_aggregation(orc):
    # <Agg(X), G> == <X, Agg^T(G)>: with W_neigh = I, W_self = 0, no activation, the layer is
    # the partitioned, masked aggregation operator and its backward is the adjoint.
    wl = synth.make_workload("c1", scale=0.1)
    n, F = wl.n, 16
    rng = np.random.default_rng(1)
    X, G = rng.standard_normal((n, F)), rng.standard_normal((n, F))
    g = orc.graph(wl.row_ptr, wl.col, wl.part, wl.parts, "sage")
    I, Z = np.eye(F), np.zeros((F, F))
    for ratio in [(1, 1), (4, 1)]:
        Y = g.layer_fwd(X, Z, I, np.zeros(F), False, ratio, KEY)[0]
        dX = g.layer_bwd(X, Y, Z, I, G, False, ratio, KEY)[0]
        assert abs(np.sum(Y * G) - np.sum(X * dX)) < 1e-9 * max(1.0, abs(np.sum(Y * G)))


# ------------------------------------------------------------------ communicated volume
def test_bytes_follow_the_rate_versus_volume_formula(orc):
    # efficiency section: the volume per round is the boundary size times the compression
    # coefficient, constant for a fixed ratio and equal to full communication x k/F.
    wl = synth.make_workload("c1", scale=0.2)
    g = orc.graph(wl.row_ptr, wl.col, wl.part, wl.parts, "gcn")
    F_in, F_out = 64, 8
    X = synth.normal_features(wl.n, F_in, 1).astype(np.float64)
    _, Wn, b = weights(F_in, F_out, False, 2)
    full = g.layer_fwd(X, None, Wn, b, True, (1, 1), (9, 0, 0), elem_bytes=4)[2]
    assert full == g.H_total * F_in * 4
    for ratio in [(2, 1), (4, 1), (64, 1)]:
        per_epoch = [g.layer_fwd(X, None, Wn, b, True, ratio, (9, e, 0), elem_bytes=4)[2] for e in range(3)]
        k = orc.kept(F_in, ratio)
        assert per_epoch == [full * k // F_in] * 3
    K = 20
    total = 0
    for e in range(K):
        ratio = orc.schedule_linear(e, K)
        Y, _, hb = g.layer_fwd(X, None, Wn, b, True, ratio, (9, e, 0), elem_bytes=4)
        hb2 = g.layer_bwd(X, Y, None, Wn, np.ones_like(Y), True, ratio, (9, e, 0), elem_bytes=4)[4]
        assert hb == hb2 == g.H_total * orc.kept(F_in, ratio) * 4
        total += hb + hb2
    ks = [orc.kept(F_in, orc.schedule_linear(e, K)) for e in range(K)]
    assert ks[:5] == [1, 1, 1, 2, 64] and ks[-1] == 64
    assert total == 2 * 4 * g.H_total * sum(ks) < 2 * K * full
