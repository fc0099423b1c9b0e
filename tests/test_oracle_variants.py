"""Pins for the scheduler variants of the appendix "Scheduler", the fixed ratios of Section V and the
"no communication" setting (Tables II-III): worked values written out by hand from the paper's three
formulas, closed forms with exact fractions, and dense brute force with all-zero masks."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import dense

from test_oracle_layer import KEY, tiny_graph, weights

GOLD = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
NO_COMM = (1, 0)


def _rows():
    out = []
    for line in open(os.path.join(GOLD, "scheduler_variants.txt")):
        if line.strip() and not line.startswith("#"):
            out.append(line.split())
    return out


def _frac(tok):
    a, b = tok.split("/")
    return int(a), int(b)


def test_worked_values_of_the_three_rate_schedules(orc):
    seen = set()
    for tok in _rows():
        name = tok[0]
        if name == "fixed_inc":
            (r0, den), (R, den2) = _frac(tok[1].split("=")[1]), _frac(tok[2].split("=")[1])
            assert den == den2
            for item in tok[3:]:
                e, want = item.split(":")
                assert orc.schedule_fixed_increment(int(e), r0, R, den) == _frac(want)
        elif name == "linear":
            (r0, den), (al, den2) = _frac(tok[1].split("=")[1]), _frac(tok[2].split("=")[1])
            assert den == den2
            for item in tok[3:]:
                e, want = item.split(":")
                assert orc.schedule_rate_linear(int(e), r0, al, den) == _frac(want)
        elif name == "exponential":
            beta, K = int(tok[1].split("=")[1]), int(tok[2].split("=")[1])
            for item in tok[3:]:
                e, want = item.split(":")
                assert orc.schedule_exponential(int(e), K, beta) == _frac(want)
        elif name == "kept":
            F = int(tok[1].split("=")[1])
            for item in tok[2:]:
                ratio, want = item.split(":")
                assert orc.kept(F, _frac(ratio)) == int(want)
        seen.add(name)
    assert seen == {"fixed_inc", "linear", "exponential", "kept"}


@pytest.mark.parametrize("r0,step,den", [(1, 1, 128), (1, 3, 64), (5, 7, 300), (2, 0, 9), (9, 4, 9)])
def test_recurrence_equals_closed_form_and_is_monotone(orc, r0, step, den):
    prev = None
    for e in range(0, 400, 3):
        rec = orc.schedule_fixed_increment(e, r0, step, den)
        lin = orc.schedule_rate_linear(e, r0, step, den)
        assert rec == lin
        rate = min(Fraction(1), Fraction(r0 + step * e, den))       # the appendix's formula, clipped at 1
        assert Fraction(rec[1], rec[0]) == rate
        assert Fraction(*rec) >= 1                                   # a ratio the compressor accepts
        if prev is not None:
            assert Fraction(*rec) <= prev                            # rate up, ratio down
        prev = Fraction(*rec)
    if step > 0:
        assert orc.schedule_rate_linear(10**6, r0, step, den) == (den, den)   # ends at full communication
        first_full = -(-(den - r0) // step)
        assert orc.schedule_rate_linear(first_full, r0, step, den) == (den, den)
        if first_full > 0:
            assert Fraction(*orc.schedule_rate_linear(first_full - 1, r0, step, den)) > 1


def test_exponential_schedule(orc):
    for beta, K in [(2, 7), (3, 5), (10, 20)]:
        prev = None
        for e in range(K + 3):
            num, den = orc.schedule_exponential(e, K, beta)
            assert den == 1 and num == min(beta ** max(K - e, 0), 2**32 - 1)
            if prev is not None:
                assert num <= prev
            prev = num
        assert orc.schedule_exponential(K - 1, K, beta) == (beta, 1)   # the last step still compresses by beta
    assert orc.kept(256, orc.schedule_exponential(0, 20, 10)) == 1     # saturated ratio keeps one element
    for bad in [(-1, 5, 2), (0, 0, 2), (0, 5, 1)]:
        with pytest.raises(ValueError):
            orc.schedule_exponential(*bad)
    with pytest.raises(ValueError):
        orc.schedule_rate_linear(0, 0, 1, 8)
    with pytest.raises(ValueError):
        orc.schedule_fixed_increment(0, 9, 1, 8)


def test_bytes_of_fixed_ratio_and_no_communication_runs(orc):
    n, P, F = 10, 3, 8
    rp, col = tiny_graph(n, 16, 4)
    part = (np.arange(n) % P).astype(np.int32)
    g = orc.graph(rp, col, part, P, "sage")
    X = np.random.default_rng(0).standard_normal((n, F))
    Ws, Wn, b = weights(F, 5, True, 1)
    full = g.layer_fwd(X, Ws, Wn, b, True, (1, 1), KEY, elem_bytes=4)[2]
    assert full == g.H_total * F * 4
    for c in (2, 4):     # fixed compression: the same volume every epoch, full volume / c
        per_epoch = {g.layer_fwd(X, Ws, Wn, b, True, (c, 1), (KEY[0], e, 0), elem_bytes=4)[2] for e in range(5)}
        assert per_epoch == {full // c}
    assert g.layer_fwd(X, Ws, Wn, b, True, NO_COMM, KEY, elem_bytes=4)[2] == 0
    packed, sent = g.compress(X, NO_COMM, KEY)
    assert packed.shape == (g.H_total, 0) and sent == 0
    assert not g.decompress(packed, F, NO_COMM, KEY).any()


@pytest.mark.parametrize("conv", ["gcn", "sage"])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_no_communication_layer_matches_dense_brute_force(orc, conv, seed):
    """Nothing sent: every remote neighbour contributes the zero vector (all-zero masks), degrees stay those
    of the whole graph.  Forward and autograd gradients of the dense formulation."""
    n, P, F_in, F_out = 10 - seed % 2, 3, 8, 5
    rp, col = tiny_graph(n, 16, seed)
    part = np.random.default_rng(seed + 7).integers(0, P, size=n).astype(np.int32)
    rng = np.random.default_rng(seed + 11)
    X = rng.standard_normal((n, F_in))
    Ws, Wn, b = weights(F_in, F_out, conv == "sage", seed)
    relu = seed % 2 == 0
    g = orc.graph(rp, col, part, P, conv)
    S = dense.dense_operator(rp, col, conv)
    M = np.zeros((n, F_in))
    Yd, Aggd = dense.layer_dense(S, part, X, M, Ws, Wn, b, relu)
    # the same thing said differently: the operator with every cross-partition entry removed
    same = (part[:, None] == part[None, :])
    assert np.allclose(Aggd, (S * same) @ X, atol=1e-14)
    Y, Agg, hb = g.layer_fwd(X, Ws, Wn, b, relu, NO_COMM, KEY, elem_bytes=4)
    assert hb == 0
    assert np.allclose(Agg, Aggd, atol=1e-12) and np.allclose(Y, Yd, atol=1e-12)
    Yr, Aggr = g.layer_fwd_rows(np.arange(n), X, Ws, Wn, b, relu, NO_COMM, KEY)
    assert np.allclose(Yr, Yd, atol=1e-12) and np.allclose(Aggr, Aggd, atol=1e-12)
    dY = rng.standard_normal((n, F_out))
    gX, gWs, gWn, gb = dense.layer_dense_grads(S, part, X, M, Ws, Wn, b, relu, dY)
    dX, dWs, dWn, db, hb2 = g.layer_bwd(X, Y, Ws, Wn, dY, relu, NO_COMM, KEY, elem_bytes=2)
    assert hb2 == 0
    assert np.allclose(dX, gX, atol=1e-12) and np.allclose(dWn, gWn, atol=1e-12) and np.allclose(db, gb, atol=1e-12)
    if conv == "sage":
        assert np.allclose(dWs, gWs, atol=1e-12)
    assert np.allclose(g.layer_dx_rows(np.arange(n), Y, Ws, Wn, dY, relu, NO_COMM, KEY), gX, atol=1e-12)
    # and it differs from the full-communication layer whenever an edge crosses partitions (the pin can fail)
    if g.cross_entries:
        assert not np.allclose(g.layer_fwd(X, Ws, Wn, b, relu, (1, 1), KEY)[1], Aggd, atol=1e-6)
