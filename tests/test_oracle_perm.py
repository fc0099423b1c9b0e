"""Pins for the oracle's shared-key permutation, compressor and scheduler."""
import os
from fractions import Fraction

import numpy as np
import pytest

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _vectors():
    out = {"idx": [], "rk0": [], "mix": []}
    for line in open(os.path.join(GOLD, "keyed_perm_vectors.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tok = line.split()
        if tok[0] == "mix64":
            out["mix"].append((int(tok[1]), int(tok[2], 16)))
        elif tok[0] == "rk0":
            out["rk0"].append(tuple(int(x) for x in tok[1:6]) + (int(tok[6], 16),))
        else:
            head, tail = line.split("|")
            out["idx"].append((tuple(int(x) for x in head.split()), [int(x) for x in tail.split()]))
    return out


def test_keyed_permutation_test_vectors(orc):
    v = _vectors()
    assert len(v["idx"]) == 6
    for (seed, t, l, node, F, k), want in v["idx"]:
        assert orc.perm_indices(seed, t, l, node, F, k).tolist() == want
    for x, want in v["mix"]:
        assert orc.mix64(x) == want
    for seed, t, l, node, F, want in v["rk0"]:
        assert int(orc.round_keys(seed, t, l, node, F)[0]) == want


@pytest.mark.parametrize("F", [1, 2, 3, 8, 47, 64, 100, 128, 256, 602])
def test_permutation_is_a_bijection_with_inverse(orc, F):
    for node in (0, 5, 2449028):
        idx = orc.perm_indices(99, 3, 1, node, F, F)
        assert sorted(idx.tolist()) == list(range(F))
        for m in range(0, F, max(1, F // 17)):
            assert orc.perm_inverse(99, 3, 1, node, F, int(idx[m])) == m


def test_prefix_property(orc):
    # the k kept positions at a lower ratio extend those at a higher ratio (same key)
    full = orc.perm_indices(7, 2, 0, 11, 256, 256)
    for k in (1, 4, 35, 255):
        assert orc.perm_indices(7, 2, 0, 11, 256, k).tolist() == full[:k].tolist()


def test_key_separates_epoch_layer_node_seed(orc):
    base = orc.perm_indices(1, 1, 1, 1, 256, 32).tolist()
    assert orc.perm_indices(2, 1, 1, 1, 256, 32).tolist() != base
    assert orc.perm_indices(1, 2, 1, 1, 256, 32).tolist() != base
    assert orc.perm_indices(1, 1, 2, 1, 256, 32).tolist() != base
    assert orc.perm_indices(1, 1, 1, 2, 256, 32).tolist() != base


@pytest.mark.parametrize("F,k", [(64, 8), (100, 14), (256, 35), (602, 60)])
def test_subset_is_close_to_uniform(orc, F, k):
    # A uniform random k-subset keeps every column with probability k/F, and for
    # x ~ N(0,1) the squared error of decompress(compress(x)) has mean F - k,
    # i.e. (1 - k/F) ||x||^2: the epsilon^2 of Definition 1, growing with the ratio.
    rows = 6000
    hits = np.zeros(F)
    rng = np.random.default_rng(0)
    err = 0.0
    for node in range(rows):
        idx = orc.perm_indices(5, 0, 0, node, F, k)
        hits[idx] += 1
        x = rng.standard_normal(F)
        m = np.zeros(F)
        m[idx] = 1
        err += np.sum((x - m * x) ** 2)
    p = k / F
    sd = np.sqrt(rows * p * (1 - p))
    assert np.all(np.abs(hits - rows * p) < 5.5 * sd)
    chi2 = np.sum((hits - rows * p) ** 2 / (rows * p * (1 - p))) / F
    assert 0.55 < chi2 < 1.45
    assert abs(err / rows - (F - k)) < 0.05 * (F - k)


def test_consecutive_epochs_overlap_like_independent_draws(orc):
    F, k, rows = 256, 32, 4000
    ov = 0
    for node in range(rows):
        a = set(orc.perm_indices(5, 3, 0, node, F, k).tolist())
        b = set(orc.perm_indices(5, 4, 0, node, F, k).tolist())
        ov += len(a & b)
    assert abs(ov / rows - k * k / F) < 0.15 * k * k / F


# ------------------------------------------------------------------ kept elements and schedule
def test_kept_is_ceil_of_width_over_ratio(orc):
    for F in (1, 8, 64, 100, 256, 602):
        for num, den in [(1, 1), (2, 1), (4, 1), (64, 1), (128, 1), (385, 4), (2560 - 127 * 5, 20), (935, 300)]:
            want = min(F, max(1, -(-F * den // num)))
            assert orc.kept(F, (num, den)) == want
            assert Fraction(F) / Fraction(num, den) <= want or want == F
    assert orc.kept(64, (1, 2)) == -1      # ratio below 1 is not a compression ratio
    assert orc.kept(64, (0, 1)) == -1


def _paper_schedule():
    d = {}
    for line in open(os.path.join(GOLD, "paper_schedule.txt")):
        if line.strip() and not line.startswith("#"):
            tok = line.split()
            d[tok[0]] = [int(x) for x in tok[1:]]
    return d


def test_schedule_paper_setting_reaches_full_communication(orc):
    d = _paper_schedule()
    K, a, cmax, cmin = d["K"][0], d["a"][0], d["c_max"][0], d["c_min"][0]
    c = [Fraction(*orc.schedule_linear(e, K, a, cmax, cmin)) for e in range(K)]
    assert c[0] == cmax
    # a straight line of slope a*(c_max-c_min)/K until it reaches c_min at e = K/a
    for e in range(K // a):
        assert c[e] == cmax - Fraction(a * (cmax - cmin) * e, K)
        assert c[e + 1] < c[e]
    assert all(x == cmin for x in c[K // a:])
    assert c[K // a - 1] > cmin
    assert c[-1] == cmin                   # ends at full communication
    for slope in d["slopes"]:
        cs = [Fraction(*orc.schedule_linear(e, K, slope, cmax, cmin)) for e in range(K)]
        assert all(cs[i + 1] <= cs[i] for i in range(K - 1))
        first_full = next(i for i, x in enumerate(cs) if x == cmin)
        assert first_full == -(-K // slope)


def test_schedule_slope_one_is_the_plain_linear_scheduler(orc):
    # Section IV: r_lin(t) = (c_min - c_max)/T * t + c_max
    T, cmax, cmin = 50, 128, 1
    for t in range(T):
        assert Fraction(*orc.schedule_linear(t, T, 1, cmax, cmin)) == Fraction(cmin - cmax, T) * t + cmax


def test_schedule_rejects_bad_arguments(orc):
    for args in [(0, 0, 5, 128, 1), (0, 10, 0, 128, 1), (0, 10, 5, 1, 2), (-1, 10, 5, 128, 1), (0, 10, 5, 128, 0)]:
        with pytest.raises(ValueError):
            orc.schedule_linear(*args)
