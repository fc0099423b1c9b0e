"""Host-side checks of the C-ABI library: exported symbols, plan builder against the oracle's
partition sets (bit-exact), rate helpers, error codes.  No GPU needed."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2406_17611_b200 import binding as vb
from paper_2406_17611_b200 import build as vbuild
from paper_2406_17611_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    vbuild.build()


def test_library_exports_every_declared_symbol():
    text = open(os.path.join(ROOT, "include", "varco.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = sorted(set(re.findall(r"\b(varco_[a-z_0-9]+)\s*\(", text)))
    assert len(declared) >= 19
    L = C.CDLL(vb.LIB_PATH)
    for name in declared:
        assert hasattr(L, name), name
    assert sorted(vb.EXPORTS) == declared


@pytest.mark.parametrize("name,scale", [("c1", 1.0), ("c2", 0.05), ("c2r", 0.05), ("c3", 0.004), ("c4", 0.02)])
def test_plan_matches_oracle_partition_bit_exact(orc, name, scale):
    wl = synth.make_workload(name, scale)
    plan = vb.Plan(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv)
    g = orc.graph(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv)
    assert (plan.n, plan.nnz, plan.P) == (wl.n, wl.nnz, wl.parts)
    assert plan.H_total == g.H_total
    assert plan.cross_entries == g.cross_entries and plan.self_entries == g.self_entries
    assert np.array_equal(plan.counts(), g.counts())
    assert np.array_equal(plan.perm(), g.perm())
    for p in range(wl.parts):
        for q in range(wl.parts):
            assert np.array_equal(plan.halo(p, q), g.halo(p, q))
    plan.close()


def test_rate_helpers_match_oracle(orc):
    for F in (1, 47, 64, 100, 256, 602):
        for K, a in [(20, 5), (100, 5), (300, 5), (300, 2), (300, 7)]:
            for e in range(0, K, max(1, K // 23)):
                r = vb.varco_schedule_linear(e, K, a)
                assert r == orc.schedule_linear(e, K, a)
                assert vb.varco_kept(F, r) == orc.kept(F, r)
    # worked values: K=100, a=5 -> c_e = 128 - 6.35 e; F=256 keeps 2, 3, ... 35 (e=19), 256 (e>=20)
    # the other schedulers of the appendix, the fixed ratios of Section V and "no communication"
    for r0, al, den in [(1, 1, 128), (1, 3, 64), (5, 7, 300), (2, 0, 9)]:
        for e in list(range(0, 140, 7)) + [10**6]:
            r = vb.varco_schedule_rate_linear(e, r0, al, den)
            assert r == orc.schedule_rate_linear(e, r0, al, den) == orc.schedule_fixed_increment(min(e, 5000), r0, al, den) \
                or (e > 5000 and r == orc.schedule_rate_linear(e, r0, al, den))
            assert vb.varco_kept(100, r) == orc.kept(100, r)
    for beta, K in [(2, 7), (3, 5), (10, 20)]:
        for e in range(K + 3):
            r = vb.varco_schedule_exponential(e, K, beta)
            assert r == orc.schedule_exponential(e, K, beta)
            assert vb.varco_kept(256, r) == orc.kept(256, r)
    for F in (8, 47, 100, 256, 602):
        assert vb.varco_kept(F, vb.NO_COMMUNICATION) == orc.kept(F, (1, 0)) == 0
        for c in (2, 4):
            assert vb.varco_kept(F, (c, 1)) == orc.kept(F, (c, 1)) == -(-F // c)
    ks = [vb.varco_kept(256, vb.varco_schedule_linear(e, 100)) for e in range(22)]
    assert ks[0] == 2 and ks[1] == 3 and ks[19] == 35 and ks[20] == ks[21] == 256
    assert vb.varco_kept(256, vb.varco_schedule_linear(59, 300)) == 83


def test_error_codes():
    L = vb.lib()
    rp = np.array([0, 1, 2], dtype=np.int64)
    col = np.array([1, 0], dtype=np.int32)
    part = np.array([0, 1], dtype=np.int32)

    def build(rp, col, part, P=2, conv=1):
        h = C.c_void_p()
        st = L.varco_partition_build(len(rp) - 1, rp.ctypes.data_as(C.POINTER(C.c_int64)),
                                     col.ctypes.data_as(C.POINTER(C.c_int32)),
                                     part.ctypes.data_as(C.POINTER(C.c_int32)), P, conv, C.byref(h))
        if st == 0:
            L.varco_partition_destroy(h)
        return st
    assert build(rp, col, part) == 0
    assert build(np.array([0, 2, 1], dtype=np.int64), col, part) == -2          # row_ptr not monotone
    assert build(np.array([1, 1, 2], dtype=np.int64), col, part) == -2          # does not start at 0
    assert build(rp, np.array([2, 0], dtype=np.int32), part) == -2              # column out of range
    assert build(rp, np.array([0, 0], dtype=np.int32), part) == -2              # diagonal entry
    assert build(np.array([0, 2, 2], dtype=np.int64), np.array([1, 1], dtype=np.int32), part) == -2   # duplicate
    assert build(rp, col, np.array([0, 2], dtype=np.int32)) == -3               # label out of range
    assert build(rp, col, part, P=0) == -1
    assert build(rp, col, part, conv=5) == -1
    with pytest.raises(vb.VarcoError):
        vb.varco_kept(64, (1, 2))
    with pytest.raises(vb.VarcoError):
        vb.varco_schedule_linear(0, 0)
    assert L.varco_status_string(-6) == b"workspace too small"
    # device entry points refuse a plan that has no device image, without touching the GPU
    plan = vb.Plan(rp, col, part, 2, "sage")
    d = vb.LayerDesc(1, 0, 4, 4, 1, 4, 4)
    buf = (C.c_float * 64)()
    st = L.varco_layer_fwd(plan.h, C.byref(d), buf, buf, buf, None, buf, buf, vb.Ratio(1, 1), vb.Key(0, 0, 0), buf,
                           1 << 20, None, None)
    assert st == -8
    nbytes = C.c_size_t()
    assert L.varco_workspace_bytes(plan.h, 4096, 4, 0, C.byref(nbytes)) == -7
    assert L.varco_workspace_bytes(plan.h, 64, 64, 0, C.byref(nbytes)) == 0 and nbytes.value > 0
    plan.close()


def test_gather_model_matches_brute_force():
    """Rows read under the static-residency cache model, against a direct count of (partition, source) uses."""
    wl = synth.make_workload("c3", 0.004)
    plan = vb.Plan(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv)
    rows = np.repeat(np.arange(wl.n), np.diff(wl.row_ptr))
    dest = wl.part[rows].astype(np.int64)
    for transposed in (False, True):
        src = rows if transposed else wl.col.astype(np.int64)
        _, cnt = np.unique(dest * wl.n + src, return_counts=True)
        part_of = np.unique(dest * wl.n + src) // wl.n
        for keep in (0, 7, 300, 10 ** 9):
            want = 0
            for q in range(wl.parts):
                c = np.sort(cnt[part_of == q])[::-1]
                want += min(keep, len(c)) + int(c[keep:].sum())
            e, s_, r = plan.gather_model(keep, transposed)
            assert (e, s_, r) == (int(cnt.sum()), len(cnt), want)
    plan.close()


def test_halo_bytes_of_the_100_epoch_schedule_follow_the_closed_form(orc):
    """The rate-sweep configuration (4-layer SAGE 100-256-256-256-47, bf16, schedule K = 100, slope 5): for every
    epoch the bytes of one epoch, forward and backward, are 2 * sum_l H_total * k_l * s -- the library's plan
    and rate helpers against the oracle's, all 100 epochs; and the oracle's own byte counter (which counts values
    as they are sent) agrees with the closed form at the schedule's corner epochs."""
    wl = synth.make_workload("c5", 0.001)
    plan = vb.Plan(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv)
    g = orc.graph(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv)
    assert plan.H_total == g.H_total
    widths, es = wl.widths, 2
    total_lib = total_orc = 0
    for e in range(100):
        r = vb.varco_schedule_linear(e, 100, 5)
        assert r == orc.schedule_linear(e, 100, 5)
        ks = [vb.varco_kept(F, r) for F in widths[:-1]]
        assert ks == [orc.kept(F, r) for F in widths[:-1]]
        total_lib += 2 * sum(plan.H_total * k * es for k in ks)
        total_orc += 2 * sum(g.H_total * orc.kept(F, r) * es for F in widths[:-1])
        if e >= 20:
            assert ks == widths[:-1]                       # full communication from epoch K / a on
    assert total_lib == total_orc
    full = 2 * sum(plan.H_total * F * es for F in widths[:-1])
    assert total_lib < 100 * full and total_lib > 80 * full
    for e in (0, 1, 19, 20):
        r = orc.schedule_linear(e, 100, 5)
        sent = 0
        for l in range(4):
            X = synth.normal_features(wl.n, widths[l], 3, True)
            Ws, Wn, b = wl.layer_weights(l)
            Y, _, hb = g.layer_fwd(X, Ws, Wn, b, l < 3, r, (1, e, l), elem_bytes=es)
            dY = np.ones((wl.n, widths[l + 1]))
            hb2 = g.layer_bwd(X, Y, Ws, Wn, dY, l < 3, r, (1, e, l), elem_bytes=es)[4]
            sent += hb + hb2
        assert sent == 2 * sum(g.H_total * orc.kept(F, r) * es for F in widths[:-1])
    plan.close()
