"""ctypes access to the C++ oracle (test infrastructure only)."""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "varco_oracle.cpp")
_LIB = os.path.join(_HERE, "libvarco_oracle.so")

GCN, SAGE = 0, 1


def build_oracle(force: bool = False) -> str:
    """Compile the oracle with g++ (-O2, OpenMP) if the library is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fopenmp", "-shared", "-fPIC", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


def _p(a, t):
    return a.ctypes.data_as(C.POINTER(t)) if a is not None else None


def _f64(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


class Oracle:
    """Scalar helpers: keyed permutation, kept elements, schedule."""

    def __init__(self):
        self.lib = C.CDLL(build_oracle())
        L = self.lib
        L.orc_mix64.restype = C.c_uint64
        L.orc_mix64.argtypes = [C.c_uint64]
        L.orc_perm_indices.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint64, C.c_int, C.c_int,
                                       C.POINTER(C.c_int32)]
        L.orc_wire_positions.argtypes = L.orc_perm_indices.argtypes
        L.orc_perm_inverse.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint64, C.c_int, C.c_int]
        L.orc_round_keys.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint64, C.c_int, C.POINTER(C.c_uint32)]
        L.orc_kept.argtypes = [C.c_int, C.c_uint64, C.c_uint64]
        L.orc_schedule_linear.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_uint64),
                                          C.POINTER(C.c_uint64)]
        L.orc_graph_create.restype = C.c_void_p
        L.orc_graph_create.argtypes = [C.c_int64, C.POINTER(C.c_int64), C.POINTER(C.c_int32), C.POINTER(C.c_int32),
                                       C.c_int, C.c_int]
        L.orc_graph_destroy.argtypes = [C.c_void_p]
        for name in ("orc_graph_H_total", "orc_graph_cross_entries", "orc_graph_self_entries"):
            getattr(L, name).restype = C.c_int64
            getattr(L, name).argtypes = [C.c_void_p]
        L.orc_graph_counts.argtypes = [C.c_void_p, C.POINTER(C.c_int64)]
        L.orc_graph_halo.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_int64)]
        L.orc_graph_perm.argtypes = [C.c_void_p, C.POINTER(C.c_int64)]
        dp = C.POINTER(C.c_double)
        key = [C.c_uint64, C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint32]  # num, den, seed, epoch, layer
        L.orc_compress.argtypes = [C.c_void_p, dp, C.c_int] + key + [dp, C.POINTER(C.c_uint64)]
        L.orc_decompress.argtypes = [C.c_void_p, dp, C.c_int] + key + [dp]
        L.orc_layer_fwd.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, dp, dp, dp, dp] + key + \
                                   [C.c_int, dp, dp, C.POINTER(C.c_uint64)]
        L.orc_layer_bwd.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, dp, dp, dp, dp, dp] + key + \
                                   [C.c_int, dp, dp, dp, dp, C.POINTER(C.c_uint64)]
        L.orc_layer_fwd_rows.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, dp, dp, dp, dp] + key + \
                                        [C.POINTER(C.c_int64), C.c_int64, dp, dp]
        L.orc_layer_dx_rows.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, dp, dp, dp, dp] + key + \
                                       [C.POINTER(C.c_int64), C.c_int64, dp]
        L.orc_set_threads.argtypes = [C.c_int]
        L.orc_get_threads.restype = C.c_int

    # -- scalars
    def mix64(self, x):
        return int(self.lib.orc_mix64(C.c_uint64(x & (2**64 - 1))))

    def perm_indices(self, seed, epoch, layer, node, F, k):
        out = np.empty(k, dtype=np.int32)
        rc = self.lib.orc_perm_indices(seed, epoch, layer, node, F, k, _p(out, C.c_int32))
        if rc != 0:
            raise ValueError("bad permutation arguments")
        return out

    def wire_positions(self, seed, epoch, layer, node, F, k):
        out = np.empty(k, dtype=np.int32)
        rc = self.lib.orc_wire_positions(seed, epoch, layer, node, F, k, _p(out, C.c_int32))
        if rc != 0:
            raise ValueError("bad arguments")
        return out

    def perm_inverse(self, seed, epoch, layer, node, F, c):
        return int(self.lib.orc_perm_inverse(seed, epoch, layer, node, F, c))

    def round_keys(self, seed, epoch, layer, node, F):
        out = np.empty(6, dtype=np.uint32)
        self.lib.orc_round_keys(seed, epoch, layer, node, F, _p(out, C.c_uint32))
        return out

    def kept(self, F, ratio):
        return int(self.lib.orc_kept(F, ratio[0], ratio[1]))

    def schedule_linear(self, epoch, K, a=5, c_max=128, c_min=1):
        num, den = C.c_uint64(), C.c_uint64()
        rc = self.lib.orc_schedule_linear(epoch, K, a, c_max, c_min, C.byref(num), C.byref(den))
        if rc != 0:
            raise ValueError("bad schedule arguments")
        return int(num.value), int(den.value)

    def schedule_fixed_increment(self, epoch, r0, R, den):
        """Ratio (num, den) of the fixed-increment rate schedule r_{k+1} = r_k + R/den, r_0 = r0/den."""
        num, d = C.c_uint64(), C.c_uint64()
        rc = self.lib.orc_schedule_fixed_increment(epoch, C.c_uint64(r0), C.c_uint64(R), C.c_uint64(den),
                                                   C.byref(num), C.byref(d))
        if rc != 0:
            raise ValueError("bad schedule arguments")
        return int(num.value), int(d.value)

    def schedule_rate_linear(self, epoch, r0, alpha, den):
        """Ratio (num, den) of the linear rate schedule r_k = (alpha k + r0) / den, clipped at 1."""
        num, d = C.c_uint64(), C.c_uint64()
        rc = self.lib.orc_schedule_rate_linear(epoch, C.c_uint64(r0), C.c_uint64(alpha), C.c_uint64(den),
                                               C.byref(num), C.byref(d))
        if rc != 0:
            raise ValueError("bad schedule arguments")
        return int(num.value), int(d.value)

    def schedule_exponential(self, epoch, K, beta):
        """Ratio (num, 1) of the exponential rate schedule r_k = beta^-(K - k + 1), k = epoch + 1."""
        num, d = C.c_uint64(), C.c_uint64()
        rc = self.lib.orc_schedule_exponential(epoch, K, beta, C.byref(num), C.byref(d))
        if rc != 0:
            raise ValueError("bad schedule arguments")
        return int(num.value), int(d.value)

    def set_threads(self, t):
        self.lib.orc_set_threads(t)

    def threads(self):
        return int(self.lib.orc_get_threads())

    def graph(self, row_ptr, col, part, P, conv):
        return OracleGraph(self, row_ptr, col, part, P, conv)


class OracleGraph:
    """A graph with partition labels; every array is in ORIGINAL node order."""

    def __init__(self, orc: Oracle, row_ptr, col, part, P, conv):
        self.o = orc
        self.lib = orc.lib
        self.rp = np.ascontiguousarray(row_ptr, dtype=np.int64)
        self.col = np.ascontiguousarray(col, dtype=np.int32)
        self.part = np.ascontiguousarray(part, dtype=np.int32)
        self.n = self.rp.shape[0] - 1
        self.P = int(P)
        self.conv = GCN if conv in (GCN, "gcn") else SAGE
        self.h = self.lib.orc_graph_create(self.n, _p(self.rp, C.c_int64), _p(self.col, C.c_int32),
                                           _p(self.part, C.c_int32), self.P, self.conv)

    def __del__(self):
        try:
            if self.h:
                self.lib.orc_graph_destroy(self.h)
                self.h = None
        except Exception:
            pass

    @property
    def H_total(self):
        return int(self.lib.orc_graph_H_total(self.h))

    @property
    def cross_entries(self):
        return int(self.lib.orc_graph_cross_entries(self.h))

    @property
    def self_entries(self):
        return int(self.lib.orc_graph_self_entries(self.h))

    def counts(self):
        out = np.zeros((self.P, self.P), dtype=np.int64)
        self.lib.orc_graph_counts(self.h, _p(out, C.c_int64))
        return out

    def halo(self, p, q):
        cnt = int(self.counts()[p, q])
        out = np.empty(cnt, dtype=np.int64)
        if cnt:
            self.lib.orc_graph_halo(self.h, p, q, _p(out, C.c_int64))
        return out

    def perm(self):
        out = np.empty(self.n, dtype=np.int64)
        self.lib.orc_graph_perm(self.h, _p(out, C.c_int64))
        return out

    def compress(self, X, ratio, key):
        X = _f64(X)
        F = X.shape[1]
        k = self.o.kept(F, ratio)
        packed = np.zeros((self.H_total, k), dtype=np.float64)
        sent = C.c_uint64()
        rc = self.lib.orc_compress(self.h, _p(X, C.c_double), F, ratio[0], ratio[1], key[0], key[1], key[2],
                                   _p(packed, C.c_double), C.byref(sent))
        assert rc == 0
        return packed, int(sent.value)

    def decompress(self, packed, F, ratio, key):
        packed = _f64(packed)
        out = np.zeros((self.H_total, F), dtype=np.float64)
        rc = self.lib.orc_decompress(self.h, _p(packed, C.c_double), F, ratio[0], ratio[1], key[0], key[1], key[2],
                                     _p(out, C.c_double))
        assert rc == 0
        return out

    def layer_fwd(self, X, W_self, W_neigh, bias, relu, ratio, key, elem_bytes=4):
        X, W_self, W_neigh, bias = _f64(X), _f64(W_self), _f64(W_neigh), _f64(bias)
        F_in, F_out = W_neigh.shape
        Y = np.zeros((self.n, F_out))
        Agg = np.zeros((self.n, F_in))
        hb = C.c_uint64()
        rc = self.lib.orc_layer_fwd(self.h, F_in, F_out, int(relu), _p(X, C.c_double), _p(W_self, C.c_double),
                                    _p(W_neigh, C.c_double), _p(bias, C.c_double), ratio[0], ratio[1], key[0],
                                    key[1], key[2], elem_bytes, _p(Y, C.c_double), _p(Agg, C.c_double),
                                    C.byref(hb))
        assert rc == 0
        return Y, Agg, int(hb.value)

    def layer_bwd(self, X, Y, W_self, W_neigh, dY, relu, ratio, key, elem_bytes=4):
        X, Y, W_self, W_neigh, dY = _f64(X), _f64(Y), _f64(W_self), _f64(W_neigh), _f64(dY)
        F_in, F_out = W_neigh.shape
        dX = np.zeros((self.n, F_in))
        dWs = np.zeros((F_in, F_out)) if self.conv == SAGE else None
        dWn = np.zeros((F_in, F_out))
        db = np.zeros(F_out)
        hb = C.c_uint64()
        rc = self.lib.orc_layer_bwd(self.h, F_in, F_out, int(relu), _p(X, C.c_double), _p(Y, C.c_double),
                                    _p(W_self, C.c_double), _p(W_neigh, C.c_double), _p(dY, C.c_double), ratio[0],
                                    ratio[1], key[0], key[1], key[2], elem_bytes, _p(dX, C.c_double),
                                    _p(dWs, C.c_double), _p(dWn, C.c_double), _p(db, C.c_double), C.byref(hb))
        assert rc == 0
        return dX, dWs, dWn, db, int(hb.value)

    def layer_fwd_rows(self, rows, X, W_self, W_neigh, bias, relu, ratio, key):
        X, W_self, W_neigh, bias = _f64(X), _f64(W_self), _f64(W_neigh), _f64(bias)
        rows = np.ascontiguousarray(rows, dtype=np.int64)
        F_in, F_out = W_neigh.shape
        Y = np.zeros((rows.shape[0], F_out))
        Agg = np.zeros((rows.shape[0], F_in))
        rc = self.lib.orc_layer_fwd_rows(self.h, F_in, F_out, int(relu), _p(X, C.c_double), _p(W_self, C.c_double),
                                         _p(W_neigh, C.c_double), _p(bias, C.c_double), ratio[0], ratio[1], key[0],
                                         key[1], key[2], _p(rows, C.c_int64), rows.shape[0], _p(Y, C.c_double),
                                         _p(Agg, C.c_double))
        assert rc == 0
        return Y, Agg

    def layer_dx_rows(self, rows, Y, W_self, W_neigh, dY, relu, ratio, key):
        Y, W_self, W_neigh, dY = _f64(Y), _f64(W_self), _f64(W_neigh), _f64(dY)
        rows = np.ascontiguousarray(rows, dtype=np.int64)
        F_in, F_out = W_neigh.shape
        dX = np.zeros((rows.shape[0], F_in))
        rc = self.lib.orc_layer_dx_rows(self.h, F_in, F_out, int(relu), _p(Y, C.c_double), _p(W_self, C.c_double),
                                        _p(W_neigh, C.c_double), _p(dY, C.c_double), ratio[0], ratio[1], key[0],
                                        key[1], key[2], _p(rows, C.c_int64), rows.shape[0], _p(dX, C.c_double))
        assert rc == 0
        return dX
