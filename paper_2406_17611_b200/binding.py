"""ctypes binding of libvarco.so: argument marshalling only.

Every step of the layer path runs in the library's CUDA kernels; PyTorch is
used here for device memory and streams.  There is no CPU fallback: if the
compiled library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libvarco.so")

F32, BF16 = 0, 1
GCN, SAGE_MEAN = 0, 1
STAGES = ["compress", "decompress", "spmm", "gemm_fwd", "gemm_dx", "gemm_dw", "spmm_t", "compress_bwd",
          "scatter_add", "aux"]

EXPORTS = ["varco_status_string", "varco_partition_build", "varco_partition_destroy", "varco_partition_info",
           "varco_partition_boundary_rows", "varco_partition_set_l2_budget", "varco_partition_gather_model", "varco_partition_counts", "varco_partition_halo", "varco_partition_perm", "varco_partition_device_bytes",
           "varco_partition_upload", "varco_workspace_bytes", "varco_kept", "varco_schedule_linear",
           "varco_schedule_rate_linear", "varco_schedule_exponential",
           "varco_compress", "varco_decompress", "varco_layer_fwd", "varco_layer_bwd", "varco_profile_enable",
           "varco_profile_reset", "varco_profile_read", "varco_profile_spans", "varco_probe_gather", "varco_debug_status", "varco_kernel_launches", "varco_workspace_status",
           "varco_exchange_noalloc"]


class Ratio(C.Structure):
    _fields_ = [("num", C.c_uint32), ("den", C.c_uint32)]


class Key(C.Structure):
    _fields_ = [("seed", C.c_uint64), ("epoch", C.c_uint32), ("layer", C.c_uint32)]


class LayerDesc(C.Structure):
    _fields_ = [("conv", C.c_int), ("dtype", C.c_int), ("F_in", C.c_int32), ("F_out", C.c_int32),
                ("relu", C.c_int32), ("ld_in", C.c_int64), ("ld_out", C.c_int64)]


class VarcoError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        super().__init__("%s: %s (%d)" % (what, lib().varco_status_string(status).decode(), status))


_lib = None


def lib():
    """Load libvarco.so (built by paper_2406_17611_b200.build); raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    path = os.environ.get("VARCO_LIBRARY", LIB_PATH)    # e.g. the debug build, libvarco_debug.so
    if not os.path.exists(path):
        raise ImportError("%s is not built: run `python -m paper_2406_17611_b200.build` "
                          "(there is no CPU fallback)" % os.path.basename(path))
    L = C.CDLL(path)
    vp, i64p, i32p = C.c_void_p, C.POINTER(C.c_int64), C.POINTER(C.c_int32)
    L.varco_status_string.restype = C.c_char_p
    L.varco_status_string.argtypes = [C.c_int]
    L.varco_partition_build.argtypes = [C.c_int64, i64p, i32p, i32p, C.c_int32, C.c_int, C.POINTER(vp)]
    L.varco_partition_destroy.argtypes = [vp]
    L.varco_partition_info.argtypes = [vp, i64p, i64p, i32p, i64p, i64p, i64p]
    L.varco_partition_counts.argtypes = [vp, i64p]
    L.varco_partition_boundary_rows.argtypes = [vp, i64p]
    L.varco_partition_set_l2_budget.argtypes = [vp, C.c_int64]
    L.varco_partition_gather_model.argtypes = [vp, C.c_int32, C.c_int64, i64p, i64p, i64p]
    L.varco_partition_halo.argtypes = [vp, C.c_int32, C.c_int32, C.POINTER(i64p), i64p]
    L.varco_partition_perm.argtypes = [vp, C.POINTER(i64p)]
    L.varco_partition_device_bytes.argtypes = [vp, C.POINTER(C.c_size_t)]
    L.varco_partition_upload.argtypes = [vp, vp, C.c_size_t, vp]
    L.varco_workspace_bytes.argtypes = [vp, C.c_int32, C.c_int32, C.c_int, C.POINTER(C.c_size_t)]
    L.varco_kept.argtypes = [C.c_int32, Ratio, i32p]
    L.varco_schedule_linear.argtypes = [C.c_int32] * 5 + [C.POINTER(Ratio)]
    L.varco_schedule_rate_linear.argtypes = [C.c_int32, C.c_uint32, C.c_uint32, C.c_uint32, C.POINTER(Ratio)]
    L.varco_schedule_exponential.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.POINTER(Ratio)]
    L.varco_compress.argtypes = [vp, vp, C.c_int64, C.c_int32, C.c_int, Ratio, Key, vp, C.POINTER(C.c_uint64), vp]
    L.varco_decompress.argtypes = [vp, vp, C.c_int32, C.c_int, Ratio, Key, vp, C.c_int64, vp]
    L.varco_exchange_noalloc.argtypes = [vp, vp, C.c_int64, C.c_int32, C.c_int, Ratio, Key, vp, C.c_int64,
                                         C.POINTER(C.c_uint64), vp]
    L.varco_layer_fwd.argtypes = [vp, C.POINTER(LayerDesc), vp, vp, vp, vp, vp, vp, Ratio, Key, vp, C.c_size_t,
                                  C.POINTER(C.c_uint64), vp]
    L.varco_layer_bwd.argtypes = [vp, C.POINTER(LayerDesc), vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, Ratio, Key, vp,
                                  C.c_size_t, C.POINTER(C.c_uint64), vp]
    L.varco_profile_enable.argtypes = [vp, C.c_int]
    L.varco_profile_reset.argtypes = [vp]
    L.varco_profile_read.argtypes = [vp, i64p, C.POINTER(C.c_double)]
    L.varco_profile_spans.argtypes = [vp, C.c_int32, C.POINTER(C.c_double), C.c_int64, i64p]
    L.varco_probe_gather.argtypes = [vp, C.c_int64, C.c_int32, vp, C.c_int64, C.c_int32, vp, vp]
    L.varco_debug_status.argtypes = [i32p, i32p]
    L.varco_kernel_launches.argtypes = [i64p]
    L.varco_workspace_status.argtypes = [vp, vp, i32p]
    _lib = L
    return L


def _check(status, what):
    if status != 0:
        raise VarcoError(status, what)


def _ratio(r):
    return r if isinstance(r, Ratio) else Ratio(int(r[0]), int(r[1]))


def _key(k):
    return k if isinstance(k, Key) else Key(int(k[0]), int(k[1]), int(k[2]))


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


# ------------------------------------------------------------------------------------------ host helpers
def varco_kept(F, ratio):
    k = C.c_int32()
    _check(lib().varco_kept(int(F), _ratio(ratio), C.byref(k)), "varco_kept")
    return int(k.value)


def varco_schedule_linear(epoch, K, slope_a=5, c_max=128, c_min=1):
    r = Ratio()
    _check(lib().varco_schedule_linear(int(epoch), int(K), int(slope_a), int(c_max), int(c_min), C.byref(r)),
           "varco_schedule_linear")
    return (int(r.num), int(r.den))


NO_COMMUNICATION = (1, 0)   # ratio with denominator 0: nothing is sent (k = 0)


def varco_schedule_rate_linear(epoch, r0, alpha, den):
    """Ratio of the rate schedule r_k = (alpha k + r0) / den (also the fixed increment r_{k+1} = r_k + alpha/den)."""
    r = Ratio()
    _check(lib().varco_schedule_rate_linear(int(epoch), int(r0), int(alpha), int(den), C.byref(r)),
           "varco_schedule_rate_linear")
    return (int(r.num), int(r.den))


def varco_schedule_exponential(epoch, K, beta):
    """Ratio beta^(K - epoch) of the exponential rate schedule r_k = beta^-(K - k + 1), k = epoch + 1."""
    r = Ratio()
    _check(lib().varco_schedule_exponential(int(epoch), int(K), int(beta), C.byref(r)), "varco_schedule_exponential")
    return (int(r.num), int(r.den))


def varco_debug_status():
    """(is this a -DVARCO_DEBUG build, first failed device-side index check since the last call or 0)."""
    dbg, word = C.c_int32(), C.c_int32()
    _check(lib().varco_debug_status(C.byref(dbg), C.byref(word)), "varco_debug_status")
    return bool(dbg.value), int(word.value)


def varco_probe_gather(table, index, out):
    """Enqueue the random-row gather probe: out[r] = XOR of table[index[r, :]] (device tensors; rows of 128, 256
    or 512 bytes)."""
    row_bytes = table.stride(0) * table.element_size()
    _check(lib().varco_probe_gather(_ptr(table), table.shape[0], row_bytes // 16, _ptr(index), index.shape[0],
                                    index.shape[1], _ptr(out), _stream()), "varco_probe_gather")


def varco_kernel_launches():
    c = C.c_int64()
    _check(lib().varco_kernel_launches(C.byref(c)), "varco_kernel_launches")
    return int(c.value)


def varco_workspace_status(workspace):
    """Device status word of the last layer call on this workspace (0 = ok); synchronises."""
    v = C.c_int32()
    _check(lib().varco_workspace_status(_ptr(workspace), _stream(), C.byref(v)), "varco_workspace_status")
    return int(v.value)


class Plan:
    """varco_partition_build and friends.  Owns the plan handle and (after upload) its device image."""

    def __init__(self, row_ptr, col, part, P, conv):
        self.rp = np.ascontiguousarray(row_ptr, dtype=np.int64)
        self.col = np.ascontiguousarray(col, dtype=np.int32)
        self.part = np.ascontiguousarray(part, dtype=np.int32)
        self.conv = GCN if conv in (GCN, "gcn") else SAGE_MEAN
        self.h = C.c_void_p()
        n = self.rp.shape[0] - 1
        st = lib().varco_partition_build(n, self.rp.ctypes.data_as(C.POINTER(C.c_int64)),
                                         self.col.ctypes.data_as(C.POINTER(C.c_int32)),
                                         self.part.ctypes.data_as(C.POINTER(C.c_int32)), int(P), self.conv,
                                         C.byref(self.h))
        _check(st, "varco_partition_build")
        self._image = None
        n_, nnz, P_, H, cross, self_e = (C.c_int64(), C.c_int64(), C.c_int32(), C.c_int64(), C.c_int64(), C.c_int64())
        _check(lib().varco_partition_info(self.h, C.byref(n_), C.byref(nnz), C.byref(P_), C.byref(H), C.byref(cross),
                                          C.byref(self_e)), "varco_partition_info")
        self.n, self.nnz, self.P, self.H_total = int(n_.value), int(nnz.value), int(P_.value), int(H.value)
        self.cross_entries, self.self_entries = int(cross.value), int(self_e.value)
        nb = C.c_int64()
        _check(lib().varco_partition_boundary_rows(self.h, C.byref(nb)), "varco_partition_boundary_rows")
        self.boundary_rows = int(nb.value)

    def close(self):
        if self.h:
            lib().varco_partition_destroy(self.h)
            self.h = C.c_void_p()
            self._image = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_l2_budget(self, nbytes):
        _check(lib().varco_partition_set_l2_budget(self.h, int(nbytes)), "varco_partition_set_l2_budget")

    def gather_model(self, resident_rows, transposed=False):
        """(row gathers issued, distinct rows gathered, rows read from memory when the `resident_rows` most used
        sources of every partition stay cached)."""
        e, s, r = C.c_int64(), C.c_int64(), C.c_int64()
        _check(lib().varco_partition_gather_model(self.h, int(bool(transposed)), int(resident_rows), C.byref(e),
                                                  C.byref(s), C.byref(r)), "varco_partition_gather_model")
        return int(e.value), int(s.value), int(r.value)

    def rows_per_partition(self):
        """Number of rows of every partition (the plan's row order is partition-contiguous)."""
        return np.bincount(self.part, minlength=self.P).astype(np.int64)

    def counts(self):
        out = np.zeros((self.P, self.P), dtype=np.int64)
        _check(lib().varco_partition_counts(self.h, out.ctypes.data_as(C.POINTER(C.c_int64))), "varco_partition_counts")
        return out

    def halo(self, p, q):
        ptr, cnt = C.POINTER(C.c_int64)(), C.c_int64()
        _check(lib().varco_partition_halo(self.h, int(p), int(q), C.byref(ptr), C.byref(cnt)), "varco_partition_halo")
        return np.ctypeslib.as_array(ptr, shape=(cnt.value,)).copy() if cnt.value else np.empty(0, dtype=np.int64)

    def perm(self):
        ptr = C.POINTER(C.c_int64)()
        _check(lib().varco_partition_perm(self.h, C.byref(ptr)), "varco_partition_perm")
        return np.ctypeslib.as_array(ptr, shape=(self.n,)).copy()

    def device_bytes(self):
        b = C.c_size_t()
        _check(lib().varco_partition_device_bytes(self.h, C.byref(b)), "varco_partition_device_bytes")
        return int(b.value)

    def upload(self, device="cuda:0"):
        import torch
        nbytes = self.device_bytes()
        self._image = torch.empty(nbytes + 256, dtype=torch.uint8, device=device)
        base = self._image.data_ptr()
        off = (-base) % 256
        with torch.cuda.device(self._image.device):
            _check(lib().varco_partition_upload(self.h, C.c_void_p(base + off), nbytes, _stream()),
                   "varco_partition_upload")
        return self

    def workspace_bytes(self, F_in_max, F_out_max, dtype):
        b = C.c_size_t()
        _check(lib().varco_workspace_bytes(self.h, int(F_in_max), int(F_out_max), int(dtype), C.byref(b)),
               "varco_workspace_bytes")
        return int(b.value)

    def workspace(self, F_in_max, F_out_max, dtype, device="cuda:0"):
        import torch
        return torch.empty(self.workspace_bytes(F_in_max, F_out_max, dtype), dtype=torch.uint8, device=device)

    # -- profiling
    def profile_enable(self, on=True):
        _check(lib().varco_profile_enable(self.h, int(bool(on))), "varco_profile_enable")

    def profile_reset(self):
        _check(lib().varco_profile_reset(self.h), "varco_profile_reset")

    def profile_read(self):
        n = len(STAGES)
        launches = (C.c_int64 * n)()
        ms = (C.c_double * n)()
        _check(lib().varco_profile_read(self.h, launches, ms), "varco_profile_read")
        return {STAGES[i]: (int(launches[i]), float(ms[i])) for i in range(n)}

    def profile_spans(self, stage):
        """Durations (ms) of the individual timed executions of one stage, in enqueue order."""
        idx = STAGES.index(stage)
        count = C.c_int64()
        _check(lib().varco_profile_spans(self.h, idx, None, 0, C.byref(count)), "varco_profile_spans")
        buf = (C.c_double * max(1, count.value))()
        _check(lib().varco_profile_spans(self.h, idx, buf, count.value, C.byref(count)), "varco_profile_spans")
        return [float(buf[i]) for i in range(count.value)]


def _dtype_of(t):
    import torch
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("activations must be float32 or bfloat16")


def varco_compress(plan: Plan, X, F, ratio, key, packed=None):
    """X: [n x ld] device tensor in plan order.  Returns (packed [H_total x k], bytes on the wire)."""
    import torch
    k = varco_kept(F, ratio)
    if packed is None:
        packed = torch.empty((plan.H_total, k), dtype=X.dtype, device=X.device)
    nbytes = C.c_uint64()
    _check(lib().varco_compress(plan.h, _ptr(X), X.stride(0), int(F), _dtype_of(X), _ratio(ratio), _key(key),
                                _ptr(packed), C.byref(nbytes), _stream()), "varco_compress")
    return packed, int(nbytes.value)


def varco_decompress(plan: Plan, packed, F, ratio, key, ld=None, out=None):
    """Returns the dense halo rows [H_total x ld] in receive order."""
    import torch
    vec = 4 if packed.dtype == torch.float32 else 8
    ld = ld or (F + vec - 1) // vec * vec
    if out is None:
        out = torch.empty((plan.H_total, ld), dtype=packed.dtype, device=packed.device)
    _check(lib().varco_decompress(plan.h, _ptr(packed), int(F), _dtype_of(packed), _ratio(ratio), _key(key),
                                  _ptr(out), ld, _stream()), "varco_decompress")
    return out


NOALLOC_SCRATCH_BYTES = 32 << 20


def varco_exchange_noalloc(plan: Plan, X, F, ratio, key, out):
    """decompress(compress(X)) into the caller's `out` [H_total x ld] using only the library's
    built-in scratch: for callers that must not allocate device memory.  Returns the wire bytes."""
    nbytes = C.c_uint64()
    _check(lib().varco_exchange_noalloc(plan.h, _ptr(X), X.stride(0), int(F), _dtype_of(X), _ratio(ratio), _key(key),
                                        _ptr(out), out.stride(0), C.byref(nbytes), _stream()),
           "varco_exchange_noalloc")
    return int(nbytes.value)


def _desc(plan, X, F_in, F_out, relu, ld_out):
    return LayerDesc(plan.conv, _dtype_of(X), int(F_in), int(F_out), int(bool(relu)), X.stride(0), int(ld_out))


def varco_layer_fwd(plan: Plan, X, W_self, W_neigh, bias, relu, ratio, key, workspace, F_in=None, Y=None, Agg=None):
    """One layer forward over all partitions.  Returns (Y, Agg_saved, halo_bytes)."""
    import torch
    F_in = F_in or W_neigh.shape[0]
    F_out = W_neigh.shape[1]
    vec = 4 if X.dtype == torch.float32 else 8
    ld_out = (F_out + vec - 1) // vec * vec
    if Y is None:
        Y = torch.zeros((plan.n, ld_out), dtype=X.dtype, device=X.device)
    if Agg is None:
        Agg = torch.zeros((plan.n, X.stride(0)), dtype=X.dtype, device=X.device)
    d = _desc(plan, X, F_in, F_out, relu, Y.stride(0))
    hb = C.c_uint64()
    _check(lib().varco_layer_fwd(plan.h, C.byref(d), _ptr(X), _ptr(W_self), _ptr(W_neigh), _ptr(bias), _ptr(Y),
                                 _ptr(Agg), _ratio(ratio), _key(key), _ptr(workspace), workspace.numel(),
                                 C.byref(hb), _stream()), "varco_layer_fwd")
    return Y, Agg, int(hb.value)


def varco_layer_bwd(plan: Plan, X, Y, Agg, W_self, W_neigh, dY, relu, ratio, key, workspace, F_in=None, dX=None,
                    dW_self=None, dW_neigh=None, dbias=None):
    """One layer backward.  Returns (dX, dW_self, dW_neigh, dbias, halo_bytes)."""
    import torch
    F_in = F_in or W_neigh.shape[0]
    F_out = W_neigh.shape[1]
    if dX is None:
        dX = torch.zeros_like(X)
    f32 = dict(dtype=torch.float32, device=X.device)
    if dW_neigh is None:
        dW_neigh = torch.zeros((F_in, F_out), **f32)
    if dW_self is None and W_self is not None:
        dW_self = torch.zeros((F_in, F_out), **f32)
    if dbias is None:
        dbias = torch.zeros((F_out,), **f32)
    d = _desc(plan, X, F_in, F_out, relu, dY.stride(0))
    hb = C.c_uint64()
    _check(lib().varco_layer_bwd(plan.h, C.byref(d), _ptr(X), _ptr(Y), _ptr(Agg), _ptr(W_self), _ptr(W_neigh),
                                 _ptr(dY), _ptr(dX), _ptr(dW_self), _ptr(dW_neigh), _ptr(dbias), _ratio(ratio),
                                 _key(key), _ptr(workspace), workspace.numel(), C.byref(hb), _stream()),
           "varco_layer_bwd")
    return dX, dW_self, dW_neigh, dbias, int(hb.value)
