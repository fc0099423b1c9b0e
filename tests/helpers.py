"""Shared plumbing of the GPU parity tests: move seeded inputs to the device in plan order and
compare device results with the oracle's (which works in original node order)."""
import numpy as np
import torch

from paper_2406_17611_b200 import binding as vb

TOL = {torch.float32: 1e-5, torch.bfloat16: 2e-2}


def vec_of(dtype):
    return 4 if dtype == torch.float32 else 8


def to_device_rows(a_host, perm, dtype, dev="cuda:0"):
    """[n x F] host array in original order -> padded [n x ld] device tensor in plan order."""
    n, F = a_host.shape
    v = vec_of(dtype)
    ld = (F + v - 1) // v * v
    t = torch.zeros((n, ld), dtype=dtype)
    t[:, :F] = torch.from_numpy(np.ascontiguousarray(a_host[perm])).to(dtype)
    return t.to(dev)


def to_host_rows(t_dev, perm, F):
    """Device tensor in plan order -> fp64 host array [n x F] in original order."""
    a = t_dev[:, :F].to(torch.float64).cpu().numpy()
    out = np.empty_like(a)
    out[perm] = a
    return out


def rel_err(got, ref):
    """max |got - ref| / max |ref| (norm-wise: element-wise ratios are meaningless at ReLU zeros)."""
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    return float(np.max(np.abs(got - ref)) / max(float(np.max(np.abs(ref))), 1e-30))


def rel_err_axis(got, ref, axis, floor=5e-2):
    """Scaled companion of rel_err: the largest |got - ref| of every column (axis=0) or row (axis=1) over that
    column's / row's own max |ref| -- not below `floor` times the tensor's max, so that a column of ReLU zeros
    does not divide by nothing.  A wrong low-magnitude column (a padded tail, one feature) or row (a high-degree
    node whose mean is small, a dropped neighbour) cannot hide behind the largest entries of the tensor."""
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    if ref.ndim == 1:
        ref, got = ref[None, :], got[None, :]
    gmax = max(float(np.abs(ref).max()), 1e-30)
    scale = np.maximum(np.abs(ref).max(axis=axis), floor * gmax)
    return float((np.abs(got - ref).max(axis=axis) / scale).max())


def close(got, ref, tol):
    """Norm-wise within tol, and within 2 tol against every column's and every row's own scale."""
    e, ec, er = rel_err(got, ref), rel_err_axis(got, ref, 0), rel_err_axis(got, ref, 1)
    ok = e <= tol and ec <= 2 * tol and er <= 2 * tol
    if not ok:
        print("close(): norm-wise %.3e, column-wise %.3e, row-wise %.3e, tol %.1e" % (e, ec, er, tol))
    return ok


def dev_weights(w, dtype, dev="cuda:0"):
    return None if w is None else torch.from_numpy(np.ascontiguousarray(w)).to(dtype).to(dev).contiguous()


def host64(t):
    return None if t is None else t.to(torch.float64).cpu().numpy()


class LayerCase:
    """One workload uploaded to the device, with its oracle graph beside it."""

    def __init__(self, orc, wl, dev="cuda:0"):
        self.wl = wl
        self.dtype = torch.bfloat16 if wl.bf16 else torch.float32
        self.es = 2 if wl.bf16 else 4
        self.plan = vb.Plan(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv).upload(dev)
        self.perm = self.plan.perm()
        self.g = orc.graph(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv)
        self.ws = self.plan.workspace(max(wl.widths[:-1]), max(wl.widths[1:]), vb.BF16 if wl.bf16 else vb.F32, dev)
        self.dev = dev
