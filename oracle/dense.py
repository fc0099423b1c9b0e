"""Dense-matrix brute force of the partitioned layer (test infrastructure only).

For graphs of a handful of nodes the aggregation matrix S is written out as an
n x n array straight from the edge list and the layer of Eq. (2) (two taps:
the node itself and one AGGREGATE) is evaluated with matrix products.  The
partitioned, compressed variant replaces a remote neighbour's row x_j by
M_j (.) x_j, M_j being the 0/1 mask of the positions that were sent
(appendix "Compression Mechanism": values in place, zero elsewhere).
Gradients come from PyTorch autograd in fp64, not from hand-derived formulas.
"""
from __future__ import annotations

import numpy as np
import torch


def dense_operator(row_ptr, col, conv: str) -> np.ndarray:
    """S as a dense array.  sage: row-normalised adjacency D^-1 A (zero rows stay zero).
    gcn: D~^-1/2 (A + I) D~^-1/2 with D~ = D + I."""
    n = len(row_ptr) - 1
    A = np.zeros((n, n))
    for i in range(n):
        for e in range(row_ptr[i], row_ptr[i + 1]):
            A[i, col[e]] = 1.0
    deg = A.sum(axis=1)
    if conv == "sage":
        inv = np.where(deg > 0, 1.0 / np.maximum(deg, 1.0), 0.0)
        return inv[:, None] * A
    d = 1.0 / np.sqrt(deg + 1.0)
    return d[:, None] * (A + np.eye(n)) * d[None, :]


def layer_dense(S, part, X, mask, W_self, W_neigh, bias, relu: bool):
    """Forward with dense matrices.  mask: [n x F] 0/1 (all ones = full communication
    = the centralized, unpartitioned layer)."""
    part = np.asarray(part)
    same = (part[:, None] == part[None, :]).astype(np.float64)
    agg = (S * same) @ X + (S * (1.0 - same)) @ (mask * X)
    z = agg @ W_neigh + bias
    if W_self is not None:
        z = z + X @ W_self
    return (np.maximum(z, 0.0) if relu else z), agg


def layer_dense_grads(S, part, X, mask, W_self, W_neigh, bias, relu: bool, dY):
    """(dX, dW_self, dW_neigh, dbias) of sum(Y * dY) by autograd, fp64."""
    t = lambda a: None if a is None else torch.tensor(np.asarray(a, dtype=np.float64), requires_grad=True)
    c = lambda a: torch.tensor(np.asarray(a, dtype=np.float64))
    Xt, Ws, Wn, bt = t(X), t(W_self), t(W_neigh), t(bias)
    part = np.asarray(part)
    same = c((part[:, None] == part[None, :]).astype(np.float64))
    St, Mt = c(S), c(mask)
    agg = (St * same) @ Xt + (St * (1.0 - same)) @ (Mt * Xt)
    z = agg @ Wn + bt
    if Ws is not None:
        z = z + Xt @ Ws
    y = torch.relu(z) if relu else z
    (y * c(dY)).sum().backward()
    g = lambda a: None if a is None else a.grad.numpy()
    return g(Xt), g(Ws), g(Wn), g(bt)
