"""Training step around the partitioned layer, in plain NumPy on top of the oracle (test infrastructure only).

Algorithm 1 of the paper, steps 4-5, with Eq. (SGD): every worker q evaluates the loss of its own training
nodes, L_q = mean over V_q of the cross-entropy; the errors are back-propagated across machines (through the
compression routine, oracle.layer_bwd); every worker applies a gradient step with the weight gradient it
accumulated, g_p, and the server averages the parameters:
    H <- mean_p (H - eta g_p) = H - (eta / Q) sum_p g_p.
The layer's backward returns exactly sum_p g_p for the upstream gradient it is given, here d(sum_q L_q)/dY.
With equal partition sizes this is plain gradient descent on the mean loss over all training nodes.
"""
from __future__ import annotations

import numpy as np


def softmax_ce_per_worker(logits, labels, train, part, P):
    """sum_q L_q and its gradient w.r.t. the logits; L_q = mean cross-entropy over worker q's training nodes."""
    z = logits - logits.max(axis=1, keepdims=True)
    logp = z - np.log(np.exp(z).sum(axis=1, keepdims=True))
    prob = np.exp(logp)
    n = logits.shape[0]
    counts = np.bincount(part[train], minlength=P).astype(np.float64)
    w = np.zeros(n)
    ok = train & (counts[part] > 0)
    w[ok] = 1.0 / counts[part[ok]]
    loss = float(-(w * logp[np.arange(n), labels]).sum())
    d = prob.copy()
    d[np.arange(n), labels] -= 1.0
    d *= w[:, None]
    return loss, d


class OracleModel:
    """Stack of partitioned layers with their weights; ReLU on all but the last layer."""

    def __init__(self, graph, part, P, widths, weights, elem_bytes=4):
        self.g, self.part, self.P = graph, np.asarray(part), P
        self.widths = list(widths)
        self.W = [[None if w is None else np.array(w, dtype=np.float64) for w in layer] for layer in weights]
        self.es = elem_bytes
        self.L = len(self.widths) - 1

    def forward(self, X, ratio, key_seed, epoch):
        acts, total = [np.asarray(X, dtype=np.float64)], 0
        for l in range(self.L):
            Ws, Wn, b = self.W[l]
            Y, _, hb = self.g.layer_fwd(acts[l], Ws, Wn, b, l < self.L - 1, ratio, (key_seed, epoch, l),
                                        elem_bytes=self.es)
            acts.append(Y)
            total += hb
        return acts, total

    def step(self, X, labels, train, ratio, key_seed, epoch, lr):
        """One pass of Algorithm 1's loop body.  Returns (sum of the workers' losses / Q, halo bytes moved)."""
        acts, total = self.forward(X, ratio, key_seed, epoch)
        loss, grad = softmax_ce_per_worker(acts[self.L], labels, train, self.part, self.P)
        for l in reversed(range(self.L)):
            Ws, Wn, b = self.W[l]
            dX, dWs, dWn, db, hb = self.g.layer_bwd(acts[l], acts[l + 1], Ws, Wn, grad, l < self.L - 1, ratio,
                                                    (key_seed, epoch, l), elem_bytes=self.es)
            total += hb
            scale = lr / self.P          # each worker steps with its own g_p, the server averages
            if Ws is not None:
                self.W[l][0] = Ws - scale * dWs
            self.W[l][1] = Wn - scale * dWn
            self.W[l][2] = b - scale * db
            grad = dX
        return loss / self.P, total

    def accuracy(self, X, labels, mask, ratio, key_seed, epoch):
        acts, _ = self.forward(X, ratio, key_seed, epoch)
        pred = acts[self.L].argmax(axis=1)
        return float((pred[mask] == labels[mask]).mean())
