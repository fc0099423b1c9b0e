"""Training step around the partitioned layer (Algorithm 1 of the paper, steps 4-5, with Eq. (SGD)).

The layers run in libvarco (varco_layer_fwd / varco_layer_bwd); the loss, its gradient with respect to the
logits and the parameter update are a few PyTorch tensor operations on the device around them.  Every worker q
evaluates the cross-entropy of its own training nodes, L_q = mean over V_q; the errors are back-propagated across
the partitions through the compression routine; every worker steps with the weight gradient it accumulated and
the server averages the parameters: H <- H - (eta / Q) sum_p g_p, where sum_p g_p is what varco_layer_bwd returns
for the upstream gradient d(sum_q L_q)/dY.  With equal partitions this is gradient descent on the mean loss.
bf16 layers keep fp32 master weights and hand the layers a bf16 copy.
"""
from __future__ import annotations

import numpy as np

from . import binding as vb


class Trainer:
    def __init__(self, plan, widths, weights, bf16: bool, device="cuda:0"):
        """plan: uploaded binding.Plan; weights: per layer (W_self or None, W_neigh, bias) as arrays;
        all node-indexed tensors handed to the methods are in the plan's row order (plan.perm())."""
        import torch
        self.torch, self.plan, self.device = torch, plan, device
        self.widths = list(widths)
        self.L = len(self.widths) - 1
        self.dt = torch.bfloat16 if bf16 else torch.float32
        self.vec = 8 if bf16 else 4
        self.ld = [(f + self.vec - 1) // self.vec * self.vec for f in self.widths]
        f32 = lambda a: None if a is None else torch.tensor(np.asarray(a, dtype=np.float32), device=device)
        self.W = [[f32(w) for w in layer] for layer in weights]
        self.ws = plan.workspace(max(self.widths[:-1]), max(self.widths[1:]), vb.BF16 if bf16 else vb.F32, device)
        n = plan.n
        self.acts = [None] + [torch.zeros((n, self.ld[l + 1]), dtype=self.dt, device=device) for l in range(self.L)]
        self.aggs = [torch.zeros((n, self.ld[l]), dtype=self.dt, device=device) for l in range(self.L)]
        self.grads = [torch.zeros((n, self.ld[l]), dtype=self.dt, device=device) for l in range(self.L + 1)]
        self.P = plan.P
        sizes = plan.rows_per_partition()
        self.part = torch.repeat_interleave(torch.arange(self.P, device=device),
                                            torch.tensor(sizes, device=device))

    def _lowp(self, w):
        return None if w is None else w.to(self.dt).contiguous()

    def forward(self, X0, ratio, seed, epoch):
        """X0: [n x ld_0] device tensor in plan order.  Returns (logits [n x ld_L], halo bytes)."""
        self.acts[0] = X0
        total = 0
        for l in range(self.L):
            Ws, Wn, b = self.W[l]
            _, _, hb = vb.varco_layer_fwd(self.plan, self.acts[l], self._lowp(Ws), self._lowp(Wn), b, l < self.L - 1,
                                          ratio, (seed, epoch, l), self.ws, F_in=self.widths[l], Y=self.acts[l + 1],
                                          Agg=self.aggs[l])
            total += hb
        return self.acts[self.L], total

    def loss_and_grad(self, logits, labels, train):
        """sum_q L_q / Q and d(sum_q L_q)/d logits (per-worker means over the training nodes)."""
        torch = self.torch
        C = self.widths[-1]
        z = logits[:, :C].float()
        logp = torch.log_softmax(z, dim=1)
        counts = torch.bincount(self.part[train], minlength=self.P).float()
        w = torch.zeros(z.shape[0], device=self.device)
        ok = train & (counts[self.part] > 0)
        w[ok] = 1.0 / counts[self.part[ok]]
        loss = -(w * logp.gather(1, labels[:, None])[:, 0]).sum() / self.P
        d = torch.exp(logp)
        d.scatter_add_(1, labels[:, None], -torch.ones_like(d[:, :1]))
        d *= w[:, None]
        g = self.grads[self.L]
        g.zero_()
        g[:, :C] = d.to(self.dt)
        return loss, g

    def step(self, X0, labels, train, ratio, seed, epoch, lr):
        """One pass of Algorithm 1's loop body.  Returns (loss as a device scalar, halo bytes of the step)."""
        logits, total = self.forward(X0, ratio, seed, epoch)
        loss, grad = self.loss_and_grad(logits, labels, train)
        scale = lr / self.P
        for l in reversed(range(self.L)):
            Ws, Wn, b = self.W[l]
            r = vb.varco_layer_bwd(self.plan, self.acts[l], self.acts[l + 1], self.aggs[l], self._lowp(Ws), self._lowp(Wn),
                                   grad, l < self.L - 1, ratio, (seed, epoch, l), self.ws, F_in=self.widths[l],
                                   dX=self.grads[l])
            dX, dWs, dWn, db, hb = r
            total += hb
            if Ws is not None:
                Ws.sub_(dWs, alpha=scale)
            Wn.sub_(dWn, alpha=scale)
            b.sub_(db, alpha=scale)
            grad = dX
        return loss, total

    def accuracy(self, X0, labels, mask, ratio, seed, epoch):
        logits, _ = self.forward(X0, ratio, seed, epoch)
        pred = logits[:, :self.widths[-1]].float().argmax(dim=1)
        return float((pred[mask] == labels[mask]).float().mean().item())
