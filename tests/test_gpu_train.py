"""The training step around the layers (Algorithm 1 steps 4-5, Eq. (SGD)) on the GPU against the oracle's:
same seeded inputs and weights, a few steps under the variable schedule; losses, updated weights and halo bytes."""
import numpy as np
import pytest
import torch

from oracle.train import OracleModel
from paper_2406_17611_b200 import binding as vb
from paper_2406_17611_b200 import synth
from paper_2406_17611_b200.train import Trainer

from helpers import rel_err

pytestmark = pytest.mark.gpu


def _run(orc, wl, X, labels, train, steps, lr, tol_loss, tol_w, ratios):
    plan = vb.Plan(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv).upload()
    g = orc.graph(wl.row_ptr, wl.col, wl.part, wl.parts, wl.conv)
    perm = plan.perm()
    weights = [list(wl.layer_weights(l)) for l in range(len(wl.widths) - 1)]
    es = 2 if wl.bf16 else 4
    ref = OracleModel(g, wl.part, wl.parts, wl.widths, weights, elem_bytes=es)
    tr = Trainer(plan, wl.widths, weights, wl.bf16)
    dt = torch.bfloat16 if wl.bf16 else torch.float32
    X0 = torch.zeros((wl.n, tr.ld[0]), dtype=dt)
    X0[:, :wl.widths[0]] = torch.from_numpy(X[perm]).to(dt)
    X0 = X0.cuda()
    lab = torch.from_numpy(labels[perm]).cuda()
    trn = torch.from_numpy(train[perm]).cuda()
    for e in range(steps):
        loss, hb = tr.step(X0, lab, trn, ratios[e], 31, e, lr)
        rloss, rhb = ref.step(X, labels, train, ratios[e], 31, e, lr)
        assert hb == rhb
        assert abs(float(loss.item()) - rloss) <= tol_loss * abs(rloss)
    for l in range(tr.L):
        for got, want in zip(tr.W[l], ref.W[l]):
            if want is not None:
                assert rel_err(got.double().cpu().numpy(), want) <= tol_w
    acc = tr.accuracy(X0, lab, ~trn, ratios[-1], 31, steps)
    racc = ref.accuracy(X, labels, ~train, ratios[-1], 31, steps)
    assert abs(acc - racc) <= 0.02
    plan.close()


def test_training_steps_match_the_oracle_fp32(orc):
    wl = synth.make_workload("c2r", 0.04)
    X, labels, train = synth.planted_task(wl.extra["block"], wl.widths[0], 5)
    ratios = [orc.schedule_linear(e, 4, 2, 16, 1) for e in range(4)] + [(1, 0)]
    _run(orc, wl, X, labels, train, 5, 0.5, 1e-5, 1e-4, ratios)


def test_training_steps_match_the_oracle_bf16(orc):
    wl = synth.make_workload("c3", 0.002)
    X = wl.features()
    labels = wl.labels()
    train = np.random.default_rng(1).random(wl.n) < 0.5
    ratios = [(16, 1), (1, 1)]
    _run(orc, wl, X, labels, train, 2, 0.2, 2e-2, 5e-2, ratios)
