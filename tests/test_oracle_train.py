"""Pins for the oracle's training step (Algorithm 1 steps 4-5, Eq. (SGD)): one step at full communication is
one gradient-descent step of the centralized model (dense matrices, PyTorch autograd); per-worker steps plus
parameter averaging are plain SGD on the mean loss when the partitions are equal; the loss of a learnable
task goes down and the bytes follow the schedule."""
import numpy as np
import torch

from oracle import dense
from oracle.train import OracleModel, softmax_ce_per_worker
from paper_2406_17611_b200 import synth

from test_oracle_layer import tiny_graph, weights


def _dense_step(S, part, P, X, labels, train, Ws_list, lr, equal_mean=False):
    """Centralized model: Y = stack of rho(X Ws + S X Wn + b); objective (1/Q) sum_q mean_{V_q} CE; one SGD step
    by autograd.  Returns (objective, new weights)."""
    t = lambda a: torch.tensor(np.asarray(a, dtype=np.float64), requires_grad=True)
    params = [[None if w is None else t(w) for w in layer] for layer in Ws_list]
    St = torch.tensor(S)
    h = torch.tensor(np.asarray(X, dtype=np.float64))
    L = len(params)
    for l, (Ws, Wn, b) in enumerate(params):
        z = (St @ h) @ Wn + b
        if Ws is not None:
            z = z + h @ Ws
        h = torch.relu(z) if l < L - 1 else z
    logp = torch.log_softmax(h, dim=1)
    nll = -logp[torch.arange(h.shape[0]), torch.tensor(labels)]
    obj = 0.0
    if equal_mean:
        obj = nll[torch.tensor(train)].mean()
    else:
        for q in range(P):
            sel = torch.tensor(train & (part == q))
            if sel.any():
                obj = obj + nll[sel].mean() / P
    obj.backward()
    new = [[None if w is None else (w - lr * w.grad).detach().numpy() for w in layer] for layer in params]
    return float(obj.detach()), new


def _setup(conv, seed, n=10, P=2):
    rp, col = tiny_graph(n, 18, seed)
    part = (np.arange(n) % P).astype(np.int32)
    rng = np.random.default_rng(seed)
    widths = [6, 5, 4]
    X = rng.standard_normal((n, widths[0]))
    labels = rng.integers(0, widths[-1], size=n)
    W = [list(weights(widths[l], widths[l + 1], conv == "sage", seed + l)) for l in range(2)]
    return rp, col, part, widths, X, labels, W


def test_full_communication_step_is_a_centralized_sgd_step(orc):
    for conv in ("sage", "gcn"):
        for seed in (0, 1):
            rp, col, part, widths, X, labels, W = _setup(conv, seed)
            train = np.ones(X.shape[0], dtype=bool)
            train[seed] = False                                   # unequal training counts per worker
            g = orc.graph(rp, col, part, 2, conv)
            m = OracleModel(g, part, 2, widths, W)
            loss, hb = m.step(X, labels, train, (1, 1), 5, 0, 0.3)
            S = dense.dense_operator(rp, col, conv)
            obj, new = _dense_step(S, part, 2, X, labels, train, W, 0.3)
            assert abs(loss - obj) < 1e-12
            for l in range(2):
                for a, b in zip(m.W[l], new[l]):
                    assert (a is None and b is None) or np.allclose(a, b, atol=1e-12)
            assert hb == 2 * g.H_total * (widths[0] + widths[1]) * 4          # forward + backward, both layers


def test_equal_partitions_give_plain_sgd_on_the_mean_loss(orc):
    rp, col, part, widths, X, labels, W = _setup("sage", 3, n=10, P=2)
    train = np.ones(10, dtype=bool)
    g = orc.graph(rp, col, part, 2, "sage")
    m = OracleModel(g, part, 2, widths, W)
    loss, _ = m.step(X, labels, train, (1, 1), 5, 0, 0.2)
    S = dense.dense_operator(rp, col, "sage")
    obj, new = _dense_step(S, part, 2, X, labels, train, W, 0.2, equal_mean=True)
    assert abs(loss - obj) < 1e-12
    assert all(np.allclose(a, b, atol=1e-12) for l in range(2) for a, b in zip(m.W[l], new[l]))
    # the per-worker normalisation itself: a 3:1 split of the training nodes is NOT the global mean
    lo, d = softmax_ce_per_worker(np.zeros((4, 3)), np.zeros(4, dtype=int), np.ones(4, dtype=bool),
                                  np.array([0, 0, 0, 1]), 2)
    assert np.isclose(lo, 2 * np.log(3)) and np.allclose(d[:, 0], [-2 / 9, -2 / 9, -2 / 9, -2 / 3])


def test_training_learns_and_counts_bytes(orc):
    """Stochastic block model, random split (most neighbours remote): the loss falls under the variable schedule,
    the bytes are the schedule's closed form, and without communication the neighbours' signal is lost."""
    n, P = 1600, 4
    rp, col, block = synth.stochastic_block_model(n, 4, 12.0, 2.0, 3)
    part = synth.partition_random_equal(n, P, 4)
    X, labels, train = synth.planted_task(block, 16, 5, signal=0.25)
    widths = [16, 16, 8]
    g = orc.graph(rp, col, part, P, "sage")
    K, lr = 30, 1.0
    runs = {}
    for name in ("varco", "none"):
        W = [[synth.glorot_uniform(widths[l], widths[l + 1], 20 + 2 * l),
              synth.glorot_uniform(widths[l], widths[l + 1], 21 + 2 * l), np.zeros(widths[l + 1])] for l in range(2)]
        m = OracleModel(g, part, P, widths, W)
        losses, total = [], 0
        for e in range(K):
            ratio = orc.schedule_linear(e, K, 5, 8, 1) if name == "varco" else (1, 0)
            lo, hb = m.step(X, labels, train, ratio, 9, e, lr)
            losses.append(lo)
            total += hb
        runs[name] = (losses, total, m.accuracy(X, labels, ~train, (1, 1) if name == "varco" else (1, 0), 9, K))
    losses, total, acc = runs["varco"]
    assert losses[-1] < 0.8 * losses[0]
    want = sum(2 * g.H_total * orc.kept(F, orc.schedule_linear(e, K, 5, 8, 1)) * 4 for e in range(K) for F in widths[:-1])
    assert total == want
    assert runs["none"][1] == 0
    assert acc > runs["none"][2] + 0.05 and acc > 0.3
