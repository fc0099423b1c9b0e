"""Synthetic generators produce graphs and partitions shaped like the paper's workloads."""
import os

import numpy as np

from paper_2406_17611_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _table1():
    rows, size = [], {}
    for line in open(os.path.join(GOLD, "paper_table1_edges.txt")):
        if not line.strip() or line.startswith("#"):
            continue
        tok = line.split()
        if tok[0] == "size":
            size[tok[1]] = (int(tok[2]), int(tok[3]))
        else:
            rows.append((tok[0], tok[1], int(tok[2]), int(tok[3]), int(tok[4])))
    return rows, size


def test_table1_random_rows_follow_one_minus_one_over_q():
    # In Table I the totals are 2 * edges + nodes (self-loops stored), and a random equal
    # Q-way split leaves a share 1 - 1/Q of the off-diagonal entries across servers.
    rows, size = _table1()
    for ds, how, Q, self_e, cross in rows:
        nodes, edges = size[ds]
        if ds == "products":
            assert self_e + cross == 2 * edges + nodes
        if how == "random":
            offdiag = self_e + cross - nodes
            assert abs(cross / offdiag - (1 - 1 / Q)) < 2e-3


def test_random_partition_cross_share(orc):
    wl = synth.make_workload("c2r", scale=0.2)
    sizes = np.bincount(wl.part, minlength=8)
    assert sizes.max() - sizes.min() <= 1
    g = orc.graph(wl.row_ptr, wl.col, wl.part, 8, "sage")
    assert g.cross_entries + g.self_entries == wl.nnz
    assert abs(g.cross_entries / wl.nnz - (1 - 1 / 8)) < 0.01


def test_sbm_community_partition_is_low_cut(orc):
    wl = synth.make_workload("c2", scale=0.2)
    g = orc.graph(wl.row_ptr, wl.col, wl.part, 8, "sage")
    assert abs(wl.nnz / wl.n - 20.0) < 0.5
    assert abs(g.cross_entries / wl.nnz - 4.0 / 20.0) < 0.01


def test_graphs_are_simple_symmetric_sorted():
    for name, scale in [("c1", 1.0), ("c2", 0.05), ("c3", 0.002), ("c4", 0.02)]:
        wl = synth.make_workload(name, scale)
        rp, col = wl.row_ptr, wl.col
        assert rp[0] == 0 and np.all(np.diff(rp) >= 0) and rp[-1] == col.shape[0]
        rows = np.repeat(np.arange(wl.n), np.diff(rp))
        assert np.all(rows != col)
        key = rows.astype(np.int64) * wl.n + col
        assert np.all(np.diff(key) > 0)                       # sorted, duplicate-free
        keyT = col.astype(np.int64) * wl.n + rows
        assert np.array_equal(np.sort(keyT), key)             # symmetric
        assert wl.part.min() >= 0 and wl.part.max() == wl.parts - 1


def test_generators_are_deterministic():
    a = synth.make_workload("c3", 0.002)
    b = synth.make_workload("c3", 0.002)
    assert np.array_equal(a.col, b.col) and np.array_equal(a.part, b.part)
    assert np.array_equal(a.features(), b.features())
    x = a.features()
    assert np.array_equal(synth.bf16_round(x), x)             # already bf16-representable
    assert abs(float(x.std()) - 1.0) < 0.02


def test_citation_shaped_workload_and_its_partition_sweep(orc):
    """The second workload (citation-network shape: 169,343 nodes, ~1.16M undirected edges, 128-d, 40 classes)
    over Q in {2, 4, 8, 16} workers: a random equal split leaves 1 - 1/Q of the entries across workers (the
    arithmetic of Table I's random rows), ranges of a breadth-first order cut fewer."""
    _, size = _table1()
    nodes, edges = size["arxiv"]
    full = synth.arxiv_shaped(16, "random")
    assert full.n == nodes and full.widths == [128, 256, 256, 40] and full.classes == 40
    assert abs(full.nnz / 2 - edges) / edges < 0.02          # duplicates dropped: within 2 % of the edge count
    for Q in (2, 4, 8, 16):
        shares = {}
        for split in ("random", "bfs"):
            wl = synth.arxiv_shaped(Q, split, scale=0.1)
            sizes = np.bincount(wl.part, minlength=Q)
            assert wl.parts == Q and sizes.max() - sizes.min() <= 1
            g = orc.graph(wl.row_ptr, wl.col, wl.part, Q, "sage")
            assert g.cross_entries + g.self_entries == wl.nnz
            shares[split] = g.cross_entries / wl.nnz
        assert abs(shares["random"] - (1 - 1 / Q)) < 0.02
        assert shares["bfs"] < shares["random"]
