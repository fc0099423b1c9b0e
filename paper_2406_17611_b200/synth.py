"""Seeded synthetic inputs: graphs, partition labels, features, weights.

This module only draws random inputs.  It holds none of the method's
arithmetic (no halo sets, no compression, no layer math), so both the CUDA
library's tests and the CPU oracle's tests may feed from it without sharing
any computation.  Everything is deterministic in its seed.

Graphs come back as a symmetric CSR adjacency (``row_ptr`` int64, ``col``
int32) with sorted, duplicate-free columns and no self-loops.  The shapes
follow the workloads of the paper's experiments section (a products-like
power-law graph with 100-d features and 47 classes, 3 x 256 SAGE layers,
2..16 workers, random and low-cut partitions); the public datasets themselves
are not used -- these inputs stand in for them.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import scipy.sparse as sp
from scipy.sparse import csgraph


# --------------------------------------------------------------------------- graphs
def _csr_from_pairs(n: int, u: np.ndarray, v: np.ndarray):
    """Undirected simple graph from endpoint pairs: drop loops, dedupe, symmetrise."""
    keep = u != v
    u, v = u[keep], v[keep]
    r = np.concatenate([u, v])
    c = np.concatenate([v, u])
    a = sp.coo_matrix((np.ones(r.shape[0], dtype=np.int8), (r, c)), shape=(n, n)).tocsr()
    a.sum_duplicates()
    a.sort_indices()
    return a.indptr.astype(np.int64), a.indices.astype(np.int32)


def erdos_renyi(n: int, avg_degree: float, seed: int):
    """G(n, m)-style Erdos-Renyi graph with about n*avg_degree/2 undirected edges."""
    rng = np.random.default_rng(seed)
    m = int(round(n * avg_degree / 2.0))
    u = rng.integers(0, n, size=m, dtype=np.int64)
    v = rng.integers(0, n, size=m, dtype=np.int64)
    return _csr_from_pairs(n, u, v)


def stochastic_block_model(n: int, blocks: int, deg_in: float, deg_out: float, seed: int):
    """Equal-size planted communities; expected degree deg_in inside, deg_out across.

    Returns (row_ptr, col, block_of_node).  Node ids are shuffled so that the
    community of a node is not a function of its id range.
    """
    rng = np.random.default_rng(seed)
    size = n // blocks
    assert size * blocks == n
    m_in = rng.poisson(size * deg_in / 2.0, size=blocks)
    us, vs = [], []
    for b in range(blocks):
        us.append(rng.integers(0, size, size=m_in[b], dtype=np.int64) + b * size)
        vs.append(rng.integers(0, size, size=m_in[b], dtype=np.int64) + b * size)
    m_out = int(rng.poisson(n * deg_out / 2.0))
    uo = rng.integers(0, n, size=m_out, dtype=np.int64)
    shift = rng.integers(1, blocks, size=m_out, dtype=np.int64)
    vo = ((uo // size + shift) % blocks) * size + rng.integers(0, size, size=m_out, dtype=np.int64)
    us.append(uo)
    vs.append(vo)
    u = np.concatenate(us)
    v = np.concatenate(vs)
    relabel = rng.permutation(n).astype(np.int64)
    block = np.empty(n, dtype=np.int32)
    block[relabel] = (np.arange(n) // size).astype(np.int32)
    row_ptr, col = _csr_from_pairs(n, relabel[u], relabel[v])
    return row_ptr, col, block


def _chung_lu(n: int, w: np.ndarray, m: int, rng):
    cdf = np.cumsum(w, dtype=np.float64)
    cdf /= cdf[-1]
    u = np.searchsorted(cdf, rng.random(m), side="right").astype(np.int64)
    v = np.searchsorted(cdf, rng.random(m), side="right").astype(np.int64)
    np.minimum(u, n - 1, out=u)
    np.minimum(v, n - 1, out=v)
    relabel = rng.permutation(n).astype(np.int64)
    return _csr_from_pairs(n, relabel[u], relabel[v])


def chung_lu_power_law(n: int, undirected_edges: int, exponent: float, seed: int):
    """Chung-Lu graph with expected degrees w_i ~ (i + i0)^(-1/(exponent-1)).

    Endpoints are drawn from the continuous density proportional to (x + i0)^-alpha on [0, n)
    by inverting its CDF in closed form, then floored to a node index.  i0 = n / 2450 keeps the
    largest expected degree near sqrt(sum w), the usual Chung-Lu condition.
    """
    rng = np.random.default_rng(seed)
    alpha = 1.0 / (exponent - 1.0)
    i0 = max(1.0, n / 2450.0)
    lo, hi = i0 ** (1.0 - alpha), (n + i0) ** (1.0 - alpha)

    def draw(m):
        x = rng.random(m)
        x *= hi - lo
        x += lo
        np.power(x, 1.0 / (1.0 - alpha), out=x)
        x -= i0
        idx = x.astype(np.int64)
        np.clip(idx, 0, n - 1, out=idx)
        return idx
    u = draw(undirected_edges)
    v = draw(undirected_edges)
    relabel = rng.permutation(n).astype(np.int64)
    return _csr_from_pairs(n, relabel[u], relabel[v])


def chung_lu_lognormal(n: int, mean_degree: float, sigma: float, seed: int):
    """Chung-Lu graph whose expected degrees are lognormal with the given mean."""
    rng = np.random.default_rng(seed)
    mu = np.log(mean_degree) - 0.5 * sigma * sigma
    w = rng.lognormal(mu, sigma, size=n)
    np.minimum(w, np.sqrt(w.sum()), out=w)
    m = int(round(w.sum() / 2.0))
    return _chung_lu(n, w, m, rng)


# --------------------------------------------------------------------------- partitions
def partition_random_equal(n: int, parts: int, seed: int) -> np.ndarray:
    """Random permutation of the nodes cut into `parts` contiguous near-equal blocks."""
    rng = np.random.default_rng(seed)
    order = rng.permutation(n)
    label = np.empty(n, dtype=np.int32)
    bounds = (np.arange(parts + 1, dtype=np.int64) * n) // parts
    for p in range(parts):
        label[order[bounds[p]:bounds[p + 1]]] = p
    return label


def partition_bfs_ranges(row_ptr: np.ndarray, col: np.ndarray, parts: int, seed: int) -> np.ndarray:
    """Breadth-first order from a seeded root (unreached nodes appended by id),
    then `parts` contiguous near-equal ranges of that order."""
    n = row_ptr.shape[0] - 1
    rng = np.random.default_rng(seed)
    a = sp.csr_matrix((np.ones(col.shape[0], dtype=np.int8), col, row_ptr), shape=(n, n))
    root = int(rng.integers(0, n))
    while row_ptr[root + 1] == row_ptr[root]:
        root = int(rng.integers(0, n))
    order = csgraph.breadth_first_order(a, root, directed=False, return_predecessors=False)
    seen = np.zeros(n, dtype=bool)
    seen[order] = True
    order = np.concatenate([order.astype(np.int64), np.nonzero(~seen)[0].astype(np.int64)])
    label = np.empty(n, dtype=np.int32)
    bounds = (np.arange(parts + 1, dtype=np.int64) * n) // parts
    for p in range(parts):
        label[order[bounds[p]:bounds[p + 1]]] = p
    return label


# --------------------------------------------------------------------------- tensors
def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bfloat16 (ties to even), returned as fp32."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    b = (b + 0x7FFF + ((b >> 16) & 1)) & 0xFFFF0000
    return b.astype(np.uint32).view(np.float32)


def normal_features(n: int, width: int, seed: int, bf16: bool = False) -> np.ndarray:
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((n, width), dtype=np.float32)
    return bf16_round(x) if bf16 else x


def glorot_uniform(fan_in: int, fan_out: int, seed: int, bf16: bool = False) -> np.ndarray:
    rng = np.random.default_rng(seed)
    lim = np.sqrt(6.0 / (fan_in + fan_out))
    w = rng.uniform(-lim, lim, size=(fan_in, fan_out)).astype(np.float32)
    return bf16_round(w) if bf16 else w


def uniform_labels(n: int, classes: int, seed: int) -> np.ndarray:
    return np.random.default_rng(seed).integers(0, classes, size=n, dtype=np.int64)


# --------------------------------------------------------------------------- workloads
@dataclass
class Workload:
    """One named configuration: graph, partition labels and model shape."""
    name: str
    row_ptr: np.ndarray
    col: np.ndarray
    part: np.ndarray
    parts: int
    conv: str                 # "gcn" or "sage"
    widths: list              # [F_0, F_1, ..., F_L]
    bf16: bool
    classes: int
    seed: int
    note: str = ""
    extra: dict = field(default_factory=dict)

    @property
    def n(self) -> int:
        return self.row_ptr.shape[0] - 1

    @property
    def nnz(self) -> int:
        return int(self.row_ptr[-1])

    def features(self) -> np.ndarray:
        return normal_features(self.n, self.widths[0], self.seed + 101, self.bf16)

    def labels(self) -> np.ndarray:
        return uniform_labels(self.n, self.classes, self.seed + 102)

    def layer_weights(self, layer: int):
        """(W_self or None, W_neigh, bias) of one layer, Glorot-uniform, seeded."""
        f_in, f_out = self.widths[layer], self.widths[layer + 1]
        s = self.seed + 1000 + 10 * layer
        w_neigh = glorot_uniform(f_in, f_out, s, self.bf16)
        w_self = glorot_uniform(f_in, f_out, s + 1, self.bf16) if self.conv == "sage" else None
        rng = np.random.default_rng(s + 2)
        bias = (0.1 * rng.standard_normal(f_out)).astype(np.float32)
        return w_self, w_neigh, bias


def planted_task(block: np.ndarray, width: int, seed: int, signal: float = 0.12, train_share: float = 0.5):
    """A node-classification task that needs the neighbours: features are N(0,1) noise plus a faint shift
    signal * mu_b shared by the nodes of community b (about one standard deviation per node along mu_b, so that
    a node's own row says little and the mean over its mostly same-community neighbours says a lot), two classes
    per community: class = 2 * community + 1[x . v > 0] for one fixed direction v (the part a node can read off
    its own row).  Returns (X fp32 [n x width], labels int64 [n], train mask bool [n]); draws inputs only."""
    rng = np.random.default_rng(seed)
    n = block.shape[0]
    nb = int(block.max()) + 1
    mu = rng.standard_normal((nb, width)).astype(np.float32)
    v = rng.standard_normal(width).astype(np.float32)
    x = rng.standard_normal((n, width), dtype=np.float32)
    x += signal * mu[block]
    coin = (x @ v > 0).astype(np.int64)
    labels = 2 * block.astype(np.int64) + coin
    train = rng.random(n) < train_share
    return x, labels, train


def make_workload(name: str, scale: float = 1.0, seed: int = 2406) -> Workload:
    """Build one of the named configurations.

    c1   Erdos-Renyi, 2,000 nodes, mean degree 10, 4 random equal parts, 2-layer GCN 64-64-8, fp32
    c2   SBM, 100,000 nodes in 8 communities (16 in / 4 out), parts = communities, SAGE 128-256-256-16, fp32
    c2r  the same graph with a random 8-way split (high cut)
    c3   Chung-Lu power law (exponent 2.1), 2.45M nodes, ~62M undirected edges, 16 BFS-range parts,
         SAGE 100-256-256-47, bf16
    c4   Chung-Lu lognormal (mean degree 490), 233,000 nodes, random 8-way split, GCN 602-256-41, bf16
    c5   the c3 graph with a 4-layer SAGE 100-256-256-256-47, bf16
    arx  citation-network shape: 169,343 nodes, ~1.16M undirected edges, 128-d, 40 classes, SAGE 128-256-256-40,
         bf16, 16 random parts (arxiv_shaped() takes the number of parts and the kind of split)

    `scale` < 1 shrinks the node count (same degree law) for tests.
    """
    key = name.lower()
    if key == "c1":
        n = max(40, int(round(2000 * scale)))
        rp, col = erdos_renyi(n, 10.0, seed)
        part = partition_random_equal(n, 4, seed + 1)
        return Workload("c1", rp, col, part, 4, "gcn", [64, 64, 8], False, 8, seed,
                        "Erdos-Renyi n=%d deg 10, 4 random equal parts" % n)
    if key in ("c2", "c2r"):
        n = max(80, int(round(100000 * scale)) // 8 * 8)
        rp, col, block = stochastic_block_model(n, 8, 16.0, 4.0, seed)
        part = block if key == "c2" else partition_random_equal(n, 8, seed + 1)
        wl = Workload(key, rp, col, part.astype(np.int32), 8, "sage", [128, 256, 256, 16], False, 16, seed,
                      "SBM n=%d, 8 communities, %s 8-way split" % (n, "community" if key == "c2" else "random"))
        wl.extra["block"] = block
        return wl
    if key in ("c3", "c5"):
        n = max(1000, int(round(2450000 * scale)))
        m = int(round(62000000 * scale))
        rp, col = chung_lu_power_law(n, m, 2.1, seed)
        part = partition_bfs_ranges(rp, col, 16, seed + 1)
        widths = [100, 256, 256, 47] if key == "c3" else [100, 256, 256, 256, 47]
        return Workload(key, rp, col, part, 16, "sage", widths, True, 47, seed,
                        "Chung-Lu power law n=%d, 16 BFS-range parts" % n)
    if key == "c4":
        n = max(2000, int(round(233000 * scale)))
        mean_deg = 490.0 if scale >= 1.0 else max(20.0, 490.0 * scale)
        rp, col = chung_lu_lognormal(n, mean_deg, 0.75, seed)
        part = partition_random_equal(n, 8, seed + 1)
        return Workload("c4", rp, col, part, 8, "gcn", [602, 256, 41], True, 41, seed,
                        "Chung-Lu lognormal n=%d mean degree %.0f, random 8-way split" % (n, mean_deg))
    if key == "arx":
        return arxiv_shaped(16, "random", scale, seed)
    raise ValueError("unknown workload %r" % name)


def arxiv_shaped(parts: int = 16, split: str = "random", scale: float = 1.0, seed: int = 2406) -> Workload:
    """A citation-network-shaped second workload: 169,343 nodes, about 1.16M undirected edges (power-law degrees,
    exponent 2.4), 128-d features, 40 classes, 3-layer SAGE 128-256-256-40, bf16; `parts` in {2, 4, 8, 16} equal
    partitions, either a random split or contiguous ranges of a breadth-first order (the low-cut stand-in for a
    partitioner).  The small-graph regime: a few MB per layer, where launches and tiny segments dominate."""
    n = max(1000, int(round(169343 * scale)))
    m = int(round(1166243 * scale))
    rp, col = chung_lu_power_law(n, m, 2.4, seed + 3)
    if split == "random":
        part = partition_random_equal(n, parts, seed + 1)
    elif split == "bfs":
        part = partition_bfs_ranges(rp, col, parts, seed + 1)
    else:
        raise ValueError("split must be 'random' or 'bfs'")
    return Workload("arx", rp, col, part, parts, "sage", [128, 256, 256, 40], True, 40, seed,
                    "Chung-Lu power law n=%d (citation-network shape), %d %s equal parts" % (n, parts, split))
