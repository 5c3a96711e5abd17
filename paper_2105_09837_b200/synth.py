"""Seeded synthetic inputs for pdADMM-G / pdADMM-G-Q workloads.

This module only draws inputs (graph, features, labels, mask, initial weights).
It contains none of the method's arithmetic, so the CPU oracle's tests and the
CUDA path's tests can both be fed from it without sharing any computation.

Every draw comes from a Philox counter-based generator keyed by
``(seed ^ workload id, purpose)``, so each array is reproducible on its own and
does not depend on the order in which the others were requested.

The five named workloads stand in for the paper's public graphs (Table "Dataset
statistics"): the items of those datasets are not reproduced here, only their
shapes, degree structure and value distributions.
"""

from __future__ import annotations

import dataclasses
from typing import List, Optional

import numpy as np

BASE_SEED = 0x9E3779B97F4A7C15

# purposes (second word of the Philox key)
_P_GRAPH, _P_FEAT, _P_LABEL, _P_MASK, _P_W = 1, 2, 3, 4, 5


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape of one synthetic training problem.

    ``n_hops`` is the highest power of the renormalised adjacency that is
    used, so the input has ``n_hops + 1`` feature blocks (powers 0..n_hops).
    ``widths`` are n_1..n_L (the last one equals ``n_classes``).
    """

    name: str
    wid: int
    n_nodes: int
    graph: str            # "er" (Erdos-Renyi) or "ba" (Barabasi-Albert)
    graph_param: float    # er: average degree; ba: edges added per new node (m)
    feat_dim: int
    feat_kind: str        # "bernoulli" or "normal"
    feat_param: float     # bernoulli: P(x=1)
    n_classes: int
    n_hops: int
    n_layers: int
    hidden: int
    quant_levels: int     # 0 = pdADMM-G, m >= 2 = pdADMM-G-Q with m uniform levels
    n_iters: int
    rho: float = 1e-3
    nu: float = 1e-3
    train_frac: float = 0.5

    @property
    def n_blocks(self) -> int:
        return self.n_hops + 1

    @property
    def n0(self) -> int:
        return self.n_blocks * self.feat_dim

    @property
    def widths(self) -> List[int]:
        return [self.hidden] * (self.n_layers - 1) + [self.n_classes]

    def scaled(self, name: str, **kw) -> "Workload":
        """A copy with some fields replaced (reduced sizes for parity tests)."""
        return dataclasses.replace(self, name=name, **kw)


WORKLOADS = {
    "c1": Workload("c1", 1, 2_000, "er", 4.0, 250, "bernoulli", 0.02, 7, 2, 10, 100, 0, 20),
    "c2": Workload("c2", 2, 20_000, "ba", 5, 700, "normal", 0.0, 10, 3, 10, 500, 0, 50),
    # c3 is c2 with quantised p: same wid on purpose, so that every input array is identical
    "c3": Workload("c3", 2, 20_000, "ba", 5, 700, "normal", 0.0, 10, 3, 10, 500, 256, 50),
    "c4": Workload("c4", 4, 170_000, "ba", 7, 128, "normal", 0.0, 40, 4, 15, 1000, 256, 30),
    "c5": Workload("c5", 5, 90_000, "ba", 5, 500, "bernoulli", 0.05, 7, 3, 30, 2000, 16, 20),
}


def _rng(w: Workload, purpose: int, sub: int = 0) -> np.random.Generator:
    key = np.array([(BASE_SEED ^ w.wid) & 0xFFFFFFFFFFFFFFFF,
                    (purpose << 32) | sub], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def _dedupe_edges(n: int, a: np.ndarray, b: np.ndarray):
    """Undirected simple graph: drop self-loops and repeated pairs; lo < hi."""
    keep = a != b
    a, b = a[keep], b[keep]
    lo, hi = np.minimum(a, b), np.maximum(a, b)
    code = np.unique(lo.astype(np.int64) * n + hi.astype(np.int64))
    return (code // n).astype(np.int32), (code % n).astype(np.int32)


def erdos_renyi(n: int, avg_deg: float, rng: np.random.Generator):
    """G(n, p) with p = avg_deg / (n - 1): a binomial number of distinct pairs."""
    pairs = n * (n - 1) // 2
    p = min(1.0, avg_deg / max(n - 1, 1))
    m = int(rng.binomial(pairs, p)) if pairs > 0 else 0
    src = np.empty(0, np.int32)
    dst = np.empty(0, np.int32)
    while src.size < m:
        need = int((m - src.size) * 1.2) + 16
        a = rng.integers(0, n, size=need)
        b = rng.integers(0, n, size=need)
        if src.size:
            a = np.concatenate([src, a])
            b = np.concatenate([dst, b])
        src, dst = _dedupe_edges(n, a, b)
    if src.size > m:                      # unique() sorted the pairs: drop a seeded subset
        keep = np.sort(rng.choice(src.size, size=m, replace=False))
        src, dst = src[keep], dst[keep]
    return src, dst


def barabasi_albert(n: int, m: int, rng: np.random.Generator):
    """Preferential attachment, m edges per new node (Batagelj-Brandes edge array).

    Edge i joins node ``m + i // m`` to the endpoint stored at a uniformly
    chosen earlier position of the edge array, which is a degree-proportional
    choice.  Repeated pairs and self-loops are dropped afterwards, so the
    average degree is slightly below 2m.
    """
    m = int(m)
    if n <= m:
        return erdos_renyi(n, n - 1, rng)
    n_e = (n - m) * m
    new = (m + np.arange(n_e) // m).astype(np.int64)
    # position 2i holds new[i]; position 2i+1 copies position r[i] <= 2i.
    # seed nodes 0..m-1: the first m edges attach to them directly.
    r = (rng.random(n_e) * (2 * np.arange(n_e) + 1)).astype(np.int64)
    ptr = r.copy()
    ptr[:m] = 2 * np.arange(m) + 1        # the first m edges go to the seed nodes 0..m-1
    # an odd position 2j+1 with j < m holds seed node j; with j >= m it copies position r[j]
    follow = ((ptr & 1) == 1) & ((ptr - 1) // 2 >= m)
    for _ in range(128):                  # pointer jumping; chains are short
        if not follow.any():
            break
        ptr[follow] = r[(ptr[follow] - 1) // 2]
        follow = ((ptr & 1) == 1) & ((ptr - 1) // 2 >= m)
    other = np.where((ptr & 1) == 0, new[ptr // 2], (ptr - 1) // 2)
    return _dedupe_edges(n, new, other)


def make_graph(w: Workload):
    """Undirected simple edge list (each edge once, src < dst), int32."""
    rng = _rng(w, _P_GRAPH)
    if w.graph == "er":
        return erdos_renyi(w.n_nodes, float(w.graph_param), rng)
    if w.graph == "ba":
        return barabasi_albert(w.n_nodes, int(w.graph_param), rng)
    raise ValueError(w.graph)


def make_features(w: Workload) -> np.ndarray:
    """Node-major [N][d] float32."""
    rng = _rng(w, _P_FEAT)
    if w.feat_kind == "bernoulli":
        return (rng.random((w.n_nodes, w.feat_dim), dtype=np.float32) < w.feat_param).astype(np.float32)
    if w.feat_kind == "normal":
        return rng.standard_normal((w.n_nodes, w.feat_dim), dtype=np.float32)
    raise ValueError(w.feat_kind)


def make_labels(w: Workload) -> np.ndarray:
    return _rng(w, _P_LABEL).integers(0, w.n_classes, size=w.n_nodes).astype(np.int32)


def make_mask(w: Workload) -> np.ndarray:
    return (_rng(w, _P_MASK).random(w.n_nodes) < w.train_frac).astype(np.uint8)


def make_weights(w: Workload) -> List[np.ndarray]:
    """W_l^0 ~ N(0, 2 / n_{l-1}) as float32 [n_l][n_{l-1}], one generator per layer."""
    out = []
    n_in = w.n0
    for l, n_out in enumerate(w.widths):
        rng = _rng(w, _P_W, l)
        std = np.float32(np.sqrt(2.0 / n_in))
        out.append(rng.standard_normal((n_out, n_in), dtype=np.float32) * std)
        n_in = n_out
    return out


@dataclasses.dataclass
class Inputs:
    workload: Workload
    edge_src: np.ndarray
    edge_dst: np.ndarray
    features: np.ndarray
    labels: np.ndarray
    train_mask: np.ndarray
    init_W: List[np.ndarray]


def make_inputs(w: Workload, with_weights: bool = True) -> Inputs:
    src, dst = make_graph(w)
    return Inputs(w, src, dst, make_features(w), make_labels(w), make_mask(w),
                  make_weights(w) if with_weights else [])


def get(name: str) -> Workload:
    return WORKLOADS[name]


def small(name: str, n_nodes: int, feat_dim: Optional[int] = None, hidden: Optional[int] = None,
          n_layers: Optional[int] = None, **kw) -> Workload:
    """A reduced copy of a named workload (same generator, smaller sizes)."""
    w = WORKLOADS[name]
    rep = dict(n_nodes=n_nodes)
    if feat_dim is not None:
        rep["feat_dim"] = feat_dim
    if hidden is not None:
        rep["hidden"] = hidden
    if n_layers is not None:
        rep["n_layers"] = n_layers
    rep.update(kw)
    return w.scaled(f"{name}-small", **rep)
