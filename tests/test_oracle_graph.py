"""Pins of the oracle's graph pre-processing, augmentation and quantisation set."""

import os

import numpy as np
import pytest

import oracle.pdadmm_oracle as o
from paper_2105_09837_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _dense_renorm(n, src, dst):
    """Dense statement of A~ = (D+I)^{-1/2}(A+I)(D+I)^{-1/2} from a set of edges."""
    A = np.zeros((n, n))
    for a, b in set((min(int(a), int(b)), max(int(a), int(b))) for a, b in zip(src, dst) if a != b):
        A[a, b] = A[b, a] = 1.0
    D = np.diag(A.sum(axis=1)) + np.eye(n)
    Dm = np.diag(1.0 / np.sqrt(np.diag(D)))
    return Dm @ (A + np.eye(n)) @ Dm


def test_golden_path_graph():
    want = np.loadtxt(os.path.join(GOLD, "path3_renormalized_adjacency.txt"))
    got = o.renormalized_adjacency(3, [0, 1], [1, 2]).toarray()
    assert np.allclose(got, want, rtol=0, atol=1e-15)


def test_golden_star_two_hops():
    want = np.loadtxt(os.path.join(GOLD, "star4_two_hop.txt"))
    A = o.renormalized_adjacency(4, [0, 0, 0], [1, 2, 3])
    X = o.augment(np.array([[1.0, 0, 0, 0]]), A, 3)
    assert np.allclose(X, want, rtol=0, atol=1e-15)


def test_adjacency_against_dense_definition_and_edge_set():
    w = synth.small("c2", 150, feat_dim=5)
    src, dst = synth.make_graph(w)
    # hand the oracle a messy list: repeats, both directions, self-loops
    s2 = np.concatenate([src, dst[:20], [3, 3]])
    d2 = np.concatenate([dst, src[:20], [3, 7]])
    A = o.renormalized_adjacency(w.n_nodes, s2, d2)
    dense = _dense_renorm(w.n_nodes, s2, d2)
    assert np.allclose(A.toarray(), dense, rtol=0, atol=1e-15)
    assert abs(A - A.T).max() < 1e-16
    # structure: the pattern of A + I, columns ascending in every row
    want = set((int(a), int(b)) for a, b in zip(s2, d2) if a != b)
    want |= set((b, a) for a, b in want) | set((i, i) for i in range(w.n_nodes))
    coo = A.tocoo()
    assert set(zip(coo.row.tolist(), coo.col.tolist())) == want
    for i in range(w.n_nodes):
        cols = A.indices[A.indptr[i]:A.indptr[i + 1]]
        assert np.all(np.diff(cols) > 0)


@pytest.mark.parametrize("name,n", [("c1", 200), ("c2", 120)])
def test_augmentation_equals_dense_matrix_powers(name, n):
    w = synth.small(name, n, feat_dim=6, n_hops=3)
    inp = synth.make_inputs(w, with_weights=False)
    A = o.renormalized_adjacency(n, inp.edge_src, inp.edge_dst)
    H = inp.features.T.astype(np.float64)
    X = o.augment(H, A, w.n_blocks)
    Ad = _dense_renorm(n, inp.edge_src, inp.edge_dst)
    want = np.concatenate([H @ np.linalg.matrix_power(Ad, k) for k in range(w.n_blocks)], axis=0)
    assert X.shape == (w.n_blocks * 6, n)
    assert np.allclose(X, want, rtol=1e-13, atol=1e-14)


def test_augmentation_fixed_vector_and_contraction():
    """h_i = sqrt(d_i + 1) is an eigenvector of A~ with eigenvalue 1, and ||A~||_2 <= 1."""
    w = synth.small("c2", 300, feat_dim=4)
    src, dst = synth.make_graph(w)
    A = o.renormalized_adjacency(w.n_nodes, src, dst)
    deg = np.bincount(np.concatenate([src, dst]), minlength=w.n_nodes)
    h = np.sqrt(deg + 1.0)[None, :]
    X = o.augment(h, A, 5)
    for k in range(5):
        assert np.allclose(X[k], h[0], rtol=1e-13)
    rng = np.random.default_rng(5)
    X = o.augment(rng.standard_normal((3, w.n_nodes)), A, 6)
    norms = [np.linalg.norm(X[3 * k:3 * k + 3]) for k in range(6)]
    assert all(norms[k + 1] <= norms[k] * (1 + 1e-12) for k in range(5))


def test_generators_are_simple_graphs_and_reproducible():
    for name, n in [("c1", 500), ("c2", 500), ("c4", 700)]:
        w = synth.small(name, n, feat_dim=3)
        s1, d1 = synth.make_graph(w)
        s2, d2 = synth.make_graph(w)
        assert np.array_equal(s1, s2) and np.array_equal(d1, d2)
        assert np.all(s1 < d1) and s1.min() >= 0 and d1.max() < n
        assert len(set(zip(s1.tolist(), d1.tolist()))) == s1.size
    w = synth.get("c2")
    s, d = synth.make_graph(w)
    assert abs(2 * s.size / w.n_nodes - 10) < 0.5          # Barabasi-Albert m=5 -> average degree about 10
    deg = np.bincount(np.concatenate([s, d]), minlength=w.n_nodes)
    assert deg.max() > 20 * deg.mean()                     # heavy tail
    assert synth.get("c3").wid == synth.get("c2").wid      # c3 shares every input with c2


# ------------------------------------------------------------------ quantisation

@pytest.mark.parametrize("m", [2, 16, 256])
def test_quantize_is_nearest_level_brute_force(m):
    rng = np.random.default_rng(m)
    scale = float(np.float32(0.0173))
    x = rng.uniform(-0.5, (m + 2) * scale, size=4000)
    x[:m] = (np.arange(m) + 0.5) * scale                    # exact half-levels: ties go up (or clamp)
    codes, vals = o.quantize(x, scale, m)
    levels = o.level_set(scale, m)
    assert codes.dtype == np.uint8 and codes.max() <= m - 1
    assert np.array_equal(vals, levels[codes])               # p is in Delta, bit for bit
    x32 = x.astype(np.float32).astype(np.float64)            # the decision is taken on the fp32 value
    dist = np.abs(x32[:, None] - levels[None, :])
    best = dist.min(axis=1)
    mine = np.abs(x32 - vals)
    # nearest up to the rounding of the fp32 division (a few ulp of x)
    assert np.all(mine <= best + 4e-7 * np.maximum(np.abs(x32), scale))
    far = np.abs(np.abs(x32 / scale - np.floor(x32 / scale)) - 0.5) > 1e-4
    assert np.array_equal(codes[far], dist.argmin(axis=1)[far].astype(np.uint8))


def test_quantize_ties_and_clamps():
    s = 0.5
    codes, vals = o.quantize(np.array([-3.0, -0.25, 0.24, 0.25, 0.75, 1.2, 100.0]), s, 4)
    assert codes.tolist() == [0, 0, 0, 1, 2, 2, 3]
    assert vals.tolist() == [0.0, 0.0, 0.0, 0.5, 1.0, 1.0, 1.5]


def test_quantization_scale():
    assert o.quantization_scale(np.array([[0.0, 2.55], [1.0, -4.0]]), 256) == float(np.float32(2.55) / np.float32(255))
    assert o.quantization_scale(np.zeros((2, 2)), 16) == 1.0
