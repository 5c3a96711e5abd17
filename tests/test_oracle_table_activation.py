"""Pins of the lookup-table z-update for smooth activations (tanh, sigmoid: the remark after Eq. "update z")."""

import numpy as np
import pytest

import oracle.pdadmm_oracle as o
from paper_2105_09837_b200 import synth

ACTS = {"tanh": np.tanh, "sigmoid": lambda x: 1.0 / (1.0 + np.exp(-x))}


def test_table_points_are_single_precision_and_span_the_range():
    pts = o.table_points(-4.0, 4.0, 257)
    assert pts.size == 257 and pts[0] == -4.0 and pts[128] == 0.0 and abs(pts[-1] - 4.0) < 1e-6
    assert np.array_equal(pts, pts.astype(np.float32).astype(np.float64))
    assert np.allclose(np.diff(pts), 8.0 / 256, rtol=0, atol=1e-6)


@pytest.mark.parametrize("name", ["tanh", "sigmoid"])
def test_table_update_is_the_best_candidate_and_close_to_the_continuous_minimum(name):
    """Brute force: the returned z has the smallest objective among all table points; against a much finer scalar grid
    (step 1e-4) its objective exceeds the continuous minimum by at most (M/2)(h/2)^2 with M a bound of the second
    derivative and h the table step, and its position is within half a step of a grid minimiser or ties it in value."""
    f = ACTS[name]
    rng = np.random.default_rng(11)
    a, q, zk = rng.normal(0, 1.2, 400), rng.normal(0, 1.0, 400), rng.normal(0, 1.2, 400)
    pts = o.table_points(-4.0, 4.0, 257)
    got = o.update_z_hidden_table(a, q, zk, f, pts)
    obj = lambda z, i: (z - a[i]) ** 2 + (q[i] - f(z)) ** 2 + (z - zk[i]) ** 2
    fine = np.arange(-4.0, 4.0 + 1e-9, 1e-4)
    h = 8.0 / 256
    for i in range(400):
        vals = obj(pts, i)
        assert got[i] in pts and abs(obj(got[i], i) - vals.min()) <= 1e-12 * vals.min()
        assert abs(got[i] - pts[np.argmin(vals)]) <= 8.0 / 256 + 1e-9 and abs(vals[np.argmin(vals)] - obj(got[i], i)) <= 1e-12 * vals.min()
        best_fine = obj(fine, i).min()
        M = 4.0 + 2.0 + 2.0 * (abs(q[i]) + 1.0)                    # |f'| <= 1, |f''| <= 1, |q - f| <= |q| + 1
        assert obj(got[i], i) <= best_fine + 0.5 * M * (h / 2) ** 2 + 1e-12


def test_table_update_reduces_to_the_midpoint_without_the_activation_term():
    """With f constant the objective is 2 (z - (a + z^k)/2)^2 + const: the table point nearest to the midpoint."""
    pts = o.table_points(-2.0, 2.0, 41)
    a, zk = np.array([0.31, -1.07, 1.96]), np.array([0.11, 0.5, 1.99])
    got = o.update_z_hidden_table(a, np.zeros(3), zk, lambda z: 0.0 * z, pts)
    mid = (a + zk) / 2
    assert np.array_equal(got, pts[np.argmin(np.abs(pts[None, :] - mid[:, None]), axis=1)])


@pytest.mark.parametrize("name", ["tanh", "sigmoid"])
def test_iteration_with_a_smooth_activation_keeps_lemma_q_opt_and_decreases_the_objective(name):
    """Lemma "q_opt" (u = nu (q - f(z))) only needs the q- and u-updates; the objective does not increase in the
    regime of the decrease lemma up to what the table's resolution costs the z-step."""
    w = synth.small("c1", 200, feat_dim=10, hidden=12, n_layers=4)
    inp = synth.make_inputs(w)
    A = o.renormalized_adjacency(w.n_nodes, inp.edge_src, inp.edge_dst)
    X = o.augment(inp.features.T.astype(np.float64), A, w.n_blocks)
    prm = o.Params(1.0, 0.01, 0, activation=name, table_size=1025)
    s = o.init_state(X, [x.astype(np.float64) for x in inp.init_W], inp.labels, inp.train_mask, prm)
    f = ACTS[name]
    assert np.allclose(s.q[0], f(s.z[0])) and np.allclose(o.residuals_sq(s), 0)
    prev = o.lagrangian(s, prm)
    pts = o.table_points(prm.table_lo, prm.table_hi, prm.table_size)
    for _ in range(6):
        s = o.iterate(s, prm)
        for l in range(s.L - 1):
            assert np.allclose(s.u[l], prm.nu * (s.q[l] - f(s.z[l])), rtol=0, atol=1e-13)
            assert np.all(np.isin(s.z[l], pts))
        cur = o.lagrangian(s, prm)
        assert cur <= prev + 1e-6 * abs(prev)
        prev = cur
    assert np.allclose(o.forward(s.p[0], s.W[:1], s.b[:1], prm.f), s.W[0] @ s.p[0] + s.b[0][:, None])
