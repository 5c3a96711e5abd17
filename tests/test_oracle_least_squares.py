"""Pins of the least-squares risk (Sec. "Problem Formulation": R only has to be convex and continuous)."""

import numpy as np

import oracle.pdadmm_oracle as o
from paper_2105_09837_b200 import synth


def test_z_last_is_the_minimiser_by_grid_search_and_stationarity():
    """Per labelled node the subproblem is (1/2)||z - e_y||^2 + (nu/2)||z - a||^2, separable over the classes: a
    dense scalar grid per class finds the same minimiser; its gradient vanishes; unlabelled nodes keep a."""
    rng = np.random.default_rng(5)
    C, n = 4, 9
    a = rng.standard_normal((C, n)) * 2.0
    y = rng.integers(0, C, n)
    mask = np.array([1, 1, 0, 1, 0, 1, 1, 1, 0], dtype=bool)
    grid = np.linspace(-6.0, 6.0, 120001)                       # step 1e-4
    for nu in (0.01, 1.0, 7.5):
        z = o.update_z_last_least_squares(a, y, mask, nu)
        for j in range(n):
            e = np.zeros(C); e[y[j]] = 1.0
            if not mask[j]:
                assert np.array_equal(z[:, j], a[:, j])
                continue
            assert np.allclose((z[:, j] - e) + nu * (z[:, j] - a[:, j]), 0.0, atol=1e-14)
            for c in range(C):
                f = 0.5 * (grid - e[c]) ** 2 + 0.5 * nu * (grid - a[c, j]) ** 2
                assert abs(grid[np.argmin(f)] - z[c, j]) <= 1e-4
    # limits: nu -> 0 gives the label, nu -> infinity gives a
    assert np.allclose(o.update_z_last_least_squares(a, y, mask, 1e-12)[:, 0], np.eye(C)[y[0]], atol=1e-10)
    assert np.allclose(o.update_z_last_least_squares(a, y, mask, 1e12)[:, 0], a[:, 0], atol=1e-10)


def test_risk_written_out_on_a_hand_example():
    z = np.array([[1.0, 0.5, 2.0], [0.0, -1.0, 3.0]])          # 2 classes, 3 nodes
    y = np.array([0, 1, 1])
    mask = np.array([True, True, False])
    # node 0: ||(1,0) - (1,0)||^2 = 0 ; node 1: ||(0.5,-1) - (0,1)||^2 = 0.25 + 4 ; node 2 is not labelled
    assert o.risk_least_squares(z, y, mask) == 0.5 * 4.25


def test_iteration_keeps_lemma_q_opt_and_decreases_the_objective():
    """The lemmas hold for any proper risk: u = nu (q - f(z)) after every iteration, and for rho large enough L_rho
    does not increase and stays above 0 (R >= 0)."""
    w = synth.small("c1", 240, feat_dim=12, hidden=14, n_layers=4)
    inp = synth.make_inputs(w)
    A = o.renormalized_adjacency(w.n_nodes, inp.edge_src, inp.edge_dst)
    X = o.augment(inp.features.T.astype(np.float64), A, w.n_blocks)
    prm = o.Params(1.0, 0.01, 0, risk="ls")
    s = o.init_state(X, [x.astype(np.float64) for x in inp.init_W], inp.labels, inp.train_mask, prm)
    prev = o.lagrangian(s, prm)
    first = prev
    for _ in range(12):
        s = o.iterate(s, prm)
        for l in range(s.L - 1):
            assert np.allclose(s.u[l], prm.nu * (s.q[l] - np.maximum(s.z[l], 0)), rtol=0, atol=1e-13)
        cur = o.lagrangian(s, prm)
        assert -1e-12 < cur <= prev + 1e-9 * abs(prev)
        prev = cur
    assert prev < 0.9 * first
    # the last layer's z is the closed form of its own inputs
    a = s.W[-1] @ s.p[-1] + s.b[-1][:, None]
    assert np.allclose(s.z[-1], o.update_z_last_least_squares(a, s.y, s.mask, prm.nu))
    # and the objective's first component is this risk, not the cross-entropy
    assert o.objective(s, prm)[0] == o.risk_least_squares(s.z[-1], s.y, s.mask)
    assert o.objective(s, prm)[0] != o.risk(s.z[-1], s.y, s.mask)
