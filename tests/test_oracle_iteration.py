"""Pins of the whole oracle iteration against the paper's lemmas and theorems."""

import numpy as np
import pytest

import oracle.pdadmm_oracle as o
from paper_2105_09837_b200 import synth


def _problem(n=240, d=12, hidden=14, L=4, name="c1"):
    w = synth.small(name, n, feat_dim=d, hidden=hidden, n_layers=L)
    inp = synth.make_inputs(w)
    A = o.renormalized_adjacency(w.n_nodes, inp.edge_src, inp.edge_dst)
    X = o.augment(inp.features.T.astype(np.float64), A, w.n_blocks)
    W0 = [x.astype(np.float64) for x in inp.init_W]
    return w, X, W0, inp.labels, inp.train_mask


def _sqdiff(a, b):
    return float(np.sum((a - b) ** 2))


def test_initial_state_is_feasible_and_satisfies_lemma_q_opt():
    w, X, W0, y, mask = _problem()
    prm = o.Params(1e-3, 1e-3, 0)
    s = o.init_state(X, W0, y, mask, prm)
    assert np.allclose(o.residuals_sq(s), 0)
    ob = o.objective(s, prm)
    assert np.allclose(ob[1:5], 0) and ob[0] > 0 and abs(ob[5] - ob[0]) < 1e-12
    for l in range(s.L - 1):
        assert np.array_equal(s.u[l], 1e-3 * (s.q[l] - o.relu(s.z[l])))
    # quantised start: p in Delta, residual not zero, one step per layer from max(q)
    prm = o.Params(1e-3, 1e-3, 16)
    s = o.init_state(X, W0, y, mask, prm)
    for l in range(1, s.L):
        lev = o.level_set(s.scale[l], 16)
        assert np.all(np.isin(s.p[l], lev))
        assert abs(s.scale[l] - float(np.float32(s.q[l - 1].max()) / np.float32(15))) == 0
        assert np.max(np.abs(s.p[l] - s.q[l - 1])) <= s.scale[l] / 2 * (1 + 1e-6)
    assert o.residuals_sq(s).sum() > 0


@pytest.mark.parametrize("m", [0, 16])
def test_lemma_q_opt_holds_every_iteration(m):
    """u_l^k = nu (q_l^k - f_l(z_l^k)) for every k (Lemma "q_opt"), with and without quantised p."""
    w, X, W0, y, mask = _problem()
    prm = o.Params(0.5, 0.02, m)
    s = o.init_state(X, W0, y, mask, prm)
    for _ in range(6):
        s = o.iterate(s, prm)
        for l in range(s.L - 1):
            assert np.allclose(s.u[l], prm.nu * (s.q[l] - o.relu(s.z[l])), rtol=0, atol=1e-13)


@pytest.mark.parametrize("m", [0, 16])
def test_objective_decrease_lemma(m):
    """rho > max(4 nu S^2, (sqrt(17)+1) nu / 2), S = 1: L_rho (beta_rho) decreases by at least the
    right-hand side of Lemma (Objective Decrease); it is bounded below (Lemma Bounded Objective)."""
    w, X, W0, y, mask = _problem()
    rho, nu = 1.0, 0.01
    assert rho > max(4 * nu, (np.sqrt(17) + 1) * nu / 2)
    C1 = nu / 2 - 2 * nu * nu / rho
    C2 = rho / 2 - 2 * nu * nu / rho - nu / 2
    prm = o.Params(rho, nu, m)
    s = o.init_state(X, W0, y, mask, prm)
    prev = o.lagrangian(s, prm)
    bounds = []
    for k in range(25):
        n = o.iterate(s, prm)
        cur = o.lagrangian(n, prm)
        L = s.L
        rhs = sum(0.5 * n.theta[l] * _sqdiff(n.W[l], s.W[l]) for l in range(L))
        rhs += sum(0.5 * nu * _sqdiff(n.b[l], s.b[l]) for l in range(L))
        rhs += sum(C1 * _sqdiff(n.z[l], s.z[l]) for l in range(L - 1)) + 0.5 * nu * _sqdiff(n.z[L - 1], s.z[L - 1])
        rhs += sum(C2 * _sqdiff(n.q[l], s.q[l]) for l in range(L - 1))
        if m == 0:
            rhs += sum(0.5 * n.tau[l] * _sqdiff(n.p[l], s.p[l]) for l in range(1, L))
        assert prev - cur >= rhs - 1e-9 * (1 + abs(prev))
        assert cur > -1e-9                      # R >= 0 and rho > nu: bounded below by 0 here
        bounds.append(rhs)
        s, prev = n, cur
    assert bounds[-1] < bounds[2]               # successive differences die out (Theorem Convergent Objective)


def test_c_k_of_the_rate_theorem_is_nonincreasing_and_summable():
    w, X, W0, y, mask = _problem(n=150, L=3)
    rho, nu = 1.0, 0.01
    C1 = nu / 2 - 2 * nu * nu / rho
    C2 = rho / 2 - 2 * nu * nu / rho - nu / 2
    prm = o.Params(rho, nu, 0)
    s = o.init_state(X, W0, y, mask, prm)
    L0 = o.lagrangian(s, prm)
    terms = []
    for k in range(30):
        n = o.iterate(s, prm)
        L = s.L
        t = sum(0.5 * n.tau[l] * _sqdiff(n.p[l], s.p[l]) for l in range(1, L))
        t += sum(0.5 * n.theta[l] * _sqdiff(n.W[l], s.W[l]) + 0.5 * nu * _sqdiff(n.b[l], s.b[l]) for l in range(L))
        t += sum(C1 * _sqdiff(n.z[l], s.z[l]) + C2 * _sqdiff(n.q[l], s.q[l]) for l in range(L - 1))
        t += 0.5 * nu * _sqdiff(n.z[L - 1], s.z[L - 1])
        terms.append(t)
        s = n
    c = np.minimum.accumulate(terms)
    assert np.all(np.diff(c) <= 0) and np.all(c >= 0)
    assert sum(terms) <= L0 - o.lagrangian(s, prm) + 1e-9


@pytest.mark.parametrize("m", [0, 256])
def test_residual_shrinks_at_rho_equal_nu(m):
    """rho = nu = 1e-3 (outside the proven regime): the primal residual sum ||p_{l+1} - q_l||^2
    falls well below its early peak and every value stays finite."""
    w, X, W0, y, mask = _problem(n=300, d=20, hidden=16, L=4)
    prm = o.Params(1e-3, 1e-3, m)
    s = o.init_state(X, W0, y, mask, prm)
    res = []
    for _ in range(30):
        s = o.iterate(s, prm)
        res.append(o.residuals_sq(s).sum())
        assert all(np.all(np.isfinite(v)) for v in s.p + s.W + s.z + s.q + s.u)
    assert res[-1] < 0.1 * max(res[:8])
    assert np.isfinite(o.lagrangian(s, prm))


def test_iteration_order_uses_new_p_in_W_and_old_q_in_p():
    """The W-update sees p^{k+1}; the p-update sees q^k, u^k (Algorithm 1)."""
    w, X, W0, y, mask = _problem(n=80, d=6, hidden=7, L=3)
    prm = o.Params(0.3, 0.05, 0)
    s = o.init_state(X, W0, y, mask, prm)
    s = o.iterate(s, prm)
    s = o.iterate(s, prm)
    n = o.iterate(s, prm)
    l = 1
    p_new, tau = o.update_p(s.p[l], s.W[l], s.b[l], s.z[l], prm.nu, s.q[l - 1], s.u[l - 1], prm.rho)
    assert np.array_equal(n.p[l], p_new)
    W_new, theta = o.update_W(p_new, s.W[l], s.b[l], s.z[l], prm.nu)
    assert np.array_equal(n.W[l], W_new)
    assert not np.array_equal(W_new, o.update_W(s.p[l], s.W[l], s.b[l], s.z[l], prm.nu)[0])
    b_new = o.update_b(p_new, W_new, s.b[l], s.z[l], prm.nu)
    assert np.array_equal(n.b[l], b_new)
    a = W_new @ p_new + b_new[:, None]
    assert np.array_equal(n.z[l], o.update_z_hidden(a, s.q[l], s.z[l]))
    assert np.array_equal(n.q[0], o.update_q(n.p[1], s.u[0], n.z[0], prm.rho, prm.nu))
    assert np.array_equal(n.u[0], o.update_u(s.u[0], n.p[1], n.q[0], prm.rho))
    assert np.array_equal(n.p[0], s.p[0])       # p_1 = X never moves


def test_single_layer_model_fixed_point_condition():
    """L = 1: the state is (W_1, b_1, z_1); after the z-update the labelled columns satisfy
    z = W X + b + (e_y - softmax(z)) / nu, the stationarity of Eq. (update zl)."""
    w, X, W0, y, mask = _problem(n=60, d=5, hidden=4, L=1)
    prm = o.Params(1.0, 0.1, 0)
    s = o.init_state(X, W0, y, mask, prm)
    assert len(s.q) == 0 and len(s.u) == 0 and len(s.p) == 1
    for _ in range(3):
        s = o.iterate(s, prm)
    a = s.W[0] @ s.p[0] + s.b[0][:, None]
    E = np.zeros_like(a)
    E[s.y, np.arange(a.shape[1])] = 1
    S = np.exp(s.z[0] - s.z[0].max(0))
    S /= S.sum(0)
    lab = s.mask
    assert np.allclose(s.z[0][:, lab], (a + (E - S) / prm.nu)[:, lab], atol=1e-9)
    assert np.array_equal(s.z[0][:, ~lab], a[:, ~lab])


def test_forward_pass_golden_and_consistency_with_a_feasible_state():
    import os
    want = np.loadtxt(os.path.join(os.path.dirname(__file__), "golden", "forward_two_layers.txt"))
    X = np.array([[1.0, 2.0], [-1.0, 0.0]])
    W = [np.array([[1.0, 0], [0, 1], [1, 1]]), np.array([[1.0, -1, 0], [0, 2, 1]])]
    b = [np.array([0.0, 1.0, -1.0]), np.array([0.5, 0.0])]
    assert np.array_equal(o.forward(X, W, b), want)
    assert o.predict(X, W, b).tolist() == [0, 1]
    assert o.accuracy([0, 1], [0, 0], [True, True]) == 0.5 and o.accuracy([0, 1], [0, 0], [True, False]) == 1.0
    # the start of Algorithm 1 is a forward pass with b = 0: its z_L is the model's output
    w, X, W0, y, mask = _problem()
    s = o.init_state(X, W0, y, mask, o.Params(1e-3, 1e-3, 0))
    assert np.allclose(o.forward(X, s.W, s.b), s.z[-1], rtol=1e-12, atol=1e-12)
    # a bias on the last layer only shifts the logits; a large one decides the class
    b2 = [x.copy() for x in s.b]
    b2[-1][3] += 1e6
    assert np.all(o.predict(X, s.W, b2) == 3)


def test_leaky_relu_keeps_lemma_q_opt_and_the_objective_decrease():
    """The proofs only use that f_l is Lipschitz with constant S <= 1, which a leaky ReLU is: Lemma "q_opt" holds
    at every iteration and, for rho large enough, L_rho does not increase."""
    w, X, W0, y, mask = _problem()
    prm = o.Params(1.0, 0.01, 0, slope=0.2)
    s = o.init_state(X, W0, y, mask, prm)
    assert np.allclose(o.residuals_sq(s), 0) and np.any(s.q[0] < 0)          # negative activations pass
    prev = o.lagrangian(s, prm)
    for _ in range(6):
        s = o.iterate(s, prm)
        for l in range(s.L - 1):
            assert np.allclose(s.u[l], prm.nu * (s.q[l] - np.where(s.z[l] > 0, s.z[l], 0.2 * s.z[l])), rtol=0, atol=1e-13)
        cur = o.lagrangian(s, prm)
        assert cur <= prev + 1e-9 * abs(prev)
        prev = cur
    # the forward pass uses the same activation
    z1 = s.W[0] @ s.p[0] + s.b[0][:, None]
    p2 = np.where(z1 > 0, z1, 0.2 * z1)
    assert np.allclose(o.forward(s.p[0], s.W[:2], s.b[:2], 0.2), s.W[1] @ p2 + s.b[1][:, None])
