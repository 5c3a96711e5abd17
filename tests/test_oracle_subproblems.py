"""Pins of every subproblem solver of the oracle against what the paper and the mathematics fix:
brute-force grid search on tiny inputs, finite differences, optimality conditions, closed forms."""

import itertools

import numpy as np
import pytest

import oracle.pdadmm_oracle as o


def _layer(rng, n_in=3, n_out=2, N=4):
    p = rng.standard_normal((n_in, N))
    W = rng.standard_normal((n_out, n_in))
    b = rng.standard_normal(n_out)
    z = rng.standard_normal((n_out, N))
    q_prev = rng.standard_normal((n_in, N))
    u_prev = rng.standard_normal((n_in, N))
    return p, W, b, z, q_prev, u_prev


NU, RHO = 0.7, 1.3


# ------------------------------------------------------------------ gradients of phi (finite differences)

def test_gradients_of_phi_by_finite_differences():
    rng = np.random.default_rng(1)
    p, W, b, z, qp, up = _layer(rng)
    h = 1e-6
    g = o.grad_p_phi(p, W, b, z, NU, qp, up, RHO)
    for idx in itertools.product(range(p.shape[0]), range(p.shape[1])):
        e = np.zeros_like(p)
        e[idx] = h
        fd = (o.phi(p + e, W, b, z, NU, qp, up, RHO) - o.phi(p - e, W, b, z, NU, qp, up, RHO)) / (2 * h)
        assert abs(fd - g[idx]) < 1e-7 * (1 + abs(fd))
    G = o.grad_W_phi(p, W, b, z, NU)
    for idx in itertools.product(range(W.shape[0]), range(W.shape[1])):
        e = np.zeros_like(W)
        e[idx] = h
        fd = (o.phi(p, W + e, b, z, NU, qp, up, RHO) - o.phi(p, W - e, b, z, NU, qp, up, RHO)) / (2 * h)
        assert abs(fd - G[idx]) < 1e-7 * (1 + abs(fd))
    gb = o.grad_b_phi(p, W, b, z, NU)
    for i in range(b.size):
        e = np.zeros_like(b)
        e[i] = h
        fd = (o.phi(p, W, b + e, z, NU, qp, up, RHO) - o.phi(p, W, b - e, z, NU, qp, up, RHO)) / (2 * h)
        assert abs(fd - gb[i]) < 1e-7 * (1 + abs(fd))


def test_phi_written_out_on_scalars():
    """phi with every array 1x1 is a formula one can evaluate by hand."""
    p, W, b, z, q, u = 2.0, 3.0, -1.0, 4.0, 0.5, 0.25
    want = 0.5 * NU * (z - W * p - b) ** 2 + u * (p - q) + 0.5 * RHO * (p - q) ** 2
    A = lambda v: np.array([[v]])
    got = o.phi(A(p), A(W), np.array([b]), A(z), NU, A(q), A(u), RHO)
    assert abs(got - want) < 1e-14
    assert abs(o.phi(A(p), A(W), np.array([b]), A(z), NU) - 0.5 * NU * (z - W * p - b) ** 2) < 1e-14


# ------------------------------------------------------------------ p-update

def test_p_update_minimises_U_grid_search():
    """On a 1x2 problem the minimiser of U_l(.; tau) over a grid is p - g/tau."""
    rng = np.random.default_rng(2)
    p, W, b, z, qp, up = _layer(rng, n_in=1, n_out=2, N=2)
    tau = 3.7
    g = o.grad_p_phi(p, W, b, z, NU, qp, up, RHO)
    want = p - g / tau
    grid = np.linspace(-0.5, 0.5, 201)
    best, arg = np.inf, None
    for d0 in grid:
        for d1 in grid:
            cand = want + np.array([[d0, d1]])
            val = o.U_model(cand, p, W, b, z, NU, qp, up, RHO, tau)
            if val < best:
                best, arg = val, cand
    assert np.allclose(arg, want, atol=1e-12)


def test_p_update_identity_and_smallest_tau():
    rng = np.random.default_rng(3)
    p, W, b, z, qp, up = _layer(rng, 5, 4, 7)
    p_new, tau = o.update_p(p, W, b, z, NU, qp, up, RHO)
    g = o.grad_p_phi(p, W, b, z, NU, qp, up, RHO)
    assert np.allclose(g + tau * (p_new - p), 0, atol=1e-12)        # optimality condition of Eq. (update p)
    phi0 = o.phi(p, W, b, z, NU, qp, up, RHO)
    Uval = o.U_model(p_new, p, W, b, z, NU, qp, up, RHO, tau)
    # phi(p^k) - U_l(p^{k+1}; tau) = (tau/2)||p^{k+1} - p^k||^2  (proof of Lemma "optimality 1")
    assert abs((phi0 - Uval) - 0.5 * tau * np.sum((p_new - p) ** 2)) < 1e-11
    # tau is admissible with equality, and 1% less is not admissible
    assert abs(o.phi(p_new, W, b, z, NU, qp, up, RHO) - Uval) < 1e-10
    t2 = 0.99 * tau
    p2 = p - g / t2
    assert o.phi(p2, W, b, z, NU, qp, up, RHO) > o.U_model(p2, p, W, b, z, NU, qp, up, RHO, t2)
    t3 = 1.01 * tau
    p3 = p - g / t3
    assert o.phi(p3, W, b, z, NU, qp, up, RHO) < o.U_model(p3, p, W, b, z, NU, qp, up, RHO, t3)
    # the generic search by definition, started below, brackets it
    tb = o.tau_by_backtracking(p, W, b, z, NU, qp, up, RHO, tau0=RHO)
    assert tau <= tb * (1 + 1e-12) and tb < 2 * tau
    assert tau >= RHO


def test_p_update_zero_gradient():
    rng = np.random.default_rng(4)
    p, W, b, z, qp, up = _layer(rng)
    z = W @ p + b[:, None]
    qp, up = p.copy(), np.zeros_like(p)
    p_new, tau = o.update_p(p, W, b, z, NU, qp, up, RHO)
    assert tau == RHO and np.array_equal(p_new, p)


# ------------------------------------------------------------------ quantised p-update

def test_quantised_p_update_properties():
    rng = np.random.default_rng(5)
    m, scale = 16, float(np.float32(0.21))
    p, W, b, z, qp, up = _layer(rng, 6, 5, 40)
    p = o.quantize(np.abs(p), scale, m)[1]
    p_new, codes, tau, trials = o.update_p_quantized(p, W, b, z, NU, qp, up, RHO, scale, m)
    levels = o.level_set(scale, m)
    assert trials >= 1
    assert np.array_equal(p_new, levels[codes])                      # p in Delta
    # accepted tau satisfies the stop condition phi(p+) <= U_l(p+; tau)
    assert o.phi(p_new, W, b, z, NU, qp, up, RHO) <= o.U_model(p_new, p, W, b, z, NU, qp, up, RHO, tau) * (1 + 1e-12) + 1e-12
    # p+ is the nearest level to the linearised step, by brute force over all levels
    g = o.grad_p_phi(p, W, b, z, NU, qp, up, RHO)
    x = (p - g / tau).astype(np.float32).astype(np.float64)
    best = np.abs(x[..., None] - levels).min(axis=-1)
    assert np.all(np.abs(x - p_new) <= best + 1e-6)
    # the quadratic-form version of the stop condition is the same statement
    d = p_new - p
    lhs = NU * np.sum((W @ d) ** 2) + RHO * np.sum(d * d)
    assert lhs <= tau * np.sum(d * d) * (1 + 1e-6)
    # beta_rho does not increase over the p-update (Lemma "optimality 1", pdADMM-G-Q line)
    assert o.phi(p_new, W, b, z, NU, qp, up, RHO) <= o.phi(p, W, b, z, NU, qp, up, RHO) + 1e-12


def test_quantised_p_update_needs_more_than_one_trial_sometimes():
    """A direction with a larger Rayleigh quotient than g forces tau to grow: the search is exercised."""
    rng = np.random.default_rng(11)
    seen = set()
    for seed in range(40):
        rng = np.random.default_rng(100 + seed)
        m, scale = 4, 1.0
        p, W, b, z, qp, up = _layer(rng, 4, 6, 3)
        W = W * 3
        p = o.quantize(np.abs(p), scale, m)[1]
        p_new, codes, tau, trials = o.update_p_quantized(p, W, b, z, 1.0, qp, up, 0.1, scale, m)
        seen.add(trials)
        d = p_new - p
        assert 1.0 * np.sum((W @ d) ** 2) + 0.1 * np.sum(d * d) <= tau * np.sum(d * d) * (1 + 1e-6)
    assert any(t > 1 for t in seen)


def test_many_levels_reproduce_unquantised_step():
    rng = np.random.default_rng(6)
    p, W, b, z, qp, up = _layer(rng, 6, 5, 30)
    p, qp = np.abs(p) + 1.0, np.abs(qp) + 1.0
    m, scale = 256, float(np.float32(6.0 / 255))
    pq = o.quantize(p, scale, m)[1]
    cont, tau_c = o.update_p(pq, W, b, z, 1e-3, qp, up, 1.0)
    disc, _, tau_q, trials = o.update_p_quantized(pq, W, b, z, 1e-3, qp, up, 1.0, scale, m)
    if trials == 1:
        assert tau_q == tau_c
        inside = (cont > 0) & (cont < 255 * scale)
        assert np.all(np.abs(disc - cont)[inside] <= scale / 2 * (1 + 1e-6))


# ------------------------------------------------------------------ W-update

def test_W_update_minimises_V_grid_search():
    rng = np.random.default_rng(7)
    p, W, b, z, _, _ = _layer(rng, n_in=2, n_out=1, N=3)
    theta = 2.9
    G = o.grad_W_phi(p, W, b, z, NU)
    want = W - G / theta
    grid = np.linspace(-0.5, 0.5, 201)
    best, arg = np.inf, None
    for d0 in grid:
        for d1 in grid:
            cand = want + np.array([[d0, d1]])
            val = o.V_model(cand, W, p, b, z, NU, theta)
            if val < best:
                best, arg = val, cand
    assert np.allclose(arg, want, atol=1e-12)


def test_W_update_identity_and_smallest_theta():
    rng = np.random.default_rng(8)
    p, W, b, z, _, _ = _layer(rng, 5, 4, 9)
    W_new, theta = o.update_W(p, W, b, z, NU)
    G = o.grad_W_phi(p, W, b, z, NU)
    assert np.allclose(G + theta * (W_new - W), 0, atol=1e-12)
    phi0 = o.phi(p, W, b, z, NU)
    Vval = o.V_model(W_new, W, p, b, z, NU, theta)
    assert abs((phi0 - Vval) - 0.5 * theta * np.sum((W_new - W) ** 2)) < 1e-11
    assert abs(o.phi(p, W_new, b, z, NU) - Vval) < 1e-10
    t2 = 0.99 * theta
    W2 = W - G / t2
    assert o.phi(p, W2, b, z, NU) > o.V_model(W2, W, p, b, z, NU, t2)
    tb = o.theta_by_backtracking(p, W, b, z, NU, theta0=theta / 1000.0)
    assert theta <= tb * (1 + 1e-12) and tb < 2 * theta
    # zero gradient: W stays
    zz = W @ p + b[:, None]
    W3, th3 = o.update_W(p, W, b, zz, NU)
    assert th3 == 0.0 and np.array_equal(W3, W)


# ------------------------------------------------------------------ b-update

def test_b_update_is_the_minimiser_grid_and_gradient():
    rng = np.random.default_rng(9)
    p, W, b, z, _, _ = _layer(rng, n_in=3, n_out=1, N=5)
    b_new = o.update_b(p, W, b, z, NU)
    assert np.allclose(b_new, np.mean(z - W @ p, axis=1))
    assert np.allclose(o.grad_b_phi(p, W, b_new, z, NU), 0, atol=1e-13)
    grid = b_new[0] + np.linspace(-1, 1, 2001)
    vals = [o.phi(p, W, np.array([v]), z, NU) for v in grid]
    assert abs(grid[int(np.argmin(vals))] - b_new[0]) < 1e-12
    # descent inequality of Lemma "optimality 1" (b line) holds with the step that is used
    assert o.phi(p, W, b, z, NU) - o.phi(p, W, b_new, z, NU) >= 0.5 * NU * np.sum((b_new - b) ** 2) - 1e-12


def test_b_update_as_printed_diverges_for_three_nodes():
    """Dividing by nu (as printed) instead of nu|V| multiplies the error by (1 - |V|) per step."""
    rng = np.random.default_rng(10)
    p, W, b, z, _, _ = _layer(rng, n_in=2, n_out=2, N=3)
    b_star = np.mean(z - W @ p, axis=1)
    b1 = o.update_b_literal(p, W, b, z, NU)
    assert np.allclose(b1 - b_star, (1 - 3) * (b - b_star))
    assert o.phi(p, W, b1, z, NU) > o.phi(p, W, b, z, NU)


# ------------------------------------------------------------------ z-update, hidden layers

def test_z_hidden_against_dense_scalar_grid():
    rng = np.random.default_rng(12)
    a = rng.uniform(-3, 3, 300)
    q = rng.uniform(-1, 3, 300)
    zk = rng.uniform(-3, 3, 300)
    got = o.update_z_hidden(a, q, zk)
    grid = np.arange(-5.0, 5.0 + 1e-9, 1e-4)
    for i in range(300):
        vals = o.z_objective_hidden(grid, a[i], q[i], zk[i])
        j = int(np.argmin(vals))
        f_got = o.z_objective_hidden(got[i], a[i], q[i], zk[i])
        assert f_got <= vals[j] + 1e-12                     # at least as good as the best grid point
        assert abs(got[i] - grid[j]) <= 1e-4 or abs(f_got - vals[j]) < 1e-7    # same point unless a near-tie
    # inequality (z minimize) of the proof: the new z is no worse than the old one
    lhs = o.z_objective_hidden(got, a, q, zk)
    rhs = (zk - a) ** 2 + (q - o.relu(zk)) ** 2
    assert np.all(lhs <= rhs + 1e-12)


@pytest.mark.parametrize("slope", [0.1, 0.3, 0.9])
def test_z_hidden_leaky_relu_against_dense_scalar_grid(slope):
    """f(x) = x for x > 0, slope * x otherwise: the z-subproblem (z-a)^2 + (q-f(z))^2 + (z-z^k)^2 per element,
    minimised over a dense grid, agrees with the closed form."""
    rng = np.random.default_rng(int(slope * 100))
    a = rng.uniform(-3, 3, 200)
    q = rng.uniform(-2, 3, 200)
    zk = rng.uniform(-3, 3, 200)
    got = o.update_z_hidden(a, q, zk, slope)
    grid = np.arange(-6.0, 6.0 + 1e-9, 1e-4)
    f_grid = np.where(grid > 0, grid, slope * grid)
    for i in range(200):
        vals = (grid - a[i]) ** 2 + (q[i] - f_grid) ** 2 + (grid - zk[i]) ** 2
        j = int(np.argmin(vals))
        f_got = (got[i] - a[i]) ** 2 + (q[i] - (got[i] if got[i] > 0 else slope * got[i])) ** 2 + (got[i] - zk[i]) ** 2
        assert f_got <= vals[j] + 1e-12
        assert abs(got[i] - grid[j]) <= 1e-4 or abs(f_got - vals[j]) < 1e-7
    assert np.array_equal(o.update_z_hidden(a, q, zk, 0.0), o.update_z_hidden(a, q, zk))     # slope 0 is ReLU


def test_z_hidden_special_cases():
    # q = a = z^k > 0: z stays ; all negative with q = 0: z stays
    assert o.update_z_hidden(np.array([2.0]), np.array([2.0]), np.array([2.0]))[0] == 2.0
    assert o.update_z_hidden(np.array([-2.0]), np.array([0.0]), np.array([-2.0]))[0] == -2.0
    # a + z^k > 0 > a + z^k + q is impossible for q >= 0; for q < 0 the negative branch clamps at 0
    z = o.update_z_hidden(np.array([1.0]), np.array([-5.0]), np.array([1.0]))[0]
    assert z == 0.0


# ------------------------------------------------------------------ z-update, last layer

def _bisect(fun, lo, hi):
    for _ in range(200):
        mid = 0.5 * (lo + hi)
        if fun(mid) > 0:
            hi = mid
        else:
            lo = mid
    return 0.5 * (lo + hi)


@pytest.mark.parametrize("nu", [1e-3, 0.05, 2.0])
def test_z_last_two_classes_is_a_logistic_prox(nu):
    """C = 2: with delta = z_0 - z_1 and the sum z_0 + z_1 = a_0 + a_1 kept, the problem is one-dimensional."""
    rng = np.random.default_rng(13)
    for _ in range(20):
        a = rng.standard_normal(2) * 3
        y = int(rng.integers(0, 2))
        z = o.prox_ce_newton(a, y, nu)
        assert abs(np.sum(z - a)) < 1e-9 / nu * 1e-2
        # stationarity in t = z_y - z_other: -sigmoid(-t) + nu (t - t_a)/2 = 0
        t_a = a[y] - a[1 - y]
        t = _bisect(lambda t: -np.exp(-np.logaddexp(0.0, t)) + 0.5 * nu * (t - t_a), t_a - 10, t_a + 2.0 / nu + 10)
        assert abs((z[y] - z[1 - y]) - t) < 1e-8


def test_z_last_stationarity_fista_and_batched_agree():
    rng = np.random.default_rng(14)
    nu = 0.05
    A = rng.standard_normal((6, 12)) * 2
    y = rng.integers(0, 6, 12)
    Zb = o.prox_ce_newton_batched(A, y, nu)
    for j in range(12):
        z = o.prox_ce_newton(A[:, j], int(y[j]), nu)
        e = np.zeros(6)
        e[y[j]] = 1
        assert np.max(np.abs(o.softmax_col(z) - e + nu * (z - A[:, j]))) < 1e-11
        assert np.allclose(Zb[:, j], z, atol=1e-9)
        if j < 4:
            assert np.allclose(o.prox_ce_fista(A[:, j], int(y[j]), nu), z, atol=1e-8)
        # a 1-D scan through the minimiser along a random direction does not find anything lower
        d = rng.standard_normal(6)
        f = lambda zz: o.cross_entropy(zz, int(y[j])) + 0.5 * nu * np.sum((zz - A[:, j]) ** 2)
        assert all(f(z + t * d) >= f(z) - 1e-13 for t in np.linspace(-1, 1, 41))


def test_z_last_unlabelled_nodes_keep_a_and_risk_is_a_masked_sum():
    rng = np.random.default_rng(15)
    a = rng.standard_normal((3, 5))
    y = np.array([0, 1, 2, 1, 0])
    mask = np.array([1, 0, 1, 0, 0], dtype=bool)
    z = o.update_z_last(a, y, mask, 0.1)
    assert np.array_equal(z[:, ~mask], a[:, ~mask])
    assert not np.allclose(z[:, mask], a[:, mask])
    want = sum(o.cross_entropy(a[:, j], int(y[j])) for j in range(5) if mask[j])
    assert abs(o.risk(a, y, mask) - want) < 1e-13
    assert abs(o.cross_entropy(np.array([0.0, 0.0]), 1) - np.log(2)) < 1e-15


# ------------------------------------------------------------------ q- and u-update

def test_q_update_gradient_and_grid():
    rng = np.random.default_rng(16)
    p_next, u, z = rng.standard_normal((3, 50))
    q = o.update_q(p_next, u, z, RHO, NU)
    # d/dq [ <u, p - q> + (rho/2)(p - q)^2 + (nu/2)(q - f(z))^2 ] = 0
    assert np.allclose(-u - RHO * (p_next - q) + NU * (q - o.relu(z)), 0, atol=1e-13)
    grid = np.linspace(-6, 6, 120001)
    for i in range(5):
        vals = u[i] * (p_next[i] - grid) + 0.5 * RHO * (p_next[i] - grid) ** 2 + 0.5 * NU * (grid - max(z[i], 0)) ** 2
        assert abs(grid[int(np.argmin(vals))] - q[i]) <= 1e-4


def test_u_update_written_out():
    u = o.update_u(np.array([1.0]), np.array([3.0]), np.array([2.5]), 0.2)
    assert abs(u[0] - (1.0 + 0.2 * 0.5)) < 1e-15
