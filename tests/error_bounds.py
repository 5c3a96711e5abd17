"""Rounding-error bounds of one device iteration, element by element.

The device holds the state in single precision and runs Algorithm 1 with the linear residual r = W p + b - z carried
along; the oracle runs the same steps in double precision.  Started from the same (single-precision representable)
state, the two differ by the roundings of the device's arithmetic and by nothing else.  The functions below propagate
those roundings through the device's sequence of operations, so that the parity tests can hold every variable to
`1e-4 relative, or the rounding level of its own computation where that is larger` instead of to hand-picked floors,
and can tell where a discrete decision (a quantisation code) is decided by rounding.  Nothing here is the method's
arithmetic: only absolute values, squares, products of those, and the constants below.

Constants
  EPS = 2^-24: unit roundoff of one single-precision operation (round to nearest).
  KAPPA: relative accuracy of a dense product as the kernels deliver it, ||fl(A B) - A B||_F <= KAPPA ||A B||_F.  It is
    not assumed: test_dense_products_keep_single_precision_accuracy_at_any_scale asserts 4e-7 for the tensor-core
    products and 1e-6 for the CUDA-core ones on every operand layout, and those two numbers are used here.
  LAMBDA = 8: an element of a product is a sum of K terms of either sign; its rounding error behaves like a sum of
    independent errors, one per term, so its size is KAPPA times the root-sum-square of the terms (the typical size of
    the sum itself), and LAMBDA such standard deviations are not exceeded by any of the 1e7..1e9 elements compared.
  A worst-case bound (sum of |a_k||b_k| instead of the root-sum-square, K 2^-24 instead of KAPPA) is a factor 30..300
  larger and would let wrong results pass; the statistical form is what keeps the tests sharp.
"""

from __future__ import annotations

import numpy as np

EPS = 2.0 ** -24
LAMBDA = 8.0


def kappa(tensor_cores: bool = True) -> float:
    return 4e-7 if tensor_cores else 1e-6


def rss(a, b):
    """Root-sum-square of the terms of every element of a @ b."""
    return np.sqrt((a * a) @ (b * b))


def _fro(a):
    return float(np.linalg.norm(a))


def iteration_bounds(prev, nxt, prm, tensor_cores=True, tau_dev=None, single=False):
    """Elementwise bounds of |device - oracle| after one iteration started from the state `prev` (already loaded into
    the device), `nxt` = oracle.iterate(prev).  Returns a dict of lists (index l-1 for layer l, the oracle's layout:
    one column per node): 'p', 'W', 'b', 'z', 'q', 'u' and 'x' (the value p - g/tau before the projection of the
    quantised update, in the same units as p).  Discrete decisions (ReLU branch, nearest level) are assumed equal:
    the callers mask the elements where the bounds themselves say that they need not be.
    single=True evaluates the magnitudes in single precision (they are error sizes, not results): twice as fast.
    """
    if single:
        import dataclasses
        f = lambda arrs: [np.asarray(a, dtype=np.float32) for a in arrs]
        prev = dataclasses.replace(prev, p=f(prev.p), W=f(prev.W), b=f(prev.b), z=f(prev.z), q=f(prev.q), u=f(prev.u))
        nxt = dataclasses.replace(nxt, p=f(nxt.p), W=f(nxt.W), b=f(nxt.b), z=f(nxt.z), q=f(nxt.q), u=f(nxt.u))
    L, rho, nu = prev.L, prm.rho, prm.nu
    quant = prm.quant_levels > 0
    A = np.abs
    out = {k: [None] * L for k in ("p", "W", "b", "z", "q", "u", "x", "r")}
    N = prev.p[0].shape[1]
    for l in range(L):
        W, p, b, z = prev.W[l], prev.p[l], prev.b[l], prev.z[l]
        n_out, n_in = W.shape
        g_in = g_out = g_nodes = LAMBDA * kappa(tensor_cores)
        a0 = W @ p + b[:, None]
        r0 = a0 - z
        # r0 = fl(P W^T + b - z): the product, then two additions
        d_r = g_in * rss(W, p) + 2 * EPS * (A(a0) + A(r0))
        p_new = nxt.p[l]
        d_p = np.zeros_like(p)
        if l >= 1:
            q_prev, u_prev = prev.q[l - 1], prev.u[l - 1]
            t = u_prev + rho * (p - q_prev)
            d_t = 2 * EPS * (A(t) + rho * A(p - q_prev))
            g = nu * (W.T @ r0) + t
            d_g = nu * (g_out * rss(W.T, r0) + rss(W.T, d_r)) + d_t + 2 * EPS * A(g)
            Wg = W @ g
            d_Wg = g_in * rss(W, g) + rss(W, d_g)
            tau = nxt.tau[l]
            gg, wgwg = _fro(g), _fro(Wg)
            # tau = rho + nu ||W g||^2 / ||g||^2: both sums of squares inherit twice the relative error of their vector
            d_tau_rel = 0.0
            if gg > 0 and wgwg > 0:
                d_tau_rel = (tau - rho) / tau * (2 * _fro(d_g) / gg + 2 * _fro(d_Wg) / wgwg + 8 * EPS)
            if tau_dev is not None and tau_dev[l]:
                d_tau_rel = max(d_tau_rel, abs(tau_dev[l] - tau) / tau)
            x = p - g / tau
            d_x = d_g / tau + A(g) / tau * (d_tau_rel + 2 * EPS) + EPS * A(x)
            out["x"][l] = d_x
            if quant:
                d = p_new - p
                d_r = d_r + g_in * rss(W, d) + EPS * A(r0 + W @ d)        # r1 = r0 + W d, p+ exact where the codes agree
            else:
                d_p = d_x
                d_r = d_r + d_Wg / tau + A(Wg) / tau * (d_tau_rel + 2 * EPS) + EPS * A(r0 - Wg / tau)
        out["p"][l] = d_p
        r1 = W @ p_new + b[:, None] - z
        # G = nu r1 p+^T over node slices, G p+, theta = nu ||G p+||^2 / ||G||^2
        G = nu * (r1 @ p_new.T)
        d_G = nu * (g_nodes * rss(r1, p_new.T) + rss(d_r, p_new.T) + rss(r1, d_p.T)) + 2 * EPS * A(G)
        Gp = G @ p_new
        d_Gp = g_in * rss(G, p_new) + rss(d_G, p_new) + rss(G, d_p)
        theta = nxt.theta[l]
        if theta > 0:
            d_theta_rel = 2 * _fro(d_G) / max(_fro(G), 1e-300) + 2 * _fro(d_Gp) / max(_fro(Gp), 1e-300) + 8 * EPS
            out["W"][l] = d_G / theta + A(G) / theta * (d_theta_rel + 2 * EPS) + EPS * A(nxt.W[l])
            r2 = r1 - Gp / theta
            d_r = d_r + d_Gp / theta + A(Gp) / theta * (d_theta_rel + 2 * EPS) + EPS * A(r2)
        else:
            out["W"][l] = np.zeros_like(W)
            r2 = r1
        # b+ = b - mean_j r2 (column sums in double precision), shift = that mean in single precision
        mean_r = r2.mean(axis=1)
        # a mean of N errors: their root-mean-square bounds it whatever their signs (Cauchy-Schwarz)
        d_b = np.sqrt((d_r * d_r).mean(axis=1)) + EPS * (A(b) + A(nxt.b[l]) + A(mean_r))
        out["b"][l] = d_b
        a = nxt.W[l] @ p_new + nxt.b[l][:, None]
        d_a = d_r + d_b[:, None] + 2 * EPS * (A(r2) + A(a))
        if l < L - 1:
            q, u = prev.q[l], prev.u[l]
            # both half-line minimisers are averages of (a, q, z) with weight at most 1/2 on a
            d_z = d_a / 2 + 3 * EPS * (A(a) + A(q) + A(z))
            out["z"][l] = d_z
            out["r"][l] = d_a + d_z
        else:
            # the proximal map of a convex risk is non-expansive in a; the Newton iteration stops at a gradient of 1e-10,
            # i.e. within 1e-10 / nu of the minimiser (nu-strong convexity); one rounding of the result
            out["z"][l] = d_a + 1e-10 / nu + EPS * A(nxt.z[l])
            out["r"][l] = d_a + out["z"][l]
    for l in range(L - 1):
        p_next_bound = out["p"][l + 1]
        q_new, u = nxt.q[l], prev.u[l]
        d_q = (rho * p_next_bound + nu * out["z"][l]) / (rho + nu) \
            + 3 * EPS * (rho * A(nxt.p[l + 1]) + A(u) + nu * A(nxt.z[l])) / (rho + nu) + EPS * A(q_new)
        out["q"][l] = d_q
        res = nxt.p[l + 1] - q_new
        out["u"][l] = rho * (p_next_bound + d_q) + EPS * (A(u) + A(nxt.u[l])) + 2 * EPS * rho * (A(nxt.p[l + 1]) + A(q_new) + A(res))
    return out
