"""Helpers of the GPU parity tests: move states between the oracle (fp64, one column per node)
and the C-ABI library (fp32, node-major), and compare them variable by variable."""

from __future__ import annotations

import numpy as np

import oracle.pdadmm_oracle as o
from paper_2105_09837_b200 import binding as B


def oracle_problem(inp, rho=None, nu=None, quant_levels=None, quantize_q=False, neg_levels=0, step=0.0, slope=0.0,
                   risk="ce", activation="relu", table=(257, -4.0, 4.0)):
    """(Params, initial oracle State) for a synth.Inputs bundle.  neg_levels / step: a fixed level set
    {(c - neg_levels) step} as the C ABI's quant_neg_levels / quant_step describe it."""
    w = inp.workload
    lo = float(np.float32(-neg_levels) * np.float32(step))
    prm = o.Params(w.rho if rho is None else rho, w.nu if nu is None else nu,
                   w.quant_levels if quant_levels is None else quant_levels,
                   quantize_q=quantize_q, level_lo=lo, level_step=step, slope=slope, risk=risk, activation=activation,
                   table_size=table[0], table_lo=table[1], table_hi=table[2])
    A = o.renormalized_adjacency(w.n_nodes, inp.edge_src, inp.edge_dst)
    X = o.augment(inp.features.T.astype(np.float64), A, w.n_blocks)
    s = o.init_state(X, [x.astype(np.float64) for x in inp.init_W], inp.labels, inp.train_mask, prm)
    return prm, s, A


def f32(a):
    return np.asarray(a, dtype=np.float32).astype(np.float64)


def round_state(s: o.State) -> o.State:
    """The oracle state with every array rounded to single precision (what the device can hold)."""
    n = s.copy()
    for name in ("p", "W", "b", "z", "q", "u"):
        setattr(n, name, [f32(a) for a in getattr(s, name)])
    return n


def load_state(ctx: B.Context, s: o.State, quantised: bool):
    """Teacher forcing: write an (already fp32-representable) oracle state into the device context."""
    L = s.L
    for l in range(1, L + 1):
        if l >= 2:
            if quantised:
                ctx.set_tensor(B.T_QSCALE, l, np.array([s.scale[l - 1]], dtype=np.float32))
            ctx.set_tensor(B.T_P, l, s.p[l - 1].T)
        ctx.set_tensor(B.T_W, l, s.W[l - 1])
        ctx.set_tensor(B.T_B, l, s.b[l - 1])
        ctx.set_tensor(B.T_Z, l, s.z[l - 1].T)
        if l < L:
            ctx.set_tensor(B.T_Q, l, s.q[l - 1].T)
            ctx.set_tensor(B.T_U, l, s.u[l - 1].T)


def read_state(ctx: B.Context) -> dict:
    L = ctx.n_layers
    out = {k: [] for k in ("p", "W", "b", "z", "q", "u")}
    for l in range(1, L + 1):
        out["p"].append(ctx.get_tensor(B.T_P, l).T.astype(np.float64))
        out["W"].append(ctx.get_tensor(B.T_W, l).astype(np.float64))
        out["b"].append(ctx.get_tensor(B.T_B, l).astype(np.float64))
        out["z"].append(ctx.get_tensor(B.T_Z, l).T.astype(np.float64))
        if l < L:
            out["q"].append(ctx.get_tensor(B.T_Q, l).T.astype(np.float64))
            out["u"].append(ctx.get_tensor(B.T_U, l).T.astype(np.float64))
    return out


def rel_err(got, want, mask=None) -> float:
    """Relative Frobenius error over the unmasked elements (the norm of the reference is taken over the same elements)."""
    if mask is not None:
        got, want = got[~mask], want[~mask]
    den = np.linalg.norm(want)
    num = np.linalg.norm(got - want)
    if den == 0.0:
        return 0.0 if num == 0.0 else np.inf
    return float(num / den)


def z_tie_mask(prev: o.State, nxt: o.State, l: int, tol=1e-5, slope=0.0):
    """Elements of hidden layer l (0-based) whose two ReLU candidates have (nearly) the same objective:
    both are minimisers there, so single and double precision may pick different ones."""
    a = nxt.W[l] @ nxt.p[l] + nxt.b[l][:, None]
    zn = np.minimum((a + slope * prev.q[l] + prev.z[l]) / (2.0 + slope * slope), 0.0)
    zp = np.maximum((a + prev.q[l] + prev.z[l]) / 3.0, 0.0)
    fn = o.z_objective_hidden(zn, a, prev.q[l], prev.z[l], slope)
    fp = o.z_objective_hidden(zp, a, prev.q[l], prev.z[l], slope)
    # equal candidates (both clamp to 0) are not a tie: either choice gives the same z
    return (np.abs(fp - fn) <= tol * (np.abs(fp) + np.abs(fn) + 1e-30)) & (zp != zn)


def band(prm: o.Params) -> float:
    """Half-width, in levels, of the band around a rounding boundary inside which single and double precision may
    round to different neighbours: 2e-4 levels, or, when there are many levels, four single-precision roundings
    (2^-24 each) of a value as large as the top level, m * 2.4e-7 levels (4096 levels: 1e-3)."""
    return max(2e-4, 2.4e-7 * prm.quant_levels)


def boundary_mask(prev: o.State, nxt: o.State, prm: o.Params, l: int, tol=None):
    """Elements of p_l (0-based l >= 1) whose pre-quantisation value lies within `tol` levels of a rounding boundary."""
    tol = band(prm) if tol is None else tol
    g = o.grad_p_phi(prev.p[l], prev.W[l], prev.b[l], prev.z[l], prm.nu, prev.q[l - 1], prev.u[l - 1], prm.rho)
    t = (prev.p[l] - g / nxt.tau[l] - prm.level_lo) / prev.scale[l]
    frac = t - np.floor(t)
    return np.abs(frac - 0.5) <= tol


def q_boundary_mask(prev: o.State, nxt: o.State, prm: o.Params, l: int, tol=None):
    """Elements of q_l (0-based l) whose value before the projection lies within `tol` levels of a rounding boundary."""
    v = o.update_q(nxt.p[l + 1], prev.u[l], nxt.z[l], prm.rho, prm.nu)
    # the value to project carries the single-precision error of z+ (a chain of products and sums, about
    # 1e-6 of the largest value), which with many levels exceeds the band of the storage roundings alone
    if tol is None:
        tol = max(band(prm), 1e-6 * float(np.abs(v).max()) / prev.scale[l + 1])
    t = (v - prm.level_lo) / prev.scale[l + 1]
    frac = t - np.floor(t)
    return np.abs(frac - 0.5) <= tol


def redo_after_p(s: o.State, n: o.State, prm: o.Params) -> o.State:
    """The rest of one iteration of Algorithm 1 (W, b, z, q, u, in that order) for the new p held in `n`, by the
    oracle's own update functions.  Used where the device and the oracle projected some entries of p, each within
    rounding of a boundary between two levels, to different neighbours: the oracle then continues from the device's
    choice, so that everything computed from p is compared on equal terms."""
    rho, nu, L = prm.rho, prm.nu, s.L
    for l in range(L):
        n.W[l], n.theta[l] = o.update_W(n.p[l], s.W[l], s.b[l], s.z[l], nu)
    for l in range(L):
        n.b[l] = o.update_b(n.p[l], n.W[l], s.b[l], s.z[l], nu)
    for l in range(L):
        a = n.W[l] @ n.p[l] + n.b[l][:, None]
        if l < L - 1:
            n.z[l] = o._update_z_hidden_for(prm, a, s.q[l], s.z[l])
        elif prm.risk == "ls":
            n.z[l] = o.update_z_last_least_squares(a, s.y, s.mask, nu)
        else:
            n.z[l] = o.update_z_last(a, s.y, s.mask, nu)
    for l in range(L - 1):
        if prm.quant_levels and prm.quantize_q:
            n.q[l] = o.update_q_quantized(n.p[l + 1], s.u[l], n.z[l], rho, nu, s.scale[l + 1], prm.quant_levels,
                                          prm.level_lo, prm.f)
        else:
            n.q[l] = o.update_q(n.p[l + 1], s.u[l], n.z[l], rho, nu, prm.f)
    for l in range(L - 1):
        n.u[l] = o.update_u(s.u[l], n.p[l + 1], n.q[l], rho)
    return n


def z_table_tie_mask(prev: o.State, nxt: o.State, prm: o.Params, l: int, tol=1e-5):
    """Lookup-table z-update of hidden layer l (0-based): elements where a neighbouring candidate of the table is
    (nearly) as good as the chosen one, so that single and double precision may pick different candidates."""
    a = nxt.W[l] @ nxt.p[l] + nxt.b[l][:, None]
    pts = o.table_points(prm.table_lo, prm.table_hi, prm.table_size)
    step = pts[1] - pts[0]
    f = prm.f
    h = lambda z: (z - a) ** 2 + (prev.q[l] - f(z)) ** 2 + (z - prev.z[l]) ** 2
    best = h(nxt.z[l])
    other = np.minimum(h(np.clip(nxt.z[l] - step, pts[0], pts[-1])), h(np.clip(nxt.z[l] + step, pts[0], pts[-1])))
    edge = (nxt.z[l] <= pts[0]) | (nxt.z[l] >= pts[-1])
    return ((other - best) <= tol * (np.abs(best) + 1e-30)) & ~edge
