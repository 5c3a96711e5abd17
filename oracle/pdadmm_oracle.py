"""fp64 CPU oracle of pdADMM-G and pdADMM-G-Q (test infrastructure, not product code).

Everything here is written in the paper's own orientation and notation:
matrices are ``width x |V|`` (one column per node), ``W_l`` is ``n_l x n_{l-1}``,
``p_l`` is the input of layer l (``p_1 = X``), ``z_l, q_l, u_l`` are ``n_l x |V|``.
Python lists are 0-based, so ``p[l-1]`` holds ``p_l`` and ``q[l-1], u[l-1]`` hold
``q_l, u_l`` (l = 1..L-1).  All arithmetic is float64 numpy; the only library
primitives are dense/sparse matrix products.

Steps follow Algorithm 1 and the appendix "Solutions to Subproblems" in the
paper's order: p (l = 2..L), W, b, z, q, residual, u.  Where the paper leaves a
choice open the reading is stated in the function's docstring.

Parity status: every function below is pinned by the CPU tests (grid search,
closed forms, invariants, hand-worked values); nothing is "parity unpinned".
"""

from __future__ import annotations

import copy
import dataclasses
from typing import List, Optional

import numpy as np
import scipy.sparse as sp


# ----------------------------------------------------------------------------
# Graph pre-processing and feature augmentation
# ----------------------------------------------------------------------------

def renormalized_adjacency(n_nodes: int, edge_src, edge_dst) -> sp.csr_matrix:
    """A~ = (D+I)^{-1/2} (A+I) (D+I)^{-1/2}, D_ii = sum_j A_ij  (Experiments, "Datasets and Settings").

    ``A`` is the symmetric 0/1 adjacency of the undirected simple graph given
    by the edge list (each edge once; self-loops and repeats are ignored).
    """
    src = np.asarray(edge_src, dtype=np.int64)
    dst = np.asarray(edge_dst, dtype=np.int64)
    keep = src != dst
    src, dst = src[keep], dst[keep]
    rows = np.concatenate([src, dst])
    cols = np.concatenate([dst, src])
    A = sp.coo_matrix((np.ones(rows.size), (rows, cols)), shape=(n_nodes, n_nodes)).tocsr()
    A.data[:] = 1.0                      # repeated pairs collapse to a single 1
    deg = np.asarray(A.sum(axis=1)).ravel()
    d_inv_sqrt = 1.0 / np.sqrt(deg + 1.0)
    A_hat = (A + sp.identity(n_nodes, format="csr")).tocsr()
    S = sp.diags(d_inv_sqrt)
    out = (S @ A_hat @ S).tocsr()
    out.sort_indices()
    return out


def augment(H: np.ndarray, A_tilde: sp.csr_matrix, n_blocks: int) -> np.ndarray:
    """X = [X_1; ...; X_K], X_k = H psi_k(A), psi = {I, A~, A~^2, ...}  (Problem Formulation).

    ``H`` is ``d x |V|``; the result is ``(n_blocks d) x |V|``.
    """
    H = np.asarray(H, dtype=np.float64)
    blocks = [H]
    for _ in range(n_blocks - 1):
        # X_{k+1} = X_k A~ ;  (X A~) = (A~^T X^T)^T and the sparse product wants the sparse factor first
        blocks.append(np.asarray((A_tilde.T @ blocks[-1].T).T))
    return np.concatenate(blocks, axis=0)


# ----------------------------------------------------------------------------
# State
# ----------------------------------------------------------------------------

@dataclasses.dataclass
class Params:
    rho: float
    nu: float
    quant_levels: int = 0                 # 0: pdADMM-G ; m >= 2: pdADMM-G-Q with m levels per layer
    max_trials: int = 30                  # cap of the tau search in the quantised p-update
    accept_slack: float = 1e-6
    quantize_q: bool = False              # the variant that also keeps q_l in Delta (end of Sec. "Quantization Extension")
    level_lo: float = 0.0                 # smallest level delta_0
    level_step: float = 0.0               # > 0: the same fixed step for every layer; 0: step from max(p) at the start
    slope: float = 0.0                    # 0: f_l = ReLU; in (0, 1): leaky ReLU with that slope for x <= 0
    risk: str = "ce"                      # R: "ce" cross-entropy (the paper's experiments), "ls" least squares
    activation: str = "relu"              # f_l: "relu" (with `slope`: leaky), or the smooth "tanh" / "sigmoid", whose
    table_lo: float = -4.0                #   z-update searches a lookup table of table_size equally spaced candidates
    table_hi: float = 4.0                 #   on [table_lo, table_hi] (remark after Eq. "update z")
    table_size: int = 257

    @property
    def f(self):
        """What the functions below take as their `slope` argument: the leaky slope, or the smooth activation itself."""
        if self.activation == "relu":
            return self.slope
        return {"tanh": np.tanh, "sigmoid": lambda x: 1.0 / (1.0 + np.exp(-x))}[self.activation]


@dataclasses.dataclass
class State:
    p: List[np.ndarray]                   # p_1..p_L ; p_1 = X is never updated
    W: List[np.ndarray]
    b: List[np.ndarray]                   # each n_l (a vector, broadcast over nodes)
    z: List[np.ndarray]
    q: List[np.ndarray]                   # q_1..q_{L-1}
    u: List[np.ndarray]                   # u_1..u_{L-1}
    y: np.ndarray                         # labels, |V| ints
    mask: np.ndarray                      # |V| bools: node contributes to R
    scale: List[float]                    # quantisation step s_l of p_l (index l-1; entry 0 unused)
    tau: List[float] = dataclasses.field(default_factory=list)     # last tau_l (index l-1; entry 0 unused)
    theta: List[float] = dataclasses.field(default_factory=list)   # last theta_l
    trials: List[int] = dataclasses.field(default_factory=list)    # trials the quantised p-update took

    @property
    def L(self) -> int:
        return len(self.W)

    def copy(self) -> "State":
        return copy.deepcopy(self)


def relu(x, slope=0.0):
    """f_l: ReLU, or, with 0 < slope < 1, the leaky ReLU f(x) = x (x > 0), slope x (x <= 0), which the paper
    names beside ReLU as an activation its assumptions cover (Sec. "Convergence Analysis").  A callable in place of
    the slope is a smooth activation (tanh, sigmoid: ``Params.f``) and is simply applied."""
    if callable(slope):
        return slope(x)
    return np.maximum(x, 0.0) if slope == 0.0 else np.where(x > 0, x, slope * x)


# ----------------------------------------------------------------------------
# phi, its gradients, and the quadratic models U_l, V_l
# ----------------------------------------------------------------------------

def phi(p, W, b, z, nu, q_prev=None, u_prev=None, rho=0.0) -> float:
    """phi(p_l,W_l,b_l,z_l[,q_{l-1},u_{l-1}])  (definition below the augmented Lagrangian).

    (nu/2)||z - W p - b||^2  [+ <u_{l-1}, p - q_{l-1}> + (rho/2)||p - q_{l-1}||^2 for l > 1].
    """
    lin = z - W @ p - b[:, None]
    val = 0.5 * nu * np.sum(lin * lin)
    if q_prev is not None:
        diff = p - q_prev
        val += np.sum(u_prev * diff) + 0.5 * rho * np.sum(diff * diff)
    return float(val)


def grad_p_phi(p, W, b, z, nu, q_prev, u_prev, rho):
    """nabla_p phi = nu W^T (W p + b - z) + u_{l-1} + rho (p - q_{l-1})."""
    return nu * (W.T @ (W @ p + b[:, None] - z)) + u_prev + rho * (p - q_prev)


def grad_W_phi(p, W, b, z, nu):
    """nabla_W phi = nu (W p + b - z) p^T."""
    return nu * ((W @ p + b[:, None] - z) @ p.T)


def grad_b_phi(p, W, b, z, nu):
    """nabla_b phi = nu sum_j (W p + b - z)_{:,j}  (b is broadcast over the |V| columns)."""
    return nu * np.sum(W @ p + b[:, None] - z, axis=1)


def U_model(p_new, p_old, W, b, z, nu, q_prev, u_prev, rho, tau) -> float:
    """U_l(p; tau) = phi(p^k) + <nabla_p phi(p^k), p - p^k> + (tau/2)||p - p^k||^2  (Eq. update p)."""
    g = grad_p_phi(p_old, W, b, z, nu, q_prev, u_prev, rho)
    d = p_new - p_old
    return phi(p_old, W, b, z, nu, q_prev, u_prev, rho) + float(np.sum(g * d)) + 0.5 * tau * float(np.sum(d * d))


def V_model(W_new, W_old, p, b, z, nu, theta) -> float:
    """V_l(W; theta) = phi(W^k) + <nabla_W phi(W^k), W - W^k> + (theta/2)||W - W^k||^2  (Eq. update W).

    The q/u terms of phi do not depend on W and cancel on both sides, so they are left out.
    """
    G = grad_W_phi(p, W_old, b, z, nu)
    D = W_new - W_old
    return phi(p, W_old, b, z, nu) + float(np.sum(G * D)) + 0.5 * theta * float(np.sum(D * D))


# ----------------------------------------------------------------------------
# p-update (Eq. update p) and its step parameter tau
# ----------------------------------------------------------------------------

def tau_smallest_admissible(g, W, nu, rho) -> float:
    """Smallest tau with phi(p - g/tau) <= U_l(p - g/tau; tau).

    The paper only states the condition.  phi is quadratic in p with Hessian
    nu W^T W + rho I, so for a step d the condition reads
    nu||W d||^2 + rho||d||^2 <= tau||d||^2; with d parallel to g the trial
    value of tau drops out and the smallest admissible value is
    rho + nu||W g||^2 / ||g||^2.  If g = 0 any tau works; rho is returned.
    """
    gg = float(np.sum(g * g))
    if gg == 0.0:
        return float(rho)
    Wg = W @ g
    return float(rho + nu * float(np.sum(Wg * Wg)) / gg)


def tau_by_backtracking(p, W, b, z, nu, q_prev, u_prev, rho, tau0=None, factor=2.0, max_trials=200):
    """Generic search by definition: grow tau geometrically until phi(p+) <= U_l(p+; tau).

    Used by the tests to bracket ``tau_smallest_admissible``; not used by ``iterate``.
    """
    g = grad_p_phi(p, W, b, z, nu, q_prev, u_prev, rho)
    tau = float(rho if tau0 is None else tau0)
    for _ in range(max_trials):
        p_new = p - g / tau
        lhs = phi(p_new, W, b, z, nu, q_prev, u_prev, rho)
        rhs = U_model(p_new, p, W, b, z, nu, q_prev, u_prev, rho, tau)
        if lhs <= rhs:
            return tau
        tau *= factor
    raise RuntimeError("tau search did not terminate")


def update_p(p, W, b, z, nu, q_prev, u_prev, rho):
    """p^{k+1} = p^k - nabla_p phi / tau^{k+1}, tau the smallest admissible value.  Returns (p+, tau)."""
    g = grad_p_phi(p, W, b, z, nu, q_prev, u_prev, rho)
    tau = tau_smallest_admissible(g, W, nu, rho)
    return p - g / tau, tau


# ----------------------------------------------------------------------------
# Quantisation set and the quantised p-update (Eq. update p quantized)
# ----------------------------------------------------------------------------

def level_set(scale: float, m: int, lo: float = 0.0) -> np.ndarray:
    """Delta = {delta_0..delta_{m-1}}, delta_c = fl32(lo + fl32(c * s)): m uniform levels starting at lo.

    The levels are single-precision numbers (one rounded multiply, one rounded
    add), so that a quantised p is exactly representable in the fp32 state of
    the CUDA path.  lo = -1, s = 1, m = 22 is the set {-1, 0, ..., 20} of the
    paper's experiments (Sec. "Datasets and Settings").
    """
    return (np.float32(lo) + np.arange(m, dtype=np.float32) * np.float32(scale)).astype(np.float64)


def nearest_level(x, scale: float, m: int, lo: float = 0.0):
    """Nearest element of Delta, element by element, by definition: argmin_{delta in Delta} |delta - x| in double
    precision, Delta = level_set(scale, m, lo).

    ||delta - x||^2 is separable, so the argmin of Eq. (update p quantized) is taken per element.  The levels are
    (nearly) uniform, so the rounding floor((x - lo)/s + 1/2) gives a candidate; because the levels themselves are
    rounded single-precision numbers the candidate and its two neighbours are then compared by their actual
    distances.  An exact tie between two levels goes to the upper one (the paper does not say; both are minimisers).
    Returns (codes, p in Delta); codes are uint8 for up to 256 levels and uint16 above (the 8- and 16-bit cases of
    Sec. "Communication Overheads").
    """
    x = np.asarray(x, dtype=np.float64)
    lev = level_set(scale, m, lo)
    c = np.clip(np.floor((x - float(np.float32(lo))) / float(np.float32(scale)) + 0.5), 0, m - 1).astype(np.int64)
    best, best_d = c, np.abs(lev[c] - x)
    for cand in (np.clip(c - 1, 0, m - 1), np.clip(c + 1, 0, m - 1)):
        d = np.abs(lev[cand] - x)
        take = (d < best_d) | ((d == best_d) & (cand > best))
        best, best_d = np.where(take, cand, best), np.where(take, d, best_d)
    return best.astype(np.uint8 if m <= 256 else np.uint16), lev[best]


def quantize(x, scale: float, m: int, lo: float = 0.0):
    """The same projection as a single-precision program computes it: code = clamp(floor((x - lo)/s + 1/2), 0, m-1)
    with x, the division, the sum and the floor all in float32 (ties at half-levels go up), value = fl32(lo + fl32(c s)).

    Not used by ``iterate``: it serves the comparisons in which both sides are handed identical float32 inputs and
    the result has to agree bit for bit.  Returns (codes, p in Delta) like ``nearest_level``.
    """
    x32 = np.asarray(x, dtype=np.float32)
    t = (x32 - np.float32(lo)) / np.float32(scale)
    c = np.floor(t + np.float32(0.5))
    c = np.clip(c, np.float32(0.0), np.float32(m - 1))
    codes = c.astype(np.uint8 if m <= 256 else np.uint16)
    vals = (np.float32(lo) + c * np.float32(scale)).astype(np.float64)
    return codes, vals


def quantization_scale(x, m: int) -> float:
    """s = max(x) / (m - 1) as a single-precision number; s = 1 if max(x) <= 0."""
    mx = np.float32(np.max(x)) if np.size(x) else np.float32(0.0)
    if not mx > 0:
        return 1.0
    return float(np.float32(mx) / np.float32(m - 1))


def update_p_quantized(p, W, b, z, nu, q_prev, u_prev, rho, scale, m, max_trials=30, slack=1e-6, lo=0.0):
    """p^{k+1} = argmin_{delta in Delta} ||delta - (p^k - nabla_p phi / tau)||.

    tau starts at the smallest value admissible for the unprojected step and
    is doubled until phi(p+) <= U_l(p+; tau) (up to a relative slack on the
    quadratic term, which only matters at exact ties).  Returns
    (p+, codes, tau, trials); trials = -1 if the cap was hit (last p+ is kept).
    """
    g = grad_p_phi(p, W, b, z, nu, q_prev, u_prev, rho)
    tau = tau_smallest_admissible(g, W, nu, rho)
    phi_old = phi(p, W, b, z, nu, q_prev, u_prev, rho)
    for trial in range(1, max_trials + 1):
        codes, p_new = nearest_level(p - g / tau, scale, m, lo)
        d = p_new - p
        dd = float(np.sum(d * d))
        lhs = phi(p_new, W, b, z, nu, q_prev, u_prev, rho)
        rhs = phi_old + float(np.sum(g * d)) + 0.5 * tau * dd
        if lhs <= rhs + 0.5 * slack * tau * dd:
            return p_new, codes, tau, trial
        tau *= 2.0
    return p_new, codes, tau, -1


# ----------------------------------------------------------------------------
# W-update (Eq. update W), b-update (Eq. update b)
# ----------------------------------------------------------------------------

def theta_smallest_admissible(G, p, nu) -> float:
    """Smallest theta with phi(W - G/theta) <= V_l(W - G/theta; theta): nu||G p||^2 / ||G||^2.

    phi is quadratic in W: phi(W + D) = phi(W) + <G, D> + (nu/2)||D p||^2.  G = 0 returns 0
    (the caller leaves W unchanged).
    """
    GG = float(np.sum(G * G))
    if GG == 0.0:
        return 0.0
    Gp = G @ p
    return float(nu * float(np.sum(Gp * Gp)) / GG)


def theta_by_backtracking(p, W, b, z, nu, theta0, factor=2.0, max_trials=400):
    """Generic search by definition on V_l (tests only)."""
    G = grad_W_phi(p, W, b, z, nu)
    theta = float(theta0)
    for _ in range(max_trials):
        W_new = W - G / theta
        if phi(p, W_new, b, z, nu) <= V_model(W_new, W, p, b, z, nu, theta):
            return theta
        theta *= factor
    raise RuntimeError("theta search did not terminate")


def update_W(p, W, b, z, nu):
    """W^{k+1} = W^k - nabla_W phi(p^{k+1}, W^k, b^k, z^k) / theta^{k+1}.  Returns (W+, theta)."""
    G = grad_W_phi(p, W, b, z, nu)
    theta = theta_smallest_admissible(G, p, nu)
    if theta == 0.0:
        return W.copy(), 0.0
    return W - G / theta, theta


def update_b(p, W, b, z, nu):
    """b^{k+1} = b^k - nabla_b phi / (nu |V|).

    The paper divides by nu, stating that nabla_b phi is nu-Lipschitz.  With b
    broadcast over |V| columns the gradient is nu sum_j(...) and its Lipschitz
    constant is nu|V|; dividing by that constant gives the exact minimiser
    mean_j (z - W p)_{:,j}, and the descent inequality of Lemma (optimality 1)
    still holds.  ``update_b_literal`` keeps the printed constant for the test
    that shows it diverges.
    """
    n_nodes = p.shape[1]
    return b - grad_b_phi(p, W, b, z, nu) / (nu * n_nodes)


def update_b_literal(p, W, b, z, nu):
    """The step exactly as printed (division by nu); tests only."""
    return b - grad_b_phi(p, W, b, z, nu) / nu


# ----------------------------------------------------------------------------
# z-update (Eq. update z, Eq. update zl)
# ----------------------------------------------------------------------------

def z_objective_hidden(c, a, q, z_old, slope: float = 0.0):
    """(c - a)^2 + (q - relu(c))^2 + (c - z^k)^2: Eq. (update z) per element, without the common nu/2."""
    return (c - a) ** 2 + (q - relu(c, slope)) ** 2 + (c - z_old) ** 2


def update_z_hidden(a, q, z_old, slope: float = 0.0):
    """ReLU closed form of Eq. (update z), a = W^{k+1} p^{k+1} + b^{k+1}.

    The printed case distinction refers to the sign of the unknown; it is
    resolved by minimising on each half-line and keeping the better of the two:
    z- = min((a + z^k)/2, 0) on z <= 0, z+ = max((a + q^k + z^k)/3, 0) on z >= 0.
    An exact tie keeps z-.  Leaky ReLU with slope s: on z <= 0 the objective is
    (z-a)^2 + (q - s z)^2 + (z - z^k)^2, stationary at (a + s q + z^k)/(2 + s^2), so
    z- = min((a + s q^k + z^k)/(2 + s^2), 0); z+ is unchanged.
    """
    z_neg = np.minimum((a + slope * q + z_old) / (2.0 + slope * slope), 0.0)
    z_pos = np.maximum((a + q + z_old) / 3.0, 0.0)
    f_neg = z_objective_hidden(z_neg, a, q, z_old, slope)
    f_pos = z_objective_hidden(z_pos, a, q, z_old, slope)
    return np.where(f_pos < f_neg, z_pos, z_neg)


def table_points(lo: float, hi: float, size: int) -> np.ndarray:
    """The candidates of the lookup table: z_i = fl32(lo + fl32(i h)), h = fl32((hi - lo) / (size - 1)), i = 0..size-1
    (single-precision numbers, so that a z taken from the table is exactly representable in the fp32 state)."""
    h = np.float32((np.float32(hi) - np.float32(lo)) / np.float32(size - 1))
    return (np.float32(lo) + np.arange(size, dtype=np.float32) * h).astype(np.float64)


def update_z_hidden_table(a, q, z_old, f, points):
    """Eq. (update z) for a smooth activation f (tanh, sigmoid), for which the paper recommends a lookup table (remark
    after Eq. "update z") instead of a closed form: the minimiser of (z - a)^2 + (q - f(z))^2 + (z - z^k)^2 over the
    table's candidate values, element by element; the first candidate wins a tie.  The result is the best point of the
    table, within half a table step of a minimiser of the continuous problem in objective value (second order)."""
    best = np.full(np.shape(a), np.inf)
    arg = np.zeros(np.shape(a))
    for zi in points:
        h = (zi - a) ** 2 + (q - f(zi)) ** 2 + (zi - z_old) ** 2
        take = h < best
        best = np.where(take, h, best)
        arg = np.where(take, zi, arg)
    return arg


def cross_entropy(z_col, y: int) -> float:
    """CE(z; y) = -z_y + log sum_c exp(z_c) for one node."""
    m = np.max(z_col)
    return float(-z_col[y] + m + np.log(np.sum(np.exp(z_col - m))))


def risk(zL, y, mask) -> float:
    """R(z_L; y) = sum over labelled nodes of the cross-entropy (an unnormalised sum,
    like the unnormalised squared norms it is added to)."""
    m = np.max(zL, axis=0)
    lse = m + np.log(np.sum(np.exp(zL - m[None, :]), axis=0))
    ce = lse - zL[y, np.arange(zL.shape[1])]
    return float(np.sum(ce[np.asarray(mask, dtype=bool)]))


def risk_least_squares(zL, y, mask) -> float:
    """R(z_L; y) = (1/2) sum over labelled nodes of ||z_L[:, j] - e_{y_j}||^2: another risk that Problem 1 admits
    (Sec. "Problem Formulation" only asks R to be convex and continuous)."""
    E = np.zeros_like(zL)
    E[np.asarray(y), np.arange(zL.shape[1])] = 1.0
    d = (zL - E)[:, np.asarray(mask, dtype=bool)]
    return float(0.5 * np.sum(d * d))


def update_z_last_least_squares(a, y, mask, nu):
    """Eq. (update zl) with the least-squares risk: argmin_z (1/2)||z - e_y||^2 + (nu/2)||z - a||^2 per labelled
    node, i.e. z = (e_y + nu a) / (1 + nu) (the stationary point of a strictly convex quadratic); unlabelled nodes
    take z = a."""
    z = np.array(a, dtype=np.float64)
    lab = np.flatnonzero(np.asarray(mask, dtype=bool))
    if lab.size:
        E = np.zeros((a.shape[0], lab.size))
        E[np.asarray(y)[lab], np.arange(lab.size)] = 1.0
        z[:, lab] = (E + nu * a[:, lab]) / (1.0 + nu)
    return z


def softmax_col(z_col):
    e = np.exp(z_col - np.max(z_col))
    return e / np.sum(e)


def prox_ce_newton(a_col, y: int, nu: float, tol=1e-12, max_iter=200):
    """argmin_z CE(z; y) + (nu/2)||z - a||^2 for one node, damped Newton.

    The objective is nu-strongly convex, so the minimiser is unique and is the
    solution of softmax(z) - e_y + nu (z - a) = 0.  The Hessian is
    diag(s) + nu I - s s^T, inverted with the rank-one update formula.
    """
    z = np.array(a_col, dtype=np.float64)
    C = z.size
    e_y = np.zeros(C)
    e_y[y] = 1.0

    def f(zz):
        return cross_entropy(zz, y) + 0.5 * nu * float(np.sum((zz - a_col) ** 2))

    fz = f(z)
    for _ in range(max_iter):
        s = softmax_col(z)
        grad = s - e_y + nu * (z - a_col)
        if np.max(np.abs(grad)) <= tol:
            break
        m_inv = 1.0 / (s + nu)
        mg = m_inv * grad
        ms = m_inv * s
        step = -(mg + ms * (np.dot(s, mg) / (1.0 - np.dot(s, ms))))
        t = 1.0
        slope = float(np.dot(grad, step))
        # once the predicted decrease is below what f can resolve in double precision the
        # iteration is in Newton's quadratic regime: full steps, no sufficient-decrease test
        resolvable = -slope > 1e-9 * (1.0 + abs(fz))
        while True:
            z_try = z + t * step
            f_try = f(z_try)
            if not resolvable or f_try <= fz + 1e-4 * t * slope or t < 1e-12:
                break
            t *= 0.5
        z, fz = z_try, f_try
    return z


def prox_ce_fista(a_col, y: int, nu: float, n_iter=20000, tol=1e-13):
    """The same minimiser by FISTA (the solver the paper names for Eq. update zl).

    Smooth part CE (gradient 1-Lipschitz, step 1), proximable part
    (nu/2)||z - a||^2 with prox(v) = (v + nu a) / (1 + nu).  Cross-check only.
    """
    C = a_col.size
    e_y = np.zeros(C)
    e_y[y] = 1.0
    x = np.array(a_col, dtype=np.float64)
    v = x.copy()
    t = 1.0
    for _ in range(n_iter):
        x_new = ((v - (softmax_col(v) - e_y)) + nu * a_col) / (1.0 + nu)
        t_new = 0.5 * (1.0 + np.sqrt(1.0 + 4.0 * t * t))
        v = x_new + ((t - 1.0) / t_new) * (x_new - x)
        done = np.max(np.abs(x_new - x)) <= tol
        x, t = x_new, t_new
        if done:
            break
    return x


def prox_ce_newton_batched(A, y, nu: float, tol=1e-12, max_iter=200):
    """``prox_ce_newton`` for many nodes at once (columns of ``A``), same steps per column.

    Each column runs its own damped Newton iteration with its own step length;
    a column stops moving once its gradient is below ``tol``.
    """
    A = np.asarray(A, dtype=np.float64)
    C, n = A.shape
    cols = np.arange(n)
    E = np.zeros((C, n))
    E[np.asarray(y, dtype=np.int64), cols] = 1.0

    def f(Z):
        m = np.max(Z, axis=0)
        lse = m + np.log(np.sum(np.exp(Z - m[None, :]), axis=0))
        return lse - np.sum(E * Z, axis=0) + 0.5 * nu * np.sum((Z - A) ** 2, axis=0)

    Z = A.copy()
    fz = f(Z)
    for _ in range(max_iter):
        Ex = np.exp(Z - np.max(Z, axis=0)[None, :])
        S = Ex / np.sum(Ex, axis=0)[None, :]
        grad = S - E + nu * (Z - A)
        active = np.max(np.abs(grad), axis=0) > tol
        if not active.any():
            break
        m_inv = 1.0 / (S + nu)
        mg = m_inv * grad
        ms = m_inv * S
        step = -(mg + ms * (np.sum(S * mg, axis=0) / (1.0 - np.sum(S * ms, axis=0)))[None, :])
        step[:, ~active] = 0.0
        slope = np.sum(grad * step, axis=0)
        t = np.ones(n)
        resolvable = -slope > 1e-9 * (1.0 + np.abs(fz))
        searching = active.copy()
        Z_try, f_try = Z.copy(), fz.copy()
        while searching.any():
            Zc = Z[:, searching] + t[searching][None, :] * step[:, searching]
            fc = f_cols(Zc, A[:, searching], E[:, searching], nu)
            ok = (~resolvable[searching]) | (fc <= fz[searching] + 1e-4 * t[searching] * slope[searching]) \
                | (t[searching] < 1e-12)
            idx = np.flatnonzero(searching)
            Z_try[:, idx[ok]] = Zc[:, ok]
            f_try[idx[ok]] = fc[ok]
            t[idx[~ok]] *= 0.5
            searching[idx[ok]] = False
        Z, fz = Z_try, f_try
    return Z


def f_cols(Z, A, E, nu):
    """CE(z; y) + (nu/2)||z - a||^2 for each column."""
    m = np.max(Z, axis=0)
    lse = m + np.log(np.sum(np.exp(Z - m[None, :]), axis=0))
    return lse - np.sum(E * Z, axis=0) + 0.5 * nu * np.sum((Z - A) ** 2, axis=0)


def update_z_last(a, y, mask, nu):
    """Eq. (update zl): labelled nodes take the proximal point of the cross-entropy,
    unlabelled nodes (no risk term) take z = a.  No proximal ||z - z^k||^2 term for l = L."""
    z = np.array(a, dtype=np.float64)
    lab = np.flatnonzero(np.asarray(mask, dtype=bool))
    if lab.size:
        z[:, lab] = prox_ce_newton_batched(a[:, lab], np.asarray(y)[lab], nu)
    return z


# ----------------------------------------------------------------------------
# q-update (Eq. update q), dual update (Eq. update u)
# ----------------------------------------------------------------------------

def update_q(p_next, u, z, rho, nu, slope=0.0):
    """q_l^{k+1} = (rho p_{l+1}^{k+1} + u_l^k + nu f_l(z_l^{k+1})) / (rho + nu)."""
    return (rho * p_next + u + nu * relu(z, slope)) / (rho + nu)


def update_q_quantized(p_next, u, z, rho, nu, scale, m, lo=0.0, slope=0.0):
    """The variant with q_l in Delta as well: q_l^{k+1} = argmin_{delta in Delta}
    ||delta - (rho p_{l+1}^{k+1} + u_l^k + nu f_l(z_l^{k+1})) / (rho + nu)||, element by element
    (Sec. "Quantization Extension", last paragraph).  Delta is the level set of p_{l+1}, which q_l has to equal."""
    return nearest_level(update_q(p_next, u, z, rho, nu, slope), scale, m, lo)[1]


def update_u(u, p_next, q, rho):
    """u_l^{k+1} = u_l^k + rho (p_{l+1}^{k+1} - q_l^{k+1})."""
    return u + rho * (p_next - q)


# ----------------------------------------------------------------------------
# Initial state, one iteration (Algorithm 1), objective and residuals
# ----------------------------------------------------------------------------

def init_state(X, W0, y, mask, prm: Params) -> State:
    """Feasible start (the paper only says "k = 0"; its theorems allow any start).

    b = 0 and a forward pass: z_l = W_l p_l, q_l = relu(z_l), p_{l+1} = q_l, u = 0.
    pdADMM-G-Q: the pass is sequential in l; the step s_{l+1} of p_{l+1} is
    max(q_l) / (m - 1) (or the fixed prm.level_step) and p_{l+1} = Proj_Delta(q_l), so the
    residual starts non-zero.  In the variant that keeps q in Delta too, q_l = p_{l+1} =
    Proj_Delta(relu(z_l)): a feasible start inside Delta.
    """
    L = len(W0)
    p = [np.asarray(X, dtype=np.float64)]
    W = [np.asarray(w, dtype=np.float64).copy() for w in W0]
    b = [np.zeros(w.shape[0]) for w in W]
    z, q, u = [], [], []
    scale = [1.0] * L
    for l in range(L):
        z.append(W[l] @ p[l])
        if l < L - 1:
            q.append(relu(z[l], prm.f))
            u.append(np.zeros_like(q[l]))
            if prm.quant_levels:
                scale[l + 1] = (float(np.float32(prm.level_step)) if prm.level_step > 0
                                else quantization_scale(q[l], prm.quant_levels))
                p.append(nearest_level(q[l], scale[l + 1], prm.quant_levels, prm.level_lo)[1])
                if prm.quantize_q:
                    q[l] = p[l + 1].copy()
            else:
                p.append(q[l].copy())
    return State(p, W, b, z, q, u, np.asarray(y), np.asarray(mask, dtype=bool), scale,
                 [0.0] * L, [0.0] * L, [0] * L)


def _update_z_hidden_for(prm: Params, a, q, z_old):
    """The z-update of a hidden layer for the activation in `prm`: closed form for (leaky) ReLU, table search else."""
    if prm.activation == "relu":
        return update_z_hidden(a, q, z_old, prm.slope)
    return update_z_hidden_table(a, q, z_old, prm.f, table_points(prm.table_lo, prm.table_hi, prm.table_size))


def iterate(s: State, prm: Params) -> State:
    """One pass of Algorithm 1: p (l=2..L), W, b, z (l=1..L), q, residual, u (l=1..L-1).

    Each family is finished for all layers before the next one starts.
    """
    rho, nu, L = prm.rho, prm.nu, s.L
    n = s.copy()
    # p_l^{k+1}, l = 2..L, from (W^k, b^k, z^k, q^k, u^k)
    for l in range(1, L):
        if prm.quant_levels:
            n.p[l], _, n.tau[l], n.trials[l] = update_p_quantized(
                s.p[l], s.W[l], s.b[l], s.z[l], nu, s.q[l - 1], s.u[l - 1], rho,
                s.scale[l], prm.quant_levels, prm.max_trials, prm.accept_slack, prm.level_lo)
        else:
            n.p[l], n.tau[l] = update_p(s.p[l], s.W[l], s.b[l], s.z[l], nu, s.q[l - 1], s.u[l - 1], rho)
    # W_l^{k+1} from (p^{k+1}, b^k, z^k)
    for l in range(L):
        n.W[l], n.theta[l] = update_W(n.p[l], s.W[l], s.b[l], s.z[l], nu)
    # b_l^{k+1} from (p^{k+1}, W^{k+1}, z^k)
    for l in range(L):
        n.b[l] = update_b(n.p[l], n.W[l], s.b[l], s.z[l], nu)
    # z_l^{k+1} from (p^{k+1}, W^{k+1}, b^{k+1}, q^k)
    for l in range(L):
        a = n.W[l] @ n.p[l] + n.b[l][:, None]
        if l < L - 1:
            n.z[l] = _update_z_hidden_for(prm, a, s.q[l], s.z[l])
        elif prm.risk == "ls":
            n.z[l] = update_z_last_least_squares(a, s.y, s.mask, nu)
        else:
            n.z[l] = update_z_last(a, s.y, s.mask, nu)
    # q_l^{k+1}, then u_l^{k+1}
    for l in range(L - 1):
        if prm.quant_levels and prm.quantize_q:
            n.q[l] = update_q_quantized(n.p[l + 1], s.u[l], n.z[l], rho, nu, s.scale[l + 1], prm.quant_levels,
                                        prm.level_lo, prm.f)
        else:
            n.q[l] = update_q(n.p[l + 1], s.u[l], n.z[l], rho, nu, prm.f)
    for l in range(L - 1):
        n.u[l] = update_u(s.u[l], n.p[l + 1], n.q[l], rho)
    return n


def residuals_sq(s: State) -> np.ndarray:
    """||r_l||^2 = ||p_{l+1} - q_l||^2, l = 1..L-1 (the residual line of Algorithm 1)."""
    return np.array([float(np.sum((s.p[l + 1] - s.q[l]) ** 2)) for l in range(s.L - 1)])


def objective(s: State, prm: Params) -> np.ndarray:
    """Components of the augmented Lagrangian L_rho and their sum:
    [R, (nu/2) sum||z - W p - b||^2, (nu/2) sum||q - f(z)||^2, sum<u, p+ - q>, (rho/2) sum||p+ - q||^2, L_rho]."""
    rho, nu, L = prm.rho, prm.nu, s.L
    R = risk_least_squares(s.z[L - 1], s.y, s.mask) if prm.risk == "ls" else risk(s.z[L - 1], s.y, s.mask)
    lin = sum(float(np.sum((s.z[l] - s.W[l] @ s.p[l] - s.b[l][:, None]) ** 2)) for l in range(L))
    act = sum(float(np.sum((s.q[l] - relu(s.z[l], prm.f)) ** 2)) for l in range(L - 1))
    dual = sum(float(np.sum(s.u[l] * (s.p[l + 1] - s.q[l]))) for l in range(L - 1))
    pen = float(np.sum(residuals_sq(s)))
    comps = [R, 0.5 * nu * lin, 0.5 * nu * act, dual, 0.5 * rho * pen]
    return np.array(comps + [sum(comps)])


def lagrangian(s: State, prm: Params) -> float:
    return float(objective(s, prm)[5])


# ----------------------------------------------------------------------------
# Greedy layer-wise training: growing a trained shallow model
# ----------------------------------------------------------------------------

def start_layers_from(s: State, prm: Params, first: int) -> State:
    """The start of Algorithm 1 for layers first..L (1-based) from the current p_first: b_l = 0, z_l = W_l p_l,
    q_l = f_l(z_l), p_{l+1} = q_l (pdADMM-G-Q: the nearest level, with the spacing taken from max(q_l) like at the very
    start), u_l = 0.  Layers below `first` are left as they are."""
    n = s.copy()
    L = n.L
    for l in range(first - 1, L):
        n.b[l] = np.zeros_like(n.b[l])
        n.z[l] = n.W[l] @ n.p[l]
        if l < L - 1:
            n.q[l] = relu(n.z[l], prm.f)
            n.u[l] = np.zeros_like(n.q[l])
            if prm.quant_levels:
                n.scale[l + 1] = (float(np.float32(prm.level_step)) if prm.level_step > 0
                                  else quantization_scale(n.q[l], prm.quant_levels))
                n.p[l + 1] = nearest_level(n.q[l], n.scale[l + 1], prm.quant_levels, prm.level_lo)[1]
                if prm.quantize_q:
                    n.q[l] = n.p[l + 1].copy()
            else:
                n.p[l + 1] = n.q[l].copy()
    return n


def grow(s: State, prm: Params, W_new: List[np.ndarray]) -> State:
    """Greedy layer-wise training (end of Sec. "The pdADMM-G Algorithm"; Sec. "Performance": 2, then 5, then 10
    layers): a trained model with L layers becomes one with L - 1 + len(W_new) layers.

    The paper says that layers are added and trained, not how they start.  Reading: the hidden layers 1..L-1 keep
    everything they have (p_l, W_l, b_l, z_l, q_l, u_l, the level spacing of p_l); the old output layer, whose width
    is the number of classes, cannot serve as a hidden layer and is dropped; the layers L.., the last of which is the
    new output layer, take the weights `W_new` (drawn by the caller like the initial ones) and start from the forward
    pass of the model trained so far, i.e. the start of Algorithm 1 from the kept p_L (``start_layers_from``): the
    constraints p_{l+1} = q_l hold for them and their duals are zero.
    """
    L_old = s.L
    keep = L_old - 1
    L_new = keep + len(W_new)
    W = [w.copy() for w in s.W[:keep]] + [np.asarray(w, dtype=np.float64).copy() for w in W_new]
    n_nodes = s.p[0].shape[1]
    b = [x.copy() for x in s.b[:keep]] + [np.zeros(w.shape[0]) for w in W_new]
    p = [x.copy() for x in s.p[:keep + 1]] + [None] * (L_new - keep - 1)
    z = [x.copy() for x in s.z[:keep]] + [None] * (L_new - keep)
    q = [x.copy() for x in s.q[:keep]] + [None] * (L_new - 1 - keep)
    u = [x.copy() for x in s.u[:keep]] + [None] * (L_new - 1 - keep)
    for l in range(keep, L_new):           # placeholders of the right shape; start_layers_from fills them
        z[l] = np.zeros((W[l].shape[0], n_nodes))
        if l < L_new - 1:
            q[l - 0] = np.zeros((W[l].shape[0], n_nodes))
            u[l - 0] = np.zeros((W[l].shape[0], n_nodes))
            p[l + 1] = np.zeros((W[l].shape[0], n_nodes))
    scale = list(s.scale[:keep + 1]) + [1.0] * (L_new - keep - 1)
    grown = State(p, W, b, z, q, u, s.y.copy(), s.mask.copy(), scale, [0.0] * L_new, [0.0] * L_new, [0] * L_new)
    return start_layers_from(grown, prm, keep + 1)


# ----------------------------------------------------------------------------
# The same iteration on node shards
# ----------------------------------------------------------------------------

def split_nodes(n_nodes: int, n_parts: int):
    """Contiguous, balanced node ranges: part r holds nodes [r N // R, (r+1) N // R)."""
    return [slice(r * n_nodes // n_parts, (r + 1) * n_nodes // n_parts) for r in range(n_parts)]


def shard_state(s: State, parts) -> List[State]:
    """The columns (nodes) of p, z, q, u, y, mask of each part; W, b and the level spacings are replicated."""
    out = []
    for sl in parts:
        out.append(State([a[:, sl].copy() for a in s.p], [w.copy() for w in s.W], [b.copy() for b in s.b],
                         [a[:, sl].copy() for a in s.z], [a[:, sl].copy() for a in s.q], [a[:, sl].copy() for a in s.u],
                         s.y[sl].copy(), s.mask[sl].copy(), list(s.scale), list(s.tau), list(s.theta), list(s.trials)))
    return out


def merge_shards(shards: List[State]) -> State:
    """Inverse of shard_state (W, b, scalars from the first shard: they are identical on all)."""
    f = shards[0]
    cat = lambda name, l: np.concatenate([getattr(x, name)[l] for x in shards], axis=1)
    return State([cat("p", l) for l in range(f.L)], [w.copy() for w in f.W], [b.copy() for b in f.b],
                 [cat("z", l) for l in range(f.L)], [cat("q", l) for l in range(f.L - 1)],
                 [cat("u", l) for l in range(f.L - 1)], np.concatenate([x.y for x in shards]),
                 np.concatenate([x.mask for x in shards]), list(f.scale), list(f.tau), list(f.theta), list(f.trials))


def _local_sum(values):
    """Sum of the partial results of this process's shards, in shard order."""
    total = values[0]
    for v in values[1:]:
        total = total + v
    return total


def iterate_sharded(shards: List[State], prm: Params, allreduce=None) -> List[State]:
    """One pass of Algorithm 1 with the nodes divided among shards (the multi-device form that the augmented MLP
    admits: once X is built, p_l, z_l, q_l, u_l are one column per node and W_l, b_l are shared).

    Every update acts on each node's column by itself except for the sums over nodes inside the step parameters
    and the shared variables: ||g||^2 and ||W g||^2 (tau, Eq. update p), the sums of the acceptance test of the
    quantised update, nabla_W phi = nu sum_j (W p + b - z)_j p_j^T and ||G p||^2 (theta, Eq. update W), and
    nabla_b phi = nu sum_j (W p + b - z)_j (Eq. update b).  Each shard forms its part of these sums; `allreduce`
    receives this process's part (its shards added in shard order) and returns the sum over all processes.  With
    allreduce=None the given shards are all there is.  The result equals `iterate` on the merged state up to the
    order of those additions.
    """
    rho, nu, L = prm.rho, prm.nu, shards[0].L
    total = (lambda parts: _local_sum(parts)) if allreduce is None else (lambda parts: allreduce(_local_sum(parts)))
    new = [s.copy() for s in shards]
    n_total = int(total([np.array(float(s.p[0].shape[1])) for s in shards]))
    # p_l^{k+1}, l = 2..L
    for l in range(1, L):
        g = [grad_p_phi(s.p[l], s.W[l], s.b[l], s.z[l], nu, s.q[l - 1], s.u[l - 1], rho) for s in shards]
        sums = total([np.array([float(np.sum(gi * gi)), float(np.sum((s.W[l] @ gi) ** 2))]) for s, gi in zip(shards, g)])
        gg, wg = float(sums[0]), float(sums[1])
        tau = float(rho) if gg == 0.0 else float(rho + nu * wg / gg)
        trials = 0
        if prm.quant_levels:
            phi_old = [phi(s.p[l], s.W[l], s.b[l], s.z[l], nu, s.q[l - 1], s.u[l - 1], rho) for s in shards]
            for trial in range(1, prm.max_trials + 1):
                p_new = [nearest_level(s.p[l] - gi / tau, s.scale[l], prm.quant_levels, prm.level_lo)[1]
                         for s, gi in zip(shards, g)]
                parts = []
                for s, gi, pn, po in zip(shards, g, p_new, phi_old):
                    d = pn - s.p[l]
                    parts.append(np.array([phi(pn, s.W[l], s.b[l], s.z[l], nu, s.q[l - 1], s.u[l - 1], rho), po,
                                           float(np.sum(gi * d)), float(np.sum(d * d))]))
                lhs, po, gd, dd = (float(x) for x in total(parts))
                trials = trial
                if lhs <= po + gd + 0.5 * tau * dd + 0.5 * prm.accept_slack * tau * dd:
                    break
                tau *= 2.0
            else:
                trials = -1
        else:
            p_new = [s.p[l] - gi / tau for s, gi in zip(shards, g)]
        for n, pn in zip(new, p_new):
            n.p[l], n.tau[l], n.trials[l] = pn, tau, trials
    # W_l^{k+1}: the gradient is a sum over nodes, theta needs ||G p||^2
    for l in range(L):
        G = total([grad_W_phi(n.p[l], s.W[l], s.b[l], s.z[l], nu) for s, n in zip(shards, new)])
        GG = float(np.sum(G * G))
        Gp2 = float(total([np.array(float(np.sum((G @ n.p[l]) ** 2))) for n in new]))
        theta = 0.0 if GG == 0.0 else float(nu * Gp2 / GG)
        for s, n in zip(shards, new):
            n.W[l] = s.W[l].copy() if theta == 0.0 else s.W[l] - G / theta
            n.theta[l] = theta
    # b_l^{k+1}: the gradient is a sum over nodes, the step is 1 / (nu |V|) with |V| the total node count
    for l in range(L):
        gb = total([grad_b_phi(n.p[l], n.W[l], s.b[l], s.z[l], nu) for s, n in zip(shards, new)])
        for s, n in zip(shards, new):
            n.b[l] = s.b[l] - gb / (nu * n_total)
    # z, q, u: node by node
    for s, n in zip(shards, new):
        for l in range(L):
            a = n.W[l] @ n.p[l] + n.b[l][:, None]
            if l < L - 1:
                n.z[l] = _update_z_hidden_for(prm, a, s.q[l], s.z[l])
            elif prm.risk == "ls":
                n.z[l] = update_z_last_least_squares(a, s.y, s.mask, nu)
            else:
                n.z[l] = update_z_last(a, s.y, s.mask, nu)
        for l in range(L - 1):
            if prm.quant_levels and prm.quantize_q:
                n.q[l] = update_q_quantized(n.p[l + 1], s.u[l], n.z[l], rho, nu, s.scale[l + 1], prm.quant_levels,
                                            prm.level_lo, prm.f)
            else:
                n.q[l] = update_q(n.p[l + 1], s.u[l], n.z[l], rho, nu, prm.f)
        for l in range(L - 1):
            n.u[l] = update_u(s.u[l], n.p[l + 1], n.q[l], rho)
    return new


def objective_sharded(shards: List[State], prm: Params, allreduce=None) -> np.ndarray:
    """The components of L_rho of the merged state: every component is a sum over nodes."""
    parts = [objective(s, prm)[:5] for s in shards]
    comps = _local_sum(parts) if allreduce is None else allreduce(_local_sum(parts))
    return np.concatenate([comps, [np.sum(comps)]])


# ----------------------------------------------------------------------------
# The trained model: forward pass, prediction, accuracy
# ----------------------------------------------------------------------------

def forward(X, W, b, slope=0.0) -> np.ndarray:
    """z_L of the GA-MLP of Problem 1 with the constraints enforced: p_1 = X,
    z_l = W_l p_l + b_l, p_{l+1} = f_l(z_l) = relu(z_l) (l < L).  Returns z_L (n_L x |V|)."""
    p = np.asarray(X, dtype=np.float64)
    for l in range(len(W)):
        z = W[l] @ p + np.asarray(b[l])[:, None]
        p = relu(z, slope)
    return z


def predict(X, W, b, slope=0.0) -> np.ndarray:
    """Class of every node: the largest entry of z_L (the class the cross-entropy risk R(z_L; y) rewards);
    the first one if several are equal."""
    return np.argmax(forward(X, W, b, slope), axis=0)


def accuracy(pred, y, mask) -> float:
    """Fraction of the nodes selected by `mask` whose predicted class equals the label (the paper's tables
    report it on the training, validation and test nodes)."""
    mask = np.asarray(mask, dtype=bool)
    return float(np.mean(np.asarray(pred)[mask] == np.asarray(y)[mask])) if mask.any() else float("nan")
