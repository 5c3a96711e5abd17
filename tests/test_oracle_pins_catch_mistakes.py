"""The pins have teeth: a plausible mistake planted in the oracle (a dropped term, a wrong sign, a transposed
operand, a wrong constant) makes at least one of the pin tests fail.  Every mistake is planted on the CPU, in the
oracle module, for the duration of one check."""

import numpy as np
import pytest

import oracle.pdadmm_oracle as o
import test_oracle_graph as tg
import test_oracle_iteration as ti
import test_oracle_objective as tobj
import test_oracle_quantised_q as tq
import test_oracle_subproblems as ts


def _fails(test, *args):
    try:
        test(*args)
    except AssertionError:
        return True
    except Exception:            # a shape error is a failure too (e.g. a transposed operand)
        return True
    return False


def _grad_p_without_dual_term(p, W, b, z, nu, q_prev, u_prev, rho):
    return nu * W.T @ (W @ p + b[:, None] - z) + rho * (p - q_prev)


def _grad_p_wrong_sign(p, W, b, z, nu, q_prev, u_prev, rho):
    return nu * W.T @ (z - W @ p - b[:, None]) + u_prev + rho * (p - q_prev)


def _grad_W_transposed(p, W, b, z, nu):
    G = nu * (W @ p + b[:, None] - z) @ p.T
    return G.T.reshape(G.shape) if G.shape[0] != G.shape[1] else G.T        # operands of the outer product swapped


def _update_u_wrong_sign(u, p_next, q, rho):
    return u - rho * (p_next - q)


def _update_q_without_nu(p_next, u, z, rho, nu, slope=0.0):
    return (rho * p_next + u + nu * o.relu(z, slope)) / rho


def _update_z_hidden_wrong_constant(a, q, z_old, slope=0.0):
    z_neg = np.minimum((a + slope * q + z_old) / (2.0 + slope * slope), 0.0)
    z_pos = np.maximum((a + q + z_old) / 2.0, 0.0)
    f_neg = o.z_objective_hidden(z_neg, a, q, z_old, slope)
    f_pos = o.z_objective_hidden(z_pos, a, q, z_old, slope)
    return np.where(f_pos < f_neg, z_pos, z_neg)


def _tau_too_small(g, W, nu, rho):
    gg = float(np.sum(g * g))
    return rho if gg == 0 else rho + 0.5 * nu * float(np.sum((W @ g) ** 2)) / gg


def _update_b_mean_of_wrong_thing(p, W, b, z, nu):
    return np.mean(z, axis=1)


def _quantize_truncating(x, scale, m, lo=0.0):
    x32 = np.asarray(x, dtype=np.float32)
    c = np.clip(np.floor((x32 - np.float32(lo)) / np.float32(scale)), 0, m - 1)
    return c.astype(np.uint8 if m <= 256 else np.uint16), (np.float32(lo) + c * np.float32(scale)).astype(np.float64)



def _objective_variant(rho_factor=1.0, dual_sign=1.0, lin_factor=1.0, act_factor=1.0, dual_factor=1.0):
    """L_rho with one component scaled, dropped or sign-flipped."""
    def wrong(s, prm):
        rho, nu, L = prm.rho, prm.nu, s.L
        R = o.risk_least_squares(s.z[L - 1], s.y, s.mask) if prm.risk == "ls" else o.risk(s.z[L - 1], s.y, s.mask)
        lin = sum(float(np.sum((s.z[l] - s.W[l] @ s.p[l] - s.b[l][:, None]) ** 2)) for l in range(L))
        act = sum(float(np.sum((s.q[l] - o.relu(s.z[l], prm.slope)) ** 2)) for l in range(L - 1))
        dual = sum(float(np.sum(s.u[l] * (s.p[l + 1] - s.q[l]))) for l in range(L - 1))
        pen = sum(float(np.sum((s.p[l + 1] - s.q[l]) ** 2)) for l in range(L - 1))
        comps = [R, lin_factor * 0.5 * nu * lin, act_factor * 0.5 * nu * act, dual_sign * dual_factor * dual,
                 rho_factor * 0.5 * rho * pen]
        return np.array(comps + [sum(comps)])
    return wrong


def _residuals_without_the_square(s):
    return np.array([float(np.sum(np.abs(s.p[l + 1] - s.q[l]))) for l in range(s.L - 1)])


def _residuals_doubled(s):
    return np.array([2.0 * float(np.sum((s.p[l + 1] - s.q[l]) ** 2)) for l in range(s.L - 1)])


def _residuals_of_the_wrong_pair(s):
    return np.array([float(np.sum((s.p[l] [:s.q[l].shape[0]] - s.q[l]) ** 2)) if s.p[l].shape[0] >= s.q[l].shape[0]
                     else 0.0 for l in range(s.L - 1)])


def _risk_as_a_mean(zL, y, mask):
    m = np.max(zL, axis=0)
    ce = m + np.log(np.sum(np.exp(zL - m[None, :]), axis=0)) - zL[y, np.arange(zL.shape[1])]
    return float(np.mean(ce[np.asarray(mask, dtype=bool)]))


def _nearest_level_rounding_down_at_ties(x, scale, m, lo=0.0):
    x = np.asarray(x, dtype=np.float64)
    lev = o.level_set(scale, m, lo)
    c = np.clip(np.ceil((x - lo) / scale - 0.5), 0, m - 1).astype(np.int64)
    return c.astype(np.uint8 if m <= 256 else np.uint16), lev[c]


def _nearest_level_truncating(x, scale, m, lo=0.0):
    x = np.asarray(x, dtype=np.float64)
    lev = o.level_set(scale, m, lo)
    c = np.clip(np.floor((x - lo) / scale), 0, m - 1).astype(np.int64)
    return c.astype(np.uint8 if m <= 256 else np.uint16), lev[c]


_GOOD_ADJACENCY = o.renormalized_adjacency


def _adjacency_without_self_loops(n, src, dst):
    import scipy.sparse as sp
    A = _GOOD_ADJACENCY(n, src, dst)
    return sp.csr_matrix(A - sp.diags(A.diagonal()))


MISTAKES = [
    ("grad_p_phi", _grad_p_without_dual_term, [ts.test_gradients_of_phi_by_finite_differences, ti.test_lemma_q_opt_holds_every_iteration], (0,)),
    ("grad_p_phi", _grad_p_wrong_sign, [ts.test_gradients_of_phi_by_finite_differences], ()),
    ("grad_W_phi", _grad_W_transposed, [ts.test_gradients_of_phi_by_finite_differences], ()),
    ("update_u", _update_u_wrong_sign, [ts.test_u_update_written_out, ti.test_lemma_q_opt_holds_every_iteration], (0,)),
    ("update_q", _update_q_without_nu, [ts.test_q_update_gradient_and_grid], ()),
    ("update_z_hidden", _update_z_hidden_wrong_constant, [ts.test_z_hidden_against_dense_scalar_grid], ()),
    ("tau_smallest_admissible", _tau_too_small, [ts.test_p_update_identity_and_smallest_tau], ()),
    ("update_b", _update_b_mean_of_wrong_thing, [ts.test_b_update_is_the_minimiser_grid_and_gradient], ()),
    ("quantize", _quantize_truncating, [tg.test_quantize_ties_and_clamps], ()),
    ("renormalized_adjacency", _adjacency_without_self_loops, [tg.test_golden_path_graph], ()),
    ("nearest_level", _nearest_level_rounding_down_at_ties, [tq.test_nearest_level_is_the_argmin_over_all_levels], (22, 1.0, -1.0)),
    ("nearest_level", _nearest_level_truncating, [tq.test_nearest_level_is_the_argmin_over_all_levels], (16, 0.0173, -0.0371)),
    ("objective", _objective_variant(rho_factor=2.0), [tobj.test_objective_components_equal_the_hand_worked_values], ()),
    ("objective", _objective_variant(dual_sign=-1.0), [tobj.test_objective_components_equal_the_hand_worked_values], ()),
    ("objective", _objective_variant(lin_factor=2.0), [tobj.test_objective_components_equal_the_hand_worked_values], ()),
    ("objective", _objective_variant(act_factor=0.0), [tobj.test_objective_components_equal_the_hand_worked_values], ()),
    ("objective", _objective_variant(dual_factor=0.0), [tobj.test_objective_components_equal_the_hand_worked_values], ()),
    ("residuals_sq", _residuals_without_the_square, [tobj.test_residuals_equal_the_hand_worked_values], ()),
    ("residuals_sq", _residuals_doubled, [tobj.test_residuals_equal_the_hand_worked_values], ()),
    ("residuals_sq", _residuals_of_the_wrong_pair, [tobj.test_residuals_equal_the_hand_worked_values], ()),
    ("risk", _risk_as_a_mean, [tobj.test_objective_components_equal_the_hand_worked_values], ()),
]


@pytest.mark.parametrize("name,wrong,tests,extra", MISTAKES, ids=[f"{i}-{m[0]}:{m[1].__name__}" for i, m in enumerate(MISTAKES)])
def test_planted_mistake_is_caught(monkeypatch, name, wrong, tests, extra):
    for t in tests:                                    # the pins pass on the oracle as it stands ...
        args = extra if t.__code__.co_argcount else ()
        t(*args)
    monkeypatch.setattr(o, name, wrong)
    caught = [t.__name__ for t in tests if _fails(t, *(extra if t.__code__.co_argcount else ()))]
    assert caught, f"no pin noticed the mistake planted in {name}"      # ... and at least one fails with the mistake
