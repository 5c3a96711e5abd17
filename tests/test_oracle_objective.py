"""Pins of the oracle's read-outs: the augmented Lagrangian L_rho with its five components, and the residuals of
Algorithm 1, against a state whose every number was worked by hand (tests/golden/lagrangian_small_state.txt)."""

import os

import numpy as np
import pytest

import oracle.pdadmm_oracle as o

GOLD = os.path.join(os.path.dirname(__file__), "golden", "lagrangian_small_state.txt")


def read_named_arrays(path):
    """Arrays of a golden file: a line "name rows cols" followed by `rows` lines of numbers; '#' starts a comment."""
    out, lines = {}, [ln.split("#")[0].strip() for ln in open(path)]
    lines = [ln for ln in lines if ln]
    i = 0
    while i < len(lines):
        name, rows, cols = lines[i].split()
        rows, cols = int(rows), int(cols)
        a = np.array([[float(x) for x in lines[i + 1 + r].split()] for r in range(rows)])
        assert a.shape == (rows, cols), name
        out[name] = a
        i += 1 + rows
    return out


def golden_state(mask=(True, True)):
    g = read_named_arrays(GOLD)
    L = 3
    s = o.State(p=[g[f"p{l}"] for l in range(1, L + 1)], W=[g[f"W{l}"] for l in range(1, L + 1)],
                b=[g[f"b{l}"].ravel() for l in range(1, L + 1)], z=[g[f"z{l}"] for l in range(1, L + 1)],
                q=[g[f"q{l}"] for l in range(1, L)], u=[g[f"u{l}"] for l in range(1, L)],
                y=g["y"].ravel().astype(int), mask=np.array(mask), scale=[1.0] * L)
    prm = o.Params(rho=float(g["rho"][0, 0]), nu=float(g["nu"][0, 0]))
    return g, s, prm


def test_objective_components_equal_the_hand_worked_values():
    g, s, prm = golden_state()
    got = o.objective(s, prm)
    assert np.allclose(got, g["components"].ravel(), rtol=0, atol=1e-13)
    assert o.lagrangian(s, prm) == got[5]
    assert abs(got[5] - sum(got[:5])) < 1e-13


def test_objective_counts_the_risk_of_labelled_nodes_only():
    g, s, prm = golden_state(mask=(True, False))
    assert np.allclose(o.objective(s, prm), g["components_node1_unlabelled"].ravel(), rtol=0, atol=1e-13)


def test_residuals_equal_the_hand_worked_values():
    g, s, prm = golden_state()
    got = o.residuals_sq(s)
    assert got.shape == (2,)
    assert np.allclose(got, g["residuals_sq"].ravel(), rtol=0, atol=1e-14)


def test_objective_responds_to_each_penalty_separately():
    """nu scales the two relaxation terms only, rho the penalty term only; R and the dual term depend on neither."""
    g, s, prm = golden_state()
    base = g["components"].ravel()
    got = o.objective(s, o.Params(rho=6.0, nu=0.125))
    want = np.array([base[0], base[1] / 4, base[2] / 4, base[3], base[4] * 3, 0.0])
    want[5] = want[:5].sum()
    assert np.allclose(got, want, rtol=0, atol=1e-13)


def test_least_squares_risk_component():
    """The same state with R = 1/2 sum ||z_L - e_y||^2: node 0 (2, 3.5) vs e_1 -> (4 + 6.25)/2, node 1 (1, 3) vs e_0 -> 9/2."""
    g, s, prm = golden_state()
    prm.risk = "ls"
    got = o.objective(s, prm)
    assert abs(got[0] - (5.125 + 4.5)) < 1e-14
    assert np.allclose(got[1:5], g["components"].ravel()[1:5], rtol=0, atol=1e-13)
