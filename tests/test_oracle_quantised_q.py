"""Pins of the pdADMM-G-Q variants: level sets that do not start at zero (the paper's own
Delta = {-1, ..., 20}) and the variant that keeps q in Delta as well."""

import os

import numpy as np
import pytest

import oracle.pdadmm_oracle as o
from paper_2105_09837_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _problem(n=200, d=10, hidden=12, L=4):
    w = synth.small("c1", n, feat_dim=d, hidden=hidden, n_layers=L)
    inp = synth.make_inputs(w)
    A = o.renormalized_adjacency(w.n_nodes, inp.edge_src, inp.edge_dst)
    X = o.augment(inp.features.T.astype(np.float64), A, w.n_blocks)
    return X, [x.astype(np.float64) for x in inp.init_W], inp.labels, inp.train_mask


def test_paper_default_level_set():
    want = np.loadtxt(os.path.join(GOLD, "paper_default_level_set.txt"))
    assert np.array_equal(o.level_set(1.0, 22, -1.0), want)
    codes, vals = o.quantize(np.array([-7.0, -1.4, -0.5, -0.51, 0.49, 3.5, 19.6, 33.0]), 1.0, 22, -1.0)
    assert vals.tolist() == [-1.0, -1.0, 0.0, -1.0, 0.0, 4.0, 20.0, 20.0]      # ties go up, ends clamp
    assert codes.tolist() == [0, 0, 1, 0, 1, 5, 21, 21]


@pytest.mark.parametrize("m,scale,lo", [(22, 1.0, -1.0), (16, 0.0173, -0.0371), (256, 0.011, 0.25), (1000, 0.003, -0.3)])
def test_quantize_with_offset_is_nearest_level_brute_force(m, scale, lo):
    rng = np.random.default_rng(m)
    scale, lo = float(np.float32(scale)), float(np.float32(lo))
    x = rng.uniform(lo - 2 * scale, lo + (m + 1) * scale, size=5000)
    codes, vals = o.quantize(x, scale, m, lo)
    levels = o.level_set(scale, m, lo)
    assert np.array_equal(vals, levels[codes])
    assert codes.dtype == (np.uint8 if m <= 256 else np.uint16) and int(codes.max()) == m - 1
    x32 = x.astype(np.float32).astype(np.float64)
    dist = np.abs(x32[:, None] - levels[None, :])
    assert np.all(np.abs(x32 - vals) <= dist.min(axis=1) + 1e-6 * scale + 4e-7 * np.abs(x32))
    t = (x32 - lo) / scale
    far = np.abs(np.abs(t - np.floor(t)) - 0.5) > 1e-3
    assert np.array_equal(codes[far], dist.argmin(axis=1)[far].astype(codes.dtype))


@pytest.mark.parametrize("m,scale,lo", [(2, 0.5, 0.0), (22, 1.0, -1.0), (16, 0.0173, -0.0371), (256, 0.011, 0.25),
                                        (1000, 0.003, -0.3)])
def test_nearest_level_is_the_argmin_over_all_levels(m, scale, lo):
    """The projection that the quantised updates use is exactly argmin_delta |delta - x| (no tolerance): brute force
    over all m levels in double precision, exact ties resolved towards the upper level, ends clamped."""
    rng = np.random.default_rng(7 * m)
    scale, lo = float(np.float32(scale)), float(np.float32(lo))
    levels = o.level_set(scale, m, lo)
    x = rng.uniform(lo - 2 * scale, lo + (m + 1) * scale, size=6000)
    x[:m - 1] = 0.5 * (levels[:-1] + levels[1:])              # exact midpoints of neighbouring levels
    x[m:2 * m] = levels + rng.uniform(-1e-9, 1e-9, size=m)    # values within rounding of a level
    codes, vals = o.nearest_level(x, scale, m, lo)
    dist = np.abs(x[:, None] - levels[None, :])
    # first minimum from the top = the upper of two tied levels
    want = (m - 1 - np.argmin(dist[:, ::-1], axis=1))
    assert np.array_equal(codes.astype(np.int64), want)
    assert np.array_equal(vals, levels[want])
    assert codes.dtype == (np.uint8 if m <= 256 else np.uint16)
    # the single-precision rounding agrees with it away from the rounding boundaries
    c32 = o.quantize(x, scale, m, lo)[0]
    t = (x - lo) / scale
    far = np.abs(np.abs(t - np.floor(t)) - 0.5) > 1e-3
    assert np.array_equal(c32[far], codes[far])


def test_quantised_q_minimises_the_q_subproblem_over_delta():
    """Brute force: per element, the level with the smallest value of the terms of L_rho that contain q_l,
    (nu/2)(q - f(z))^2 + u (p_next - q) + (rho/2)(p_next - q)^2, is the one update_q_quantized returns."""
    rng = np.random.default_rng(3)
    rho, nu, m, lo = 0.7, 0.3, 22, -1.0
    p_next = o.quantize(rng.uniform(-2, 21, (6, 50)), 1.0, m, lo)[1]
    u = rng.normal(0, 0.4, (6, 50))
    z = rng.normal(3, 5, (6, 50))
    got = o.update_q_quantized(p_next, u, z, rho, nu, 1.0, m, lo)
    levels = o.level_set(1.0, m, lo)
    f = o.relu(z)
    cost = (0.5 * nu * (levels[:, None, None] - f) ** 2 + u * (p_next - levels[:, None, None])
            + 0.5 * rho * (p_next - levels[:, None, None]) ** 2)
    best = cost.min(axis=0)
    mine = 0.5 * nu * (got - f) ** 2 + u * (p_next - got) + 0.5 * rho * (p_next - got) ** 2
    assert np.all(np.isin(got, levels))
    assert np.all(mine <= best + 1e-6 * (1 + np.abs(best)))
    # away from ties the minimiser is unique
    srt = np.sort(cost, axis=0)
    clear = srt[1] - srt[0] > 1e-4
    assert np.array_equal(got[clear], levels[cost.argmin(axis=0)][clear])


@pytest.mark.parametrize("lo,step", [(0.0, 0.0), (-1.0, 1.0)])
def test_iterates_stay_in_delta_and_start_is_feasible(lo, step):
    X, W0, y, mask = _problem()
    m = 22 if step else 16
    prm = o.Params(0.5, 0.02, m, quantize_q=True, level_lo=lo, level_step=step)
    s = o.init_state(X, W0, y, mask, prm)
    assert np.allclose(o.residuals_sq(s), 0)                     # q_l = p_{l+1} = Proj(relu(z_l))
    for l in range(1, s.L):
        if step:
            assert s.scale[l] == step
        if not step:                                              # a fixed set may clamp at its top
            assert np.max(np.abs(s.p[l] - o.relu(s.z[l - 1]))) <= s.scale[l] / 2 * (1 + 1e-6)
    for _ in range(4):
        s = o.iterate(s, prm)
        for l in range(1, s.L):
            lev = o.level_set(s.scale[l], m, lo)
            assert np.all(np.isin(s.p[l], lev)) and np.all(np.isin(s.q[l - 1], lev))
        assert np.all(np.isfinite(o.objective(s, prm)))


def test_fine_level_set_reproduces_the_unquantised_q_update():
    """With a fine set that covers the values, one q-update from the same state differs from the
    real-valued one by at most half a step per element."""
    X, W0, y, mask = _problem()
    base = o.Params(0.5, 0.02, 256)
    s = o.init_state(X, W0, y, mask, base)
    s = o.iterate(s, base)
    a = o.iterate(s, base)
    b = o.iterate(s, o.Params(0.5, 0.02, 256, quantize_q=True))
    for l in range(s.L - 1):
        inside = a.q[l] <= 255 * s.scale[l + 1]
        assert np.max(np.abs(a.q[l] - b.q[l])[inside]) <= s.scale[l + 1] / 2 * (1 + 1e-5)
        assert np.array_equal(a.p[l + 1], b.p[l + 1])            # p does not depend on the choice for q
