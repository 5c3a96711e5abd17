"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same seeded inputs.

Tolerances: integer work (CSR structure, quantisation codes on identical inputs) is bit-exact; every
floating-point variable of the state agrees within a relative Frobenius error of 1e-4 after one
teacher-forced iteration; the augmented Lagrangian agrees within 1e-3 after 20 free-running iterations.
"""

import numpy as np
import pytest

import oracle.pdadmm_oracle as o
from paper_2105_09837_b200 import binding as B
from paper_2105_09837_b200 import synth
import error_bounds as EB
import parity_util as U

pytestmark = pytest.mark.gpu

TOL = 1e-4


def _cases():
    # name, base workload, overrides: sizes span several 128-row tiles with ragged tails and odd widths
    return {
        "er-small": ("c1", dict(n_nodes=700, feat_dim=18, hidden=36, n_layers=4)),
        "ba-ragged": ("c2", dict(n_nodes=1237, feat_dim=37, hidden=150, n_layers=5, n_hops=2)),
        "ba-wide": ("c2", dict(n_nodes=901, feat_dim=50, hidden=260, n_layers=3)),
        "c4-like": ("c4", dict(n_nodes=1500, feat_dim=16, hidden=130, n_layers=4)),
    }


def _inputs(case, **extra):
    base, kw = _cases()[case]
    kw = dict(kw)
    kw.update(extra)
    return synth.make_inputs(synth.small(base, **kw))


# ----------------------------------------------------------------------------- init: graph, augmentation, forward pass

@pytest.mark.parametrize("case", ["er-small", "ba-ragged", "c4-like"])
def test_init_graph_augmentation_and_forward_pass(case):
    inp = _inputs(case, quant_levels=0)
    prm, s, A = U.oracle_problem(inp)
    ctx = B.from_inputs(inp)
    # CSR structure is integer work: bit-exact
    assert np.array_equal(ctx.get_tensor(B.T_CSR_ROWPTR), A.indptr.astype(np.int32))
    assert np.array_equal(ctx.get_tensor(B.T_CSR_COLIDX), A.indices.astype(np.int32))
    assert np.allclose(ctx.get_tensor(B.T_CSR_VAL), A.data, rtol=3e-7, atol=0)
    X = ctx.get_tensor(B.T_X).T.astype(np.float64)
    d = inp.workload.feat_dim
    assert np.array_equal(X[:d], s.p[0][:d])                                  # block 0 is H itself
    assert U.rel_err(X, s.p[0]) < 1e-6
    st = U.read_state(ctx)
    for l in range(s.L):
        assert U.rel_err(st["z"][l], s.z[l]) < 1e-5
        assert U.rel_err(st["p"][l], s.p[l]) < 1e-5
        assert np.all(st["b"][l] == 0)
    for l in range(s.L - 1):
        assert U.rel_err(st["q"][l], s.q[l]) < 1e-5
        assert np.all(st["u"][l] == 0)
    ob_g, ob_o = ctx.objective(), o.objective(s, prm)
    assert abs(ob_g[0] - ob_o[0]) <= 1e-5 * ob_o[0]
    assert np.allclose(ctx.residuals(), 0)
    ctx.destroy()


def test_init_quantised_start():
    inp = _inputs("ba-ragged", quant_levels=16)
    prm, s, _ = U.oracle_problem(inp)
    ctx = B.from_inputs(inp)
    for l in range(2, s.L + 1):
        scale = ctx.get_tensor(B.T_QSCALE, l)[0]
        assert abs(scale - s.scale[l - 1]) <= 2e-6 * s.scale[l - 1]
        codes = ctx.get_tensor(B.T_CODES, l)
        p = ctx.get_tensor(B.T_P, l)
        assert codes.max() <= 15
        assert np.array_equal(p, codes.astype(np.float32) * np.float32(scale))   # p in Delta, bit for bit
    assert ctx.residuals().sum() > 0
    ctx.destroy()


def test_setting_p_or_its_spacing_keeps_p_equal_to_the_levels_of_its_codes():
    """The kernels of pdADMM-G-Q read p_l through its codes, so whatever a caller stores must end up as a pair
    (codes, p = levels of those codes): values off the level set are projected (Eq. "update p quantized": nearest level),
    and a new spacing moves p_l to the new level set."""
    inp = _inputs("ba-ragged", quant_levels=16)
    ctx = B.from_inputs(inp)
    rng = np.random.default_rng(5)
    for l in (2, 3):
        s = np.float32(ctx.get_tensor(B.T_QSCALE, l)[0])
        p = ctx.get_tensor(B.T_P, l)
        noisy = (p + np.float32(0.3) * s * rng.uniform(-1, 1, p.shape).astype(np.float32)).astype(np.float32)
        ctx.set_tensor(B.T_P, l, noisy)
        want_codes, want_p = o.quantize(noisy, float(s), 16)           # both sides get the same fp32 input: bit for bit
        assert np.array_equal(ctx.get_tensor(B.T_CODES, l), want_codes)
        assert np.array_equal(ctx.get_tensor(B.T_P, l), want_p.astype(np.float32))
        s2 = np.float32(1.5) * s
        ctx.set_tensor(B.T_QSCALE, l, np.array([s2], dtype=np.float32))
        want_codes, want_p = o.quantize(want_p.astype(np.float32), float(s2), 16)
        assert np.array_equal(ctx.get_tensor(B.T_CODES, l), want_codes)
        assert np.array_equal(ctx.get_tensor(B.T_P, l), want_p.astype(np.float32))
    ctx.step(2)                                                        # and the iteration keeps the pair together
    for l in (2, 3):
        s = np.float32(ctx.get_tensor(B.T_QSCALE, l)[0])
        assert np.array_equal(ctx.get_tensor(B.T_P, l), ctx.get_tensor(B.T_CODES, l).astype(np.float32) * s)
    ctx.destroy()


# ----------------------------------------------------------------------------- one teacher-forced iteration

def _compare_iteration(ctx, prev, prm, label, tensor_cores=True, report=None, single_bounds=False):
    """prev: fp32-representable oracle state, already loaded.  Steps both sides once and compares every variable:
    relative Frobenius error <= 1e-4 and largest elementwise error <= 1e-4 of the largest element.  Where a variable
    is a small difference of large terms (b, u) the bar is the rounding level of its own computation as
    error_bounds.iteration_bounds propagates it, if that is larger.  Discrete decisions are compared exactly outside
    the elements whose deciding value lies within its own rounding bound of the boundary.  `report`, if a dict,
    receives the measured numbers."""
    nxt = o.iterate(prev, prm)
    ctx.step(1)
    got = U.read_state(ctx)
    L = prev.L
    quant = prm.quant_levels > 0
    tau_dev = [0.0] + [float(ctx.get_tensor(B.T_TAU, l + 1)[0]) for l in range(1, L)]
    bd = EB.iteration_bounds(prev, nxt, prm, tensor_cores, tau_dev, single=single_bounds)
    worst, worst_el, stats = {}, {}, {}

    def compare(name, g, w, delta=None, mask=None):
        """Frobenius and elementwise errors of one variable outside `mask`; delta: elementwise rounding bound that may
        replace the 1e-4 bar where it is larger (None: the plain bar)."""
        keep = slice(None) if mask is None else ~mask
        g, w = g[keep], w[keep]
        err = np.abs(g - w)
        floor_f = 0.0 if delta is None else float(np.linalg.norm(delta[keep]))
        worst[name] = float(np.linalg.norm(err) / max(np.linalg.norm(w), floor_f / TOL, 1e-300))
        el_bar = TOL * float(np.abs(w).max(initial=0.0))
        if delta is None:
            worst_el[name] = float(err.max(initial=0.0) / max(el_bar, 1e-300))
        else:
            worst_el[name] = float((err / np.maximum(el_bar, delta[keep])).max(initial=0.0))
        stats[name] = (float(np.linalg.norm(err) / max(np.linalg.norm(w), 1e-300)), float(err.max(initial=0.0)),
                       float(np.abs(w).max(initial=0.0)))

    flipped = 0
    masks = [None] * L
    for l in range(1, L):
        if not quant:
            continue
        trials = int(ctx.get_tensor(B.T_TRIALS, l + 1)[0])
        if trials != nxt.trials[l]:
            # the accept test is a floating-point decision; it may differ only at a (relative) tie
            pytest.skip(f"{label}: tau search took {trials} trials on the device, {nxt.trials[l]} in the oracle")
        # the value before the projection carries the rounding bound bd['x']: inside that distance of a boundary
        # between two levels either neighbour is the nearest level of a value the device could have computed
        mask = U.boundary_mask(prev, nxt, prm, l, tol=bd["x"][l] / prev.scale[l])
        codes = ctx.get_tensor(B.T_CODES, l + 1).T
        want_codes = np.rint((nxt.p[l] - prm.level_lo) / prev.scale[l]).astype(codes.dtype)
        diff = codes != want_codes
        stats[f"codes{l + 1}"] = (float(mask.mean()), int(diff.sum()), float(np.median(bd["x"][l] / prev.scale[l])))
        assert not np.any(diff & ~mask), f"{label}: codes differ away from a rounding boundary (layer {l + 1})"
        assert np.all(np.abs(codes.astype(int) - want_codes.astype(int)) <= 1)
        assert mask.mean() < (5e-3 if prm.quant_levels <= 256 else 5e-2), mask.mean()
        scale = np.float32(prev.scale[l])
        assert np.array_equal(got["p"][l].astype(np.float32), np.float32(prm.level_lo) + codes.astype(np.float32) * scale)
        if diff.any():
            # both neighbours are nearest levels of a value inside the rounding bound: the oracle continues from
            # the device's choice there, so that W, b, z, q, u (which all depend on p) are compared on equal terms
            flipped += int(diff.sum())
            nxt.p[l] = np.where(diff, got["p"][l], nxt.p[l])
        masks[l] = mask
    if flipped:
        nxt = U.redo_after_p(prev, nxt, prm)
    stats["flipped_codes"] = flipped
    for l in range(1, L):
        compare(f"p{l + 1}", got["p"][l], nxt.p[l], None, None)
        # tau is a ratio of two norms of the gradient; when the step it scales is itself at rounding level
        # (a nearly feasible state) the ratio is not determined, so it is compared only for real steps
        if np.linalg.norm(nxt.p[l] - prev.p[l]) > 1e-3 * np.linalg.norm(prev.p[l]):
            assert abs(tau_dev[l] - nxt.tau[l]) <= 1e-3 * nxt.tau[l], f"{label}: tau_{l + 1} {tau_dev[l]} vs {nxt.tau[l]}"
    for l in range(L):
        compare(f"W{l + 1}", got["W"][l], nxt.W[l])
        # b_l = mean_j (z - W p)_j is a small difference of terms of the size of W p: the bar is 1e-4 of ||b|| or the
        # propagated rounding of that mean, whichever is larger
        compare(f"b{l + 1}", got["b"][l], nxt.b[l], bd["b"][l])
        if np.linalg.norm(nxt.W[l] - prev.W[l]) > 1e-3 * np.linalg.norm(prev.W[l]):
            theta = float(ctx.get_tensor(B.T_THETA, l + 1)[0])
            assert abs(theta - nxt.theta[l]) <= 1e-3 * nxt.theta[l], f"{label}: theta_{l + 1} {theta} vs {nxt.theta[l]}"
        if l < L - 1:
            tie = (U.z_tie_mask(prev, nxt, l, slope=prm.slope) if prm.activation == "relu"
                   else U.z_table_tie_mask(prev, nxt, prm, l))
            # a coarse fixed level set (integers) makes q exactly 0 or a whole number in many places, and with it
            # exact ties between the two ReLU candidates; elsewhere ties are rare
            # with a lookup table a state that has not moved yet (a = z^k, q = f(z^k)) sits between two candidates that are
            # equally good up to the tiny asymmetry of f: ties are common in the first iterations
            assert tie.mean() < (0.5 if prm.activation != "relu" else (0.1 if prm.level_step else 1e-2))
            if quant and prm.quantize_q:
                # q is a discrete decision as well: on the level set bit for bit, equal to the oracle's except where
                # the value before the projection lies within its rounding bound of a boundary (one level off at most)
                lev = o.level_set(prev.scale[l + 1], prm.quant_levels, prm.level_lo)
                assert np.all(np.isin(got["q"][l], lev)), f"{label}: q_{l + 1} left the level set"
                qb = U.q_boundary_mask(prev, nxt, prm, l, tol=np.maximum(bd["q"][l] / prev.scale[l + 1], 1e-9)) | tie
                dq = np.abs(got["q"][l] - nxt.q[l])
                assert np.all(dq[~tie] <= prev.scale[l + 1] * (1 + 1e-4))      # levels are rounded fp32 numbers
                assert not np.any((dq > 0) & ~qb), f"{label}: q_{l + 1} differs away from a rounding boundary"
                stats[f"qcodes{l + 1}"] = (float(qb.mean()), int((dq > 0).sum()))
                # With rho = nu, u = 0 and an inactive ReLU the value to project is p_{l+1}/2: an exact tie between two
                # levels whenever the code of p_{l+1} is odd, so boundary elements are common here.  Both neighbours
                # minimise the q-subproblem there; they are left out of the comparison of q and of u (nothing else
                # in the iteration depends on q).
                tie = qb
            compare(f"z{l + 1}", got["z"][l], nxt.z[l], None, tie)
            compare(f"q{l + 1}", got["q"][l], nxt.q[l], None, tie)
            # u_l = u_l + rho (p_{l+1} - q_l) is a small difference of terms of size rho |p|: 1e-4 of ||u||, or the
            # propagated rounding of that difference where it is larger (a start where p = q has u = 0)
            um = tie
            compare(f"u{l + 1}", got["u"][l], nxt.u[l], bd["u"][l], um)
        else:
            compare(f"z{l + 1}", got["z"][l], nxt.z[l])
    if report is not None:
        report.update(stats=stats, frob=dict(worst), elementwise=dict(worst_el))
    bad = {k: v for k, v in worst.items() if not v <= TOL}
    bad.update({k + "(elementwise)": v for k, v in worst_el.items() if not v <= 1.0})
    assert not bad, f"{label}: errors above the bar: {bad} (Frobenius: {worst}; elementwise / bar: {worst_el})"
    return nxt


@pytest.mark.parametrize("case,levels,flags", [
    ("er-small", 0, 0), ("ba-ragged", 0, 0), ("ba-wide", 0, 0), ("c4-like", 0, 0),
    ("er-small", 16, 0), ("ba-ragged", 256, 0), ("c4-like", 256, 0),
    ("ba-wide", 1024, 0),          # 16-bit codes that are still exact in one fp16 plane (integer operands)
    ("ba-ragged", 0, B.FLAG_SIMT_GEMM), ("ba-ragged", 256, B.FLAG_SIMT_GEMM),
])
def test_teacher_forced_iterations(case, levels, flags):
    inp = _inputs(case, quant_levels=levels)
    prm, s, _ = U.oracle_problem(inp)
    ctx = B.from_inputs(inp, flags=flags)
    quant = levels > 0
    for k in range(5):
        prev = U.round_state(s)
        U.load_state(ctx, prev, quant)
        nxt = _compare_iteration(ctx, prev, prm, f"{case}/m={levels}/k={k}", tensor_cores=not (flags & B.FLAG_SIMT_GEMM))
        s = nxt
    ctx.destroy()


@pytest.mark.parametrize("case,levels,neg,step,quant_q", [
    ("er-small", 16, 0, 0.0, True),          # q kept on the level set of p_{l+1} as well
    ("ba-ragged", 256, 0, 0.0, True),
    ("er-small", 22, 1, 1.0, False),         # the level set {-1, 0, ..., 20} of the paper's experiments
    ("ba-ragged", 22, 1, 1.0, True),
    ("c4-like", 64, 3, 0.125, True),
    ("ba-ragged", 4096, 0, 0.0, True),       # 16-bit codes
])
def test_teacher_forced_level_set_variants(case, levels, neg, step, quant_q):
    inp = _inputs(case, quant_levels=levels)
    prm, s, _ = U.oracle_problem(inp, quantize_q=quant_q, neg_levels=neg, step=step)
    ctx = B.from_inputs(inp, flags=B.FLAG_QUANT_Q if quant_q else 0, quant_neg_levels=neg, quant_step=step)
    # the start: same level spacing, p (and q) on the level set, equal to the oracle's away from rounding boundaries
    st = U.read_state(ctx)
    for l in range(1, s.L):
        dev_scale = float(ctx.get_tensor(B.T_QSCALE, l + 1)[0])       # from the device's own max: last-bit differences
        assert dev_scale == pytest.approx(s.scale[l], rel=1e-6)
        lev = o.level_set(dev_scale, levels, prm.level_lo)
        assert np.all(np.isin(st["p"][l], lev))
        assert np.mean(np.abs(st["p"][l] - s.p[l]) > 0.5 * s.scale[l]) < 5e-3
        if quant_q:
            assert np.array_equal(st["q"][l - 1], st["p"][l])
    for k in range(4):
        prev = U.round_state(s)
        U.load_state(ctx, prev, True)
        s = _compare_iteration(ctx, prev, prm, f"{case}/m={levels}/neg={neg}/q={quant_q}/k={k}")
    # free-running: the iterates stay on the level set
    ctx.step(3)
    st = U.read_state(ctx)
    for l in range(1, s.L):
        lev = o.level_set(float(ctx.get_tensor(B.T_QSCALE, l + 1)[0]), levels, prm.level_lo)
        assert np.all(np.isin(st["p"][l], lev))
        if quant_q:
            assert np.all(np.isin(st["q"][l - 1], lev))
    assert np.all(np.isfinite(ctx.objective()))
    ctx.destroy()


@pytest.mark.parametrize("case,slope,levels,neg,step", [("er-small", 0.2, 0, 0, 0.0), ("ba-ragged", 0.05, 0, 0, 0.0),
                                                       ("c4-like", 0.3, 64, 8, 0.125)])
def test_teacher_forced_leaky_relu(case, slope, levels, neg, step):
    """f_l = leaky ReLU (the other activation the paper names): z-update by its own closed form, q, u, the
    objective's activation term and the forward pass all use it."""
    inp = _inputs(case, quant_levels=levels)
    prm, s, _ = U.oracle_problem(inp, neg_levels=neg, step=step, slope=slope)
    ctx = B.from_inputs(inp, quant_neg_levels=neg, quant_step=step, leaky_slope=slope)
    st = U.read_state(ctx)
    if not levels:
        for l in range(s.L - 1):
            assert U.rel_err(st["q"][l], s.q[l]) < 1e-5 and st["q"][l].min() < 0
    for k in range(4):
        prev = U.round_state(s)
        U.load_state(ctx, prev, levels > 0)
        s = _compare_iteration(ctx, prev, prm, f"{case}/slope={slope}/k={k}")
    got, want = ctx.objective(), o.objective(s, prm)
    assert abs(got[2] - want[2]) <= 1e-3 * abs(want[2]) + 1e-12 and abs(got[5] - want[5]) <= 1e-3 * abs(want[5])
    logits, pred, _ = ctx.predict()
    want_logits = o.forward(s.p[0], [U.f32(w) for w in ctx_weights(ctx)[0]], [U.f32(b) for b in ctx_weights(ctx)[1]], slope)
    assert U.rel_err(logits.T.astype(np.float64), want_logits) < TOL
    ctx.destroy()


@pytest.mark.parametrize("case,levels", [("er-small", 0), ("ba-ragged", 0), ("c4-like", 64)])
def test_teacher_forced_least_squares_risk(case, levels):
    """R = least squares (PDADMM_FLAG_LEAST_SQUARES): the last layer's z-update is its closed form and the
    objective's first component is that risk; everything else is unchanged."""
    inp = _inputs(case, quant_levels=levels)
    prm, s, _ = U.oracle_problem(inp, risk="ls")
    ctx = B.from_inputs(inp, flags=B.FLAG_LEAST_SQUARES)
    for k in range(4):
        prev = U.round_state(s)
        U.load_state(ctx, prev, levels > 0)
        s = _compare_iteration(ctx, prev, prm, f"{case}/ls/k={k}")
    got, want = ctx.objective(), o.objective(s, prm)
    assert abs(got[0] - want[0]) <= 1e-4 * abs(want[0]) and abs(got[5] - want[5]) <= 1e-3 * abs(want[5])
    assert abs(want[0] - o.risk(s.z[-1], s.y, s.mask)) > 1e-2 * abs(want[0])     # not the cross-entropy
    ctx.destroy()


@pytest.mark.parametrize("case,name,code,levels,neg,step", [("er-small", "tanh", B.ACT_TANH, 0, 0, 0.0),
                                                            ("ba-ragged", "sigmoid", B.ACT_SIGMOID, 0, 0, 0.0),
                                                            ("c4-like", "tanh", B.ACT_TANH, 64, 32, 1.0 / 32)])
def test_teacher_forced_smooth_activation_with_lookup_table(case, name, code, levels, neg, step):
    """f_l = tanh or sigmoid: the z-update takes the best candidate of a lookup table (remark after Eq. "update z"),
    q, u, the objective's activation term, the start and the forward pass use the activation itself.  z must equal the
    oracle's candidate exactly except where a neighbouring candidate ties."""
    table = (513, -6.0, 6.0)
    inp = _inputs(case, quant_levels=levels)
    prm, s, _ = U.oracle_problem(inp, neg_levels=neg, step=step, activation=name, table=table)
    ctx = B.from_inputs(inp, quant_neg_levels=neg, quant_step=step, activation=code, table=table)
    st = U.read_state(ctx)
    if not levels:
        for l in range(s.L - 1):
            assert U.rel_err(st["q"][l], s.q[l]) < 1e-5
    pts = o.table_points(*table[1:], table[0])
    for k in range(4):
        prev = U.round_state(s)
        U.load_state(ctx, prev, levels > 0)
        s = _compare_iteration(ctx, prev, prm, f"{case}/{name}/k={k}")
        got = U.read_state(ctx)
        for l in range(s.L - 1):
            assert np.all(np.isin(got["z"][l], pts)), "z left the table"
            tie = U.z_table_tie_mask(prev, s, prm, l)
            assert np.array_equal(got["z"][l][~tie], s.z[l][~tie])
    got, want = ctx.objective(), o.objective(s, prm)
    assert abs(got[2] - want[2]) <= 1e-3 * abs(want[2]) + 1e-12 and abs(got[5] - want[5]) <= 1e-3 * abs(want[5])
    logits, pred, _ = ctx.predict()
    Ws, bs = ctx_weights(ctx)
    want_logits = o.forward(s.p[0], [U.f32(w) for w in Ws], [U.f32(b) for b in bs], prm.f)
    assert U.rel_err(logits.T.astype(np.float64), want_logits) < TOL
    ctx.destroy()


def ctx_weights(ctx):
    L = ctx.n_layers
    return ([ctx.get_tensor(B.T_W, l).astype(np.float64) for l in range(1, L + 1)],
            [ctx.get_tensor(B.T_B, l).astype(np.float64) for l in range(1, L + 1)])


@pytest.mark.parametrize("rho,nu", [(1.0, 0.01), (0.05, 0.5)])
def test_teacher_forced_other_penalties(rho, nu):
    inp = _inputs("er-small", quant_levels=0)
    prm, s, _ = U.oracle_problem(inp, rho=rho, nu=nu)
    ctx = B.from_inputs(inp, rho=rho, nu=nu)
    for k in range(4):
        prev = U.round_state(s)
        U.load_state(ctx, prev, False)
        s = _compare_iteration(ctx, prev, prm, f"rho={rho}/k={k}")
    ctx.destroy()


# ----------------------------------------------------------------------------- free-running trajectories

# Free-running pdADMM-G-Q: the projection is a discrete decision.  Where p - g/tau lies within single-precision
# rounding of a boundary between two levels the device and the fp64 oracle may round to different neighbours;
# both are nearest levels of their own value.  Each such flip moves one entry by a whole level and the two
# trajectories then separate slowly, so the free-running comparison is looser for -Q (1e-2), while the
# teacher-forced tests above hold every single iteration to 1e-4.
@pytest.mark.parametrize("case,levels,tol", [("er-small", 0, 1e-3), ("ba-ragged", 0, 1e-3), ("c4-like", 0, 1e-3),
                                             ("ba-ragged", 256, 1e-2), ("er-small", 16, 1e-2)])
def test_objective_after_20_free_iterations(case, levels, tol):
    inp = _inputs(case, quant_levels=levels)
    prm, s, _ = U.oracle_problem(inp)
    ctx = B.from_inputs(inp)
    for _ in range(20):
        s = o.iterate(s, prm)
    ctx.step(20)
    want, got = o.objective(s, prm), ctx.objective()
    assert abs(got[5] - want[5]) <= tol * abs(want[5]), (got, want)
    res_g, res_o = ctx.residuals(), o.residuals_sq(s)
    assert np.allclose(res_g, res_o, rtol=30 * tol, atol=1e-6 * max(res_o.max(), 1e-30))
    # Lemma q_opt on the device state: u = nu (q - ReLU(z)) (holds for p-only quantisation too)
    st = U.read_state(ctx)
    for l in range(s.L - 1):
        lhs, rhs = st["u"][l], prm.nu * (st["q"][l] - np.maximum(st["z"][l], 0))
        assert np.linalg.norm(lhs - rhs) <= 1e-4 * max(np.linalg.norm(lhs), 1e-12)
    if levels:
        for l in range(2, s.L + 1):
            codes, p = ctx.get_tensor(B.T_CODES, l), ctx.get_tensor(B.T_P, l)
            assert np.array_equal(p, codes.astype(np.float32) * ctx.get_tensor(B.T_QSCALE, l)[0])
    ctx.destroy()


def test_graph_replay_equals_direct_launches():
    inp = _inputs("ba-ragged", quant_levels=0)
    a, b = B.from_inputs(inp), B.from_inputs(inp, flags=B.FLAG_NO_GRAPH)
    a.step(5)
    b.step(5)
    assert a.launches() == b.launches() > 0
    sa, sb = U.read_state(a), U.read_state(b)
    for k in sa:
        for x, y in zip(sa[k], sb[k]):
            assert np.array_equal(x, y), k
    a.destroy()
    b.destroy()


def test_step_is_deterministic_and_split_calls_agree():
    inp = _inputs("ba-ragged", quant_levels=0)
    a, b = B.from_inputs(inp), B.from_inputs(inp)
    a.step(6)
    for _ in range(3):
        b.step(2)
    sa, sb = U.read_state(a), U.read_state(b)
    for k in sa:
        for x, y in zip(sa[k], sb[k]):
            assert np.array_equal(x, y), k                      # fixed-order reductions: bit-identical runs
    a.destroy()
    b.destroy()


# ----------------------------------------------------------------------------- the trained model: forward pass, classes

@pytest.mark.parametrize("case,levels,flags", [("er-small", 0, 0), ("ba-ragged", 0, 0), ("c4-like", 256, 0),
                                               ("ba-ragged", 0, B.FLAG_SIMT_GEMM)])
def test_prediction_matches_the_oracle_forward_pass(case, levels, flags):
    inp = _inputs(case, quant_levels=levels)
    prm, s, _ = U.oracle_problem(inp)
    ctx = B.from_inputs(inp, flags=flags)
    mask = inp.train_mask.astype(bool)
    for k in range(3):
        if k:                                   # weights after some iterations, carried over from the oracle
            for _ in range(2):
                s = o.iterate(s, prm)
            U.load_state(ctx, U.round_state(s), levels > 0)
        Wf = [U.f32(w) for w in s.W]
        bf = [U.f32(b) for b in s.b]
        want = o.forward(s.p[0], Wf, bf)
        logits, pred, counts = ctx.predict()
        assert U.rel_err(logits.T.astype(np.float64), want) < TOL
        # classes: equal wherever the two largest logits are further apart than the tolerance allows them to move
        srt = np.sort(want, axis=0)
        clear = (srt[-1] - srt[-2]) > 4 * TOL * np.abs(want).max()
        want_pred = np.argmax(want, axis=0)
        assert clear.mean() > 0.9
        assert np.array_equal(pred[clear], want_pred[clear])
        assert np.array_equal(pred, np.argmax(logits, axis=1))          # the device's own logits decide, first one wins
        hit = pred == inp.labels
        assert counts.tolist() == [int(hit[mask].sum()), int(mask.sum()), int(hit[~mask].sum()), int((~mask).sum())]
        assert abs(counts[0] / counts[1] - o.accuracy(want_pred, inp.labels, mask)) <= (~clear).mean() + 1e-12
    # the state of the iteration is untouched: one more step gives what it gives without the call in between
    ref = B.from_inputs(inp, flags=flags)
    U.load_state(ref, U.round_state(s), levels > 0)
    ref.step(1)
    ctx.step(1)
    a, b = U.read_state(ctx), U.read_state(ref)
    for name in ("p", "W", "b", "z", "q", "u"):
        for x, y in zip(a[name], b[name]):
            assert np.array_equal(x, y)
    ctx.destroy()
    ref.destroy()


@pytest.mark.parametrize("levels", [0, 16])
def test_gradient_constant_kept_by_the_q_u_kernel_equals_the_recomputed_one(levels):
    """t_l = u_{l-1} + rho (p_l - q_{l-1}) is written by the kernel that updates q and u and recomputed from the stored
    iterates after the caller sets a tensor: both routes give the same bits, iteration after iteration."""
    inp = _inputs("ba-ragged", quant_levels=levels)
    a = B.from_inputs(inp)
    b = B.from_inputs(inp)
    for k in range(4):
        a.step(1)
        b.set_tensor(B.T_U, 1, b.get_tensor(B.T_U, 1))          # same values: only forces the recomputation
        b.step(1)
        sa, sb = U.read_state(a), U.read_state(b)
        for name in ("p", "W", "b", "z", "q", "u"):
            for x, y in zip(sa[name], sb[name]):
                assert np.array_equal(x, y), f"{name} differs at iteration {k}"
    a.destroy()
    b.destroy()
