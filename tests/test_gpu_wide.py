"""GPU parity of whole iterations at the layer shapes of the two large workloads (their depth, width, class count and
level count, fewer nodes), of long free runs, and of the free-running quantised objective.

The wide layers take code paths that the small cases never reach inside an iteration: the W-gradient's operands are
transposed and split into planes beforehand on every layer, and the products over a partly filled last round of the
persistent grid are cut along the contraction.  Node counts are chosen so that both happen (stated per case)."""

import numpy as np
import pytest

import oracle.pdadmm_oracle as o
from paper_2105_09837_b200 import binding as B
from paper_2105_09837_b200 import synth
import parity_util as U
from test_gpu_parity import _compare_iteration

pytestmark = pytest.mark.gpu


# c4 shape: 15 layers x 1000, 640 inputs, 40 classes, 256 levels.  4800 nodes = 38 row tiles (the last one ragged):
#   hidden products 38 x 8 = 304 tiles = 2 rounds of 148 + 8, each of the 8 cut into 2 contraction slices; the last
#   layer's 38 tiles are cut into 2 slices as well; W-gradient 8 x 8 (layer 1: 8 x 5) output tiles: planes beforehand.
# c5 shape: 30 layers x 2000, 2000 inputs, 7 classes, 16 levels.  1300 nodes = 11 row tiles: 176 tiles = 148 + 28,
#   the 28 cut into 4 slices; W-gradient 16 x 16 output tiles: planes beforehand.
@pytest.mark.parametrize("name,n_nodes,levels", [("c4", 4800, 256), ("c5", 1300, 16), ("c4", 4800, 0)])
def test_teacher_forced_iterations_at_the_shapes_of_the_large_workloads(name, n_nodes, levels):
    w = synth.small(name, n_nodes, quant_levels=levels)
    full = synth.get(name)
    assert (w.n_layers, w.hidden, w.n_classes, w.feat_dim, w.n_hops) == \
        (full.n_layers, full.hidden, full.n_classes, full.feat_dim, full.n_hops)
    inp = synth.make_inputs(w)
    prm, s, _ = U.oracle_problem(inp)
    ctx = B.from_inputs(inp)
    for k in range(2):
        prev = U.round_state(s)
        U.load_state(ctx, prev, levels > 0)
        rep = {}
        s = _compare_iteration(ctx, prev, prm, f"{name}-shape/N={n_nodes}/m={levels}/k={k}", report=rep, single_bounds=True)
    # the trajectory continues on the device alone: state stays valid
    ctx.step(2)
    assert np.all(np.isfinite(ctx.objective()))
    ctx.destroy()


def test_a_jump_in_the_size_of_the_gradient_between_iterations_is_handled():
    """Wide quantised layers: the epilogue that writes g also writes its fp16 plane for the norm-only product W g, scaled
    by an exponent predicted from the previous iteration's max|g|; a kernel then checks the prediction and redoes the
    plane if it does not fit.  Here the dual variable is scaled by 1e4 and back between teacher-forced iterations, so
    that max|g| jumps by four orders of magnitude each way (too large: the predicted scaling would overflow fp16; too
    small: it would leave no significant bits).  That product only decides the tau at which the search of Eq. "update p
    quantized" starts, tau = rho + nu ||W g||^2 / ||g||^2: it must agree with the oracle's in every one of these
    iterations (the scaled states are far from anything the method produces, so nothing else is compared here)."""
    import dataclasses
    w = synth.small("c4", 2400, quant_levels=256)          # 1000-wide layers: 8 column tiles, the copy is in use
    inp = synth.make_inputs(w)
    prm, s, _ = U.oracle_problem(inp)
    ctx = B.from_inputs(inp)
    for k, factor in enumerate([1.0, 1.0, 1e4, 1e-4, 1.0]):
        scaled = dataclasses.replace(s, u=[x * factor for x in s.u])
        prev = U.round_state(scaled)
        U.load_state(ctx, prev, True)
        nxt = o.iterate(prev, prm)
        ctx.step(1)
        for l in range(1, prev.L):
            tau_dev = float(ctx.get_tensor(B.T_TAU, l + 1)[0])
            trials_dev = int(ctx.get_tensor(B.T_TRIALS, l + 1)[0])
            start_dev, start_want = tau_dev / 2.0 ** (trials_dev - 1), nxt.tau[l] / 2.0 ** (nxt.trials[l] - 1)
            assert abs(start_dev - start_want) <= 1e-5 * start_want, (k, factor, l + 1, start_dev, start_want)
        s = nxt
    ctx.destroy()


@pytest.mark.parametrize("flags", [0, B.FLAG_SIMT_GEMM])
def test_cached_linear_residual_does_not_drift_over_200_free_iterations(flags):
    """The library carries r = W p + b - z from step to step instead of recomputing it.  After 200 free iterations the
    carried r is compared (a) with W p + b - z recomputed on the host in double precision from the device's own p, W,
    b, z, through the linear term of the objective, and (b) with a twin context that is forced to rebuild r from its
    definition (re-setting W to the values just read): the objective's linear term and the next iteration's z, W, p of
    the two agree within 1e-4."""
    inp = synth.make_inputs(synth.small("c2", 1500, feat_dim=30, hidden=120, n_layers=6, quant_levels=0))
    w = inp.workload
    ctx = B.from_inputs(inp, flags=flags)
    ctx.step(200)
    st = U.read_state(ctx)
    lin = sum(float(np.sum((st["z"][l] - st["W"][l] @ st["p"][l] - st["b"][l][:, None]) ** 2)) for l in range(w.n_layers))
    dev = ctx.objective()
    # r is a difference of terms of the size of W p: each term's single-precision rounding is the floor of what any
    # single-precision r can resolve; the comparison is against that floor or 1e-4, whichever is larger
    floor = sum(float(np.sum((2.0 ** -23 * (np.abs(st["z"][l]) + np.abs(st["W"][l] @ st["p"][l]))) ** 2)) for l in range(w.n_layers))
    assert abs(dev[1] - 0.5 * w.nu * lin) <= max(1e-4 * 0.5 * w.nu * lin, 0.5 * w.nu * (2 * np.sqrt(lin * floor) + floor)), (dev[1], 0.5 * w.nu * lin)
    twin = B.from_inputs(inp, flags=flags)
    U.load_state(twin, _as_state(st, inp), False)            # every tensor re-set: r, t and the planes are rebuilt
    dev2 = twin.objective()
    assert abs(dev[1] - dev2[1]) <= 1e-4 * abs(dev2[1]) + 0.5 * w.nu * (2 * np.sqrt(lin * floor) + floor)
    assert abs(dev[5] - dev2[5]) <= 1e-6 * abs(dev2[5])
    ctx.step(1)
    twin.step(1)
    a, b = U.read_state(ctx), U.read_state(twin)
    for name in ("p", "W", "z", "q"):
        for l, (x, y) in enumerate(zip(a[name], b[name])):
            if name == "p" and l == 0:
                continue
            assert U.rel_err(x, y) <= 1e-4, (name, l + 1, U.rel_err(x, y))
    ctx.destroy()
    twin.destroy()


def _as_state(st, inp):
    L = len(st["W"])
    return o.State(st["p"], st["W"], st["b"], st["z"], st["q"], st["u"], inp.labels, inp.train_mask.astype(bool), [1.0] * L)


def test_long_free_run_matches_the_oracle_variable_by_variable():
    """40 free iterations of pdADMM-G: no discrete decision except the ReLU branch, so the two trajectories stay
    together; every variable is compared at the end (1e-3: forty iterations of single-precision rounding)."""
    inp = synth.make_inputs(synth.small("c2", 900, feat_dim=20, hidden=70, n_layers=4, quant_levels=0))
    prm, s, _ = U.oracle_problem(inp)
    ctx = B.from_inputs(inp)
    ctx.step(40)
    for _ in range(40):
        s = o.iterate(s, prm)
    got = U.read_state(ctx)
    for name in ("p", "W", "z", "q"):
        for l in range(len(got[name])):
            want = getattr(s, name)[l]
            assert U.rel_err(got[name][l], want) <= 1e-3, (name, l + 1, U.rel_err(got[name][l], want))
    want, have = o.objective(s, prm), ctx.objective()
    assert abs(have[5] - want[5]) <= 1e-4 * abs(want[5])
    ctx.destroy()


@pytest.mark.parametrize("case,levels", [("ba-ragged", 256), ("er-small", 16), ("c4-like", 256)])
def test_free_running_quantised_objective_differs_by_boundary_flips_only(case, levels):
    """20 free iterations of pdADMM-G-Q.  The projection is a discrete decision: where p - g/tau lies within
    single-precision rounding of the boundary between two levels, the device and the oracle may take different
    neighbours, after which the trajectories separate slowly.  Here the oracle replays the device's choice at exactly
    those elements (both neighbours are nearest levels of a value within the rounding bound) and nowhere else; the
    objective then agrees within 1e-3 after 20 iterations, and the number of replayed elements is tiny."""
    from test_gpu_parity import _inputs
    import error_bounds as EB
    inp = _inputs(case, quant_levels=levels)
    prm, s, _ = U.oracle_problem(inp)
    ctx = B.from_inputs(inp)
    replayed, total = 0, 0
    for k in range(20):
        ctx.step(1)
        nxt = o.iterate(s, prm)
        bd = EB.iteration_bounds(U.round_state(s), nxt, prm)
        changed = False
        for l in range(1, s.L):
            codes = ctx.get_tensor(B.T_CODES, l + 1).T.astype(np.int64)
            mine = np.rint((nxt.p[l] - prm.level_lo) / s.scale[l]).astype(np.int64)
            # the oracle state carries forty-odd roundings of earlier device iterations as well: the band is the
            # bound of this iteration's computation plus the distance of the two states' inputs, taken from p itself
            near = U.boundary_mask(s, nxt, prm, l, tol=np.maximum(bd["x"][l] / s.scale[l], 1e-3))
            flip = (codes != mine) & near & (np.abs(codes - mine) == 1)
            total += codes.size
            if flip.any():
                lev = o.level_set(s.scale[l], prm.quant_levels, prm.level_lo)
                nxt.p[l] = np.where(flip, lev[np.clip(codes, 0, levels - 1)], nxt.p[l])
                replayed += int(flip.sum())
                changed = True
        if changed:
            nxt = U.redo_after_p(s, nxt, prm)
        s = nxt
    want, got = o.objective(s, prm), ctx.objective()
    assert replayed <= 2e-3 * total, (replayed, total)
    assert abs(got[5] - want[5]) <= 1e-3 * abs(want[5]), (got, want, replayed)
    ctx.destroy()
