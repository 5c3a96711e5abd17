"""GPU parity at the full sizes of the five workloads, in the launch configuration bench.py times.

c1, c2, c3: the oracle can afford whole iterations, so one teacher-forced iteration (after two oracle
iterations, when every layer has started to move) is compared variable by variable, and c1 also runs its
20 free iterations.  c4, c5: the oracle cannot afford an iteration (1e13..1e14 flop in fp64, >200 GB), so the
parts it can compute are compared (the whole augmented input, the forward pass on sampled nodes) and the state
after two device iterations is checked against properties that hold at any size (Lemma "q_opt", p on the level
set, finite and decreasing objective).
"""

import numpy as np
import pytest

import oracle.pdadmm_oracle as o
from paper_2105_09837_b200 import binding as B
from paper_2105_09837_b200 import synth
import parity_util as U
from test_gpu_parity import _compare_iteration

pytestmark = pytest.mark.gpu


def test_c1_full_teacher_forced_and_20_free_iterations():
    inp = synth.make_inputs(synth.get("c1"))
    prm, s, _ = U.oracle_problem(inp)
    ctx = B.from_inputs(inp)
    free = B.from_inputs(inp)
    free.step(20)
    for k in range(20):
        if k in (2, 7, 15):
            prev = U.round_state(s)
            U.load_state(ctx, prev, False)
            _compare_iteration(ctx, prev, prm, f"c1/k={k}")
        s = o.iterate(s, prm)
    want, got = o.objective(s, prm), free.objective()
    assert abs(got[5] - want[5]) <= 1e-3 * abs(want[5]), (got, want)
    ctx.destroy()
    free.destroy()


@pytest.mark.parametrize("name", ["c2", "c3"])
def test_c2_c3_full_one_teacher_forced_iteration(name):
    inp = synth.make_inputs(synth.get(name))
    prm, s, A = U.oracle_problem(inp)
    ctx = B.from_inputs(inp)
    X = ctx.get_tensor(B.T_X).T.astype(np.float64)
    assert U.rel_err(X, s.p[0]) < 1e-6
    del X
    for _ in range(2):
        s = o.iterate(s, prm)
    prev = U.round_state(s)
    del s
    U.load_state(ctx, prev, prm.quant_levels > 0)
    _compare_iteration(ctx, prev, prm, f"{name}/k=2")
    ctx.destroy()


@pytest.mark.parametrize("name", ["c4", "c5"])
def test_c4_c5_full_size_parts_and_invariants(name):
    w = synth.get(name)
    inp = synth.make_inputs(w)
    ctx = B.from_inputs(inp)
    # the whole augmented input against the oracle (sparse products are cheap for it)
    A = o.renormalized_adjacency(w.n_nodes, inp.edge_src, inp.edge_dst)
    assert np.array_equal(ctx.get_tensor(B.T_CSR_ROWPTR), A.indptr.astype(np.int32))
    assert np.array_equal(ctx.get_tensor(B.T_CSR_COLIDX), A.indices.astype(np.int32))
    X = o.augment(inp.features.T.astype(np.float64), A, w.n_blocks)
    Xg = ctx.get_tensor(B.T_X)
    assert U.rel_err(Xg.T.astype(np.float64), X) < 1e-6
    # forward pass of layer 1 on sampled nodes, one by one
    rng = np.random.default_rng(7)
    nodes = rng.choice(w.n_nodes, size=64, replace=False)
    z1 = ctx.get_tensor(B.T_Z, 1)
    want = (inp.init_W[0].astype(np.float64) @ X[:, nodes]).T
    assert U.rel_err(z1[nodes].astype(np.float64), want) < 1e-5
    del X, Xg, z1
    L, m = w.n_layers, w.quant_levels
    obj0 = ctx.objective()
    ctx.step(2)
    obj2 = ctx.objective()
    assert np.all(np.isfinite(obj2)) and obj2[5] < obj0[5]
    res = ctx.residuals()
    assert res.shape == (L - 1,) and np.all(np.isfinite(res))
    for l in (1, L // 2, L - 1):
        # Lemma q_opt: u_l = nu (q_l - ReLU(z_l)) after every iteration
        u, q, z = ctx.get_tensor(B.T_U, l), ctx.get_tensor(B.T_Q, l), ctx.get_tensor(B.T_Z, l)
        rhs = np.float32(w.nu) * (q - np.maximum(z, 0))
        assert np.linalg.norm((u - rhs).ravel()) <= 1e-4 * max(np.linalg.norm(rhs.ravel()), 1e-12)
        del u, q, z, rhs
        # p on the level set, bit for bit
        codes, p = ctx.get_tensor(B.T_CODES, l + 1), ctx.get_tensor(B.T_P, l + 1)
        scale = ctx.get_tensor(B.T_QSCALE, l + 1)[0]
        assert int(codes.max()) <= m - 1
        assert np.array_equal(p, codes.astype(np.float32) * scale)
        del codes, p
        assert 1 <= int(ctx.get_tensor(B.T_TRIALS, l + 1)[0]) <= 30
    ctx.destroy()


def _rows(ctx, kind, layer, nodes):
    """Rows `nodes` of a node-major tensor as the oracle's columns (float64)."""
    return ctx.get_tensor(kind, layer)[nodes].T.astype(np.float64)


@pytest.mark.parametrize("name", ["c4", "c5"])
def test_c4_c5_full_size_node_wise_updates_on_sampled_nodes(name):
    """At full size the oracle cannot afford an iteration, but every update except the sums over nodes acts on one
    node's column at a time.  So for 48 sampled nodes the p-, z-, q- and u-updates of one device iteration are
    recomputed by the oracle's own update functions from the device's state before the iteration and the quantities
    that are sums over all nodes as the device has them afterwards (tau, W+, b+, which the reduced-size tests compare
    with the oracle).  Launch configuration: exactly what bench.py times."""
    w = synth.get(name)
    inp = synth.make_inputs(w)
    ctx = B.from_inputs(inp)
    ctx.step(2)                                      # leave the feasible start
    rng = np.random.default_rng(5)
    nodes = np.sort(rng.choice(w.n_nodes, size=48, replace=False))
    L, m, rho, nu = w.n_layers, w.quant_levels, w.rho, w.nu
    layers = sorted(set([1, 2, L // 2, L - 1, L]))
    before = {}
    for l in layers:
        before[l] = dict(p=_rows(ctx, B.T_P, l, nodes), z=_rows(ctx, B.T_Z, l, nodes),
                         W=ctx.get_tensor(B.T_W, l).astype(np.float64), b=ctx.get_tensor(B.T_B, l).astype(np.float64))
        if l < L:
            before[l].update(q=_rows(ctx, B.T_Q, l, nodes), u=_rows(ctx, B.T_U, l, nodes))
        if l >= 2:
            before[l].update(q_prev=_rows(ctx, B.T_Q, l - 1, nodes), u_prev=_rows(ctx, B.T_U, l - 1, nodes))
    ctx.step(1)
    y, mask = inp.labels[nodes], inp.train_mask[nodes].astype(bool)
    for l in layers:
        s0 = before[l]
        p_new = _rows(ctx, B.T_P, l, nodes)
        if l >= 2:
            tau = float(ctx.get_tensor(B.T_TAU, l)[0])
            scale = float(ctx.get_tensor(B.T_QSCALE, l)[0])
            g = o.grad_p_phi(s0["p"], s0["W"], s0["b"], s0["z"], nu, s0["q_prev"], s0["u_prev"], rho)
            x = s0["p"] - g / tau
            codes, want_p = o.nearest_level(x, scale, m)
            t = x / scale
            clear = np.abs(t - np.floor(t) - 0.5) > 2e-3          # away from a rounding boundary (x carries fp32 rounding)
            assert np.array_equal(p_new[clear], want_p[clear]), (name, l)
            assert np.max(np.abs(p_new - want_p)) <= scale * (1 + 1e-6) and clear.mean() > 0.99
        else:
            assert np.array_equal(p_new, s0["p"])                # p_1 = X never moves
        W1, b1 = ctx.get_tensor(B.T_W, l).astype(np.float64), ctx.get_tensor(B.T_B, l).astype(np.float64)
        a = W1 @ p_new + b1[:, None]
        z_new = _rows(ctx, B.T_Z, l, nodes)
        if l < L:
            want_z = o.update_z_hidden(a, s0["q"], s0["z"])
            zn = np.minimum((a + s0["z"]) / 2, 0.0)
            zp = np.maximum((a + s0["q"] + s0["z"]) / 3, 0.0)
            fn, fp = o.z_objective_hidden(zn, a, s0["q"], s0["z"]), o.z_objective_hidden(zp, a, s0["q"], s0["z"])
            tie = (np.abs(fp - fn) <= 1e-5 * (np.abs(fp) + np.abs(fn) + 1e-30)) & (zp != zn)
            assert U.rel_err(z_new, want_z, tie) < 1e-4, (name, l)
            p_next = _rows(ctx, B.T_P, l + 1, nodes)
            q_new, u_new = _rows(ctx, B.T_Q, l, nodes), _rows(ctx, B.T_U, l, nodes)
            want_q = o.update_q(p_next, s0["u"], z_new, rho, nu)
            assert U.rel_err(q_new, want_q) < 1e-5, (name, l)
            want_u = o.update_u(s0["u"], p_next, q_new, rho)
            assert np.linalg.norm(u_new - want_u) <= 1e-5 * max(np.linalg.norm(want_u), rho * np.linalg.norm(p_next) * 1e-2), (name, l)
        else:
            want_z = o.update_z_last(a, y, mask, nu)
            assert U.rel_err(z_new, want_z) < 1e-4, (name, l)
    ctx.destroy()


def test_c4_full_size_level_set_variant_and_prediction():
    """Workload c4 with the paper's level set {-1..20} for p and q: after two iterations both are on the set bit
    for bit, and the forward pass of the trained model agrees with the oracle on sampled nodes."""
    w = synth.get("c4")
    inp = synth.make_inputs(w)
    m, neg, step = 22, 1, 1.0
    ctx = B.from_inputs(inp, flags=B.FLAG_QUANT_Q, quant_levels=m, quant_neg_levels=neg, quant_step=step)
    ctx.step(2)
    assert np.all(np.isfinite(ctx.objective()))
    lev = o.level_set(step, m, -1.0).astype(np.float32)
    for l in (1, w.n_layers // 2, w.n_layers - 1):
        assert float(ctx.get_tensor(B.T_QSCALE, l + 1)[0]) == step
        p, q, codes = ctx.get_tensor(B.T_P, l + 1), ctx.get_tensor(B.T_Q, l), ctx.get_tensor(B.T_CODES, l + 1)
        assert np.array_equal(p, np.float32(-1.0) + codes.astype(np.float32) * np.float32(step))
        assert np.all(np.isin(q, lev))
        del p, q, codes
    logits, pred, counts = ctx.predict()
    assert counts[1] + counts[3] == w.n_nodes and counts[1] == int(inp.train_mask.sum())
    assert np.array_equal(pred, np.argmax(logits, axis=1))
    rng = np.random.default_rng(11)
    nodes = rng.choice(w.n_nodes, size=48, replace=False)
    X = ctx.get_tensor(B.T_X)[nodes].T.astype(np.float64)
    Ws = [ctx.get_tensor(B.T_W, l).astype(np.float64) for l in range(1, w.n_layers + 1)]
    bs = [ctx.get_tensor(B.T_B, l).astype(np.float64) for l in range(1, w.n_layers + 1)]
    want = o.forward(X, Ws, bs)
    assert U.rel_err(logits[nodes].T.astype(np.float64), want) < 1e-4
    ctx.destroy()
