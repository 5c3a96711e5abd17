"""Pins of the oracle's node-sharded iteration: it is the same iteration."""

import numpy as np
import pytest

import oracle.pdadmm_oracle as o
from paper_2105_09837_b200 import synth


def _problem(m=0, n=210, L=4, **kw):
    w = synth.small("c2", n, feat_dim=9, hidden=13, n_layers=L, quant_levels=m)
    inp = synth.make_inputs(w)
    prm = o.Params(0.5, 0.02, m, **kw)
    A = o.renormalized_adjacency(w.n_nodes, inp.edge_src, inp.edge_dst)
    X = o.augment(inp.features.T.astype(np.float64), A, w.n_blocks)
    s = o.init_state(X, [x.astype(np.float64) for x in inp.init_W], inp.labels, inp.train_mask, prm)
    return s, prm


def _assert_same_state(t, got, tol):
    """Equal up to the order of additions; b is a mean of residuals that may itself be at rounding level, so it is
    measured against the size of the terms that are averaged (the entries of z)."""
    for name in ("p", "W", "b", "z", "q", "u"):
        for l, (a, b) in enumerate(zip(getattr(t, name), getattr(got, name))):
            scale = np.linalg.norm(a)
            if name == "b":
                scale = max(scale, np.abs(t.z[l]).max() * np.sqrt(a.size))
            if name == "u":
                scale = max(scale, np.linalg.norm(t.q[l]) * 1e-3)
            assert np.linalg.norm(a - b) <= tol * max(scale, 1e-30), (name, l)


def _assert_same_steps(prev, t, got, tol):
    """tau and theta are ratios of norms of a gradient; while a layer's gradient is itself at rounding level (the
    start is feasible, the risk's pull reaches layer l only after L - l iterations) the ratio is noise, so they are
    compared where the step they scale is a real one."""
    for l in range(t.L):
        if l >= 1 and np.linalg.norm(t.p[l] - prev.p[l]) > 1e-6 * np.linalg.norm(prev.p[l]):
            assert abs(got.tau[l] - t.tau[l]) <= tol * t.tau[l], ("tau", l)
        if np.linalg.norm(t.W[l] - prev.W[l]) > 1e-6 * np.linalg.norm(prev.W[l]):
            assert abs(got.theta[l] - t.theta[l]) <= tol * t.theta[l], ("theta", l)
    assert got.trials == t.trials


def test_split_shard_merge_round_trip():
    s, prm = _problem()
    parts = o.split_nodes(210, 4)
    assert [p.start for p in parts] == [0, 52, 105, 157] and parts[-1].stop == 210
    sh = o.shard_state(s, parts)
    assert sum(x.p[0].shape[1] for x in sh) == 210
    back = o.merge_shards(sh)
    for name in ("p", "W", "b", "z", "q", "u"):
        for a, b in zip(getattr(s, name), getattr(back, name)):
            assert np.array_equal(a, b)
    assert np.array_equal(back.y, s.y) and np.array_equal(back.mask, s.mask)


@pytest.mark.parametrize("m,kw", [(0, {}), (16, {}), (16, dict(quantize_q=True)), (0, dict(slope=0.2)), (0, dict(risk="ls"))])
def test_one_shard_is_the_plain_iteration(m, kw):
    s, prm = _problem(m, **kw)
    t = s
    sh = o.shard_state(s, o.split_nodes(210, 1))
    for _ in range(4):
        prev = t
        t = o.iterate(t, prm)
        sh = o.iterate_sharded(sh, prm)
    _assert_same_state(t, sh[0], 1e-12)           # the library products may round differently for another memory layout
    _assert_same_steps(prev, t, sh[0], 1e-9)


@pytest.mark.parametrize("m", [0, 16])
@pytest.mark.parametrize("R", [2, 3, 7])
def test_sharded_iterations_equal_the_plain_ones_up_to_summation_order(m, R):
    s, prm = _problem(m)
    t = s
    sh = o.shard_state(s, o.split_nodes(210, R))
    for _ in range(5):
        prev = t
        t = o.iterate(t, prm)
        sh = o.iterate_sharded(sh, prm)
        # the shared variables stay identical on all shards
        for x in sh[1:]:
            for l in range(t.L):
                assert np.array_equal(x.W[l], sh[0].W[l]) and np.array_equal(x.b[l], sh[0].b[l])
    got = o.merge_shards(sh)
    _assert_same_state(t, got, 1e-10)
    _assert_same_steps(prev, t, got, 1e-8)
    assert np.allclose(o.objective_sharded(sh, prm), o.objective(t, prm), rtol=1e-10, atol=1e-12)


def test_a_sum_left_unreduced_is_caught():
    """A shard that uses its own part of a sum over nodes instead of the total follows another trajectory."""
    s, prm = _problem(0)
    s = o.iterate(o.iterate(s, prm), prm)                         # leave the feasible start, where every gradient is zero
    ref = o.iterate(s, prm)
    sh = o.shard_state(s, o.split_nodes(210, 2))
    alone = [o.iterate_sharded([x], prm)[0] for x in sh]          # each shard as if it were the whole graph
    last = ref.L - 1                                              # the layer that moves in the very first iteration
    assert np.linalg.norm(alone[0].W[last] - ref.W[last]) > 1e-6 * np.linalg.norm(ref.W[last])
    together = o.merge_shards(o.iterate_sharded(sh, prm))
    assert np.linalg.norm(together.W[last] - ref.W[last]) <= 1e-12 * np.linalg.norm(ref.W[last])
