"""GPU parity of the greedy layer-wise schedule: growing a trained context by layers, against the oracle's `grow`."""

import numpy as np
import pytest

import oracle.pdadmm_oracle as o
from paper_2105_09837_b200 import binding as B
from paper_2105_09837_b200 import greedy, synth
import parity_util as U
from test_gpu_parity import _compare_iteration

pytestmark = pytest.mark.gpu


def _inputs(depth, levels):
    return synth.make_inputs(synth.small("c2", 1000, feat_dim=20, hidden=72, n_layers=depth, quant_levels=levels))


@pytest.mark.parametrize("levels", [0, 16])
def test_growing_a_trained_context_matches_the_oracle(levels):
    inp2, inp5 = _inputs(2, levels), _inputs(5, levels)
    prm, s, _ = U.oracle_problem(inp2)
    for _ in range(4):
        s = o.iterate(s, prm)
    s = U.round_state(s)
    ctx2 = B.from_inputs(inp2)
    U.load_state(ctx2, s, levels > 0)                 # the device continues from the oracle's trained shallow model
    want = o.grow(s, prm, [x.astype(np.float64) for x in inp5.init_W[1:]])
    ctx5 = greedy.grow_context(ctx2, inp5)
    ctx2.destroy()
    got = U.read_state(ctx5)
    assert ctx5.n_layers == 5
    # kept layer: bit for bit what was loaded
    for name in ("W", "b", "z", "q", "u"):
        assert np.array_equal(got[name][0], getattr(want, name)[0]), name
    assert np.array_equal(got["p"][1], want.p[1])
    # added layers: the forward pass of the model so far
    for l in range(1, 5):
        assert np.array_equal(got["W"][l], U.f32(want.W[l])) and np.all(got["b"][l] == 0)
        assert U.rel_err(got["z"][l], want.z[l]) < 1e-5, l
        if l < 4:
            assert np.all(got["u"][l] == 0)
            if levels:
                scale = float(ctx5.get_tensor(B.T_QSCALE, l + 2)[0])
                assert scale == pytest.approx(want.scale[l + 1], rel=1e-5)
                assert np.all(np.isin(got["p"][l + 1], o.level_set(scale, levels)))
                assert np.mean(np.abs(got["p"][l + 1] - want.p[l + 1]) > 0.5 * scale) < 5e-3
            else:
                assert U.rel_err(got["q"][l], want.q[l]) < 1e-5 and np.array_equal(got["p"][l + 1], got["q"][l])
    res = ctx5.residuals()
    assert abs(res[0] - o.residuals_sq(want)[0]) <= 1e-4 * o.residuals_sq(want)[0] + 1e-12
    if not levels:
        assert np.all(res[1:] == 0)
    # and the grown context iterates like the oracle's grown state
    prm5 = o.Params(prm.rho, prm.nu, levels)
    state = want
    for k in range(3):
        prev = U.round_state(state)
        U.load_state(ctx5, prev, levels > 0)
        state = _compare_iteration(ctx5, prev, prm5, f"grown/m={levels}/k={k}")
    ctx5.destroy()


def test_greedy_schedule_two_four_six_layers_free_running():
    """The whole schedule on the device alone against the same schedule in the oracle: the objective of the deepest
    model agrees within 1e-3."""
    depths, iters = (2, 4, 6), (6, 6, 8)
    ctx = greedy.train(lambda d: _inputs(d, 0), depths, iters)
    prm, s, _ = U.oracle_problem(_inputs(2, 0))
    for _ in range(iters[0]):
        s = o.iterate(s, prm)
    for d, k in zip(depths[1:], iters[1:]):
        s = o.grow(s, prm, [x.astype(np.float64) for x in _inputs(d, 0).init_W[s.L - 1:]])
        for _ in range(k):
            s = o.iterate(s, prm)
    assert ctx.n_layers == 6 and s.L == 6
    want, got = o.objective(s, prm), ctx.objective()
    assert abs(got[5] - want[5]) <= 1e-3 * abs(want[5]), (got, want)
    st = U.read_state(ctx)
    for l in range(6):
        assert U.rel_err(st["W"][l], s.W[l]) < 1e-3
    ctx.destroy()
    with pytest.raises(ValueError):
        greedy.train(lambda d: _inputs(d, 0), (4, 2), (1, 1))
