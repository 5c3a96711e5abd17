"""Pins of the oracle's layer-wise growth (greedy training schedule)."""

import numpy as np
import pytest

import oracle.pdadmm_oracle as o
from paper_2105_09837_b200 import synth


def _stage(n_layers, m=0, n=160):
    w = synth.small("c2", n, feat_dim=7, hidden=12, n_layers=n_layers, quant_levels=m)
    inp = synth.make_inputs(w)
    A = o.renormalized_adjacency(w.n_nodes, inp.edge_src, inp.edge_dst)
    X = o.augment(inp.features.T.astype(np.float64), A, w.n_blocks)
    return w, inp, X


@pytest.mark.parametrize("m", [0, 16])
def test_growth_keeps_the_trained_layers_and_starts_the_new_ones_feasibly(m):
    w2, inp2, X = _stage(2, m)
    w5, inp5, _ = _stage(5, m)
    prm = o.Params(0.5, 0.02, m)
    s = o.init_state(X, [x.astype(np.float64) for x in inp2.init_W], inp2.labels, inp2.train_mask, prm)
    for _ in range(6):
        s = o.iterate(s, prm)
    W_new = [x.astype(np.float64) for x in inp5.init_W[1:]]            # layers 2..5 of the deeper model
    g = o.grow(s, prm, W_new)
    assert g.L == 5 and len(g.q) == 4 and len(g.u) == 4 and len(g.p) == 5
    # layer 1 is untouched, including the input of the old output layer
    for name in ("W", "b", "z", "q", "u"):
        assert np.array_equal(getattr(g, name)[0], getattr(s, name)[0])
    assert np.array_equal(g.p[0], s.p[0]) and np.array_equal(g.p[1], s.p[1])
    assert g.scale[1] == s.scale[1]
    # the new layers: the forward pass of the model so far, written out here step by step
    p = s.p[1]
    for l in range(1, 5):
        assert np.array_equal(g.W[l], W_new[l - 1]) and np.all(g.b[l] == 0)
        z = W_new[l - 1] @ p
        assert np.array_equal(g.z[l], z)
        if l < 4:
            q = np.maximum(z, 0)
            assert np.array_equal(g.q[l], q) and np.all(g.u[l] == 0)
            if m:
                lev = o.level_set(g.scale[l + 1], m)
                assert np.all(np.isin(g.p[l + 1], lev)) and np.max(np.abs(g.p[l + 1] - q)) <= g.scale[l + 1] / 2 * (1 + 1e-6)
                assert g.scale[l + 1] == o.quantization_scale(q, m)
            else:
                assert np.array_equal(g.p[l + 1], q)
            p = g.p[l + 1]
    # the residuals of the new boundaries vanish (pdADMM-G), the old one keeps its value
    res = o.residuals_sq(g)
    assert res[0] == o.residuals_sq(s)[0]
    if not m:
        assert np.all(res[1:] == 0)
    # and the grown model trains on: finite, and the kept layer keeps moving
    for _ in range(3):
        g = o.iterate(g, prm)
    assert np.isfinite(o.lagrangian(g, prm))


def test_growing_twice_reaches_the_full_depth():
    prm = o.Params(1.0, 0.01, 0)
    w2, inp2, X = _stage(2)
    w4, inp4, _ = _stage(4)
    w7, inp7, _ = _stage(7)
    s = o.init_state(X, [x.astype(np.float64) for x in inp2.init_W], inp2.labels, inp2.train_mask, prm)
    for _ in range(3):
        s = o.iterate(s, prm)
    s = o.grow(s, prm, [x.astype(np.float64) for x in inp4.init_W[1:]])
    for _ in range(3):
        s = o.iterate(s, prm)
    W3_trained = s.W[2].copy()
    s = o.grow(s, prm, [x.astype(np.float64) for x in inp7.init_W[3:]])
    assert s.L == 7 and np.array_equal(s.W[2], W3_trained)
    assert [w.shape[0] for w in s.W] == [12] * 6 + [w7.n_classes]
    before = o.lagrangian(s, prm)
    for _ in range(4):
        s = o.iterate(s, prm)
    assert o.lagrangian(s, prm) <= before + 1e-9 * abs(before)          # rho = 1, nu = 0.01: the decrease lemma's regime


def test_start_layers_from_the_first_layer_is_the_initial_state():
    w, inp, X = _stage(4, 16)
    prm = o.Params(0.5, 0.02, 16)
    s = o.init_state(X, [x.astype(np.float64) for x in inp.init_W], inp.labels, inp.train_mask, prm)
    t = o.iterate(s, prm)
    r = o.start_layers_from(t, prm, 1)                 # forgets the iteration except for W (which moved)
    ref = o.init_state(X, t.W, inp.labels, inp.train_mask, prm)
    for name in ("p", "z", "q", "u", "b"):
        for a, b in zip(getattr(r, name), getattr(ref, name)):
            assert np.array_equal(a, b), name
    assert r.scale == ref.scale
