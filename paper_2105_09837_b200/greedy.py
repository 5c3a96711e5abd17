"""Greedy layer-wise training (paper, end of Section "The pdADMM-G Algorithm" and Section "Performance": a two-layer
GA-MLP first, then five layers, then all ten): a driver around the C-ABI calls, no arithmetic of its own.

Growing keeps the hidden layers of the trained model with their whole state, drops its output layer (its width is the
number of classes), and starts the added layers, the last of which is the new output layer, from the forward pass of
the model trained so far (``pdadmm_start_layers_from``).
"""

from __future__ import annotations

from typing import Callable, List, Sequence

import numpy as np

from . import binding as B


def grow_context(old: B.Context, new_inputs, **ctx_kwargs) -> B.Context:
    """A context for `new_inputs` (same graph, features, labels; more layers; its init_W supply the weights of the
    added layers) that continues the training of `old`: layers 1..L_old-1 are copied over, the rest start from the
    forward pass.  `old` is left untouched; the caller destroys it."""
    w = new_inputs.workload
    keep = old.n_layers - 1
    if w.n_layers <= keep:
        raise ValueError("the grown model must be deeper than the kept layers")
    if old.widths[:keep] != list(w.widths[:keep]):
        raise ValueError("the kept hidden layers must have the same widths in the grown model")
    new = B.from_inputs(new_inputs, **ctx_kwargs)
    quantised = new.quant_levels > 0
    for l in range(1, keep + 1):
        new.set_tensor(B.T_W, l, old.get_tensor(B.T_W, l))
        new.set_tensor(B.T_B, l, old.get_tensor(B.T_B, l))
        new.set_tensor(B.T_Z, l, old.get_tensor(B.T_Z, l))
        new.set_tensor(B.T_Q, l, old.get_tensor(B.T_Q, l))
        new.set_tensor(B.T_U, l, old.get_tensor(B.T_U, l))
        # p_{l+1}: the input of the next layer (for l = keep: of the first added layer), on its level set in -Q
        if quantised:
            new.set_tensor(B.T_QSCALE, l + 1, old.get_tensor(B.T_QSCALE, l + 1))
        new.set_tensor(B.T_P, l + 1, old.get_tensor(B.T_P, l + 1))
    new.start_layers_from(keep + 1)
    return new


def train(inputs_for_depth: Callable[[int], object], depths: Sequence[int], iterations: Sequence[int],
          **ctx_kwargs) -> B.Context:
    """Trains models of increasing depth, e.g. depths (2, 5, 10): `iterations[i]` iterations at depth `depths[i]`.
    `inputs_for_depth(L)` returns the inputs bundle of the L-layer model (same graph and features every time).
    Returns the context of the deepest model."""
    if len(depths) != len(iterations) or not depths or any(b <= a for a, b in zip(depths, depths[1:])):
        raise ValueError("depths must increase and come with one iteration count each")
    ctx = B.from_inputs(inputs_for_depth(depths[0]), **ctx_kwargs)
    ctx.step(iterations[0])
    for depth, n_iter in zip(depths[1:], iterations[1:]):
        grown = grow_context(ctx, inputs_for_depth(depth), **ctx_kwargs)
        ctx.destroy()
        ctx = grown
        ctx.step(n_iter)
    return ctx
