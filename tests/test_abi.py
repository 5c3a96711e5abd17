"""CPU checks of the C-ABI library: it builds, loads, exports every declared symbol, and fails loudly without a GPU."""

import ctypes
import os
import re

import numpy as np
import pytest

from paper_2105_09837_b200 import binding as B
from paper_2105_09837_b200 import build as build_mod
from paper_2105_09837_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "pdadmm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pdadmm_[a-z_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build_mod.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    names = _declared()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(B.EXPORTS) == names          # the Python binding covers the same entry points


def test_no_device_means_an_error_not_a_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    inp = synth.make_inputs(synth.small("c1", 50, feat_dim=4, hidden=5, n_layers=2))
    with pytest.raises(B.PdadmmError) as e:
        B.from_inputs(inp)
    assert e.value.code == B.ECUDA


def test_argument_checks_need_no_device():
    inp = synth.make_inputs(synth.small("c1", 50, feat_dim=4, hidden=5, n_layers=2))
    w = inp.workload
    bad = np.array(inp.labels)
    bad[3] = 99
    with pytest.raises(B.PdadmmError) as e:
        B.Context(w.n_nodes, inp.edge_src, inp.edge_dst, inp.features, w.n_hops, w.n_classes, bad, inp.train_mask,
                  w.widths, 1e-3, 1e-3, 0, inp.init_W)
    assert e.value.code == B.EINVAL and "label" in str(e.value)
    with pytest.raises(B.PdadmmError) as e:
        B.Context(w.n_nodes, inp.edge_src, inp.edge_dst, inp.features, w.n_hops, w.n_classes, inp.labels,
                  inp.train_mask, w.widths, -1.0, 1e-3, 0, inp.init_W)
    assert e.value.code == B.EINVAL
    with pytest.raises(B.PdadmmError) as e:
        B.Context(w.n_nodes, inp.edge_src, inp.edge_dst, inp.features, w.n_hops, w.n_classes, inp.labels,
                  inp.train_mask, w.widths, 1e-3, 1e-3, 70000, inp.init_W)
    assert e.value.code == B.EINVAL
    with pytest.raises(B.PdadmmError):
        B.quantize(np.zeros(4, np.float32), 0.0, 16)
    with pytest.raises(B.PdadmmError):
        B.spmm([0, 2], [0, 5], [1.0, 1.0], np.zeros((1, 4), np.float32))      # column out of range
    assert B.lib().pdadmm_destroy(None) == 0
