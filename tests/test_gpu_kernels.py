"""GPU tests of single kernels and of edge cases, through the C ABI."""

import numpy as np
import pytest
import scipy.sparse as sp

import oracle.pdadmm_oracle as o
from paper_2105_09837_b200 import binding as B
from paper_2105_09837_b200 import synth
import parity_util as U

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("m,scale", [(2, 0.75), (16, 0.0173), (256, 0.011764706)])
def test_quantise_kernel_is_bit_exact(m, scale):
    rng = np.random.default_rng(m)
    scale = float(np.float32(scale))
    n = 1_000_003                                                   # ragged tail
    x = rng.uniform(-2 * scale, (m + 1) * scale, n).astype(np.float32)
    x[:m] = (np.arange(m, dtype=np.float32) + np.float32(0.5)) * np.float32(scale)   # half levels
    x[m:2 * m] = np.arange(m, dtype=np.float32) * np.float32(scale)                  # exact levels
    codes, p = B.quantize(x, scale, m)
    want_codes, want_p = o.quantize(x, scale, m)
    assert np.array_equal(codes, want_codes)
    assert np.array_equal(p, want_p.astype(np.float32))
    assert np.array_equal(p, codes.astype(np.float32) * np.float32(scale))
    lev = o.level_set(scale, m)
    assert np.all(np.isin(p.astype(np.float64), lev))


@pytest.mark.parametrize("m,scale,lo", [(22, 1.0, -1.0), (16, 0.0173, -0.0346), (256, 0.011, 0.25),
                                        (4096, 0.0007, -0.07), (65536, 0.00004, 0.0)])
def test_quantise_kernel_with_offset_is_bit_exact(m, scale, lo):
    """Level sets that do not start at zero, e.g. {-1, ..., 20}: same codes and values as the oracle's projection."""
    rng = np.random.default_rng(m)
    scale, lo = float(np.float32(scale)), float(np.float32(lo))
    x = rng.uniform(lo - 2 * scale, lo + (m + 1) * scale, size=200003).astype(np.float32)
    x[:m] = (lo + (np.arange(m) + 0.5) * scale).astype(np.float32)
    codes, p = B.quantize(x, scale, m, lo=lo)
    assert codes.dtype == (np.uint8 if m <= 256 else np.uint16)
    want_codes, want_p = o.quantize(x, scale, m, lo)
    assert np.array_equal(codes, want_codes)
    assert np.array_equal(p, want_p.astype(np.float32))


def test_quantise_empty_input():
    codes, p = B.quantize(np.zeros(0, np.float32), 1.0, 4)
    assert codes.size == 0 and p.size == 0


@pytest.mark.parametrize("width", [1, 6, 64, 250, 700])
def test_spmm_against_sparse_library(width):
    w = synth.small("c2", 3001, feat_dim=4)
    src, dst = synth.make_graph(w)
    A = o.renormalized_adjacency(w.n_nodes, src, dst)
    x = np.random.default_rng(width).standard_normal((w.n_nodes, width)).astype(np.float32)
    y = B.spmm(A.indptr, A.indices, A.data.astype(np.float32), x)
    want = A.astype(np.float64) @ x.astype(np.float64)
    assert U.rel_err(y.astype(np.float64), want) < 1e-6
    # empty rows and an empty matrix
    E = sp.csr_matrix((5, 5))
    assert np.all(B.spmm(E.indptr, E.indices, E.data, np.ones((5, 3), np.float32)) == 0)


@pytest.mark.parametrize("mode,M,N,K", [(0, 300, 200, 100), (1, 300, 200, 100), (2, 300, 200, 1000), (0, 1000, 500, 500),
                                        (1, 1000, 500, 500), (2, 500, 500, 5000), (0, 129, 7, 65), (1, 5, 131, 3),
                                        (2, 7, 100, 129), (2, 1000, 600, 333), (0, 2500, 120, 1100), (1, 1300, 250, 2100),
                                        (0, 30000, 300, 200), (1, 26000, 200, 330), (2, 1500, 1400, 3000)])
@pytest.mark.parametrize("kind", ["normal", "positive", "tiny", "huge", "mixed"])
def test_dense_products_keep_single_precision_accuracy_at_any_scale(mode, M, N, K, kind):
    """The tensor-core products split each operand into two half-precision planes after scaling it by a power of two
    taken from its largest magnitude: the result must be as accurate as a single-precision product (relative
    Frobenius error below 4e-7 against the product in double precision) whatever the magnitude of the operands,
    also when the entries of one operand span many orders of magnitude, for all three operand layouts, with ragged
    tiles and with contraction lengths that are not a multiple of the K block.  The last shape has enough output
    tiles (40) for the contraction over rows to take its operands as planes split beforehand; the smaller ones
    split them inside the product.  The last two have a partly filled last round of the persistent grid and a long
    contraction, so their tiles are cut into 2 and 4 contraction slices that one warp per tile adds up.  The last three
    have several output tiles per block of the persistent grid (705, 408 and 132 x 8 slices on 148 blocks), so the two
    accumulate sets of a block alternate many times."""
    rng = np.random.default_rng(1000 * mode + M + N + K)
    a = rng.standard_normal((K, M) if mode == 2 else (M, K))
    b = rng.standard_normal((N, K) if mode == 0 else (K, N))
    if kind == "positive":
        a, b = np.abs(a), np.abs(b)
    elif kind == "tiny":
        a, b = a * 1e-20, b * 1e-9
    elif kind == "huge":
        a, b = a * 1e12, b * 3e7
    elif kind == "mixed":
        a = a * np.exp(rng.uniform(-12, 12, size=a.shape))
        b = b * np.exp(rng.uniform(-8, 8, size=b.shape))
    a, b = a.astype(np.float32), b.astype(np.float32)
    a64, b64 = a.astype(np.float64), b.astype(np.float64)
    want = a64 @ b64.T if mode == 0 else (a64 @ b64 if mode == 1 else a64.T @ b64)
    got, ss = B.matmul(mode, a, b)
    assert U.rel_err(got.astype(np.float64), want) < 4e-7
    if kind in ("normal", "positive", "mixed"):          # the sum of squares is taken in single precision per thread
                                                         # (1e-19 < |C| < 1e19), which the other two kinds leave
        assert abs(ss - np.sum(want ** 2)) <= 2e-6 * np.sum(want ** 2)
    ref, _ = B.matmul(mode, a, b, flags=B.FLAG_SIMT_GEMM)             # the CUDA-core product of the same library
    assert U.rel_err(ref.astype(np.float64), want) < 1e-6


def test_single_layer_model_and_zero_hops():
    inp = synth.make_inputs(synth.small("c1", 333, feat_dim=9, hidden=5, n_layers=1, n_hops=0))
    prm, s, _ = U.oracle_problem(inp)
    ctx = B.from_inputs(inp)
    assert ctx.residuals().size == 0
    for k in range(3):
        prev = U.round_state(s)
        U.load_state(ctx, prev, False)
        s = o.iterate(prev, prm)
        ctx.step(1)
        st = U.read_state(ctx)
        assert U.rel_err(st["W"][0], s.W[0]) < 1e-4
        assert U.rel_err(st["z"][0], s.z[0]) < 1e-4
        assert np.linalg.norm(st["b"][0] - s.b[0]) <= 1e-4 * max(np.linalg.norm(s.b[0]), 1e-3)
    assert abs(ctx.objective()[5] - o.objective(s, prm)[5]) <= 1e-4 * abs(o.objective(s, prm)[5])
    ctx.destroy()


def test_graph_without_edges_and_tiny_node_counts():
    for n in (1, 2, 5):
        w = synth.small("c1", n, feat_dim=3, hidden=4, n_layers=3)
        inp = synth.make_inputs(w)
        inp.edge_src = np.zeros(0, np.int32)
        inp.edge_dst = np.zeros(0, np.int32)
        inp.train_mask[:] = 1
        prm, s, A = U.oracle_problem(inp)
        ctx = B.from_inputs(inp)
        assert np.array_equal(ctx.get_tensor(B.T_CSR_COLIDX), np.arange(n, dtype=np.int32))
        assert np.allclose(ctx.get_tensor(B.T_CSR_VAL), 1.0)
        assert U.rel_err(ctx.get_tensor(B.T_X).T.astype(np.float64), s.p[0]) < 1e-6
        ctx.step(3)
        for _ in range(3):
            s = o.iterate(s, prm)
        got = ctx.objective()
        assert np.all(np.isfinite(got))
        assert abs(got[5] - o.objective(s, prm)[5]) <= 1e-3 * abs(o.objective(s, prm)[5]) + 1e-9
        ctx.destroy()


def test_csr_from_messy_edge_list_with_a_hub_is_bit_exact():
    """Repeats, both directions, self-loops and a node with more neighbours than one warp sorts."""
    w = synth.small("c2", 2500, feat_dim=3, hidden=4, n_layers=2)
    inp = synth.make_inputs(w)
    hub = 17
    others = np.setdiff1d(np.arange(w.n_nodes, dtype=np.int32), [hub])[::-1][:1400]      # descending ids
    src = np.concatenate([inp.edge_src, inp.edge_dst[:300], np.full(others.size, hub, np.int32), [5, 9, 9]])
    dst = np.concatenate([inp.edge_dst, inp.edge_src[:300], others, [5, 9, 11]])
    perm = np.random.default_rng(3).permutation(src.size)
    inp.edge_src, inp.edge_dst = src[perm].astype(np.int32), dst[perm].astype(np.int32)
    A = o.renormalized_adjacency(w.n_nodes, inp.edge_src, inp.edge_dst)
    ctx = B.from_inputs(inp)
    assert np.array_equal(ctx.get_tensor(B.T_CSR_ROWPTR), A.indptr.astype(np.int32))
    assert np.array_equal(ctx.get_tensor(B.T_CSR_COLIDX), A.indices.astype(np.int32))
    assert np.allclose(ctx.get_tensor(B.T_CSR_VAL), A.data, rtol=3e-7, atol=0)
    ctx.destroy()


def test_edge_with_node_id_out_of_range_is_rejected():
    w = synth.small("c1", 50, feat_dim=3, hidden=4, n_layers=2)
    inp = synth.make_inputs(w)
    inp.edge_dst = inp.edge_dst.copy()
    inp.edge_dst[4] = 50
    with pytest.raises(RuntimeError, match="edge 4"):
        B.from_inputs(inp)


def test_all_nodes_unlabelled_keeps_z_equal_to_a():
    inp = synth.make_inputs(synth.small("c1", 200, feat_dim=5, hidden=6, n_layers=2))
    inp.train_mask[:] = 0
    prm, s, _ = U.oracle_problem(inp)
    ctx = B.from_inputs(inp)
    ctx.step(2)
    for _ in range(2):
        s = o.iterate(s, prm)
    assert ctx.objective()[0] == 0.0
    assert U.rel_err(ctx.get_tensor(B.T_Z, 2).T.astype(np.float64), s.z[1]) < 1e-4
    ctx.destroy()


def test_get_set_round_trip_and_size_checks():
    inp = synth.make_inputs(synth.small("c2", 300, feat_dim=7, hidden=10, n_layers=3, quant_levels=16))
    ctx = B.from_inputs(inp)
    rng = np.random.default_rng(0)
    for kind, layer in [(B.T_W, 2), (B.T_B, 1), (B.T_Z, 3), (B.T_Q, 1), (B.T_U, 2)]:
        shape, dt = ctx._shape(kind, layer)
        v = rng.standard_normal(shape).astype(dt)
        ctx.set_tensor(kind, layer, v)
        assert np.array_equal(ctx.get_tensor(kind, layer), v)
    scale = ctx.get_tensor(B.T_QSCALE, 2)[0]
    codes = rng.integers(0, 16, size=ctx._shape(B.T_P, 2)[0]).astype(np.uint8)
    ctx.set_tensor(B.T_P, 2, codes.astype(np.float32) * scale)
    assert np.array_equal(ctx.get_tensor(B.T_CODES, 2), codes)
    lib = B.lib()
    buf = np.zeros(10, np.float32)
    assert lib.pdadmm_get_tensor(ctx._h, B.T_W, 1, buf.ctypes.data, 12) == B.EINVAL        # wrong size
    assert lib.pdadmm_get_tensor(ctx._h, B.T_Q, 3, buf.ctypes.data, 40) == B.EINVAL        # q_L does not exist
    assert lib.pdadmm_set_tensor(ctx._h, B.T_TAU, 2, buf.ctypes.data, 8) == B.EINVAL       # read-only
    assert lib.pdadmm_set_tensor(ctx._h, 99, 1, buf.ctypes.data, 8) == B.EINVAL
    assert "kind" in lib.pdadmm_last_error().decode()
    assert lib.pdadmm_step(ctx._h, -1) == B.EINVAL
    ctx.destroy()


@pytest.mark.parametrize("levels", [0, 16])
def test_lanes_and_graph_replay_do_not_change_a_bit(levels):
    """The layers' kernels run on two concurrent lanes and, for pdADMM-G, from a captured graph.  Every reduction
    has a fixed order and every lane its own scratch, so the iterates must be bit-identical to those of a run that
    queues everything on one stream and launches directly: a difference would mean a race between lanes."""
    inp = synth.make_inputs(synth.small("c2", 3000, feat_dim=40, hidden=150, n_layers=5, quant_levels=levels))
    ref = None
    for flags in (B.FLAG_ONE_LANE | B.FLAG_NO_GRAPH, B.FLAG_ONE_LANE, B.FLAG_NO_GRAPH, 0):
        ctx = B.from_inputs(inp, flags=flags)
        ctx.step(2)
        ctx.step(3)                                   # the second call replays the graph where there is one
        st = U.read_state(ctx)
        obj = ctx.objective()
        ctx.destroy()
        if ref is None:
            ref = (st, obj)
            continue
        for k in st:
            for a, b in zip(st[k], ref[0][k]):
                assert np.array_equal(a, b), (flags, k)
        assert np.array_equal(obj, ref[1])


def test_profile_counters_and_launch_count():
    inp = synth.make_inputs(synth.small("c2", 400, feat_dim=8, hidden=12, n_layers=3))
    ctx = B.from_inputs(inp)
    ctx.step(1)                       # the first step also prepares what later steps carry along
    n0 = ctx.launches()
    ctx.step(1)
    n1 = ctx.launches() - n0
    assert n1 > 0
    ctx.profile(True)
    ctx.step(2)
    prof = ctx.profile_read()
    assert ctx.launches() == n0 + 3 * n1
    assert sum(v["launches"] for v in prof.values()) == 2 * n1
    assert prof["zqu"]["launches"] == 2 * 2 and prof["zqu"]["ms"] > 0 and prof["zqu"]["bytes"] > 0
    assert prof["gemm_gradw"]["flops"] > 0
    ctx.profile(False)
    ctx.destroy()


def test_non_finite_state_is_reported_not_propagated_silently():
    """A NaN written into W by the caller: the next step returns ENUMERIC (the gradient norms see it)."""
    inp = synth.make_inputs(synth.small("c1", 300, feat_dim=6, hidden=8, n_layers=3))
    ctx = B.from_inputs(inp)
    ctx.step(1)
    W2 = ctx.get_tensor(B.T_W, 2)
    W2[1, 2] = np.nan
    ctx.set_tensor(B.T_W, 2, W2)
    with pytest.raises(B.PdadmmError) as e:
        ctx.step(1)
    assert e.value.code == B.ENUMERIC
    ctx.destroy()


def test_bounded_wait_runs_out_and_the_device_stays_usable():
    """A wait that nothing satisfies gives up after its cycle limit, the kernel returns by itself, the host reports
    PDADMM_ETIMEOUT, and a tensor-core product launched afterwards in the same process is correct."""
    rc, waited, text = B.selftest_bounded_wait(limit_cycles=100000)
    assert rc == B.ETIMEOUT and "expired" in text
    assert 100000 < waited < 50_000_000              # gave up soon after the limit (polled every 256 probes)
    rng = np.random.default_rng(0)
    a = rng.standard_normal((300, 200)).astype(np.float32)
    b = rng.standard_normal((150, 200)).astype(np.float32)
    c, _ = B.matmul(0, a, b)
    want = a.astype(np.float64) @ b.astype(np.float64).T
    assert U.rel_err(c.astype(np.float64), want) < 1e-6
    with pytest.raises(B.PdadmmError):
        B._check(B.lib().pdadmm_selftest_bounded_wait(0, 0, None))       # limit out of range: EINVAL, nothing launched
