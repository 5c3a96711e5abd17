"""The node-sharded iteration on the GPU: two contexts, each owning half of the nodes, driven by two host threads on
one device.  The reduction callback is answered on the host: each thread waits for its own stream, the two partial
buffers are added on the host, and both contexts receive the total.  No kernel waits for another one; the threads
meet at a host barrier."""

import threading

import numpy as np
import pytest
import torch

import oracle.pdadmm_oracle as o
from paper_2105_09837_b200 import binding as B
from paper_2105_09837_b200 import sharded, synth
import parity_util as U

pytestmark = pytest.mark.gpu


class HostAllReduce:
    """Adds (or maximises) the callers' device buffers over `world` threads, in rank order, on the host."""

    def __init__(self, world):
        self.world, self.barrier, self.parts = world, threading.Barrier(world), [None] * world
        self.calls = [0] * world

    def callback(self, rank):
        def cb(user, buf, count, dtype, op, stream):
            try:
                torch.cuda.ExternalStream(stream, device="cuda:0").synchronize()
                t = sharded.tensor_at(buf, count, dtype, 0)
                self.parts[rank] = t.cpu().numpy().copy()
                self.barrier.wait(timeout=60)
                tot = self.parts[0].copy()
                for r in range(1, self.world):
                    tot = np.maximum(tot, self.parts[r]) if op == sharded.MAX else tot + self.parts[r]
                self.barrier.wait(timeout=60)
                t.copy_(torch.from_numpy(tot))
                torch.cuda.current_stream().synchronize()
                self.calls[rank] += 1
                return 0
            except Exception:
                import traceback
                traceback.print_exc()
                self.barrier.abort()
                return 1
        return B.ALLREDUCE_FN(cb)


def _run_sharded(inp, world, n_iters, flags=0, teacher=None):
    """`world` contexts on device 0, one thread each; returns (merged device state, objective, residuals, contexts' extras)."""
    w = inp.workload
    red = HostAllReduce(world)
    out, errs = [None] * world, []

    def work(rank):
        try:
            lo, cnt = sharded.node_range(rank, world, w.n_nodes)
            ctx = B.from_inputs(inp, flags=flags, shard=(lo, cnt, red.callback(rank)))
            if teacher is not None:
                U.load_state(ctx, teacher[rank], w.quant_levels > 0)
            ctx.step(n_iters)
            st = U.read_state(ctx)
            st["objective"], st["residuals"] = ctx.objective(), ctx.residuals()
            st["tau"] = [0.0] + [float(ctx.get_tensor(B.T_TAU, l)[0]) for l in range(2, w.n_layers + 1)]
            st["comm_bytes"], st["x"] = ctx.comm_bytes(), ctx.get_tensor(B.T_X)
            ctx.destroy()
            out[rank] = st
        except Exception as e:          # noqa: BLE001
            errs.append(e)
            red.barrier.abort()

    threads = [threading.Thread(target=work, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=600)
    assert not errs, errs
    assert len(set(red.calls)) == 1 and red.calls[0] > 0          # every shard issued the same number of reductions
    return out


@pytest.mark.parametrize("levels,flags", [(0, 0), (16, 0), (0, B.FLAG_SIMT_GEMM)])
def test_two_shards_on_one_device_follow_the_oracle(levels, flags):
    inp = synth.make_inputs(synth.small("c2", 1100, feat_dim=24, hidden=90, n_layers=4, quant_levels=levels))
    w = inp.workload
    prm, s, _ = U.oracle_problem(inp)
    for _ in range(2):
        s = o.iterate(s, prm)                     # a state in which every layer moves
    prev = U.round_state(s)
    parts = o.split_nodes(w.n_nodes, 2)
    out = _run_sharded(inp, 2, 1, flags=flags, teacher=o.shard_state(prev, parts))
    want = o.merge_shards(o.iterate_sharded(o.shard_state(prev, parts), prm))
    plain = o.iterate(prev, prm)
    # X of a shard is its rows of the whole graph's X
    X = np.concatenate([out[0]["x"], out[1]["x"]], axis=0).T.astype(np.float64)
    assert U.rel_err(X, prev.p[0]) < 1e-6
    # the replicated variables are bit-identical on both shards
    for name in ("W", "b"):
        for a, b in zip(out[0][name], out[1][name]):
            assert np.array_equal(a, b), name
    assert out[0]["tau"] == out[1]["tau"]
    assert np.array_equal(out[0]["objective"], out[1]["objective"])
    merged = {k: [np.concatenate([out[0][k][l], out[1][k][l]], axis=1) for l in range(len(out[0][k]))] for k in ("p", "z", "q", "u")}
    for name in ("p", "z", "q"):
        for l in range(len(merged[name])):
            if levels and name == "p" and l >= 1:
                frac = np.mean(merged[name][l] != getattr(want, name)[l])
                assert frac < 2e-3, (name, l, frac)            # codes may take the other neighbour on a rounding boundary
            else:
                tie = None
                if name in ("z", "q") and l < w.n_layers - 1:
                    tie = U.z_tie_mask(prev, want, l)
                    if levels:
                        tie = tie | np.any(merged["p"][l] != want.p[l], axis=0)[None, :] | (merged["p"][l + 1] != want.p[l + 1])
                e = U.rel_err(merged[name][l], getattr(want, name)[l], tie)
                assert e < 1e-4, (name, l, e)
    for l in range(w.n_layers):
        assert U.rel_err(out[0]["W"][l], want.W[l]) < (1e-4 if not levels else 1e-3)
    # the sharded oracle is the plain oracle
    assert U.rel_err(want.W[-1], plain.W[-1]) < 1e-10
    obj = o.objective(o.State(want.p, want.W, want.b, want.z, want.q, want.u, want.y, want.mask, want.scale), prm)
    assert abs(out[0]["objective"][5] - obj[5]) <= 1e-3 * abs(obj[5])
    assert np.allclose(out[0]["residuals"], o.residuals_sq(want), rtol=1e-2, atol=1e-9 * max(o.residuals_sq(want).max(), 1e-30))
    # volume entering the all-reduces of one iteration: every layer's W-gradient and column sums, and the scalars
    widths_in = [w.n0] + w.widths[:-1]
    ld = lambda n: (n + 31) // 32 * 32
    per_iter = sum(4 * no * ld(ni) + 8 * ld(no) + 8 for ni, no in zip(widths_in, w.widths)) + 16 * (w.n_layers - 1)
    assert out[0]["comm_bytes"] >= per_iter            # the quantised update adds 16 bytes per trial


def test_free_run_on_two_shards_matches_one_context():
    inp = synth.make_inputs(synth.small("c2", 900, feat_dim=16, hidden=70, n_layers=5, quant_levels=0))
    out = _run_sharded(inp, 2, 12)
    one = B.from_inputs(inp)
    one.step(12)
    want = U.read_state(one)
    obj = one.objective()
    one.destroy()
    for name in ("z", "q"):
        for l in range(len(want[name])):
            got = np.concatenate([out[0][name][l], out[1][name][l]], axis=1)
            assert U.rel_err(got, want[name][l]) < 1e-3, (name, l)
    for l in range(5):
        assert U.rel_err(out[0]["W"][l], want["W"][l]) < 1e-3
    assert abs(out[0]["objective"][5] - obj[5]) <= 1e-4 * abs(obj[5])


def test_shard_arguments_are_checked():
    inp = synth.make_inputs(synth.small("c1", 60, feat_dim=4, hidden=5, n_layers=2))
    with pytest.raises(B.PdadmmError):
        B.from_inputs(inp, shard=(50, 20, B.ALLREDUCE_FN(lambda *a: 0)))       # reaches past the last node
    with pytest.raises(B.PdadmmError):
        B.from_inputs(inp, shard=(0, 30, B.ALLREDUCE_FN()))                    # part of the graph, no callback


def test_nccl_callback_with_one_rank_equals_the_unsharded_context():
    """The callback that bench.py uses on several GPUs (torch.distributed all_reduce on the library's stream, on a
    tensor that wraps the library's buffer), here in a process group of one NCCL rank: every sum over shards is the
    shard's own value, so the iterates equal those of a context without a callback."""
    import os
    import socket
    import torch.distributed as dist
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        inp = synth.make_inputs(synth.small("c2", 700, feat_dim=12, hidden=40, n_layers=4, quant_levels=16))
        red = sharded.TorchAllReduce(0)
        a = B.from_inputs(inp, shard=(0, 700, red.fn))
        b = B.from_inputs(inp)
        a.step(4)
        b.step(4)
        assert red.calls > 0 and red.bytes - a.comm_bytes() == 4 * 3     # the context counts pdadmm_step's traffic; the start
        #                                                                   reduced one float per level spacing (3 layers)
        sa, sb = U.read_state(a), U.read_state(b)
        for name in ("p", "W", "z", "q"):
            for x, y in zip(sa[name], sb[name]):
                assert U.rel_err(x, y) < 1e-5, name
        assert abs(a.objective()[5] - b.objective()[5]) <= 1e-5 * abs(b.objective()[5])
        a.destroy()
        b.destroy()
    finally:
        dist.destroy_process_group()
