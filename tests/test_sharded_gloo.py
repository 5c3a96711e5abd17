"""The node-sharded iteration on two CPU ranks (gloo): host logic of the multi-GPU path."""

import os
import socket

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle.pdadmm_oracle as o
from paper_2105_09837_b200 import sharded, synth


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _problem(m):
    w = synth.small("c2", 180, feat_dim=8, hidden=11, n_layers=4, quant_levels=m)
    inp = synth.make_inputs(w)
    prm = o.Params(0.5, 0.02, m)
    A = o.renormalized_adjacency(w.n_nodes, inp.edge_src, inp.edge_dst)
    X = o.augment(inp.features.T.astype(np.float64), A, w.n_blocks)
    return w, o.init_state(X, [x.astype(np.float64) for x in inp.init_W], inp.labels, inp.train_mask, prm), prm


def _worker(rank, world, port, m, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w, s, prm = _problem(m)                                   # every rank builds the graph and X; it keeps its nodes
    lo, cnt = sharded.node_range(rank, world, w.n_nodes)
    mine = o.shard_state(s, [slice(lo, lo + cnt)])
    reduce = sharded.oracle_allreduce(dist)
    for _ in range(4):
        mine = o.iterate_sharded(mine, prm, allreduce=reduce)
    obj = o.objective_sharded(mine, prm, allreduce=reduce)
    out[rank] = dict(p=[a.copy() for a in mine[0].p], W=[a.copy() for a in mine[0].W], b=[a.copy() for a in mine[0].b],
                     z=[a.copy() for a in mine[0].z], tau=list(mine[0].tau), theta=list(mine[0].theta),
                     trials=list(mine[0].trials), obj=obj)
    dist.barrier()
    dist.destroy_process_group()


def _run(m):
    world, port = 2, _free_port()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, m, out), nprocs=world, join=True)
    return [out[r] for r in range(world)]


def test_two_ranks_give_the_bits_of_two_shards_in_one_process():
    """2 x N/2 on two gloo ranks equals the same two shards iterated in one process, bit for bit: every reduction adds
    the same two numbers (a sum of two is commutative), everything else is local."""
    for m in (0, 16):
        ranks = _run(m)
        w, s, prm = _problem(m)
        sh = o.shard_state(s, o.split_nodes(w.n_nodes, 2))
        for _ in range(4):
            sh = o.iterate_sharded(sh, prm)
        for r in range(2):
            for name in ("p", "W", "b", "z"):
                for a, b in zip(ranks[r][name], getattr(sh[r], name)):
                    assert np.array_equal(a, b), (m, r, name)
            assert ranks[r]["tau"] == sh[r].tau and ranks[r]["theta"] == sh[r].theta and ranks[r]["trials"] == sh[r].trials
        assert np.array_equal(ranks[0]["obj"], ranks[1]["obj"])
        assert np.array_equal(ranks[0]["obj"], o.objective_sharded(sh, prm))
        for l in range(4):                                    # the shared variables are the same on both ranks
            assert np.array_equal(ranks[0]["W"][l], ranks[1]["W"][l]) and np.array_equal(ranks[0]["b"][l], ranks[1]["b"][l])
        # and the whole thing is the plain iteration up to the order of the additions
        t = s
        for _ in range(4):
            t = o.iterate(t, prm)
        got = np.concatenate([ranks[0]["z"][-1], ranks[1]["z"][-1]], axis=1)
        assert np.linalg.norm(got - t.z[-1]) <= 1e-10 * np.linalg.norm(t.z[-1])


def test_node_ranges_cover_every_node_once():
    for n, world in [(10, 3), (20000, 8), (7, 7), (5, 8)]:
        ranges = [sharded.node_range(r, world, n) for r in range(world)]
        assert ranges[0][0] == 0 and sum(c for _, c in ranges) == n
        for (a, ca), (b, _) in zip(ranges, ranges[1:]):
            assert a + ca == b
        assert max(c for _, c in ranges) - min(c for _, c in ranges) <= 1


def test_communication_volume_of_the_two_sharding_schemes():
    """Workload c2 (N = 20000, 10 layers x 500, 2800 inputs) on 2 ranks.  Node sharding: a ring all-reduce over 2
    ranks sends the buffer once: 4 (500 x 2800 + 8 x 500 x 500 + 10 x 500) floats + 8-byte sums.  Layer sharding
    (the paper's scheme): one boundary after layer 5 carrying 500 x 20000 values of p one way, q and u the other."""
    win = [2800] + [500] * 9
    wout = [500] * 9 + [10]
    nodes = sharded.comm_bytes(20000, win, wout, "nodes", world=2)
    want = 4 * (500 * 2800 + 8 * 500 * 500 + 10 * 500) + 8 * (9 * 500 + 10) + 8 * 10 + 16 * 9
    assert nodes == want
    e = 20000 * 500
    assert sharded.comm_bytes(20000, win, wout, "layers", world=2) == 8 * e                 # q and u in float32
    assert sharded.comm_bytes(20000, win, wout, "layers", world=2, p_bits=8) == 8 * e       # the busiest rank still sends q, u
    assert sharded.comm_bytes(20000, win, wout, "layers", world=2, p_bits=8, q_bits=8) == 5 * e
    assert nodes < 0.2 * 8 * e                                 # O(L h^2) against O(N h)
