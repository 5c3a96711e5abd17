"""Host-side logic of the node-sharded iteration: one process per GPU, each with the nodes of one contiguous range.

After the feature augmentation every update of Algorithm 1 acts on one node's column at a time, except for a few sums
over nodes (inside tau, theta, the W-gradient, the b-update and the acceptance test of the quantised p-update).  A rank
therefore keeps p, z, q, u of its own nodes and a full copy of W and b, and per iteration the ranks add up, for every
layer, the n_l x n_{l-1} W-gradient, the n_l column sums of the b-update and a handful of scalars.  The paper instead
gives every layer to a client and sends p_{l+1} one way and q_l, u_l the other way across each layer boundary
(Sec. "The pdADMM-G Algorithm"), optionally as 8- or 16-bit codes (Sec. "Quantization Extension", "Communication
Overheads"); `comm_bytes` counts both schemes.

The library calls back for every sum (``pdadmm_allreduce_fn`` of include/pdadmm.h); `TorchAllReduce` answers with
``torch.distributed`` (NCCL on GPUs; the tensors it reduces are the library's own device buffers, which lie in this
GPU's memory).
"""

from __future__ import annotations

import ctypes as C
from typing import List, Tuple

import numpy as np

from .binding import ALLREDUCE_FN
F32, F64 = 0, 1
SUM, MAX = 0, 1


def node_range(rank: int, world: int, n_nodes: int) -> Tuple[int, int]:
    """(first node, node count) of a rank: contiguous, balanced, every node owned exactly once."""
    lo, hi = rank * n_nodes // world, (rank + 1) * n_nodes // world
    return lo, hi - lo


def comm_bytes(n_nodes: int, widths_in: List[int], widths_out: List[int], scheme: str, world: int = 2,
               p_bits: int = 32, q_bits: int = 32, trials: float = 1.0) -> int:
    """Bytes one rank sends per iteration (received bytes are the same by symmetry).

    scheme "nodes":  every layer's W-gradient (float32, n_l x n_{l-1}), column sums (float64, n_l) and scalars
                     (float64: 2 for tau, 1 for theta, 2 per trial of the quantised update) enter an all-reduce; a ring
                     all-reduce sends 2 (R-1)/R of the buffer per rank.
    scheme "layers": the paper's layer-per-client exchange.  Across the boundary between layers l and l+1 the owner
                     of l+1 sends p_{l+1} (n_l x |V| values of p_bits each) and the owner of l sends q_l (q_bits) and
                     u_l (float32).  With `world` clients owning contiguous blocks of layers there are world-1
                     boundaries; a rank in the middle sends across two of them: counted here is the busiest rank.
    """
    L = len(widths_out)
    if scheme == "nodes":
        buf = 0
        for l in range(L):
            buf += 4 * widths_out[l] * widths_in[l] + 8 * widths_out[l] + 8 * 1
            if l >= 1:
                buf += 8 * 2 + (8 * 2 * trials if p_bits < 32 else 0)
        return int(round(2 * (world - 1) / world * buf))
    if scheme == "layers":
        # boundaries after layers L/world, 2L/world, ...: every boundary carries the widths of that layer's output
        cuts = sorted(set(r * L // world for r in range(1, world)))
        per_boundary = [n_nodes * widths_out[c - 1] * (p_bits + q_bits + 32) // 8 for c in cuts if 1 <= c <= L - 1]
        if not per_boundary:
            return 0
        # a boundary's traffic is split between its two sides: p one way, q and u the other
        send_up = [n_nodes * widths_out[c - 1] * (q_bits + 32) // 8 for c in cuts if 1 <= c <= L - 1]     # owner of l
        send_down = [n_nodes * widths_out[c - 1] * p_bits // 8 for c in cuts if 1 <= c <= L - 1]           # owner of l+1
        busiest = 0
        for r in range(world):
            sent = (send_up[r] if r < len(send_up) else 0) + (send_down[r - 1] if 1 <= r <= len(send_down) else 0)
            busiest = max(busiest, sent)
        return int(busiest)
    raise ValueError(scheme)


class _DevicePointer:
    """A device buffer of the library as an object torch can wrap without copying."""

    def __init__(self, ptr: int, count: int, typestr: str):
        self.__cuda_array_interface__ = {"shape": (count,), "typestr": typestr, "data": (int(ptr), False), "version": 2}


def tensor_at(ptr: int, count: int, dtype: int, device: int):
    import torch
    return torch.as_tensor(_DevicePointer(ptr, count, "<f8" if dtype == F64 else "<f4"), device=f"cuda:{device}")


class TorchAllReduce:
    """The library's reduction callback answered by ``torch.distributed.all_reduce`` on the library's stream."""

    def __init__(self, device: int, group=None):
        import torch
        import torch.distributed as dist
        self.device, self.group, self.calls, self.bytes = device, group, 0, 0

        def cb(user, buf, count, dtype, op, stream):
            try:
                t = tensor_at(buf, count, dtype, device)
                with torch.cuda.stream(torch.cuda.ExternalStream(stream, device=f"cuda:{device}")):
                    dist.all_reduce(t, op=dist.ReduceOp.MAX if op == MAX else dist.ReduceOp.SUM, group=self.group)
                self.calls += 1
                self.bytes += count * (8 if dtype == F64 else 4)
                return 0
            except Exception:          # an exception must not cross the C boundary
                import traceback
                traceback.print_exc()
                return 1
        self.fn = ALLREDUCE_FN(cb)      # keep the object alive as long as the context uses it


def oracle_allreduce(dist, group=None):
    """All-reduce (sum) of a float64 numpy array over the ranks of a process group, for the oracle's sharded
    iteration on CPU ranks (``oracle.iterate_sharded(..., allreduce=...)``)."""
    import torch

    def f(x):
        t = torch.from_numpy(np.ascontiguousarray(np.asarray(x, dtype=np.float64)).copy().reshape(-1))
        dist.all_reduce(t, group=group)
        return t.numpy().reshape(np.shape(x)).copy()
    return f
