"""ctypes binding of ``libpdadmm.so``: the same entry points as ``include/pdadmm.h``.

Argument marshalling only -- every step of the iteration runs in the library's kernels.
The library must have been built (``python -m paper_2105_09837_b200.build``); loading fails
loudly otherwise, and there is no CPU fallback.
"""

from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import numpy as np

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libpdadmm.so")
_lib = None

# tensor kinds (pdadmm_tensor)
T_X, T_P, T_W, T_B, T_Z, T_Q, T_U, T_CODES, T_TAU, T_THETA, T_QSCALE, T_CSR_ROWPTR, T_CSR_COLIDX, T_CSR_VAL, T_TRIALS = range(15)
FLAG_SIMT_GEMM = 1
FLAG_QUANT_Q = 2
FLAG_NO_GRAPH = 4
FLAG_ONE_LANE = 8
FLAG_LEAST_SQUARES = 16
ACT_RELU, ACT_TANH, ACT_SIGMOID = 0, 1, 2

OK, EINVAL, ENOMEM, ECUDA, ETIMEOUT, ENUMERIC, ENOTCONV = 0, -1, -2, -3, -4, -5, -6

EXPORTS = [
    "pdadmm_init", "pdadmm_init_sharded", "pdadmm_comm_bytes", "pdadmm_start_layers_from", "pdadmm_step", "pdadmm_last_step_ms", "pdadmm_objective", "pdadmm_residuals", "pdadmm_get_tensor",
    "pdadmm_set_tensor", "pdadmm_predict", "pdadmm_quantize", "pdadmm_spmm", "pdadmm_matmul", "pdadmm_matmul_tn_static", "pdadmm_selftest_bounded_wait",
    "pdadmm_profile", "pdadmm_profile_classes",
    "pdadmm_profile_name", "pdadmm_profile_read", "pdadmm_launches", "pdadmm_time_augmentation", "pdadmm_destroy", "pdadmm_last_error",
]


class PdadmmError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"pdadmm error {code}: {text}")
        self.code = code


class _Config(C.Structure):
    _fields_ = [
        ("n_nodes", C.c_int64), ("n_edges", C.c_int64),
        ("edge_src", C.POINTER(C.c_int32)), ("edge_dst", C.POINTER(C.c_int32)),
        ("feat_dim", C.c_int32), ("features", C.POINTER(C.c_float)),
        ("n_hops", C.c_int32), ("n_classes", C.c_int32),
        ("labels", C.POINTER(C.c_int32)), ("train_mask", C.POINTER(C.c_uint8)),
        ("n_layers", C.c_int32), ("layer_widths", C.POINTER(C.c_int32)),
        ("rho", C.c_float), ("nu", C.c_float), ("quant_levels", C.c_int32),
        ("quant_neg_levels", C.c_int32), ("quant_step", C.c_float), ("leaky_slope", C.c_float),
        ("activation", C.c_int32), ("table_size", C.c_int32), ("table_lo", C.c_float), ("table_hi", C.c_float),
        ("init_W", C.POINTER(C.POINTER(C.c_float))),
        ("device", C.c_int32), ("flags", C.c_uint32),
    ]


ALLREDUCE_FN = C.CFUNCTYPE(C.c_int, C.c_void_p, C.c_void_p, C.c_size_t, C.c_int, C.c_int, C.c_void_p)


class _Shard(C.Structure):
    _fields_ = [("node_begin", C.c_int64), ("node_count", C.c_int64), ("allreduce", ALLREDUCE_FN), ("user", C.c_void_p)]


def lib() -> C.CDLL:
    """Load the shared library (once)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2105_09837_b200.build`")
        L = C.CDLL(_LIB_PATH)
        L.pdadmm_last_error.restype = C.c_char_p
        L.pdadmm_profile_name.restype = C.c_char_p
        L.pdadmm_init.argtypes = [C.POINTER(_Config), C.POINTER(C.c_void_p)]
        L.pdadmm_init_sharded.argtypes = [C.POINTER(_Config), C.POINTER(_Shard), C.POINTER(C.c_void_p)]
        L.pdadmm_comm_bytes.argtypes = [C.c_void_p, C.POINTER(C.c_int64)]
        L.pdadmm_start_layers_from.argtypes = [C.c_void_p, C.c_int]
        L.pdadmm_step.argtypes = [C.c_void_p, C.c_int]
        L.pdadmm_last_step_ms.argtypes = [C.c_void_p, C.POINTER(C.c_double)]
        L.pdadmm_objective.argtypes = [C.c_void_p, C.POINTER(C.c_double)]
        L.pdadmm_residuals.argtypes = [C.c_void_p, C.POINTER(C.c_double), C.c_int]
        L.pdadmm_get_tensor.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_size_t]
        L.pdadmm_set_tensor.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_size_t]
        L.pdadmm_predict.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.pdadmm_quantize.argtypes = [C.c_int, C.c_void_p, C.c_size_t, C.c_float, C.c_float, C.c_int, C.c_void_p,
                                      C.c_void_p]
        L.pdadmm_spmm.argtypes = [C.c_int, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
        L.pdadmm_matmul.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                    C.POINTER(C.c_double), C.c_uint32]
        L.pdadmm_matmul_tn_static.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_void_p, C.c_int,
                                              C.c_void_p, C.c_void_p]
        L.pdadmm_selftest_bounded_wait.argtypes = [C.c_int, C.c_longlong, C.POINTER(C.c_longlong)]
        L.pdadmm_profile.argtypes = [C.c_void_p, C.c_int]
        L.pdadmm_profile_name.argtypes = [C.c_int]
        L.pdadmm_profile_read.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_int64),
                                          C.POINTER(C.c_double), C.POINTER(C.c_double)]
        L.pdadmm_launches.argtypes = [C.c_void_p, C.POINTER(C.c_int64)]
        L.pdadmm_time_augmentation.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_double)]
        L.pdadmm_destroy.argtypes = [C.c_void_p]
        _lib = L
    return _lib


def _check(rc: int):
    if rc != 0:
        raise PdadmmError(rc, lib().pdadmm_last_error().decode())


def _ptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(C.POINTER(ctype))


class Context:
    """One problem on one device (``pdadmm_ctx``)."""

    def __init__(self, n_nodes: int, edge_src, edge_dst, features, n_hops: int, n_classes: int, labels, train_mask,
                 layer_widths: Sequence[int], rho: float, nu: float, quant_levels: int, init_W: List[np.ndarray],
                 device: int = 0, flags: int = 0, quant_neg_levels: int = 0, quant_step: float = 0.0,
                 leaky_slope: float = 0.0, shard=None, activation: int = 0, table=(0, 0.0, 0.0)):
        """shard: None, or (node_begin, node_count, allreduce) with allreduce an ``ALLREDUCE_FN`` object (kept alive
        here): the context then owns those nodes only (``pdadmm_init_sharded``)."""
        self._h = C.c_void_p()
        src = np.ascontiguousarray(edge_src, dtype=np.int32)
        dst = np.ascontiguousarray(edge_dst, dtype=np.int32)
        feat = np.ascontiguousarray(features, dtype=np.float32)
        lab = np.ascontiguousarray(labels, dtype=np.int32)
        msk = np.ascontiguousarray(train_mask, dtype=np.uint8)
        widths = np.ascontiguousarray(layer_widths, dtype=np.int32)
        Ws = [np.ascontiguousarray(w, dtype=np.float32) for w in init_W]
        if feat.ndim != 2 or feat.shape[0] != n_nodes:
            raise ValueError("features must be [n_nodes][feat_dim]")
        n_in = (n_hops + 1) * feat.shape[1]
        if len(Ws) != len(widths):
            raise ValueError("one initial weight matrix per layer is required")
        for w, n_out in zip(Ws, widths):
            if w.shape != (int(n_out), n_in):
                raise ValueError(f"init_W has shape {w.shape}, expected {(int(n_out), n_in)}")
            n_in = int(n_out)
        if lab.shape != (n_nodes,) or msk.shape != (n_nodes,) or src.shape != dst.shape:
            raise ValueError("labels/mask must be [n_nodes]; edge arrays must have equal length")
        wp = (C.POINTER(C.c_float) * len(Ws))(*[_ptr(w, C.c_float) for w in Ws])
        cfg = _Config(n_nodes, src.size, _ptr(src, C.c_int32), _ptr(dst, C.c_int32), feat.shape[1],
                      _ptr(feat, C.c_float), n_hops, n_classes, _ptr(lab, C.c_int32), _ptr(msk, C.c_uint8),
                      len(widths), _ptr(widths, C.c_int32), rho, nu, quant_levels, quant_neg_levels, quant_step, leaky_slope,
                      int(activation), int(table[0]), float(table[1]), float(table[2]), wp, device, flags)
        self.n_nodes, self.n_layers = int(n_nodes), len(widths)
        self.n_nodes_total = int(n_nodes)
        self.n0 = (n_hops + 1) * feat.shape[1]
        self.widths = [int(x) for x in widths]
        self.quant_levels = int(quant_levels)
        if shard is None:
            _check(lib().pdadmm_init(C.byref(cfg), C.byref(self._h)))
        else:
            begin, count, fn = shard
            self._allreduce = fn                      # the library keeps the pointer: the object must outlive the context
            sh = _Shard(int(begin), int(count), fn, None)
            self.n_nodes = int(count)
            _check(lib().pdadmm_init_sharded(C.byref(cfg), C.byref(sh), C.byref(self._h)))

    # ---- same names as the C ABI
    def step(self, n_iters: int = 1):
        _check(lib().pdadmm_step(self._h, int(n_iters)))

    def start_layers_from(self, first_layer: int):
        _check(lib().pdadmm_start_layers_from(self._h, int(first_layer)))

    def last_step_ms(self) -> float:
        ms = C.c_double()
        _check(lib().pdadmm_last_step_ms(self._h, C.byref(ms)))
        return ms.value

    def objective(self) -> np.ndarray:
        out = (C.c_double * 6)()
        _check(lib().pdadmm_objective(self._h, out))
        return np.array(out[:])

    def residuals(self) -> np.ndarray:
        n = self.n_layers - 1
        out = (C.c_double * max(n, 1))()
        _check(lib().pdadmm_residuals(self._h, out if n else None, n))
        return np.array(out[:n])

    def predict(self):
        """``pdadmm_predict``: (logits [N][C] float32, classes [N] int32, counts [4] int64)."""
        logits = np.empty((self.n_nodes, self.widths[-1]), dtype=np.float32)
        pred = np.empty(self.n_nodes, dtype=np.int32)
        counts = np.zeros(4, dtype=np.int64)
        _check(lib().pdadmm_predict(self._h, logits.ctypes.data_as(C.c_void_p), pred.ctypes.data_as(C.c_void_p),
                                    counts.ctypes.data_as(C.c_void_p)))
        return logits, pred, counts

    def _shape(self, kind: int, layer: int):
        n_in = self.n0 if layer <= 1 else self.widths[layer - 2]
        n_out = self.widths[layer - 1] if 1 <= layer <= self.n_layers else 0
        N = self.n_nodes
        if kind == T_X:
            return (N, self.n0), np.float32
        if kind == T_P:
            return (N, n_in), np.float32
        if kind == T_W:
            return (n_out, n_in), np.float32
        if kind == T_B:
            return (n_out,), np.float32
        if kind in (T_Z, T_Q, T_U):
            return (N, n_out), np.float32
        if kind == T_CODES:
            return (N, n_in), (np.uint16 if self.quant_levels > 256 else np.uint8)
        if kind in (T_TAU, T_THETA):
            return (1,), np.float64
        if kind == T_QSCALE:
            return (1,), np.float32
        if kind == T_TRIALS:
            return (1,), np.int32
        if kind == T_CSR_ROWPTR:
            return (self.n_nodes_total + 1,), np.int32
        raise ValueError(kind)

    def get_tensor(self, kind: int, layer: int = 1) -> np.ndarray:
        if kind in (T_CSR_COLIDX, T_CSR_VAL):
            nnz = int(self.get_tensor(T_CSR_ROWPTR)[-1])
            shape, dt = (nnz,), (np.int32 if kind == T_CSR_COLIDX else np.float32)
        else:
            shape, dt = self._shape(kind, layer)
        out = np.empty(shape, dtype=dt)
        _check(lib().pdadmm_get_tensor(self._h, kind, layer, out.ctypes.data_as(C.c_void_p), out.nbytes))
        return out

    def set_tensor(self, kind: int, layer: int, value):
        shape, dt = self._shape(kind, layer)
        a = np.ascontiguousarray(value, dtype=dt)
        if a.shape != shape:
            raise ValueError(f"tensor kind {kind} layer {layer} has shape {shape}, got {a.shape}")
        _check(lib().pdadmm_set_tensor(self._h, kind, layer, a.ctypes.data_as(C.c_void_p), a.nbytes))

    def profile(self, enable: bool):
        _check(lib().pdadmm_profile(self._h, int(bool(enable))))

    def profile_read(self) -> dict:
        out = {}
        for k in range(lib().pdadmm_profile_classes()):
            ms, n, by, fl = C.c_double(), C.c_int64(), C.c_double(), C.c_double()
            _check(lib().pdadmm_profile_read(self._h, k, C.byref(ms), C.byref(n), C.byref(by), C.byref(fl)))
            out[lib().pdadmm_profile_name(k).decode()] = dict(ms=ms.value, launches=n.value, bytes=by.value, flops=fl.value)
        return out

    def time_augmentation(self, reps: int = 20):
        """``pdadmm_time_augmentation``: (ms per hop, algorithmic bytes per hop)."""
        ms, by = C.c_double(), C.c_double()
        _check(lib().pdadmm_time_augmentation(self._h, reps, C.byref(ms), C.byref(by)))
        return ms.value, by.value

    def comm_bytes(self) -> int:
        n = C.c_int64()
        _check(lib().pdadmm_comm_bytes(self._h, C.byref(n)))
        return n.value

    def launches(self) -> int:
        n = C.c_int64()
        _check(lib().pdadmm_launches(self._h, C.byref(n)))
        return n.value

    def destroy(self):
        if self._h:
            lib().pdadmm_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def from_inputs(inp, device: int = 0, flags: int = 0, rho: Optional[float] = None, nu: Optional[float] = None,
                quant_levels: Optional[int] = None, quant_neg_levels: int = 0, quant_step: float = 0.0,
                leaky_slope: float = 0.0, shard=None, activation: int = 0, table=(0, 0.0, 0.0)) -> Context:
    """Context for a ``synth.Inputs`` bundle."""
    w = inp.workload
    return Context(w.n_nodes, inp.edge_src, inp.edge_dst, inp.features, w.n_hops, w.n_classes, inp.labels,
                   inp.train_mask, w.widths, w.rho if rho is None else rho, w.nu if nu is None else nu,
                   w.quant_levels if quant_levels is None else quant_levels, inp.init_W, device, flags,
                   quant_neg_levels, quant_step, leaky_slope, shard, activation, table)


def quantize(x, scale: float, levels: int, device: int = 0, lo: float = 0.0):
    """``pdadmm_quantize``: (codes uint8, p float32) for a float32 array; ``lo`` is the smallest level."""
    a = np.ascontiguousarray(x, dtype=np.float32)
    codes = np.empty(a.shape, dtype=np.uint16 if levels > 256 else np.uint8)
    p = np.empty(a.shape, dtype=np.float32)
    _check(lib().pdadmm_quantize(device, a.ctypes.data_as(C.c_void_p), a.size, scale, lo, levels,
                                 codes.ctypes.data_as(C.c_void_p), p.ctypes.data_as(C.c_void_p)))
    return codes, p


def spmm(row_ptr, col_idx, val, x, device: int = 0) -> np.ndarray:
    """``pdadmm_spmm``: Y = A X for a CSR matrix and a node-major float32 matrix."""
    rp = np.ascontiguousarray(row_ptr, dtype=np.int32)
    ci = np.ascontiguousarray(col_idx, dtype=np.int32)
    v = np.ascontiguousarray(val, dtype=np.float32)
    a = np.ascontiguousarray(x, dtype=np.float32)
    y = np.empty_like(a)
    _check(lib().pdadmm_spmm(device, rp.size - 1, rp.ctypes.data_as(C.c_void_p), ci.ctypes.data_as(C.c_void_p),
                             v.ctypes.data_as(C.c_void_p), a.ctypes.data_as(C.c_void_p), a.shape[1],
                             y.ctypes.data_as(C.c_void_p)))
    return y


def matmul(mode: int, A, B, flags: int = 0, device: int = 0):
    """``pdadmm_matmul``: (C, sum(C^2)).  mode 0: A[M,K] B[N,K]^T; 1: A[M,K] B[K,N]; 2: A[K,M]^T B[K,N]."""
    a = np.ascontiguousarray(A, dtype=np.float32)
    b = np.ascontiguousarray(B, dtype=np.float32)
    if mode == 0:
        (M, K), (N, K2) = a.shape, b.shape
    elif mode == 1:
        (M, K), (K2, N) = a.shape, b.shape
    else:
        (K, M), (K2, N) = a.shape, b.shape
    if K != K2:
        raise ValueError("contraction lengths differ")
    c = np.empty((M, N), dtype=np.float32)
    ss = C.c_double()
    _check(lib().pdadmm_matmul(device, mode, M, N, K, a.ctypes.data_as(C.c_void_p), b.ctypes.data_as(C.c_void_p),
                               c.ctypes.data_as(C.c_void_p), C.byref(ss), flags))
    return c, ss.value


def matmul_tn_static(dA: int, lda: int, dB: int, ldb: int, dC: int, M: int, N: int, K: int, stream: int = 0,
                     device: int = 0):
    """``pdadmm_matmul_tn_static``: C = A^T B on device buffers given by their addresses; allocates nothing.

    The kernels are only enqueued on ``stream``; the caller synchronises before reading C.
    """
    _check(lib().pdadmm_matmul_tn_static(device, M, N, K, C.c_void_p(dA), lda, C.c_void_p(dB), ldb, C.c_void_p(dC),
                                         C.c_void_p(stream)))


def selftest_bounded_wait(limit_cycles: int = 100000, device: int = 0):
    """``pdadmm_selftest_bounded_wait``: returns (status code, cycles waited); the status is ETIMEOUT by design."""
    waited = C.c_longlong(0)
    rc = lib().pdadmm_selftest_bounded_wait(device, limit_cycles, C.byref(waited))
    return rc, int(waited.value), lib().pdadmm_last_error().decode()
