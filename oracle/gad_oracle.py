"""ctypes wrapper around the C oracle (``gad_oracle.c``).

TEST INFRASTRUCTURE: only the tests, the smoke check and the CPU-baseline leg of the benchmark
may import this module.  The CUDA library and its Python binding never do.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gad_oracle.c")
_LIB = os.path.join(_HERE, "libgad_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP over output rows) if it is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _p(a, t):
    return a.ctypes.data_as(C.POINTER(t)) if a is not None else None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.orc_create.restype = C.c_void_p
        L.orc_param_count.restype = C.c_int64
        L.orc_get_epoch.restype = C.c_int64
        L.orc_zeta_aggregate.restype = C.c_double
        L.orc_zeta_pairwise.restype = C.c_double
        _lib = L
    return _lib


def threads() -> int:
    """Threads the OpenMP loops of the oracle will use."""
    n = os.environ.get("OMP_NUM_THREADS")
    if n:
        return int(n.split(",")[0])
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


class Store:
    """The block-diagonal store of the K augmented subgraphs, as the oracle builds it."""

    def __init__(self, n, rowptr, col, core_ptr, core_nodes, halo_ptr, halo_nodes, weights=None):
        L = lib()
        rowptr = np.ascontiguousarray(rowptr, dtype=np.int64)
        col = np.ascontiguousarray(col, dtype=np.int32)
        core_ptr = np.ascontiguousarray(core_ptr, dtype=np.int64)
        core_nodes = np.ascontiguousarray(core_nodes, dtype=np.int32)
        halo_ptr = np.ascontiguousarray(halo_ptr, dtype=np.int64)
        halo_nodes = np.ascontiguousarray(halo_nodes, dtype=np.int32)
        w = None if weights is None else np.ascontiguousarray(weights, dtype=np.float32)
        K = core_ptr.shape[0] - 1
        npr, nnz = C.c_int64(0), C.c_int64(0)
        rc = L.orc_store_sizes(C.c_int32(n), _p(rowptr, C.c_int64), _p(col, C.c_int32), C.c_int32(K),
                               _p(core_ptr, C.c_int64), _p(core_nodes, C.c_int32), _p(halo_ptr, C.c_int64),
                               _p(halo_nodes, C.c_int32), C.byref(npr), C.byref(nnz))
        if rc != 0:
            raise ValueError("oracle store: error %d" % rc)
        self.K = K
        self.n_prime, self.nnz = npr.value, nnz.value
        self.rowptr = np.zeros(self.n_prime + 1, dtype=np.int64)
        self.col = np.zeros(max(self.nnz, 1), dtype=np.int32)
        self.val = np.zeros(max(self.nnz, 1), dtype=np.float64)
        self.sub_off = np.zeros(K + 1, dtype=np.int32)
        self.gid = np.zeros(max(self.n_prime, 1), dtype=np.int32)
        self.deg = np.zeros(max(self.n_prime, 1), dtype=np.int32)
        rc = L.orc_store_build(C.c_int32(n), _p(rowptr, C.c_int64), _p(col, C.c_int32), _p(w, C.c_float),
                               C.c_int32(K), _p(core_ptr, C.c_int64), _p(core_nodes, C.c_int32),
                               _p(halo_ptr, C.c_int64), _p(halo_nodes, C.c_int32), _p(self.rowptr, C.c_int64),
                               _p(self.col, C.c_int32), _p(self.val, C.c_double), _p(self.sub_off, C.c_int32),
                               _p(self.gid, C.c_int32), _p(self.deg, C.c_int32))
        if rc != 0:
            raise ValueError("oracle store: error %d" % rc)
        self.col = self.col[: self.nnz]
        self.val = self.val[: self.nnz]
        self.gid = self.gid[: self.n_prime]
        self.deg = self.deg[: self.n_prime]
        self.core_count = np.diff(core_ptr).astype(np.int64)


class Model:
    """K GCN replicas over the K augmented subgraphs, trained as in Algorithm 2 of the paper."""

    def __init__(self, store: Store, X, labels, split, dims, params0, *, lr=0.01, dropout=0.0, seed=0,
                 beta=1.0, weighted=True, zeta_mode=0):
        L = lib()
        self.store = store
        self.dims = tuple(int(d) for d in dims)
        self.K = store.K
        X = np.ascontiguousarray(X, dtype=np.float32)
        labels = np.ascontiguousarray(labels, dtype=np.int32)
        split = np.ascontiguousarray(split, dtype=np.uint8)
        dims_a = np.asarray(self.dims, dtype=np.int32)
        params0 = np.ascontiguousarray(params0, dtype=np.float32)
        h = L.orc_create(C.c_int64(store.n_prime), C.c_int64(store.nnz), _p(store.rowptr, C.c_int64),
                         _p(store.col, C.c_int32), _p(store.val, C.c_double), C.c_int32(store.K),
                         _p(store.sub_off, C.c_int32), _p(store.gid, C.c_int32), _p(store.deg, C.c_int32),
                         _p(store.core_count, C.c_int64), _p(X, C.c_float), _p(labels, C.c_int32),
                         _p(split, C.c_uint8), C.c_int32(len(self.dims) - 1), _p(dims_a, C.c_int32),
                         C.c_double(lr), C.c_double(dropout), C.c_uint64(seed), C.c_double(beta),
                         C.c_int32(1 if weighted else 0), C.c_int32(zeta_mode), _p(params0, C.c_float))
        if not h:
            raise MemoryError("oracle model: allocation failed")
        self._h = C.c_void_p(h)
        self.P = int(L.orc_param_count(self._h))
        assert self.P == params0.shape[0]

    def close(self):
        if self._h is not None:
            lib().orc_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def train_epoch(self) -> np.ndarray:
        out = np.zeros(self.K + 1, dtype=np.float64)
        lib().orc_train_epoch(self._h, _p(out, C.c_double))
        return out

    def forward_loss(self) -> np.ndarray:
        out = np.zeros(self.K, dtype=np.float64)
        lib().orc_forward_loss(self._h, _p(out, C.c_double))
        return out

    def forward_backward(self) -> np.ndarray:
        out = np.zeros(self.K, dtype=np.float64)
        lib().orc_forward_backward(self._h, _p(out, C.c_double))
        return out

    def forward(self) -> np.ndarray:
        """Inference forward; returns the logits of every store row [N' x C]."""
        lib().orc_forward(self._h)
        return self.activation(len(self.dims) - 1)

    def forward_global(self, n: int) -> np.ndarray:
        """Logits scattered to graph-node order [n x C]; rows no subgraph owns stay zero."""
        lg = self.forward()
        out = np.zeros((n, self.dims[-1]), dtype=np.float64)
        s = self.store
        for k in range(self.K):
            r0 = int(s.sub_off[k])
            nc = int(s.core_count[k])
            out[s.gid[r0:r0 + nc]] = lg[r0:r0 + nc]
        return out

    def activation(self, l: int) -> np.ndarray:
        out = np.zeros((self.store.n_prime, self.dims[l]), dtype=np.float64)
        lib().orc_get_activation(self._h, C.c_int32(l), _p(out, C.c_double))
        return out

    def subgraph_weights(self):
        z = np.zeros(self.K, dtype=np.float64)
        w = np.zeros(self.K, dtype=np.float64)
        lib().orc_subgraph_weights(self._h, _p(z, C.c_double), _p(w, C.c_double))
        return z, w

    def consensus(self):
        lib().orc_consensus(self._h)

    def get_params(self, k: int) -> np.ndarray:
        out = np.zeros(self.P, dtype=np.float64)
        lib().orc_get_params(self._h, C.c_int32(k), _p(out, C.c_double))
        return out

    def set_params(self, k: int, p):
        p = np.ascontiguousarray(p, dtype=np.float64)
        assert p.shape[0] == self.P
        lib().orc_set_params(self._h, C.c_int32(k), _p(p, C.c_double))

    def get_grads(self, k: int) -> np.ndarray:
        out = np.zeros(self.P, dtype=np.float64)
        lib().orc_get_grads(self._h, C.c_int32(k), _p(out, C.c_double))
        return out

    def set_relu_branch(self, layer: int, rows, cols, side: int):
        """Prescribes the ReLU branch (1 on, 2 off, 0 undecided again) of hidden units of H^(layer) at the kink."""
        rows = np.ascontiguousarray(rows, dtype=np.int64)
        cols = np.ascontiguousarray(cols, dtype=np.int32)
        rc = lib().orc_set_relu_branch(self._h, C.c_int32(layer), C.c_int64(rows.shape[0]), _p(rows, C.c_int64),
                                       _p(cols, C.c_int32), C.c_int32(side))
        if rc != 0:
            raise ValueError("orc_set_relu_branch: error %d" % rc)

    def clear_relu_branches(self):
        for l in range(1, len(self.dims) - 1):
            lib().orc_set_relu_branch(self._h, C.c_int32(l), C.c_int64(-1), None, None, C.c_int32(0))

    def ntrain(self) -> np.ndarray:
        out = np.zeros(self.K, dtype=np.int64)
        lib().orc_get_ntrain(self._h, _p(out, C.c_int64))
        return out

    @property
    def epoch(self) -> int:
        return int(lib().orc_get_epoch(self._h))

    @epoch.setter
    def epoch(self, e: int):
        lib().orc_set_epoch(self._h, C.c_int64(e))


def zeta_aggregate(deg, X, beta=1.0) -> float:
    deg = np.ascontiguousarray(deg, dtype=np.int32)
    X = np.ascontiguousarray(X, dtype=np.float64).reshape(deg.shape[0], -1)
    return float(lib().orc_zeta_aggregate(_p(deg, C.c_int32), _p(X, C.c_double), C.c_int64(deg.shape[0]),
                                          C.c_int(X.shape[1]), C.c_double(beta)))


def zeta_pairwise(deg, X, beta=1.0) -> float:
    deg = np.ascontiguousarray(deg, dtype=np.int32)
    X = np.ascontiguousarray(X, dtype=np.float64).reshape(deg.shape[0], -1)
    return float(lib().orc_zeta_pairwise(_p(deg, C.c_int32), _p(X, C.c_double), C.c_int64(deg.shape[0]),
                                         C.c_int(X.shape[1]), C.c_double(beta)))


def zeta_pair_sums(deg, X):
    deg = np.ascontiguousarray(deg, dtype=np.int32)
    X = np.ascontiguousarray(X, dtype=np.float64).reshape(deg.shape[0], -1)
    out = np.zeros(2, dtype=np.float64)
    lib().orc_zeta_pair_sums(_p(deg, C.c_int32), _p(X, C.c_double), C.c_int64(deg.shape[0]), C.c_int(X.shape[1]),
                             _p(out, C.c_double))
    return float(out[0]), float(out[1])


def keep_unit(seed, epoch, layer, row, col, p) -> bool:
    return bool(lib().orc_keep_unit(C.c_uint64(seed), C.c_int64(epoch), C.c_int(layer), C.c_int64(row), C.c_int(col),
                                    C.c_double(p)))


def from_workload(w, params0, **kw):
    """Convenience: oracle store + model for a ``gad_synth.Workload``."""
    cp, cn, hp, hn = w.flat_partition()
    st = Store(w.n, w.rowptr, w.col, cp, cn, hp, hn)
    kw.setdefault("lr", w.lr)
    return Model(st, w.X, w.labels, w.split, w.dims, params0, **kw)
