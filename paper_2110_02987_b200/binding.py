"""Thin ctypes binding of the C-ABI library ``libgad.so`` (see ``include/gad.h``).

Argument marshalling only: every step of the epoch runs in the library's CUDA kernels.  PyTorch is
used for what the boundary leaves to the caller: the device workspace and the stream.  There is no
CPU fallback; importing works without a GPU (so the exported symbols can be checked), but every
compute call needs the built library and a CUDA device and raises otherwise.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgad.so")

GAD_OK = 0
ERRORS = {-1: "GAD_ERR_ARG", -2: "GAD_ERR_RANGE", -3: "GAD_ERR_UNSORTED", -4: "GAD_ERR_DUPLICATE", -5: "GAD_ERR_OOM",
          -6: "GAD_ERR_NONFINITE", -7: "GAD_ERR_DEVICE_TIMEOUT", -8: "GAD_ERR_CUDA", -9: "GAD_ERR_UNSUPPORTED"}

# Every symbol include/gad.h declares.
SYMBOLS = (
    "gad_workspace_bytes", "gad_create", "gad_train_epoch", "gad_get_loss", "gad_forward", "gad_subgraph_weights",
    "gad_consensus", "gad_get_params", "gad_set_params", "gad_get_grads", "gad_param_count", "gad_store_sizes",
    "gad_get_store", "gad_get_activation", "gad_set_inputs", "gad_read_loss_async", "gad_synchronize", "gad_get_epoch", "gad_set_epoch", "gad_profile_enable",
    "gad_profile_reset", "gad_profile_count", "gad_profile_read", "gad_subgraph_weights_static", "gad_launch_count",
    "gad_last_error", "gad_destroy", "gad_train_epoch_local", "gad_consensus_floats", "gad_consensus_partial",
    "gad_consensus_apply", "gad_export_params", "gad_get_train_counts", "gad_augment_workspace_bytes", "gad_augment",
    "gad_augment_last_error", "gad_debug_expire_wait", "gad_default_params", "gad_check_store",
)


class GadError(RuntimeError):
    def __init__(self, code, msg=""):
        self.code = code
        super().__init__("%s (%d)%s" % (ERRORS.get(code, "GAD_ERR_?"), code, ": " + msg if msg else ""))


class gad_csr(C.Structure):
    _fields_ = [("n", C.c_int32), ("nnz", C.c_int64), ("rowptr", C.POINTER(C.c_int64)), ("col", C.POINTER(C.c_int32)),
                ("w", C.POINTER(C.c_float))]


class gad_partition(C.Structure):
    _fields_ = [("K", C.c_int32), ("core_ptr", C.POINTER(C.c_int64)), ("core_nodes", C.POINTER(C.c_int32)),
                ("halo_ptr", C.POINTER(C.c_int64)), ("halo_nodes", C.POINTER(C.c_int32))]


class gad_config(C.Structure):
    _fields_ = [("L", C.c_int32), ("dims", C.POINTER(C.c_int32)), ("lr", C.c_float), ("dropout", C.c_float),
                ("seed", C.c_uint64), ("gemm_mode", C.c_int32), ("zeta_mode", C.c_int32), ("beta", C.c_float),
                ("weighted", C.c_int32), ("flags", C.c_int32)]


_lib = None


def load():
    """Loads libgad.so; raises if it has not been built (``python -m paper_2110_02987_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libgad.so is missing: build it with paper_2110_02987_b200/build.py "
                               "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        L.gad_last_error.restype = C.c_char_p
        L.gad_last_error.argtypes = [C.c_void_p]
        L.gad_destroy.restype = None
        L.gad_destroy.argtypes = [C.c_void_p]
        _lib = L
    return _lib


def _ptr(a, t):
    return a.ctypes.data_as(C.POINTER(t)) if a is not None else None


def _arr(a, dtype):
    return None if a is None else np.ascontiguousarray(a, dtype=dtype)


class _Inputs:
    """Keeps the marshalled host arrays alive for the duration of a call."""

    def __init__(self, n, rowptr, col, weights, core_ptr, core_nodes, halo_ptr, halo_nodes, dims, lr, dropout, seed,
                 gemm_mode, zeta_mode, beta, weighted, flags):
        self.rowptr = _arr(rowptr, np.int64)
        self.col = _arr(col, np.int32)
        self.w = _arr(weights, np.float32)
        self.core_ptr = _arr(core_ptr, np.int64)
        self.core_nodes = _arr(core_nodes, np.int32)
        self.halo_ptr = _arr(halo_ptr, np.int64)
        self.halo_nodes = _arr(halo_nodes, np.int32)
        self.dims = np.asarray(dims, dtype=np.int32)
        self.csr = gad_csr(int(n), int(self.rowptr[-1]) if self.rowptr is not None and self.rowptr.size else 0,
                           _ptr(self.rowptr, C.c_int64), _ptr(self.col, C.c_int32), _ptr(self.w, C.c_float))
        self.part = gad_partition(int(self.core_ptr.shape[0] - 1), _ptr(self.core_ptr, C.c_int64),
                                  _ptr(self.core_nodes, C.c_int32), _ptr(self.halo_ptr, C.c_int64),
                                  _ptr(self.halo_nodes, C.c_int32))
        self.cfg = gad_config(int(self.dims.shape[0] - 1), _ptr(self.dims, C.c_int32), float(lr), float(dropout), int(seed),
                              int(gemm_mode), int(zeta_mode), float(beta), 1 if weighted else 0, int(flags))


def gad_workspace_bytes(n, rowptr, col, core_ptr, core_nodes, halo_ptr, halo_nodes, dims, *, weights=None, lr=0.01,
                        dropout=0.0, seed=0, gemm_mode=0, zeta_mode=0, beta=1.0, weighted=True, flags=0) -> int:
    L = load()
    inp = _Inputs(n, rowptr, col, weights, core_ptr, core_nodes, halo_ptr, halo_nodes, dims, lr, dropout, seed, gemm_mode,
                  zeta_mode, beta, weighted, flags)
    out = C.c_size_t(0)
    rc = L.gad_workspace_bytes(C.byref(inp.csr), C.byref(inp.part), C.byref(inp.cfg), C.byref(out))
    if rc != GAD_OK:
        raise GadError(rc, (L.gad_last_error(None) or b"").decode())
    return int(out.value)


class Gad:
    """One library context: K GCN replicas over K augmented subgraphs on the current CUDA device.

    Methods carry the names of the C entry points (without the ``gad_`` prefix where it reads better as a method:
    ``train_epoch``, ``forward``, ``subgraph_weights``, ``consensus`` ...).
    """

    def __init__(self, n, rowptr, col, core_ptr, core_nodes, halo_ptr, halo_nodes, X, labels, split, dims, *,
                 init_params=None, weights=None, lr=0.01, dropout=0.0, seed=0, gemm_mode=0, zeta_mode=0, beta=1.0,
                 weighted=True, flags=0, stream=None, device=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("the GAD library needs a CUDA device (there is no CPU fallback)")
        L = load()
        self._L = L
        self._h = None
        self.n = int(n)
        self.dims = tuple(int(d) for d in dims)
        inp = _Inputs(n, rowptr, col, weights, core_ptr, core_nodes, halo_ptr, halo_nodes, dims, lr, dropout, seed,
                      gemm_mode, zeta_mode, beta, weighted, flags)
        self.K = int(inp.part.K)
        X = _arr(X, np.float32)
        labels = _arr(labels, np.int32)
        split = _arr(split, np.uint8)
        if X.shape != (self.n, self.dims[0]) or labels.shape != (self.n,) or split.shape != (self.n,):
            raise GadError(-1, "X / labels / split have the wrong shape")
        init = _arr(init_params, np.float32)
        nbytes = C.c_size_t(0)
        rc = L.gad_workspace_bytes(C.byref(inp.csr), C.byref(inp.part), C.byref(inp.cfg), C.byref(nbytes))
        if rc != GAD_OK:
            raise GadError(rc, (L.gad_last_error(None) or b"").decode())
        self.device = torch.device(device if device is not None else "cuda:%d" % torch.cuda.current_device())
        self.workspace_bytes = int(nbytes.value)
        with torch.cuda.device(self.device):
            self._ws = torch.empty(self.workspace_bytes + 256, dtype=torch.uint8, device=self.device)
            base = self._ws.data_ptr()
            aligned = (base + 255) // 256 * 256
            self._stream = stream if stream is not None else torch.cuda.current_stream(self.device)
            h = C.c_void_p(None)
            rc = L.gad_create(C.byref(h), C.byref(inp.csr), C.byref(inp.part), _ptr(X, C.c_float), _ptr(labels, C.c_int32),
                              _ptr(split, C.c_uint8), C.byref(inp.cfg), _ptr(init, C.c_float), C.c_void_p(aligned),
                              C.c_size_t(self.workspace_bytes), C.c_void_p(self._stream.cuda_stream))
        if rc != GAD_OK:
            raise GadError(rc, (L.gad_last_error(None) or b"").decode())
        self._h = h
        P = C.c_int64(0)
        self._ck(L.gad_param_count(self._h, C.byref(P)))
        self.P = int(P.value)
        a, b = C.c_int64(0), C.c_int64(0)
        self._ck(L.gad_store_sizes(self._h, C.byref(a), C.byref(b)))
        self.n_prime, self.nnz_prime = int(a.value), int(b.value)

    # -- plumbing ------------------------------------------------------------------------------
    def _ck(self, rc):
        if rc != GAD_OK:
            raise GadError(rc, (self._L.gad_last_error(self._h) or b"").decode())

    def destroy(self):
        if self._h is not None:
            self._L.gad_destroy(self._h)
            self._h = None
            self._ws = None

    close = destroy

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.destroy()

    # -- the epoch -----------------------------------------------------------------------------
    def train_epoch(self, loss_out=None, wait=True):
        """gad_train_epoch.  With wait=True returns the float32 [K+1] losses (and waits for the stream); with
        wait=False only enqueues the epoch and returns None.  ``loss_out`` may be a preallocated float32 [K+1]
        array (e.g. a view of pinned memory); with wait=False it must be pinned and receives the losses once the
        stream gets there (gad_read_loss_async; call synchronize() before reading it)."""
        if not wait:
            self._ck(self._L.gad_train_epoch(self._h, None))
            if loss_out is not None:
                self._ck(self._L.gad_read_loss_async(self._h, _ptr(loss_out, C.c_float)))
            return None
        out = loss_out if loss_out is not None else np.zeros(self.K + 1, dtype=np.float32)
        self._ck(self._L.gad_train_epoch(self._h, _ptr(out, C.c_float)))
        return out

    def synchronize(self):
        """gad_synchronize: waits for everything enqueued on the context's two streams."""
        self._ck(self._L.gad_synchronize(self._h))

    def get_loss(self):
        out = np.zeros(self.K + 1, dtype=np.float32)
        self._ck(self._L.gad_get_loss(self._h, _ptr(out, C.c_float)))
        return out

    def forward(self):
        out = np.zeros((self.n, self.dims[-1]), dtype=np.float32)
        self._ck(self._L.gad_forward(self._h, _ptr(out, C.c_float)))
        return out

    def subgraph_weights(self):
        z = np.zeros(self.K, dtype=np.float32)
        w = np.zeros(self.K, dtype=np.float32)
        self._ck(self._L.gad_subgraph_weights(self._h, _ptr(z, C.c_float), _ptr(w, C.c_float)))
        return z, w

    def consensus(self):
        self._ck(self._L.gad_consensus(self._h))

    # -- the subgraphs spread over several contexts ---------------------------------------------
    def train_epoch_local(self, wait=True):
        """gad_train_epoch_local: forward, loss, backward and zeta; no update, no consensus.  Returns the float32 [K+1]
        losses with wait=True, None otherwise."""
        if not wait:
            self._ck(self._L.gad_train_epoch_local(self._h, None))
            return None
        out = np.zeros(self.K + 1, dtype=np.float32)
        self._ck(self._L.gad_train_epoch_local(self._h, _ptr(out, C.c_float)))
        return out

    def ntrain(self):
        """gad_get_train_counts: |T_k| of every subgraph, int64 [K]."""
        out = np.zeros(self.K, dtype=np.int64)
        self._ck(self._L.gad_get_train_counts(self._h, _ptr(out, C.c_int64)))
        return out

    def consensus_floats(self) -> int:
        n = C.c_int64(0)
        self._ck(self._L.gad_consensus_floats(self._h, C.byref(n)))
        return int(n.value)

    def new_consensus_buffer(self):
        """A float32 CUDA tensor of gad_consensus_floats elements on this context's device."""
        import torch
        return torch.zeros(self.consensus_floats(), dtype=torch.float32, device=self.device)

    def consensus_partial(self, zeta_total, out, with_step=True):
        """gad_consensus_partial into the CUDA tensor ``out`` (see new_consensus_buffer)."""
        self._check_buffer(out)
        self._ck(self._L.gad_consensus_partial(self._h, C.c_double(float(zeta_total)), C.c_int32(1 if with_step else 0),
                                               C.c_void_p(out.data_ptr())))
        return out

    def consensus_apply(self, buf):
        self._check_buffer(buf)
        self._ck(self._L.gad_consensus_apply(self._h, C.c_void_p(buf.data_ptr())))

    def export_params(self, k, out):
        self._check_buffer(out)
        self._ck(self._L.gad_export_params(self._h, C.c_int32(k), C.c_void_p(out.data_ptr())))
        return out

    def _check_buffer(self, t):
        import torch
        if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()
                and t.numel() >= self.consensus_floats()):
            raise GadError(-1, "a consensus buffer is a contiguous float32 CUDA tensor of consensus_floats() elements")

    # -- accessors -----------------------------------------------------------------------------
    def get_params(self, k):
        out = np.zeros(self.P, dtype=np.float32)
        self._ck(self._L.gad_get_params(self._h, C.c_int32(k), _ptr(out, C.c_float)))
        return out

    def set_params(self, k, p):
        p = _arr(p, np.float32)
        if p.shape != (self.P,):
            raise GadError(-1, "parameter vector has the wrong length")
        self._ck(self._L.gad_set_params(self._h, C.c_int32(k), _ptr(p, C.c_float)))

    def get_grads(self, k):
        out = np.zeros(self.P, dtype=np.float32)
        self._ck(self._L.gad_get_grads(self._h, C.c_int32(k), _ptr(out, C.c_float)))
        return out

    def get_store(self):
        rowptr = np.zeros(self.n_prime + 1, dtype=np.int64)
        col = np.zeros(self.nnz_prime, dtype=np.int32)
        val = np.zeros(self.nnz_prime, dtype=np.float32)
        sub_off = np.zeros(self.K + 1, dtype=np.int32)
        gid = np.zeros(self.n_prime, dtype=np.int32)
        deg = np.zeros(self.n_prime, dtype=np.int32)
        self._ck(self._L.gad_get_store(self._h, _ptr(rowptr, C.c_int64), _ptr(col, C.c_int32), _ptr(val, C.c_float),
                                       _ptr(sub_off, C.c_int32), _ptr(gid, C.c_int32), _ptr(deg, C.c_int32)))
        return dict(rowptr=rowptr, col=col, val=val, sub_off=sub_off, gid=gid, deg=deg)

    def get_activation(self, l):
        out = np.zeros((self.n_prime, self.dims[l]), dtype=np.float32)
        self._ck(self._L.gad_get_activation(self._h, C.c_int32(l), _ptr(out, C.c_float)))
        return out

    def set_inputs(self, X=None, labels=None):
        """gad_set_inputs.  X / labels may be numpy arrays or (pinned) CPU torch tensors; they must stay alive
        until the stream has consumed them."""
        def host_ptr(a, ctype, np_dtype):
            if a is None:
                return None, None
            if hasattr(a, "data_ptr"):
                return a, C.cast(C.c_void_p(a.data_ptr()), C.POINTER(ctype))
            a = _arr(a, np_dtype)
            return a, _ptr(a, ctype)
        kx, px = host_ptr(X, C.c_float, np.float32)
        kl, pl = host_ptr(labels, C.c_int32, np.int32)
        self._keep = (kx, kl)
        self._ck(self._L.gad_set_inputs(self._h, px, pl))

    @property
    def epoch(self):
        e = C.c_int64(0)
        self._ck(self._L.gad_get_epoch(self._h, C.byref(e)))
        return int(e.value)

    @epoch.setter
    def epoch(self, e):
        self._ck(self._L.gad_set_epoch(self._h, C.c_int64(e)))

    def check_store(self):
        """gad_check_store: every index of the device store and its work lists tested against its range; returns the
        number of violations (0) or raises."""
        v = C.c_int64(0)
        self._ck(self._L.gad_check_store(self._h, C.byref(v)))
        return int(v.value)

    def debug_expire_wait(self, polls=1000):
        """gad_debug_expire_wait: makes one bounded device-side wait run out (for testing the time-out path)."""
        self._ck(self._L.gad_debug_expire_wait(self._h, C.c_uint32(polls)))

    # -- profiling -----------------------------------------------------------------------------
    def profile_enable(self, on=True):
        self._ck(self._L.gad_profile_enable(self._h, C.c_int32(1 if on else 0)))

    def profile_reset(self):
        self._ck(self._L.gad_profile_reset(self._h))

    def profile_read(self):
        """List of dicts: name, launches, total_ms, bytes_per_launch, flops_per_launch."""
        cnt = C.c_int32(0)
        self._ck(self._L.gad_profile_count(self._h, C.byref(cnt)))
        out = []
        for i in range(cnt.value):
            name = C.create_string_buffer(64)
            n, ms, by, fl = C.c_int64(0), C.c_double(0), C.c_double(0), C.c_double(0)
            self._ck(self._L.gad_profile_read(self._h, C.c_int32(i), name, C.byref(n), C.byref(ms), C.byref(by), C.byref(fl)))
            out.append(dict(name=name.value.decode(), launches=int(n.value), total_ms=float(ms.value),
                            bytes_per_launch=float(by.value), flops_per_launch=float(fl.value)))
        return out


def subgraph_weights_static(X, deg, sub_off, F, zeta_out, w_out, *, beta=1.0, weighted=True, stream=None):
    """gad_subgraph_weights_static: zeta_k and w_k without a context, a workspace or any allocation.

    For callers that may not allocate device memory (see include/gad.h).  Every argument is a CUDA torch tensor the
    caller already owns: X float32 [rows, ld] (ld a multiple of 4), deg int32 [rows], sub_off int32 [K+1], and the
    outputs zeta_out / w_out float32 [K].  The kernels are enqueued on ``stream`` (default: torch's current stream);
    the call does not wait.  Limits: K <= 256, ld <= 4096, K * ld <= 16384."""
    import torch
    if stream is None:
        stream = torch.cuda.current_stream(X.device)
    if not (X.is_cuda and X.dtype == torch.float32 and X.dim() == 2 and X.is_contiguous()):
        raise GadError(-1, "X must be a contiguous float32 CUDA matrix")
    for t, dt in ((deg, torch.int32), (sub_off, torch.int32), (zeta_out, torch.float32), (w_out, torch.float32)):
        if not (t.is_cuda and t.dtype == dt and t.is_contiguous()):
            raise GadError(-1, "deg / sub_off must be int32 and zeta_out / w_out float32 contiguous CUDA tensors")
    K = int(sub_off.numel()) - 1
    if zeta_out.numel() != K or w_out.numel() != K or deg.numel() != X.shape[0]:
        raise GadError(-1, "tensor sizes do not match")
    rc = load().gad_subgraph_weights_static(
        C.c_void_p(X.data_ptr()), C.c_int64(X.shape[0]), C.c_int32(int(F)), C.c_int32(X.shape[1]), C.c_void_p(deg.data_ptr()),
        C.c_void_p(sub_off.data_ptr()), C.c_int32(K), C.c_float(beta), C.c_int32(1 if weighted else 0),
        C.c_void_p(zeta_out.data_ptr()), C.c_void_p(w_out.data_ptr()), C.c_void_p(stream.cuda_stream))
    if rc != GAD_OK:
        raise GadError(rc, "gad_subgraph_weights_static")


def launch_count() -> int:
    """gad_launch_count: CUDA kernels launched by the library in this process so far."""
    n = C.c_int64(0)
    rc = load().gad_launch_count(C.byref(n))
    if rc != GAD_OK:
        raise GadError(rc)
    return int(n.value)


class _AugmentConfig(C.Structure):
    _fields_ = [("steps", C.c_int32), ("cap", C.c_int32), ("alpha", C.c_double), ("E", C.c_double), ("zc", C.c_double),
                ("seed", C.c_uint64), ("graph_resident", C.c_int32)]


def default_params(dims, seed=0):
    """gad_default_params: the seeded Glorot-uniform initialisation gad_create uses when it is given none (host-only)."""
    dims_a = np.asarray(dims, dtype=np.int32)
    P = int(sum(int(dims_a[l]) * int(dims_a[l + 1]) + int(dims_a[l + 1]) for l in range(len(dims_a) - 1)))
    out = np.zeros(P, dtype=np.float32)
    rc = load().gad_default_params(C.c_int32(len(dims_a) - 1), _ptr(dims_a, C.c_int32), C.c_uint64(seed), _ptr(out, C.c_float))
    if rc != GAD_OK:
        raise GadError(rc)
    return out


class Augmenter:
    """gad_augment for one graph and several calls: the device workspace is kept between calls, and from the second call
    on (same workspace, same graph) the graph is not copied to the device again (``graph_resident``)."""

    def __init__(self, n, rowptr, col):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("the GAD library needs a CUDA device (there is no CPU fallback)")
        self._L = load()
        self._L.gad_augment_last_error.restype = C.c_char_p
        self.n = int(n)
        self.rowptr = _arr(rowptr, np.int64)
        self.col = _arr(col, np.int32)
        self._csr = gad_csr(self.n, int(self.rowptr[-1]), _ptr(self.rowptr, C.c_int64), _ptr(self.col, C.c_int32), None)
        self._ws = None
        self._ws_bytes = 0
        self._resident = False

    def _fail(self, rc):
        raise GadError(rc, (self._L.gad_augment_last_error() or b"").decode())

    def run(self, cores, steps, *, alpha=0.01, E=0.05, zc=1.96, seed=0, cap=4, stream=None):
        """The replication-node list of every core set (Algorithm 1 of the paper) on the current CUDA device.
        Returns (list of int32 arrays in selection order, int64 array of the walks drawn per subgraph)."""
        import torch
        L = self._L
        K = len(cores)
        cp = np.zeros(K + 1, dtype=np.int64)
        np.cumsum([len(c) for c in cores], out=cp[1:])
        cn = _arr(np.concatenate(cores) if cp[-1] > 0 else np.empty(0, np.int32), np.int32)
        cfg = _AugmentConfig(int(steps), int(cap), float(alpha), float(E), float(zc), int(seed), 0)
        nbytes = C.c_size_t(0)
        rc = L.gad_augment_workspace_bytes(C.byref(self._csr), C.c_int32(K), _ptr(cp, C.c_int64), _ptr(cn, C.c_int32), C.byref(cfg),
                                           C.byref(nbytes))
        if rc != GAD_OK:
            self._fail(rc)
        if self._ws is None or int(nbytes.value) > self._ws_bytes:
            self._ws = torch.empty(int(nbytes.value) + 256, dtype=torch.uint8, device="cuda")
            self._ws_bytes = int(nbytes.value)
            self._resident = False
        cfg.graph_resident = 1 if self._resident else 0
        aligned = (self._ws.data_ptr() + 255) // 256 * 256
        st = stream if stream is not None else torch.cuda.current_stream()
        capacity = int(sum(int(np.floor(alpha * 2.0 * len(c))) for c in cores)) + 1
        halo_ptr = np.zeros(K + 1, dtype=np.int64)
        halo = np.zeros(capacity, dtype=np.int32)
        walks = np.zeros(K, dtype=np.int64)
        rc = L.gad_augment(C.byref(self._csr), C.c_int32(K), _ptr(cp, C.c_int64), _ptr(cn, C.c_int32), C.byref(cfg), C.c_void_p(aligned),
                           C.c_size_t(self._ws_bytes), C.c_void_p(st.cuda_stream), _ptr(halo_ptr, C.c_int64), _ptr(halo, C.c_int32),
                           C.c_int64(capacity), _ptr(walks, C.c_int64))
        if rc != GAD_OK:
            self._resident = False
            self._fail(rc)
        self._resident = True
        return [halo[halo_ptr[k]:halo_ptr[k + 1]].copy() for k in range(K)], walks


def augment(n, rowptr, col, cores, steps, *, alpha=0.01, E=0.05, zc=1.96, seed=0, cap=4, stream=None):
    """gad_augment, one call: the replication-node list of every core set (Algorithm 1 of the paper) on the current CUDA
    device.  Returns (list of int32 arrays in selection order, int64 array of the walks drawn per subgraph)."""
    return Augmenter(n, rowptr, col).run(cores, steps, alpha=alpha, E=E, zc=zc, seed=seed, cap=cap, stream=stream)


def from_workload(w, init_params, **kw):
    """A context for a ``gad_synth.Workload``."""
    cp, cn, hp, hn = w.flat_partition()
    kw.setdefault("lr", w.lr)
    return Gad(w.n, w.rowptr, w.col, cp, cn, hp, hn, w.X, w.labels, w.split, w.dims, init_params=init_params, **kw)
