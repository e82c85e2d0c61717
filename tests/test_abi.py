"""CPU checks of the boundary: the library loads, exports every declared symbol, and its host-side
validation (reached through gad_workspace_bytes, which touches no GPU) rejects malformed inputs."""
import os
import re

import numpy as np
import pytest

import __graft_entry__ as entry
import paper_2110_02987_b200 as pkg
from paper_2110_02987_b200 import GadError, gad_workspace_bytes
from conftest import small_random_case, flat

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    entry.build()


def test_library_exports_every_symbol_the_header_declares():
    text = open(os.path.join(ROOT, "include", "gad.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(gad_[a-z_]+)\s*\(", text))
    assert declared == set(pkg.SYMBOLS)
    lib = pkg.load()
    for name in declared:
        assert getattr(lib, name) is not None


def _ws(case, dims=(6, 5, 3), **kw):
    n, rowptr, col, w, core, halo = case
    return gad_workspace_bytes(n, rowptr, col, *flat(core), *flat(halo), dims, **kw)


def test_workspace_bytes_is_host_only_and_grows_with_the_problem():
    a = _ws(small_random_case(0))
    b = _ws(small_random_case(0), dims=(6, 50, 3))
    c = _ws(small_random_case(0, n=80))
    assert a > 0 and b > a and c > a and a % 256 == 0


def test_malformed_inputs_are_rejected_on_the_host():
    n, rowptr, col, w, core, halo = small_random_case(1)
    bad = col.copy(); bad[3] = n
    with pytest.raises(GadError) as e:
        _ws((n, rowptr, bad, w, core, halo))
    assert e.value.code == -2
    rp = rowptr.copy(); rp[5], rp[6] = rp[6] + 1, rp[5]
    with pytest.raises(GadError) as e:
        _ws((n, rp, col, w, core, halo))
    assert e.value.code in (-3, -1)
    dup = [c.copy() for c in core]; dup[1] = np.concatenate([dup[1], core[0][:1]])
    with pytest.raises(GadError) as e:
        _ws((n, rowptr, col, w, dup, halo))
    assert e.value.code == -4
    h2 = [h.copy() for h in halo]; h2[0] = np.concatenate([h2[0], core[0][:1]])
    with pytest.raises(GadError) as e:
        _ws((n, rowptr, col, w, core, h2))
    assert e.value.code == -4
    h3 = [h.copy() for h in halo]; h3[2] = np.concatenate([h3[2], np.array([-1], dtype=np.int32)])
    with pytest.raises(GadError) as e:
        _ws((n, rowptr, col, w, core, h3))
    assert e.value.code == -2
    for kw, code in ((dict(dropout=1.0), -1), (dict(zeta_mode=3), -1), (dict(gemm_mode=7), -1), (dict(beta=0.0), -1)):
        with pytest.raises(GadError) as e:
            _ws((n, rowptr, col, w, core, halo), **kw)
        assert e.value.code == code
    with pytest.raises(GadError):
        _ws((n, rowptr, col, w, core, halo), dims=(6, 0, 3))


def test_compute_calls_fail_loudly_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    n, rowptr, col, w, core, halo = small_random_case(2)
    with pytest.raises(RuntimeError):
        pkg.Gad(n, rowptr, col, *flat(core), *flat(halo), np.zeros((n, 6), np.float32), np.zeros(n, np.int32),
                np.zeros(n, np.uint8), (6, 5, 3))


def test_augment_arguments_are_checked_on_the_host():
    import ctypes as C
    from paper_2110_02987_b200 import binding as b
    L = pkg.load()
    n, rowptr, col, w, core, halo = small_random_case(4)
    cp, cn = flat(core)
    rowptr = np.ascontiguousarray(rowptr, np.int64); col = np.ascontiguousarray(col, np.int32)
    csr = b.gad_csr(int(n), int(rowptr[-1]), b._ptr(rowptr, C.c_int64), b._ptr(col, C.c_int32), None)

    def ws(steps=2, cap=4, alpha=0.01, E=0.05, zc=1.96, nodes=cn, graph=csr):
        cfg = b._AugmentConfig(steps, cap, alpha, E, zc, 0)
        out = C.c_size_t(0)
        rc = L.gad_augment_workspace_bytes(C.byref(graph), C.c_int32(len(core)), b._ptr(cp, C.c_int64), b._ptr(nodes, C.c_int32),
                                           C.byref(cfg), C.byref(out))
        return rc, out.value

    rc, nbytes = ws()
    assert rc == 0 and nbytes > 0 and nbytes % 256 == 0
    assert ws(steps=0)[0] == -1 and ws(steps=9)[0] == -1 and ws(cap=0)[0] == -1 and ws(E=0.0)[0] == -1 and ws(alpha=-1.0)[0] == -1
    bad = cn.copy(); bad[0] = n
    assert ws(nodes=bad)[0] == -2
    assert ws(cap=8)[1] > nbytes                      # room for more walks
    # the caller's CSR is checked like gad_create checks it: the kernels index with its values
    badcol = col.copy(); badcol[2] = n
    assert ws(graph=b.gad_csr(int(n), int(rowptr[-1]), b._ptr(rowptr, C.c_int64), b._ptr(badcol, C.c_int32), None))[0] == -2
    badcol[2] = -1
    assert ws(graph=b.gad_csr(int(n), int(rowptr[-1]), b._ptr(rowptr, C.c_int64), b._ptr(badcol, C.c_int32), None))[0] == -2
    rp = rowptr.copy(); rp[5], rp[6] = rp[6] + 1, rp[5]
    assert ws(graph=b.gad_csr(int(n), int(rowptr[-1]), b._ptr(rp, C.c_int64), b._ptr(col, C.c_int32), None))[0] == -3
    assert ws(graph=b.gad_csr(int(n), int(rowptr[-1]) + 1, b._ptr(rowptr, C.c_int64), b._ptr(col, C.c_int32), None))[0] == -1


def test_default_initialisation_is_seeded_glorot_uniform():
    """gad_default_params (what gad_create uses when no parameters are passed in): every weight inside the Glorot range
    of its layer, spread over it like a uniform variable, biases zero, a pure function of the seed."""
    dims = (40, 64, 7)
    a = pkg.default_params(dims, seed=3)
    assert np.array_equal(a, pkg.default_params(dims, seed=3))
    assert not np.array_equal(a, pkg.default_params(dims, seed=4))
    o = 0
    for fi, fo in zip(dims[:-1], dims[1:]):
        W, b = a[o:o + fi * fo], a[o + fi * fo:o + fi * fo + fo]
        o += fi * fo + fo
        lim = np.sqrt(6.0 / (fi + fo))
        assert np.all(np.abs(W) < lim) and np.all(b == 0.0)
        assert abs(W.mean()) < 4 * lim / np.sqrt(3 * W.size)            # mean 0, variance lim^2 / 3
        assert abs(W.var() - lim * lim / 3) < 0.1 * lim * lim / 3
        assert np.unique(W).size > 0.99 * W.size
    assert o == a.size
    with pytest.raises(GadError):
        pkg.default_params((4, 0, 2))
