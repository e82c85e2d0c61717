import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def rel_err(a, b) -> float:
    """Per-tensor error used by every parity check: max|a-b| / max(max|b|, 1e-30)."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    if a.size == 0:
        return 0.0
    return float(np.max(np.abs(a - b)) / max(float(np.max(np.abs(b))), 1e-30))


@pytest.fixture(scope="session")
def tiny():
    from gad_synth import make_workload
    return make_workload("tiny")


@pytest.fixture(scope="session")
def tiny_signal():
    from gad_synth import make_workload
    return make_workload("tiny_signal")


def small_random_case(seed, n=40, K=3, p=0.15, directed=False, weighted=False, halo=True):
    """A small random graph with an arbitrary (non-contiguous, partly uncovered) partition."""
    rng = np.random.default_rng(seed)
    A = rng.random((n, n)) < p
    if not directed:
        A = np.triu(A, 1)
        A = A | A.T
    np.fill_diagonal(A, rng.random(n) < 0.3)       # some nodes already carry a self-loop
    src, dst = np.nonzero(A)
    rowptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(np.bincount(src, minlength=n), out=rowptr[1:])
    col = dst.astype(np.int32)
    w = None
    if weighted:
        Wm = rng.uniform(0.5, 2.0, size=(n, n))
        if not directed:
            Wm = (Wm + Wm.T) / 2
        w = Wm[src, dst].astype(np.float32)
    perm = rng.permutation(n)
    covered = perm[: n - 3]                          # three nodes belong to no subgraph
    core = [np.sort(c).astype(np.int32)[::-1].copy() for c in np.array_split(covered, K)]
    halos = []
    for c in core:
        others = np.setdiff1d(np.arange(n), c)
        take = rng.permutation(others)[: (4 if halo else 0)]
        halos.append(take.astype(np.int32))
    return n, rowptr, col, w, core, halos


def flat(lists):
    ptr = np.zeros(len(lists) + 1, dtype=np.int64)
    np.cumsum([len(a) for a in lists], out=ptr[1:])
    nodes = np.concatenate(lists).astype(np.int32) if ptr[-1] > 0 else np.empty(0, dtype=np.int32)
    return ptr, nodes
