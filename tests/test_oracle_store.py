"""Pins for the oracle's block-diagonal store of the augmented subgraphs.

The expected values come from dense matrices built straight from the definitions
(g'_i = (v_i + v'_i, e_i + e'_i), Algorithm 1; A~ = D~^-1/2 (A + I) D~^-1/2, Section 3.3),
not from the oracle's own row-by-row routine.
"""
import numpy as np
import pytest

from oracle import gad_oracle as orc
from conftest import small_random_case, flat


def dense_graph(n, rowptr, col, w):
    A = np.zeros((n, n))
    for u in range(n):
        for e in range(rowptr[u], rowptr[u + 1]):
            A[u, col[e]] += 1.0 if w is None else float(w[e])
    return A


def dense_hat(A, idx):
    """Normalised adjacency of the subgraph induced on idx, self-loop added where missing."""
    S = A[np.ix_(idx, idx)].copy()
    for i in range(len(idx)):
        if S[i, i] == 0.0:
            S[i, i] = 1.0
    d = S.sum(axis=1)
    return S / np.sqrt(np.outer(d, d)), d


def store_block(st, k):
    r0, r1 = int(st.sub_off[k]), int(st.sub_off[k + 1])
    B = np.zeros((r1 - r0, r1 - r0))
    for r in range(r0, r1):
        for e in range(st.rowptr[r], st.rowptr[r + 1]):
            c = st.col[e]
            assert r0 <= c < r1, "column leaves its diagonal block"
            assert B[r - r0, c - r0] == 0.0, "duplicate column in a row"
            B[r - r0, c - r0] = st.val[e]
        cols = st.col[st.rowptr[r]:st.rowptr[r + 1]]
        assert np.all(np.diff(cols) > 0), "columns not strictly ascending"
    return B


@pytest.mark.parametrize("seed,directed,weighted", [(0, False, False), (1, False, True), (2, True, False),
                                                     (3, True, True)])
def test_store_matches_dense_definition(seed, directed, weighted):
    n, rowptr, col, w, core, halo = small_random_case(seed, directed=directed, weighted=weighted)
    cp, cn = flat(core)
    hp, hn = flat(halo)
    st = orc.Store(n, rowptr, col, cp, cn, hp, hn, weights=w)
    A = dense_graph(n, rowptr, col, w)
    assert st.n_prime == sum(len(c) + len(h) for c, h in zip(core, halo))
    row = 0
    for k in range(len(core)):
        idx = np.concatenate([core[k], halo[k]])
        assert np.array_equal(st.gid[row:row + len(idx)], idx)
        assert st.sub_off[k] == row
        hat, d = dense_hat(A, idx)
        B = store_block(st, k)
        assert np.allclose(B, hat, rtol=1e-14, atol=0)
        assert np.array_equal(B != 0, hat != 0)
        # sqrt(d~) is an eigenvector of A~ with eigenvalue 1 when A~ is built from row sums
        if not directed:
            assert np.allclose(B @ np.sqrt(d), np.sqrt(d), rtol=1e-12)
            assert np.allclose(B, B.T, rtol=1e-14)
        # local degree = distinct neighbours inside the subgraph, self excluded
        sub = A[np.ix_(idx, idx)] != 0
        np.fill_diagonal(sub, False)
        assert np.array_equal(st.deg[row:row + len(idx)], sub.sum(axis=1))
        row += len(idx)
    assert st.sub_off[-1] == st.n_prime
    assert st.rowptr[-1] == st.nnz


def test_parallel_edges_are_summed_and_self_loops_not_doubled():
    # node 0 -- node 1 listed twice (weights 1 and 2), node 0 has a self-loop of weight 3, node 1 has none
    rowptr = np.array([0, 3, 4], dtype=np.int64)
    col = np.array([1, 0, 1, 0], dtype=np.int32)
    w = np.array([1.0, 3.0, 2.0, 3.0], dtype=np.float32)
    st = orc.Store(2, rowptr, col, *flat([np.array([0, 1], dtype=np.int32)]), *flat([np.empty(0, np.int32)]), weights=w)
    S = np.array([[3.0, 3.0], [3.0, 1.0]])
    d = S.sum(axis=1)
    assert np.allclose(store_block(st, 0), S / np.sqrt(np.outer(d, d)))
    assert list(st.deg) == [1, 1]


def test_store_rejects_bad_partitions():
    n, rowptr, col, w, core, halo = small_random_case(5)
    cp, cn = flat(core)
    bad = [h.copy() for h in halo]
    bad[0] = np.concatenate([bad[0], core[0][:1]])          # a replicated node that is also a core node
    with pytest.raises(ValueError):
        orc.Store(n, rowptr, col, cp, cn, *flat(bad))
    bad = [h.copy() for h in halo]
    bad[1] = np.concatenate([bad[1], np.array([n], dtype=np.int32)])   # out of range
    with pytest.raises(ValueError):
        orc.Store(n, rowptr, col, cp, cn, *flat(bad))


def test_empty_subgraph_and_isolated_node():
    # 3 nodes, no edges; subgraph 1 is empty
    rowptr = np.zeros(4, dtype=np.int64)
    col = np.empty(0, dtype=np.int32)
    core = [np.array([2, 0], dtype=np.int32), np.empty(0, np.int32), np.array([1], dtype=np.int32)]
    halo = [np.empty(0, np.int32)] * 3
    st = orc.Store(3, rowptr, col, *flat(core), *flat(halo))
    assert list(st.sub_off) == [0, 2, 2, 3]
    assert st.nnz == 3 and np.allclose(st.val, 1.0)       # only the added self-loops, A~ = I
    assert list(st.col) == [0, 1, 2]
    assert list(st.deg) == [0, 0, 0]


def test_tiny_workload_bookkeeping(tiny):
    cp, cn, hp, hn = tiny.flat_partition()
    st = orc.Store(tiny.n, tiny.rowptr, tiny.col, cp, cn, hp, hn)
    assert st.n_prime == cn.size + hn.size
    assert st.K == 4
    # every stored value is 1/sqrt(d_i d_j) for an unweighted graph
    d = np.zeros(st.n_prime)
    np.add.at(d, np.repeat(np.arange(st.n_prime), np.diff(st.rowptr)), 1.0)
    rows = np.repeat(np.arange(st.n_prime), np.diff(st.rowptr))
    assert np.allclose(st.val, 1.0 / np.sqrt(d[rows] * d[st.col]), rtol=1e-14)
