"""Pins for the variance-based importance weight (Section 3.4.1) and the weighted global consensus
(Definition 3, Section 3.4.2)."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import gad_oracle as orc
from gad_synth import glorot_params
from conftest import flat, rel_err
from test_oracle_gcn import make_case

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "zeta_example.txt")


def golden_rows():
    rows = []
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        fig, val, seq = line.split()
        rows.append((fig, float(val), [int(t) for t in seq.split(",")]))
    return rows


@pytest.mark.parametrize("fig,printed,degs", golden_rows())
def test_paper_worked_example(fig, printed, degs):
    # all pairwise distances are zero in the example: identical feature vectors
    X = np.full((len(degs), 3), 0.7)
    for fn in (orc.zeta_aggregate, orc.zeta_pairwise):
        z = fn(degs, X, beta=1.0)
        assert round(10 * z, 2) == printed, (fig, fn.__name__, z)
    # exact rational value of sum_{i<j} p_i p_j
    tot = sum(degs)
    exact = sum(Fraction(degs[i], tot) * Fraction(degs[j], tot) for i in range(4) for j in range(i + 1, 4))
    assert abs(orc.zeta_aggregate(degs, X) - float(exact)) < 1e-15


def test_printed_order_of_the_example():
    rows = {fig: orc.zeta_aggregate(degs, np.zeros((4, 1))) for fig, _, degs in golden_rows()}
    assert rows["4.a"] > rows["4.c"] > rows["4.b"]


@pytest.mark.parametrize("n", [2, 5, 64])
def test_property2_equal_probabilities_maximise_the_pair_sum(n):
    X = np.zeros((n, 2))
    best = orc.zeta_aggregate(np.full(n, 3), X)
    assert abs(best - (n - 1) / (2.0 * n)) < 1e-15
    rng = np.random.default_rng(n)
    for _ in range(20):
        deg = rng.integers(1, 9, size=n)
        assert orc.zeta_aggregate(deg, X) <= best + 1e-15


def test_closed_forms_match_the_pair_definitions():
    rng = np.random.default_rng(0)
    n, F = 150, 7
    deg = rng.integers(0, 12, size=n)
    X = rng.standard_normal((n, F)) * rng.uniform(0.1, 3.0, size=F) + rng.uniform(-5, 5, size=F)
    S, Q = orc.zeta_pair_sums(deg, X)
    # numpy restatement of the two pair sums, independent of the C loops
    p = deg / deg.sum()
    iu, ju = np.triu_indices(n, 1)
    d2 = ((X[iu] - X[ju]) ** 2).sum(axis=1)
    assert abs(S - (p[iu] * p[ju]).sum()) < 1e-14
    assert abs(Q - (p[iu] * p[ju] * d2).sum()) < 1e-11
    want = S / (np.sqrt(Q / S) + 1.0)
    assert abs(orc.zeta_aggregate(deg, X) - want) < 1e-13
    lit = (p[iu] * p[ju] / (np.sqrt(d2) + 1.0)).sum()
    assert abs(orc.zeta_pairwise(deg, X) - lit) < 1e-13


def test_pairwise_reading_dominates_aggregate_reading_and_they_meet_on_equal_distances():
    rng = np.random.default_rng(1)
    for n in (2, 3, 30):
        deg = rng.integers(1, 6, size=n)
        X = rng.standard_normal((n, 4))
        assert orc.zeta_pairwise(deg, X) >= orc.zeta_aggregate(deg, X) - 1e-15
    # two nodes: a single pair, both readings are p_0 p_1 / (d + beta)
    X = np.array([[0.0, 0.0], [3.0, 4.0]])
    z = orc.zeta_aggregate([1, 3], X, beta=0.5)
    assert abs(z - (0.25 * 0.75) / (5.0 + 0.5)) < 1e-15
    assert abs(orc.zeta_pairwise([1, 3], X, beta=0.5) - z) < 1e-15
    # regular simplex: all pairwise distances sqrt(2)
    X = np.eye(5)
    deg = [1, 2, 3, 4, 5]
    assert abs(orc.zeta_pairwise(deg, X) - orc.zeta_aggregate(deg, X)) < 1e-15


def test_degenerate_subgraphs():
    assert orc.zeta_aggregate([0], np.ones((1, 3))) == 0.0            # a single node has no pair
    z = orc.zeta_aggregate([0, 0, 0], np.zeros((3, 2)))              # no edges: uniform p
    assert abs(z - 1.0 / 3.0) < 1e-15


def test_translation_and_large_offsets_do_not_change_zeta():
    rng = np.random.default_rng(2)
    deg = rng.integers(1, 7, size=40)
    X = rng.standard_normal((40, 5))
    assert abs(orc.zeta_aggregate(deg, X) - orc.zeta_aggregate(deg, X + 1e4)) < 1e-9


def _model(seed=0, K_identical=False, **kw):
    dims = (6, 5, 3)
    n, rowptr, col, w, core, halo, X, y, split, theta, st = make_case(seed, dims)
    return orc.Model(st, X, y, split, dims, theta, **kw), theta


def test_weights_sum_to_one_and_follow_zeta():
    m, _ = _model(0)
    z, w = m.subgraph_weights()
    assert abs(w.sum() - 1.0) < 1e-15
    assert np.allclose(w, z / z.sum(), rtol=1e-15)
    assert len(set(np.round(z, 12))) > 1
    m2, _ = _model(0, weighted=False)
    assert np.allclose(m2.subgraph_weights()[1], 1.0 / m2.K)


def test_consensus_is_weighted_mean_idempotent_and_identity_for_one_replica():
    m, theta = _model(1)
    rng = np.random.default_rng(0)
    copies = [theta.astype(np.float64) + rng.standard_normal(theta.size) for _ in range(m.K)]
    for k in range(m.K):
        m.set_params(k, copies[k])
    _, w = m.subgraph_weights()
    m.consensus()
    want = sum(w[k] * copies[k] for k in range(m.K))
    for k in range(m.K):
        assert rel_err(m.get_params(k), want) < 1e-15
    once = m.get_params(0).copy()
    m.consensus()
    assert rel_err(m.get_params(0), once) < 1e-15
    # one replica: the consensus changes nothing
    dims = (6, 5, 3)
    n, rowptr, col, wgt, core, halo, X, y, split, theta, _ = make_case(2, dims)
    st = orc.Store(n, rowptr, col, *flat([np.arange(n, dtype=np.int32)]), *flat([np.empty(0, np.int32)]))
    one = orc.Model(st, X, y, split, dims, theta)
    p = one.get_params(0).copy()
    one.consensus()
    assert np.array_equal(one.get_params(0), p)
    assert one.subgraph_weights()[1][0] == 1.0


def test_equal_importance_gives_the_plain_average_of_definition_3():
    # two identical subgraphs => equal zeta => weights 1/2 => plain average
    rng = np.random.default_rng(3)
    n0 = 10
    A = np.triu(rng.random((n0, n0)) < 0.4, 1)
    A = A | A.T
    big = np.zeros((2 * n0, 2 * n0), dtype=bool)
    big[:n0, :n0] = A
    big[n0:, n0:] = A
    src, dst = np.nonzero(big)
    rowptr = np.zeros(2 * n0 + 1, dtype=np.int64)
    np.cumsum(np.bincount(src, minlength=2 * n0), out=rowptr[1:])
    X0 = rng.standard_normal((n0, 4)).astype(np.float32)
    X = np.vstack([X0, X0])
    dims = (4, 3)
    core = [np.arange(n0, dtype=np.int32), np.arange(n0, 2 * n0, dtype=np.int32)]
    st = orc.Store(2 * n0, rowptr, dst.astype(np.int32), *flat(core), *flat([np.empty(0, np.int32)] * 2))
    theta = glorot_params(dims, rng)
    m = orc.Model(st, X, np.zeros(2 * n0, np.int32), np.zeros(2 * n0, np.uint8), dims, theta)
    z, w = m.subgraph_weights()
    assert z[0] == z[1] and np.allclose(w, 0.5)
    a, b = rng.standard_normal(m.P), rng.standard_normal(m.P)
    m.set_params(0, a)
    m.set_params(1, b)
    m.consensus()
    assert rel_err(m.get_params(0), (a + b) / 2) < 1e-15


def test_parameter_consensus_equals_weighted_gradient_step():
    # from identical copies: sum_k w_k (theta - eta g_k) = theta - eta sum_k w_k g_k  (Section 3.4.2)
    m, theta = _model(4, lr=0.05)
    m.forward_backward()
    g = [m.get_grads(k) for k in range(m.K)]
    _, w = m.subgraph_weights()
    want = theta.astype(np.float64) - 0.05 * sum(w[k] * g[k] for k in range(m.K))
    m2, _ = _model(4, lr=0.05)
    m2.train_epoch()
    for k in range(m2.K):
        assert rel_err(m2.get_params(k), want) < 1e-12


def test_layer_sum_reading_against_pair_loops_over_every_layer():
    """zeta_mode 2 keeps the sum over the layers of the variance equation.  Pinned against O(n^2) pair loops written
    here: S from the degrees, and the p-weighted squared distances added up layer by layer over the activations the
    forward pass left (one loop nest per layer, not the concatenation the oracle forms)."""
    dims = (6, 5, 4, 3)
    n, rowptr, col, w, core, halo, X, y, split, theta, st = make_case(8, dims, n=36, K=2)
    m = orc.Model(st, X, y, split, dims, theta, zeta_mode=2, beta=0.7)
    m.forward()
    zeta, wts = m.subgraph_weights()
    acts = [m.activation(l) for l in range(len(dims) - 1)]
    for k in range(st.K):
        r0, r1 = int(st.sub_off[k]), int(st.sub_off[k + 1])
        deg = st.deg[r0:r1].astype(np.float64)
        p = deg / deg.sum() if deg.sum() > 0 else np.full(r1 - r0, 1.0 / (r1 - r0))
        S = Q = 0.0
        for i in range(r1 - r0):
            for j in range(i + 1, r1 - r0):
                S += p[i] * p[j]
                for H in acts:
                    d = H[r0 + i] - H[r0 + j]
                    Q += p[i] * p[j] * float(d @ d)
        want = S / (np.sqrt(Q / S) + 0.7)
        assert abs(zeta[k] - want) <= 1e-12 * want
    assert abs(wts.sum() - 1.0) < 1e-15


def test_layer_sum_reading_with_one_layer_is_the_aggregate_reading():
    dims = (6, 3)
    n, rowptr, col, w, core, halo, X, y, split, theta, st = make_case(9, dims)
    a = orc.Model(st, X, y, split, dims, theta, zeta_mode=0)
    b = orc.Model(st, X, y, split, dims, theta, zeta_mode=2)
    for _ in range(2):
        assert np.array_equal(a.train_epoch(), b.train_epoch())
    assert np.array_equal(a.get_params(0), b.get_params(0))
    assert np.array_equal(a.subgraph_weights()[0], b.subgraph_weights()[0])


def test_layer_sum_reading_changes_with_the_model():
    """With hidden layers the weights follow the activations: they differ from the input-only reading and move as
    the parameters move (the input-only weights never do)."""
    dims = (6, 5, 3)
    n, rowptr, col, w, core, halo, X, y, split, theta, st = make_case(10, dims)
    a = orc.Model(st, X, y, split, dims, theta, zeta_mode=0, lr=0.5)
    b = orc.Model(st, X, y, split, dims, theta, zeta_mode=2, lr=0.5)
    b.train_epoch(); a.train_epoch()
    z0, zb0 = a.subgraph_weights()[0].copy(), b.subgraph_weights()[0].copy()
    assert np.all(zb0 < z0)            # more squared distance in the denominator
    b.train_epoch(); a.train_epoch()
    assert np.array_equal(a.subgraph_weights()[0], z0)
    assert not np.array_equal(b.subgraph_weights()[0], zb0)
