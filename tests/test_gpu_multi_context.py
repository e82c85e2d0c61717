"""GPU parity of Algorithm 2 with the subgraphs spread over several contexts (gad_train_epoch_local,
gad_consensus_partial, gad_consensus_apply, gad_export_params), through the C ABI, against the oracle.  Two contexts
on the one GPU stand for two GPUs: they run one after the other, and a tensor addition stands for the all-reduce."""
import numpy as np
import pytest

import __graft_entry__ as entry
from gad_synth import glorot_params
from conftest import small_random_case, flat, rel_err

pytestmark = pytest.mark.gpu
TOL = 1e-4
DIMS = (24, 40, 5)


@pytest.fixture(scope="module", autouse=True)
def built():
    entry.build()


def _inputs(case, seed=7):
    n = case[0]
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((n, DIMS[0])).astype(np.float32)
    y = rng.integers(0, DIMS[-1], size=n).astype(np.int32)
    split = rng.integers(0, 3, size=n).astype(np.uint8)
    return X, y, split, glorot_params(DIMS, rng, bias_scale=0.2)


def _gad(case, subgraphs, X, y, split, theta, **kw):
    import paper_2110_02987_b200 as pkg
    n, rowptr, col, w, core, halo = case
    cp, cn = flat([core[k] for k in subgraphs])
    hp, hn = flat([halo[k] for k in subgraphs])
    return pkg.Gad(n, rowptr, col, cp, cn, hp, hn, X, y, split, DIMS, init_params=theta, weights=w, **kw)


def _oracle(case, subgraphs, X, y, split, theta, **kw):
    from oracle import gad_oracle as orc
    n, rowptr, col, w, core, halo = case
    cp, cn = flat([core[k] for k in subgraphs])
    hp, hn = flat([halo[k] for k in subgraphs])
    st = orc.Store(n, rowptr, col, cp, cn, hp, hn, weights=w)
    return orc.Model(st, X, y, split, DIMS, theta, **kw)


@pytest.mark.parametrize("weighted", [True, False])
def test_two_contexts_add_up_to_the_consensus_over_all_subgraphs(weighted):
    case = small_random_case(41, n=300, K=5, p=0.03)
    X, y, split, theta = _inputs(case)
    ref = _oracle(case, range(5), X, y, split, theta, lr=0.2, weighted=weighted)
    parts = [[0, 2, 4], [1, 3]]
    with _gad(case, parts[0], X, y, split, theta, lr=0.2, weighted=weighted) as a, \
            _gad(case, parts[1], X, y, split, theta, lr=0.2, weighted=weighted) as b, \
            _gad(case, range(5), X, y, split, theta, lr=0.2, weighted=weighted) as whole:
        zeta_total = float(sum(np.sum(g.subgraph_weights()[0].astype(np.float64)) for g in (a, b))) if weighted else 5.0
        bufs = [a.new_consensus_buffer(), b.new_consensus_buffer()]
        for _ in range(3):
            la, lb = a.train_epoch_local(), b.train_epoch_local()
            a.consensus_partial(zeta_total, bufs[0])
            b.consensus_partial(zeta_total, bufs[1])
            total = bufs[0] + bufs[1]                 # the all-reduce
            a.consensus_apply(total)
            b.consensus_apply(total)
            lw = whole.train_epoch()
            lr_ = ref.train_epoch()
            got = np.zeros(5)
            got[parts[0]], got[parts[1]] = la[:-1], lb[:-1]
            assert np.max(np.abs(got - lr_[:-1])) <= 1e-4
            assert np.max(np.abs(got - lw[:-1])) <= 1e-5
        want = ref.get_params(0)
        for g in (a, b):
            for k in range(g.K):
                assert rel_err(g.get_params(k), want) <= TOL
                assert rel_err(g.get_params(k), whole.get_params(0)) <= 1e-5    # same arithmetic, another grouping of the sum
        nt = np.concatenate([a.ntrain(), b.ntrain()])
        assert np.array_equal(np.sort(nt), np.sort(ref.ntrain()))


def test_sharded_epoch_on_one_rank_equals_the_fused_epoch():
    import paper_2110_02987_b200 as pkg
    case = small_random_case(42, n=300, K=4, p=0.03)
    X, y, split, theta = _inputs(case)
    with _gad(case, range(4), X, y, split, theta, lr=0.2) as a, _gad(case, range(4), X, y, split, theta, lr=0.2) as b:
        sh = pkg.ShardedEpoch(a)
        for _ in range(3):
            loss = sh.step()
            want = b.train_epoch()
            assert abs(loss - float(want[-1])) <= 1e-5
        for k in range(4):
            assert rel_err(a.get_params(k), b.get_params(k)) <= 1e-5


def test_rounds_on_the_gpu_against_the_oracle():
    import paper_2110_02987_b200 as pkg
    case = small_random_case(43, n=300, K=4, p=0.03)
    X, y, split, theta = _inputs(case)
    oa = _oracle(case, [0, 1], X, y, split, theta, lr=0.2)
    ob = _oracle(case, [2, 3], X, y, split, theta, lr=0.2)
    with _gad(case, [0, 1], X, y, split, theta, lr=0.2) as a, _gad(case, [2, 3], X, y, split, theta, lr=0.2) as b:
        rounds = pkg.RoundsEpoch([a, b])
        for _ in range(2):
            got = rounds.step()
            la = oa.train_epoch()
            for k in range(2):
                ob.set_params(k, oa.get_params(0))
            lb = ob.train_epoch()
            for k in range(2):
                oa.set_params(k, ob.get_params(0))
            assert np.max(np.abs(got[0] - la)) <= 1e-4 and np.max(np.abs(got[1] - lb)) <= 1e-4
        for k in range(2):
            assert rel_err(a.get_params(k), oa.get_params(k)) <= TOL
            assert rel_err(b.get_params(k), ob.get_params(k)) <= TOL
        assert np.array_equal(a.get_params(0), b.get_params(1))      # the hand-over is an exact copy


def test_consensus_of_the_parameters_as_they_are():
    """with_step = 0: the share of a plain consensus; with one context and its own total it must equal gad_consensus."""
    case = small_random_case(44, n=200, K=3, p=0.04)
    X, y, split, theta = _inputs(case)
    rng = np.random.default_rng(3)
    with _gad(case, range(3), X, y, split, theta) as a, _gad(case, range(3), X, y, split, theta) as b:
        for k in range(3):
            p = (theta + rng.standard_normal(theta.shape[0]) * 0.1).astype(np.float32)
            a.set_params(k, p)
            b.set_params(k, p)
        zeta_total = float(np.sum(a.subgraph_weights()[0].astype(np.float64)))
        buf = a.new_consensus_buffer()
        a.consensus_partial(zeta_total, buf, with_step=False)
        a.consensus_apply(buf)
        b.consensus()
        for k in range(3):
            assert rel_err(a.get_params(k), b.get_params(0)) <= 1e-6
