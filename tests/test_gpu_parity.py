"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element, on the same
seeded inputs.  Tolerances: integer bookkeeping bit-exact; floating-point tensors (logits, gradients,
parameters) max|a-b| / max|b| <= 1e-4 in fp32 mode; the 10-epoch loss curve within 1e-3."""
import numpy as np
import pytest

import __graft_entry__ as entry
from gad_synth import make_workload, glorot_params
from conftest import small_random_case, flat, rel_err

pytestmark = pytest.mark.gpu

TOL = 1e-4
LOSS_TOL = 1e-3


@pytest.fixture(scope="module", autouse=True)
def built():
    entry.build()


def pkg():
    import paper_2110_02987_b200 as p
    return p


def orc():
    from oracle import gad_oracle
    return gad_oracle


def make_pair(case, dims, seed=0, X=None, **kw):
    n, rowptr, col, w, core, halo = case
    rng = np.random.default_rng(1000 + seed)
    if X is None:
        X = rng.standard_normal((n, dims[0])).astype(np.float32)
    y = rng.integers(0, dims[-1], size=n).astype(np.int32)
    split = rng.integers(0, 3, size=n).astype(np.uint8)
    theta = glorot_params(dims, rng, bias_scale=0.2)
    cp, cn = flat(core)
    hp, hn = flat(halo)
    st = orc().Store(n, rowptr, col, cp, cn, hp, hn, weights=w)
    okw = {k: v for k, v in kw.items() if k in ("lr", "dropout", "seed", "beta", "weighted", "zeta_mode")}
    ref = orc().Model(st, X, y, split, dims, theta, **okw)
    g = pkg().Gad(n, rowptr, col, cp, cn, hp, hn, X, y, split, dims, init_params=theta, weights=w, **kw)
    return g, ref, st


def check_store(g, st):
    assert g.check_store() == 0          # the library's own index check of the device store and its work lists
    s = g.get_store()
    assert np.array_equal(s["rowptr"], st.rowptr)
    assert np.array_equal(s["col"], st.col)
    assert np.array_equal(s["sub_off"], st.sub_off)
    assert np.array_equal(s["gid"], st.gid)
    assert np.array_equal(s["deg"], st.deg)
    want = st.val.astype(np.float32)
    ulp = np.abs(s["val"].view(np.int32).astype(np.int64) - want.view(np.int32).astype(np.int64))
    assert ulp.max(initial=0) <= 1


def relu_kink_units(g, ref, tol):
    """Hidden units that are zero on one side and not on the other.  A unit whose pre-activation is zero within rounding
    can land on either side of the ReLU in fp32 and in the fp64 oracle; both are valid, but the gradient path differs by
    a finite amount.  Such units must be genuine ties: magnitude at most max(1e-5, tol / 10) of the layer's largest value.
    Returns {layer: (rows, cols, on the GPU's side?)}."""
    out = {}
    for l in range(1, len(g.dims) - 1):
        a, b = g.get_activation(l), ref.activation(l)
        diff = (a == 0) != (b == 0)
        if diff.any():
            worst = float(np.max(np.maximum(np.abs(a[diff]), np.abs(b[diff]))) / np.max(np.abs(b)))
            assert worst <= max(1e-5, 0.1 * tol), "a hidden unit differs across the ReLU and is not a tie (%g)" % worst
            rows, cols = np.nonzero(diff)
            out[l] = (rows, cols, a[rows, cols] != 0)
    return out


def oracle_step(g, ref, tol=TOL, step="train_epoch"):
    """The oracle's counterpart of the step the library has just run (`step`: train_epoch or forward_backward), with the
    ReLU decision of units at the kink taken as the library took it: the step is run; if units fell on different
    sides it is run again from the same state with their branch prescribed (orc_set_relu_branch), until none differ.
    The comparison that follows needs no widened tolerance.  Returns (the step's result, number of tie units)."""
    saved = [ref.get_params(k) for k in range(ref.K)]
    epoch = ref.epoch
    out = getattr(ref, step)()
    total = 0
    for _ in range(4):
        ties = relu_kink_units(g, ref, tol)
        if not ties:
            break
        for l, (rows, cols, on) in ties.items():
            total += len(rows)
            ref.set_relu_branch(l, rows[on], cols[on], 1)
            ref.set_relu_branch(l, rows[~on], cols[~on], 2)
        for k in range(ref.K):
            ref.set_params(k, saved[k])
        ref.epoch = epoch
        out = getattr(ref, step)()
    else:
        raise AssertionError("units at the ReLU kink keep changing sides")
    ref.clear_relu_branches()
    if total:
        print("ReLU ties: %d hidden units at the kink took the library's branch in the oracle" % total)
    return out, total


def check_epoch(g, ref, tol=TOL, loss_tol=1e-5):
    lg = g.train_epoch()
    lr, _ = oracle_step(g, ref, tol)
    assert np.max(np.abs(lg - lr)) <= loss_tol + 1e-5 * np.max(np.abs(lr)), (lg, lr)
    L = len(g.dims) - 1
    for l in range(1, L + 1):
        assert rel_err(g.get_activation(l), ref.activation(l)) <= tol, "activation %d" % l
    for k in range(g.K):
        assert rel_err(g.get_grads(k), ref.get_grads(k)) <= tol, "grads %d" % k
        assert rel_err(g.get_params(k), ref.get_params(k)) <= tol, "params %d" % k


@pytest.mark.parametrize("seed,directed,weighted,dims", [
    (0, False, False, (6, 5, 3)),
    (1, False, True, (13, 7, 5, 3)),
    (2, True, False, (6, 5, 3)),
    (3, True, True, (33, 130, 4)),
    (4, False, False, (8, 4)),
    (5, False, False, (10, 150)),
    (6, True, False, (7, 9, 40)),
])
def test_small_cases_store_and_one_epoch(seed, directed, weighted, dims):
    case = small_random_case(seed, n=70, K=3, directed=directed, weighted=weighted)
    g, ref, st = make_pair(case, dims, seed, lr=0.1)
    with g:
        check_store(g, st)
        check_epoch(g, ref)
        check_epoch(g, ref)


def test_tiny_ten_epoch_loss_curve_and_parameters(tiny):
    theta = glorot_params(tiny.dims, np.random.default_rng(0))
    ref = orc().from_workload(tiny, theta)
    with pkg().from_workload(tiny, theta) as g:
        check_store(g, ref.store)
        lg = np.array([g.train_epoch() for _ in range(10)])
        lr = np.array([ref.train_epoch() for _ in range(10)])
        assert np.max(np.abs(lg - lr)) <= LOSS_TOL
        assert np.max(np.abs(lg - lr)) <= 2e-5          # far inside the bar in fp32 mode
        for k in range(g.K):
            assert rel_err(g.get_params(k), ref.get_params(k)) <= TOL
            assert rel_err(g.get_grads(k), ref.get_grads(k)) <= TOL
        out = g.forward()
        assert rel_err(out, ref.forward_global(tiny.n)) <= TOL


def test_tiny_signal_learns_and_tracks_the_oracle(tiny_signal):
    w = tiny_signal
    theta = glorot_params(w.dims, np.random.default_rng(2))
    ref = orc().from_workload(w, theta)
    with pkg().from_workload(w, theta) as g:
        lg = np.array([g.train_epoch() for _ in range(10)])
        lr = np.array([ref.train_epoch() for _ in range(10)])
        assert lr[-1, -1] < lr[0, -1] - 0.1
        assert np.max(np.abs(lg - lr)) <= LOSS_TOL
        for k in range(g.K):
            assert rel_err(g.get_params(k), ref.get_params(k)) <= TOL


def test_dropout_mask_matches_the_counter_based_definition(tiny_signal):
    w = tiny_signal
    theta = glorot_params(w.dims, np.random.default_rng(3))
    ref = orc().from_workload(w, theta, dropout=0.25, seed=77)
    with pkg().from_workload(w, theta, dropout=0.25, seed=77) as g:
        for _ in range(3):
            lg, lr = g.train_epoch(), ref.train_epoch()
            assert np.max(np.abs(lg - lr)) <= 1e-4
            h1g, h1r = g.get_activation(1), ref.activation(1)
            assert np.array_equal(h1g == 0, h1r == 0)             # the same units dropped
            assert rel_err(h1g, h1r) <= TOL
        assert (h1r == 0).mean() > 0.3
        for k in range(g.K):
            assert rel_err(g.get_params(k), ref.get_params(k)) <= TOL
        # inference applies no dropout
        assert rel_err(g.forward(), ref.forward_global(w.n)) <= TOL


def test_importance_weights_and_consensus(tiny):
    theta = glorot_params(tiny.dims, np.random.default_rng(4))
    ref = orc().from_workload(tiny, theta)
    with pkg().from_workload(tiny, theta) as g:
        zg, wg = g.subgraph_weights()
        zr, wr = ref.subgraph_weights()
        assert np.max(np.abs(zg - zr) / zr) <= 1e-6
        assert np.max(np.abs(wg - wr)) <= 1e-6 and abs(float(wg.sum()) - 1.0) <= 1e-6
        rng = np.random.default_rng(0)
        for k in range(g.K):
            t = theta + rng.standard_normal(theta.size).astype(np.float32)
            g.set_params(k, t)
            ref.set_params(k, t)
        g.consensus()
        ref.consensus()
        first = g.get_params(0)
        for k in range(g.K):
            assert rel_err(g.get_params(k), ref.get_params(k)) <= 1e-6
            assert np.array_equal(g.get_params(k), first)          # every replica holds the same bits
        g.consensus()
        assert rel_err(g.get_params(0), first) <= 1e-6              # a second consensus changes nothing
    with pkg().from_workload(tiny, theta, weighted=False) as g:
        assert np.allclose(g.subgraph_weights()[1], 0.25)


@pytest.mark.parametrize("flags", [0, 16])
@pytest.mark.parametrize("seed,n,K,F", [(0, 70, 3, 6), (1, 700, 2, 37), (2, 3000, 3, 64), (3, 1500, 1, 130)])
def test_pairwise_importance_weights(seed, n, K, F, flags):
    """zeta_mode 1: the printed formula taken literally, sum_{i<j} p_i p_j / (|x_i - x_j| + beta), against the oracle's
    double loop; then an epoch whose consensus uses them.  flags 0: squared distances from a Gram matrix on the tensor
    cores, tiles of 128 x 128 pairs; flags 16: from the differences on the FP32 ALUs, tiles of 64 x 64.  Ragged last
    tiles, subgraphs of less than one tile, feature widths that are not multiples of the MMA's K."""
    case = small_random_case(seed, n=n, K=K, p=min(0.15, 8.0 / n))
    g, ref, st = make_pair(case, (F, 8, 3), seed, lr=0.1, zeta_mode=1, flags=flags)
    with g:
        zg, wg = g.subgraph_weights()
        zr, wr = ref.subgraph_weights()
        assert np.max(np.abs(zg - zr)) <= 2e-6 * np.max(zr)
        assert np.max(np.abs(wg - wr)) <= 2e-6
        check_epoch(g, ref)


@pytest.mark.parametrize("flags", [0, 16])
def test_pairwise_importance_of_identical_points_is_the_closed_form(flags):
    """All features equal: every distance is 0 and zeta = S / beta with S = (1 - sum p^2) / 2.  (For the Gram-matrix
    kernel this is the worst case of its cancellation: every pair is recomputed from the differences.)"""
    case = small_random_case(5, n=300, K=2, p=0.05)
    n = case[0]
    X = np.ones((n, 12), dtype=np.float32) * 0.75
    g, ref, st = make_pair(case, (12, 5, 3), 5, X=X, zeta_mode=1, beta=0.5, flags=flags)
    with g:
        zg, _ = g.subgraph_weights()
    for k in range(st.K):
        d = st.deg[st.sub_off[k]:st.sub_off[k + 1]].astype(np.float64)
        p = d / d.sum() if d.sum() > 0 else np.full(len(d), 1.0 / len(d))
        assert abs(zg[k] - 0.5 * (1.0 - np.sum(p * p)) / 0.5) <= 1e-6


def test_large_feature_offsets_do_not_break_the_variance_statistics():
    case = small_random_case(11, n=90, K=3)
    X = (np.random.default_rng(5).standard_normal((90, 9)) + 300.0).astype(np.float32)
    g, ref, _ = make_pair(case, (9, 4, 3), 11, X=X)
    with g:
        zg, wg = g.subgraph_weights()
        zr, wr = ref.subgraph_weights()
        assert np.max(np.abs(zg - zr) / zr) <= 1e-5


def test_single_replica_and_degenerate_subgraphs():
    # K = 1: the consensus is the identity; an empty subgraph and a subgraph without training nodes are legal
    n, rowptr, col, w, core, halo = small_random_case(6, n=50, K=1, halo=False)
    g, ref, st = make_pair((n, rowptr, col, w, core, halo), (6, 5, 3), 6, lr=0.2)
    with g:
        check_store(g, st)
        check_epoch(g, ref)
        before = g.get_params(0)
        g.consensus()
        assert np.array_equal(g.get_params(0), before)
        assert g.subgraph_weights()[1][0] == 1.0
    n, rowptr, col, w, core, halo = small_random_case(7, n=60, K=3)
    core = [core[0], np.empty(0, np.int32), core[2]]
    halo = [halo[0], np.empty(0, np.int32), halo[2]]
    g, ref, st = make_pair((n, rowptr, col, w, core, halo), (6, 5, 3), 7, lr=0.2)
    with g:
        check_store(g, st)
        check_epoch(g, ref)
        zg, wg = g.subgraph_weights()
        assert zg[1] == 0.0 and wg[1] == 0.0


def test_many_subgraphs_and_a_deep_network():
    """K = 40 small subgraphs (several row tiles and chunks end inside a subgraph of a few rows) and L = 5 layers."""
    case = small_random_case(31, n=600, K=40, p=0.02)
    g, ref, st = make_pair(case, (20, 24, 40, 16, 12, 5), 31, lr=0.05)
    with g:
        check_store(g, st)
        check_epoch(g, ref)
        check_epoch(g, ref)


@pytest.mark.parametrize("flags", [0, 1])
@pytest.mark.parametrize("dims", [(24, 40, 6), (100, 20, 6)])
def test_dropout_through_both_layer_orders_and_transform_paths(flags, dims):
    """Dropout after the ReLU when layer 0 aggregates first (mask applied in the transform's epilogue: tensor-core
    kernel, or the FP32-ALU one with flags bit 0) and when it transforms first (mask applied in the SpMM epilogue)."""
    case = small_random_case(33, n=500, K=3, p=0.02)
    g, ref, st = make_pair(case, dims, 33, lr=0.05, dropout=0.4, flags=flags)
    with g:
        for _ in range(2):
            lg, lr = g.train_epoch(), ref.train_epoch()
            assert np.max(np.abs(lg - lr)) <= 1e-4
            h1g, h1r = g.get_activation(1), ref.activation(1)
            assert np.array_equal(h1g == 0, h1r == 0)
            assert rel_err(h1g, h1r) <= TOL
        for k in range(g.K):
            assert rel_err(g.get_params(k), ref.get_params(k)) <= TOL


def test_wide_input_aggregated_first():
    """F_0 = 1100 > 1024 aggregated first (two column slabs in the SpMM, a 1100-deep reduction in the transform)."""
    case = small_random_case(35, n=400, K=2, p=0.03)
    g, ref, st = make_pair(case, (1100, 600, 4), 35, lr=0.02)
    with g:
        check_epoch(g, ref)


def test_pairwise_importance_with_degenerate_subgraphs():
    """zeta_mode 1 with an empty subgraph (zeta 0), a single-row subgraph (no pair: zeta 0) and a subgraph without edges
    (uniform p)."""
    n = 40
    rowptr = np.zeros(n + 1, dtype=np.int64)
    src = np.array([0, 1, 1, 2, 2, 3], dtype=np.int64)
    dst = np.array([1, 0, 2, 1, 3, 2], dtype=np.int32)
    np.cumsum(np.bincount(src, minlength=n), out=rowptr[1:])
    core = [np.arange(0, 10, dtype=np.int32), np.empty(0, np.int32), np.array([10], dtype=np.int32), np.arange(20, 40, dtype=np.int32)]
    halo = [np.empty(0, np.int32)] * 4
    g, ref, st = make_pair((n, rowptr, dst, None, core, halo), (5, 4, 3), 37, zeta_mode=1)
    with g:
        zg, wg = g.subgraph_weights()
        zr, wr = ref.subgraph_weights()
        assert zg[1] == 0.0 and zg[2] == 0.0
        assert np.max(np.abs(zg - zr)) <= 1e-6 and np.max(np.abs(wg - wr)) <= 1e-6
        check_epoch(g, ref)


def test_isolated_nodes_and_no_edges():
    n = 40
    rowptr = np.zeros(n + 1, dtype=np.int64)
    col = np.empty(0, dtype=np.int32)
    core = [np.arange(0, 25, dtype=np.int32), np.arange(25, 40, dtype=np.int32)]
    halo = [np.array([30], dtype=np.int32), np.empty(0, np.int32)]
    g, ref, st = make_pair((n, rowptr, col, None, core, halo), (5, 4, 3), 8, lr=0.3)
    with g:
        check_store(g, st)
        check_epoch(g, ref)
        zg, _ = g.subgraph_weights()
        zr, _ = ref.subgraph_weights()
        assert np.allclose(zg, zr, rtol=1e-6)


def test_hub_rows_and_wide_features():
    # a star with 5000 leaves puts one row far above the hub threshold; 1030 features need two column slabs
    n = 5001
    leaves = np.arange(1, n)
    src = np.concatenate([np.zeros(n - 1, dtype=np.int64), leaves])
    dst = np.concatenate([leaves, np.zeros(n - 1, dtype=np.int64)])
    order = np.lexsort((dst, src))
    src, dst = src[order], dst[order]
    rowptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(np.bincount(src, minlength=n), out=rowptr[1:])
    core = [np.arange(0, 3000, dtype=np.int32), np.arange(3000, n, dtype=np.int32)]
    halo = [np.arange(3000, 3100, dtype=np.int32), np.array([0], dtype=np.int32)]
    g, ref, st = make_pair((n, rowptr, dst.astype(np.int32), None, core, halo), (12, 1030, 3), 9, lr=0.05)
    with g:
        check_store(g, st)
        check_epoch(g, ref)


@pytest.mark.parametrize("directed,weighted,dims", [(False, False, (24, 40, 5)), (True, True, (24, 40, 70)), (True, False, (16, 6))])
def test_last_backward_aggregation_over_the_rows_that_carry_loss(directed, weighted, dims):
    """d loss / d logits is zero on replicated rows and on core rows outside the training split, so by default the last
    layer's backward aggregation runs over a store without the entries that read such rows.  Same gradients as the
    full store (flag bit 6) up to the grouping of a cut row's partial sums, and as the oracle; subgraph 1 has no
    training node at all, subgraph 0 holds a hub row that is cut into parts."""
    n, rowptr, col, w, core, halo = small_random_case(31, n=1500, K=3, p=0.004, directed=directed, weighted=weighted)
    # a hub: node core[0][0] gains an edge from and to every other node of its subgraph
    hub, others = int(core[0][0]), [int(v) for v in core[0][1:]]
    src = np.repeat(np.arange(n, dtype=np.int64), np.diff(rowptr))
    pairs = set(zip(src.tolist(), col.tolist()))
    extra = [(hub, v) for v in others if (hub, v) not in pairs] + [(v, hub) for v in others if (v, hub) not in pairs]
    es = np.concatenate([src, np.array([e[0] for e in extra], dtype=np.int64)])
    ed = np.concatenate([col.astype(np.int64), np.array([e[1] for e in extra], dtype=np.int64)])
    ew = None if w is None else np.concatenate([w, np.ones(len(extra), dtype=np.float32)])
    order = np.lexsort((ed, es))
    es, ed = es[order], ed[order]
    ew = None if ew is None else ew[order]
    rowptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(np.bincount(es, minlength=n), out=rowptr[1:])
    col = ed.astype(np.int32)
    rng = np.random.default_rng(77)
    X = rng.standard_normal((n, dims[0])).astype(np.float32)
    y = rng.integers(0, dims[-1], size=n).astype(np.int32)
    split = rng.integers(0, 3, size=n).astype(np.uint8)
    split[core[1]] = 1 + (split[core[1]] & 1)          # no training node in subgraph 1
    theta = glorot_params(dims, rng, bias_scale=0.2)
    cp, cn = flat(core)
    hp, hn = flat(halo)
    st = orc().Store(n, rowptr, col, cp, cn, hp, hn, weights=ew)
    ref = orc().Model(st, X, y, split, dims, theta, lr=0.05)
    a = pkg().Gad(n, rowptr, col, cp, cn, hp, hn, X, y, split, dims, init_params=theta, weights=ew, lr=0.05)
    b = pkg().Gad(n, rowptr, col, cp, cn, hp, hn, X, y, split, dims, init_params=theta, weights=ew, lr=0.05, flags=64)
    with a, b:
        assert a.check_store() == 0 and b.check_store() == 0
        assert a.ntrain()[1] == 0
        for _ in range(2):
            b.train_epoch()
            check_epoch(a, ref)
            assert np.array_equal(a.get_activation(len(dims) - 1), b.get_activation(len(dims) - 1))   # the forward pass does not differ
            for k in range(a.K):
                assert rel_err(a.get_grads(k), b.get_grads(k)) <= 1e-6
                assert rel_err(a.get_params(k), b.get_params(k)) <= 1e-6


def test_runs_are_bitwise_reproducible_and_resume_is_exact(tiny_signal):
    w = tiny_signal
    theta = glorot_params(w.dims, np.random.default_rng(5))
    with pkg().from_workload(w, theta, dropout=0.25, seed=3) as a:
        la = np.array([a.train_epoch() for _ in range(10)])
        pa = a.get_params(0)
    with pkg().from_workload(w, theta, dropout=0.25, seed=3) as b:
        lb = [b.train_epoch() for _ in range(5)]
        saved = [b.get_params(k) for k in range(b.K)]
        epoch = b.epoch
    with pkg().from_workload(w, theta, dropout=0.25, seed=3) as c:
        for k in range(c.K):
            c.set_params(k, saved[k])
        c.epoch = epoch
        lb += [c.train_epoch() for _ in range(5)]
        pc = c.get_params(0)
    assert np.array_equal(la, np.array(lb))
    assert np.array_equal(pa, pc)


def test_set_inputs_replaces_features_and_labels(tiny):
    w = tiny
    theta = glorot_params(w.dims, np.random.default_rng(6))
    rng = np.random.default_rng(9)
    X2 = rng.standard_normal(w.X.shape).astype(np.float32)
    y2 = rng.integers(0, 4, size=w.n).astype(np.int32)
    cp, cn, hp, hn = w.flat_partition()
    st = orc().Store(w.n, w.rowptr, w.col, cp, cn, hp, hn)
    ref = orc().Model(st, X2, y2, w.split, w.dims, theta, lr=w.lr)
    with pkg().from_workload(w, theta) as g:
        g.set_inputs(X2, y2)
        lg, lr = g.train_epoch(), ref.train_epoch()
        assert np.max(np.abs(lg - lr)) <= 1e-5
        assert rel_err(g.get_grads(1), ref.get_grads(1)) <= TOL


def test_pipelined_inputs_and_asynchronous_loss_reads(tiny):
    """A loop that never waits inside a step: inputs alternate between two pinned buffers (the copies go out on the
    context's second stream into alternating staging buffers), losses come back asynchronously."""
    import torch
    w = tiny
    theta = glorot_params(w.dims, np.random.default_rng(11))
    rng = np.random.default_rng(12)
    Xs = [w.X, rng.standard_normal(w.X.shape).astype(np.float32), rng.standard_normal(w.X.shape).astype(np.float32)]
    pinned = [torch.from_numpy(x).pin_memory() for x in Xs]
    labels = torch.from_numpy(w.labels).pin_memory()
    losses = torch.zeros((5, w.K + 1), dtype=torch.float32).pin_memory()
    cp, cn, hp, hn = w.flat_partition()
    st = orc().Store(w.n, w.rowptr, w.col, cp, cn, hp, hn)
    with pkg().from_workload(w, theta) as g:
        for i in range(5):
            g.set_inputs(pinned[i % 3], labels)
            g.train_epoch(loss_out=losses[i].numpy(), wait=False)
        g.synchronize()
        params = theta
        for i in range(5):
            ref = orc().Model(st, Xs[i % 3], w.labels, w.split, w.dims, params, lr=w.lr)
            want = ref.train_epoch()
            params = ref.get_params(0)      # identical replicas after the weighted consensus
            assert np.max(np.abs(losses[i].numpy() - want)) <= 1e-5, "step %d" % i
        assert rel_err(g.get_params(0), params) <= TOL


def test_kept_input_aggregation_follows_new_features(tiny):
    """flags bit 1 keeps A~ H^(0) across epochs; new features must replace it."""
    w = tiny
    theta = glorot_params(w.dims, np.random.default_rng(8))
    rng = np.random.default_rng(10)
    X2 = rng.standard_normal(w.X.shape).astype(np.float32)
    cp, cn, hp, hn = w.flat_partition()
    st = orc().Store(w.n, w.rowptr, w.col, cp, cn, hp, hn)
    ref = orc().Model(st, w.X, w.labels, w.split, w.dims, theta, lr=w.lr)
    with pkg().from_workload(w, theta, flags=2) as g:
        for _ in range(2):
            assert np.max(np.abs(g.train_epoch() - ref.train_epoch())) <= 1e-5
        ref2 = orc().Model(st, X2, w.labels, w.split, w.dims, ref.get_params(0), lr=w.lr)
        for k in range(1, g.K):
            ref2.set_params(k, ref.get_params(k))
        g.set_inputs(X2, None)
        for _ in range(2):
            assert np.max(np.abs(g.train_epoch() - ref2.train_epoch())) <= 1e-5
        assert rel_err(g.get_params(0), ref2.get_params(0)) <= TOL


def test_non_finite_loss_is_reported_not_trapped(tiny):
    w = tiny
    theta = glorot_params(w.dims, np.random.default_rng(7))
    X = w.X.copy()
    X[w.core[0][0], 0] = np.inf
    cp, cn, hp, hn = w.flat_partition()
    with pkg().Gad(w.n, w.rowptr, w.col, cp, cn, hp, hn, X, w.labels, w.split, w.dims, init_params=theta) as g:
        with pytest.raises(pkg().GadError) as e:
            g.train_epoch()
        assert e.value.code == -6
        g.set_inputs(w.X)                                   # the context stays usable
        for k in range(g.K):
            g.set_params(k, theta)
        assert np.all(np.isfinite(g.train_epoch()))


def test_c2_two_epochs_full_size():
    w = make_workload("c2")
    theta = glorot_params(w.dims, np.random.default_rng(0))
    ref = orc().from_workload(w, theta)
    with pkg().from_workload(w, theta) as g:
        check_store(g, ref.store)
        ties = 0
        for _ in range(2):
            lg = g.train_epoch()
            lr, t = oracle_step(g, ref)
            ties += t
            assert np.max(np.abs(lg - lr)) <= 1e-4
        assert ties <= 64, "%d hidden units at the ReLU kink: more than rounding explains" % ties
        L = len(w.dims) - 1
        assert rel_err(g.get_activation(L), ref.activation(L)) <= TOL
        for k in range(g.K):
            assert rel_err(g.get_grads(k), ref.get_grads(k)) <= TOL, "replica %d" % k
            assert rel_err(g.get_params(k), ref.get_params(k)) <= TOL
        zg, wg = g.subgraph_weights()
        zr, wr = ref.subgraph_weights()
        assert np.max(np.abs(wg - wr)) <= 1e-6


def test_c2_ten_epoch_loss_curve_full_size_in_the_benchmark_configuration():
    """The launch configuration bench.py times: full-size c2 on a stream of its own, so epochs 2 .. 10 are graph
    replays.  Loss curve within 1e-3 of the oracle's over ten epochs (lr 0.5 so that it moves), parameters and
    logits within 1e-4 at the end."""
    import torch
    w = make_workload("c2")
    theta = glorot_params(w.dims, np.random.default_rng(0))
    ref = orc().from_workload(w, theta, lr=0.5)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        with pkg().from_workload(w, theta, lr=0.5, stream=stream) as g:
            n0 = pkg().launch_count()
            lg = np.array([g.train_epoch() for _ in range(10)])
            assert pkg().launch_count() - n0 == 10 * 18
            lr = np.array([ref.train_epoch() for _ in range(10)])
            assert np.max(np.abs(lg - lr)) <= LOSS_TOL
            assert lr[0, -1] - lr[-1, -1] > 5e-3          # the curve moves by several times the tolerance
            for k in (0, g.K - 1):
                assert rel_err(g.get_params(k), ref.get_params(k)) <= TOL
            assert rel_err(g.forward(), ref.forward_global(w.n)) <= TOL


@pytest.mark.parametrize("gemm_mode,flags,tol", [(0, 0, TOL), (0, 1, TOL), (1, 0, 5e-2), (0, 2, TOL), (0, 3, TOL)])
@pytest.mark.parametrize("dims", [(96, 160, 40, 8), (602, 256, 41), (20, 300, 130, 3)])
def test_transform_paths_tensor_core_and_simt(gemm_mode, flags, tol, dims):
    """The grouped H.W transform on tensor cores (split-TF32: fp32 bar; single-pass TF32 operands: 5e-2 bar) and
    on the FP32 ALUs (flags bit 0), over row tiles with ragged ends and feature widths that are not tile multiples.
    Layer 0 transforms first when F_0 > 2 F_1 (the 602-wide case) and aggregates first otherwise; flags bit 1 makes it
    aggregate first everywhere and keeps the aggregated features between epochs."""
    case = small_random_case(21, n=900, K=3, p=0.01)
    g, ref, st = make_pair(case, dims, 21, lr=0.05, gemm_mode=gemm_mode, flags=flags)
    with g:
        for _ in range(2):
            lg = g.train_epoch()
            lr, _ = oracle_step(g, ref, tol)
            assert np.max(np.abs(lg - lr)) <= (1e-4 if gemm_mode == 0 else 5e-2)
        L = len(dims) - 1
        for l in range(1, L + 1):
            assert rel_err(g.get_activation(l), ref.activation(l)) <= tol, "activation %d" % l
        for k in range(g.K):
            assert rel_err(g.get_grads(k), ref.get_grads(k)) <= tol
            assert rel_err(g.get_params(k), ref.get_params(k)) <= tol
        assert rel_err(g.forward(), ref.forward_global(case[0])) <= tol


def test_split_transform_keeps_the_bits_below_tf32():
    """The fp32-accurate transforms hand the tensor core the activation tile as loaded and add the product with
    lo = x - (x without its 13 lowest mantissa bits): right only if the tensor core drops those bits of an fp32 operand
    rather than rounding them.  Features whose 13 lowest mantissa bits are all ones make the difference as large as it
    gets (rounding would move every one of them up by a TF32 ulp, 5e-4 to 1e-3 of the value, always away from zero);
    on a graph without edges (A~ = I) layer 0 is the transform alone.  Bar: 2e-5 of the largest entry, forward (row
    kernel) and weight gradient (reduction over rows): several times what the split leaves, and far below the 7e-4 that
    rounded hi parts under the same lo parts give on these inputs (worked out in fp64 on the host)."""
    n, K, dims = 700, 2, (256, 256, 8)
    rowptr = np.zeros(n + 1, dtype=np.int64)
    col = np.empty(0, dtype=np.int32)
    core = [np.arange(0, 350, dtype=np.int32), np.arange(350, n, dtype=np.int32)]
    halo = [np.empty(0, np.int32), np.empty(0, np.int32)]
    X = np.random.default_rng(5).standard_normal((n, dims[0])).astype(np.float32)
    X = (X.view(np.uint32) | np.uint32(0x1FFF)).view(np.float32)
    g, ref, st = make_pair((n, rowptr, col, None, core, halo), dims, 5, X=X, lr=0.05)
    with g:
        lg = g.train_epoch()
        lr, _ = oracle_step(g, ref, 2e-5)
        assert np.max(np.abs(lg - lr)) <= 1e-5
        assert rel_err(g.get_activation(1), ref.activation(1)) <= 2e-5
        for k in range(K):
            assert rel_err(g.get_grads(k), ref.get_grads(k)) <= 2e-5


@pytest.mark.parametrize("flags", [0, 4])
@pytest.mark.parametrize("dims,dropout", [((40, 128, 16), 0.0), ((30, 200, 12), 0.0), ((24, 500, 7), 0.3), ((100, 8, 3), 0.0),
                                          ((16, 130, 16, 4), 0.25), ((12, 256, 5), 0.0), ((9, 516, 4), 0.0), ((20, 100, 10), 0.0), ((12, 128, 16, 100, 8), 0.0)])
def test_layers_of_at_most_sixteen_output_columns(flags, dims, dropout):
    """The backward pass of a layer l >= 1 with at most 16 output columns runs as one stream on the FP32 ALUs (dW and
    the masked input gradient in one pass over H and dZ), or with flags bit 2 through the tensor-core transforms like
    any other layer.  Input widths of one, two and four 128-column slabs, ragged ones, one beyond the kernel's limit
    (516) and some below it (under 96 columns: tensor cores again), a narrow layer in the middle of the network (its
    kernel also sums the bias gradient of the layer below) and one that is layer 0 (tensor cores)."""
    case = small_random_case(31, n=1500, K=3, p=0.006)
    g, ref, st = make_pair(case, dims, 31, lr=0.05, dropout=dropout, flags=flags)
    with g:
        for _ in range(2):
            lg = g.train_epoch()
            lr, _ = oracle_step(g, ref)
            assert np.max(np.abs(lg - lr)) <= 1e-4
        L = len(dims) - 1
        for l in range(1, L + 1):
            assert rel_err(g.get_activation(l), ref.activation(l)) <= TOL, "activation %d" % l
        for k in range(g.K):
            assert rel_err(g.get_grads(k), ref.get_grads(k)) <= TOL
            assert rel_err(g.get_params(k), ref.get_params(k)) <= TOL
        assert rel_err(g.forward(), ref.forward_global(case[0])) <= TOL


@pytest.mark.parametrize("dims,dropout", [((12, 40, 9, 4), 0.0), ((130, 24, 6), 0.3), ((10, 5), 0.0)])
def test_importance_weights_summed_over_the_layers(dims, dropout):
    """zeta_mode 2: the aggregate distance term with the sum over layers kept (inputs H^(0) .. H^(L-1) of the epoch's own
    forward pass).  Weights, losses and parameters against the oracle over three epochs, and the standalone call."""
    case = small_random_case(51, n=400, K=4, p=0.02)
    g, ref, st = make_pair(case, dims, 51, lr=0.2, dropout=dropout, zeta_mode=2, beta=0.5)
    with g:
        zg, wg = g.subgraph_weights()          # before any epoch: an inference pass provides the activations
        ref.forward()
        zr, wr = ref.subgraph_weights()
        assert np.max(np.abs(wg - wr)) <= 1e-5 and rel_err(zg, zr) <= 1e-5
        for _ in range(3):
            lg = g.train_epoch()
            lr, _ = oracle_step(g, ref)
            assert np.max(np.abs(lg - lr)) <= 1e-4
        zg, wg = g.subgraph_weights()
        zr, wr = ref.subgraph_weights()
        assert np.max(np.abs(wg - wr)) <= 1e-5 and rel_err(zg, zr) <= 1e-5
        for k in range(g.K):
            assert rel_err(g.get_grads(k), ref.get_grads(k)) <= TOL
            assert rel_err(g.get_params(k), ref.get_params(k)) <= TOL


@pytest.mark.parametrize("dims,zeta_mode", [((24, 40, 5), 0), ((130, 128, 16), 0), ((12, 20, 9, 4), 2), ((40, 12, 64, 5), 1)])
def test_epochs_replayed_as_a_graph_equal_epochs_enqueued_one_by_one(dims, zeta_mode):
    """On a stream of its own the library captures the epoch's launches after the first epoch and replays them as one
    CUDA graph; flags bit 3 keeps the launches one by one.  Same kernels in the same order: the results must agree
    bit for bit, the launch counter must advance alike, and both must match the oracle."""
    import torch
    case = small_random_case(61, n=500, K=4, p=0.02)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        g, ref, st = make_pair(case, dims, 61, lr=0.1, zeta_mode=zeta_mode, stream=stream)
        h, _, _ = make_pair(case, dims, 61, lr=0.1, zeta_mode=zeta_mode, stream=stream, flags=8)
        with g, h:
            for epoch in range(4):
                n0 = pkg().launch_count()
                lg = g.train_epoch()
                n1 = pkg().launch_count()
                lh = h.train_epoch()
                n2 = pkg().launch_count()
                lr = ref.train_epoch()
                assert np.array_equal(lg, lh) and n1 - n0 == n2 - n1 > 0
                assert np.max(np.abs(lg - lr)) <= 1e-4
            for k in range(g.K):
                assert np.array_equal(g.get_params(k), h.get_params(k))
                assert np.array_equal(g.get_grads(k), h.get_grads(k))
                assert rel_err(g.get_params(k), ref.get_params(k)) <= TOL
            # the epoch without update and consensus has a graph of its own
            for _ in range(3):
                assert np.array_equal(g.train_epoch_local(), h.train_epoch_local())
            assert np.array_equal(g.get_grads(1), h.get_grads(1))
            # new inputs between replays
            X2 = np.random.default_rng(9).standard_normal((case[0], dims[0])).astype(np.float32)
            g.set_inputs(X2); h.set_inputs(X2)
            assert np.array_equal(g.train_epoch(), h.train_epoch())
            assert np.array_equal(g.get_params(0), h.get_params(0))


def test_reduced_precision_mode_on_a_power_law_graph():
    """gemm_mode 1 (one TF32 pass per transform, the aggregation gathering a bfloat16 copy of its operand) on a scaled
    c2: hub rows cut into parts, wide and narrow aggregations, graph replay.  Bar of this mode: 5e-2."""
    import torch
    w = make_workload("c2", scale=0.2)
    theta = glorot_params(w.dims, np.random.default_rng(0), bias_scale=0.1)
    ref = orc().from_workload(w, theta, lr=0.5)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        with pkg().from_workload(w, theta, lr=0.5, gemm_mode=1, stream=stream) as g:
            for _ in range(3):
                lg, lr = g.train_epoch(), ref.train_epoch()
                assert np.max(np.abs(lg - lr)) <= 5e-2
            L = len(w.dims) - 1
            assert rel_err(g.get_activation(L), ref.activation(L)) <= 5e-2
            for k in range(g.K):
                assert rel_err(g.get_grads(k), ref.get_grads(k)) <= 5e-2
                assert rel_err(g.get_params(k), ref.get_params(k)) <= 5e-2
            # and it is not the fp32 path in disguise: the rounding of the operands shows
            assert rel_err(g.get_activation(L), ref.activation(L)) > 1e-5


def test_a_bounded_wait_that_runs_out_is_reported_and_leaves_the_model_untouched(tiny_signal):
    """The transforms bound every device-side wait.  gad_debug_expire_wait makes one such wait run out on purpose (a
    one-thread kernel polling, 1000 times, a barrier nothing arrives at): the kernel returns, the error word is raised,
    the epoch enqueued behind it skips its update and consensus, the next waiting call returns
    GAD_ERR_DEVICE_TIMEOUT, and the context goes on working from the unchanged parameters."""
    w = tiny_signal
    theta = glorot_params(w.dims, np.random.default_rng(13))
    ref = orc().from_workload(w, theta)
    with pkg().from_workload(w, theta) as g:
        assert np.max(np.abs(g.train_epoch() - ref.train_epoch())) <= 1e-5
        before = [g.get_params(k) for k in range(g.K)]
        g.debug_expire_wait(1000)
        g.train_epoch(wait=False)                       # enqueued behind the failed wait
        with pytest.raises(pkg().GadError) as e:
            g.synchronize()
        assert e.value.code == -7
        for k in range(g.K):
            assert np.array_equal(g.get_params(k), before[k])
        g.synchronize()                                  # reported once, then cleared
        g.debug_expire_wait(1)
        with pytest.raises(pkg().GadError) as e:
            g.get_loss()
        assert e.value.code == -7
        # the run continues as if the skipped epoch had not been asked for
        g.epoch = ref.epoch
        assert np.max(np.abs(g.train_epoch() - ref.train_epoch())) <= 1e-5
        for k in range(g.K):
            assert rel_err(g.get_params(k), ref.get_params(k)) <= TOL
        with pytest.raises(pkg().GadError):
            g.debug_expire_wait(0)


def test_set_inputs_rejects_labels_outside_the_classes(tiny):
    w = tiny
    theta = glorot_params(w.dims, np.random.default_rng(14))
    with pkg().from_workload(w, theta) as g:
        bad = w.labels.copy()
        bad[7] = w.dims[-1]
        with pytest.raises(pkg().GadError) as e:
            g.set_inputs(None, bad)
        assert e.value.code == -2
        bad[7] = -1
        with pytest.raises(pkg().GadError) as e:
            g.set_inputs(w.X, bad)
        assert e.value.code == -2
        assert np.all(np.isfinite(g.train_epoch()))      # nothing was enqueued; the old labels are still in place


def test_pairwise_importance_of_near_duplicates_and_offset_features():
    """The Gram form |x|^2 + |y|^2 - 2 x.y cancels for rows that are close compared with their norms.  Features with a
    large common offset (every pair is close in that sense) and a block of near-duplicate rows must still give the
    oracle's zeta: such pairs take the difference form."""
    case = small_random_case(41, n=600, K=2, p=0.02)
    n = case[0]
    rng = np.random.default_rng(41)
    X = (rng.standard_normal((n, 20)) + 40.0).astype(np.float32)
    X[100:200] = X[100] + 1e-3 * rng.standard_normal((100, 20)).astype(np.float32)
    g, ref, st = make_pair(case, (20, 5, 3), 41, X=X, zeta_mode=1)
    with g:
        zg, wg = g.subgraph_weights()
        zr, wr = ref.subgraph_weights()
        assert np.max(np.abs(zg - zr)) <= 2e-6 * np.max(zr)
        assert np.max(np.abs(wg - wr)) <= 2e-6


def test_pairwise_importance_of_a_large_subgraph():
    """One subgraph of 36 000 rows (more than the 32 768 the FP32-ALU kernel takes; 282 x 282 / 2 tiles, the last ones
    ragged) and one of 5 000, against the oracle's pair loop (6.6e8 pairs); twice, for run-to-run equality."""
    rng = np.random.default_rng(43)
    n, F = 41000, 24
    src = rng.integers(0, n, size=4 * n)
    dst = rng.integers(0, n, size=4 * n)
    keep = src != dst
    src, dst = np.concatenate([src[keep], dst[keep]]), np.concatenate([dst[keep], src[keep]])
    order = np.lexsort((dst, src))
    src, dst = src[order], dst[order]
    rowptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(np.bincount(src, minlength=n), out=rowptr[1:])
    core = [np.arange(0, 36000, dtype=np.int32), np.arange(36000, n, dtype=np.int32)]
    halo = [np.empty(0, np.int32), np.empty(0, np.int32)]
    X = rng.standard_normal((n, F)).astype(np.float32)
    X[:, :3] *= 4.0
    g, ref, st = make_pair((n, rowptr, dst.astype(np.int32), None, core, halo), (F, 6, 3), 43, X=X, zeta_mode=1)
    with g:
        zg, wg = g.subgraph_weights()
        zg2, _ = g.subgraph_weights()
        assert np.array_equal(zg, zg2)
        zr, wr = ref.subgraph_weights()
        assert np.max(np.abs(zg - zr)) <= 2e-6 * np.max(zr)
        assert np.max(np.abs(wg - wr)) <= 2e-6
    with pytest.raises(pkg().GadError) as e:           # the FP32-ALU form keeps its limit
        make_pair((n, rowptr, dst.astype(np.int32), None, core, halo), (F, 6, 3), 43, X=X, zeta_mode=1, flags=16)
    assert e.value.code == -9


@pytest.mark.parametrize("flags", [0, 1, 32])
@pytest.mark.parametrize("dims,dropout", [((16, 8, 256, 4), 0.0), ((12, 40, 9, 64, 5), 0.3), ((20, 6, 30, 140, 3), 0.0)])
def test_layers_beyond_the_first_choose_the_order_of_aggregation_and_transform(flags, dims, dropout):
    """A layer l >= 1 whose input is narrower than its output aggregates first, sigma((A~ H^(l)) W + b): forward SpMM at
    the input width, dW = (A~ H^(l))^T dPre, dH^(l) = A~^T (dPre W^T) followed by the ReLU mask of the layer below.  On
    the tensor cores, on the FP32 ALUs (flags bit 0), and with the choice switched off (flags bit 5): all against the
    oracle, which always computes A~ (H W)."""
    case = small_random_case(71, n=700, K=3, p=0.012, directed=(flags == 1))
    g, ref, st = make_pair(case, dims, 71, lr=0.05, dropout=dropout, flags=flags)
    with g:
        for _ in range(2):
            lg = g.train_epoch()
            lr, _ = oracle_step(g, ref)
            assert np.max(np.abs(lg - lr)) <= 1e-4
        L = len(dims) - 1
        for l in range(1, L + 1):
            assert rel_err(g.get_activation(l), ref.activation(l)) <= TOL, "activation %d" % l
        for k in range(g.K):
            assert rel_err(g.get_grads(k), ref.get_grads(k)) <= TOL
            assert rel_err(g.get_params(k), ref.get_params(k)) <= TOL
        assert rel_err(g.forward(), ref.forward_global(case[0])) <= TOL


def test_reduced_precision_mode_with_a_layer_that_aggregates_first():
    """gemm_mode 1 through a net whose middle layer aggregates first (8 -> 200): the bfloat16 operand copies are made by
    the conversion pass for that layer's two aggregations and by the transform's epilogue for the others.  Bar: 5e-2."""
    case = small_random_case(73, n=900, K=3, p=0.01)
    dims = (150, 8, 200, 6)
    g, ref, st = make_pair(case, dims, 73, lr=0.05, gemm_mode=1)
    with g:
        for _ in range(2):
            lg = g.train_epoch()
            lr, _ = oracle_step(g, ref, 5e-2)
            assert np.max(np.abs(lg - lr)) <= 5e-2
        for l in range(1, len(dims)):
            assert rel_err(g.get_activation(l), ref.activation(l)) <= 5e-2, "activation %d" % l
        for k in range(g.K):
            assert rel_err(g.get_grads(k), ref.get_grads(k)) <= 5e-2
            assert rel_err(g.get_params(k), ref.get_params(k)) <= 5e-2
