"""GPU parity of gad_augment (importance-based subgraph augmentation, Algorithm 1) through the C ABI: integer work
with a counter-based generator on both sides, so the replication-node lists and the numbers of walks must equal the
oracle's exactly."""
import numpy as np
import pytest

import __graft_entry__ as entry
from gad_synth import make_workload, glorot_params
from gad_synth.graphs import sbm_graph
from gad_synth.partition import contiguous_partition, bfs_partition
from conftest import small_random_case, rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    entry.build()


def _both(n, rowptr, col, cores, steps, **kw):
    import paper_2110_02987_b200 as pkg
    from oracle import augment_oracle as aug
    got, walks = pkg.augment(n, rowptr, col, cores, steps, **kw)
    want, info = aug.augment(n, rowptr, col, cores, steps, **kw)
    assert walks.tolist() == [it["n"] for it in info]
    assert len(got) == len(want)
    for k, (a, b) in enumerate(zip(got, want)):
        assert np.array_equal(a, b), "subgraph %d" % k
    return got, info


@pytest.mark.parametrize("steps,alpha,seed", [(1, 0.05, 0), (2, 0.08, 7), (3, 0.02, 123456789), (4, 0.3, 5)])
def test_block_model_partition(steps, alpha, seed):
    rng = np.random.default_rng(seed)
    rowptr, col, block = sbm_graph(4, 200, 0.05, 0.004, rng)
    got, info = _both(800, rowptr, col, contiguous_partition(800, 4), steps, alpha=alpha, seed=seed)
    assert sum(len(h) for h in got) > 0


def test_power_law_graph_with_breadth_first_blocks_and_more_walks_than_the_first_batch():
    w = make_workload("c2", scale=0.02)
    cores = bfs_partition(w.rowptr, w.col, 4)
    got, info = _both(w.n, w.rowptr, w.col, cores, 2, alpha=0.05, E=0.02, seed=3, cap=6)
    assert any(it["n"] > it["n0"] for it in info)          # the error equation asked for more walks somewhere


def test_degenerate_partitions():
    n, rowptr, col, w, core, halo = small_random_case(5, n=60, K=3)
    cores = [np.arange(n, dtype=np.int32)]                  # no boundary at all
    _both(n, rowptr, col, cores, 2)
    cores = [np.array([7], dtype=np.int32), np.empty(0, dtype=np.int32), np.setdiff1d(np.arange(n), [7]).astype(np.int32)]
    _both(n, rowptr, col, cores, 3, alpha=0.5, seed=2)      # a single node, an empty set, the rest


def test_augmented_subgraphs_train_like_the_oracle():
    """The lists go straight into gad_create as the replicated nodes."""
    import paper_2110_02987_b200 as pkg
    from oracle import gad_oracle as orc
    w = make_workload("tiny_signal")
    cores = w.core
    halos, _ = pkg.augment(w.n, w.rowptr, w.col, cores, len(w.dims) - 1, alpha=0.05, seed=1)
    assert all(len(h) > 0 for h in halos)
    w.halo = halos
    theta = glorot_params(w.dims, np.random.default_rng(2))
    ref = orc.from_workload(w, theta)
    with pkg.from_workload(w, theta) as g:
        for _ in range(3):
            assert np.max(np.abs(g.train_epoch() - ref.train_epoch())) <= 1e-4
        assert rel_err(g.get_params(0), ref.get_params(0)) <= 1e-4


def test_leading_walks_that_do_not_suffice():
    """The device hands the host only the best-ranked walks (here 1024 of about 9000).  3000 core nodes that all touch one
    outside hub and one private outside node each: every top-ranked walk ends on the hub, so the leading stretch yields a
    single replication node and the ranking of all walks has to follow - with the same lists as the oracle."""
    m = 3000
    hub = m
    src = np.concatenate([np.arange(m), np.full(m, hub), np.arange(m), m + 1 + np.arange(m)])
    dst = np.concatenate([np.full(m, hub), np.arange(m), m + 1 + np.arange(m), np.arange(m)])
    ring = np.arange(m)
    src = np.concatenate([src, ring, (ring + 1) % m]); dst = np.concatenate([dst, (ring + 1) % m, ring])
    n = 2 * m + 1
    order = np.lexsort((dst, src))
    src, dst = src[order], dst[order]
    rowptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(np.bincount(src, minlength=n), out=rowptr[1:])
    cores = [np.arange(m, dtype=np.int32), np.arange(m, n, dtype=np.int32)]
    got, info = _both(n, rowptr, dst.astype(np.int32), cores, 1, alpha=0.05, seed=9)
    assert len(got[0]) > 100 and info[0]["n"] > 1024


def test_a_second_call_reuses_the_graph_on_the_device():
    """Augmenter keeps its workspace: from the second call on the graph is not uploaded again (graph_resident), whatever
    the partition, the seed or the walk length of that call; a call that needs a larger workspace uploads it afresh."""
    import paper_2110_02987_b200 as pkg
    from oracle import augment_oracle as aug
    w = make_workload("c2", scale=0.03)
    a = pkg.Augmenter(w.n, w.rowptr, w.col)
    for K, steps, seed, cap in ((4, 2, 0, 4), (4, 3, 5, 4), (6, 2, 1, 2), (2, 2, 2, 8)):
        cores = bfs_partition(w.rowptr, w.col, K)
        got, walks = a.run(cores, steps, alpha=0.03, seed=seed, cap=cap)
        want, info = aug.augment(w.n, w.rowptr, w.col, cores, steps, alpha=0.03, seed=seed, cap=cap)
        assert walks.tolist() == [it["n"] for it in info]
        for x, y in zip(got, want):
            assert np.array_equal(x, y)
