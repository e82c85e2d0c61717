"""Pins for the augmentation oracle (Algorithm 1, Section 3.2.2): the generator against the published splitmix64
vectors, the walks against the graph, the counts against a recount written here, the number of walks against the
Monte-Carlo error equation evaluated with numpy's mean and standard deviation, the visit frequencies against their
exact probabilities for one-step walks, and the selection against the properties the paper states for it."""
import math
import os

import numpy as np

from oracle import augment_oracle as aug
from conftest import small_random_case
from gad_synth.graphs import sbm_graph
from gad_synth.partition import contiguous_partition

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "splitmix64.txt")


def test_mix_is_the_splitmix64_output_function():
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        seed, *outs = [int(t) for t in line.split()]
        state = np.uint64(seed)
        for want in outs:
            with np.errstate(over="ignore"):
                state = state + aug.G64
            assert int(aug.mix64(state)) == want


def _graph(seed=0):
    rng = np.random.default_rng(seed)
    rowptr, col, block = sbm_graph(4, 60, 0.08, 0.01, rng)
    return 240, rowptr, col, contiguous_partition(240, 4)


def test_walks_start_on_the_boundary_and_follow_edges():
    n, rowptr, col, cores = _graph()
    halos, info = aug.augment(n, rowptr, col, cores, 3, alpha=0.05, seed=5)
    for k, it in enumerate(info):
        B = set(int(b) for b in it["boundary"])
        inside = np.zeros(n, bool); inside[cores[k]] = True
        for b in B:     # a boundary node is a core node with an outside neighbour, and every such node is listed
            assert inside[b] and np.any(~inside[col[rowptr[b]:rowptr[b + 1]]])
        assert len(B) == sum(1 for v in cores[k] if np.any(~inside[col[rowptr[v]:rowptr[v + 1]]]))
        assert it["n0"] == sum(int(rowptr[b + 1] - rowptr[b]) for b in B)      # d |B| with d the average boundary degree
        for w in it["walks"]:
            assert int(w[0]) in B
            for a, b in zip(w[:-1], w[1:]):
                assert int(b) in set(int(c) for c in col[rowptr[a]:rowptr[a + 1]])


def test_counts_scores_and_number_of_walks():
    n, rowptr, col, cores = _graph(1)
    halos, info = aug.augment(n, rowptr, col, cores, 2, alpha=0.05, E=0.05, seed=9, cap=3)
    for k, it in enumerate(info):
        inside = np.zeros(n, bool); inside[cores[k]] = True
        recount = np.zeros(n, np.int64)
        for w in it["walks"]:
            for v in np.unique(w):
                if not inside[v]:
                    recount[v] += 1
        assert np.array_equal(recount, it["count"])
        assert not np.any(it["count"][cores[k]])
        want = np.array([sum(int(recount[v]) for v in np.unique(w) if not inside[v]) for w in it["walks"]])
        assert np.array_equal(want, it["scores"])
        # the number of walks from the first batch alone, by the error equation with numpy's statistics
        first = np.zeros(n, np.int64)
        for w in it["walks"][: it["n0"]]:
            for v in np.unique(w):
                if not inside[v]:
                    first[v] += 1
        prob = first[first > 0] / float(it["n0"])
        direct = (1.96 * prob.std() / (prob.mean() * 0.05)) ** 2
        assert it["n"] == max(it["n0"], min(3 * it["n0"], math.ceil(direct))) or abs(it["n"] - math.ceil(direct)) <= 1
        assert it["n0"] <= it["n"] <= 3 * it["n0"] and it["walks"].shape[0] == it["n"]


def test_one_step_visit_frequencies_approach_their_probabilities():
    n, rowptr, col, cores = _graph(2)
    halos, info = aug.augment(n, rowptr, col, cores, 1, alpha=0.05, seed=3, cap=8)
    it = info[0]
    B = it["boundary"]
    p = np.zeros(n)
    for b in B:                       # P(walk visits v) = sum_b 1/|B| * (edges b -> v) / deg(b)
        nb = col[rowptr[b]:rowptr[b + 1]]
        for v in nb:
            p[v] += 1.0 / (len(B) * len(nb))
    inside = np.zeros(n, bool); inside[cores[0]] = True
    p[inside] = 0.0
    freq = it["count"] / float(it["n"])
    sigma = np.sqrt(p * (1 - p) / it["n"])
    assert np.all(np.abs(freq - p) <= 5 * sigma + 1e-12)
    assert np.all((p > 0) | (it["count"] == 0))


def test_selection_takes_walks_in_order_of_importance_without_dangling_nodes():
    n, rowptr, col, cores = _graph(3)
    halos, info = aug.augment(n, rowptr, col, cores, 3, alpha=0.08, seed=11)
    for k, (h, it) in enumerate(zip(halos, info)):
        inside = np.zeros(n, bool); inside[cores[k]] = True
        nv = len(cores[k])
        directed = sum(int(np.sum(inside[col[rowptr[v]:rowptr[v + 1]]] & (col[rowptr[v]:rowptr[v + 1]] != v))) for v in cores[k])
        dens = directed / (nv * (nv - 1.0))
        assert it["n_rep"] == min(math.floor(0.08 * (1 + dens) * nv), int(np.sum(it["count"] > 0)))
        assert len(h) == it["n_rep"] and len(set(h.tolist())) == len(h) and not np.any(inside[h])
        # no dangling node: each selected node is joined to the subgraph through nodes selected before it
        reach = inside.copy()
        for v in h:
            assert np.any(reach[col[rowptr[v]:rowptr[v + 1]]]) or np.any([v in col[rowptr[u]:rowptr[u + 1]] for u in np.nonzero(reach)[0]])
            reach[v] = True
        # the first selected nodes are the outside nodes of the best walk
        best = int(np.lexsort((np.arange(it["n"]), -it["scores"]))[0])
        first = []
        for v in it["walks"][best]:
            if not inside[v] and int(v) not in first:
                first.append(int(v))
        assert h[: len(first)].tolist() == first[: len(h)]


def test_density_of_a_complete_core_and_determinism():
    n = 30
    A = np.ones((n, n), bool)
    src, dst = np.nonzero(A)
    rowptr = np.zeros(n + 1, np.int64); np.cumsum(np.bincount(src, minlength=n), out=rowptr[1:])
    cores = [np.arange(0, 15, dtype=np.int32), np.arange(15, 30, dtype=np.int32)]
    halos, info = aug.augment(n, rowptr, dst.astype(np.int32), cores, 2, alpha=0.1, seed=1)
    assert [it["n_rep"] for it in info] == [3, 3]           # floor(0.1 * (1 + 1) * 15)
    again, _ = aug.augment(n, rowptr, dst.astype(np.int32), cores, 2, alpha=0.1, seed=1)
    other, _ = aug.augment(n, rowptr, dst.astype(np.int32), cores, 2, alpha=0.1, seed=2)
    assert all(np.array_equal(a, b) for a, b in zip(halos, again))
    assert any(not np.array_equal(a, b) for a, b in zip(halos, other))


def test_a_subgraph_without_boundary_gets_no_replication_nodes():
    n, rowptr, col, w, core, halo = small_random_case(3, n=30, K=2)
    whole = [np.arange(n, dtype=np.int32)]
    halos, info = aug.augment(n, rowptr, col, whole, 2)
    assert len(halos[0]) == 0 and info[0]["n"] == 0
