"""GPU parity at the largest configurations (c4: 2.45 M nodes, 118 M entries, K = 16, 100-256-256-47; c3 with
K = 8 and K = 4: 233 000 nodes of mean degree 490, 602-256-41, the layer that transforms before it aggregates; one
point of the sweep: 1 M nodes, mean degree 32, 256 features, K = 8), where a whole oracle epoch takes minutes:
  - bit-exact store bookkeeping, sampled output rows the oracle's definitions give one by one (layer 1 from the
    inputs alone; deeper layers from the layer below), and properties that hold at any size (scatter of the logits,
    loss from the logits, equal replicas after the consensus, importance weights);
  - the whole forward and backward pass of single subgraphs (the first, the middle one and the last) against the
    oracle run on that subgraph alone: a replica's activations, loss and gradient depend on its own subgraph only, so an
    oracle with K = 1 over g'_k gives them exactly; then the parameters after the epoch against theta - eta sum_k w_k g_k
    formed with those oracle gradients;
  - the ten-epoch loss curve of c3 (K = 8) against whole oracle epochs."""
import functools

import numpy as np
import pytest

import __graft_entry__ as entry
from gad_synth import make_workload, glorot_params
from conftest import rel_err
from test_gpu_parity import check_store

pytestmark = pytest.mark.gpu

TOL = 1e-4


@functools.lru_cache(maxsize=2)
def workload(name):
    """The two workloads built last stay in memory (a few GB): the tests of c4 and c3k8 alternate."""
    if name.startswith("sweep"):
        _, deg, F, K = name.split("_")
        return make_workload("sweep", mean_deg=float(deg[1:]), F=int(F[1:]), K=int(K[1:]))
    return make_workload(name)


def unpack(theta, dims):
    """[W_0, b_0, W_1, b_1, ...] from the flat parameter vector (W_l row-major [F_l x F_{l+1}])."""
    out, o = [], 0
    for fi, fo in zip(dims[:-1], dims[1:]):
        W = theta[o:o + fi * fo].reshape(fi, fo).astype(np.float64); o += fi * fo
        b = theta[o:o + fo].astype(np.float64); o += fo
        out.append((W, b))
    assert o == theta.shape[0]
    return out


@pytest.mark.parametrize("name", ["c4", "c3k8"])
def test_full_size_sampled_rows_and_properties(name):
    entry.build()
    import paper_2110_02987_b200 as pkg
    from oracle import gad_oracle as orc
    orc.build()
    w = workload(name)
    dims = tuple(w.dims)
    L = len(dims) - 1
    theta = glorot_params(dims, np.random.default_rng(0), bias_scale=0.2)
    cp, cn, hp, hn = w.flat_partition()
    st = orc.Store(w.n, w.rowptr, w.col, cp, cn, hp, hn)
    layers = unpack(theta, dims)
    rng = np.random.default_rng(123)
    with pkg.from_workload(w, theta) as g:
        check_store(g, st)                                   # every index bit-exact, every value within 1 ulp
        logits = g.forward()
        H = [None] + [g.get_activation(l) for l in range(1, L + 1)]

        # rows to check: the longest row, the first and last row of some subgraphs, a few halo rows, random rows
        lens = np.diff(st.rowptr)
        rows = {int(np.argmax(lens)), 0, st.n_prime - 1}
        for k in (0, st.K // 2, st.K - 1):
            rows.update({int(st.sub_off[k]), int(st.sub_off[k + 1] - 1), int(st.sub_off[k] + st.core_count[k])})
        rows.update(int(r) for r in rng.integers(0, st.n_prime, size=40))
        rows = sorted(r for r in rows if 0 <= r < st.n_prime)

        for l in range(L):
            W_b = layers[l]
            got = H[l + 1][rows].astype(np.float64)
            want = np.empty_like(got)
            for i, r in enumerate(rows):
                e0, e1 = st.rowptr[r], st.rowptr[r + 1]
                cols, vals = st.col[e0:e1], st.val[e0:e1]
                below = w.X[st.gid[cols]].astype(np.float64) if l == 0 else H[l][cols].astype(np.float64)
                pre = (vals @ below) @ W_b[0] + W_b[1]
                want[i] = pre if l == L - 1 else np.maximum(pre, 0.0)
            err = np.max(np.abs(got - want)) / np.max(np.abs(want))
            assert err <= TOL, "layer %d sampled rows: %g" % (l + 1, err)

        # logits in global node order are the core rows of H^(L), bit for bit; uncovered rows stay zero
        core_rows = np.concatenate([np.arange(st.sub_off[k], st.sub_off[k] + st.core_count[k]) for k in range(st.K)])
        assert np.array_equal(logits[st.gid[core_rows]], H[L][core_rows])

        # one epoch: each subgraph's loss is the mean cross-entropy of its own training core rows
        loss = g.train_epoch()
        z = H[L].astype(np.float64)
        total, count = 0.0, 0
        for k in range(st.K):
            r = np.arange(st.sub_off[k], st.sub_off[k] + st.core_count[k])
            r = r[w.split[st.gid[r]] == 0]
            zz = z[r]
            m = zz.max(axis=1)
            ce = m + np.log(np.exp(zz - m[:, None]).sum(axis=1)) - zz[np.arange(len(r)), w.labels[st.gid[r]]]
            assert abs(loss[k] - ce.mean()) <= 1e-4 * max(1.0, abs(ce.mean())), "loss of subgraph %d" % k
            total += ce.sum(); count += len(r)
        assert abs(loss[st.K] - total / count) <= 1e-4 * max(1.0, total / count)

        # weighted consensus leaves K identical replicas; the weights are those of the oracle's zeta
        p0 = g.get_params(0)
        assert np.all(np.isfinite(p0))
        for k in (1, st.K - 1):
            assert np.array_equal(p0, g.get_params(k))
        zg, wg = g.subgraph_weights()
        zr = np.array([orc.zeta_aggregate(st.deg[st.sub_off[k]:st.sub_off[k + 1]], w.X[st.gid[st.sub_off[k]:st.sub_off[k + 1]]])
                       for k in range(st.K)])
        assert np.max(np.abs(zg - zr)) <= 1e-6 * np.max(zr)
        assert np.max(np.abs(wg - zr / zr.sum())) <= 1e-6


def one_subgraph(w, k):
    """The workload reduced to subgraph k (for an oracle with K = 1)."""
    sub = type(w)(**{**w.__dict__})
    sub.core, sub.halo = [w.core[k]], [w.halo[k]]
    return sub


@pytest.mark.parametrize("name", ["c4", "c3k8", "c3k4", "sweep_d32_f256_k8"])
def test_full_size_backward_pass_of_single_subgraphs(name):
    """Everything the backward pass writes, at full size, in the launch configuration the benchmark times (a stream of
    its own: the second and third epoch below are graph replays): for k in {0, K/2, K-1} the oracle runs forward,
    loss and backward on g'_k alone and the library's replica k must match it element by element - activations of
    every layer, the subgraph loss, and the gradient of every parameter - within 1e-4; the parameters after the
    epoch must be theta - eta sum_k w_k g_k with the oracle's gradients for those k (the library's own for the
    others) and the oracle's importance weights."""
    import torch
    entry.build()
    import paper_2110_02987_b200 as pkg
    from oracle import gad_oracle as orc
    orc.build()
    w = workload(name)
    dims = tuple(w.dims)
    L = len(dims) - 1
    theta = glorot_params(dims, np.random.default_rng(0), bias_scale=0.2)
    lr = 0.5                                     # large enough for the update to show in the parameters
    ks = sorted({0, w.K // 2, w.K - 1})
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        with pkg.from_workload(w, theta, lr=lr, stream=stream) as g:
            off = g.get_store()["sub_off"]
            g.train_epoch_local()                # enqueued launch by launch
            loss = g.train_epoch_local()         # the same pass again, replayed as a graph: same parameters, same result
            grads = [g.get_grads(k) for k in range(g.K)]
            H = [None] + [g.get_activation(l) for l in range(1, L + 1)]
            oracle_grads = {}
            for k in ks:
                ref = orc.from_workload(one_subgraph(w, k), theta, lr=lr)
                r0, r1 = int(off[k]), int(off[k + 1])
                lk = ref.forward_backward()
                # hidden units at the ReLU kink take the library's branch in the oracle (see test_gpu_parity.oracle_step)
                ties = 0
                for _ in range(4):
                    found = False
                    for l in range(1, L):
                        a, b = H[l][r0:r1], ref.activation(l)
                        diff = (a == 0) != (b == 0)
                        if diff.any():
                            worst = float(np.max(np.maximum(np.abs(a[diff]), np.abs(b[diff]))) / np.max(np.abs(b)))
                            assert worst <= 1e-5, "a hidden unit differs across the ReLU and is not a tie (%g)" % worst
                            rows, cols = np.nonzero(diff)
                            on = a[rows, cols] != 0
                            ref.set_relu_branch(l, rows[on], cols[on], 1)
                            ref.set_relu_branch(l, rows[~on], cols[~on], 2)
                            ties += len(rows)
                            found = True
                    if not found:
                        break
                    lk = ref.forward_backward()
                print("%s subgraph %d: %d rows, %d ReLU ties" % (name, k, r1 - r0, ties))
                assert ties <= 64, "%d hidden units at the ReLU kink: more than rounding explains" % ties
                for l in range(1, L + 1):
                    assert rel_err(H[l][r0:r1], ref.activation(l)) <= TOL, "activation %d of subgraph %d" % (l, k)
                assert abs(loss[k] - lk[0]) <= 1e-5 * max(1.0, abs(lk[0])), "loss of subgraph %d" % k
                oracle_grads[k] = ref.get_grads(0)
                assert rel_err(grads[k], oracle_grads[k]) <= TOL, "gradient of replica %d" % k
                # and layer by layer, so that a small layer cannot hide behind a large one
                o = 0
                for l in range(L):
                    for size, what in ((dims[l] * dims[l + 1], "dW"), (dims[l + 1], "db")):
                        assert rel_err(grads[k][o:o + size], oracle_grads[k][o:o + size]) <= TOL, "%s_%d of replica %d" % (what, l, k)
                        o += size
                ref.close()
            # the epoch proper: same gradients (same parameters), then the update and the weighted consensus
            g.train_epoch()
            assert np.array_equal(g.get_grads(ks[-1]), grads[ks[-1]])
            st = g.get_store()
            X0 = g.get_activation(0)
            zeta = np.array([orc.zeta_aggregate(st["deg"][off[k]:off[k + 1]], X0[off[k]:off[k + 1]]) for k in range(g.K)])
            wts = zeta / zeta.sum()
            want = theta.astype(np.float64).copy()
            for k in range(g.K):
                want -= lr * wts[k] * (oracle_grads[k] if k in oracle_grads else grads[k].astype(np.float64))
            got = g.get_params(0)
            assert rel_err(got, want) <= TOL
            step = want - theta.astype(np.float64)
            assert np.max(np.abs(step)) > 1e-3 * np.max(np.abs(theta))          # the update is visible at this tolerance
            assert rel_err(got.astype(np.float64) - theta.astype(np.float64), step) <= 1e-3   # fp32 parameters: 6e-8 |theta| of rounding in the difference
            for k in (1, g.K - 1):
                assert np.array_equal(got, g.get_params(k))


def test_c3k8_ten_epoch_loss_curve_against_whole_oracle_epochs():
    """The loss curve over ten epochs at full size (c3, K = 8), in the benchmark's launch configuration, within 1e-3 of
    the oracle's whole epochs; parameters within 1e-4 at the end."""
    import torch
    entry.build()
    import paper_2110_02987_b200 as pkg
    from oracle import gad_oracle as orc
    orc.build()
    w = workload("c3k8")
    theta = glorot_params(w.dims, np.random.default_rng(0), bias_scale=0.2)
    lr = 0.5
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        with pkg.from_workload(w, theta, lr=lr, stream=stream) as g:
            lg = np.array([g.train_epoch() for _ in range(10)])
            pg = g.get_params(0)
    ref = orc.from_workload(w, theta, lr=lr)
    lo = np.array([ref.train_epoch() for _ in range(10)])
    assert np.max(np.abs(lg - lo)) <= 1e-3, np.max(np.abs(lg - lo))
    assert lo[0, -1] - lo[-1, -1] > 5e-3                  # the curve moves by several times the tolerance
    assert rel_err(pg, ref.get_params(0)) <= TOL
