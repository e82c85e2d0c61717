"""GPU parity at the two largest configurations (c4: 2.45 M nodes, 118 M entries, K = 16, 100-256-256-47; c3 with
K = 8: 233 000 nodes of mean degree 490, 602-256-41, the layer that transforms before it aggregates), where a whole
oracle epoch takes minutes: bit-exact store bookkeeping, sampled output rows the oracle's definitions
give one by one (layer 1 from the inputs alone; deeper layers from the layer below), and properties that hold at
any size (scatter of the logits, loss from the logits, equal replicas after the consensus, importance weights)."""
import numpy as np
import pytest

import __graft_entry__ as entry
from gad_synth import make_workload, glorot_params
from test_gpu_parity import check_store

pytestmark = pytest.mark.gpu

TOL = 1e-4


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
    w = make_workload(name)
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
