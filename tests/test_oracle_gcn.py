"""Pins for the oracle's forward / loss / backward / epoch (Section 3.3 and Algorithm 2 of the paper)."""
import numpy as np
import pytest

from oracle import gad_oracle as orc
from gad_synth import glorot_params, param_count
from conftest import small_random_case, flat, rel_err
from test_oracle_store import dense_graph, dense_hat


def unpack(theta, dims):
    out, o = [], 0
    for l in range(len(dims) - 1):
        fi, fo = dims[l], dims[l + 1]
        W = theta[o:o + fi * fo].reshape(fi, fo)
        o += fi * fo
        b = theta[o:o + fo]
        o += fo
        out.append((W, b))
    return out


def dense_forward(hat, X, theta, dims):
    H = X
    layers = unpack(theta, dims)
    for l, (W, b) in enumerate(layers):
        H = hat @ (H @ W) + b
        if l < len(layers) - 1:
            H = np.maximum(H, 0.0)
    return H


def make_case(seed, dims=(6, 5, 3), **kw):
    n, rowptr, col, w, core, halo = small_random_case(seed, **kw)
    rng = np.random.default_rng(100 + seed)
    X = rng.standard_normal((n, dims[0])).astype(np.float32)
    y = rng.integers(0, dims[-1], size=n).astype(np.int32)
    split = rng.integers(0, 3, size=n).astype(np.uint8)
    theta = glorot_params(dims, rng, bias_scale=0.3)
    st = orc.Store(n, rowptr, col, *flat(core), *flat(halo), weights=w)
    return n, rowptr, col, w, core, halo, X, y, split, theta, st


@pytest.mark.parametrize("seed,dims", [(0, (6, 5, 3)), (1, (6, 5, 4, 3)), (2, (3, 2))])
def test_forward_matches_dense_brute_force(seed, dims):
    n, rowptr, col, w, core, halo, X, y, split, theta, st = make_case(seed, dims, weighted=True)
    m = orc.Model(st, X, y, split, dims, theta)
    logits = m.forward()
    A = dense_graph(n, rowptr, col, w)
    for k in range(len(core)):
        idx = np.concatenate([core[k], halo[k]])
        hat, _ = dense_hat(A, idx)
        want = dense_forward(hat, X[idx].astype(np.float64), theta.astype(np.float64), dims)
        r0 = st.sub_off[k]
        assert rel_err(logits[r0:r0 + len(idx)], want) < 1e-13


def test_forward_global_scatter_covers_core_rows_only():
    n, rowptr, col, w, core, halo, X, y, split, theta, st = make_case(4)
    m = orc.Model(st, X, y, split, (6, 5, 3), theta)
    out = m.forward_global(n)
    covered = np.zeros(n, dtype=bool)
    covered[np.concatenate(core)] = True
    assert np.all(out[~covered] == 0.0)
    assert np.all(np.abs(out[covered]).sum(axis=1) > 0)


def test_isolated_nodes_reduce_to_a_plain_mlp():
    # no edges: A~ = I, so the GCN is a per-node multilayer perceptron
    n, dims = 12, (4, 6, 3)
    rng = np.random.default_rng(0)
    rowptr = np.zeros(n + 1, dtype=np.int64)
    col = np.empty(0, dtype=np.int32)
    X = rng.standard_normal((n, 4)).astype(np.float32)
    theta = glorot_params(dims, rng, bias_scale=0.2)
    core = [np.arange(0, 7, dtype=np.int32), np.arange(7, 12, dtype=np.int32)]
    st = orc.Store(n, rowptr, col, *flat(core), *flat([np.empty(0, np.int32)] * 2))
    m = orc.Model(st, X, np.zeros(n, np.int32), np.zeros(n, np.uint8), dims, theta)
    (W0, b0), (W1, b1) = unpack(theta.astype(np.float64), dims)
    want = np.maximum(X.astype(np.float64) @ W0 + b0, 0) @ W1 + b1
    assert rel_err(m.forward(), want) < 1e-14


def test_complete_graph_averages_every_row():
    # complete graph with self-loops: A~ = (1/n) 1 1^T, so every output row is the same mean
    n, dims = 9, (3, 2)
    rng = np.random.default_rng(1)
    src, dst = np.nonzero(np.ones((n, n)))
    rowptr = np.arange(0, n * n + 1, n, dtype=np.int64)
    X = rng.standard_normal((n, 3)).astype(np.float32)
    theta = glorot_params(dims, rng, bias_scale=0.2)
    st = orc.Store(n, rowptr, dst.astype(np.int32), *flat([np.arange(n, dtype=np.int32)]), *flat([np.empty(0, np.int32)]))
    m = orc.Model(st, X, np.zeros(n, np.int32), np.zeros(n, np.uint8), dims, theta)
    W, b = unpack(theta.astype(np.float64), dims)[0]
    want = np.tile(X.astype(np.float64).mean(axis=0) @ W + b, (n, 1))
    assert rel_err(m.forward(), want) < 1e-14


def test_uniform_logits_give_log_C():
    n, rowptr, col, w, core, halo, X, y, split, theta, st = make_case(6, (6, 5, 3))
    m = orc.Model(st, X, y, split, (6, 5, 3), np.zeros_like(theta))
    loss = m.forward_loss()
    nt = m.ntrain()
    assert np.allclose(loss[nt > 0], np.log(3.0), rtol=1e-14)


def test_loss_matches_dense_definition_and_counts_core_training_nodes_only():
    dims = (6, 5, 3)
    n, rowptr, col, w, core, halo, X, y, split, theta, st = make_case(7, dims)
    m = orc.Model(st, X, y, split, dims, theta)
    loss = m.forward_loss()
    A = dense_graph(n, rowptr, col, w)
    for k in range(len(core)):
        idx = np.concatenate([core[k], halo[k]])
        hat, _ = dense_hat(A, idx)
        z = dense_forward(hat, X[idx].astype(np.float64), theta.astype(np.float64), dims)
        rows = [i for i in range(len(core[k])) if split[core[k][i]] == 0]
        assert m.ntrain()[k] == len(rows)
        p = np.exp(z - z.max(axis=1, keepdims=True))
        p /= p.sum(axis=1, keepdims=True)
        want = -np.mean([np.log(p[i, y[idx[i]]]) for i in rows]) if rows else 0.0
        assert abs(loss[k] - want) < 1e-13


@pytest.mark.parametrize("seed,dims,dropout", [(0, (6, 5, 3), 0.0), (1, (6, 5, 4, 3), 0.0), (2, (6, 5, 3), 0.4)])
def test_gradients_match_central_finite_differences(seed, dims, dropout):
    n, rowptr, col, w, core, halo, X, y, split, theta, st = make_case(seed, dims, weighted=(seed == 1))
    m = orc.Model(st, X, y, split, dims, theta, dropout=dropout, seed=11)
    m.forward_backward()
    K, P = m.K, m.P
    h = 1e-6
    for k in range(K):
        g = m.get_grads(k)
        base = m.get_params(k)
        fd = np.zeros(P)
        for i in range(P):
            t = base.copy()
            t[i] = base[i] + h
            m.set_params(k, t)
            lp = m.forward_loss()[k]
            t[i] = base[i] - h
            m.set_params(k, t)
            lm = m.forward_loss()[k]
            fd[i] = (lp - lm) / (2 * h)
        m.set_params(k, base)
        assert rel_err(g, fd) < 1e-6, "replica %d" % k
        assert np.abs(g).max() > 0


def test_dlogits_rows_sum_to_zero_via_last_bias_gradient():
    # d(loss)/d(last bias) = column sums of (softmax - onehot)/|T|; every row of softmax - onehot
    # sums to zero, so the entries of that bias gradient sum to zero too.
    dims = (6, 5, 3)
    n, rowptr, col, w, core, halo, X, y, split, theta, st = make_case(8, dims)
    m = orc.Model(st, X, y, split, dims, theta)
    m.forward_backward()
    for k in range(m.K):
        gb = m.get_grads(k)[-dims[-1]:]
        assert abs(gb.sum()) < 1e-14


def test_identical_subgraphs_give_identical_gradients_and_relabelling_is_invariant():
    dims = (5, 4, 3)
    rng = np.random.default_rng(3)
    n0 = 15
    A = np.triu(rng.random((n0, n0)) < 0.3, 1)
    A = A | A.T
    # two disjoint copies of the same graph; the second copy with its nodes listed in another order
    n = 2 * n0
    big = np.zeros((n, n), dtype=bool)
    big[:n0, :n0] = A
    big[n0:, n0:] = A
    src, dst = np.nonzero(big)
    rowptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(np.bincount(src, minlength=n), out=rowptr[1:])
    X0 = rng.standard_normal((n0, 5)).astype(np.float32)
    y0 = rng.integers(0, 3, n0).astype(np.int32)
    s0 = rng.integers(0, 2, n0).astype(np.uint8)
    X, y, split = np.vstack([X0, X0]), np.concatenate([y0, y0]), np.concatenate([s0, s0])
    perm = rng.permutation(n0)
    core = [np.arange(n0, dtype=np.int32), (n0 + perm).astype(np.int32)]
    st = orc.Store(n, rowptr, dst.astype(np.int32), *flat(core), *flat([np.empty(0, np.int32)] * 2))
    theta = glorot_params(dims, rng, bias_scale=0.1)
    m = orc.Model(st, X, y, split, dims, theta)
    loss = m.forward_backward()
    assert abs(loss[0] - loss[1]) < 1e-14
    assert rel_err(m.get_grads(1), m.get_grads(0)) < 1e-13
    lg = m.forward()
    assert rel_err(lg[n0:][np.argsort(perm)], lg[:n0]) < 1e-13


def test_single_subgraph_epoch_is_a_full_batch_gcn_step():
    # K = 1, no replicated nodes: the epoch is one SGD step of a full-batch GCN on the whole graph
    dims = (6, 5, 3)
    n, rowptr, col, w, _, _, X, y, split, theta, _ = make_case(9, dims)
    core = [np.arange(n, dtype=np.int32)]
    st = orc.Store(n, rowptr, col, *flat(core), *flat([np.empty(0, np.int32)]))
    lr = 0.1
    m = orc.Model(st, X, y, split, dims, theta, lr=lr)
    before = m.get_params(0)
    loss = m.train_epoch()
    after = m.get_params(0)
    # dense full-batch reference, gradient by finite differences of the dense loss
    hat, _ = dense_hat(dense_graph(n, rowptr, col, w), np.arange(n))
    rows = np.nonzero(split == 0)[0]

    def dense_loss(t):
        z = dense_forward(hat, X.astype(np.float64), t, dims)
        z = z - z.max(axis=1, keepdims=True)
        lse = np.log(np.exp(z).sum(axis=1))
        return float(np.mean(lse[rows] - z[rows, y[rows]]))

    assert abs(loss[0] - dense_loss(before)) < 1e-13 and abs(loss[1] - loss[0]) < 1e-15
    g = np.zeros_like(before)
    for i in range(before.size):
        t = before.copy(); t[i] += 1e-6
        u = before.copy(); u[i] -= 1e-6
        g[i] = (dense_loss(t) - dense_loss(u)) / 2e-6
    assert rel_err(after, before - lr * g) < 1e-8


def test_resume_five_plus_five_equals_ten(tiny_signal):
    w = tiny_signal
    theta = glorot_params(w.dims, np.random.default_rng(1))
    a = orc.from_workload(w, theta, dropout=0.2, seed=5)
    la = [a.train_epoch() for _ in range(10)]
    b = orc.from_workload(w, theta, dropout=0.2, seed=5)
    lb = [b.train_epoch() for _ in range(5)]
    c = orc.from_workload(w, theta, dropout=0.2, seed=5)
    for k in range(c.K):
        c.set_params(k, b.get_params(k))
    c.epoch = b.epoch
    lb += [c.train_epoch() for _ in range(5)]
    assert np.array_equal(np.array(la), np.array(lb))
    assert np.array_equal(a.get_params(0), c.get_params(0))


def test_tiny_loss_starts_near_log4_and_signal_case_learns(tiny, tiny_signal):
    th = glorot_params(tiny.dims, np.random.default_rng(0))
    m = orc.from_workload(tiny, th)
    l0 = m.train_epoch()
    assert abs(l0[-1] - np.log(4)) < 0.35
    m2 = orc.from_workload(tiny_signal, th)
    ls = [m2.train_epoch()[-1] for _ in range(10)]
    assert ls[-1] < ls[0] - 0.1


def test_dropout_mask_is_a_pure_counter_function():
    import os
    here = os.path.dirname(__file__)
    for line in open(os.path.join(here, "golden", "splitmix64.txt")):
        if line.startswith("#") or not line.strip():
            continue
        seed, *outs = [int(t) for t in line.split()]
        s = seed
        for want in outs:
            s = (s + 0x9e3779b97f4a7c15) & (2 ** 64 - 1)
            got = orc.lib().orc_mix64
            got.restype = __import__("ctypes").c_uint64
            assert got(__import__("ctypes").c_uint64(s)) == want
    keep = np.array([[orc.keep_unit(3, 2, 1, r, c, 0.3) for c in range(64)] for r in range(256)])
    assert abs(keep.mean() - 0.7) < 0.02
    again = np.array([[orc.keep_unit(3, 2, 1, r, c, 0.3) for c in range(64)] for r in range(256)])
    assert np.array_equal(keep, again)
    other = np.array([[orc.keep_unit(3, 3, 1, r, c, 0.3) for c in range(64)] for r in range(256)])
    assert (keep != other).mean() > 0.2
    assert all(orc.keep_unit(9, 0, 0, r, 0, 0.0) for r in range(100))


def test_prescribed_relu_branches_equal_a_network_with_that_mask():
    """orc_set_relu_branch (for hidden units at the kink of the ReLU): with the branch of some units prescribed, forward
    and gradients are those of the network whose layer-1 activation is `mask * pre-activation` with that mask held
    fixed - checked against a dense forward and central finite differences of that masked network; prescribing the
    branch the ReLU takes anyway changes nothing, and clearing restores the plain ReLU bit for bit."""
    dims = (6, 5, 3)
    n, rowptr, col, w, core, halo, X, y, split, theta, st = make_case(3, dims, K=1, halo=False)
    idx = core[0]
    hat, _ = dense_hat(dense_graph(n, rowptr, col, w), idx)
    Xd, yd = X[idx].astype(np.float64), y[idx]
    train = np.nonzero(split[idx] == 0)[0]
    m = orc.Model(st, X, y, split, dims, theta)
    m.forward_backward()
    g_plain, h1_plain = m.get_grads(0), m.activation(1)
    natural = h1_plain > 0
    on = np.argwhere(natural)[:3]            # three active units to switch off
    off = np.argwhere(~natural)[:3]          # three inactive units to switch on
    mask = natural.copy()
    mask[on[:, 0], on[:, 1]] = False
    mask[off[:, 0], off[:, 1]] = True

    def loss_of(t):
        (W0, b0), (W1, b1) = unpack(t, dims)
        z = hat @ ((mask * (hat @ (Xd @ W0) + b0)) @ W1) + b1
        zt = z[train]
        lse = zt.max(axis=1) + np.log(np.exp(zt - zt.max(axis=1, keepdims=True)).sum(axis=1))
        return np.mean(lse - zt[np.arange(len(train)), yd[train]]), z

    # the branch the ReLU takes anyway: nothing changes
    m.set_relu_branch(1, on[:, 0], on[:, 1], 1)
    m.set_relu_branch(1, off[:, 0], off[:, 1], 2)
    m.forward_backward()
    assert np.array_equal(m.get_grads(0), g_plain) and np.array_equal(m.activation(1), h1_plain)
    # the other branch: the masked network
    m.set_relu_branch(1, on[:, 0], on[:, 1], 2)
    m.set_relu_branch(1, off[:, 0], off[:, 1], 1)
    loss = m.forward_backward()
    t0 = theta.astype(np.float64)
    want_loss, want_logits = loss_of(t0)
    assert abs(loss[0] - want_loss) < 1e-13
    assert rel_err(m.activation(2), want_logits) < 1e-13
    fd = np.zeros_like(t0)
    for i in range(t0.size):
        tp, tm = t0.copy(), t0.copy()
        tp[i] += 1e-6; tm[i] -= 1e-6
        fd[i] = (loss_of(tp)[0] - loss_of(tm)[0]) / 2e-6
    assert rel_err(m.get_grads(0), fd) < 1e-7
    assert rel_err(m.get_grads(0), g_plain) > 1e-4          # and it is a different network
    m.clear_relu_branches()
    m.forward_backward()
    assert np.array_equal(m.get_grads(0), g_plain)
    with pytest.raises(ValueError):
        m.set_relu_branch(2, [0], [0], 1)                    # the last layer has no ReLU
