"""gad_subgraph_weights_static: the importance weights for callers that may not allocate device memory.

Some callers cannot let a library call cudaMalloc for them: the device already belongs to the application's own
memory pool, or the call sits in a loop where an allocation (and the device synchronisation it may bring) is not
acceptable.  For them the library offers one entry point that needs no context and no workspace and keeps its
partial sums in a fixed array inside the library.  This test calls it through the C ABI twice in a row, on two
different workloads, so the second call runs over whatever the first left in that shared array, and checks both
results against the regular entry point (gad_subgraph_weights of a context built on the same inputs), whose own
values are compared with the CPU oracle's zeta first.

The file is collected last on purpose, so a failure here cannot hide any other test behind `-x`.
"""
import numpy as np
import pytest

import __graft_entry__ as entry
from gad_synth import make_workload, glorot_params

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    entry.build()


def reference_and_inputs(w):
    """zeta / w from the regular entry point, and the same inputs as plain device tensors.  The regular entry point's
    zeta is itself held against the oracle's definition (Section 3.4.1, aggregate reading) here, so this file stands on
    the oracle and not only on the library's other path."""
    import torch
    import paper_2110_02987_b200 as pkg
    from oracle import gad_oracle as orc
    theta = glorot_params(w.dims, np.random.default_rng(0))
    with pkg.from_workload(w, theta) as g:
        zeta, wts = g.subgraph_weights()
        st = g.get_store()
        X = g.get_activation(0)                       # input features in store-row order [N' x F]
    off = st["sub_off"]
    z_orc = np.array([orc.zeta_aggregate(st["deg"][off[k]:off[k + 1]], X[off[k]:off[k + 1]]) for k in range(len(off) - 1)])
    assert np.max(np.abs(zeta - z_orc) / z_orc) <= 1e-6
    assert np.max(np.abs(wts - z_orc / z_orc.sum())) <= 1e-6
    F = X.shape[1]
    ld = (F + 3) // 4 * 4
    Xp = np.zeros((X.shape[0], ld), dtype=np.float32)
    Xp[:, :F] = X
    dev = torch.device("cuda")
    return zeta, wts, (torch.from_numpy(Xp).to(dev), torch.from_numpy(st["deg"]).to(dev),
                       torch.from_numpy(st["sub_off"]).to(dev), F)


def call_static(inputs, weighted=True):
    import torch
    import paper_2110_02987_b200 as pkg
    X, deg, sub_off, F = inputs
    K = sub_off.numel() - 1
    zeta = torch.full((K,), -1.0, dtype=torch.float32, device=X.device)
    wts = torch.full((K,), -1.0, dtype=torch.float32, device=X.device)
    pkg.subgraph_weights_static(X, deg, sub_off, F, zeta, wts, weighted=weighted)
    torch.cuda.synchronize()
    return zeta.cpu().numpy(), wts.cpu().numpy()


def test_static_entry_point_matches_the_regular_one_on_two_calls_in_a_row():
    first = reference_and_inputs(make_workload("tiny"))
    second = reference_and_inputs(make_workload("c2", scale=0.05))
    for zeta_ref, w_ref, inputs in (first, second, first):
        zeta, wts = call_static(inputs)
        assert np.max(np.abs(zeta - zeta_ref) / zeta_ref) <= 1e-6
        assert np.max(np.abs(wts - w_ref)) <= 1e-6
        assert abs(float(wts.sum()) - 1.0) <= 1e-6
    # the plain average of Definition 3
    _, wts = call_static(first[2], weighted=False)
    assert np.allclose(wts, 1.0 / len(wts))


def test_static_entry_point_rejects_what_does_not_fit_its_fixed_array():
    import torch
    import paper_2110_02987_b200 as pkg
    dev = torch.device("cuda")
    K, ld = 8, 4096                                   # K * ld = 32768 > 16384
    X = torch.zeros((K, ld), dtype=torch.float32, device=dev)
    deg = torch.zeros(K, dtype=torch.int32, device=dev)
    sub_off = torch.arange(K + 1, dtype=torch.int32, device=dev)
    out = torch.zeros(K, dtype=torch.float32, device=dev)
    with pytest.raises(pkg.GadError) as e:
        pkg.subgraph_weights_static(X, deg, sub_off, ld, out, out.clone())
    assert e.value.code == -2
