"""The sweep generator that draws a graph once per mean degree must hand out the very workloads make_workload builds."""
import numpy as np

from gad_synth import make_workload, sweep_family


def test_sweep_family_equals_the_single_workloads():
    seen = 0
    for w in sweep_family(8, (2, 4), (16, 32), scale=0.01):
        r = make_workload("sweep", scale=0.01, mean_deg=8, F=w.dims[0], K=w.K)
        assert w.name == r.name and w.dims == r.dims == (w.dims[0], w.dims[0], w.dims[0], 16)
        for a, b in ((w.rowptr, r.rowptr), (w.col, r.col), (w.X, r.X), (w.labels, r.labels), (w.split, r.split)):
            assert np.array_equal(a, b)
        for a, b in zip(w.core + w.halo, r.core + r.halo):
            assert np.array_equal(a, b)
        seen += 1
    assert seen == 4
