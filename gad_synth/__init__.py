"""Seeded synthetic inputs for the GAD training-epoch path.

This package only *makes inputs*: graphs in CSR form, node partitions with their
replicated (halo) node lists, features, labels, data splits and initial
parameters.  It contains none of the method's arithmetic (no adjacency
normalisation, no GCN layer, no importance weight, no consensus), so that the
CPU oracle and the CUDA library can both be fed from it without sharing any of
the code under test.

The paper trains on Cora, Pubmed, Flicker and Reddit (Table 1).  Those datasets
are not available here; the generators below only borrow their shapes (node and
edge counts, feature widths, class counts) and a power-law / community degree
structure.
"""
from .graphs import (  # noqa: F401
    sbm_graph,
    chung_lu_graph,
    planted_community_graph,
    csr_from_pairs,
)
from .partition import (  # noqa: F401
    contiguous_partition,
    bfs_partition,
    one_hop_halo,
)
from .workloads import (  # noqa: F401
    Workload,
    make_workload,
    sweep_family,
    glorot_params,
    param_count,
    WORKLOADS,
)
