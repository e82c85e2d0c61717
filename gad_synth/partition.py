"""Stand-ins for GAD-Partition's output: node partitions and replicated-node lists.

The paper produces its partitions with a multi-level (Metis-like) method and
selects the replicated nodes with Monte-Carlo random walks.  Both are *inputs* to
the training epoch; here they are replaced by simple deterministic rules that give
lists of the same kind (disjoint core sets, a bounded list of boundary-adjacent
replicated nodes per subgraph).
"""
from __future__ import annotations

import numpy as np


def contiguous_partition(n: int, K: int) -> list[np.ndarray]:
    """K node ranges [k*ceil(n/K), (k+1)*ceil(n/K))."""
    size = -(-n // K)
    return [np.arange(k * size, min((k + 1) * size, n), dtype=np.int32) for k in range(K)]


def _neighbours_in_order(rowptr: np.ndarray, col: np.ndarray, frontier: np.ndarray) -> np.ndarray:
    """Concatenated neighbour lists of ``frontier`` (frontier order, ascending id inside a list)."""
    start = rowptr[frontier]
    cnt = rowptr[frontier + 1] - start
    total = int(cnt.sum())
    if total == 0:
        return np.empty(0, dtype=np.int64)
    offs = np.repeat(start - np.concatenate([[0], np.cumsum(cnt)[:-1]]), cnt)
    return col[np.arange(total, dtype=np.int64) + offs].astype(np.int64)


def bfs_partition(rowptr: np.ndarray, col: np.ndarray, K: int) -> list[np.ndarray]:
    """BFS-grown blocks of ceil(n/K) nodes.

    A block starts at the lowest unassigned node id and grows in breadth-first
    queue order (neighbours in ascending id); when the queue empties before the
    block is full it restarts from the lowest unassigned id.  A block that
    reaches its size is closed and the next block starts with a fresh queue.
    Node order inside a block is the visit order.
    """
    n = rowptr.shape[0] - 1
    size = -(-n // K)
    assigned = np.zeros(n, dtype=bool)
    parts: list[np.ndarray] = []
    next_free = 0
    for _ in range(K):
        block: list[np.ndarray] = []
        have = 0
        remaining = n - int(assigned.sum())
        want = min(size, remaining)
        frontier = np.empty(0, dtype=np.int64)
        while have < want:
            if frontier.size == 0:
                while next_free < n and assigned[next_free]:
                    next_free += 1
                frontier = np.array([next_free], dtype=np.int64)
                assigned[next_free] = True
                block.append(frontier)
                have += 1
                continue
            nb = _neighbours_in_order(rowptr, col, frontier)
            nb = nb[~assigned[nb]]
            if nb.size:
                _, first = np.unique(nb, return_index=True)
                nb = nb[np.sort(first)]
            if have + nb.size > want:
                nb = nb[: want - have]
            assigned[nb] = True
            if nb.size:
                block.append(nb)
                have += nb.size
            frontier = nb
        parts.append(np.concatenate(block).astype(np.int32) if block else np.empty(0, np.int32))
    return parts


def one_hop_halo(rowptr: np.ndarray, col: np.ndarray, parts: list[np.ndarray], *,
                 frac_of_candidates: float | None = None,
                 frac_of_core: float | None = None) -> list[np.ndarray]:
    """Replicated-node list per subgraph.

    Candidates are the 1-hop neighbours of the core set that lie outside it
    (Definition 2 of the paper with x = 1).  They are ranked by (degree in the
    whole graph, descending; node id, ascending) and the first
    ``ceil(frac_of_candidates*|C_k|)`` or ``min(|C_k|, ceil(frac_of_core*|V_k|))``
    are kept.
    """
    n = rowptr.shape[0] - 1
    deg = np.diff(rowptr)
    halos = []
    inside = np.zeros(n, dtype=bool)
    for core in parts:
        core64 = core.astype(np.int64)
        inside[core64] = True
        nb = _neighbours_in_order(rowptr, col, core64)
        cand = np.unique(nb[~inside[nb]])
        inside[core64] = False
        if frac_of_candidates is not None:
            keep = int(np.ceil(frac_of_candidates * cand.size))
        else:
            keep = min(cand.size, int(np.ceil(frac_of_core * core.size)))
        order = np.lexsort((cand, -deg[cand]))
        halos.append(cand[order[:keep]].astype(np.int32))
    return halos
