"""Seeded random graphs, returned as CSR (rowptr int64, col int32, sorted columns)."""
from __future__ import annotations

import numpy as np


def csr_from_pairs(n: int, u: np.ndarray, v: np.ndarray, *, symmetrise: bool = True,
                   self_loops: bool = True) -> tuple[np.ndarray, np.ndarray]:
    """Build an unweighted CSR graph from endpoint pairs.

    Self-pairs are dropped, duplicates are merged, the pair set is made
    symmetric when ``symmetrise`` and one self-loop per node is added when
    ``self_loops``.  Columns are ascending within each row.
    """
    u = np.asarray(u, dtype=np.int64)
    v = np.asarray(v, dtype=np.int64)
    keep = u != v
    u, v = u[keep], v[keep]
    if symmetrise:
        lo = np.minimum(u, v)
        hi = np.maximum(u, v)
        key = np.unique(lo * n + hi)
        lo, hi = key // n, key % n
        del key
        src = np.concatenate([lo, hi])
        dst = np.concatenate([hi, lo])
        del lo, hi
    else:
        key = np.unique(u * n + v)
        src, dst = key // n, key % n
        del key
    if self_loops:
        loop = np.arange(n, dtype=np.int64)
        src = np.concatenate([src, loop])
        dst = np.concatenate([dst, loop])
    key = src * n + dst
    del src, dst
    key.sort()
    src = key // n
    col = (key % n).astype(np.int32)
    del key
    counts = np.bincount(src, minlength=n)
    rowptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(counts, out=rowptr[1:])
    return rowptr, col


def sbm_graph(n_blocks: int, block_size: int, p_in: float, p_out: float,
              rng: np.random.Generator) -> tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Stochastic block model: one Bernoulli draw per unordered node pair.

    Returns (rowptr, col, block_id).  Undirected, with self-loops.
    """
    n = n_blocks * block_size
    block = np.repeat(np.arange(n_blocks, dtype=np.int32), block_size)
    iu, ju = np.triu_indices(n, k=1)
    prob = np.where(block[iu] == block[ju], p_in, p_out)
    hit = rng.random(iu.shape[0]) < prob
    rowptr, col = csr_from_pairs(n, iu[hit], ju[hit])
    return rowptr, col, block


def _capped_weights(n: int, gamma: float, mean_deg: float, i0: float = 10.0) -> np.ndarray:
    """Expected degrees w_i proportional to (i+i0)^(-1/(gamma-1)), mean ``mean_deg``,
    each capped at sqrt(sum w) so that pair probabilities stay below one."""
    w = (np.arange(n, dtype=np.float64) + i0) ** (-1.0 / (gamma - 1.0))
    w *= mean_deg * n / w.sum()
    for _ in range(8):
        cap = np.sqrt(w.sum())
        over = w > cap
        if not over.any():
            break
        w[over] = cap
        free = ~over
        target = mean_deg * n - cap * over.sum()
        if target > 0 and free.any():
            w[free] *= target / w[free].sum()
    return np.minimum(w, np.sqrt(w.sum()))


def chung_lu_graph(n: int, gamma: float, mean_deg: float, n_comm: int, p_intra: float,
                   rng: np.random.Generator) -> tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Power-law (Chung-Lu) graph with a planted community signal.

    ``n*mean_deg/2`` endpoint pairs are drawn with probability proportional to
    the expected degrees.  Every node gets a community uniformly at random; with
    probability ``p_intra`` the second endpoint of a pair is drawn (again
    proportionally to expected degree) inside the first endpoint's community.
    Returns (rowptr, col, community).  Undirected, with self-loops.
    """
    w = _capped_weights(n, gamma, mean_deg)
    comm = rng.integers(0, n_comm, size=n).astype(np.int32)
    m = int(n * mean_deg / 2)
    cdf = np.cumsum(w)
    first = np.searchsorted(cdf, rng.random(m) * cdf[-1], side="right").astype(np.int64)
    np.minimum(first, n - 1, out=first)
    # nodes grouped by community, with a cumulative weight inside that ordering
    order = np.argsort(comm, kind="stable")
    cdf_c = np.cumsum(w[order])
    c_end = np.cumsum(np.bincount(comm, minlength=n_comm))
    c_start = c_end - np.bincount(comm, minlength=n_comm)
    base = np.where(c_start > 0, cdf_c[np.maximum(c_start - 1, 0)], 0.0)
    top = cdf_c[c_end - 1]
    intra = rng.random(m) < p_intra
    r = rng.random(m)
    second = np.empty(m, dtype=np.int64)
    # inside the first endpoint's community
    cf = comm[first[intra]]
    pos = np.searchsorted(cdf_c, base[cf] + r[intra] * (top[cf] - base[cf]), side="right")
    pos = np.clip(pos, c_start[cf], c_end[cf] - 1)
    second[intra] = order[pos]
    # anywhere
    pos = np.searchsorted(cdf, r[~intra] * cdf[-1], side="right")
    second[~intra] = np.minimum(pos, n - 1)
    rowptr, col = csr_from_pairs(n, first, second)
    return rowptr, col, comm


def planted_community_graph(n: int, n_comm: int, mean_deg: float, frac_in: float,
                            rng: np.random.Generator) -> tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Dense-community graph: ``n_comm`` equal contiguous communities; a fraction
    ``frac_in`` of the ``n*mean_deg/2`` uniform node pairs falls inside one
    community, the rest anywhere.  Returns (rowptr, col, community)."""
    size = -(-n // n_comm)
    comm = (np.arange(n, dtype=np.int64) // size).astype(np.int32)
    m = int(n * mean_deg / 2)
    m_in = int(m * frac_in)
    c = rng.integers(0, n_comm, size=m_in)
    lo = c * size
    span = np.minimum(lo + size, n) - lo
    u_in = lo + (rng.random(m_in) * span).astype(np.int64)
    v_in = lo + (rng.random(m_in) * span).astype(np.int64)
    u_out = rng.integers(0, n, size=m - m_in)
    v_out = rng.integers(0, n, size=m - m_in)
    rowptr, col = csr_from_pairs(n, np.concatenate([u_in, u_out]), np.concatenate([v_in, v_out]))
    return rowptr, col, comm
