"""Oracle for importance-based subgraph augmentation (Algorithm 1 of the paper, Section 3.2.2), plain numpy.

TEST INFRASTRUCTURE: only the tests and the CPU-baseline leg of the benchmark may import this module.

For every subgraph g_i = (v_i, e_i) of a partition of G (steps in the order of Algorithm 1):

  boundary B(g_i)    the nodes of v_i with a neighbour outside v_i, in ascending node id
  first walks        d |B| walks with d the average degree of the boundary nodes, i.e. n0 = sum of their degrees;
                     a walk starts at a boundary node drawn uniformly and takes l steps (l = number of GCN layers,
                     Property 1), each to a uniformly drawn neighbour in G
  visit counts       count[v] = number of walks that contain v, for v outside v_i  (I(v) = count[v] / n, importance equation)
  number of walks    n = (z_c sigma / (mean E))^2 from the mean and standard deviation of I over the visited
                     candidates (Monte-Carlo error equation); the walks n0 .. n-1 are added when n > n0
  replication count  n(g_i) = alpha (1 + d(g_i)) |v_i| with the density d(g_i) = 2 |e_i| / (|v_i| (|v_i| - 1))
  selection          walks in descending order of I(RW) = sum of I(v) over the walk's nodes outside v_i; the nodes of a
                     walk that lie outside v_i and are not selected yet are added in walk order until n(g_i) are selected
                     ("depth-first": a selected node is reached from v_i through selected nodes of the same walk)

Readings where the paper is silent: the random draws come from a counter-based generator,
draw(i, j, s) = mix(mix(mix(seed + G (1 + i)) + G (1 + j)) + G (1 + s)) with the splitmix64 output function `mix` and
its increment G, reduced modulo the number of choices; a node counts once per walk; sigma is the population standard
deviation; sigma / mean is evaluated from the integer sums of the counts, n = ceil((z_c / E)^2 (m S2 / S1^2 - 1));
the number of walks is capped at `cap` times n0; walks of equal score keep their index order; n(g_i) is rounded down
and cannot exceed the number of visited candidates; self-loops stored in G count as neighbours.
"""
from __future__ import annotations

import math

import numpy as np

G64 = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def mix64(z):
    """Output function of splitmix64 on uint64 arrays (wrap-around arithmetic)."""
    z = np.asarray(z, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


def draw(seed: int, i: int, j, s: int):
    """The random 64-bit number of subgraph i, walk(s) j, step s (step 0 chooses the start)."""
    j = np.asarray(j, dtype=np.uint64)
    with np.errstate(over="ignore"):
        h = mix64(np.uint64(seed) + G64 * np.uint64(1 + i))
        h = mix64(h + G64 * (np.uint64(1) + j))
        return mix64(h + G64 * np.uint64(1 + s))


def boundary(rowptr, col, core, n):
    inside = np.zeros(n, dtype=bool)
    inside[core] = True
    out = []
    for v in np.sort(core):
        nb = col[rowptr[v]:rowptr[v + 1]]
        if np.any(~inside[nb]):
            out.append(int(v))
    return np.asarray(out, dtype=np.int64), inside


def walks(rowptr, col, B, seed, i, j0, j1, steps):
    """Node sequences of the walks j0 .. j1-1 of subgraph i: int64 [j1 - j0, steps + 1]."""
    j = np.arange(j0, j1, dtype=np.uint64)
    seq = np.empty((j.shape[0], steps + 1), dtype=np.int64)
    cur = B[(draw(seed, i, j, 0) % np.uint64(B.shape[0])).astype(np.int64)]
    seq[:, 0] = cur
    deg = np.diff(rowptr)
    for s in range(1, steps + 1):
        d = deg[cur]
        r = draw(seed, i, j, s)
        pick = (r % np.maximum(d, 1).astype(np.uint64)).astype(np.int64)
        nxt = col[np.minimum(rowptr[cur] + pick, col.shape[0] - 1)]
        cur = np.where(d > 0, nxt, cur)
        seq[:, s] = cur
    return seq


def _count(seq, inside, count):
    """count[v] += 1 for every walk and every distinct node v of it outside the subgraph."""
    for w in seq:
        seen = set()
        for v in w:
            v = int(v)
            if not inside[v] and v not in seen:
                seen.add(v)
                count[v] += 1


def walk_scores(seq, inside, count):
    out = np.zeros(seq.shape[0], dtype=np.int64)
    for a, w in enumerate(seq):
        seen = set()
        for v in w:
            v = int(v)
            if not inside[v] and v not in seen:
                seen.add(v)
                out[a] += int(count[v])
    return out


def number_of_walks(count, n0, zc, E, cap):
    c = count[count > 0].astype(np.int64)
    m, S1, S2 = int(c.shape[0]), int(c.sum()), int((c * c).sum())
    if m == 0:
        return n0
    ratio = (float(m) * float(S2)) / (float(S1) * float(S1)) - 1.0
    n = int(math.ceil((zc / E) * (zc / E) * ratio)) if ratio > 0.0 else 0
    return max(n0, min(n, cap * n0))


def replication_count(rowptr, col, core, inside, alpha):
    nv = int(core.shape[0])
    if nv < 2:
        return 0
    directed = 0
    for v in core:
        nb = col[rowptr[v]:rowptr[v + 1]]
        directed += int(np.sum(inside[nb] & (nb != v)))
    dens = float(directed) / (float(nv) * float(nv - 1))      # 2 |e_i| = directed entries inside, self-loops left out
    return int(math.floor(alpha * (1.0 + dens) * float(nv)))


def augment(n, rowptr, col, cores, steps, *, alpha=0.01, E=0.05, zc=1.96, seed=0, cap=4):
    """Replication-node list of every subgraph, plus what the steps produced on the way (for the tests)."""
    rowptr = np.asarray(rowptr, dtype=np.int64)
    col = np.asarray(col, dtype=np.int64)
    halos, info = [], []
    for i, core in enumerate(cores):
        core = np.asarray(core, dtype=np.int64)
        B, inside = boundary(rowptr, col, core, n)
        count = np.zeros(n, dtype=np.int64)
        if B.shape[0] == 0:
            halos.append(np.empty(0, dtype=np.int32))
            info.append({"boundary": B, "n0": 0, "n": 0, "count": count, "n_rep": 0, "scores": np.empty(0, np.int64)})
            continue
        n0 = int(np.sum(np.diff(rowptr)[B]))
        seq = walks(rowptr, col, B, seed, i, 0, n0, steps)
        _count(seq, inside, count)
        nw = number_of_walks(count, n0, zc, E, cap)
        if nw > n0:
            more = walks(rowptr, col, B, seed, i, n0, nw, steps)
            _count(more, inside, count)
            seq = np.concatenate([seq, more])
        scores = walk_scores(seq, inside, count)
        n_rep = min(replication_count(rowptr, col, core, inside, alpha), int(np.sum(count > 0)))
        order = np.lexsort((np.arange(nw), -scores))
        chosen, have = [], set()
        for a in order:
            if len(chosen) >= n_rep:
                break
            for v in seq[a]:
                v = int(v)
                if not inside[v] and v not in have and len(chosen) < n_rep:
                    have.add(v)
                    chosen.append(v)
        halos.append(np.asarray(chosen, dtype=np.int32))
        info.append({"boundary": B, "n0": n0, "n": nw, "count": count, "n_rep": n_rep, "scores": scores, "walks": seq})
    return halos, info
