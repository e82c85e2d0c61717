"""The named synthetic workloads (graph + partition + features + labels + layer sizes)."""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from .graphs import sbm_graph, chung_lu_graph, planted_community_graph
from .partition import contiguous_partition, bfs_partition, one_hop_halo


@dataclass
class Workload:
    name: str
    n: int
    rowptr: np.ndarray          # int64 [n+1]
    col: np.ndarray             # int32 [nnz], ascending inside a row
    X: np.ndarray               # float32 [n, dims[0]]
    labels: np.ndarray          # int32 [n], 0..C-1
    split: np.ndarray           # uint8 [n]: 0 train, 1 validation, 2 test
    core: list                  # K int32 arrays (disjoint)
    halo: list                  # K int32 arrays (disjoint from the matching core)
    dims: tuple                 # (F_0, ..., F_L)
    lr: float = 0.01
    epochs: int = 10
    seed: int = 0
    recipe: str = ""
    extra: dict = field(default_factory=dict)

    @property
    def K(self) -> int:
        return len(self.core)

    @property
    def nnz(self) -> int:
        return int(self.rowptr[-1])

    def flat_partition(self):
        """(core_ptr int64[K+1], core_nodes int32, halo_ptr int64[K+1], halo_nodes int32)."""
        def flat(lists):
            ptr = np.zeros(len(lists) + 1, dtype=np.int64)
            np.cumsum([len(a) for a in lists], out=ptr[1:])
            nodes = (np.concatenate(lists).astype(np.int32) if ptr[-1] > 0
                     else np.empty(0, dtype=np.int32))
            return ptr, np.ascontiguousarray(nodes)
        cp, cn = flat(self.core)
        hp, hn = flat(self.halo)
        return cp, cn, hp, hn


def param_count(dims) -> int:
    return int(sum(dims[l] * dims[l + 1] + dims[l + 1] for l in range(len(dims) - 1)))


def glorot_params(dims, rng: np.random.Generator, bias_scale: float = 0.0) -> np.ndarray:
    """One replica's parameters, float32 [P], laid out [W_0 (F_0 x F_1 row-major), b_0, W_1, b_1, ...].
    W_l is uniform in +-sqrt(6/(F_l+F_{l+1})); b_l is zero unless ``bias_scale`` asks for a
    small uniform value (useful to exercise the bias path in tests)."""
    out = []
    for l in range(len(dims) - 1):
        fi, fo = dims[l], dims[l + 1]
        a = np.sqrt(6.0 / (fi + fo))
        out.append(rng.uniform(-a, a, size=fi * fo))
        out.append(rng.uniform(-bias_scale, bias_scale, size=fo) if bias_scale > 0 else np.zeros(fo))
    return np.concatenate(out).astype(np.float32)


def _split(n: int, rng: np.random.Generator, fr=(0.6, 0.2, 0.2)) -> np.ndarray:
    perm = rng.permutation(n)
    split = np.full(n, 2, dtype=np.uint8)
    a = int(round(fr[0] * n))
    b = a + int(round(fr[1] * n))
    split[perm[:a]] = 0
    split[perm[a:b]] = 1
    return split


def _noisy_labels(base: np.ndarray, n_classes: int, noise: float, rng) -> np.ndarray:
    y = base.astype(np.int32) % n_classes
    flip = rng.random(y.shape[0]) < noise
    y[flip] = rng.integers(0, n_classes, size=int(flip.sum()))
    return y.astype(np.int32)


def _tiny(rng, signal: bool, scale: float):
    bs = max(8, int(round(500 * scale)))
    rowptr, col, block = sbm_graph(4, bs, 0.02, 0.001, rng)
    n = 4 * bs
    X = rng.standard_normal((n, 32)).astype(np.float32)
    y = _noisy_labels(block, 4, 0.10, rng)
    if signal:
        X[np.arange(n), y] += 1.0
    split = _split(n, rng)
    core = contiguous_partition(n, 4)
    halo = one_hop_halo(rowptr, col, core, frac_of_candidates=0.05)
    return Workload(
        name="tiny_signal" if signal else "tiny", n=n, rowptr=rowptr, col=col, X=X, labels=y,
        split=split, core=core, halo=halo, dims=(32, 16, 4), lr=0.5 if signal else 0.01, epochs=10,
        recipe="SBM 4x%d p_in=.02 p_out=.001; N(0,1)^32%s; K=4 contiguous; top-5%% 1-hop halo" %
               (bs, " +1 on coordinate y" if signal else ""))


def _chung_lu(name, n, gamma, mean_deg, n_comm, n_classes, F, K, halo_r, dims, epochs, rng, scale):
    n = max(64 * K, int(round(n * scale)))
    rowptr, col, comm = chung_lu_graph(n, gamma, mean_deg, n_comm, 0.7, rng)
    X = rng.standard_normal((n, F), dtype=np.float32)
    y = (comm % n_classes).astype(np.int32)
    split = _split(n, rng)
    core = bfs_partition(rowptr, col, K)
    halo = one_hop_halo(rowptr, col, core, frac_of_core=halo_r)
    return Workload(
        name=name, n=n, rowptr=rowptr, col=col, X=X, labels=y, split=split, core=core, halo=halo,
        dims=tuple(dims), lr=0.01, epochs=epochs,
        recipe="Chung-Lu gamma=%.1f mean degree %g, %d planted communities (p_intra .7); N(0,1)^%d; "
               "K=%d BFS blocks; halo %g of core" % (gamma, mean_deg, n_comm, F, K, halo_r))


def _c3(K, rng, scale):
    n = max(64 * K, int(round(233_000 * scale)))
    mean_deg = 490.0 if scale >= 1.0 else max(8.0, 490.0 * max(scale, 0.02))
    rowptr, col, comm = planted_community_graph(n, 50, mean_deg, 0.8, rng)
    X = rng.standard_normal((n, 602), dtype=np.float32)
    y = (comm % 41).astype(np.int32)
    split = _split(n, rng)
    # contiguous blocks follow the planted communities, as a minimum-cut partition would; breadth-first
    # blocks do not (two hops reach the whole graph), and cut about 70 % of the edges
    core = contiguous_partition(n, K)
    halo = one_hop_halo(rowptr, col, core, frac_of_core=0.05)
    return Workload(
        name="c3k%d" % K, n=n, rowptr=rowptr, col=col, X=X, labels=y, split=split, core=core, halo=halo,
        dims=(602, 256, 41), lr=0.01, epochs=20,
        recipe="50 planted communities, mean degree %g, 80%% intra; N(0,1)^602; K=%d contiguous blocks; "
               "halo .05 of core" % (mean_deg, K))


def sweep_family(mean_deg: float, Ks, Fs, *, seed: int = 0, scale: float = 1.0):
    """The sweep workloads of one mean degree, for every feature width in ``Fs`` and every K in ``Ks``, with the graph
    drawn once and every partition grown once.  Each yielded workload equals ``make_workload("sweep", mean_deg=...,
    F=..., K=...)`` bit for bit (the generator draws the graph before the features, and the partition draws nothing)."""
    rng = np.random.default_rng(seed)
    n = max(64 * max(Ks), int(round(1_000_000 * scale)))
    rowptr, col, comm = chung_lu_graph(n, 2.1, mean_deg, 16, 0.7, rng)
    state = rng.bit_generator.state
    y = (comm % 16).astype(np.int32)
    parts = {}
    for K in Ks:
        core = bfs_partition(rowptr, col, K)
        parts[K] = (core, one_hop_halo(rowptr, col, core, frac_of_core=0.05))
    for F in Fs:
        rng.bit_generator.state = state
        X = rng.standard_normal((n, F), dtype=np.float32)
        split = _split(n, rng)
        for K in Ks:
            core, halo = parts[K]
            w = Workload(
                name="sweep_d%g_f%d_k%d" % (mean_deg, F, K), n=n, rowptr=rowptr, col=col, X=X, labels=y, split=split, core=core,
                halo=halo, dims=(F, F, F, 16), lr=0.01, epochs=1,
                recipe="Chung-Lu gamma=%.1f mean degree %g, %d planted communities (p_intra .7); N(0,1)^%d; "
                       "K=%d BFS blocks; halo %g of core" % (2.1, mean_deg, 16, F, K, 0.05))
            w.seed = seed
            yield w


WORKLOADS = ("tiny", "tiny_signal", "c2", "c3k4", "c3k8", "c4", "sweep")


def make_workload(name: str, *, seed: int = 0, scale: float = 1.0, **kw) -> Workload:
    """Build one of the named workloads from ``numpy.random.default_rng(seed)``.

    ``scale`` < 1 shrinks the node count (and, for the dense-community graph, the mean
    degree) while keeping the recipe, for parity cases that a CPU oracle finishes quickly.
    ``sweep`` takes ``mean_deg``, ``F`` and ``K`` keywords.
    """
    rng = np.random.default_rng(seed)
    if name == "tiny":
        w = _tiny(rng, False, scale)
    elif name == "tiny_signal":
        w = _tiny(rng, True, scale)
    elif name == "c2":
        w = _chung_lu("c2", 100_000, 2.1, 20, 16, 16, 128, 8, 0.10, (128, 128, 16), 50, rng, scale)
    elif name in ("c3k4", "c3k8"):
        w = _c3(int(name[3:]), rng, scale)
    elif name == "c4":
        w = _chung_lu("c4", 2_450_000, 2.2, 50, 47, 47, 100, 16, 0.05, (100, 256, 256, 47), 10, rng, scale)
    elif name == "sweep":
        F = int(kw.get("F", 128))
        K = int(kw.get("K", 8))
        deg = float(kw.get("mean_deg", 32))
        w = _chung_lu("sweep_d%g_f%d_k%d" % (deg, F, K), 1_000_000, 2.1, deg, 16, 16, F, K, 0.05,
                      (F, F, F, 16), 1, rng, scale)
    else:
        raise ValueError("unknown workload %r" % name)
    w.seed = seed
    return w
