"""Algorithm 2 with the subgraphs spread over several contexts: several GPUs (one context each, one all-reduce per
step), or several rounds of an epoch (z subgraphs per processor, one context per round).

Only orchestration lives here: which context runs when, and the sums over contexts.  Every step of the method runs
in the library (``gad_train_epoch_local``, ``gad_consensus_partial``, ``gad_consensus_apply``, ``gad_export_params``).
An *engine* is anything with the methods of :class:`paper_2110_02987_b200.Gad` used below; the tests drive the same
classes with a CPU engine to check the sums over ranks.
"""
from __future__ import annotations

import numpy as np


def shard_subgraphs(K: int, world: int, rank: int) -> list[int]:
    """Subgraphs k = rank, rank + world, ... (the round-robin assignment of K subgraphs to `world` processors)."""
    return list(range(rank, K, world))


class ShardedEpoch:
    """One training step of K subgraphs spread over the ranks of a ``torch.distributed`` group, one engine per rank.

    Per step every rank runs its local epoch and its share of the weighted consensus; ONE all-reduce (sum) of the
    consensus buffer gives every rank the same model, which it writes to its replicas.  The importance weights depend
    only on the graph and the features, so their total over all ranks is reduced once, at set-up (call
    :meth:`refresh_weights` after new features).
    """

    def __init__(self, engine, group=None, weighted=True):
        import torch.distributed as dist
        self.engine = engine
        self.group = group
        self.dist = dist
        self.weighted = weighted
        self.buf = engine.new_consensus_buffer()
        self.refresh_weights()

    def _sum(self, values):
        import torch
        t = torch.tensor(values, dtype=torch.float64)
        if self.dist.is_initialized() and self.dist.get_world_size(self.group) > 1:
            dev = self.buf.device if self.dist.get_backend(self.group) == "nccl" else "cpu"
            t = t.to(dev)
            self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM, group=self.group)
        return t.cpu().numpy()

    def refresh_weights(self):
        zeta, _ = self.engine.subgraph_weights()
        local = float(np.sum(np.asarray(zeta, dtype=np.float64))) if self.weighted else float(self.engine.K)
        self.zeta_total = float(self._sum([local])[0])
        if not self.zeta_total > 0.0:   # every zeta is zero: the plain average
            self.weighted_total = None
            raise ValueError("all importance weights are zero; use weighted=False")

    def step(self, want_loss=True):
        """One epoch over all ranks' subgraphs.  Returns the global mean training loss (or None)."""
        losses = self.engine.train_epoch_local(wait=want_loss)
        self.engine.consensus_partial(self.zeta_total, self.buf, with_step=True)
        if self.dist.is_initialized() and self.dist.get_world_size(self.group) > 1:
            self.dist.all_reduce(self.buf, op=self.dist.ReduceOp.SUM, group=self.group)
        self.engine.consensus_apply(self.buf)
        if not want_loss:
            return None
        nt = np.asarray(self.engine.ntrain(), dtype=np.float64)
        num, den = self._sum([float(np.sum(nt * np.asarray(losses[:-1], dtype=np.float64))), float(np.sum(nt))])
        return num / den if den > 0 else 0.0


class RoundsEpoch:
    """z rounds per epoch: the engines (one per round, same layer sizes, same device) train one after the other,
    each starting from the model the round before it left (last paragraph of Section 3.3)."""

    def __init__(self, engines):
        self.engines = list(engines)
        self.buf = self.engines[0].new_consensus_buffer()

    def step(self):
        """One epoch = every round once.  Returns the list of the rounds' loss arrays."""
        out = []
        z = len(self.engines)
        for r, eng in enumerate(self.engines):
            out.append(eng.train_epoch())
            nxt = self.engines[(r + 1) % z]
            if nxt is not eng:
                eng.export_params(0, self.buf)   # after the consensus every replica holds the same model
                nxt.consensus_apply(self.buf)
        return out
