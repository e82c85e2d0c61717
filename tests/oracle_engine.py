"""A CPU engine with the method names the orchestration classes use, backed by the oracle (fp64).  Test helper: it
lets the sums over ranks and the hand-over between rounds be checked without a GPU."""
import numpy as np
import torch

from conftest import flat


class OracleEngine:
    def __init__(self, case, subgraphs, X, y, split, dims, theta, lr, weighted=True):
        from oracle import gad_oracle as orc
        n, rowptr, col, w, core, halo = case
        cp, cn = flat([core[k] for k in subgraphs])
        hp, hn = flat([halo[k] for k in subgraphs])
        self.store = orc.Store(n, rowptr, col, cp, cn, hp, hn, weights=w)
        self.model = orc.Model(self.store, X, y, split, dims, theta, lr=lr, weighted=weighted)
        self.K, self.lr, self.weighted, self.P = len(subgraphs), lr, weighted, self.model.P

    def subgraph_weights(self):
        return self.model.subgraph_weights()

    def ntrain(self):
        return self.model.ntrain()

    def train_epoch(self):
        return self.model.train_epoch()

    def train_epoch_local(self, wait=True):
        losses = self.model.forward_backward()
        nt = self.ntrain().astype(np.float64)
        return np.concatenate([losses, [np.sum(nt * losses) / max(nt.sum(), 1.0)]])

    def new_consensus_buffer(self):
        return torch.zeros(self.P, dtype=torch.float64)

    def consensus_partial(self, zeta_total, out, with_step=True):
        zeta, _ = self.model.subgraph_weights()
        acc = np.zeros(self.P)
        for k in range(self.K):
            wk = (zeta[k] if self.weighted else 1.0) / zeta_total
            acc += wk * (self.model.get_params(k) - (self.lr * self.model.get_grads(k) if with_step else 0.0))
        out.copy_(torch.from_numpy(acc))
        return out

    def consensus_apply(self, buf):
        for k in range(self.K):
            self.model.set_params(k, buf.numpy())

    def export_params(self, k, out):
        out.copy_(torch.from_numpy(self.model.get_params(k)))
        return out
