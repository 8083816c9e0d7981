"""Test-only stand-in for the CUDA meetings of the ring driver: the same three methods, computed on the CPU in
float64 from the oracle's Fold and the textbook residual.  It lets the multi-rank schedule (who meets whom, what
travels, what comes home) be checked with gloo ranks where no GPU is available."""
import numpy as np
import torch

from oracle import vpce_oracle as orc

PHASE_RESIDUAL, PHASE_INPUT_GRAD, PHASE_WEIGHT_GRAD = 1, 2, 4


class OracleMeetings:
    def __init__(self):
        self.calls = []

    def workspace(self, N, d, S, device):
        return {}                                            # holds the residual strip between the phases of a meeting

    def forward_meeting(self, X, W, t, v_lo, V, ignore_index, state, first, last, loss, lse, ws):
        Xn, Wn, tn = X.double().numpy(), W.double().numpy(), t.numpy().astype(np.int64)
        valid = tn != ignore_index
        N = Xn.shape[0]
        if first:
            S = (np.full(N, -np.inf), np.zeros(N), np.zeros(N))
        else:
            S = tuple(state[k].double().numpy().copy() for k in range(3))
        S, _ = orc.fold(S, Xn @ Wn.T, np.where(valid, tn, -1), v_lo, v_lo + Wn.shape[0])
        for k in range(3):
            state[k].copy_(torch.from_numpy(S[k]).to(state.dtype))
        if last:
            m, z, y = S
            l = m + np.log(z)
            lse.copy_(torch.from_numpy(l).to(lse.dtype))
            loss.copy_(torch.from_numpy(np.where(valid, l - y, 0.0)).to(loss.dtype))
        self.calls.append(("fwd", v_lo, Wn.shape[0], bool(first), bool(last)))

    def backward_meeting(self, X, W, t, lse, dloss, v_lo, V, ignore_index, phases, dX_acc, first, last, dX, dW,
                         accumulate_dW, ws):
        Xn, Wn, tn = X.double().numpy(), W.double().numpy(), t.numpy().astype(np.int64)
        if phases & PHASE_RESIDUAL:
            valid = tn != ignore_index
            G = np.exp(Xn @ Wn.T - lse.double().numpy()[:, None])
            own = valid & (tn >= v_lo) & (tn < v_lo + Wn.shape[0])
            rows = np.nonzero(own)[0]
            G[rows, tn[rows] - v_lo] -= 1.0
            G *= np.where(valid, dloss.double().numpy(), 0.0)[:, None]
            ws["G"] = G
        if phases & PHASE_INPUT_GRAD:
            part = ws["G"] @ Wn
            total = part if first else dX_acc.double().numpy() + part
            if last:
                dX.copy_(torch.from_numpy(total).to(dX.dtype))
            else:
                dX_acc.copy_(torch.from_numpy(total).to(dX_acc.dtype))
        if phases & PHASE_WEIGHT_GRAD:
            part = ws["G"].T @ Xn
            if accumulate_dW:
                dW.add_(torch.from_numpy(part).to(dW.dtype))
            else:
                dW.copy_(torch.from_numpy(part).to(dW.dtype))
        self.calls.append(("bwd", v_lo, Wn.shape[0], phases, bool(first), bool(last)))


    def count_valid(self, t, V, ignore_index):
        tn = t.numpy()
        return int(((tn != ignore_index) & (tn >= 0) & (tn < V)).sum())

    def mean_dloss(self, t, V, ignore_index, n_valid_total):
        tn = t.numpy()
        valid = (tn != ignore_index) & (tn >= 0) & (tn < V)
        out = np.where(valid, 1.0 / n_valid_total if n_valid_total else 0.0, 0.0)
        return torch.from_numpy(out.astype(np.float32))


def global_problem(P, N, d, V, seed, ignore_frac=0.1, ignore_index=-100):
    """One seeded problem for a whole group: per-rank batches X_r [N, d], targets, and the full weight."""
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((P * N, d))
    W = rng.standard_normal((V, d)) / np.sqrt(d)
    t = rng.integers(0, V, size=P * N).astype(np.int32)
    t[rng.random(P * N) < ignore_frac] = ignore_index
    t[0] = 0
    t[-1] = V - 1                                          # first and last vocabulary id are targets
    return X, W, t
