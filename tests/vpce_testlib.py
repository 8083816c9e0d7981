"""Helpers shared by the GPU parity tests: move seeded inputs to the device, call the C-ABI
through the Python binding, and measure errors against the float64 oracle."""
import numpy as np
import torch

import paper_2609_14306_b200 as vp
from synth_inputs import IGNORE_INDEX, bf16_bits_to_f64

TOL_TOKEN = 2e-3      # |err| of per-token lse and loss
TOL_MEAN_REL = 1e-4   # relative error of the mean loss
TOL_GRAD = 1e-2       # relative Frobenius error of dH, dW


def to_dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def relF(a: np.ndarray, ref: np.ndarray) -> float:
    den = float(np.linalg.norm(ref))
    num = float(np.linalg.norm(np.asarray(a, dtype=np.float64) - ref))
    return num / den if den > 0 else num


class DeviceRun:
    """Device buffers and results of one forward(+backward) call."""

    def __init__(self, H_bits, W_bits, labels, block_v, T_chunk, chunk_index_base=0, ignore_index=IGNORE_INDEX,
                 W_dev=None, dW=None):
        self.T, self.d = H_bits.shape
        self.V = W_bits.shape[0] if W_dev is None else W_dev.shape[0]
        self.block_v, self.T_chunk, self.base, self.ignore_index = block_v, T_chunk, chunk_index_base, ignore_index
        self.H = to_dev_bf16(H_bits)
        self.W = to_dev_bf16(W_bits) if W_dev is None else W_dev
        self.labels = torch.from_numpy(np.ascontiguousarray(labels, dtype=np.int32)).cuda()
        self.ws_bytes = vp.vp_ce_workspace_bytes(T_chunk, self.d, block_v)
        assert self.ws_bytes > 0, "shape rejected by vp_ce_workspace_bytes"
        self.ws = torch.empty(self.ws_bytes, dtype=torch.uint8, device="cuda")
        self.loss = torch.full((self.T,), float("nan"), dtype=torch.float32, device="cuda")
        self.lse = torch.full((self.T,), float("nan"), dtype=torch.float32, device="cuda")
        self.dH = None
        self.dW = dW

    def forward(self):
        vp.vp_ce_forward(self.H, self.W, self.labels, self.block_v, self.ignore_index, self.loss, self.lse,
                         self.T_chunk, self.base, self.ws)
        torch.cuda.synchronize()
        self.fwd_status = vp.vp_ce_device_status(self.ws)
        return self

    def backward(self, dloss=None, accumulate=False):
        if self.dH is None:
            self.dH = torch.full((self.T, self.d), float("nan"), dtype=torch.bfloat16, device="cuda")
        if self.dW is None:
            self.dW = torch.full((self.V, self.d), float("nan"), dtype=torch.float32, device="cuda")
        dl = None if dloss is None else torch.from_numpy(np.ascontiguousarray(dloss, dtype=np.float32)).cuda()
        vp.vp_ce_backward(self.H, self.W, self.labels, self.lse, dl, self.dH, self.dW, self.block_v,
                          self.ignore_index, self.T_chunk, self.base, accumulate, self.ws)
        torch.cuda.synchronize()
        self.bwd_status = vp.vp_ce_device_status(self.ws)
        return self

    def mean(self):
        m = torch.zeros(1, dtype=torch.float32, device="cuda")
        n = torch.zeros(1, dtype=torch.int32, device="cuda")
        vp.vp_ce_mean_loss(self.loss, self.labels, self.V, self.ignore_index, m, n)
        torch.cuda.synchronize()
        return float(m.item()), int(n.item())

    # host copies
    def np_lse(self): return self.lse.cpu().numpy().astype(np.float64)
    def np_loss(self): return self.loss.cpu().numpy().astype(np.float64)
    def np_dH(self): return self.dH.float().cpu().numpy().astype(np.float64)
    def np_dW(self): return self.dW.cpu().numpy().astype(np.float64)


def softmax_only_residuals(dH, dW, H64, W64, labels, dloss64, ignore_index=IGNORE_INDEX):
    """Adds the exactly-known one-hot terms back, leaving only the softmax part of each gradient
    (the one-hot part dominates the norm by ~sqrt(V) and would hide a wrong softmax term)."""
    lab = np.asarray(labels).astype(np.int64)
    valid = lab != ignore_index
    dl = np.where(valid, dloss64, 0.0)
    dH_s = dH.copy()
    dW_s = dW.copy()
    rows = np.nonzero(valid)[0]
    dH_s[rows] += dl[rows, None] * W64[lab[rows]]
    np.add.at(dW_s, lab[rows], dl[rows, None] * H64[rows])
    return dH_s, dW_s


def check_against_oracle(run: DeviceRun, ref: dict, H64, W64, labels, dloss64, tag=""):
    """Asserts the acceptance tolerances and returns the measured errors."""
    e = {}
    e["lse"] = float(np.abs(run.np_lse() - ref["lse"]).max())
    e["loss"] = float(np.abs(run.np_loss() - ref["loss"]).max())
    mean, n_valid = run.mean()
    e["mean_rel"] = abs(mean - ref["mean"]) / max(abs(ref["mean"]), 1e-30) if ref["n_valid"] else abs(mean)
    assert n_valid == ref["n_valid"], tag
    dH, dW = run.np_dH(), run.np_dW()
    e["dH"], e["dW"] = relF(dH, ref["dH"]), relF(dW, ref["dW"])
    sH, sW = softmax_only_residuals(dH, dW, H64, W64, labels, dloss64)
    rH, rW = softmax_only_residuals(ref["dH"], ref["dW"], H64, W64, labels, dloss64)
    e["dH_softmax_only"], e["dW_softmax_only"] = relF(sH, rH), relF(sW, rW)
    e["dW_colsum_rel"] = float(np.linalg.norm(dW.sum(0)) / max(np.linalg.norm(dW), 1e-300))
    assert np.isfinite(dH).all() and np.isfinite(dW).all(), tag
    assert e["lse"] <= TOL_TOKEN and e["loss"] <= TOL_TOKEN, (tag, e)
    assert e["mean_rel"] <= TOL_MEAN_REL, (tag, e)
    assert e["dH"] <= TOL_GRAD and e["dW"] <= TOL_GRAD, (tag, e)
    # Stricter than the acceptance gate, and free of the one-hot term's rounding: the rows of dW whose vocabulary
    # id is no token's target consist of the softmax part alone (sum_n dloss_n p[n, v] H_n), so a wrong softmax term
    # reads ~1 here whatever V is, while a right one differs from the oracle by the bf16 rounding of G only.
    never = untargeted_ids(labels, dW.shape[0])
    if len(never):
        e["dW_untargeted_rows"] = relF(dW[never], ref["dW"][never])
        assert e["dW_untargeted_rows"] <= TOL_GRAD, (tag, e)
    # The softmax-only parts of the FULL gradients (one-hot part added back exactly on the host).  The one-hot entries of
    # the staged residual are rounded to bf16 like the rest, but the library adds the rounding residue of every token's
    # one-hot entry back in fp32 (exact one-hot terms), so these too must match the oracle to the gradient tolerance.
    assert e["dW_softmax_only"] <= TOL_GRAD, (tag, e)
    # dH is a bf16 OUTPUT: its own rounding (up to 2^-9 of each element, one-hot part included) is the floor here
    floor = 2.0 ** -9 * np.linalg.norm(ref["dH"]) / max(np.linalg.norm(rH), 1e-300)
    e["dH_softmax_only_bound"] = TOL_GRAD + floor
    assert e["dH_softmax_only"] <= TOL_GRAD + floor, (tag, e)
    return e


def untargeted_ids(labels, V, ignore_index=IGNORE_INDEX):
    """Vocabulary ids that are the target of no valid token."""
    lab = np.asarray(labels).astype(np.int64)
    lab = lab[(lab != ignore_index) & (lab >= 0) & (lab < V)]
    return np.setdiff1d(np.arange(V), lab)
