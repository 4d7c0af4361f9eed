"""Helpers of the GPU parity tests: move a seeded workload to the device and compare with the oracle."""
import numpy as np

from oracle import feplb_oracle as O
from paper_2604_19654_b200 import feplb as F
from paper_2604_19654_b200 import workloads as W

# |gpu - ref| <= ATOL_REL * max|ref| + RTOL * |ref| for bf16 inputs with fp32 accumulation
ATOL_REL = 1e-2
RTOL = 1e-2


def assert_close(gpu_f64: np.ndarray, ref: np.ndarray, what=""):
    bound = ATOL_REL * np.abs(ref).max() + RTOL * np.abs(ref)
    err = np.abs(gpu_f64 - ref)
    bad = err > bound
    assert not bad.any(), (f"{what}: {int(bad.sum())} of {bad.size} elements out of tolerance; "
                           f"max err {err.max():.3e}, max|ref| {np.abs(ref).max():.3e}, "
                           f"first bad index {np.argwhere(bad)[0].tolist()}")
    return float((err / (bound + 1e-300)).max())


class DeviceCase:
    """Inputs of one micro-batch on the device plus a context and buffers."""

    def __init__(self, w, mb=0, weights=None, **cfg_kw):
        import torch
        self.w = w
        self.cfg = F.config_from_workload(w, **cfg_kw)
        self.x, self.ids, self.gates = W.gen_microbatch(w, mb)
        self.w1, self.w3, self.w2 = weights if weights is not None else W.gen_weights(w)
        self.ctx = F.Context(self.cfg)
        self.buf = F.Buffers(self.cfg)
        self.d_x = F.bf16_tensor(self.x)
        self.d_ids = torch.from_numpy(self.ids).cuda()
        self.d_gates = torch.from_numpy(self.gates).cuda()
        self.d_w1, self.d_w3, self.d_w2 = (F.bf16_tensor(a) for a in (self.w1, self.w3, self.w2))

    def close(self):
        self.ctx.close()


def oracle_mask(counts, w):
    return O.select_dynamic(counts, w.E, w.R, w.dyn)


def upload_groups(groups):
    import torch
    a = F.groups_to_numpy(groups)
    if a.shape[0] == 0:
        a = np.zeros((1, 5), np.int32)
    return torch.from_numpy(a).cuda()
