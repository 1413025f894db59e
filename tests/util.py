"""Shared helpers of the GPU tests: move a Workload to the device, run it through the
C ABI (paper_2608_05033_b200 binding), bring C back."""
import numpy as np
import torch

import paper_2608_05033_b200 as sd
import workloads as W


def dev(a: np.ndarray):
    """numpy -> cuda tensor (uint16 bf16 bit patterns travel as int16)."""
    if a.dtype == np.uint16:
        a = a.view(np.int16)
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


class DeviceWorkload:
    def __init__(self, w: W.Workload):
        self.w = w
        self.rowptr = dev(w.rowptr)
        self.colind = dev(w.colind) if w.colind.size else torch.zeros(1, dtype=torch.int32, device="cuda")
        self.vals = dev(w.vals) if w.vals.size else torch.zeros(1, dtype=torch.float32, device="cuda")

    def plan(self, family=sd.SD_AUTO, windows=0, validate=False, N=None, heavy_len=0):
        w = self.w
        return sd.Plan(self.rowptr, self.colind, self.vals, w.M, w.K, w.N if N is None else N,
                       dtype=w.dtype, family=family, windows=windows, validate=validate, heavy_len=heavy_len)


def run_spmm(plan, w: W.Workload, pad_b=0, pad_c=0, offset=0, c_fill=None, alpha=None, beta=None):
    """Runs sd_spmm on device copies of w.B / w.C0.  pad_*: extra leading-dimension columns
    filled with sentinels; offset: element offset of the base pointers (breaks 16-byte
    alignment when not a multiple of 4).  Returns (C [M,N] float32, padding_intact)."""
    alpha = w.alpha if alpha is None else alpha
    beta = w.beta if beta is None else beta
    M, K, N = w.M, w.K, w.N
    bdt = np.float32 if w.dtype == W.SD_F32 else np.uint16
    Bh = np.full(K * (N + pad_b) + offset + 8, 0x7F7F if bdt == np.uint16 else 1e30, dtype=bdt)
    Bview = Bh[offset:offset + K * (N + pad_b)].reshape(K, N + pad_b)
    Bview[:, :N] = w.B
    Ch = np.full(M * (N + pad_c) + offset + 8, -7.25, dtype=np.float32)
    Cview = Ch[offset:offset + M * (N + pad_c)].reshape(M, N + pad_c)
    if c_fill is not None:
        Cview[:, :N] = c_fill
    elif w.C0 is not None:
        Cview[:, :N] = w.C0
    Bd, Cd = dev(Bh), dev(Ch)
    sd.sd_spmm(plan.handle, Bd.data_ptr() + offset * Bd.element_size(), N + pad_b,
               Cd.data_ptr() + offset * 4, N + pad_c, alpha, beta)
    torch.cuda.synchronize()
    out = Cd.cpu().numpy()
    got = out[offset:offset + M * (N + pad_c)].reshape(M, N + pad_c)
    intact = bool(np.all(got[:, N:] == np.float32(-7.25)) and np.all(out[:offset] == np.float32(-7.25))
                  and np.all(out[offset + M * (N + pad_c):] == np.float32(-7.25)))
    return np.ascontiguousarray(got[:, :N]), intact
