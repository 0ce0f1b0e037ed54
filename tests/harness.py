"""Test-side plumbing: lay numpy variables out in the library's arenas, run the CUDA library
through its C-ABI binding on torch-allocated device memory, and pull results back per variable.
No arithmetic of the method lives here."""
from __future__ import annotations

import numpy as np
import torch

import paper_2205_03494_b200 as omc


def to_full(plan, arrays) -> np.ndarray:
    """Variables -> one FP32 array in the plan's full layout (padding zero)."""
    out = np.zeros(plan.full_elems, np.float32)
    for i, a in enumerate(arrays):
        out[plan.full_off[i]:plan.full_off[i] + plan.numel[i]] = np.asarray(a, np.float32).ravel()
    return out


def from_full(plan, full: np.ndarray, i: int) -> np.ndarray:
    return full[plan.full_off[i]:plan.full_off[i] + plan.numel[i]]


class DeviceModel:
    """Device buffers of one compressed model plus helpers to move variables in and out."""

    def __init__(self, plan: omc.Plan, device="cuda:0"):
        self.plan = plan
        self.dev = torch.device(device)
        z = lambda n, dt: torch.zeros(max(int(n), 16), dtype=dt, device=self.dev)
        self.packed = z(plan.packed_bytes, torch.uint8)
        self.resid = z(plan.resid_elems, torch.float32)
        self.sb = z(2 * plan.n_quantised, torch.float32)
        self.ws = z(plan.workspace_bytes, torch.uint8)
        plan.prepare(self.ws.data_ptr(), torch.cuda.current_stream().cuda_stream)

    def _s(self):
        return torch.cuda.current_stream().cuda_stream

    def upload_full(self, arrays) -> torch.Tensor:
        return torch.from_numpy(to_full(self.plan, arrays)).to(self.dev)

    def compress(self, params_full: torch.Tensor):
        self.plan.compress(params_full.data_ptr(), self.packed.data_ptr(), self.resid.data_ptr(),
                           self.sb.data_ptr(), self.ws.data_ptr(), self._s())

    def decompress(self, first_var=0, n_vars=None, out=None) -> torch.Tensor:
        if out is None:
            out = torch.zeros(self.plan.full_elems, dtype=torch.float32, device=self.dev)
        self.plan.decompress(self.packed.data_ptr(), self.resid.data_ptr(), self.sb.data_ptr(),
                             out.data_ptr(), first_var, n_vars, self._s())
        return out

    def update(self, grads_full: torch.Tensor, lr: float, w_out: torch.Tensor | None = None):
        self.plan.update_recompress(self.packed.data_ptr(), self.resid.data_ptr(), self.sb.data_ptr(),
                                    grads_full.data_ptr(), lr, self.ws.data_ptr(),
                                    None if w_out is None else w_out.data_ptr(), self._s())

    # ---- per-variable views on the host
    def host_state(self):
        torch.cuda.synchronize()
        assert self.plan.status(self._s()) == 0, "a kernel gave up waiting for one of its copies"
        return (self.packed.cpu().numpy(), self.resid.cpu().numpy(), self.sb.cpu().numpy())

    def var_packed(self, packed_host, i):
        p = self.plan
        return packed_host[p.packed_off[i]:p.packed_off[i] + p.var_packed_bytes[i]]

    def var_resid(self, resid_host, i):
        p = self.plan
        return resid_host[p.resid_off[i]:p.resid_off[i] + p.numel[i]]

    def var_sb(self, sb_host, i):
        k = self.plan.sb_slot[i]
        return sb_host[2 * k], sb_host[2 * k + 1]


def same_f32(a, b) -> bool:
    """Bit-for-bit equal, except that any NaN equals any NaN."""
    a = np.asarray(a, np.float32).ravel()
    b = np.asarray(b, np.float32).ravel()
    na, nb = np.isnan(a), np.isnan(b)
    return bool(np.array_equal(na, nb) and np.array_equal(a.view(np.uint32)[~na], b.view(np.uint32)[~nb]))


def ulp_diff(a: np.float32, b: np.float32) -> int:
    """Distance in FP32 units in the last place (NaN vs NaN = 0; sign change = large)."""
    a, b = np.float32(a), np.float32(b)
    if np.isnan(a) and np.isnan(b):
        return 0
    if np.isnan(a) or np.isnan(b):
        return 1 << 30

    def key(x):
        u = int(np.float32(x).view(np.uint32))
        return u if u < 0x80000000 else 0x80000000 - u
    return abs(key(a) - key(b))
