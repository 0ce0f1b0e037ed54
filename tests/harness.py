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


GUARD_BYTES = 1024
GUARD_BYTE = 0xA5


class Guarded:
    """A device buffer followed by canary bytes: no race detector or sanitizer is available for the
    GPU runs, so every buffer a kernel writes is followed by a known pattern that the tests check
    after the calls (a store past the end of an arena shows up here)."""

    def __init__(self, n: int, dtype, dev, fill=None):
        self.n = max(int(n), 16)
        item = torch.empty(0, dtype=dtype).element_size()
        nbytes = (self.n * item + 15) // 16 * 16
        self.raw = torch.empty(nbytes + GUARD_BYTES, dtype=torch.uint8, device=dev)
        self.raw[nbytes:] = GUARD_BYTE
        self.t = self.raw[:self.n * item].view(dtype)
        if fill is None:
            self.t.zero_()
            self.raw[self.n * item:nbytes] = 0
        else:
            self.t.fill_(fill)
            self.raw[self.n * item:nbytes] = GUARD_BYTE
        self._tail = self.n * item if fill is not None else nbytes

    def intact(self) -> bool:
        return bool((self.raw[self._tail:] == GUARD_BYTE).all())


class DeviceModel:
    """Device buffers of one compressed model plus helpers to move variables in and out."""

    def __init__(self, plan: omc.Plan, device="cuda:0"):
        self.plan = plan
        self.dev = torch.device(device)
        self.guards = {}

        def z(name, n, dt):
            g = Guarded(n, dt, self.dev)
            self.guards[name] = g
            return g.t
        self.packed = z("packed", plan.packed_bytes, torch.uint8)
        self.resid = z("resid", plan.resid_elems, torch.float32)
        self.sb = z("sb", 2 * plan.n_quantised, torch.float32)
        self.ws = z("workspace", plan.workspace_bytes, torch.uint8)
        plan.prepare(self.ws.data_ptr(), torch.cuda.current_stream().cuda_stream)

    def check_guards(self):
        """The canary bytes behind every arena are untouched."""
        for name, g in self.guards.items():
            assert g.intact(), "a kernel wrote past the end of the %s arena" % name

    def _s(self):
        return torch.cuda.current_stream().cuda_stream

    def upload_full(self, arrays) -> torch.Tensor:
        return torch.from_numpy(to_full(self.plan, arrays)).to(self.dev)

    def full_buffer(self, name: str) -> torch.Tensor:
        """A zeroed FP32 buffer in the full layout with canary bytes behind it (for outputs)."""
        g = Guarded(self.plan.full_elems, torch.float32, self.dev)
        self.guards[name] = g
        return g.t[:self.plan.full_elems]

    def compress(self, params_full: torch.Tensor):
        self.plan.compress(params_full.data_ptr(), self.packed.data_ptr(), self.resid.data_ptr(),
                           self.sb.data_ptr(), self.ws.data_ptr(), self._s())

    def decompress(self, first_var=0, n_vars=None, out=None) -> torch.Tensor:
        if out is None:
            out = self.full_buffer("decompress output")
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
        self.check_guards()
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
