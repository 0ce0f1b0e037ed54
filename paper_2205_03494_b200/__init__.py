"""Python binding of libomc (Online Model Compression parameter store for B200).

Argument marshalling only: every function below forwards to the C-ABI entry point of the same name
in ``include/omc.h``; all arithmetic runs in the library's CUDA kernels.  Device buffers are passed
as integer addresses (e.g. ``torch.Tensor.data_ptr()``), streams as ``cudaStream_t`` integers.
There is no CPU fallback: if ``libomc.so`` has not been built, importing the binding's functions
raises.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libomc.so")

KIND_WEIGHT_MATRIX, KIND_BIAS, KIND_NORM, KIND_OTHER = 0, 1, 2, 3
PLAN_PVT, PLAN_WEIGHTS_ONLY = 1, 2
PLAN_DEFAULT = PLAN_PVT | PLAN_WEIGHTS_ONLY
FORMAT_FIXED_POINT = 1

EXPORTS = ["omc_strerror", "omc_last_cuda_error", "omc_plan", "omc_plan_destroy", "omc_plan_seed", "omc_plan_sizes",
           "omc_plan_var", "omc_plan_division", "omc_plan_prepare", "omc_plan_status", "omc_plan_inject_wait_timeout", "omc_compress", "omc_decompress",
           "omc_update_recompress", "omc_update_recompress_host", "omc_transition", "omc_aggregate", "omc_aggregate_sum", "omc_aggregate_add", "omc_divide", "omc_matmul",
           "omc_compress_var_static", "omc_static_status"]
STATIC_MAX_NUMEL = 1 << 28


class OmcError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().omc_strerror(status).decode()
        if status == -6:
            msg += " [cudaError %d]" % lib().omc_last_cuda_error()
        super().__init__("%s: %s (%d)" % (where, msg, status))


class Format(C.Structure):
    _fields_ = [("sign_bits", C.c_uint8), ("exp_bits", C.c_uint8), ("man_bits", C.c_uint8),
                ("flags", C.c_uint8)]


class VarDesc(C.Structure):
    _fields_ = [("numel", C.c_uint64), ("kind", C.c_uint32), ("reserved", C.c_uint32)]


_lib = None


def lib():
    """The loaded shared library (built in-tree by ``python -m paper_2205_03494_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libomc.so is missing: build it with "
                               "`python -m paper_2205_03494_b200.build` (no fallback exists)")
        L = C.CDLL(LIB_PATH)
        vp, u64p, u32p = C.c_void_p, C.POINTER(C.c_uint64), C.POINTER(C.c_uint32)
        L.omc_strerror.argtypes = [C.c_int]
        L.omc_strerror.restype = C.c_char_p
        L.omc_last_cuda_error.restype = C.c_int
        L.omc_plan.argtypes = [C.POINTER(VarDesc), C.c_uint32, Format, C.c_double, C.c_uint64,
                               C.POINTER(C.c_uint8), C.c_uint32, C.POINTER(vp)]
        L.omc_plan_destroy.argtypes = [vp]
        L.omc_plan_seed.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32]
        L.omc_plan_seed.restype = C.c_uint64
        L.omc_plan_sizes.argtypes = [vp, u64p, u64p, u64p, u32p, u64p, u64p]
        L.omc_plan_var.argtypes = [vp, C.c_uint32, C.POINTER(C.c_int), u64p, u64p, u64p, u64p, u32p]
        L.omc_plan_division.argtypes = [vp, u32p, u32p, u64p, C.POINTER(u64p)]
        L.omc_plan_prepare.argtypes = [vp, vp, vp]
        L.omc_plan_status.argtypes = [vp, vp, u32p]
        L.omc_plan_inject_wait_timeout.argtypes = [vp, C.c_uint32]
        L.omc_compress.argtypes = [vp, vp, vp, vp, vp, vp, vp]
        L.omc_decompress.argtypes = [vp, vp, vp, vp, C.c_uint32, C.c_uint32, vp, vp]
        L.omc_update_recompress.argtypes = [vp, vp, vp, vp, vp, C.c_float, vp, vp, vp]
        L.omc_update_recompress_host.argtypes = [vp, vp, vp, vp, vp, C.c_float, vp, vp, vp, vp]
        L.omc_transition.argtypes = [vp] * 10
        L.omc_matmul.argtypes = [vp, C.c_uint32, vp, vp, vp, C.c_uint32, C.c_uint32, C.c_uint32, vp, vp, vp]
        L.omc_aggregate.argtypes = [C.POINTER(vp), C.c_uint32, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), vp, vp]
        L.omc_aggregate_sum.argtypes = L.omc_aggregate.argtypes
        L.omc_aggregate_add.argtypes = L.omc_aggregate.argtypes
        L.omc_divide.argtypes = [vp, vp, C.c_uint32, vp]
        L.omc_compress_var_static.argtypes = [vp, C.c_uint64, Format, C.c_uint32, vp, vp, vp]
        L.omc_static_status.argtypes = [vp, u32p]
        _lib = L
    return _lib


def _check(status: int, where: str):
    if status != 0:
        raise OmcError(status, where)


class Plan:
    """Handle of an ``omc_plan_t``; attributes mirror omc_plan_sizes / omc_plan_var."""

    def __init__(self, numel, kinds, fmt, fraction=1.0, seed=0, mask=None, flags=PLAN_DEFAULT, fixed=False):
        """fmt = (E, M) of S1EyMz, or with fixed=True (integer bits, fraction bits) of the fixed-point
        variant S1IxFy."""
        n = len(numel)
        descs = (VarDesc * max(n, 1))()
        for i in range(n):
            descs[i].numel, descs[i].kind, descs[i].reserved = int(numel[i]), int(kinds[i]), 0
        S, E, M = (1, fmt[0], fmt[1]) if len(fmt) == 2 else fmt
        self.E, self.M, self.B = int(E), int(M), 1 + int(E) + int(M)
        f = Format(S, E, M, FORMAT_FIXED_POINT if fixed else 0)
        self.fixed = bool(fixed)
        mk = None
        if mask is not None:
            mk = (C.c_uint8 * n)(*[1 if m else 0 for m in mask])
        h = C.c_void_p()
        _check(lib().omc_plan(descs, n, f, float(fraction), int(seed), mk, int(flags), C.byref(h)),
               "omc_plan")
        self._h = h
        self.nvars = n
        self.flags = flags
        a, b, c, e, g = (C.c_uint64() for _ in range(5))
        d = C.c_uint32()
        _check(lib().omc_plan_sizes(h, C.byref(a), C.byref(b), C.byref(c), C.byref(d), C.byref(e),
                                    C.byref(g)), "omc_plan_sizes")
        self.full_elems, self.resid_elems, self.packed_bytes = a.value, b.value, c.value
        self.n_quantised, self.workspace_bytes, self.closed_form_bytes = d.value, e.value, g.value
        self.numel = [int(x) for x in numel]
        self.quantised, self.full_off, self.resid_off = [], [], []
        self.packed_off, self.var_packed_bytes, self.sb_slot = [], [], []
        q = C.c_int()
        o1, o2, o3, o4 = (C.c_uint64() for _ in range(4))
        sl = C.c_uint32()
        for i in range(n):
            _check(lib().omc_plan_var(h, i, C.byref(q), C.byref(o1), C.byref(o2), C.byref(o3),
                                      C.byref(o4), C.byref(sl)), "omc_plan_var")
            self.quantised.append(bool(q.value))
            self.full_off.append(o1.value)
            self.resid_off.append(o2.value)
            self.packed_off.append(o3.value)
            self.var_packed_bytes.append(o4.value)
            self.sb_slot.append(sl.value)

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            lib().omc_plan_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def division(self):
        """omc_plan_division: (n_warps, n_tiles, [run_start[0], ..., run_start[n_runs]])."""
        nw, nr, nt, tab = C.c_uint32(), C.c_uint32(), C.c_uint64(), C.POINTER(C.c_uint64)()
        _check(lib().omc_plan_division(self._h, C.byref(nw), C.byref(nr), C.byref(nt), C.byref(tab)),
               "omc_plan_division")
        return nw.value, nt.value, [tab[i] for i in range(nr.value + 1)]

    # ---- device calls (addresses are ints; 0/None = NULL) -----------------------------------
    def prepare(self, workspace, stream=0):
        _check(lib().omc_plan_prepare(self._h, workspace, stream), "omc_plan_prepare")

    def inject_wait_timeout(self, polls: int):
        """omc_plan_inject_wait_timeout: the next launch gives up its waits (diagnostics)."""
        _check(lib().omc_plan_inject_wait_timeout(self._h, int(polls)), "omc_plan_inject_wait_timeout")

    def status(self, stream=0) -> int:
        st = C.c_uint32(0)
        _check(lib().omc_plan_status(self._h, stream, C.byref(st)), "omc_plan_status")
        return st.value

    def compress(self, params, packed, resid, sb, workspace, stream=0):
        _check(lib().omc_compress(self._h, params, packed, resid, sb, workspace, stream),
               "omc_compress")

    def decompress(self, packed, resid, sb, out, first_var=0, n_vars=None, stream=0):
        n_vars = self.nvars - first_var if n_vars is None else n_vars
        _check(lib().omc_decompress(self._h, packed, resid, sb, first_var, n_vars, out, stream),
               "omc_decompress")

    def update_recompress(self, packed, resid, sb, grads, lr, workspace, debug_w_out=None,
                          stream=0):
        _check(lib().omc_update_recompress(self._h, packed, resid, sb, grads, float(lr),
                                           debug_w_out, workspace, stream), "omc_update_recompress")

    def update_recompress_host(self, packed, resid, sb, host_grads, lr, grads_staging, host_sb_out,
                               workspace, stream=0):
        _check(lib().omc_update_recompress_host(self._h, packed, resid, sb, host_grads, float(lr),
                                                grads_staging, host_sb_out, workspace, stream),
               "omc_update_recompress_host")


def plan_seed(base_seed: int, round_: int, client: int) -> int:
    """omc_plan_seed: the selection seed of (round, client) under one job seed (Sec. 3.1)."""
    return int(lib().omc_plan_seed(int(base_seed), int(round_), int(client)))


def transition(plan_from: Plan, plan_to: Plan, packed_from, resid_from, sb_from, packed_to, resid_to, sb_to,
               workspace_to, stream=0):
    """omc_transition: state under plan_from -> state under plan_to (addresses are ints)."""
    _check(lib().omc_transition(plan_from._h, plan_to._h, packed_from, resid_from, sb_from, packed_to, resid_to,
                                sb_to, workspace_to, stream), "omc_transition")


def matmul(plan: Plan, var, packed, sb, x_half, M, N, K, y, rowsum_scratch, stream=0):
    """omc_matmul: Y = X * Wbar^T straight from the codes of variable `var` (addresses are ints)."""
    _check(lib().omc_matmul(plan._h, var, packed, sb, x_half, M, N, K, y, rowsum_scratch, stream), "omc_matmul")


def aggregate(plans, packed, resid, sb, out, stream=0):
    """omc_aggregate: mean of the clients' decompressed models into `out` (addresses are ints)."""
    k = len(plans)
    arr = lambda xs: (C.c_void_p * k)(*[x if not hasattr(x, "_h") else x._h.value for x in xs])
    _check(lib().omc_aggregate(arr(plans), k, arr(packed), arr(resid), arr(sb), out, stream), "omc_aggregate")


def aggregate_sum(plans, packed, resid, sb, out, stream=0):
    """omc_aggregate_sum: the clients' decompressed models added up, not divided (addresses are ints)."""
    k = len(plans)
    arr = lambda xs: (C.c_void_p * k)(*[x if not hasattr(x, "_h") else x._h.value for x in xs])
    _check(lib().omc_aggregate_sum(arr(plans), k, arr(packed), arr(resid), arr(sb), out, stream), "omc_aggregate_sum")


MAX_CLIENTS_PER_CALL = 16      # of omc_aggregate, omc_aggregate_sum and omc_aggregate_add


def aggregate_add(plans, packed, resid, sb, out, stream=0):
    """omc_aggregate_add: this batch of clients added, in index order, to the sum `out` already holds."""
    k = len(plans)
    arr = lambda xs: (C.c_void_p * k)(*[x if not hasattr(x, "_h") else x._h.value for x in xs])
    _check(lib().omc_aggregate_add(arr(plans), k, arr(packed), arr(resid), arr(sb), out, stream), "omc_aggregate_add")


def divide(plan: Plan, values, divisor: int, stream=0):
    """omc_divide: values[e] /= divisor over a buffer in the plan's full layout."""
    _check(lib().omc_divide(plan._h, values, int(divisor), stream), "omc_divide")


def compress_var_static(values, numel, fmt, packed, sb, flags=PLAN_PVT, stream=0, fixed=False):
    """omc_compress_var_static: one variable, no plan, no workspace, no allocation (addresses are
    ints).  Raises OmcError like the other calls (status -8 = numel beyond STATIC_MAX_NUMEL)."""
    S, E, M = (1, fmt[0], fmt[1]) if len(fmt) == 2 else fmt
    _check(lib().omc_compress_var_static(values, int(numel), Format(S, E, M, FORMAT_FIXED_POINT if fixed else 0),
                                         int(flags), packed, sb,
                                         stream), "omc_compress_var_static")


def static_status(stream=0) -> int:
    """omc_static_status: the status word of the most recent compress_var_static on this device."""
    st = C.c_uint32(0)
    _check(lib().omc_static_status(stream, C.byref(st)), "omc_static_status")
    return st.value
