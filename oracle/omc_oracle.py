"""ctypes front end of the CPU oracle (``omc_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the benchmark's CPU-baseline
leg.  It shares nothing with the CUDA library and the library never imports it.

The wrapper marshals numpy arrays and loops over variables; all of the method's arithmetic is in
the C file.  A model state is a plain dict (see :func:`compress`).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "omc_oracle.c")
_LIB = os.path.join(_HERE, "libomc_oracle.so")

KIND_WEIGHT_MATRIX, KIND_BIAS, KIND_NORM, KIND_OTHER = 0, 1, 2, 3


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fused multiply-add contraction) and return the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC", "-std=gnu11",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u8p, u32p, u64p = C.POINTER(C.c_uint8), C.POINTER(C.c_uint32), C.POINTER(C.c_uint64)
        f32p, f64p = C.POINTER(C.c_float), C.POINTER(C.c_double)
        L.orc_format_ok.argtypes = [C.c_int, C.c_int]
        L.orc_decode.argtypes = [C.c_uint32, C.c_int, C.c_int]
        L.orc_decode.restype = C.c_float
        L.orc_encode.argtypes = [C.c_float, C.c_int, C.c_int]
        L.orc_encode.restype = C.c_uint32
        L.orc_fixed_format_ok.argtypes = [C.c_int, C.c_int]
        L.orc_decode_fixed.argtypes = [C.c_uint32, C.c_int, C.c_int]
        L.orc_decode_fixed.restype = C.c_float
        L.orc_encode_fixed.argtypes = [C.c_float, C.c_int, C.c_int]
        L.orc_encode_fixed.restype = C.c_uint32
        L.orc_decode_fixed_array.argtypes = [u32p, C.c_uint64, C.c_int, C.c_int, f32p]
        L.orc_encode_fixed_array.argtypes = [f32p, C.c_uint64, C.c_int, C.c_int, u32p]
        L.orc_compress_var_fx.argtypes = [f32p, C.c_uint64, C.c_int, C.c_int, C.c_int, C.c_int, u8p, f32p, f32p]
        L.orc_decompress_var_fx.argtypes = [u8p, C.c_uint64, C.c_int, C.c_int, C.c_int, C.c_float, C.c_float,
                                            f32p]
        L.orc_update_recompress_var_fx.argtypes = [u8p, C.c_uint64, C.c_int, C.c_int, C.c_int, C.c_int, f32p,
                                                   f32p, f32p, C.c_float, f32p]
        L.orc_decode_array.argtypes = [u32p, C.c_uint64, C.c_int, C.c_int, f32p]
        L.orc_encode_array.argtypes = [f32p, C.c_uint64, C.c_int, C.c_int, u32p]
        L.orc_packed_bytes.argtypes = [C.c_uint64, C.c_int]
        L.orc_packed_bytes.restype = C.c_uint64
        L.orc_pack.argtypes = [u32p, C.c_uint64, C.c_int, u8p]
        L.orc_unpack.argtypes = [u8p, C.c_uint64, C.c_int, u32p]
        L.orc_unpack_one.argtypes = [u8p, C.c_uint64, C.c_int]
        L.orc_unpack_one.restype = C.c_uint32
        L.orc_exact_sum.argtypes = [f64p, C.c_uint64]
        L.orc_exact_sum.restype = C.c_double
        L.orc_fit.argtypes = [f32p, f32p, C.c_uint64, C.c_int, f32p, f32p, f64p]
        L.orc_compress_var.argtypes = [f32p, C.c_uint64, C.c_int, C.c_int, C.c_int, u8p, f32p, f32p]
        L.orc_decompress_var.argtypes = [u8p, C.c_uint64, C.c_int, C.c_int, C.c_float, C.c_float,
                                         f32p]
        L.orc_update_recompress_var.argtypes = [u8p, C.c_uint64, C.c_int, C.c_int, C.c_int, f32p,
                                                f32p, f32p, C.c_float, f32p]
        L.orc_sgd_var.argtypes = [f32p, f32p, C.c_uint64, C.c_float]
        L.orc_aggregate_var.argtypes = [C.POINTER(f32p), C.c_uint32, C.c_uint64, f32p]
        L.orc_sum_var.argtypes = [C.POINTER(f32p), C.c_uint32, C.c_uint64, f32p]
        L.orc_divide_var.argtypes = [f32p, C.c_uint64, C.c_uint32, f32p]
        L.orc_splitmix64.argtypes = [C.c_uint64, C.c_uint32]
        L.orc_splitmix64.restype = C.c_uint64
        L.orc_plan_seed.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32]
        L.orc_plan_seed.restype = C.c_uint64
        L.orc_select.argtypes = [u8p, C.c_uint32, C.c_double, C.c_uint64, u8p]
        L.orc_model_bytes.argtypes = [u64p, u8p, C.c_uint32, C.c_int]
        L.orc_model_bytes.restype = C.c_uint64
        _lib = L
    return _lib


def _p(a: np.ndarray, ct):
    return a.ctypes.data_as(C.POINTER(ct))


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


# --------------------------------------------------------------------------------------------
# scalar / array codec

def decode(codes, E: int, M: int, fixed: bool = False) -> np.ndarray:
    """fixed=True: the fixed-point variant, (E, M) = (integer bits, fraction bits)."""
    codes = np.ascontiguousarray(codes, dtype=np.uint32).ravel()
    out = np.empty(codes.size, np.float32)
    fn = lib().orc_decode_fixed_array if fixed else lib().orc_decode_array
    fn(_p(codes, C.c_uint32), codes.size, E, M, _p(out, C.c_float))
    return out


def encode(x, E: int, M: int, fixed: bool = False) -> np.ndarray:
    x = _f32(x).ravel()
    out = np.empty(x.size, np.uint32)
    fn = lib().orc_encode_fixed_array if fixed else lib().orc_encode_array
    fn(_p(x, C.c_float), x.size, E, M, _p(out, C.c_uint32))
    return out


def packed_bytes(n: int, B: int) -> int:
    return int(lib().orc_packed_bytes(n, B))


def pack(codes, B: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint32).ravel()
    out = np.empty(packed_bytes(codes.size, B), np.uint8)
    lib().orc_pack(_p(codes, C.c_uint32), codes.size, B, _p(out, C.c_uint8))
    return out


def unpack(packed, n: int, B: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    out = np.empty(n, np.uint32)
    lib().orc_unpack(_p(packed, C.c_uint8), n, B, _p(out, C.c_uint32))
    return out


def exact_sum(x) -> float:
    x = np.ascontiguousarray(x, dtype=np.float64).ravel()
    return float(lib().orc_exact_sum(_p(x, C.c_double), x.size))


def fit(V, Vt, pvt: bool = True, want_sums: bool = False):
    V, Vt = _f32(V).ravel(), _f32(Vt).ravel()
    s, b = C.c_float(), C.c_float()
    sums = np.zeros(4, np.float64)
    lib().orc_fit(_p(V, C.c_float), _p(Vt, C.c_float), V.size, int(pvt), C.byref(s), C.byref(b),
                  _p(sums, C.c_double))
    if want_sums:
        return np.float32(s.value), np.float32(b.value), sums
    return np.float32(s.value), np.float32(b.value)


# --------------------------------------------------------------------------------------------
# per-variable operations

def compress_var(V, E: int, M: int, pvt: bool = True, fixed: bool = False):
    V = _f32(V).ravel()
    out = np.empty(packed_bytes(V.size, 1 + E + M), np.uint8)
    s, b = C.c_float(), C.c_float()
    lib().orc_compress_var_fx(_p(V, C.c_float), V.size, int(fixed), E, M, int(pvt), _p(out, C.c_uint8),
                              C.byref(s), C.byref(b))
    return out, np.float32(s.value), np.float32(b.value)


def decompress_var(packed, n: int, E: int, M: int, s, b, fixed: bool = False) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    out = np.empty(n, np.float32)
    lib().orc_decompress_var_fx(_p(packed, C.c_uint8), n, int(fixed), E, M, C.c_float(float(s)),
                                C.c_float(float(b)), _p(out, C.c_float))
    return out


def update_recompress_var(packed, n: int, E: int, M: int, s, b, g, lr: float, pvt: bool = True,
                          want_w: bool = False, fixed: bool = False):
    """Returns (new_packed, s', b'[, W]); the input array is not modified."""
    packed = np.array(packed, dtype=np.uint8, copy=True)
    g = _f32(g).ravel()
    sc, bc = C.c_float(float(s)), C.c_float(float(b))
    w = np.empty(n, np.float32) if want_w else None
    lib().orc_update_recompress_var_fx(_p(packed, C.c_uint8), n, int(fixed), E, M, int(pvt), C.byref(sc),
                                       C.byref(bc), _p(g, C.c_float), C.c_float(lr),
                                       _p(w, C.c_float) if want_w else None)
    if want_w:
        return packed, np.float32(sc.value), np.float32(bc.value), w
    return packed, np.float32(sc.value), np.float32(bc.value)


def sgd_var(v, g, lr: float) -> np.ndarray:
    v = np.array(v, dtype=np.float32, copy=True).ravel()
    g = _f32(g).ravel()
    lib().orc_sgd_var(_p(v, C.c_float), _p(g, C.c_float), v.size, C.c_float(lr))
    return v


def aggregate_var(client_values) -> np.ndarray:
    """FP32 mean of one variable over the clients (their decompressed or FP32 values), clients
    added in index order, one division at the end."""
    xs = [_f32(x).ravel() for x in client_values]
    n = xs[0].size
    ptrs = (C.POINTER(C.c_float) * len(xs))(*[_p(x, C.c_float) for x in xs])
    out = np.empty(n, np.float32)
    lib().orc_aggregate_var(ptrs, len(xs), n, _p(out, C.c_float))
    return out


def sum_var(client_values) -> np.ndarray:
    """Un-divided FP32 sum of one variable over clients, in index order."""
    xs = [_f32(x).ravel() for x in client_values]
    n = xs[0].size
    ptrs = (C.POINTER(C.c_float) * len(xs))(*[_p(x, C.c_float) for x in xs])
    out = np.empty(n, np.float32)
    lib().orc_sum_var(ptrs, len(xs), n, _p(out, C.c_float))
    return out


def divide_var(x, K: int) -> np.ndarray:
    x = _f32(x).ravel()
    out = np.empty(x.size, np.float32)
    lib().orc_divide_var(_p(x, C.c_float), x.size, K, _p(out, C.c_float))
    return out


def aggregate_two_stage(states_by_holder, threads: int = 1) -> list:
    """Mean over the clients of several holders (servers, GPUs): per-holder sums in client order,
    the holders' sums added in holder order, one division by the number of all clients."""
    holders = [h for h in states_by_holder if h]
    k_total = sum(len(h) for h in holders)
    sums = []
    for h in holders:
        dec = [decompress(st, threads) for st in h]
        sums.append([sum_var([d[i] for d in dec]) for i in range(len(dec[0]))])
    return [divide_var(sum_var([s[i] for s in sums]), k_total) for i in range(len(sums[0]))]


def aggregate(states, threads: int = 1) -> list:
    """Server-side mean of the clients' models: every client's state is decompressed, then each
    variable is averaged by :func:`aggregate_var`."""
    dec = [decompress(st, threads) for st in states]
    return _map(lambda i: aggregate_var([d[i] for d in dec]), range(len(dec[0])), threads)


# --------------------------------------------------------------------------------------------
# plan-level: selection, sizes, whole-model state

def splitmix64(seed: int, nth: int) -> int:
    return int(lib().orc_splitmix64(seed, nth))


def plan_seed(base: int, round_: int, client: int) -> int:
    """Selection seed of (round, client) under one job seed (Sec. 3.1)."""
    return int(lib().orc_plan_seed(base, round_, client))


def select(kinds, fraction: float, seed: int, weights_only: bool = True) -> np.ndarray:
    kinds = np.asarray(kinds)
    eligible = (kinds == KIND_WEIGHT_MATRIX) if weights_only else np.ones(kinds.size, bool)
    eligible = np.ascontiguousarray(eligible, dtype=np.uint8)
    sel = np.zeros(kinds.size, np.uint8)
    lib().orc_select(_p(eligible, C.c_uint8), kinds.size, float(fraction), seed,
                     _p(sel, C.c_uint8))
    return sel.astype(bool)


def model_bytes(numel, selected, B: int) -> int:
    numel = np.ascontiguousarray(numel, dtype=np.uint64)
    sel = np.ascontiguousarray(selected, dtype=np.uint8)
    return int(lib().orc_model_bytes(_p(numel, C.c_uint64), _p(sel, C.c_uint8), numel.size, B))


def _map(fn, items, threads: int):
    if threads <= 1:
        return [fn(it) for it in items]
    with ThreadPoolExecutor(max_workers=threads) as ex:      # the C calls release the GIL
        return list(ex.map(fn, items))


def compress(variables, selected, E: int, M: int, pvt: bool = True, threads: int = 1,
             fixed: bool = False) -> dict:
    """Model state: {'E','M','fixed','pvt','n': [...], 'sel': [...], 'packed': {i: u8}, 's': {i: f32},
    'b': {i: f32}, 'fp32': {i: f32 array}} -- variables not selected stay in FP32 (Sec. 2.4)."""
    st = {"E": E, "M": M, "fixed": bool(fixed), "pvt": pvt, "n": [int(np.asarray(v).size) for v in variables],
          "sel": [bool(x) for x in selected], "packed": {}, "s": {}, "b": {}, "fp32": {}}

    def one(i):
        if st["sel"][i]:
            return compress_var(variables[i], E, M, pvt, fixed)
        return np.array(variables[i], dtype=np.float32, copy=True).ravel()

    for i, r in enumerate(_map(one, range(len(variables)), threads)):
        if st["sel"][i]:
            st["packed"][i], st["s"][i], st["b"][i] = r
        else:
            st["fp32"][i] = r
    return st


def decompress(st: dict, threads: int = 1) -> list:
    def one(i):
        if st["sel"][i]:
            return decompress_var(st["packed"][i], st["n"][i], st["E"], st["M"], st["s"][i],
                                  st["b"][i], st.get("fixed", False))
        return st["fp32"][i].copy()

    return _map(one, range(len(st["n"])), threads)


def update_recompress(st: dict, grads, lr: float, threads: int = 1, want_w: bool = False):
    """One OMC round over the whole model, in place on ``st``.  Returns the list of W if asked."""
    def one(i):
        if st["sel"][i]:
            return update_recompress_var(st["packed"][i], st["n"][i], st["E"], st["M"], st["s"][i],
                                         st["b"][i], grads[i], lr, st["pvt"], want_w=want_w,
                                         fixed=st.get("fixed", False))
        return sgd_var(st["fp32"][i], grads[i], lr)

    ws = []
    for i, r in enumerate(_map(one, range(len(st["n"])), threads)):
        if st["sel"][i]:
            st["packed"][i], st["s"][i], st["b"][i] = r[0], r[1], r[2]
            if want_w:
                ws.append(r[3])
        else:
            st["fp32"][i] = r
            if want_w:
                ws.append(r)
    return ws if want_w else None
