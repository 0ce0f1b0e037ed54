"""Seeded synthetic parameter sets shaped like the paper's speech-recognition models.

Input generation only: this module holds none of the method's arithmetic and is the one piece the
tests hand to both the CUDA library and the CPU oracle.  Every variable and every gradient has its
own counter-seeded numpy stream (PCG64 from SeedSequence([seed, tag, variable, round])), so any
subset can be generated alone, in any order, on any number of threads, with identical values.

The sets stand in for the paper's Conformer models (Sec. 3.1): they take the variable shapes, the
share of weight matrices (99.8%, Sec. 2.4) and plausible value distributions, not the trained
weights or the data, which are not available.
"""
from __future__ import annotations

import math
import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field

import numpy as np

KIND_WEIGHT_MATRIX, KIND_BIAS, KIND_NORM, KIND_OTHER = 0, 1, 2, 3
_TAG_PARAM, _TAG_GRAD, _TAG_SHAPE = 1, 2, 3


def _rng(seed, tag, i, rnd=0):
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, tag, i, rnd])))


def default_threads() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return os.cpu_count() or 1


@dataclass
class Var:
    name: str
    shape: tuple
    kind: int
    init: tuple           # ("normal", std) | ("glorot",) | ("const", c) | ("outlier", std, p, std2)
    grad_std: float

    @property
    def numel(self) -> int:
        return int(np.prod(self.shape))


@dataclass
class Workload:
    name: str
    vars: list
    fmt: tuple            # (E, M)
    fraction: float
    seed: int
    lr: float
    rounds: int
    sel_seed: int = 0
    notes: str = ""
    _extra: dict = field(default_factory=dict)

    @property
    def numel(self):
        return [v.numel for v in self.vars]

    @property
    def kinds(self):
        return [v.kind for v in self.vars]

    @property
    def total(self) -> int:
        return sum(self.numel)

    def params(self, i: int) -> np.ndarray:
        v = self.vars[i]
        g = _rng(self.seed, _TAG_PARAM, i)
        n = v.numel
        kind = v.init[0]
        if kind == "const":
            return np.full(n, v.init[1], np.float32)
        if kind == "normal":
            x = g.standard_normal(n, dtype=np.float32)
            x *= np.float32(v.init[1])
            return x
        if kind == "glorot":
            fan_in, fan_out = v.shape[0], v.shape[-1]
            lim = math.sqrt(6.0 / (fan_in + fan_out))
            x = g.random(n, dtype=np.float32)
            x *= np.float32(2 * lim)
            x -= np.float32(lim)
            return x
        if kind == "outlier":
            _, std, p, std2 = v.init
            x = g.standard_normal(n, dtype=np.float32)
            pick = g.random(n, dtype=np.float32) < np.float32(p)
            x *= np.where(pick, np.float32(std2), np.float32(std))
            return x
        raise ValueError(kind)

    def grads(self, i: int, rnd: int = 0) -> np.ndarray:
        v = self.vars[i]
        x = _rng(self.seed, _TAG_GRAD, i, rnd).standard_normal(v.numel, dtype=np.float32)
        x *= np.float32(v.grad_std)
        return x

    def all_params(self, threads: int = 0, which=None) -> list:
        return _pmap(self.params, which if which is not None else range(len(self.vars)), threads)

    def all_grads(self, rnd: int = 0, threads: int = 0, which=None) -> list:
        return _pmap(lambda i: self.grads(i, rnd), which if which is not None else range(len(self.vars)),
                     threads)


def _pmap(fn, items, threads):
    threads = threads or default_threads()
    items = list(items)
    if threads <= 1 or len(items) <= 1:
        return [fn(i) for i in items]
    with ThreadPoolExecutor(max_workers=threads) as ex:
        return list(ex.map(fn, items))


# ------------------------------------------------------------------------------------------------

def tiny(fmt=(5, 2), fraction=1.0, sel_seed=0) -> Workload:
    """Four 256x256 weight matrices ~ N(0, 0.05^2) and four zero bias vectors of length 256;
    gradients ~ N(0, (1e-3)^2); one round at lr = 0.01."""
    vs = []
    for k in range(4):
        vs.append(Var("dense%d/w" % k, (256, 256), KIND_WEIGHT_MATRIX, ("normal", 0.05), 1e-3))
        vs.append(Var("dense%d/b" % k, (256,), KIND_BIAS, ("const", 0.0), 1e-3))
    return Workload("tiny", vs, fmt, fraction, seed=0, lr=0.01, rounds=1, sel_seed=sel_seed)


def conformer_like(blocks: int = 17, d: int = 512, fmt=(5, 10)) -> Workload:
    """Conformer-shaped encoder: per block two feed-forward modules (d x 4d, 4d x d), attention
    Q/K/V/O (d x d), convolution module (pointwise d x 2d and d x d, depthwise d x 32), five
    LayerNorms and one bias per matrix.  Weights Glorot-uniform, norm gains 1, biases 0; gradients
    ~ N(0, (1e-4)^2).  17 blocks at d = 512: 102,776,832 weight parameters in 187 matrices, 99.8%
    of the model."""
    vs = []
    for bl in range(blocks):
        mats = [("ffn1/w1", (d, 4 * d)), ("ffn1/w2", (4 * d, d)), ("att/q", (d, d)), ("att/k", (d, d)),
                ("att/v", (d, d)), ("att/o", (d, d)), ("conv/pw1", (d, 2 * d)), ("conv/dw", (d, 32)),
                ("conv/pw2", (d, d)), ("ffn2/w1", (d, 4 * d)), ("ffn2/w2", (4 * d, d))]
        norms = ["ffn1/ln", "att/ln", "conv/ln", "ffn2/ln", "out/ln"]
        order = [(0, 0), (1, 0), (0, 1), (1, 1), (0, 2), (0, 3), (0, 4), (0, 5), (1, 2), (0, 6), (0, 7),
                 (0, 8), (1, 3), (0, 9), (0, 10), (1, 4)]
        for what, j in order:
            if what == 0:
                nm, shp = mats[j]
                vs.append(Var("b%d/%s" % (bl, nm), shp, KIND_WEIGHT_MATRIX, ("glorot",), 1e-4))
                vs.append(Var("b%d/%s_bias" % (bl, nm), (shp[1],), KIND_BIAS, ("const", 0.0), 1e-4))
            else:
                vs.append(Var("b%d/%s/gain" % (bl, norms[j]), (d,), KIND_NORM, ("const", 1.0), 1e-4))
                vs.append(Var("b%d/%s/bias" % (bl, norms[j]), (d,), KIND_NORM, ("const", 0.0), 1e-4))
    return Workload("conformer_like_%db_d%d" % (blocks, d), vs, fmt, 1.0, seed=1, lr=0.01, rounds=100)


def large_transformer(layers: int = 32, d: int = 2048, fmt=(5, 6)) -> Workload:
    """Per layer: feed-forward d x 4d and 4d x d, four d x d attention matrices; weights
    ~ N(0, 0.02^2) with each element replaced, with probability 0.01, by N(0, 0.5^2); gradients
    ~ N(0, (1e-4)^2).  32 layers at d = 2048: 1,610,612,736 parameters; 20 layers: 1,006,632,960."""
    vs = []
    init = ("outlier", 0.02, 0.01, 0.5)
    for l in range(layers):
        vs.append(Var("l%d/att/q" % l, (d, d), KIND_WEIGHT_MATRIX, init, 1e-4))
        vs.append(Var("l%d/att/k" % l, (d, d), KIND_WEIGHT_MATRIX, init, 1e-4))
        vs.append(Var("l%d/att/v" % l, (d, d), KIND_WEIGHT_MATRIX, init, 1e-4))
        vs.append(Var("l%d/att/o" % l, (d, d), KIND_WEIGHT_MATRIX, init, 1e-4))
        vs.append(Var("l%d/ffn/w1" % l, (d, 4 * d), KIND_WEIGHT_MATRIX, init, 1e-4))
        vs.append(Var("l%d/ffn/w2" % l, (4 * d, d), KIND_WEIGHT_MATRIX, init, 1e-4))
    return Workload("large_transformer_%dl_d%d" % (layers, d), vs, fmt, 1.0, seed=2, lr=0.01, rounds=10)


def ragged(nvars: int = 4096, lo: int = 64, hi: int = 1 << 20, fmt=(5, 2)) -> Workload:
    """Many small variables: element counts log-uniform in [lo, hi], each variable with its own
    scale s log-uniform in [1e-4, 1]: values ~ N(0, s^2), gradients ~ N(0, (0.01 s)^2)."""
    g = _rng(3, _TAG_SHAPE, 0)
    n = np.floor(np.exp(g.uniform(math.log(lo), math.log(hi), nvars))).astype(np.int64)
    s = np.exp(g.uniform(math.log(1e-4), math.log(1.0), nvars))
    vs = [Var("v%d" % i, (int(n[i]),), KIND_WEIGHT_MATRIX, ("normal", float(s[i])), 0.01 * float(s[i]))
          for i in range(nvars)]
    return Workload("ragged_%d" % nvars, vs, fmt, 1.0, seed=3, lr=0.01, rounds=3)


def sweep():
    """Partial-quantisation sweep on the tiny set: (fraction, format) combinations."""
    for p in (0.25, 0.5, 0.75, 1.0):
        for fmt in ((4, 3), (5, 6), (5, 10)):
            yield tiny(fmt=fmt, fraction=p, sel_seed=11)
