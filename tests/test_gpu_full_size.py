"""Parity at the benchmark configurations' full sizes, in the launch configuration bench.py times
(whole-model plans, one kernel launch per call).  The GPU processes every variable; the oracle
recomputes a sample of variables (largest, smallest, first, last, FP32-only ones) completely, so
every code, (s, b) and W of those variables is compared; the rest is covered by the status word and
by the zero-padding and determinism checks."""
import numpy as np
import pytest
import torch

import paper_2205_03494_b200 as omc
from paper_2205_03494_b200 import workloads
from test_gpu_parity import Lockstep

pytestmark = pytest.mark.gpu


def pick(wl, extra=()):
    n = np.array(wl.numel)
    q = [i for i, k in enumerate(wl.kinds) if k == 0]
    o = [i for i, k in enumerate(wl.kinds) if k != 0]
    s = {q[0], q[-1], q[int(np.argmax(n[q]))], q[int(np.argmin(n[q]))], *extra}
    if o:
        s |= {o[0], o[-1]}
    return sorted(s)


def test_conformer_like_100m_three_rounds():
    wl = workloads.conformer_like()
    sample = pick(wl, extra=(2, 20, 300, 301))
    params = wl.all_params()
    ls = Lockstep(wl.numel, wl.kinds, wl.fmt, params, sample=sample, threads=8)
    del params
    ls.check_decompress()
    for r in range(3):
        packed = ls.round(wl.all_grads(r), wl.lr if r < 2 else 30.0)
    ls.check_padding(packed)
    ls.check_decompress()
    assert ls.sb_ulp_cases <= 1, ls.sb_ulp_cases


def test_ragged_4096_variables_two_rounds():
    wl = workloads.ragged()
    n = np.array(wl.numel)
    order = np.argsort(n)
    sample = sorted({int(i) for i in list(order[:6]) + list(order[-3:]) + list(order[::400])} | {0, 4095})
    params = wl.all_params()
    ls = Lockstep(wl.numel, wl.kinds, wl.fmt, params, sample=sample, threads=8)
    del params
    ls.check_decompress()
    for r in range(2):
        packed = ls.round(wl.all_grads(r), 0.01 if r == 0 else 20.0, want_w=(r == 1))
    ls.check_padding(packed)
    assert ls.sb_ulp_cases <= 2, ls.sb_ulp_cases


def test_large_transformer_1p6b_one_round():
    """32 layers at d = 2048, 12-bit codes: 1,610,612,736 parameters, one round."""
    free, _ = torch.cuda.mem_get_info()
    if free < 24e9:
        pytest.skip("needs about 24 GB of free device memory")
    wl = workloads.large_transformer()
    sample = [0, 4, 95, 191]          # two attention matrices, a 2048x8192 and the last 8192x2048
    params = wl.all_params()
    ls = Lockstep(wl.numel, wl.kinds, wl.fmt, params, sample=sample, threads=4)
    del params
    torch.cuda.empty_cache()
    packed = ls.round(wl.all_grads(0), 2.0, want_w=False)
    ls.check_padding(packed)
    assert ls.sb_ulp_cases <= 1, ls.sb_ulp_cases
