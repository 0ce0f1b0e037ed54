"""Randomised parity: seeded random models (variable counts, sizes from one element to tens of
tiles, kinds, value scales), random formats of both codec families (compiled and run-time),
random fractions and plan switches, a few rounds with random step sizes, alternately with and
without the W output, then a re-selection and a server-side mean -- every step against the oracle,
bit for bit (codes, padding, FP32 variables, W, decompressed values; (s, b) within one unit in
the last place).  The seeds are fixed, so a failure reproduces."""
import numpy as np
import pytest
import torch

import paper_2205_03494_b200 as omc
from oracle import omc_oracle as orc
from harness import DeviceModel, from_full, same_f32
from test_gpu_parity import Lockstep, oracle_transition

pytestmark = pytest.mark.gpu

FLOAT_FORMATS = [(5, 2), (4, 3), (5, 6), (5, 10), (4, 14), (3, 7), (2, 3), (3, 9), (4, 8), (5, 7), (8, 7), (8, 23),
                 (6, 5), (2, 0), (7, 22), (3, 4)]
FIXED_FORMATS = [(0, 7), (0, 11), (0, 15), (1, 6), (2, 9), (0, 20)]


def random_model(rng):
    nvars = int(rng.integers(1, 24))
    numel, kinds = [], []
    for _ in range(nvars):
        kind = rng.choice([0, 0, 0, 1, 2, 3])
        if kind == 0:
            n = int(np.exp(rng.uniform(0, np.log(40000))))
            if rng.random() < 0.3:
                n = int(rng.choice([1024, 2048, 4096, 8192, 512, 1536]))     # whole granules, too
        else:
            n = int(rng.integers(1, 3000))
        numel.append(max(n, 1))
        kinds.append(int(kind))
    if 0 not in kinds:
        kinds[0] = 0
    return numel, kinds


@pytest.mark.parametrize("seed", range(24))
def test_random_model_against_oracle(seed):
    rng = np.random.default_rng(1000 + seed)
    fixed = bool(seed % 3 == 2)
    fmt = (FIXED_FORMATS if fixed else FLOAT_FORMATS)[int(rng.integers(0, 6 if fixed else len(FLOAT_FORMATS)))]
    numel, kinds = random_model(rng)
    span = 2.0 ** fmt[0] if fixed else min(2.0 ** ((1 << (fmt[0] - 1)) - 2), 4.0)
    scales = [span * 10.0 ** rng.uniform(-4, 0) for _ in numel]
    params = [(rng.standard_normal(n) * sc).astype(np.float32) for n, sc in zip(numel, scales)]
    flags = (omc.PLAN_PVT if rng.random() < 0.8 else 0) | (omc.PLAN_WEIGHTS_ONLY if rng.random() < 0.7 else 0)
    fraction = float(rng.choice([1.0, 0.9, 0.5, 0.25]))
    ls = Lockstep(numel, kinds, fmt, params, fraction=fraction, seed=int(rng.integers(0, 1 << 30)), flags=flags, fixed=fixed)
    ls.check_padding(ls.check_state("compress-again", resync=False))
    ls.check_decompress()
    if len(numel) > 2:
        first = int(rng.integers(0, len(numel) - 1))
        ls.check_decompress(first=first, count=int(rng.integers(1, len(numel) - first + 1)))
    for r in range(3):
        grads = [(rng.standard_normal(n) * sc * 0.3).astype(np.float32) for n, sc in zip(numel, scales)]
        packed = ls.round(grads, float(10.0 ** rng.uniform(-2, 0.5)), want_w=bool((seed + r) % 2))
        ls.check_padding(packed)
    ls.check_decompress()
    # re-selection to another random subset, one more round there
    plan_to = omc.Plan(numel, kinds, fmt, fraction=float(rng.choice([1.0, 0.75, 0.4])), seed=int(rng.integers(0, 1 << 30)),
                       flags=flags, fixed=fixed)
    st = torch.cuda.current_stream().cuda_stream
    if not (fixed and fmt not in [(0, 7), (0, 11), (0, 15)]) and not (not fixed and fmt in [(6, 5), (2, 0), (7, 22), (3, 4)]):
        dm_to = DeviceModel(plan_to)
        a, b = ls.dm, dm_to
        omc.transition(ls.plan, plan_to, a.packed.data_ptr(), a.resid.data_ptr(), a.sb.data_ptr(),
                       b.packed.data_ptr(), b.resid.data_ptr(), b.sb.data_ptr(), b.ws.data_ptr(), st)
        ls.st = oracle_transition(ls.st, plan_to.quantised)
        ls.plan, ls.dm = plan_to, dm_to
        ls.check_padding(ls.check_state("transition"))
        grads = [(rng.standard_normal(n) * sc * 0.3).astype(np.float32) for n, sc in zip(numel, scales)]
        ls.round(grads, 0.3, want_w=False)
        # the mean of this client and a second one with its own subset
        other = Lockstep(numel, kinds, fmt, [p * np.float32(1.01) for p in params], fraction=0.6,
                         seed=int(rng.integers(0, 1 << 30)), flags=flags, fixed=fixed)
        out = torch.zeros(ls.plan.full_elems, dtype=torch.float32, device="cuda")
        cl = [ls, other]
        omc.aggregate([c.plan for c in cl], [c.dm.packed.data_ptr() for c in cl], [c.dm.resid.data_ptr() for c in cl],
                      [c.dm.sb.data_ptr() for c in cl], out.data_ptr(), st)
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        want = orc.aggregate([c.st for c in cl])
        for i in range(len(numel)):
            assert same_f32(from_full(ls.plan, got, i), want[i]), i
    else:       # formats that run on the run-time kernels have no transition / aggregation kernel
        assert omc.lib().omc_transition(ls.plan._h, plan_to._h, 0, 0, 0, 0, 0, 0, 0, None) in (-5, -2, -3)
    assert ls.sb_ulp_cases <= 3, ls.sb_ulp_cases
