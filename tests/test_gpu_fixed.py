"""GPU parity of the fixed-point codec variant (Sec. 2.2 names fixed-point formats as an
alternative; S1IxFy as include/omc.h defines it) against the oracle's: codes, padding, decompressed
values, W and FP32 variables bit-exact, (s, b) within one FP32 unit in the last place, exactly as
for the floating-point codes.  Q7, Q11 and Q15 run the compiled kernels, the other formats the
kernels that take the format at run time."""
import numpy as np
import pytest
import torch

import paper_2205_03494_b200 as omc
from paper_2205_03494_b200 import workloads
from oracle import omc_oracle as orc
from harness import DeviceModel, from_full, same_f32
from test_gpu_parity import Lockstep, oracle_transition, WANT_W

pytestmark = pytest.mark.gpu

FIXED_FORMATS = [(0, 7), (0, 11), (0, 15),                                   # compiled
                 (2, 3), (1, 6), (8, 15), (0, 23), (3, 0), (0, 1), (4, 8)]   # format at run time


@WANT_W
@pytest.mark.parametrize("fmt", FIXED_FORMATS, ids=lambda f: "I%dF%d" % f)
def test_ragged_small_fixed_point(fmt, want_w):
    """Ragged sizes, mixed kinds, values from far inside the range to beyond it (saturation), three
    rounds with steps of several code steps."""
    I, F = fmt
    rng = np.random.default_rng(I * 100 + F)
    numel = [1, 2, 3, 5, 31, 32, 33, 127, 128, 129, 1023, 1024, 1025, 2047, 4096, 5000, 3 * 1024 + 7, 777, 8, 16,
             12289]
    kinds = [0] * len(numel)
    for j in (3, 9, 14):
        kinds[j] = 1
    span = 2.0 ** I
    params = [(rng.standard_normal(n) * span * [0.7, 0.2, 0.02, 2.0 ** -F, 0.4, 1.5][j % 6]).astype(np.float32)
              for j, n in enumerate(numel)]
    ls = Lockstep(numel, kinds, fmt, params, fixed=True)
    packed = ls.check_state("compress-again", resync=False)
    ls.check_padding(packed)
    ls.check_decompress()
    ls.check_decompress(first=4, count=9)
    for r in range(3):
        grads = [(rng.standard_normal(n) * 0.3 * span).astype(np.float32) for n in numel]
        packed = ls.round(grads, [0.01, 1.0, 0.5][r], want_w=want_w)
        ls.check_padding(packed)
    ls.check_decompress()
    assert ls.sb_ulp_cases <= 3, ls.sb_ulp_cases


@WANT_W
@pytest.mark.parametrize("fmt", [(0, 7), (0, 15), (2, 3), (0, 23)], ids=lambda f: "I%dF%d" % f)
def test_special_values_fixed_point(fmt, want_w):
    """Every tie between neighbouring values with its FP32 neighbours, both ends of the range and
    beyond, zeros of both signs, FP32 subnormals, infinities (saturate) and NaNs (become 0), laid
    out as whole tiles (the kernels' full-granule path) and as a ragged variable."""
    I, F = fmt
    B = 1 + I + F
    step = 2.0 ** -F
    ks = np.arange(-2 ** (B - 1) - 3, 2 ** (B - 1) + 3, dtype=np.float64)
    if ks.size > 6000:
        ks = np.unique(np.concatenate([ks[:200], ks[-200:], ks[::max(1, ks.size // 5000)], np.arange(-100, 100)]))
    ties = ((ks + 0.5) * step).astype(np.float32)
    near = np.concatenate([ties, np.nextafter(ties, np.float32(9e9)), np.nextafter(ties, np.float32(-9e9)),
                           (ks * step).astype(np.float32)])
    specials = np.array([0.0, -0.0, 1e-45, -1e-45, 1e-30, -1e-30, np.inf, -np.inf, 3.4e38, -3.4e38, 2.0 ** I,
                         -(2.0 ** I), 2.0 ** I - step, 2.0 ** I - step / 2], np.float32)
    nans = np.array([0x7FC00000, 0xFFC00000, 0x7F800001, 0x7FFFFFFF], np.uint32).view(np.float32)
    rng = np.random.default_rng(4)
    vals = np.concatenate([near, specials, nans, (rng.standard_normal(3000) * 2.0 ** I * 0.5).astype(np.float32)])
    n = (vals.size + 4095) // 4096 * 4096
    vals = np.concatenate([vals, np.resize(ties, n - vals.size)])
    rng.shuffle(vals)
    finite = vals[np.isfinite(vals)][:5000]                       # a ragged variable with a finite fit
    params = [vals, finite, np.full(1500, 0.3 * 2.0 ** I, np.float32), np.zeros(130, np.float32),
              np.array([0.25 * 2.0 ** I], np.float32)]
    numel = [p.size for p in params]
    ls = Lockstep(numel, [0] * len(numel), fmt, params, fixed=True)
    ls.check_decompress()
    grads = [(rng.standard_normal(k) * 0.1 * 2.0 ** I).astype(np.float32) for k in numel]
    grads[1][:6] = [np.inf, -np.inf, np.nan, 1e38, -1e38, -0.0]
    ls.round(grads, 1.0, want_w=want_w)
    ls.check_decompress()
    ls.round([np.zeros(k, np.float32) for k in numel], 1.0, want_w=want_w)     # decode, then encode again
    ls.check_decompress()


def test_tiny_and_ragged_sets_in_q7():
    """The tiny set (one round, as its configuration states) and the 4096-variable ragged set (two
    rounds, every variable compared) in 8-bit fixed point.  The ragged set's scales reach down to
    1e-4, far below Q7's step of 1/128: most of its variables quantise to a handful of codes, or to
    a single one, which is what the per-variable transformation's degenerate case is for."""
    wl = workloads.tiny()
    ls = Lockstep(wl.numel, wl.kinds, (0, 7), wl.all_params(), fixed=True)
    ls.check_decompress()
    ls.check_padding(ls.round(wl.all_grads(0), wl.lr, want_w=False))
    ls.check_padding(ls.round(wl.all_grads(0), 10.0))
    ls.check_decompress()
    wl = workloads.ragged()
    params = wl.all_params()
    ls = Lockstep(wl.numel, wl.kinds, (0, 7), params, threads=8, fixed=True)
    del params
    for r in range(2):
        packed = ls.round(wl.all_grads(r), 0.01 if r == 0 else 20.0, want_w=False)
    ls.check_padding(packed)
    ls.check_decompress()
    assert ls.sb_ulp_cases <= 4, ls.sb_ulp_cases


@pytest.mark.parametrize("fmt", [(0, 11), (0, 15)], ids=lambda f: "I%dF%d" % f)
def test_conformer_like_100m_fixed_point(fmt):
    """The 100M set in 12- and 16-bit fixed point with a tenth of the matrices left in FP32, every
    variable compared, the launch a training loop makes."""
    wl = workloads.conformer_like()
    params = wl.all_params()
    ls = Lockstep(wl.numel, wl.kinds, fmt, params, fraction=0.9, seed=5, threads=8, fixed=True)
    del params
    for r in range(2):
        packed = ls.round(wl.all_grads(r), 30.0, want_w=False)
    ls.check_padding(packed)
    ls.check_decompress()
    assert ls.sb_ulp_cases <= 1, ls.sb_ulp_cases


@pytest.mark.parametrize("fmt", [(0, 7), (0, 15)], ids=lambda f: "I%dF%d" % f)
def test_transition_and_aggregate_fixed_point(fmt):
    rng = np.random.default_rng(12)
    numel = [5000, 1, 1024, 70000, 333, 2048, 12289, 4096, 100]
    kinds = [0, 0, 0, 0, 1, 0, 0, 0, 2]
    params = [(rng.standard_normal(n) * 0.3).astype(np.float32) for n in numel]
    ls = Lockstep(numel, kinds, fmt, params, fraction=0.5, seed=1, fixed=True)
    plan_to = omc.Plan(numel, kinds, fmt, fraction=0.7, seed=2, fixed=True)
    assert plan_to.quantised != ls.plan.quantised
    dm_to = DeviceModel(plan_to)
    a, b = ls.dm, dm_to
    st = torch.cuda.current_stream().cuda_stream
    omc.transition(ls.plan, plan_to, a.packed.data_ptr(), a.resid.data_ptr(), a.sb.data_ptr(),
                   b.packed.data_ptr(), b.resid.data_ptr(), b.sb.data_ptr(), b.ws.data_ptr(), st)
    ls.st = oracle_transition(ls.st, plan_to.quantised)
    ls.plan, ls.dm = plan_to, dm_to
    ls.check_padding(ls.check_state("transition"))
    ls.round([(rng.standard_normal(n) * 0.05).astype(np.float32) for n in numel], 0.5, want_w=False)
    # a floating-point plan of the same widths is another format: refused
    other = omc.Plan(numel, kinds, (5, 2) if fmt == (0, 7) else (5, 10))
    do = DeviceModel(other)
    assert omc.lib().omc_transition(other._h, plan_to._h, do.packed.data_ptr(), do.resid.data_ptr(), do.sb.data_ptr(),
                                    b.packed.data_ptr(), b.resid.data_ptr(), b.sb.data_ptr(), b.ws.data_ptr(), None) == -5
    # server-side mean of three clients
    clients = [ls]
    for k in (1, 2):
        pk = [p + np.float32(0.01 * k) for p in params]
        clients.append(Lockstep(numel, kinds, fmt, pk, fraction=0.6, seed=20 + k, fixed=True))
    out = torch.zeros(ls.plan.full_elems, dtype=torch.float32, device="cuda")
    omc.aggregate([c.plan for c in clients], [c.dm.packed.data_ptr() for c in clients],
                  [c.dm.resid.data_ptr() for c in clients], [c.dm.sb.data_ptr() for c in clients], out.data_ptr(), st)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    want = orc.aggregate([c.st for c in clients])
    for i in range(len(numel)):
        assert same_f32(from_full(ls.plan, got, i), want[i]), i


def test_fixed_point_format_limits_and_matmul_refusal():
    L = omc.lib()
    h = omc.C.c_void_p()
    d = (omc.VarDesc * 1)()
    d[0].numel, d[0].kind = 128 * 64, 0
    for I, F, ok in [(0, 7, True), (8, 15, True), (0, 23, True), (0, 0, False), (1, 23, False), (9, 3, False)]:
        rc = L.omc_plan(d, 1, omc.Format(1, I, F, omc.FORMAT_FIXED_POINT), 1.0, 0, None, omc.PLAN_DEFAULT, omc.C.byref(h))
        assert (rc == 0) == ok, (I, F, rc)
        if rc == 0:
            L.omc_plan_destroy(h)
    assert L.omc_plan(d, 1, omc.Format(1, 5, 2, 2), 1.0, 0, None, omc.PLAN_DEFAULT, omc.C.byref(h)) == -2   # unknown flag
    plan = omc.Plan([128 * 64], [0], (2, 9), fixed=True)        # omc_matmul decodes S1I0F7 / F11 / F15 only
    dm = DeviceModel(plan)
    x = torch.zeros(128 * 64, dtype=torch.float16, device="cuda")
    y = torch.zeros(128 * 128, dtype=torch.float32, device="cuda")
    assert L.omc_matmul(plan._h, 0, dm.packed.data_ptr(), dm.sb.data_ptr(), x.data_ptr(), 128, 128, 64, y.data_ptr(),
                        y.data_ptr(), None) == -2
