"""GPU parity: the CUDA library (through its C-ABI) against the CPU oracle on the same seeded
inputs.  Packed codes (whole arena, zero padding included), decompressed values, the updated FP32
values W and the FP32 variables must be bit-exact.  (s, b) come from fp64 sums whose order the
paper does not fix: the oracle sums exactly, the GPU in a fixed order in fp64, so the two may
differ by one FP32 unit in the last place in rare near-midpoint cases; the tests allow that, count
it, and then continue from the oracle's (s, b) so that a difference cannot compound.  For nearly
lossless formats b is a difference of almost equal sums; there the bound is the summation error
itself, 4 n 2^-53 mean|V|, far below anything a stored value can show.
"""
import numpy as np
import pytest
import torch

import paper_2205_03494_b200 as omc
from paper_2205_03494_b200 import workloads
from oracle import omc_oracle as orc
from harness import DeviceModel, from_full, same_f32, to_full, ulp_diff

pytestmark = pytest.mark.gpu

ALL_FORMATS = [(5, 2), (4, 3), (5, 6), (5, 10), (4, 14), (3, 7), (2, 3), (3, 9), (4, 8), (5, 7), (8, 7),
               (8, 23),
               # no compiled specialisation: these take the run-time-format kernels
               (2, 0), (3, 2), (6, 5), (7, 22), (4, 23), (8, 10), (5, 3), (2, 23)]


class Lockstep:
    """Runs the oracle and the GPU side by side on a (sub)set of variables and compares."""

    def __init__(self, numel, kinds, fmt, params, *, fraction=1.0, seed=0, mask=None,
                 flags=omc.PLAN_DEFAULT, sample=None, threads=4, fixed=False):
        self.E, self.M = fmt
        self.fixed = fixed
        self.B = 1 + self.E + self.M
        self.plan = omc.Plan(numel, kinds, fmt, fraction=fraction, seed=seed, mask=mask, flags=flags, fixed=fixed)
        self.pvt = bool(flags & omc.PLAN_PVT)
        self.dm = DeviceModel(self.plan)
        self.idx = list(range(len(numel))) if sample is None else list(sample)
        self.threads = threads
        self.sb_ulp_cases = 0
        self.b_cancellation_cases = 0
        self.sb_checked = 0
        # initial compression on both sides
        full = self.dm.upload_full(params)
        self.dm.compress(full)
        del full
        sel = [self.plan.quantised[i] for i in self.idx]
        self.st = orc.compress([params[i] for i in self.idx], sel, self.E, self.M, self.pvt, threads, fixed=fixed)
        self.check_state("compress")

    def check_state(self, what, resync=True):
        packed, resid, sb = self.dm.host_state()
        fix = []
        for k, i in enumerate(self.idx):
            if self.plan.quantised[i]:
                got = self.dm.var_packed(packed, i)
                assert np.array_equal(got, self.st["packed"][k]), \
                    "%s: codes of variable %d differ at byte %s" % (
                        what, i, np.flatnonzero(got != self.st["packed"][k])[:5])
                s, b = self.dm.var_sb(sb, i)
                for name, g, w in (("s", s, self.st["s"][k]), ("b", b, self.st["b"][k])):
                    d = ulp_diff(g, w)
                    self.sb_checked += 1
                    if d > 1 and name == "b" and np.isfinite(g) and np.isfinite(w):
                        # b = (Sum V - s Sum Vt)/n cancels almost completely when the code is nearly
                        # lossless; what the fixed-order fp64 sums can differ by is then larger than
                        # an ulp of the tiny b: 4 n 2^-53 mean|V| bounds it (worst-case summation).
                        n = self.plan.numel[i]
                        scale = float(np.mean(np.abs(orc.decompress_var(
                            self.st["packed"][k], n, self.E, self.M, self.st["s"][k], self.st["b"][k], self.fixed))))
                        assert abs(float(g) - float(w)) <= 4 * n * 2.0 ** -53 * scale, (what, i, g, w, scale)
                        self.b_cancellation_cases += 1
                        fix.append((i, k))
                        continue
                    assert d <= 1, "%s: %s of variable %d: gpu %r oracle %r" % (what, name, i, g, w)
                    if d:
                        self.sb_ulp_cases += 1
                        fix.append((i, k))
            else:
                assert same_f32(self.dm.var_resid(resid, i), self.st["fp32"][k]), (what, i)
        if fix and resync:
            for i, k in fix:
                slot = self.plan.sb_slot[i]
                self.dm.sb[2 * slot] = float(self.st["s"][k])
                self.dm.sb[2 * slot + 1] = float(self.st["b"][k])
        return packed

    def check_padding(self, packed):
        """The bits after a variable's last code, up to its 16-byte boundary, are zero."""
        for i in range(self.plan.nvars):
            if self.plan.quantised[i]:
                arr = self.dm.var_packed(packed, i)
                nbits = self.plan.numel[i] * self.B
                assert arr.size % 16 == 0 and not arr[(nbits + 7) // 8:].any(), i
                if nbits % 8:
                    assert int(arr[nbits // 8]) >> (nbits % 8) == 0, i

    def check_decompress(self, first=0, count=None):
        out = self.dm.decompress(first, count)
        torch.cuda.synchronize()
        self.dm.check_guards()
        out = out.cpu().numpy()
        want = orc.decompress(self.st, self.threads)
        hi = self.plan.nvars if count is None else first + count
        for k, i in enumerate(self.idx):
            if first <= i < hi:
                assert same_f32(from_full(self.plan, out, i), want[k]), ("decompress", i)
        return out

    def round(self, grads, lr, want_w=True):
        """grads: list over all variables (GPU) -- the oracle takes the sampled ones."""
        gfull = self.dm.upload_full(grads)
        w_out = self.dm.full_buffer("W output") if want_w else None
        self.dm.update(gfull, lr, w_out)
        ws = orc.update_recompress(self.st, [grads[i] for i in self.idx], lr, self.threads, want_w=True)
        packed = self.check_state("update")
        if want_w:
            w_host = w_out.cpu().numpy()
            for k, i in enumerate(self.idx):
                assert same_f32(from_full(self.plan, w_host, i), ws[k]), ("W", i)
        return packed


# ---------------------------------------------------------------------------------------------

WANT_W = pytest.mark.parametrize("want_w", [True, False], ids=["w_out", "production"])


@WANT_W
@pytest.mark.parametrize("lr", [0.01, 10.0])
def test_tiny_set_one_round(lr, want_w):
    """Tiny set, 1/5/2, all four matrices: compress, decompress, one update round.  lr = 10 makes
    the step larger than the code spacing so that the re-encode path really changes codes.
    want_w = False is the launch a training loop makes (W is never stored); want_w = True the
    instantiation that also writes W, so that W itself is compared."""
    wl = workloads.tiny()
    params = wl.all_params()
    ls = Lockstep(wl.numel, wl.kinds, wl.fmt, params)
    before = ls.dm.packed.cpu().numpy().copy()
    ls.check_decompress()
    packed = ls.round(wl.all_grads(0), lr, want_w=want_w)
    ls.check_padding(packed)
    ls.check_decompress()
    changed = np.count_nonzero(before != packed[:before.size])
    if lr == 10.0:
        assert changed > before.size // 10
    assert ls.sb_ulp_cases <= 2


@pytest.mark.parametrize("wl", list(workloads.sweep()), ids=lambda w: "p%g-E%dM%d" % (w.fraction, *w.fmt))
def test_partial_quantisation_sweep(wl):
    """Quantised fraction x format sweep on the tiny set: parity, stored bytes against the closed
    form, and the quantisation error against the half-spacing bound."""
    params = wl.all_params()
    ls = Lockstep(wl.numel, wl.kinds, wl.fmt, params, fraction=wl.fraction, seed=wl.sel_seed)
    E, M = wl.fmt
    B = 1 + E + M
    sel = orc.select(wl.kinds, wl.fraction, wl.sel_seed)
    assert ls.plan.quantised == list(sel)
    assert ls.plan.closed_form_bytes == orc.model_bytes(wl.numel, sel, B)
    out = ls.check_decompress()
    # error of the plain code against the bound 2^(max(e, emin) - M - 1)
    emin = 2 - (1 << (E - 1))
    for i in range(len(params)):
        if not sel[i]:
            continue
        v = params[i].astype(np.float64)
        vt = orc.decode(orc.unpack(ls.dm.var_packed(ls.dm.packed.cpu().numpy(), i), v.size, B), E, M)
        nz = v != 0
        bound = np.exp2(np.maximum(np.floor(np.log2(np.abs(v[nz]))), emin) - M - 1)
        assert np.all(np.abs(vt[nz] - v[nz]) <= bound)
        # uniform-noise model: the error in units of the local spacing is spread evenly over
        # [-1/2, 1/2], so its RMS is 1/sqrt(12) (sanity check, 10 %)
        rms = float(np.sqrt(np.mean(((vt[nz] - v[nz]) / (2 * bound)) ** 2)))
        assert 0.9 / np.sqrt(12) <= rms <= 1.1 / np.sqrt(12), (i, rms)
        rec = from_full(ls.plan, out, i).astype(np.float64)
        assert np.linalg.norm(rec - v) <= np.linalg.norm(vt - v) * (1 + 1e-6)
    for r in range(3):      # the last round without the W output: the launch that takes FP32 tiles from the queue
        ls.round(wl.all_grads(r), 0.01 if r == 0 else 5.0, want_w=(r < 2))
    ls.check_decompress()


@WANT_W
@pytest.mark.parametrize("fmt", ALL_FORMATS, ids=lambda f: "E%dM%d" % f)
def test_ragged_small_all_formats(fmt, want_w):
    """Ragged list (sizes 1 .. a few tiles, not multiples of anything), mixed kinds, three rounds
    with a step large enough to move codes across binades and into the subnormal range."""
    rng = np.random.default_rng(fmt[0] * 100 + fmt[1])
    numel = [1, 2, 3, 5, 31, 32, 33, 127, 128, 129, 1023, 1024, 1025, 2047, 4096, 5000, 3 * 1024 + 7,
             777, 8, 16, 12289]
    kinds = [0] * len(numel)
    for j in (3, 9, 14):
        kinds[j] = 1
    E, M = fmt
    span = min(2.0 ** ((1 << (E - 1)) - 2), 4.0)
    params = []
    for j, n in enumerate(numel):
        scale = span * 10.0 ** (-(j % 6))
        params.append((rng.standard_normal(n) * scale).astype(np.float32))
    ls = Lockstep(numel, kinds, fmt, params)
    packed = ls.check_state("compress-again", resync=False)
    ls.check_padding(packed)
    ls.check_decompress()
    ls.check_decompress(first=4, count=9)
    for r in range(3):
        grads = [(rng.standard_normal(n) * 0.3 * span * 10.0 ** (-(j % 6))).astype(np.float32)
                 for j, n in enumerate(numel)]
        packed = ls.round(grads, [0.01, 1.0, 0.5][r], want_w=want_w)
        ls.check_padding(packed)
    ls.check_decompress()
    assert ls.sb_ulp_cases <= 3, ls.sb_ulp_cases


@pytest.mark.parametrize("fmt", [(5, 2), (5, 6), (5, 10), (4, 3), (3, 7), (8, 7), (2, 3), (6, 5), (8, 10), (3, 0)],
                         ids=lambda f: "E%dM%d" % f)
@WANT_W
def test_special_values(fmt, want_w):
    """Zeros of both signs, FP32 subnormals, ties, the overflow threshold, infinities and NaNs with
    payloads, a constant variable, a one-element variable."""
    E, M = fmt
    bias = (1 << (E - 1)) - 1
    emin, emax = 1 - bias, bias
    tiny = 2.0 ** (emin - M)
    top = 2.0 ** emax * (2 - 2.0 ** -M)
    thr = 2.0 ** emax * (2 - 2.0 ** -(M + 1))
    f32 = np.float32
    specials = np.array([0.0, -0.0, 1e-45, -1e-45, 1e-40, tiny, tiny / 2, -tiny / 2, 1.5 * tiny, 2.5 * tiny,
                         np.nextafter(f32(tiny / 2), f32(1)), 2.0 ** emin, np.nextafter(f32(2.0 ** emin), f32(0)),
                         1.0, 1 + 2.0 ** -(M + 1), 1 + 3 * 2.0 ** -(M + 1), np.nextafter(f32(2.0), f32(0)),
                         min(top, 3.4e38), min(thr, 3.4e38), np.nextafter(f32(min(thr, 3.4e38)), f32(0)),
                         -min(thr, 3.4e38), 3.4028235e38, -3.4028235e38, np.inf, -np.inf], np.float32)
    nans = np.array([0x7FC00000, 0xFFC00000, 0x7F800001, 0xFF800001, 0x7FFFFFFF, 0x7FA00000, 0x7F801000],
                    np.uint32).view(np.float32)
    rng = np.random.default_rng(5)
    body = (rng.standard_normal(3000) * 0.05).astype(np.float32)
    v_finite = np.concatenate([specials[:-4], body])           # no Inf/NaN: the fit stays finite
    v_inf = np.concatenate([specials, body[:100]])
    v_nan = np.concatenate([nans, body[:200]])
    v_const = np.full(1500, 0.3, np.float32)
    v_cell = np.linspace(0.26, 0.2600001, 700).astype(np.float32)       # one quantisation cell
    v_one = np.array([0.7], np.float32)
    v_zero = np.zeros(130, np.float32)
    v_pm0 = np.array([0.0, -0.0] * 40, np.float32)
    params = [v_finite, v_inf, v_nan, v_const, v_cell, v_one, v_zero, v_pm0, body]
    numel = [p.size for p in params]
    ls = Lockstep(numel, [0] * len(numel), fmt, params)
    ls.check_decompress()
    grads = [(rng.standard_normal(n) * 0.05).astype(np.float32) for n in numel]
    grads[0][:8] = [np.inf, -np.inf, np.nan, 1e38, -1e38, 0.0, -0.0, 1e-45]
    ls.round(grads, 1.0, want_w=want_w)
    ls.check_decompress()
    grads = [(rng.standard_normal(n) * 0.05).astype(np.float32) for n in numel]
    ls.round(grads, 0.5, want_w=want_w)
    ls.check_decompress()


@pytest.mark.parametrize("fmt", [(5, 2), (4, 3), (2, 3), (5, 6), (3, 7), (5, 10), (4, 8), (8, 7)],
                         ids=lambda f: "E%dM%d" % f)
@WANT_W
def test_rounding_boundaries_through_the_fast_path(fmt, want_w):
    """Every midpoint between neighbouring values of the format (up to 4096 of them, the lowest
    and the highest always included), each with its two FP32 neighbours and in both signs, and a
    log-uniform sweep from below the smallest subnormal to beyond the overflow threshold, laid out
    as variables of whole tiles so that the kernels take their full-granule path (hardware
    narrow-float and FP16 conversions where the format has them) and not the careful one.
    Compress and one update round (zero gradient: decode, then encode again) against the oracle."""
    E, M = fmt
    bias = (1 << (E - 1)) - 1
    emin, emax = 1 - bias, bias
    # finite magnitudes of the format, ascending: m * 2^(emin - M) for the subnormals, then the binades
    mags = [m * 2.0 ** (emin - M) for m in range(1 << M)]
    for e in range(emin, emax + 1):
        mags += [(1 + m / 2.0 ** M) * 2.0 ** e for m in range(1 << M)]
    mags = np.array(mags, np.float64)
    mids = 0.5 * (mags[:-1] + mags[1:])
    mids = np.append(mids, 2.0 ** emax * (2 - 2.0 ** -(M + 1)))      # the overflow threshold
    mids = mids[mids < 3.4e38]
    if mids.size > 4096:
        keep = np.unique(np.concatenate([np.arange(64), np.arange(mids.size - 64, mids.size),
                                         np.linspace(0, mids.size - 1, 3968).astype(np.int64)]))
        mids = mids[keep]
    m32 = mids.astype(np.float32)
    near = np.concatenate([m32, np.nextafter(m32, np.float32(0)), np.nextafter(m32, np.float32(np.inf))])
    rng = np.random.default_rng(E * 31 + M)
    lo, hi = np.log(max(2.0 ** (emin - M - 3), 1e-44)), np.log(min(2.0 ** (emax + 2), 3e38))
    sweep = np.exp(rng.uniform(lo, hi, 60000)).astype(np.float32) * rng.choice([-1.0, 1.0], 60000).astype(np.float32)
    vals = np.concatenate([near, -near, sweep])
    n = (vals.size + 4095) // 4096 * 4096                       # whole tiles, whatever the granule size
    vals = np.concatenate([vals, np.resize(m32, n - vals.size)])
    rng.shuffle(vals)
    in_range = vals[np.abs(vals) < 2.0 ** emax]                 # a second variable with no overflow: finite fit
    in_range = in_range[:in_range.size // 4096 * 4096]
    params = [vals, in_range]
    ls = Lockstep([p.size for p in params], [0, 0], fmt, params)
    ls.check_decompress()
    ls.round([np.zeros(p.size, np.float32) for p in params], 1.0, want_w=want_w)
    ls.check_decompress()


@pytest.mark.parametrize("fmt", [(5, 10), (5, 2), (3, 7)], ids=lambda f: "E%dM%d" % f)
def test_twenty_rounds_free_running(fmt):
    """The GPU and the oracle each run twenty rounds on their own, neither seeing the other's
    (s, b) in between; afterwards the decompressed models agree to 1e-6 relative.  A one-ulp
    difference in some (s, b) along the way (fp64 sums in another order, about once in 2^16
    fits) could flip a few codes in later rounds, so a 1e-5 share of the elements may differ."""
    wl = workloads.conformer_like(blocks=1)
    wl.fmt = fmt
    params = wl.all_params()
    plan = omc.Plan(wl.numel, wl.kinds, fmt)
    dm = DeviceModel(plan)
    dm.compress(dm.upload_full(params))
    st = orc.compress(params, plan.quantised, fmt[0], fmt[1], True, 8)
    for r in range(20):
        grads = wl.all_grads(r)
        dm.update(dm.upload_full(grads), 50.0)          # large steps: the codes keep moving
        orc.update_recompress(st, grads, 50.0, 8)
    got = dm.decompress().cpu().numpy()
    want = orc.decompress(st, 8)
    bad = total = 0
    for i in range(plan.nvars):
        g, w = from_full(plan, got, i), want[i]
        bad += int(np.count_nonzero(~np.isclose(g, w, rtol=1e-6, atol=0.0, equal_nan=True)))
        total += w.size
    assert bad <= 1e-5 * total, (bad, total)
    assert plan.status() == 0


def test_plan_switches():
    """Per-variable transformation off (s = 1, b = 0 stay put), weights-only off, explicit mask."""
    wl = workloads.tiny()
    params = wl.all_params()
    ls = Lockstep(wl.numel, wl.kinds, wl.fmt, params, flags=omc.PLAN_WEIGHTS_ONLY)
    _, _, sb = ls.dm.host_state()
    assert np.array_equal(sb[:8], np.array([1, 0] * 4, np.float32))
    ls.round(wl.all_grads(0), 10.0)
    ls.check_decompress()
    ls = Lockstep(wl.numel, wl.kinds, wl.fmt, params, flags=omc.PLAN_PVT)
    assert all(ls.plan.quantised)
    ls.round(wl.all_grads(0), 10.0)
    ls = Lockstep(wl.numel, wl.kinds, wl.fmt, params, mask=[1, 0, 0, 0, 0, 0, 1, 0])
    assert sum(ls.plan.quantised) == 2
    ls.round(wl.all_grads(0), 10.0)
    ls.check_decompress()


def test_repeatable_and_workspace_reuse():
    """Two runs from the same state give identical bytes; the workspace needs no clearing between
    calls; a second plan with its own workspace is independent."""
    wl = workloads.ragged(nvars=300, hi=30000)
    params = wl.all_params()
    plan = omc.Plan(wl.numel, wl.kinds, wl.fmt)
    outs = []
    for rep in range(2):
        dm = DeviceModel(plan)
        dm.compress(dm.upload_full(params))
        for r in range(3):
            dm.update(dm.upload_full(wl.all_grads(r)), 0.5)
        outs.append(dm.host_state())
    for a, b in zip(*outs):
        assert np.array_equal(a.view(np.uint8), b.view(np.uint8))


def test_device_call_argument_errors():
    wl = workloads.tiny()
    plan = omc.Plan(wl.numel, wl.kinds, wl.fmt)
    dm = DeviceModel(plan)
    L = omc.lib()
    h, ws, pk, rs, sb = plan._h, dm.ws.data_ptr(), dm.packed.data_ptr(), dm.resid.data_ptr(), dm.sb.data_ptr()
    full = torch.zeros(plan.full_elems, device="cuda")
    assert L.omc_compress(h, None, pk, rs, sb, ws, None) == -3
    assert L.omc_compress(h, full.data_ptr() + 4, pk, rs, sb, ws, None) == -4
    assert L.omc_decompress(h, pk, rs, sb, 0, 0, full.data_ptr(), None) == -1
    assert L.omc_decompress(h, pk, rs, sb, 7, 2, full.data_ptr(), None) == -1
    assert L.omc_decompress(h, pk, rs, sb, 0, 8, None, None) == -3
    assert L.omc_update_recompress(h, pk, rs, sb, None, 0.1, None, ws, None) == -3
    assert L.omc_update_recompress(h, pk + 8, rs, sb, full.data_ptr(), 0.1, None, ws, None) == -4
    assert L.omc_plan_prepare(h, None, None) == -3
    torch.cuda.synchronize()


def oracle_transition(st, sel_to):
    """The oracle's state under another selection, composed from its own operations: released
    variables are decompressed, newly selected ones compressed, the others kept."""
    E, M, pvt = st["E"], st["M"], st["pvt"]
    fixed = st.get("fixed", False)
    new = {"E": E, "M": M, "fixed": fixed, "pvt": pvt, "n": list(st["n"]), "sel": [bool(x) for x in sel_to],
           "packed": {}, "s": {}, "b": {}, "fp32": {}}
    for i, n in enumerate(st["n"]):
        was, now = st["sel"][i], bool(sel_to[i])
        if was and now:
            new["packed"][i], new["s"][i], new["b"][i] = st["packed"][i], st["s"][i], st["b"][i]
        elif not was and not now:
            new["fp32"][i] = st["fp32"][i]
        elif was:
            new["fp32"][i] = orc.decompress_var(st["packed"][i], n, E, M, st["s"][i], st["b"][i], fixed)
        else:
            new["packed"][i], new["s"][i], new["b"][i] = orc.compress_var(st["fp32"][i], E, M, pvt, fixed)
    return new


@pytest.mark.parametrize("fmt", [(5, 2), (5, 6), (5, 10), (4, 14), (3, 7)], ids=lambda f: "E%dM%d" % f)
def test_transition_between_selections(fmt):
    """Re-selection: a round under one random subset, then the state is carried to another subset
    (other seed, other fraction) and training continues there; every step against the oracle."""
    rng = np.random.default_rng(99)
    numel = [5000, 1, 1024, 70000, 333, 2048, 12289, 4096, 100, 9000, 513, 65536]
    kinds = [0, 0, 0, 0, 1, 0, 0, 0, 2, 0, 0, 0]
    params = [(rng.standard_normal(n) * 0.1).astype(np.float32) for n in numel]
    ls = Lockstep(numel, kinds, fmt, params, fraction=0.5, seed=1)
    ls.round([(rng.standard_normal(n) * 0.05).astype(np.float32) for n in numel], 1.0)
    for frac, seed in [(0.6, 2), (1.0, 3), (0.3, 4)]:
        plan_to = omc.Plan(numel, kinds, fmt, fraction=frac, seed=seed)
        assert plan_to.quantised != ls.plan.quantised
        dm_to = DeviceModel(plan_to)
        a, b = ls.dm, dm_to
        omc.transition(ls.plan, plan_to, a.packed.data_ptr(), a.resid.data_ptr(), a.sb.data_ptr(),
                       b.packed.data_ptr(), b.resid.data_ptr(), b.sb.data_ptr(), b.ws.data_ptr(),
                       torch.cuda.current_stream().cuda_stream)
        ls.st = oracle_transition(ls.st, plan_to.quantised)
        ls.plan, ls.dm = plan_to, dm_to
        packed = ls.check_state("transition")
        ls.check_padding(packed)
        ls.check_decompress()
        ls.round([(rng.standard_normal(n) * 0.05).astype(np.float32) for n in numel], 0.5)
        ls.round([(rng.standard_normal(n) * 0.05).astype(np.float32) for n in numel], 0.5, want_w=False)
    assert ls.sb_ulp_cases <= 2


@pytest.mark.parametrize("fmt", [(5, 10), (4, 3)], ids=lambda f: "E%dM%d" % f)
def test_transition_extreme_selections(fmt):
    """Selections at the ends: nothing quantised -> everything -> the same again -> nothing, and a
    model of one single-element variable.  The launch's own division of the work then has only
    copies, only conversions, or fewer tiles than one warp's share."""
    rng = np.random.default_rng(5)
    for numel in ([3000, 1, 1024, 70001, 2048, 12289, 64], [1]):
        kinds = [0] * len(numel)
        params = [(rng.standard_normal(n) * 0.1).astype(np.float32) for n in numel]
        none, every = [0] * len(numel), [1] * len(numel)
        ls = Lockstep(numel, kinds, fmt, params, mask=none)
        for mask in (every, every, none, none):
            plan_to = omc.Plan(numel, kinds, fmt, mask=mask)
            dm_to = DeviceModel(plan_to)
            a, b = ls.dm, dm_to
            omc.transition(ls.plan, plan_to, a.packed.data_ptr(), a.resid.data_ptr(), a.sb.data_ptr(),
                           b.packed.data_ptr(), b.resid.data_ptr(), b.sb.data_ptr(), b.ws.data_ptr(),
                           torch.cuda.current_stream().cuda_stream)
            ls.st = oracle_transition(ls.st, plan_to.quantised)
            ls.plan, ls.dm = plan_to, dm_to
            ls.check_padding(ls.check_state("transition"))
            ls.round([(rng.standard_normal(n) * 0.05).astype(np.float32) for n in numel], 0.5)
        assert ls.plan.status() == 0


def test_transition_refuses_mismatched_plans():
    a = omc.Plan([100, 200], [0, 0], (5, 2))
    b = omc.Plan([100, 201], [0, 0], (5, 2))
    c = omc.Plan([100, 200], [0, 0], (5, 6))
    da, db, dc = DeviceModel(a), DeviceModel(b), DeviceModel(c)
    args = lambda x, y: (x.packed.data_ptr(), x.resid.data_ptr(), x.sb.data_ptr(), y.packed.data_ptr(),
                         y.resid.data_ptr(), y.sb.data_ptr(), y.ws.data_ptr(), None)
    L = omc.lib()
    assert L.omc_transition(a._h, b._h, *args(da, db)) == -5
    assert L.omc_transition(a._h, c._h, *args(da, dc)) == -5
    never = omc.Plan([100, 200], [0, 0], (5, 2))
    assert L.omc_transition(a._h, never._h, *args(da, da)) == -5
    torch.cuda.synchronize()


@pytest.mark.parametrize("K", [5, 8, 16], ids=lambda k: "K%d" % k)
@pytest.mark.parametrize("fmt", [(5, 2), (4, 3), (2, 3), (5, 6), (5, 10), (3, 7), (5, 7), (4, 14), (8, 7), (8, 23)],
                         ids=lambda f: "E%dM%d" % f)
def test_aggregate_client_replicas(fmt, K):
    """Server-side mean of K clients that each quantised their own random subset (Sec. 2.5) against
    the oracle's aggregate (every client decompressed, FP32 mean in client order, one division)."""
    rng = np.random.default_rng(7)
    numel = [3000, 1, 1024, 5121, 333, 40000, 12289, 77]
    kinds = [0, 0, 0, 0, 1, 0, 0, 2]
    base = [(rng.standard_normal(n) * 0.1).astype(np.float32) for n in numel]
    clients = []
    for k in range(K):
        params = [(p + rng.standard_normal(p.size).astype(np.float32) * np.float32(0.01)) for p in base]
        if k == 2:
            params[0][:6] = [np.inf, -np.inf, np.nan, 1e30, -0.0, 1e-45]
        ls = Lockstep(numel, kinds, fmt, params, fraction=0.6, seed=10 + k)
        clients.append(ls)
    assert len({tuple(c.plan.quantised) for c in clients}) > 1
    out = torch.zeros(clients[0].plan.full_elems, dtype=torch.float32, device="cuda")
    omc.aggregate([c.plan for c in clients], [c.dm.packed.data_ptr() for c in clients],
                  [c.dm.resid.data_ptr() for c in clients], [c.dm.sb.data_ptr() for c in clients],
                  out.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    for c in clients:
        c.dm.check_guards()
    got = out.cpu().numpy()
    dec = [orc.decompress(c.st) for c in clients]
    want = orc.aggregate([c.st for c in clients])
    for i in range(len(numel)):
        assert same_f32(from_full(clients[0].plan, got, i), want[i]), i
    # one client alone: the mean is its decompressed model
    omc.aggregate([clients[1].plan], [clients[1].dm.packed.data_ptr()], [clients[1].dm.resid.data_ptr()],
                  [clients[1].dm.sb.data_ptr()], out.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    for i in range(len(numel)):
        assert same_f32(from_full(clients[1].plan, got, i), dec[1][i]), i
    L = omc.lib()
    assert L.omc_aggregate(None, 1, None, None, None, out.data_ptr(), None) == -3


@pytest.mark.parametrize("fmt", [(3, 7), (4, 14), (5, 7), (4, 3), (5, 6)], ids=lambda f: "E%dM%d" % f)
def test_aggregate_with_extreme_transformations(fmt):
    """(s, b) are data to the aggregation: whatever a client delivers, each value is
    fma(s, Vt, b).  Huge, tiny, negative and non-finite scales, written into the clients' (s, b)
    arrays on both sides, take the kernel off any path that pre-scales s."""
    rng = np.random.default_rng(41)
    numel = [2048, 700, 1024, 3333, 5000, 64, 1500]
    kinds = [0] * len(numel)
    odd = [(1e30, 0.5), (np.inf, 0.0), (np.nan, 1.0), (1e-42, -2.0), (-3.0e37, 1e38), (16.0, 0.0), (-0.0, -0.0)]
    clients = []
    for k in range(4):
        params = [(rng.standard_normal(n) * 0.1).astype(np.float32) for n in numel]
        c = Lockstep(numel, kinds, fmt, params, seed=70 + k)
        for i in range(len(numel)):
            if (i + k) % 2 == 0:
                sv, bv = odd[(i + 2 * k) % len(odd)]
                slot = c.plan.sb_slot[i]
                c.dm.sb[2 * slot], c.dm.sb[2 * slot + 1] = float(sv), float(bv)
                c.st["s"][i], c.st["b"][i] = np.float32(sv), np.float32(bv)
        clients.append(c)
    out = clients[0].dm.full_buffer("mean")
    omc.aggregate([c.plan for c in clients], [c.dm.packed.data_ptr() for c in clients],
                  [c.dm.resid.data_ptr() for c in clients], [c.dm.sb.data_ptr() for c in clients],
                  out.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    clients[0].dm.check_guards()
    got = out.cpu().numpy()
    want = orc.aggregate([c.st for c in clients])
    for i in range(len(numel)):
        assert same_f32(from_full(clients[0].plan, got, i), want[i]), i


@pytest.mark.parametrize("fmt", [(5, 10), (5, 2), (3, 7), (4, 14)], ids=lambda f: "E%dM%d" % f)
def test_aggregate_more_clients_than_one_call_takes(fmt):
    """Forty clients in batches of 16, 16 and 8 (omc_aggregate_sum, then omc_aggregate_add twice,
    then omc_divide): the same FP32 additions in the same order as one pass over all forty, so the
    result equals the oracle's mean over the forty bit for bit."""
    from paper_2205_03494_b200 import replicas
    rng = np.random.default_rng(57)
    numel = [3000, 1, 1024, 5121, 333, 20000, 77]
    kinds = [0, 0, 0, 0, 1, 0, 2]
    base = [(rng.standard_normal(n) * 0.1).astype(np.float32) for n in numel]
    clients = []
    for k in range(40):
        params = [(p + rng.standard_normal(p.size).astype(np.float32) * np.float32(0.01)) for p in base]
        if k == 21:
            params[0][:4] = [np.inf, np.nan, -0.0, 1e-45]
        clients.append(Lockstep(numel, kinds, fmt, params, fraction=0.6, seed=300 + k))
    st = torch.cuda.current_stream().cuda_stream
    plan0 = clients[0].plan
    args = lambda cs: ([c.plan for c in cs], [c.dm.packed.data_ptr() for c in cs], [c.dm.resid.data_ptr() for c in cs],
                       [c.dm.sb.data_ptr() for c in cs])
    out = clients[0].dm.full_buffer("running sum")
    out.fill_(123.0)                                  # the first batch must not read it
    omc.aggregate_sum(*args(clients[:16]), out.data_ptr(), st)
    omc.aggregate_add(*args(clients[16:32]), out.data_ptr(), st)
    omc.aggregate_add(*args(clients[32:]), out.data_ptr(), st)
    omc.divide(plan0, out.data_ptr(), 40, st)
    torch.cuda.synchronize()
    clients[0].dm.check_guards()
    got = out.cpu().numpy()
    want = orc.aggregate([c.st for c in clients])
    for i in range(len(numel)):
        assert same_f32(from_full(plan0, got, i), want[i]), i
    # the helper cuts any number of local clients into such batches
    out2 = torch.zeros(plan0.full_elems, dtype=torch.float32, device="cuda")
    k = replicas.mean_of_local_and_remote_clients(*args(clients), out2, st)
    torch.cuda.synchronize()
    assert k == 40 and torch.equal(out2.view(torch.int32), out.view(torch.int32))
    L = omc.lib()
    assert L.omc_aggregate_add(None, 1, None, None, None, out.data_ptr(), None) == -3


@pytest.mark.parametrize("fmt", [(5, 10), (5, 2), (3, 7)], ids=lambda f: "E%dM%d" % f)
def test_aggregate_in_two_stages(fmt):
    """The mean over clients held by several GPUs (omc_aggregate_sum per holder, the holders' sums
    added, omc_divide), with the collective's addition stood in for by one FP32 addition in holder
    order: bit-exact against the oracle's two-stage mean; one holder alone equals omc_aggregate."""
    from paper_2205_03494_b200 import replicas
    rng = np.random.default_rng(31)
    numel = [3000, 1, 1024, 5121, 333, 40000, 77]
    kinds = [0, 0, 0, 0, 1, 0, 2]
    base = [(rng.standard_normal(n) * 0.1).astype(np.float32) for n in numel]
    clients = []
    for k in range(7):
        params = [(p + rng.standard_normal(p.size).astype(np.float32) * np.float32(0.01)) for p in base]
        clients.append(Lockstep(numel, kinds, fmt, params, fraction=0.6, seed=50 + k))
    holders = [clients[:3], clients[3:5], clients[5:]]
    st = torch.cuda.current_stream().cuda_stream
    plan0 = clients[0].plan
    sums = []
    for h in holders:
        buf = clients[0].dm.full_buffer("partial sum %d" % len(sums))
        omc.aggregate_sum([c.plan for c in h], [c.dm.packed.data_ptr() for c in h], [c.dm.resid.data_ptr() for c in h],
                          [c.dm.sb.data_ptr() for c in h], buf.data_ptr(), st)
        sums.append(buf)
    total = sums[0].clone()
    for s in sums[1:]:
        total += s                                  # what the all-reduce does, here in holder order
    omc.divide(plan0, total.data_ptr(), 7, st)
    torch.cuda.synchronize()
    clients[0].dm.check_guards()
    got = total.cpu().numpy()
    want = orc.aggregate_two_stage([[c.st for c in h] for h in holders])
    for i in range(len(numel)):
        assert same_f32(from_full(plan0, got, i), want[i]), i
    # one process, no process group: the two library steps in a row are omc_aggregate
    out = torch.zeros(plan0.full_elems, dtype=torch.float32, device="cuda")
    k = replicas.mean_of_local_and_remote_clients([c.plan for c in clients], [c.dm.packed.data_ptr() for c in clients],
                                                  [c.dm.resid.data_ptr() for c in clients],
                                                  [c.dm.sb.data_ptr() for c in clients], out, st)
    ref = torch.zeros_like(out)
    omc.aggregate([c.plan for c in clients], [c.dm.packed.data_ptr() for c in clients],
                  [c.dm.resid.data_ptr() for c in clients], [c.dm.sb.data_ptr() for c in clients], ref.data_ptr(), st)
    torch.cuda.synchronize()
    assert k == 7 and torch.equal(out.view(torch.int32), ref.view(torch.int32))
    L = omc.lib()
    assert L.omc_divide(plan0._h, out.data_ptr(), 0, None) == -1
    assert L.omc_divide(plan0._h, None, 3, None) == -3
