"""Host-only checks of libomc: the shared library loads and exports what include/omc.h declares,
omc_plan's selection, layouts and size accounting agree with the oracle and with the closed form,
and bad arguments come back as error codes.  No GPU needed."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import paper_2205_03494_b200 as omc
from paper_2205_03494_b200 import workloads
from oracle import omc_oracle as orc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "omc.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(omc_[a-z_]+)\s*\(", hdr))
    assert declared == set(omc.EXPORTS), declared ^ set(omc.EXPORTS)
    L = omc.lib()
    for name in declared:
        assert getattr(L, name) is not None
    assert L.omc_strerror(0) == b"ok" and b"format" in L.omc_strerror(-2)


def test_plan_selection_matches_oracle():
    for wl in [workloads.tiny(), workloads.conformer_like(blocks=2), workloads.ragged(nvars=50)]:
        for frac in (0.25, 0.5, 0.9, 1.0):
            for seed in (0, 5):
                p = omc.Plan(wl.numel, wl.kinds, wl.fmt, fraction=frac, seed=seed)
                want = orc.select(wl.kinds, frac, seed)
                assert p.quantised == list(want)
                B = 1 + wl.fmt[0] + wl.fmt[1]
                assert p.closed_form_bytes == orc.model_bytes(wl.numel, want, B)
    wl = workloads.conformer_like(blocks=1)
    p = omc.Plan(wl.numel, wl.kinds, wl.fmt, fraction=0.5, seed=1, flags=omc.PLAN_PVT)
    assert p.quantised == list(orc.select(wl.kinds, 0.5, 1, weights_only=False))


def test_plan_layout_rules():
    numel = [5, 1024, 1025, 3, 64, 1 << 20, 7]
    kinds = [0, 0, 1, 0, 2, 0, 0]
    for fmt in [(5, 2), (5, 6), (5, 10), (4, 14), (2, 3), (8, 23)]:
        B = 1 + sum(fmt)
        p = omc.Plan(numel, kinds, fmt, fraction=1.0)
        assert p.quantised == [k == 0 for k in kinds]
        full = resid = packed = 0
        slot = 0
        for i, n in enumerate(numel):
            assert p.full_off[i] == full and full % 4 == 0
            full += (n + 3) // 4 * 4
            if p.quantised[i]:
                assert p.packed_off[i] == packed and packed % 16 == 0
                assert p.var_packed_bytes[i] == orc.packed_bytes(n, B)
                packed += p.var_packed_bytes[i]
                assert p.sb_slot[i] == slot
                slot += 1
            else:
                assert p.resid_off[i] == resid
                resid += (n + 3) // 4 * 4
        assert (p.full_elems, p.resid_elems, p.packed_bytes, p.n_quantised) == (full, resid, packed, slot)
        assert p.workspace_bytes >= 256 and p.workspace_bytes % 256 == 0


def test_plan_mask_and_errors():
    numel, kinds = [10, 20, 30], [0, 1, 0]
    p = omc.Plan(numel, kinds, (5, 2), mask=[0, 0, 1])
    assert p.quantised == [False, False, True]
    with pytest.raises(omc.OmcError) as e:
        omc.Plan(numel, kinds, (5, 2), mask=[0, 1, 0])            # a bias is not eligible
    assert e.value.status == -1
    omc.Plan(numel, kinds, (5, 2), mask=[0, 1, 0], flags=omc.PLAN_PVT)   # eligible without the rule
    for bad_fmt in [(1, 5), (9, 3), (5, 24), (0, 5, 2), (2, 5, 2)]:
        with pytest.raises(omc.OmcError) as e:
            omc.Plan(numel, kinds, bad_fmt)
        assert e.value.status == -2
    for frac in (0.0, -0.5, 1.5, float("nan")):
        with pytest.raises(omc.OmcError) as e:
            omc.Plan(numel, kinds, (5, 2), fraction=frac)
        assert e.value.status == -1
    with pytest.raises(omc.OmcError):
        omc.Plan([10, 0], [0, 0], (5, 2))                         # empty variable
    with pytest.raises(omc.OmcError):
        omc.Plan([10], [7], (5, 2))                               # unknown kind
    with pytest.raises(omc.OmcError):
        omc.Plan([], [], (5, 2))
    with pytest.raises(omc.OmcError):
        omc.Plan(numel, kinds, (5, 2), flags=8)
    L = omc.lib()
    assert L.omc_plan(None, 1, omc.Format(1, 5, 2, 0), 1.0, 0, None, 3, None) == -3
    assert L.omc_plan_destroy(None) == -3
    assert L.omc_plan_sizes(None, None, None, None, None, None, None) == -3
    # device calls on a plan that was never prepared are refused before anything is launched
    assert L.omc_compress(p._h, 16, 16, 16, 16, 16, None) == -5
    assert L.omc_decompress(p._h, 16, 16, 16, 0, 1, 16, None) == -5
    assert L.omc_update_recompress(p._h, 16, 16, 16, 16, 0.1, None, 16, None) == -5
    assert L.omc_plan_var(p._h, 3, None, None, None, None, None, None) == -1


def test_sweep_sizes_against_closed_form():
    """Partial-quantisation sweep on the tiny set: stored bytes equal the closed form
    (1 - w p) + w p B / 32 up to the 8 bytes of (s, b) per matrix."""
    for wl in workloads.sweep():
        p = omc.Plan(wl.numel, wl.kinds, wl.fmt, fraction=wl.fraction, seed=wl.sel_seed)
        B = 1 + sum(wl.fmt)
        k = sum(p.quantised)
        assert k == int(np.floor(wl.fraction * 4 + 0.5))
        w = 4 * 65536 / wl.total
        pq = k / 4
        closed = ((1 - w * pq) + w * pq * B / 32) * 4 * wl.total + 8 * k
        assert abs(p.closed_form_bytes - closed) < 1e-6 * closed
        assert p.packed_bytes == k * 65536 * B // 8


def test_workload_shapes():
    wl = workloads.conformer_like()
    w = sum(n for n, k in zip(wl.numel, wl.kinds) if k == 0)
    assert w == 102_776_832 and sum(1 for k in wl.kinds if k == 0) == 187
    assert wl.total - w == 235_552 and abs(w / wl.total - 0.998) < 5e-4     # Sec. 2.4: 99.8%
    assert workloads.large_transformer().total == 1_610_612_736
    assert workloads.large_transformer(layers=20).total == 1_006_632_960
    assert workloads.tiny().total == 263_168
    r = workloads.ragged()
    assert len(r.numel) == 4096 and min(r.numel) >= 64 and max(r.numel) <= 1 << 20
    a, b = workloads.tiny().params(0), workloads.tiny().params(0)
    assert np.array_equal(a, b) and abs(a.std() - 0.05) < 2e-3
    g = workloads.tiny().grads(0, 1)
    assert not np.array_equal(g, workloads.tiny().grads(0, 0)) and abs(g.std() - 1e-3) < 1e-4


def test_division_of_the_tiles_into_runs():
    """Every tile belongs to exactly one run, runs are contiguous and in order, their number is a
    whole multiple of the warps launched, and no run is much longer than an equal share: at most
    the share plus three tiles for every quantised variable that starts inside it (what the plan
    charges a run for entering one)."""
    rag = workloads.ragged()
    conf = workloads.conformer_like()
    cases = [(rag.numel, rag.kinds, rag.fmt, 1.0), (conf.numel, conf.kinds, conf.fmt, 1.0),
             (conf.numel, conf.kinds, conf.fmt, 0.5), ([5, 1024, 1025, 3, 64, 7], [0, 0, 1, 0, 2, 0], (5, 2), 1.0),
             ([1], [0], (5, 10), 1.0), ([1 << 40], [0], (5, 2), 1.0), ([3] * 5000, [0] * 5000, (4, 3), 1.0)]
    for numel, kinds, fmt, frac in cases:
        p = omc.Plan(numel, kinds, fmt, fraction=frac)
        nwarps, ntiles, rs = p.division()
        tiles = [(n + 1023) // 1024 for n in numel]
        assert ntiles == sum(tiles)
        assert rs[0] == 0 and rs[-1] == ntiles and all(a <= b for a, b in zip(rs, rs[1:]))
        nruns = len(rs) - 1
        assert 1 <= nwarps <= ntiles and nruns % nwarps == 0 and nruns // nwarps <= 64
        if ntiles > 1 << 24:
            continue
        # tile index at which each variable starts, to count the variables a run enters
        starts = np.cumsum([0] + tiles[:-1])
        qstarts = np.array([t for t, q in zip(starts, p.quantised) if q])
        cost_share = (ntiles + 3 * len(qstarts)) / nruns
        for r in range(nruns):
            run = rs[r + 1] - rs[r]
            entered = int(np.searchsorted(qstarts, rs[r + 1]) - np.searchsorted(qstarts, rs[r]))
            assert run <= cost_share + 2, (r, run, cost_share)
            assert run + 3 * entered >= cost_share - 5, (r, run, entered, cost_share)


def test_plan_seed_matches_oracle_and_published_values():
    want = [int(l, 16) for l in open(os.path.join(os.path.dirname(__file__), "golden", "splitmix64_seed0.txt"))
            if l.strip() and not l.startswith("#")]
    assert [omc.plan_seed(0, 0, c) for c in range(len(want))] == want
    rng = np.random.default_rng(8)
    for _ in range(200):
        base = int(rng.integers(0, 2 ** 63)) * 2 + int(rng.integers(0, 2))
        r, c = int(rng.integers(0, 2 ** 32)), int(rng.integers(0, 2 ** 32))
        assert omc.plan_seed(base, r, c) == orc.plan_seed(base, r, c)
    # N client plans from one seed: the library's plans equal the oracle's selections
    wl = workloads.conformer_like(blocks=2)
    for client in range(4):
        seed = omc.plan_seed(77, 3, client)
        plan = omc.Plan(wl.numel, wl.kinds, (3, 7), fraction=0.9, seed=seed)
        assert plan.quantised == list(orc.select(wl.kinds, 0.9, orc.plan_seed(77, 3, client)))
