"""Parity at the benchmark configurations' full sizes, in the launch configuration bench.py times
(whole-model plans, one kernel launch per call).  On the 100M and the ragged set every variable is
compared with the oracle; on the 1.6-billion-parameter set the oracle recomputes a sample of
variables completely (every code, (s, b) and W of those), the rest is covered by the status word
and the zero-padding check."""
import numpy as np
import pytest
import torch

import paper_2205_03494_b200 as omc
from paper_2205_03494_b200 import workloads
from test_gpu_parity import Lockstep

pytestmark = pytest.mark.gpu


def test_conformer_like_100m_three_rounds():
    """The bench workload, every variable compared in every round; the last round is the launch
    bench.py times (W not stored) with a step large enough to move most codes."""
    wl = workloads.conformer_like()
    params = wl.all_params()
    ls = Lockstep(wl.numel, wl.kinds, wl.fmt, params, threads=8)
    del params
    ls.check_decompress()
    for r in range(3):
        packed = ls.round(wl.all_grads(r), wl.lr if r < 2 else 30.0, want_w=(r < 2))
    ls.check_padding(packed)
    ls.check_decompress()
    assert ls.sb_ulp_cases <= 1, ls.sb_ulp_cases


@pytest.mark.parametrize("fmt,fraction", [((5, 6), 1.0), ((3, 7), 0.9), ((4, 14), 0.9), ((5, 2), 0.5)],
                         ids=lambda v: str(v).replace(" ", ""))
def test_conformer_like_100m_other_formats(fmt, fraction):
    """The 100M set in the formats of Tables 1-2 and with a share of the matrices left in FP32 (the
    launch that takes FP32 tiles from the queue), every variable compared, W not stored."""
    wl = workloads.conformer_like()
    params = wl.all_params()
    ls = Lockstep(wl.numel, wl.kinds, fmt, params, fraction=fraction, seed=5, threads=8)
    del params
    for r in range(2):
        packed = ls.round(wl.all_grads(r), 30.0, want_w=False)
    ls.check_padding(packed)
    ls.check_decompress()
    assert ls.sb_ulp_cases <= 1, ls.sb_ulp_cases


def test_ragged_4096_variables_two_rounds():
    """The ragged set, every one of its 4096 variables compared; the second round is the launch a
    training loop makes (W not stored) with a large step."""
    wl = workloads.ragged()
    params = wl.all_params()
    ls = Lockstep(wl.numel, wl.kinds, wl.fmt, params, threads=8)
    del params
    ls.check_decompress()
    for r in range(2):
        packed = ls.round(wl.all_grads(r), 0.01 if r == 0 else 20.0, want_w=(r == 0))
    ls.check_padding(packed)
    assert ls.sb_ulp_cases <= 4, ls.sb_ulp_cases


def test_large_transformer_1p6b_one_round():
    """32 layers at d = 2048, 12-bit codes: 1,610,612,736 parameters, one round."""
    free, _ = torch.cuda.mem_get_info()
    if free < 24e9:
        pytest.skip("needs about 24 GB of free device memory")
    wl = workloads.large_transformer()
    sample = list(range(0, 6)) + [95, 100] + list(range(186, 192))     # the first and the last layer whole, two in the middle
    params = wl.all_params()
    ls = Lockstep(wl.numel, wl.kinds, wl.fmt, params, sample=sample, threads=4)
    del params
    torch.cuda.empty_cache()
    packed = ls.round(wl.all_grads(0), 2.0, want_w=False)
    ls.check_padding(packed)
    assert ls.sb_ulp_cases <= 1, ls.sb_ulp_cases


@pytest.mark.parametrize("fmt", [(5, 10), (5, 2)], ids=lambda f: "E%dM%d" % f)
def test_conformer_like_100m_transition_between_90pct_subsets(fmt):
    """omc_transition at the size bench.py times it: the whole 100M set from one random 90 % of the
    matrices to another (its division of the work is made on the device by several thread blocks
    and has thousands of runs here), every variable against the oracle, then one more round."""
    from test_gpu_parity import oracle_transition
    wl = workloads.conformer_like()
    params = wl.all_params()
    ls = Lockstep(wl.numel, wl.kinds, fmt, params, fraction=0.9, seed=21, threads=8)
    del params
    plan_to = omc.Plan(wl.numel, wl.kinds, fmt, fraction=0.9, seed=22)
    changing = sum(a != b for a, b in zip(ls.plan.quantised, plan_to.quantised))
    assert changing >= 10
    from harness import DeviceModel
    dm_to = DeviceModel(plan_to)
    a, b = ls.dm, dm_to
    omc.transition(ls.plan, plan_to, a.packed.data_ptr(), a.resid.data_ptr(), a.sb.data_ptr(),
                   b.packed.data_ptr(), b.resid.data_ptr(), b.sb.data_ptr(), b.ws.data_ptr(),
                   torch.cuda.current_stream().cuda_stream)
    ls.st = oracle_transition(ls.st, plan_to.quantised)
    ls.plan, ls.dm = plan_to, dm_to
    packed = ls.check_state("transition")
    ls.check_padding(packed)
    ls.round(wl.all_grads(0), 5.0, want_w=False)
    assert ls.sb_ulp_cases <= 1, ls.sb_ulp_cases


@pytest.mark.parametrize("fmt,K", [((5, 10), 3), ((5, 6), 4), ((3, 7), 3)], ids=lambda v: str(v).replace(" ", ""))
def test_conformer_like_100m_aggregate(fmt, K):
    """omc_aggregate at the size bench.py times it: K clients of the 100M set, each with its own
    random 90 % of the matrices, every element of the mean against the oracle.  The launch has
    about a hundred tiles per warp here, so every warp walks over many tiles and across variable
    boundaries."""
    from oracle import omc_oracle as orc
    from harness import from_full, same_f32
    wl = workloads.conformer_like()
    base = wl.all_params()
    clients = []
    for k in range(K):
        rng = np.random.default_rng(500 + k)
        params = [p + np.float32(0.003 * (k + 1)) * rng.standard_normal(p.size, dtype=np.float32) for p in base]
        clients.append(Lockstep(wl.numel, wl.kinds, fmt, params, fraction=0.9, seed=40 + k, threads=8))
        del params
    assert len({tuple(c.plan.quantised) for c in clients}) == K
    out = torch.full((clients[0].plan.full_elems,), float("nan"), dtype=torch.float32, device="cuda")
    omc.aggregate([c.plan for c in clients], [c.dm.packed.data_ptr() for c in clients],
                  [c.dm.resid.data_ptr() for c in clients], [c.dm.sb.data_ptr() for c in clients],
                  out.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    want = orc.aggregate([c.st for c in clients], threads=8)
    for i in range(len(wl.numel)):
        assert same_f32(from_full(clients[0].plan, got, i), want[i]), i


@pytest.mark.parametrize("fmt", [(5, 2), (3, 7), (5, 10)], ids=lambda f: "E%dM%d" % f)
def test_one_variable_beyond_32_bit_indexing(fmt):
    """A single variable of 2^32 + 1,081,344 elements (8-, 11- and 16-bit codes, fit on): element and byte offsets
    no longer fit 32 bits.  The variable is one block of 2^20 + 264 values repeated 4096 times, so the
    oracle's answer for the block is the answer for the whole: the codes repeat, and the least-squares
    fit of a repeated sample is the fit of the sample (all sums and n scale by 4096 = 2^12, which the
    closed form cancels exactly; checked below on the CPU with 4 repeats).  Everything is compared on
    the device, every byte and every value."""
    from oracle import omc_oracle as orc
    from harness import ulp_diff
    free, _ = torch.cuda.mem_get_info()
    if free < 80e9:
        pytest.skip("needs about 70 GB of free device memory")
    (E, M), R, m = fmt, 4096, (1 << 20) + 264
    bb = m * (1 + E + M) // 8                 # bytes of one block's codes (m is a multiple of 8)
    n_big = R * m
    assert n_big > (1 << 32)
    rng = np.random.default_rng(2205)
    block = (rng.standard_normal(m) * 0.05).astype(np.float32)
    block[:8] = [0.0, -0.0, 1e-8, -3e-6, 6.1e-5, 0.4375, -3.5, 1e-45]
    gblock = (rng.standard_normal(m) * 1e-3).astype(np.float32)
    small = [(rng.standard_normal(k) * 0.05).astype(np.float32) for k in (1000, 77)]
    # oracle on the block (and the invariance it rests on)
    pk0, s0, b0 = orc.compress_var(block, E, M)
    pk4, s4, b4 = orc.compress_var(np.tile(block, 4), E, M)
    assert (s0, b0) == (s4, b4) and np.array_equal(np.tile(pk0[:bb], 4), pk4[:4 * bb])

    plan = omc.Plan([1000, n_big, 77], [0, 0, 1], (E, M))
    dev = torch.device("cuda:0")
    st = torch.cuda.current_stream().cuda_stream
    z = lambda k, dt: torch.zeros(max(int(k), 16), dtype=dt, device=dev)
    full = z(plan.full_elems, torch.float32)
    off = plan.full_off[1]
    blk_d = torch.from_numpy(block).to(dev)
    full[off:off + n_big].view(R, m).copy_(blk_d.unsqueeze(0).expand(R, m))
    full[plan.full_off[0]:plan.full_off[0] + 1000] = torch.from_numpy(small[0]).to(dev)
    full[plan.full_off[2]:plan.full_off[2] + 77] = torch.from_numpy(small[1]).to(dev)
    packed, resid = z(plan.packed_bytes, torch.uint8), z(plan.resid_elems, torch.float32)
    sb, ws = z(2 * plan.n_quantised, torch.float32), z(plan.workspace_bytes, torch.uint8)
    plan.prepare(ws.data_ptr(), st)
    plan.compress(full.data_ptr(), packed.data_ptr(), resid.data_ptr(), sb.data_ptr(), ws.data_ptr(), st)
    torch.cuda.synchronize()
    assert plan.status(st) == 0

    def check_codes(pk_block, s_want, b_want):
        po = plan.packed_off[1]
        want = torch.from_numpy(pk_block[:bb].copy()).to(dev)
        got = packed[po:po + R * bb].view(R, bb)
        assert bool((got == want.unsqueeze(0)).all())
        assert plan.var_packed_bytes[1] == R * bb          # a multiple of 16: no padding to check
        k = plan.sb_slot[1]
        s_got, b_got = np.float32(sb[2 * k].item()), np.float32(sb[2 * k + 1].item())
        assert ulp_diff(s_got, s_want) <= 1, (s_got, s_want)
        assert abs(float(b_got) - float(b_want)) <= 4 * n_big * 2.0 ** -53 * float(np.abs(block).mean()) + 2.0 ** -23 * abs(float(b_want))
        return s_got, b_got

    s_g, b_g = check_codes(pk0, s0, b0)
    # the small neighbours are untouched by the big one
    pk_s, s_s, b_s = orc.compress_var(small[0], E, M)
    assert np.array_equal(packed[plan.packed_off[0]:plan.packed_off[0] + pk_s.size].cpu().numpy(), pk_s)
    assert np.array_equal(resid[plan.resid_off[2]:plan.resid_off[2] + 77].cpu().numpy(), small[1])

    # decompress: the oracle's values for the block under the (s, b) the library stored
    del full
    out = z(plan.full_elems, torch.float32)
    plan.decompress(packed.data_ptr(), resid.data_ptr(), sb.data_ptr(), out.data_ptr(), 0, None, st)
    torch.cuda.synchronize()
    want = torch.from_numpy(orc.decompress_var(pk0, m, E, M, s_g, b_g)).to(dev)
    assert bool((out[off:off + n_big].view(R, m).view(torch.int32) == want.view(torch.int32).unsqueeze(0)).all())

    # one fused round with a repeated gradient block
    out.zero_()
    out[off:off + n_big].view(R, m).copy_(torch.from_numpy(gblock).to(dev).unsqueeze(0).expand(R, m))
    plan.update_recompress(packed.data_ptr(), resid.data_ptr(), sb.data_ptr(), out.data_ptr(), 2.0, ws.data_ptr(), None, st)
    torch.cuda.synchronize()
    assert plan.status(st) == 0
    pk1, s1, b1 = orc.update_recompress_var(pk0, m, E, M, s_g, b_g, gblock, 2.0)
    check_codes(pk1, s1, b1)
    assert not np.array_equal(pk1[:bb], pk0[:bb])
