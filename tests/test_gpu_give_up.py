"""The give-up path of the bounded waits, run in the one form that cannot fault or hang:
omc_plan_inject_wait_timeout makes the next launch announce its asynchronous loads to their
barriers without issuing them, so every wait runs out after a few thousand polls with no copy in
flight; the kernel must set the plan's status word and return, the context must stay usable, and
after omc_plan_prepare the same plan must work bit-exactly again."""
import numpy as np
import pytest
import torch

import paper_2205_03494_b200 as omc
from oracle import omc_oracle as orc
from harness import DeviceModel
from test_gpu_parity import Lockstep

pytestmark = pytest.mark.gpu

NUMEL = [5000, 300, 4096, 70001, 64]
KINDS = [0, 1, 0, 0, 2]


def fresh(fmt, rng):
    params = [(rng.standard_normal(n) * 0.1).astype(np.float32) for n in NUMEL]
    return params, Lockstep(NUMEL, KINDS, fmt, params)


@pytest.mark.parametrize("fmt", [(5, 10), (5, 6), (5, 2), (3, 7)], ids=lambda f: "E%dM%d" % f)
@pytest.mark.parametrize("call", ["compress", "decompress", "update", "transition"])
def test_wait_runs_out_then_plan_works_again(call, fmt):
    rng = np.random.default_rng(17)
    params, ls = fresh(fmt, rng)
    dm, plan = ls.dm, ls.plan
    st = torch.cuda.current_stream().cuda_stream
    grads = [(rng.standard_normal(n) * 0.05).astype(np.float32) for n in NUMEL]
    assert plan.status(st) == 0
    plan.inject_wait_timeout(1 << 12)
    if call == "compress":
        dm.compress(dm.upload_full(params))
    elif call == "decompress":
        dm.decompress()
    elif call == "update":
        dm.update(dm.upload_full(grads), 0.5)
    else:
        other = omc.Plan(NUMEL, KINDS, fmt, mask=[0, 0, 1, 0, 0])
        do = DeviceModel(other)
        omc.transition(other, plan, do.packed.data_ptr(), do.resid.data_ptr(), do.sb.data_ptr(),
                       dm.packed.data_ptr(), dm.resid.data_ptr(), dm.sb.data_ptr(), dm.ws.data_ptr(), st)
    torch.cuda.synchronize()                       # the launch ends by itself
    assert plan.status(st) != 0                    # and says that it gave up
    dm.check_guards()
    # back to a usable state: prepare again, compress again, then a normal round against the oracle
    plan.prepare(dm.ws.data_ptr(), st)
    assert plan.status(st) == 0
    dm.compress(dm.upload_full(params))
    ls.check_state("compress after a give-up")
    ls.round(grads, 0.5, want_w=False)
    ls.check_decompress()


@pytest.mark.parametrize("fmt", [(5, 10), (5, 2), (3, 7)], ids=lambda f: "E%dM%d" % f)
def test_aggregate_wait_runs_out_then_works_again(fmt):
    """omc_aggregate streams the clients' codes through bounded waits of its own; the give-up is
    reported through the first plan's status word."""
    rng = np.random.default_rng(23)
    clients = []
    for k in range(3):
        params = [(rng.standard_normal(n) * 0.1).astype(np.float32) for n in NUMEL]
        clients.append(Lockstep(NUMEL, KINDS, fmt, params, fraction=0.7, seed=5 + k))
    plan0, dm0 = clients[0].plan, clients[0].dm
    st = torch.cuda.current_stream().cuda_stream
    out = dm0.full_buffer("mean")
    run = lambda: omc.aggregate([c.plan for c in clients], [c.dm.packed.data_ptr() for c in clients],
                                [c.dm.resid.data_ptr() for c in clients], [c.dm.sb.data_ptr() for c in clients],
                                out.data_ptr(), st)
    plan0.inject_wait_timeout(1 << 10)
    run()
    torch.cuda.synchronize()
    assert plan0.status(st) != 0
    for c in clients:
        c.dm.check_guards()
    plan0.prepare(dm0.ws.data_ptr(), st)
    assert plan0.status(st) == 0
    run()
    torch.cuda.synchronize()
    assert plan0.status(st) == 0
    dm0.check_guards()
    got = out.cpu().numpy()
    want = orc.aggregate([c.st for c in clients])
    for i in range(len(NUMEL)):
        o = plan0.full_off[i]
        assert np.array_equal(got[o:o + NUMEL[i]].view(np.uint32), want[i].view(np.uint32)), i


def test_matmul_wait_runs_out_then_works_again():
    rng = np.random.default_rng(3)
    N, K, M = 256, 128, 200
    w = (rng.standard_normal(N * K) * 0.05).astype(np.float32)
    x = (rng.standard_normal((M, K)) * 0.5).astype(np.float16)
    for fmt, fixed, M in [((5, 10), False, 200), ((5, 10), False, 300), ((5, 2), False, 200), ((0, 15), True, 200)]:
        # 300 rows of S1E5M10 take the kernel that pairs two SMs on a tile
        x = (rng.standard_normal((M, K)) * 0.5).astype(np.float16)
        plan = omc.Plan([N * K], [0], fmt, fixed=fixed)
        dm = DeviceModel(plan)
        dm.compress(dm.upload_full([w]))
        xd = torch.from_numpy(x).cuda()
        y = torch.zeros((M, N), dtype=torch.float32, device="cuda")
        scratch = torch.zeros(M, dtype=torch.float32, device="cuda")
        st = torch.cuda.current_stream().cuda_stream
        run = lambda: omc.matmul(plan, 0, dm.packed.data_ptr(), dm.sb.data_ptr(), xd.data_ptr(), M, N, K,
                                 y.data_ptr(), scratch.data_ptr(), st)
        plan.inject_wait_timeout(1 << 10)
        run()
        torch.cuda.synchronize()
        assert plan.status(st) != 0
        plan.prepare(dm.ws.data_ptr(), st)
        assert plan.status(st) == 0
        run()
        torch.cuda.synchronize()
        assert plan.status(st) == 0
        state = orc.compress([w], [True], *fmt, fixed=fixed)
        wbar = orc.decompress_var(state["packed"][0], N * K, fmt[0], fmt[1], state["s"][0], state["b"][0], fixed)
        want = x.astype(np.float64) @ wbar.reshape(N, K).astype(np.float64).T
        assert np.allclose(y.cpu().numpy(), want, rtol=1e-4, atol=1e-4)


def test_injection_argument_checks():
    plan = omc.Plan([100], [0], (5, 2))
    L = omc.lib()
    assert L.omc_plan_inject_wait_timeout(None, 10) == -3
    assert L.omc_plan_inject_wait_timeout(plan._h, 0) == -1
    assert L.omc_plan_inject_wait_timeout(plan._h, (1 << 24) + 1) == -1
