"""omc_compress_var_static: the entry point for callers that cannot allocate device memory (code
running inside another framework's memory pool, services with all buffers reserved up front,
plug-ins handed only their inputs and outputs).  Its scratch is a fixed array inside the library,
so the test checks what such a caller relies on: the output equals omc_compress's on a one-variable
plan, bit for bit (and the CPU oracle's: codes bit for bit, (s, b) within one FP32 unit in the
last place, the tolerance of every other parity test), on two calls in a row that share the array (different sizes and formats, so the
second call meets whatever the first one left), and oversize requests are refused untouched.
Collected last on purpose (file name), and self-contained so it also passes in a fresh process."""
import numpy as np
import pytest
import torch

import paper_2205_03494_b200 as omc
from oracle import omc_oracle as orc
from harness import ulp_diff

pytestmark = pytest.mark.gpu


def reference(values: torch.Tensor, fmt, flags, fixed=False):
    """omc_compress on a plan holding just this variable."""
    n = values.numel()
    plan = omc.Plan([n], [omc.KIND_WEIGHT_MATRIX], fmt, flags=flags | omc.PLAN_WEIGHTS_ONLY, fixed=fixed)
    dev = values.device
    packed = torch.zeros(plan.packed_bytes, dtype=torch.uint8, device=dev)
    resid = torch.zeros(16, dtype=torch.float32, device=dev)
    sb = torch.zeros(2, dtype=torch.float32, device=dev)
    ws = torch.zeros(plan.workspace_bytes, dtype=torch.uint8, device=dev)
    s = torch.cuda.current_stream().cuda_stream
    plan.prepare(ws.data_ptr(), s)
    plan.compress(values.data_ptr(), packed.data_ptr(), resid.data_ptr(), sb.data_ptr(), ws.data_ptr(), s)
    torch.cuda.synchronize()
    assert plan.status(s) == 0
    return packed.cpu().numpy(), sb.cpu().numpy()


def static_call(values: torch.Tensor, fmt, flags, fixed=False):
    n = values.numel()
    B = 1 + fmt[0] + fmt[1]
    nbytes = ((n * B + 7) // 8 + 15) // 16 * 16
    packed = torch.full((nbytes,), 0xAB, dtype=torch.uint8, device=values.device)   # must be overwritten
    sb = torch.full((2,), 7.0, dtype=torch.float32, device=values.device)
    omc.compress_var_static(values.data_ptr(), n, fmt, packed.data_ptr(), sb.data_ptr(), flags=flags,
                            stream=torch.cuda.current_stream().cuda_stream, fixed=fixed)
    torch.cuda.synchronize()
    assert omc.static_status(torch.cuda.current_stream().cuda_stream) == 0
    return packed.cpu().numpy(), sb.cpu().numpy()


def padded(n, gen, scale):
    """Device tensor with n values followed by zero padding up to a multiple of 4 floats."""
    t = torch.zeros((n + 3) // 4 * 4, dtype=torch.float32, device="cuda")
    t[:n] = torch.randn(n, generator=gen, device="cuda") * scale
    return t[:n]


def test_two_calls_in_a_row_match_omc_compress():
    gen = torch.Generator(device="cuda")
    gen.manual_seed(1234)
    calls = [(3_000_001, (5, 10), omc.PLAN_PVT, 0.05, False),      # many warps, ragged end
             (70_001, (5, 2), omc.PLAN_PVT, 0.3, False),           # fewer warps than the first call used
             (513, (5, 6), 0, 0.02, False),                        # no transformation: s = 1, b = 0
             (200_003, (0, 11), omc.PLAN_PVT, 0.3, True),          # the fixed-point variant
             (1, (4, 3), omc.PLAN_PVT, 1.0, False)]                # a single element
    for n, fmt, flags, scale, fixed in calls:
        v = padded(n, gen, scale)
        got_p, got_sb = static_call(v, fmt, flags, fixed)
        want_p, want_sb = reference(v, fmt, flags, fixed)
        assert np.array_equal(got_p, want_p), (n, fmt)
        assert np.array_equal(got_sb.view(np.uint32), want_sb.view(np.uint32)), (n, fmt, got_sb, want_sb)
        # and against the CPU oracle itself, so that a defect shared by both entry points shows
        orc_p, orc_s, orc_b = orc.compress_var(v.cpu().numpy(), fmt[0], fmt[1], bool(flags & omc.PLAN_PVT), fixed)
        assert np.array_equal(got_p, orc_p), (n, fmt)
        assert ulp_diff(got_sb[0], orc_s) <= 1 and ulp_diff(got_sb[1], orc_b) <= 1, (n, fmt, got_sb, orc_s, orc_b)
    # same input twice through the shared array: identical bytes
    v = padded(200_000, gen, 0.1)
    a = static_call(v, (5, 10), omc.PLAN_PVT)
    b = static_call(v, (5, 10), omc.PLAN_PVT)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1].view(np.uint32), b[1].view(np.uint32))


def test_refusals_touch_nothing():
    L = omc.lib()
    v = torch.zeros(1024, dtype=torch.float32, device="cuda")
    out = torch.full((4096,), 0xCD, dtype=torch.uint8, device="cuda")
    sb = torch.full((2,), 3.0, dtype=torch.float32, device="cuda")
    f = omc.Format(1, 5, 10, 0)
    args = (v.data_ptr(), out.data_ptr(), sb.data_ptr())
    assert L.omc_compress_var_static(args[0], omc.STATIC_MAX_NUMEL + 1, f, 1, args[1], args[2], None) == -8
    assert b"capacity" in L.omc_strerror(-8)
    assert L.omc_compress_var_static(args[0], 0, f, 1, args[1], args[2], None) == -1
    assert L.omc_compress_var_static(None, 16, f, 1, args[1], args[2], None) == -3
    assert L.omc_compress_var_static(args[0] + 4, 16, f, 1, args[1], args[2], None) == -4
    assert L.omc_compress_var_static(args[0], 16, omc.Format(1, 9, 3, 0), 1, args[1], args[2], None) == -2
    assert L.omc_compress_var_static(args[0], 16, f, 2, args[1], args[2], None) == -1
    torch.cuda.synchronize()
    assert bool((out == 0xCD).all()) and bool((sb == 3.0).all())
