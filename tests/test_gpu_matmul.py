"""omc_matmul: the forward-path product computed straight from the codes (tensor cores) against
the definition: decompress the variable with the oracle, then Y = X Wbar^T in fp64 (numpy matmul).
Tolerance: X and the codes are exact FP16 inputs and their products are exact in FP32, so the only
errors are the FP32 accumulation over K in the tensor cores (at most one unit in the last place per
addition, i.e. K 2^-23 of sum |x||w|, if the accumulator truncates), the same for rowsum(X), the
rounding of Wbar = s*Wt + b in the definition and the epilogue's two roundings: the bound is
(4 K + 8) 2^-24 (|s| sum_k |x||wt| + |b| sum_k |x|), a factor two above that worst case."""
import numpy as np
import pytest
import torch

import paper_2205_03494_b200 as omc
from oracle import omc_oracle as orc
from harness import DeviceModel, Guarded

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("fmt", [(5, 10), (5, 6), (5, 2), (4, 3), (2, 3)], ids=lambda f: "E%dM%d" % f)
@pytest.mark.parametrize("M,N,K", [(128, 128, 64), (200, 256, 192), (1000, 384, 512), (64, 128, 1024),
                                   (4000, 4224, 192), (256, 256, 64), (300, 256, 1024)])
def test_matmul_from_codes_matches_definition(M, N, K, fmt):
    """The last shape has 32 x 17 = 544 tiles of 128 x 256 (M and N not multiples of the tile), so
    every persistent CTA walks over three or four tiles: both accumulators in tensor memory are
    reused, the producer runs ahead across tile boundaries, and the epilogue of one tile overlaps
    the products of the next.  From 256 rows and columns on the product runs on pairs of SMs; the last
    two shapes are its smallest (one tile, one K block) and one tile with more K blocks than stages."""
    rng = np.random.default_rng(M + N + K)
    numel = [777, N * K, 64, 128 * 64]
    kinds = [0, 0, 1, 0]
    scale = 1.0 if fmt == (2, 3) else 0.05          # S1E2M3 resolves nothing below 1/8 ...
    params = [np.clip(rng.standard_normal(n) * scale + 0.2 * scale, -3.5, 3.5).astype(np.float32)
              for n in numel]                        # ... and overflows from 3.875 on
    plan = omc.Plan(numel, kinds, fmt)
    dm = DeviceModel(plan)
    dm.compress(dm.upload_full(params))
    st = orc.compress(params, plan.quantised, *fmt)
    x = (rng.standard_normal((M, K)) * 0.5).astype(np.float16)
    xd = torch.from_numpy(x).cuda()
    yg = Guarded(M * N, torch.float32, "cuda", fill=float("nan"))
    y = yg.t[:M * N].view(M, N)
    scratch = torch.zeros(M, dtype=torch.float32, device="cuda")
    omc.matmul(plan, 1, dm.packed.data_ptr(), dm.sb.data_ptr(), xd.data_ptr(), M, N, K, y.data_ptr(),
               scratch.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert plan.status() == 0
    assert yg.intact()
    E_, M_ = fmt
    s_, b_ = float(st["s"][1]), float(st["b"][1])
    wbar = orc.decompress_var(st["packed"][1], N * K, E_, M_, st["s"][1], st["b"][1]).reshape(N, K).astype(np.float64)
    wt = orc.decode(orc.unpack(st["packed"][1], N * K, 1 + E_ + M_), E_, M_).reshape(N, K).astype(np.float64)
    x64 = x.astype(np.float64)
    want = x64 @ wbar.T
    bound = (4 * K + 8) * 2.0 ** -24 * (abs(s_) * (np.abs(x64) @ np.abs(wt).T)
                                        + abs(b_) * np.abs(x64).sum(1, keepdims=True)) + 1e-30
    got = y.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    assert np.all(np.abs(got - want) <= bound), float(np.max(np.abs(got - want) / bound))


@pytest.mark.parametrize("fmt", [(5, 7), (3, 7), (3, 9), (4, 8), (4, 14)], ids=lambda f: "E%dM%d" % f)
@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (200, 256, 384), (1000, 384, 512), (4000, 4224, 256)])
def test_matmul_from_odd_width_codes(M, N, K, fmt):
    """The 11- and 13-bit formats of Table 2 and Sec. 3.5.3: a K block of their codes starts 8
    bytes off the 16-byte grid every other time, the E = 3 and E = 4 formats are FP16 values only
    after a change of the exponent bias, and their subnormal codes are normal FP16 numbers.  S1E4M14
    (Table 1, 19 bits) has more significant bits than FP16: its weights go in as two FP16 terms and
    every K step makes two products.  Weights are scaled so that they reach from the format's
    subnormal range to near its largest value."""
    E_, M_ = fmt
    rng = np.random.default_rng(M + N + K + E_)
    top = 2.0 ** ((1 << (E_ - 1)) - 1) * (2 - 2.0 ** -M_)
    scale = min(0.2 * top, 2.0)
    w = (rng.standard_normal(N * K) * scale * 10.0 ** rng.uniform(-4, 0, N * K)).astype(np.float32)
    w = np.clip(w, -0.9 * top, 0.9 * top)
    numel, kinds = [333, N * K, 64], [0, 0, 1]
    params = [rng.standard_normal(333).astype(np.float32) * np.float32(0.1), w, np.zeros(64, np.float32)]
    plan = omc.Plan(numel, kinds, fmt)
    dm = DeviceModel(plan)
    dm.compress(dm.upload_full(params))
    st = orc.compress(params, plan.quantised, *fmt)
    x = (rng.standard_normal((M, K)) * 0.5).astype(np.float16)
    xd = torch.from_numpy(x).cuda()
    yg = Guarded(M * N, torch.float32, "cuda", fill=float("nan"))
    y = yg.t[:M * N].view(M, N)
    scratch = torch.zeros(M, dtype=torch.float32, device="cuda")
    omc.matmul(plan, 1, dm.packed.data_ptr(), dm.sb.data_ptr(), xd.data_ptr(), M, N, K, y.data_ptr(),
               scratch.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert plan.status() == 0 and yg.intact()
    s_, b_ = float(st["s"][1]), float(st["b"][1])
    wbar = orc.decompress_var(st["packed"][1], N * K, E_, M_, st["s"][1], st["b"][1]).reshape(N, K).astype(np.float64)
    wt = orc.decode(orc.unpack(st["packed"][1], N * K, 1 + E_ + M_), E_, M_).reshape(N, K).astype(np.float64)
    x64 = x.astype(np.float64)
    want = x64 @ wbar.T
    bound = (4 * K + 8) * 2.0 ** -24 * (abs(s_) * (np.abs(x64) @ np.abs(wt).T)
                                        + abs(b_) * np.abs(x64).sum(1, keepdims=True)) + 1e-30
    got = y.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    assert np.all(np.abs(got - want) <= bound), float(np.max(np.abs(got - want) / bound))
    # a row of 11- or 13-bit codes must be whole 16-byte units: K = 64 is refused before any launch
    if (N * K) % 64 == 0:
        assert omc.lib().omc_matmul(plan._h, 1, dm.packed.data_ptr(), dm.sb.data_ptr(), xd.data_ptr(), M, N * K // 64, 64,
                                    y.data_ptr(), scratch.data_ptr(), None) == -1


@pytest.mark.parametrize("fmt", [(0, 7), (0, 11), (0, 15)], ids=lambda f: "I%dF%d" % f)
@pytest.mark.parametrize("M,N,K", [(128, 128, 64), (200, 256, 192), (1000, 384, 512), (4000, 4224, 192)])
def test_matmul_from_fixed_point_codes(M, N, K, fmt):
    """The fixed-point variant (Sec. 2.2): two's-complement codes become FP16 values in the decoder
    warps without an integer conversion; S1I0F15 has more significant bits than FP16 and goes in as
    two terms.  The weights cover the whole range, both ends (the most negative code -1 and the
    largest value 1 - 2^-y, reached by saturation) and the smallest steps included."""
    I_, F_ = fmt
    rng = np.random.default_rng(M + N + K + F_)
    w = (rng.standard_normal(N * K) * 0.4 * 10.0 ** rng.uniform(-4, 0, N * K)).astype(np.float32)
    w[:64] = np.linspace(-1.5, 1.5, 64, dtype=np.float32)        # saturates at both ends
    w[64:72] = [-1.0, 1.0, 2.0 ** -F_, -(2.0 ** -F_), 0.0, -0.0, 1 - 2.0 ** -F_, 2.0 ** -(F_ + 2)]
    numel, kinds = [333, N * K, 64], [0, 0, 1]
    params = [rng.standard_normal(333).astype(np.float32) * np.float32(0.1), w, np.zeros(64, np.float32)]
    plan = omc.Plan(numel, kinds, fmt, fixed=True)
    dm = DeviceModel(plan)
    dm.compress(dm.upload_full(params))
    st = orc.compress(params, plan.quantised, I_, F_, fixed=True)
    x = (rng.standard_normal((M, K)) * 0.5).astype(np.float16)
    xd = torch.from_numpy(x).cuda()
    yg = Guarded(M * N, torch.float32, "cuda", fill=float("nan"))
    y = yg.t[:M * N].view(M, N)
    scratch = torch.zeros(M, dtype=torch.float32, device="cuda")
    omc.matmul(plan, 1, dm.packed.data_ptr(), dm.sb.data_ptr(), xd.data_ptr(), M, N, K, y.data_ptr(),
               scratch.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert plan.status() == 0 and yg.intact()
    s_, b_ = float(st["s"][1]), float(st["b"][1])
    wbar = orc.decompress_var(st["packed"][1], N * K, I_, F_, st["s"][1], st["b"][1], fixed=True).reshape(N, K).astype(np.float64)
    codes = orc.unpack(st["packed"][1], N * K, 1 + I_ + F_)
    wt = orc.decode(codes, I_, F_, fixed=True).reshape(N, K).astype(np.float64)
    assert wt.min() == -1.0 and wt.max() == 1 - 2.0 ** -F_          # both ends of the range are in the matrix
    x64 = x.astype(np.float64)
    want = x64 @ wbar.T
    bound = (4 * K + 8) * 2.0 ** -24 * (abs(s_) * (np.abs(x64) @ np.abs(wt).T)
                                        + abs(b_) * np.abs(x64).sum(1, keepdims=True)) + 1e-30
    got = y.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    assert np.all(np.abs(got - want) <= bound), float(np.max(np.abs(got - want) / bound))


def test_matmul_fixed_point_exact_small_case():
    """With s = 1, b = 0, one-hot rows of X and weights that are whole codes, every output is one
    weight exactly: the decoders' FP16 values are the codes' values bit for bit, for every code of
    the three formats."""
    for F_, (N, K, M) in [(f, shape) for f in (7, 11, 15) for shape in ((128, 512, 512), (256, 256, 256))]:
        # 128 rows of W: one SM per tile; 256 x 256: the kernel on pairs of SMs
        B = 1 + F_
        ks = (np.arange(N * K, dtype=np.int64) % (1 << B)) - (1 << (B - 1))     # every code (all 65536 of S1I0F15 once)
        w = (ks.astype(np.float64) * 2.0 ** -F_).astype(np.float32)
        plan = omc.Plan([N * K], [0], (0, F_), fixed=True, flags=omc.PLAN_WEIGHTS_ONLY)    # no transformation
        dm = DeviceModel(plan)
        dm.compress(dm.upload_full([w]))
        x = np.zeros((M, K), np.float16)
        assert M == K
        x[np.arange(M), np.arange(M)] = 1.0                                       # row m picks column m of W^T
        xd = torch.from_numpy(x).cuda()
        y = torch.zeros((M, N), dtype=torch.float32, device="cuda")
        scratch = torch.zeros(M, dtype=torch.float32, device="cuda")
        omc.matmul(plan, 0, dm.packed.data_ptr(), dm.sb.data_ptr(), xd.data_ptr(), M, N, K, y.data_ptr(),
                   scratch.data_ptr(), torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert plan.status() == 0
        want = w.reshape(N, K).T                                                   # y[m, n] = W[n, m]
        assert np.array_equal(y.cpu().numpy(), want), (F_, N)


@pytest.mark.parametrize("fmt,fixed", [((5, 10), False), ((5, 2), False), ((3, 7), False), ((4, 14), False),
                                       ((0, 11), True), ((0, 15), True)], ids=lambda v: str(v))
def test_matmul_repeated_launches_give_the_same_bits(fmt, fixed):
    """Ten launches in a row on pairs of SMs (several tiles per pair, ragged M and N): the same bits
    every time and a clean status word, i.e. no stage was read before it was ready."""
    rng = np.random.default_rng(5)
    M, N, K = 1000, 384, 512
    w = (rng.standard_normal(N * K) * 0.05).astype(np.float32)
    plan = omc.Plan([N * K], [0], fmt, fixed=fixed)
    dm = DeviceModel(plan)
    dm.compress(dm.upload_full([w]))
    xd = torch.from_numpy((rng.standard_normal((M, K)) * 0.5).astype(np.float16)).cuda()
    scratch = torch.zeros(M, dtype=torch.float32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    first = None
    for i in range(10):
        y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        omc.matmul(plan, 0, dm.packed.data_ptr(), dm.sb.data_ptr(), xd.data_ptr(), M, N, K, y.data_ptr(),
                   scratch.data_ptr(), st)
        torch.cuda.synchronize()
        assert plan.status(st) == 0 and not torch.isnan(y).any()
        if first is None:
            first = y
        else:
            assert torch.equal(first.view(torch.int32), y.view(torch.int32)), i


def test_matmul_argument_checks():
    plan = omc.Plan([128 * 64, 100], [0, 1], (5, 10))
    dm = DeviceModel(plan)
    p8 = omc.Plan([128 * 64], [0], (6, 5))
    d8 = DeviceModel(p8)
    x = torch.zeros(128 * 64, dtype=torch.float16, device="cuda")
    y = torch.zeros(128 * 128, dtype=torch.float32, device="cuda")
    L = omc.lib()
    a = (dm.packed.data_ptr(), dm.sb.data_ptr(), x.data_ptr())
    assert L.omc_matmul(plan._h, 1, *a, 128, 128, 64, y.data_ptr(), y.data_ptr(), None) == -1     # FP32 variable
    assert L.omc_matmul(plan._h, 0, *a, 128, 128, 32, y.data_ptr(), y.data_ptr(), None) == -1     # K % 64
    assert L.omc_matmul(plan._h, 0, *a, 128, 64, 128, y.data_ptr(), y.data_ptr(), None) == -1     # N % 128
    assert L.omc_matmul(plan._h, 0, *a, 128, 128, 128, y.data_ptr(), y.data_ptr(), None) == -1    # N*K != numel
    assert L.omc_matmul(p8._h, 0, d8.packed.data_ptr(), d8.sb.data_ptr(), x.data_ptr(), 128, 128, 64, y.data_ptr(),
                        y.data_ptr(), None) == -2
    assert L.omc_matmul(plan._h, 0, *a, 128, 128, 64, None, y.data_ptr(), None) == -3
    pf = omc.Plan([128 * 64], [0], (1, 6), fixed=True)          # a fixed-point format the product has no decoder for
    df = DeviceModel(pf)
    assert L.omc_matmul(pf._h, 0, df.packed.data_ptr(), df.sb.data_ptr(), x.data_ptr(), 128, 128, 64, y.data_ptr(),
                        y.data_ptr(), None) == -2
    torch.cuda.synchronize()


@pytest.mark.parametrize("size", [128, 384], ids=lambda n: "n%d" % n)
@pytest.mark.parametrize("fmt", [(4, 3), (2, 3), (3, 7), (4, 8), (3, 9), (4, 14)], ids=lambda f: "E%dM%d" % f)
def test_matmul_weights_at_the_top_of_the_range(fmt, size):
    """Weights that are infinite, NaN or the largest finite value of S1E4M3 / S1E2M3: the hardware
    narrow-float types have other values at those codes, so the decoder patches them.  A row of W
    with an infinity gives an infinite or NaN output column, a row with the largest finite value
    the exact product.  (128: the kernel with one SM per tile; 384: the one on pairs of SMs, the
    second CTA's rows included.)"""
    E, M = fmt
    N, K, Mr = size, 128, size
    top = 2.0 ** ((1 << (E - 1)) - 1) * (2 - 2.0 ** -M)
    w = np.full((N, K), 0.5 * top, np.float32)           # a value of the format in both cases
    w[3, 5] = np.inf
    w[7, 9] = -np.inf
    w[11, 0] = np.nan
    w[20, :] = top
    w[21, :] = -top
    w[N - 5, :] = top                                     # in the second CTA's half of a pair's tile
    w[N - 9, 17] = -np.inf
    plan = omc.Plan([N * K], [0], fmt, flags=omc.PLAN_WEIGHTS_ONLY)       # no transformation: s = 1, b = 0
    dm = DeviceModel(plan)
    dm.compress(dm.upload_full([w.reshape(-1)]))
    x = np.ones((Mr, K), np.float16)
    xd = torch.from_numpy(x).cuda()
    y = torch.zeros((Mr, N), dtype=torch.float32, device="cuda")
    scratch = torch.zeros(Mr, dtype=torch.float32, device="cuda")
    omc.matmul(plan, 0, dm.packed.data_ptr(), dm.sb.data_ptr(), xd.data_ptr(), Mr, N, K, y.data_ptr(),
               scratch.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    got = y.cpu().numpy()
    assert np.all(got[:, 3] == np.inf) and np.all(got[:, 7] == -np.inf) and np.all(np.isnan(got[:, 11]))
    assert np.all(got[:, 20] == np.float32(top * K)) and np.all(got[:, 21] == np.float32(-top * K))
    assert np.all(got[:, 0] == np.float32(0.5 * top * K))
    assert np.all(got[:, N - 5] == np.float32(top * K)) and np.all(got[:, N - 9] == -np.inf)

