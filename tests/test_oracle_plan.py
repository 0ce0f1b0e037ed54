"""Pins for the oracle's selection rule (Sec. 2.4, 2.5, 3.1) and its size accounting, the latter
against the parameter-memory figures the paper prints (Tables 1 and 2, Sec. 3.4, Sec. 3.5.3)."""
import os

import numpy as np
import pytest

from oracle import omc_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rows(name):
    out = []
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            out.append([c.strip() for c in line.split("|")])
    return out


def model_with_share(weight_share, n_mats=1000, mat=4096):
    """n_mats equal weight matrices plus one FP32-only vector sized to give the stated share."""
    total_w = n_mats * mat
    other = round(total_w * (1 - weight_share) / weight_share) if weight_share < 1 else 0
    numel = [mat] * n_mats + ([other] if other else [])
    kinds = [orc.KIND_WEIGHT_MATRIX] * n_mats + ([orc.KIND_NORM] if other else [])
    return np.array(numel, np.uint64), np.array(kinds)


def test_splitmix64_published_vectors():
    want = [int(l, 16) for l in open(os.path.join(GOLDEN, "splitmix64_seed0.txt"))
            if l.strip() and not l.startswith("#")]
    assert [orc.splitmix64(0, i) for i in range(len(want))] == want


def test_selection_rule():
    kinds = np.array([0, 1, 0, 2, 0, 0, 3, 0, 0, 0, 1, 0, 0])   # 9 weight matrices
    for p, k in [(0.25, 2), (0.5, 5), (0.75, 7), (0.9, 8), (1.0, 9), (0.05, 0)]:
        sel = orc.select(kinds, p, seed=7)
        assert sel.sum() == k == int(np.floor(p * 9 + 0.5))
        assert not sel[kinds != 0].any()                        # weight matrices only (Sec. 2.4)
        assert np.array_equal(sel, orc.select(kinds, p, seed=7))
    # without the weights-only rule every variable is eligible
    assert orc.select(kinds, 1.0, 0, weights_only=False).all()
    # the subset varies with the seed (Sec. 3.1: from round to round, client to client)
    kinds = np.zeros(40, int)
    masks = {tuple(orc.select(kinds, 0.5, s)) for s in range(20)}
    assert len(masks) > 15
    # every matrix is picked about equally often
    hits = sum(orc.select(kinds, 0.5, s).astype(int) for s in range(2000))
    assert hits.min() > 850 and hits.max() < 1150


def test_selection_is_fisher_yates_prefix():
    """Independent restatement: descending Fisher-Yates on the ascending eligible indices driven by
    the published generator, first k taken."""
    kinds = np.array([0, 2, 0, 0, 1, 0, 0, 0, 3, 0, 0])
    elig = [i for i, k in enumerate(kinds) if k == 0]
    for seed in [0, 1, 12345]:
        perm = list(elig)
        draws = iter(orc.splitmix64(seed, i) for i in range(len(perm)))
        for i in range(len(perm) - 1, 0, -1):
            j = next(draws) % (i + 1)
            perm[i], perm[j] = perm[j], perm[i]
        for frac, k in [(0.5, 4), (0.125, 1), (0.9, 7)]:              # k = floor(frac*8 + 0.5)
            want = np.zeros(kinds.size, bool)
            want[perm[:k]] = True
            assert np.array_equal(orc.select(kinds, frac, seed), want)


@pytest.mark.parametrize("label,fp32_mb,omc_mb,bits,frac,share,src", rows("paper_sizes.txt"))
def test_sizes_reproduce_paper_tables(label, fp32_mb, omc_mb, bits, frac, share, src):
    numel, kinds = model_with_share(float(share))
    sel = orc.select(kinds, float(frac), seed=1)
    ratio = orc.model_bytes(numel, sel, int(bits)) / (4.0 * float(numel.sum()))
    assert abs(ratio * float(fp32_mb) - float(omc_mb)) <= 1.5, (label, ratio * float(fp32_mb))
    # and the closed form (1 - w p) + w p B / 32 (+ 8 bytes of (s, b) per matrix)
    w, p, B = float(share), float(frac), int(bits)
    closed = (1 - w * p) + w * p * B / 32
    assert abs(ratio - closed) < 1e-3


def test_ratios_stated_in_text():
    r = {k: (float(v), float(t)) for k, v, t, _ in rows("paper_ratios.txt")}
    numel, kinds = model_with_share(0.998)
    sel = orc.select(kinds, 0.9, seed=3)
    full = 4.0 * float(numel.sum())
    ratio11 = orc.model_bytes(numel, sel, 11) / full
    assert abs((1 - ratio11) - r["headline_reduction"][0]) <= r["headline_reduction"][1]
    assert abs(ratio11 - r["table2_ratio_11bit"][0]) <= r["table2_ratio_11bit"][1]
    ratio16 = orc.model_bytes(numel, sel, 16) / full
    assert abs((1 - ratio16) - r["pixel4_3block_reduction"][0]) <= r["pixel4_3block_reduction"][1]
    numel1, kinds1 = model_with_share(1.0)
    sel1 = orc.select(kinds1, 0.9, seed=3)
    ratio19 = orc.model_bytes(numel1, sel1, 19) / (4.0 * float(numel1.sum()))
    assert abs(ratio19 - r["table1_ratio"][0]) <= r["table1_ratio"][1]
    # average bit width with 90% of the parameters at 11 bits
    avg_bits = 32 * orc.model_bytes(numel1, sel1, 11) / (4.0 * float(numel1.sum()))
    assert abs((avg_bits - 11) - r["avg_bitwidth_increase"][0]) <= r["avg_bitwidth_increase"][1]


def test_model_bytes_exact():
    numel = np.array([10, 7, 100], np.uint64)
    assert orc.model_bytes(numel, [1, 0, 1], 12) == (15 + 8) + 28 + (150 + 8)
    assert orc.model_bytes(numel, [0, 0, 0], 12) == 4 * 117
    assert orc.model_bytes(numel, [1, 1, 1], 3) == (4 + 8) + (3 + 8) + (38 + 8)


def test_whole_model_state_round():
    rng = np.random.default_rng(0)
    variables = [rng.standard_normal(n).astype(np.float32) * 0.05 for n in (300, 20, 129)]
    grads = [rng.standard_normal(v.size).astype(np.float32) * 1e-3 for v in variables]
    st = orc.compress(variables, [True, False, True], 5, 2)
    dec = orc.decompress(st)
    assert np.array_equal(dec[1], variables[1])
    ws = orc.update_recompress(st, grads, 0.01, want_w=True, threads=2)
    assert np.array_equal(ws[1], orc.sgd_var(variables[1], grads[1], 0.01))
    p, s, b = orc.compress_var(ws[0], 5, 2)
    assert np.array_equal(st["packed"][0], p) and st["s"][0] == s and st["b"][0] == b


def test_plan_seed_is_the_kth_output_of_the_published_generator():
    """Seeds per (round, client), Sec. 3.1: output number round * 2^32 + client of the stream seeded
    with the job's seed.  For seed 0, round 0 these are the generator's published check values; for
    other arguments the oracle's direct jump must land where stepping through the stream arrives."""
    want = [int(l, 16) for l in open(os.path.join(GOLDEN, "splitmix64_seed0.txt"))
            if l.strip() and not l.startswith("#")]
    assert [orc.plan_seed(0, 0, c) for c in range(len(want))] == want
    for base in (0, 1, 0xDEADBEEF, 2 ** 64 - 1):
        for c in (0, 1, 7, 500, 1999):
            assert orc.plan_seed(base, 0, c) == orc.splitmix64(base, c)
    # a round is 2^32 outputs further on: the same as entering the stream of another seed
    gamma = 0x9E3779B97F4A7C15
    for base, rnd, c in [(5, 1, 0), (5, 3, 9), (123456789, 1000, 77)]:
        shifted = (base + ((rnd << 32) * gamma)) % 2 ** 64
        assert orc.plan_seed(base, rnd, c) == orc.splitmix64(shifted, c)
    # all different over a grid of rounds and clients, and the selections they give vary
    seeds = {orc.plan_seed(42, r, c) for r in range(50) for c in range(128)}
    assert len(seeds) == 50 * 128
    kinds = np.zeros(40, int)
    masks = {tuple(orc.select(kinds, 0.9, orc.plan_seed(42, r, c))) for r in range(4) for c in range(16)}
    assert len(masks) > 55
