"""Aggregation of clients spread over several ranks (Sec. 1, Sec. 2.5), bookkeeping on CPU: two
and three gloo ranks with unequal numbers of clients (one rank with none), the library's two GPU
steps replaced by the oracle's sum and division, the result against the oracle's two-stage mean
and, within the stated bound, against the plain mean over all clients."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

NUMEL = [300, 17, 1000, 64]
FMT = (5, 2)


def client_state(c):
    from oracle import omc_oracle as orc
    rng = np.random.default_rng(100 + c)
    params = [(rng.standard_normal(n) * 0.1).astype(np.float32) for n in NUMEL]
    sel = [bool((c + i) % 3) for i in range(len(NUMEL))]
    return orc.compress(params, sel, *FMT)


def clients_of(rank, world):
    table = {2: [[0, 1, 2], [3, 4]], 3: [[0, 1], [], [2, 3, 4]]}[world]
    return table[rank]


def _rank(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    from oracle import omc_oracle as orc
    from paper_2205_03494_b200 import replicas
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [client_state(c) for c in clients_of(rank, world)]
    total = sum(NUMEL)
    offs = np.concatenate([[0], np.cumsum(NUMEL)])

    def local_sum(t):
        t.zero_()
        if mine:
            dec = [orc.decompress(st) for st in mine]
            for i in range(len(NUMEL)):
                t[offs[i]:offs[i + 1]] = torch.from_numpy(orc.sum_var([d[i] for d in dec]))

    def divide(t, k):
        t.copy_(torch.from_numpy(orc.divide_var(t.numpy(), k)))

    buf = torch.empty(total, dtype=torch.float32)
    k_total = replicas.mean_across_ranks(buf, len(mine), local_sum, divide)
    out[rank] = (k_total, buf.numpy().copy())
    dist.barrier()
    dist.destroy_process_group()


def run(world):
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    out = mp.Manager().dict()
    mp.spawn(_rank, args=(world, port, out), nprocs=world, join=True)
    return out


def check(world):
    from oracle import omc_oracle as orc
    out = run(world)
    holders = [[client_state(c) for c in clients_of(r, world)] for r in range(world)]
    want = np.concatenate(orc.aggregate_two_stage(holders))
    plain = np.concatenate(orc.aggregate([st for h in holders for st in h]))
    k = sum(len(h) for h in holders)
    mags = np.zeros_like(want, dtype=np.float64)
    for h in holders:
        for st in h:
            mags += np.abs(np.concatenate(orc.decompress(st))).astype(np.float64)
    bound = (k - 1) * 2.0 ** -24 * mags / k + 2.0 ** -23 * np.abs(plain)
    for r in range(world):
        k_total, got = out[r]
        assert k_total == k == 5
        if world == 2:          # two addends commute: every rank holds exactly the oracle's two-stage mean
            assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
        assert np.all(np.abs(got.astype(np.float64) - plain.astype(np.float64)) <= bound)
    assert all(np.array_equal(out[0][1], out[r][1]) for r in range(world))   # one result on all ranks


def test_two_ranks_with_three_and_two_clients():
    check(2)


def test_three_ranks_one_without_clients():
    check(3)


def test_single_process_needs_no_group():
    from paper_2205_03494_b200 import replicas
    buf = torch.empty(8)
    k = replicas.mean_across_ranks(buf, 4, lambda t: t.fill_(8.0), lambda t, k: t.div_(k))
    assert k == 4 and bool((buf == 2.0).all())
