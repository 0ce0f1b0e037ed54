"""The multi-rank (replica) bookkeeping of bench.py on CPU: two gloo ranks, the slowest rank's time
is what every rank ends up with, and the reported value counts all replicas' parameters."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _rank(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))
    dist.barrier()
    out[rank] = (ms, bench.replica_value(1000, world, ms))
    dist.destroy_process_group()


def test_two_gloo_ranks_report_slowest_time_and_whole_job_value():
    import socket
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    out = mp.Manager().dict()
    mp.spawn(_rank, args=(2, port, out), nprocs=2, join=True)
    assert out[0] == out[1] == (15.0, 2 * 1000 / 15e-3)


def test_single_rank_is_identity():
    import bench
    assert bench.max_over_ranks(3.5, None, None) == 3.5
    assert bench.replica_value(10, 1, 2.0) == 5000.0


def test_traffic_row_is_reported_only_for_the_sources_it_was_captured_with(tmp_path, monkeypatch):
    """roofline.traffic comes from profiles/dram_traffic.txt and goes back to null as soon as the
    kernel's sources differ from the ones the counters were taken with."""
    import bench
    prof = tmp_path / "profiles"
    prof.mkdir()
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    monkeypatch.setattr(bench, "kernel_source_hash", lambda: "abc123")
    (prof / "dram_traffic.txt").write_text("# comment\nsome_set 1000 abc123\nother_set 5 ffffff\n")
    assert bench.ncu_traffic("some_set") == 1000
    assert bench.ncu_traffic("other_set") is None          # captured with other sources
    assert bench.ncu_traffic("missing") is None
    (prof / "dram_traffic.txt").unlink()
    assert bench.ncu_traffic("some_set") is None


def test_algorithmic_bytes_rule():
    """4 + B/4 bytes per quantised parameter (code in, gradient in, code out) plus 16 per variable
    for (s, b) read and written; 12 per FP32 parameter."""
    import bench

    class P:
        numel, quantised, B = [1000, 64, 333], [True, False, True], 12
    assert bench.algorithmic_bytes(P) == (1000 * 4 + 2 * 1500 + 16) + 12 * 64 + (333 * 4 + 2 * 500 + 16)
