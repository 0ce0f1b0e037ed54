#!/usr/bin/env python
"""Throughput of the OMC hot path on B200: one step = one round of the fused
decode -> SGD update -> re-encode over a whole synthetic parameter set (one kernel launch).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload conformer|large|large:<layers>|ragged|tiny]
    python bench.py --impl reference ...      # times the CPU oracle instead (rank 0 only)

Prints one JSON line.  Multi-GPU runs are independent replicas (the path has no exchange step):
every rank runs the same workload on its own GPU; the value is all ranks' parameters over the
slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "params/s, fused decode->update->re-encode"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

KERNEL_SOURCES = ("kernels.cuh", "codec.cuh", "omc_internal.h", "omc_api.cu", "omc_plan.cpp")


def kernel_source_hash() -> str:
    """Hash of the sources the fused kernel and its launch are built from."""
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2205_03494_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def ncu_traffic(workload_key: str):
    """DRAM bytes per launch of the fused kernel (dram__bytes_read.sum + dram__bytes_write.sum of
    one ncu capture), from profiles/dram_traffic.txt: lines of `workload-key bytes source-hash`.
    None when no capture exists for the workload or the kernel's sources changed since it was taken."""
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.txt")) as f:
            rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    except OSError:
        return None
    now = kernel_source_hash()
    for r in rows:
        if len(r) >= 3 and r[0] == workload_key and r[2] == now:
            return int(r[1])
    return None


def make_workload(name):
    from paper_2205_03494_b200 import workloads
    if name == "conformer":
        return workloads.conformer_like()
    if name == "large":
        return workloads.large_transformer()
    if name.startswith("large:"):            # e.g. large:20 = the 20-layer cut (1,006,632,960 params)
        return workloads.large_transformer(layers=int(name.split(":")[1]))
    if name == "ragged":
        return workloads.ragged()
    if name == "tiny":
        return workloads.tiny()
    raise SystemExit("unknown workload " + name)


def algorithmic_bytes(plan) -> int:
    """Bytes one fused round must move: code in + gradient in + code out per quantised parameter
    (4 + B/4), 12 per FP32 parameter, 16 for each variable's (s, b) read and written."""
    total = 0
    for i, n in enumerate(plan.numel):
        if plan.quantised[i]:
            total += n * 4 + 2 * ((n * plan.B + 7) // 8) + 16
        else:
            total += 12 * n
    return total


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            pass
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            c = [x.strip() for x in r.split(",")]
            if len(c) < 7:
                continue
            try:
                sm.append(float(c[0])); mx.append(float(c[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------

def cpu_oracle_rate(wl, threads, which, rounds=1):
    """Parameters per second of the CPU oracle's update-recompress on variables `which`."""
    from oracle import omc_oracle as orc
    from paper_2205_03494_b200 import workloads  # noqa: F401
    params = wl.all_params(which=which)
    grads = wl.all_grads(0, which=which)
    sel = orc.select(wl.kinds, wl.fraction, wl.sel_seed)
    st = orc.compress(params, [bool(sel[i]) for i in which], wl.fmt[0], wl.fmt[1], True, threads)
    n = sum(wl.numel[i] for i in which)
    t0 = time.perf_counter()
    for _ in range(rounds):
        orc.update_recompress(st, grads, wl.lr, threads)
    dt = time.perf_counter() - t0
    return n * rounds / dt, n, dt


def sample_vars(wl, budget_params):
    """Leading variables of the workload up to a parameter budget (at least one)."""
    which, tot = [], 0
    for i, n in enumerate(wl.numel):
        if which and tot + n > budget_params:
            break
        which.append(i)
        tot += n
    return which


def run_reference(args):
    """Reference arm: the CPU oracle as it stands, on the host cores, on a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2205_03494_b200.workloads import default_threads
    wl = make_workload(args.workload)
    threads = default_threads()
    which = sample_vars(wl, 12_500_000)
    from oracle import omc_oracle as orc
    params = wl.all_params(which=which)
    grads = wl.all_grads(0, which=which)
    sel = orc.select(wl.kinds, wl.fraction, wl.sel_seed)
    st = orc.compress(params, [bool(sel[i]) for i in which], wl.fmt[0], wl.fmt[1], True, threads)
    n = sum(wl.numel[i] for i in which)
    for _ in range(args.warmup):
        orc.update_recompress(st, grads, wl.lr, threads)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        orc.update_recompress(st, grads, wl.lr, threads)
    dt = time.perf_counter() - t0
    value = n * args.steps / dt
    sample = "first %d variables (%d params) of %s per step" % (len(which), n, wl.name)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "params/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": "%s S1E%dM%d p=%g" % (wl.name, wl.fmt[0], wl.fmt[1], wl.fraction),
                   "sample": sample},
        "cpu_baseline": {"value": value, "unit": "params/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "params/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def max_over_ranks(ms: float, dist, device) -> float:
    """The slowest rank's time: what a multi-rank (replica) run reports."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_value(nparams: int, world: int, ms_per_step: float) -> float:
    """Whole-job parameters per second of `world` independent replicas."""
    return world * nparams / (ms_per_step * 1e-3)


class FusedRun:
    """One workload resident on the device, ready for rounds of the fused update-recompress."""

    def __init__(self, wl, plan, dev, stream):
        import numpy as np
        import torch
        self.wl, self.plan, self.dev, self.stream = wl, plan, dev, stream
        z = lambda n, dt: torch.zeros(max(int(n), 16), dtype=dt, device=dev)
        self.packed, self.resid = z(plan.packed_bytes, torch.uint8), z(plan.resid_elems, torch.float32)
        self.sb, self.ws = z(2 * plan.n_quantised, torch.float32), z(plan.workspace_bytes, torch.uint8)
        plan.prepare(self.ws.data_ptr(), stream)
        params = self.upload(wl.params)
        plan.compress(params.data_ptr(), self.packed.data_ptr(), self.resid.data_ptr(), self.sb.data_ptr(),
                      self.ws.data_ptr(), stream)
        torch.cuda.synchronize()
        del params
        self.grads = self.upload(lambda i: wl.grads(i, 0))
        self.nparams = wl.total
        self.step_bytes = algorithmic_bytes(plan)

    def upload(self, make):
        """The seeded variables `make(i)`, generated on the host cores a few at a time and copied to
        their places in a device array in the plan's full layout (never the whole model on the host)."""
        import torch
        from concurrent.futures import ThreadPoolExecutor
        from paper_2205_03494_b200.workloads import default_threads
        plan = self.plan
        out = torch.zeros(plan.full_elems, dtype=torch.float32, device=self.dev)
        idx = list(range(plan.nvars))
        group = max(1, default_threads())
        with ThreadPoolExecutor(max_workers=group) as ex:
            for g0 in range(0, len(idx), 4 * group):
                chunk = idx[g0:g0 + 4 * group]
                for i, x in zip(chunk, ex.map(make, chunk)):
                    out[plan.full_off[i]:plan.full_off[i] + plan.numel[i]].copy_(torch.from_numpy(x))
        return out

    def step(self):
        self.plan.update_recompress(self.packed.data_ptr(), self.resid.data_ptr(), self.sb.data_ptr(),
                                    self.grads.data_ptr(), self.wl.lr, self.ws.data_ptr(), None, self.stream)

    def timed(self, steps):
        """Milliseconds for `steps` back-to-back rounds (CUDA events on the launching stream)."""
        import torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            self.step()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    def roofline(self, ms_per_step, traffic_key=None):
        peak, peak_kind = measured_peak()
        achieved = self.step_bytes / (ms_per_step * 1e6)       # GB/s
        return {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "frac_of_nominal_8tbs": achieved / NOMINAL_HBM_GBS,
                "peak_source": peak_kind + " copy bandwidth", "kernel": "omc_kernel<UPDATE>",
                "traffic": ncu_traffic(traffic_key) if traffic_key else None}

    def sustained(self, seconds, local, est_ms):
        """A run of at least `seconds` of back-to-back rounds with the clocks sampled: long enough for
        the power cap to act on the SM clock, which the short timed region never sees."""
        steps = max(10, int(seconds * 1e3 / est_ms) + 1)
        sampler = ClockSampler(local)
        sampler.start()
        time.sleep(0.25)
        ms = self.timed(steps)
        clocks = sampler.stop()
        per = ms / steps
        out = {"steps": steps, "seconds": ms * 1e-3, "ms_per_step": per, "params_per_s": self.nparams / (per * 1e-3),
               "roofline": self.roofline(per), "clocks": clocks}
        if clocks.get("sm_mhz"):
            out["ms_x_sm_ghz"] = per * clocks["sm_mhz"] * 1e-3       # time x clock: compares runs at different clocks
        return out


def config_label(wl, fixed=False):
    return "%s S1%s%d%s%d p=%g" % (wl.name, "I" if fixed else "E", wl.fmt[0], "F" if fixed else "M", wl.fmt[1], wl.fraction)


def bench_other_config(name, local, dev, stream, seconds):
    """A sub-record for one of the other target configurations: its own rounds as the configuration
    states them, the spread, and a sustained run, each with its roofline fraction."""
    import torch
    import paper_2205_03494_b200 as omc
    wl = make_workload(name)
    plan = omc.Plan(wl.numel, wl.kinds, wl.fmt, fraction=wl.fraction, seed=wl.sel_seed)
    run = FusedRun(wl, plan, dev, stream)
    for _ in range(3):
        run.step()
    rounds = max(wl.rounds, 10)
    chunks = sorted(run.timed(rounds) / rounds for _ in range(5))
    per = chunks[len(chunks) // 2]
    rec = {"config": config_label(wl), "params": run.nparams, "variables": plan.nvars,
           "bytes_per_step": run.step_bytes, "rounds_per_timing": rounds,
           "ms_per_step": per, "ms_per_step_spread": {"chunks": 5, "best": chunks[0], "median": per, "worst": chunks[-1]},
           "params_per_s": run.nparams / (per * 1e-3), "roofline": run.roofline(per),
           "sustained": run.sustained(seconds, local, per), "status": plan.status(stream)}
    del run
    torch.cuda.empty_cache()
    return rec


def run_ours(args):
    import numpy as np
    import torch
    import paper_2205_03494_b200 as omc
    from paper_2205_03494_b200.workloads import default_threads

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    wl = make_workload(args.workload)
    if args.format:
        wl.fmt = tuple(int(x) for x in args.format.split(","))
    if args.fraction:
        wl.fraction = args.fraction
    flags = (0 if args.no_pvt else omc.PLAN_PVT) | (0 if args.all_variables else omc.PLAN_WEIGHTS_ONLY)
    plan = omc.Plan(wl.numel, wl.kinds, wl.fmt, fraction=wl.fraction, seed=wl.sel_seed, flags=flags,
                    fixed=args.fixed)
    stream = torch.cuda.current_stream().cuda_stream
    run = FusedRun(wl, plan, dev, stream)
    packed, resid, sb, ws, grads = run.packed, run.resid, run.sb, run.ws, run.grads
    nparams, step_bytes = run.nparams, run.step_bytes
    step = run.step
    z = lambda n, dt: torch.zeros(max(int(n), 16), dtype=dt, device=dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()          # before the warm-up, so that a short timed region still has samples around it
    for _ in range(args.warmup):
        step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if rank == 0 else None
    ms = max_over_ranks(ms, dist, dev)
    ms_per_step = ms / args.steps

    # ---- spread of the same step: ten more chunks, each timed by its own pair of events
    chunk = max(1, args.steps // 10)
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(11)]
    evs[0].record()
    for c in range(10):
        for _ in range(chunk):
            step()
        evs[c + 1].record()
    torch.cuda.synchronize()
    chunk_ms = sorted(evs[c].elapsed_time(evs[c + 1]) / chunk for c in range(10))
    spread = {"chunks": 10, "steps_per_chunk": chunk, "best": chunk_ms[0], "median": 0.5 * (chunk_ms[4] + chunk_ms[5]),
              "worst": chunk_ms[-1]}

    # ---- the same step for two seconds and more, clocks sampled (rank 0 reports its own GPU)
    sustained = run.sustained(args.sustain, local, ms_per_step) if (rank == 0 and args.sustain > 0) else None

    # ---- end to end: gradients start in pinned host memory, (s, b) is read back, every step
    host_grads = torch.empty(plan.full_elems, dtype=torch.float32, pin_memory=True)
    host_grads.copy_(grads)
    host_sb = torch.zeros(max(2 * plan.n_quantised, 1), dtype=torch.float32, pin_memory=True)
    e2e_steps = max(3, min(args.steps, 10))

    def e2e_step():
        plan.update_recompress_host(packed.data_ptr(), resid.data_ptr(), sb.data_ptr(), host_grads.data_ptr(),
                                    wl.lr, grads.data_ptr(), host_sb.data_ptr(), ws.data_ptr(), stream)

    e2e_step()
    barrier()
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    e2e_ms = max_over_ranks(e2e_ms, dist, dev)
    del host_grads

    # ---- the two other kernels, for context (not part of the step)
    extra = {}
    if rank == 0 and not args.no_extra:
        out = torch.empty(plan.full_elems, dtype=torch.float32, device=dev)
        for name, fn, nbytes in (
            ("decompress", lambda: plan.decompress(packed.data_ptr(), resid.data_ptr(), sb.data_ptr(),
                                                   out.data_ptr(), 0, None, stream),
             sum((n * plan.B + 7) // 8 + 4 * n if q else 8 * n for n, q in zip(plan.numel, plan.quantised))),
            ("compress", lambda: plan.compress(out.data_ptr(), packed.data_ptr(), resid.data_ptr(), sb.data_ptr(),
                                               ws.data_ptr(), stream),
             sum((n * plan.B + 7) // 8 + 4 * n if q else 8 * n for n, q in zip(plan.numel, plan.quantised))),
        ):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            reps = 20
            e0.record()
            for _ in range(reps):
                fn()
            e1.record()
            torch.cuda.synchronize()
            t_ms = e0.elapsed_time(e1) / reps
            extra[name] = {"ms": t_ms, "params_per_s": nparams / (t_ms * 1e-3), "gbs": nbytes / (t_ms * 1e6)}

        # the forward path as Sec. 2.1 describes it: only the parameters the next layer needs are
        # decompressed, i.e. one call per group of consecutive variables (here 17 equal groups: the
        # Conformer-like set has 17 blocks of 32 variables) instead of one call for the model
        groups = 17 if plan.nvars >= 17 else 1
        bounds = [plan.nvars * g // groups for g in range(groups + 1)]

        def layerwise():
            for g in range(groups):
                plan.decompress(packed.data_ptr(), resid.data_ptr(), sb.data_ptr(), out.data_ptr(), bounds[g],
                                bounds[g + 1] - bounds[g], stream)

        for _ in range(3):
            layerwise()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(20):
            layerwise()
        e1.record()
        torch.cuda.synchronize()
        t_ms = e0.elapsed_time(e1) / 20
        extra["decompress_in_%d_calls" % groups] = {"ms": t_ms, "params_per_s": nparams / (t_ms * 1e-3),
                                                    "gbs": extra["decompress"]["gbs"] * extra["decompress"]["ms"] / t_ms}

        # re-selection between two random 90% subsets (Sec. 3.1), state A -> state B
        pa = omc.Plan(wl.numel, wl.kinds, wl.fmt, fraction=0.9, seed=1, fixed=args.fixed)
        pb = omc.Plan(wl.numel, wl.kinds, wl.fmt, fraction=0.9, seed=2, fixed=args.fixed)
        if pa.n_quantised and pa.quantised != pb.quantised:
            bufs = {}
            for nm, pl in (("a", pa), ("b", pb)):
                bufs[nm] = (z(pl.packed_bytes, torch.uint8), z(pl.resid_elems, torch.float32),
                            z(2 * pl.n_quantised, torch.float32), z(pl.workspace_bytes, torch.uint8))
                pl.prepare(bufs[nm][3].data_ptr(), stream)
            A, Bf = bufs["a"], bufs["b"]
            pa.compress(out.data_ptr(), A[0].data_ptr(), A[1].data_ptr(), A[2].data_ptr(), A[3].data_ptr(), stream)
            fn = lambda: omc.transition(pa, pb, A[0].data_ptr(), A[1].data_ptr(), A[2].data_ptr(), Bf[0].data_ptr(),
                                        Bf[1].data_ptr(), Bf[2].data_ptr(), Bf[3].data_ptr(), stream)
            nbytes = 0
            for n, qa, qb in zip(pa.numel, pa.quantised, pb.quantised):
                cb = (n * pa.B + 7) // 8
                nbytes += 2 * cb if (qa and qb) else 8 * n if not (qa or qb) else cb + 4 * n
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            e0.record()
            for _ in range(20):
                fn()
            e1.record()
            torch.cuda.synchronize()
            t_ms = e0.elapsed_time(e1) / 20
            extra["transition_90pct_to_90pct"] = {"ms": t_ms, "params_per_s": nparams / (t_ms * 1e-3),
                                                  "gbs": nbytes / (t_ms * 1e6),
                                                  "variables_changing": sum(a != b for a, b in zip(pa.quantised, pb.quantised))}

        # server-side mean of 8 client replicas, each with its own random 90% subset (Sec. 2.5)
        K = 8
        cl16 = []
        for k in range(16):
            pl = omc.Plan(wl.numel, wl.kinds, wl.fmt, fraction=0.9, seed=100 + k, fixed=args.fixed)
            b4 = (z(pl.packed_bytes, torch.uint8), z(pl.resid_elems, torch.float32),
                  z(2 * pl.n_quantised, torch.float32), z(pl.workspace_bytes, torch.uint8))
            pl.prepare(b4[3].data_ptr(), stream)
            pl.compress(out.data_ptr(), b4[0].data_ptr(), b4[1].data_ptr(), b4[2].data_ptr(), b4[3].data_ptr(), stream)
            cl16.append((pl, b4))
        cl = cl16[:K]
        mean = torch.empty(plan.full_elems, dtype=torch.float32, device=dev)
        try:
            fn = lambda: omc.aggregate([c[0] for c in cl], [c[1][0].data_ptr() for c in cl],
                                       [c[1][1].data_ptr() for c in cl], [c[1][2].data_ptr() for c in cl],
                                       mean.data_ptr(), stream)
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            e0.record()
            for _ in range(20):
                fn()
            e1.record()
            torch.cuda.synchronize()
            t_ms = e0.elapsed_time(e1) / 20
            nbytes = 4 * nparams + sum(((n * pl.B + 7) // 8) if q else 4 * n
                                       for pl, _ in cl for n, q in zip(pl.numel, pl.quantised))
            extra["aggregate_8_clients"] = {"ms": t_ms, "params_per_s": nparams / (t_ms * 1e-3),
                                            "gbs": nbytes / (t_ms * 1e6)}
            # the paper's round (Sec. 3.1: 128 clients), more than one call takes: eight batches of 16
            # (omc_aggregate_sum, seven times omc_aggregate_add, omc_divide); sixteen different
            # states, the same sixteen in every batch (3.6 GB a batch: nothing of it is left in the
            # L2 when the next batch reads it)
            lists = lambda cs: ([c[0] for c in cs], [c[1][0].data_ptr() for c in cs], [c[1][1].data_ptr() for c in cs],
                                [c[1][2].data_ptr() for c in cs])
            batches = [lists(cl16) for _ in range(8)]

            def fn128():
                omc.aggregate_sum(*batches[0], mean.data_ptr(), stream)
                for bt in batches[1:]:
                    omc.aggregate_add(*bt, mean.data_ptr(), stream)
                omc.divide(cl[0][0], mean.data_ptr(), 128, stream)
            for _ in range(2):
                fn128()
            torch.cuda.synchronize()
            e0.record()
            for _ in range(5):
                fn128()
            e1.record()
            torch.cuda.synchronize()
            t_ms = e0.elapsed_time(e1) / 5
            # the clients' bytes; `out` written once, then read and written by each further batch and by the division
            per_client = sum(((n * pl.B + 7) // 8) if q else 4 * n
                             for pl, _ in cl16 for n, q in zip(pl.numel, pl.quantised))
            nbytes128 = 8 * per_client + (4 + 8 * 8) * nparams
            extra["aggregate_128_clients_in_8_calls"] = {"ms": t_ms, "params_per_s": nparams / (t_ms * 1e-3),
                                                         "gbs": nbytes128 / (t_ms * 1e6)}
        except omc.OmcError as err:
            extra["aggregate_8_clients"] = {"unavailable": str(err)}

        # forward path fused into a GEMM (tensor cores): a 2048 x 8192 feed-forward matrix, 8192 tokens
        Mm, Nm, Km = 8192, 8192, 2048
        wsrc = torch.randn(Nm * Km, device=dev) * 0.02
        xh = (torch.randn(Mm, Km, device=dev) * 0.5).half()
        yo = torch.empty(Mm, Nm, dtype=torch.float32, device=dev)
        rs = torch.empty(Mm, dtype=torch.float32, device=dev)
        for mfmt in ((5, 10), (5, 6), (5, 2), (4, 3), (2, 3), (5, 7), (3, 7), (3, 9), (4, 8), (4, 14),
                     (0, 7, "fixed"), (0, 11, "fixed"), (0, 15, "fixed")):
            mfixed = len(mfmt) == 3
            mfmt = mfmt[:2]
            key = "matmul_from_codes_8192x8192x2048_" + ("S1I%dF%d" if mfixed else "S1E%dM%d") % mfmt
            try:
                pm = omc.Plan([Nm * Km], [0], mfmt, fixed=mfixed)
                bm = (z(pm.packed_bytes, torch.uint8), z(16, torch.float32), z(2, torch.float32),
                      z(pm.workspace_bytes, torch.uint8))
                pm.prepare(bm[3].data_ptr(), stream)
                wfmt = wsrc * 25.0 if mfmt == (2, 3) and not mfixed else wsrc       # S1E2M3 resolves nothing below 1/8
                pm.compress(wfmt.data_ptr(), bm[0].data_ptr(), bm[1].data_ptr(), bm[2].data_ptr(), bm[3].data_ptr(), stream)
                torch.cuda.synchronize()
                del wfmt
                fn = lambda: omc.matmul(pm, 0, bm[0].data_ptr(), bm[2].data_ptr(), xh.data_ptr(), Mm, Nm, Km,
                                        yo.data_ptr(), rs.data_ptr(), stream)
                for _ in range(3):
                    fn()
                torch.cuda.synchronize()
                e0.record()
                for _ in range(10):
                    fn()
                e1.record()
                torch.cuda.synchronize()
                t_ms = e0.elapsed_time(e1) / 10
                extra[key] = {"ms": t_ms, "tflops": 2.0 * Mm * Nm * Km / (t_ms * 1e9), "status": pm.status(stream)}
            except omc.OmcError as err:
                extra[key] = {"unavailable": str(err)}
        del wsrc, xh, yo

    # ---- the other target configurations as sub-records (default workload, one GPU only)
    other_configs = []
    if rank == 0 and world == 1 and args.workload == "conformer" and not args.no_other_configs and \
            not (args.format or args.fixed or args.fraction or args.no_pvt or args.all_variables):
        del packed, resid, sb, ws, grads
        run.packed = run.resid = run.sb = run.ws = run.grads = None
        torch.cuda.empty_cache()
        for name in ("large", "ragged"):
            try:
                other_configs.append(bench_other_config(name, local, dev, stream, args.sustain or 2.0))
            except (RuntimeError, MemoryError) as err:      # e.g. a GPU with less free memory than the set needs
                other_configs.append({"config": name, "unavailable": str(err).splitlines()[0][:200]})

    if dist is not None:
        dist.barrier()
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    achieved = step_bytes / (ms_per_step * 1e6)       # GB/s
    threads = default_threads()
    cpu = None
    if world == 1 and not args.no_cpu:
        which = list(range(len(wl.numel))) if wl.total <= 120_000_000 else sample_vars(wl, 100_000_000)
        rate, n_s, dt = cpu_oracle_rate(wl, threads, which)
        cpu = {"value": rate, "unit": "params/s", "cores": threads, "kind": "oracle",
               "sample": "1 round over %d variables (%d params) of %s, %.1f s wall" % (len(which), n_s, wl.name, dt)}
        which1 = sample_vars(wl, 20_000_000)
        rate1, n1, dt1 = cpu_oracle_rate(wl, 1, which1)
        cpu["single_thread"] = {"value": rate1, "unit": "params/s", "cores": 1,
                                "sample": "1 round over %d variables (%d params), %.1f s wall" % (len(which1), n1, dt1)}
    line = {
        "metric": METRIC, "value": replica_value(nparams, world, ms_per_step), "unit": "params/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "ms_per_step_spread": spread,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": config_label(wl, args.fixed),
                   "params": nparams, "variables": plan.nvars, "quantised_variables": plan.n_quantised,
                   "bytes_per_step": step_bytes, "lr": wl.lr, "pvt": not args.no_pvt, "weights_only": not args.all_variables, "gradients": "one seeded buffer reused every step",
                   "l2": ("inputs per step (%.0f MB) exceed the 126 MB L2; no flush" % (step_bytes / 1e6)
                          if step_bytes > 126e6 else
                          "inputs per step (%.1f MB) fit the 126 MB L2 and are not flushed: a latency figure, "
                          "not a bandwidth one" % (step_bytes / 1e6)),
                   "multi_gpu": "replicas only"},
        "hbm_gbs": achieved, "pct_of_8tbs": 100 * achieved / NOMINAL_HBM_GBS,
        "clocks": clocks,
        "e2e": {"value": replica_value(nparams, world, e2e_ms / e2e_steps), "unit": "params/s",
                "h2d_bytes_per_step": 4 * plan.full_elems, "d2h_bytes_per_step": 8 * plan.n_quantised,
                "ms_per_step": e2e_ms / e2e_steps, "steps": e2e_steps},
        "gpu_launches": args.steps,
        "roofline": run.roofline(ms_per_step, None if (args.format or args.fixed or args.fraction or args.no_pvt or args.all_variables)
                                 else wl.name),
        "sustained": sustained,
        "other_configs": other_configs,
        "cpu_baseline": cpu,
        "other_kernels": extra,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="conformer")
    ap.add_argument("--format", default="", help="override the workload's format: E,M (e.g. 3,7 = S1E3M7)")
    ap.add_argument("--fixed", action="store_true",
                    help="read --format as I,F of the fixed-point variant S1IxFy (e.g. 0,15 = Q15)")
    ap.add_argument("--fraction", type=float, default=0.0, help="override the quantised fraction of weight matrices")
    ap.add_argument("--no-pvt", action="store_true", help="ablation: without the per-variable transformation")
    ap.add_argument("--all-variables", action="store_true", help="ablation: biases and norms are eligible too")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--no-extra", action="store_true", help="skip timing the decompress / compress kernels")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the sub-records of the large transformer and the ragged set")
    ap.add_argument("--sustain", type=float, default=2.0,
                    help="seconds of back-to-back steps in the sustained sub-record (0 = skip)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
