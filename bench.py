#!/usr/bin/env python
"""Benchmark of the DeMo optimizer transform (compress x W + decode) on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload decoder_1b] [--impl ours|reference]

One "step" is one optimizer step of the whole hot path: W x demo_compress + 1 x demo_decode_apply
over a synthetic parameter set resident in HBM.  Prints ONE JSON line (rank 0).  With N > 1 (torchrun)
every rank runs an independent replica of the same workload -- the path has no exchange step on one
GPU per replica -- and `value` is the work of all ranks over the slowest rank's time.
`--impl reference` times the fp64 CPU oracle on a bounded sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "optimizer-step params/s (compress+decode)"
UNIT = "params/s"


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json, device-to-device copy)"
    return 6650.0, "fallback (earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml

            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(0.05)

    def start(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()

    def stop(self):
        self._stop.set()
        if self._thr is not None:
            self._thr.join()
        med = sorted(self.samples)[len(self.samples) // 2] if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def algorithmic_bytes(wl, gbytes: int):
    """Bytes the method must move per step: per worker read g and m, write m; once read and write x.
    Payload traffic (written once, read once) is reported separately."""
    P = wl.n_params
    core = P * (wl.num_workers * (gbytes + 8) + 8)
    payload = 2 * wl.num_workers * wl.records_per_worker() * 8
    return core, payload


def cpu_sample(wl, target_s: float):
    """A bounded sample of the workload for the oracle: n chunks of 2-D tiles through W compress passes
    and one decode, n sized by a short probe so that one pass takes about target_s seconds.  The inputs
    are drawn once (the values do not change the work); returns (timed pass, n, cores)."""
    import numpy as np

    from oracle import demo_oracle as orc

    s, k, W = wl.chunk, wl.topk, wl.num_workers
    M = s * s
    rng = np.random.default_rng(0)

    def draw(n):
        return (rng.standard_normal((W, n, M)) * 1e-3, rng.standard_normal((W, n, M)) * 1e-2,
                rng.standard_normal((n, M)) * 0.02)

    def run(data):
        g, m, x = data
        n = x.shape[0]
        recs = np.zeros((W, n, min(k, M)), dtype=orc.RECORD_DTYPE)
        t0 = time.perf_counter()
        for w in range(W):
            out = orc.compress_chunks(g[w], m[w], s, s, k, wl.beta)
            recs[w]["idx"] = out["idx"]
            recs[w]["val"] = out["val"].astype(np.float32)
        orc.decode_chunks(recs, x, s, s, wl.lr, wl.weight_decay)
        return time.perf_counter() - t0

    cores = orc.max_threads()
    n0 = max(cores, 16)
    t_probe = run(draw(n0))
    n = int(min(max(n0, n0 * target_s / max(t_probe, 1e-6)), 1 << 16))
    data = draw(n)
    return (lambda: run(data)), n, cores


def cpu_baseline(wl, target_s: float = 20.0, sample=None):
    """Time the oracle, as it stands, on a bounded sample.  Returns (record, parameters, seconds)."""
    s, k, W = wl.chunk, wl.topk, wl.num_workers
    M = s * s
    run, n, cores = sample if sample is not None else cpu_sample(wl, target_s)
    t = run()
    return {"value": n * M / t, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "%d chunks of %dx%d (k=%d) through W=%d compress passes + 1 decode, %.1f s" % (n, s, s, k, W, t)}, n * M, t


def run_reference(args, rank):
    from paper_2411_19870_b200 import inputs

    if rank != 0:
        return
    wl = inputs.by_name(args.workload)
    times, units = [], 0
    base = None
    per_step = max(2.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    sample = cpu_sample(wl, per_step)  # sized and drawn once: every step is one pass over the same sample
    for i in range(args.warmup + args.steps):
        base, n_par, t = cpu_baseline(wl, sample=sample)
        if i >= args.warmup:
            times.append(t)
            units += n_par
    value = units / sum(times)
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / len(times), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "chunk": wl.chunk, "topk": wl.topk, "num_workers": wl.num_workers,
                   "note": "fp64 CPU oracle on a bounded chunk sample per step"},
        "cpu_baseline": dict(base, value=value),
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)


def run_ours(args, rank, world):
    import torch

    import paper_2411_19870_b200 as demo
    from paper_2411_19870_b200 import inputs

    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod

        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)

    wl = inputs.by_name(args.workload)
    if args.chunk or args.topk:  # ablation: same tensors, other chunk size / k (not the headline configuration)
        import dataclasses

        wl = dataclasses.replace(wl, chunk=args.chunk or wl.chunk, topk=args.topk or wl.topk)
    W, T = wl.num_workers, len(wl.shapes)
    gbytes = 2 if wl.grad_dtype == torch.bfloat16 else 4
    chunk_shapes = None
    if args.chunk_shape:  # ablation: rectangular chunks AxB for the matrices (B for the vectors), N-D kernels
        ca, cb = (int(v) for v in args.chunk_shape.lower().split("x"))
        chunk_shapes = [(ca, cb) if len(shp) == 2 else (cb,) for shp in wl.shapes]
        args.no_cpu_baseline = True  # the timed CPU baseline covers the square-chunk headline only
    tr = demo.DemoTransform(wl.shapes, chunk=wl.chunk, topk=wl.topk, beta=wl.beta, lr=wl.lr,
                            weight_decay=wl.weight_decay, num_workers=W,
                            grad_dtype=demo.DEMO_BF16 if gbytes == 2 else demo.DEMO_F32, device=local,
                            chunk_shapes=chunk_shapes)
    if args.path == "generic":
        tr.set_path(demo.DEMO_PATH_GENERIC)
    if args.momentum_domain == "dct":  # experiment, not the headline: momentum of 2-D tensors kept as DCT tiles
        tr.set_momentum_domain(demo.DEMO_MOMENTUM_DCT)
    if args.basis == "identity":
        tr.set_basis(torch.eye(wl.chunk))
    elif args.basis == "random":  # Gaussian draws seeded by a step number, orthonormalised on the device
        tr.set_basis_gaussian(inputs.basis_gaussian(1, wl.chunk))
    P0 = wl.n_params
    params = inputs.make_params(wl, dev)
    mom = [inputs.make_momentum(wl, dev) for _ in range(W)]
    streams = [inputs.GradStream(wl, w, dev) for w in range(W)]
    for st in streams:  # ablation: row-sparse embedding gradients
        st.embedding_active_rows = args.embedding_active_rows or None
    grads = [st.next() for st in streams]  # one seeded set per worker, reused
    payloads = [torch.empty(tr.payload_bytes, dtype=torch.uint8, device=dev) for _ in range(W)]
    torch.cuda.synchronize()

    def step(events=None):
        for w in range(W):
            if events is not None:
                e0 = torch.cuda.Event(enable_timing=True)
                e0.record()
            tr.compress(w, grads[w], mom[w], payloads[w])
            if events is not None:
                e1 = torch.cuda.Event(enable_timing=True)
                e1.record()
                events["compress"].append((e0, e1))
        if events is not None:
            e0 = torch.cuda.Event(enable_timing=True)
            e0.record()
        tr.decode_apply(payloads, params)
        if events is not None:
            e1 = torch.cuda.Event(enable_timing=True)
            e1.record()
            events["decode"].append((e0, e1))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = tr.launch_count
    events = {"compress": [], "decode": []}
    # Working sets that fit in the 126 MB L2 twice over are flushed out of it between timed steps by a
    # 256 MB write; the step is then timed by its own pair of events and the flushes are left out.
    working_set = W * P0 * (gbytes + 4) + 4 * P0 + W * tr.payload_bytes
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if working_set < (252 << 20) else None
    if flush is None:
        t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        marks = [t_start]
        t_start.record()
        for _ in range(args.steps):
            step(events)
            marks.append(torch.cuda.Event(enable_timing=True))
            marks[-1].record()
        t_end.record()
        barrier()
        ms_local = t_start.elapsed_time(t_end)
        per_step = [a.elapsed_time(b) for a, b in zip(marks[:-1], marks[1:])]
    else:
        pairs = []
        for _ in range(args.steps):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            step(events)
            e1.record()
            pairs.append((e0, e1))
        barrier()
        per_step = [a.elapsed_time(b) for a, b in pairs]
        ms_local = sum(per_step)
    clocks = sampler.stop()
    launches = tr.launch_count - launches0
    ms_total = max_over_ranks(ms_local, dist, dev)
    ms_step = ms_total / args.steps
    assert tr.device_status() == 0

    P = wl.n_params
    value = replica_throughput(P, world, ms_step)
    core_bytes, payload_bytes = algorithmic_bytes(wl, gbytes)
    peak, peak_src = _peaks()
    c_ms = [a.elapsed_time(b) for a, b in events["compress"]]
    d_ms = [a.elapsed_time(b) for a, b in events["decode"]]
    c_avg = sum(c_ms) / len(c_ms)
    d_avg = sum(d_ms) / len(d_ms)
    compress_bytes = P * (gbytes + 8)  # read g, read m, write m for one worker
    achieved = compress_bytes / (c_avg * 1e-3) / 1e9
    roofline = {
        "bound": "hbm", "kernel": "demo_compress (one worker: fused momentum+DCT+top-k+residual over all tensors)",
        "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src,
        "traffic": None, "algorithmic_bytes_per_launch": compress_bytes, "avg_launch_ms": c_avg,
        "decode": {"avg_launch_ms": d_avg, "algorithmic_bytes_per_launch": P * 8 + payload_bytes // 2,
                   "achieved": (P * 8 + payload_bytes // 2) / (d_avg * 1e-3) / 1e9},
        "step": {"algorithmic_bytes": core_bytes, "payload_bytes": payload_bytes,
                 "achieved": core_bytes / (ms_step * 1e-3) / 1e9, "frac_of_measured": core_bytes / (ms_step * 1e-3) / 1e9 / peak,
                 "frac_of_nominal_8TBs": core_bytes / (ms_step * 1e-3) / 8e12},
    }
    traffic_file = os.path.join(ROOT, "profiles", "traffic.json")
    headline_kernels = not args.chunk_shape and args.basis == "dct" and args.path == "auto" and not args.chunk
    if os.path.exists(traffic_file) and headline_kernels:  # the capture is of the fast DCT kernels at s = 64
        try:
            with open(traffic_file) as f:
                tj = json.load(f)
            per_param = tj.get("compress_dram_bytes_per_param")
            if per_param is not None:
                roofline["traffic"] = per_param * P
                roofline["traffic_source"] = tj.get("source")
        except Exception:
            pass

    # end to end through the host-buffer entry point: H2D of every worker's gradients from pinned
    # memory, the step, D2H of the W payloads
    e2e = None
    if not args.no_e2e:
        try:
            e2e = run_e2e(torch, tr, wl, grads, mom, payloads, params, dev, world, dist, gbytes, args)
        except Exception as ex:  # pragma: no cover
            e2e = {"value": None, "unit": UNIT, "error": repr(ex)}

    # Beside the headline (never part of it): the same step with the momentum buffers of the 2-D tensors kept in
    # the transform domain (demo_set_momentum_domain).  Runs after everything above, on the same buffers.
    side = None
    if (headline_kernels and args.momentum_domain == "spatial" and wl.chunk == 64 and not args.no_momentum_dct_line
            and not args.embedding_active_rows):
        try:
            tr.set_momentum_domain(demo.DEMO_MOMENTUM_DCT)
            for mw in mom:
                for t in mw:
                    t.zero_()          # m = 0 in either representation
            for _ in range(max(3, args.warmup)):
                step()
            barrier()
            sampler2 = ClockSampler(local)
            sampler2.start()
            ev = {"compress": [], "decode": []}
            s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s0.record()
            for _ in range(args.steps):
                if flush is not None:
                    flush.fill_(1)
                step(ev)
            s1.record()
            barrier()
            clocks2 = sampler2.stop()
            assert tr.device_status() == 0
            cm = sum(a.elapsed_time(b) for a, b in ev["compress"]) / len(ev["compress"])
            dm = sum(a.elapsed_time(b) for a, b in ev["decode"]) / len(ev["decode"])
            ms2 = (W * cm + dm) if flush is not None else max_over_ranks(s0.elapsed_time(s1), dist, dev) / args.steps
            side = {"momentum_domain": "dct", "note": "opt-in representation, not the contract of the metric",
                    "ms_per_step": ms2, "value": replica_throughput(P, world, ms2), "unit": UNIT,
                    "compress_avg_launch_ms": cm, "decode_avg_launch_ms": dm,
                    "compress_frac": compress_bytes / (cm * 1e-3) / 1e9 / peak,
                    "step_frac_of_measured": core_bytes / (ms2 * 1e-3) / 1e9 / peak,
                    "step_frac_of_nominal_8TBs": core_bytes / (ms2 * 1e-3) / 8e12, "clocks": clocks2}
            tr.set_momentum_domain(demo.DEMO_MOMENTUM_SPATIAL)
        except Exception as ex:  # pragma: no cover
            side = {"momentum_domain": "dct", "error": repr(ex)}

    base = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        base, _, _ = cpu_baseline(wl)

    if rank == 0:
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "ms_per_step_median": sorted(per_step)[len(per_step) // 2],
            "ms_per_step_min": min(per_step), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl.name, "n_params": P, "n_tensors": T, "chunk": wl.chunk, "topk": wl.topk,
                       "num_workers": W, "beta": wl.beta, "grad_dtype": "bf16" if gbytes == 2 else "f32",
                       "parallelism": "replicas only (one GPU per replica, no collective)" if world > 1 else "1 GPU",
                       "worker_params_per_s": value * W, "l2": ("inputs (%.1f GB resident in HBM) are larger than the 126 MB L2; no flush needed" % (working_set / 1e9))
                       if flush is None else ("working set %.1f MB: L2 flushed by a 256 MB write before every timed step"
                                              % (working_set / 1e6)), "kernel_path": args.path,
                       "gradients": "one seeded gradient set per worker, reused every step on purpose (a second set "
                                    "per worker does not fit beside the %d momenta; the momentum still changes "
                                    "every step)" % W,
                       "momentum_domain": args.momentum_domain,
                       "basis": args.basis, "chunk_shape": args.chunk_shape or None,
                       "embedding_active_rows": args.embedding_active_rows or None},
            "roofline": roofline, "clocks": clocks, "gpu_launches": int(launches), "e2e": e2e,
        }
        if base is not None:
            out["cpu_baseline"] = base
        if side is not None:
            out["momentum_dct"] = side
        print(json.dumps(out), flush=True)
    tr.close()
    if dist is not None:
        dist.destroy_process_group()


def run_e2e(torch, tr, wl, grads, mom, payloads, params, dev, world, dist, gbytes, args):
    W = wl.num_workers
    P = wl.n_params
    import psutil

    need = W * P * gbytes + W * tr.payload_bytes
    distinct = psutil.virtual_memory().available > 2.5 * need * max(1, world)
    if distinct:
        host = [[g.cpu().pin_memory() for g in gw] for gw in grads]
        note = "distinct pinned gradient set per worker"
    else:
        one = [g.cpu().pin_memory() for g in grads[0]]
        host = [one for _ in range(W)]
        note = "one pinned gradient set copied for every worker (host memory too small for W sets)"
    out = torch.empty(W * tr.payload_bytes, dtype=torch.uint8).pin_memory()
    steps = max(1, min(args.steps, args.e2e_steps))
    tr.step_host(host, grads, mom, payloads, params, out)  # warm-up
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        tr.step_host(host, grads, mom, payloads, params, out)
    e1.record()
    torch.cuda.synchronize()
    ms = max_over_ranks(e0.elapsed_time(e1) / steps, dist, dev)
    return {"value": replica_throughput(P, world, ms), "unit": UNIT, "ms_per_step": ms, "steps": steps,
            "h2d_bytes_per_step": W * P * gbytes, "d2h_bytes_per_step": W * tr.payload_bytes, "note": note}


def max_over_ranks(ms: float, dist, device) -> float:
    """Device time of the slowest rank (identity when there is one process)."""
    if dist is None:
        return float(ms)
    import torch

    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_throughput(units_per_rank: float, world: int, ms: float) -> float:
    """Whole-job throughput of `world` independent replicas: all units over the slowest rank's time."""
    return world * units_per_rank / (ms * 1e-3)


def spawn_ranks(args) -> int:
    """`python bench.py --gpus N` outside a launcher: start N ranks of this script on this node, one per GPU,
    under torch.distributed.run (rendezvous on 127.0.0.1) and pass their output through.  The ranks stay
    independent replicas: the process group only carries the barrier and the MAX over ranks of the device time."""
    import socket
    import subprocess

    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def run_standin(args, rank, world):
    """The launch, rendezvous and reporting path of the N-rank benchmark with a CPU stand-in for the timed region
    (a gloo group, a short host loop per step): what can be checked of `--gpus N` on a machine without GPUs.
    Prints the same JSON shape with "standin": "cpu"; never a benchmark number."""
    import numpy as np
    import torch
    import torch.distributed as dist

    if world > 1:
        dist.init_process_group("gloo")
    a = np.random.default_rng(rank).standard_normal((64, 64))
    for _ in range(args.warmup):
        a = a @ a.T / 64.0
    if world > 1:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        a = a @ a.T / 64.0
    ms_local = (time.perf_counter() - t0) * 1e3
    ms = max_over_ranks(ms_local, dist if world > 1 else None, torch.device("cpu")) / args.steps
    if world > 1:
        dist.barrier()
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": replica_throughput(float(a.size), world, ms), "unit": UNIT,
                          "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
                          "higher_is_better": True, "scaling": "weak", "standin": "cpu",
                          "config": {"workload": "launcher check", "parallelism": "replicas only"}}), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_grid(args):
    """Ablation grid of the stress configuration (heavy-tailed gradients with tie-maker chunks):
    chunk s x k x fan-in W, ms per optimizer step, one JSON line per cell.  The 4096 x 4096 matrix runs
    every cell; `--grid-set` adds the 1B-class set for the cells that fit in memory (W <= 16)."""
    import torch

    import paper_2411_19870_b200 as demo
    from paper_2411_19870_b200 import inputs

    dev = torch.device("cuda", 0)
    for full in ([False, True] if args.grid_set else [False]):
        for s in (32, 64, 128):
            for k in (1, 8, 32, 128):
                for W in (1, 8, 64):
                    if full and W > 16:
                        continue  # 64 momentum sets of the 1B-class set do not fit in 180 GB
                    wl = inputs.stress(chunk=s, topk=k, num_workers=W, full_set=full)
                    tr = demo.DemoTransform(wl.shapes, chunk=s, topk=k, beta=wl.beta, lr=wl.lr,
                                            weight_decay=wl.weight_decay, num_workers=W)
                    params = inputs.make_params(wl, dev)
                    mom = [inputs.make_momentum(wl, dev) for _ in range(W)]
                    grads = [inputs.GradStream(wl, w, dev).next() for w in range(W)]
                    payloads = [torch.empty(tr.payload_bytes, dtype=torch.uint8, device=dev) for _ in range(W)]

                    def step():
                        for w in range(W):
                            tr.compress(w, grads[w], mom[w], payloads[w])
                        tr.decode_apply(payloads, params)

                    for _ in range(3):
                        step()
                    torch.cuda.synchronize()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    n = 5
                    e0.record()
                    for _ in range(n):
                        step()
                    e1.record()
                    torch.cuda.synchronize()
                    ms = e0.elapsed_time(e1) / n
                    assert tr.device_status() == 0
                    core, _ = algorithmic_bytes(wl, 2)
                    print(json.dumps({"workload": wl.name, "n_params": wl.n_params, "chunk": s, "topk": k,
                                      "num_workers": W, "ms_per_step": ms, "params_per_s": wl.n_params / (ms * 1e-3),
                                      "algorithmic_GBps": core / (ms * 1e-3) / 1e9,
                                      "kernels": "fast"}), flush=True)
                    tr.close()
                    del params, mom, grads, payloads
                    torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="decoder_1b")
    ap.add_argument("--path", default="auto", choices=["auto", "generic"])
    ap.add_argument("--chunk", type=int, default=0, help="override the workload's chunk size (ablation)")
    ap.add_argument("--topk", type=int, default=0, help="override the workload's k (ablation)")
    ap.add_argument("--embedding-active-rows", type=int, default=0,
                    help="rows per chunk-row block of the embedding that get a gradient (ablation; 0 = all)")
    ap.add_argument("--chunk-shape", default="", help="AxB: rectangular chunks through the N-D kernels (ablation)")
    ap.add_argument("--basis", default="dct", choices=["dct", "identity", "random"],
                    help="transform basis; anything but dct takes the dense-transform kernels (not the headline)")
    ap.add_argument("--momentum-domain", default="spatial", choices=["spatial", "dct"],
                    help="dct: the opt-in representation of demo_set_momentum_domain (a second, non-headline line)")
    ap.add_argument("--no-momentum-dct-line", action="store_true",
                    help="skip the extra measurement of the opt-in transform-domain momentum after the headline run")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--grid", action="store_true", help="print the stress/ablation grid instead of the benchmark line")
    ap.add_argument("--grid-set", action="store_true", help="with --grid: also run the 1B-class set")
    ap.add_argument("--standin", default="", choices=["", "cpu"],
                    help="cpu: run the launcher / rendezvous / reporting path with a host stand-in for the timed "
                         "region (checks `--gpus N` without GPUs; not a benchmark)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = max(args.warmup, 1)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and "RANK" not in os.environ and not args.grid:
        # not under a launcher: become one (N ranks, one per GPU; each rank re-enters main() with RANK set)
        raise SystemExit(spawn_ranks(args))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.standin == "cpu":
        run_standin(args, rank, world)
    elif args.grid:
        if rank == 0:
            run_grid(args)
    elif args.impl == "reference":
        run_reference(args, rank)
    else:
        run_ours(args, rank, world)


if __name__ == "__main__":
    main()
