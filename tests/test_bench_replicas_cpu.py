"""The N > 1 path of bench.py is "replicas only": every rank runs the same single-GPU workload and
rank 0 reports all ranks' work over the slowest rank's device time.  The host-side part of that
(rendezvous, MAX reduction, aggregation) is exercised here with two gloo ranks on CPU."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, out):
    import bench

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 10.0 + 5.0 * rank            # rank 1 is the slow one
    ms = bench.max_over_ranks(ms_local, dist, torch.device("cpu"))
    dist.barrier()
    if rank == 0:
        out.put((ms, bench.replica_throughput(1000.0, world, ms)))
    dist.destroy_process_group()


def test_two_gloo_ranks_report_slowest_time_and_total_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    ms, value = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ms == 15.0
    assert value == pytest.approx(2 * 1000.0 / 0.015)


def test_single_process_is_identity():
    import bench

    assert bench.max_over_ranks(3.5, None, None) == 3.5
    assert bench.replica_throughput(10.0, 1, 1000.0) == 10.0


def test_reference_arm_prints_one_json_line_quickly():
    import json
    import subprocess

    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "params/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


def test_gpus_2_outside_a_launcher_starts_two_ranks():
    """`python bench.py --gpus 2` with no launcher around it re-executes itself under torch.distributed.run; the
    CPU stand-in replaces only the timed region, so launch, rendezvous on 127.0.0.1, MAX over ranks and the single
    JSON line of rank 0 are the real ones."""
    import json
    import subprocess

    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "3", "--warmup", "3",
                        "--standin", "cpu"], capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1                      # rank 0 alone prints
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["standin"] == "cpu" and line["value"] > 0


def test_under_a_launcher_bench_does_not_spawn_again():
    import json
    import subprocess

    env = dict(os.environ, RANK="0", WORLD_SIZE="1", LOCAL_RANK="0", MASTER_ADDR="127.0.0.1", MASTER_PORT="29999")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1", "--warmup", "0",
                        "--standin", "cpu"], capture_output=True, text=True, timeout=120, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["n_gpus"] == 1                  # the launcher's world size is what counts
