"""The multi-GPU path is "replicas only": no data-path collective, only the barrier and the reduction of the
timing statistics.  That host logic is exercised here with two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    # replica `rank` took (10 + rank) ms and committed 100 * (rank + 1) tokens
    res = bench.combine_replica_stats(10.0 + rank, 100 * (rank + 1), 0.02 * (rank + 1), 50 + rank, dist, "cpu")
    dist.barrier()
    out.put((rank, res))
    dist.destroy_process_group()


def test_replica_statistics_max_time_sum_tokens():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = dict(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank in (0, 1):
        total_ms, committed, e2e_s, e2e_committed = results[rank]
        assert total_ms == 11.0 and committed == 300.0           # slowest replica's time, all replicas' tokens
        assert abs(e2e_s - 0.04) < 1e-12 and e2e_committed == 101.0


def test_bench_gpus_2_without_a_launcher_spawns_two_ranks():
    """`python bench.py --gpus 2` run as one plain process must become two ranks (here: gloo on CPU, made-up
    statistics) and report their combined figures -- never one replica's work under n_gpus = 2."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--replica-selftest"],
                         capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [json.loads(l) for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                           # rank 0 alone prints
    line = lines[0]
    assert line["n_gpus"] == 2 and line["world"] == 2
    assert line["total_ms"] == 11.0 and line["committed"] == 300.0   # slowest replica's time, both replicas' tokens
    # a launcher that gave another number of ranks than --gpus is refused
    env_bad = dict(env, WORLD_SIZE="1", RANK="0")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--replica-selftest"],
                         capture_output=True, text=True, timeout=120, env=env_bad, cwd=ROOT)
    assert res.returncode == 2 and "WORLD_SIZE" in res.stderr


def test_single_replica_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.combine_replica_stats(5.0, 7, 0.1, 3, None, "cpu") == (5.0, 7.0, 0.1, 3.0)


def test_roofline_object_prefers_in_stream_durations():
    """The roofline's launch duration: device timestamps when that pass ran, the event-bracketed figure otherwise,
    and the event-bracketed figure is always kept beside the first."""
    sys.path.insert(0, ROOT)
    import bench
    peak = 6000.0
    # 100 launches of 120 MB each: 40 us per launch by events, 30 us per launch in the stream
    r = bench.roofline_object({"gemm": [50, 1500.0], "attention": [10, 160.0]}, 4.0, 100 * 120e6, 100, 5.0, peak, "test", 121e6)
    assert abs(r["frac_with_activations"] - r["frac"]) < 1e-12          # no weights-only figure given: the two agree
    rw = bench.roofline_object({"gemm": [50, 1500.0], "attention": [10, 160.0]}, 4.0, 100 * 120e6, 100, 5.0, peak, "test", 121e6,
                               weight_bytes_per_launch=90e6)
    assert abs(rw["achieved"] - 90e6 / 30e-6 / 1e9) < 1e-6 and abs(rw["frac_with_activations"] - r["frac"]) < 1e-12
    assert rw["traffic_note"] and abs(rw["event_bracketed"]["achieved"] - 90e6 / 40e-6 / 1e9) < 1e-6
    assert abs(r["avg_launch_us"] - 30.0) < 1e-9 and r["launches_timed"] == 50
    assert abs(r["achieved"] - 120e6 / 30e-6 / 1e9) < 1e-6 and abs(r["frac"] - r["achieved"] / peak) < 1e-12
    assert abs(r["event_bracketed"]["avg_launch_us"] - 40.0) < 1e-9
    assert abs(r["event_bracketed"]["achieved"] - 120e6 / 40e-6 / 1e9) < 1e-6
    assert r["attention_avg_launch_us"] == 16.0 and r["bound"] == "hbm" and r["traffic"] == 121e6
    r2 = bench.roofline_object(None, 4.0, 100 * 120e6, 100, 5.0, peak, "test", None)
    assert abs(r2["avg_launch_us"] - 40.0) < 1e-9 and "event_bracketed" not in r2
    assert abs(r2["frac"] - (120e6 / 40e-6 / 1e9) / peak) < 1e-12
