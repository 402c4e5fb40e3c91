"""The N > 1 plumbing of bench.py (replicas only: barrier + max-over-ranks timing), on CPU with gloo."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 if rank == 0 else 25.0                      # rank 1 is the slow one
    bench.dist_barrier()
    value, ms_per_step = bench.aggregate_steps_per_s(50, local_ms, world, torch.device("cpu"))
    q.put((rank, value, ms_per_step, bench.dist_max(float(rank), torch.device("cpu"))))
    dist.destroy_process_group()


def test_two_rank_aggregate_uses_the_slowest_rank():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, value, ms_per_step, mx in res:
        assert abs(value - 2 * 50 / 0.025) < 1e-6 and abs(ms_per_step - 0.5) < 1e-9 and mx == 1.0


def test_single_process_is_a_noop():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.dist_max(3.5, torch.device("cpu")) == 3.5
    v, ms = bench.aggregate_steps_per_s(10, 5.0, 1, torch.device("cpu"))
    assert abs(v - 2000.0) < 1e-9 and abs(ms - 0.5) < 1e-12


def test_reference_arm_prints_one_contract_line():
    """`bench.py --impl reference` (the oracle on the host cores) prints exactly one JSON line with the contract's keys."""
    import json
    import subprocess
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "0",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in d, key
    assert d["impl"] == "reference" and d["vs_baseline"] is None and d["config"]["workload"] == "tiny"
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0


def test_gpus_flag_brings_up_the_replicas_by_itself():
    """`bench.py --gpus 2` started without a launcher (no WORLD_SIZE) spawns two ranks, which rendezvous on 127.0.0.1,
    time the (stub) step, take the max over ranks and print ONE line with n_gpus == 2.  --dry-run keeps it off the GPU."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "20", "--warmup", "3",
                        "--dry-run", "--backend", "gloo", "--config", "0"], capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.strip().startswith("{")]
    assert len(lines) == 1, r.stdout
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["steps"] == 20 and d["dry_run"] is True
    # rank 1 sleeps 2 ms per step, rank 0 1 ms: the slowest rank sets the time, both ranks' steps count
    assert d["ms_per_step"] >= 2.0 and abs(d["value"] - 2 * 1e3 / d["ms_per_step"]) < 1e-6 * d["value"]


def test_gpus_flag_refuses_more_ranks_than_devices():
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "4096", "--steps", "1"],
                       capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode == 2 and "CUDA device" in r.stderr
