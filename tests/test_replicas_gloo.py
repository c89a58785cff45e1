"""The multi-GPU path on CPU: two gloo ranks.

The step has no exchange between sequences, so N GPUs run N independent replicas.  What a multi-rank
bench run adds to the single-GPU one is host logic only: every rank draws its own seeded batch, the
job's time is the slowest rank's, throughput is the sum over replicas, and the reference arm runs on
rank 0 alone.  These tests run that logic in two processes over gloo."""
import json
import os
import subprocess
import sys
from pathlib import Path

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parents[1]
sys.path.insert(0, str(ROOT))


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, str(ROOT))
    import bench
    from paper_2601_17917_b200 import workloads as wl
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = bench.rank_config(wl.CONFIGS["tiny"], rank)
        z = wl.logits(cfg)
        my_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
        job_ms = bench.max_over_ranks(my_ms, world, torch.device("cpu"))
        res = {"rank": rank, "seed": cfg.seed, "checksum": float(z.double().sum()), "job_ms": job_ms,
               "value": bench.job_throughput(world, job_ms)}
        Path(out_dir, f"r{rank}.json").write_text(json.dumps(res))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_own_batches_and_slowest_rank_time(tmp_path):
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0, r1 = (json.loads((tmp_path / f"r{r}.json").read_text()) for r in (0, 1))
    assert r0["seed"] != r1["seed"] and r0["checksum"] != r1["checksum"]      # independent batches
    assert r0["job_ms"] == r1["job_ms"] == 15.0                               # max over ranks, on every rank
    assert r0["value"] == r1["value"] == 2 * 1e3 / 15.0                       # whole-job steps/s


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(3.5, 1, torch.device("cpu")) == 3.5
    assert bench.job_throughput(1, 2.0) == 500.0


def test_reference_arm_runs_on_rank_0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1", MASTER_ADDR="127.0.0.1")
    p = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0", "--config", "tiny"], env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0 and p.stdout.strip() == ""
    env["RANK"] = "0"
    p = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0", "--config", "tiny"], env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


def test_bare_gpus_flag_starts_its_own_ranks():
    """`python bench.py --gpus 2` without a launcher around it starts two ranks itself; with --dry-run the ranks
    do the host-side part only (gloo): own seeds per rank, max over ranks, n_gpus = 2 in the one line printed."""
    import bench
    cmd = bench.replica_command(2, ["--gpus", "2", "--dry-run"], port=29431)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"] and "--nproc-per-node=2" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[-3:] == ["--gpus", "2", "--dry-run"]
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_PORT")}
    p = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--gpus", "2", "--dry-run", "--config", "tiny"], env=env,
                       capture_output=True, text=True, timeout=600)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [json.loads(l) for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                   # rank 0 alone prints
    line = lines[0]
    assert line["dry_run"] and line["n_gpus"] == 2 and line["config"]["parallelism"] == "replicas x2"
    assert len(set(line["rank_seeds"])) == 2                 # every replica draws its own batch
    assert line["ms_per_step"] == 2.0 and line["value"] == 2 * 1e3 / 2.0     # slowest rank's time; whole-job steps/s
