"""The N > 1 path of the benchmark on CPU: two gloo ranks, each with its own (independent)
dock workload; the only exchange is the max-over-ranks of the timings, and rank 0 reports the
whole-job rate.  Also the reference arm under a multi-rank launch: only rank 0 works."""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    from paper_2507_19017_b200 import workloads as wl
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    # every rank draws its own batch (different seed), as bench.py does
    w = wl.make_config(1, seed=wl.BASE_SEED + 1 + 1000 * rank)
    ms = [1.0 + rank, 0.25 * (2 - rank)]          # rank 1 is slower on the first, faster on the second
    got = bench.max_over_ranks(dist, ms, torch.device("cpu"))
    rate = bench.whole_job_rate(world, w.n * len(w.consumers), got[0] * 1e-3)
    dist.barrier()
    with open(out + f".{rank}", "w") as f:
        json.dump({"max": got, "rate": rate, "tokens": w.tokens_total()}, f)
    dist.destroy_process_group()


def test_two_gloo_ranks_reduce_timings_and_scale_weakly(tmp_path):
    import torch.multiprocessing as mp
    port, out = _free_port(), str(tmp_path / "r")
    mp.spawn(_rank_main, args=(2, port, out), nprocs=2, join=True)
    r0, r1 = (json.load(open(out + f".{r}")) for r in (0, 1))
    assert r0["max"] == r1["max"] == [2.0, 0.5]
    assert r0["rate"] == r1["rate"] == pytest.approx(2 * 64 * 4 / 2.0e-3)
    assert r0["tokens"] != r1["tokens"]          # independent batches, no shared data


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--config", "1", "--cpu-seconds", "0.2"], env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0 and res.stdout.strip() == ""
    env["RANK"] = "0"; env["LOCAL_RANK"] = "0"
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--config", "1", "--cpu-seconds", "0.2"], env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["value"] == line["value"] and line["unit"] == "samples/s"
