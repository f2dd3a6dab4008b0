"""Host logic of the N > 1 benchmark path on CPU: two gloo ranks on 127.0.0.1.

The hot path shards by (batch, head) with no data-path collective, so a multi-GPU run is one
layer instance per rank; the only exchange is the max-over-ranks of the device timings and the
barriers around the timed region.  This checks that exchange and the reference arm's rank rule."""
import os
import subprocess
import sys

import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    torch.distributed.init_process_group("gloo", rank=rank, world_size=world)
    torch.distributed.barrier()
    mine = [10.0 + 5.0 * rank, 100.0 - 30.0 * rank]          # rank 1 slower on [0], rank 0 on [1]
    got = bench.max_over_ranks(mine, world, torch.device("cpu"))
    out.put((rank, got, bench.job_value(world, 2.0e12, got[0])))
    torch.distributed.barrier()
    torch.distributed.destroy_process_group()


def test_timings_are_the_maximum_over_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, value in res:
        assert got == [15.0, 100.0]                            # both ranks see the slowest rank
        assert value == pytest.approx(2 * 2.0e12 / 15.0e-3 / 1e12)   # whole job: both instances


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], 1, torch.device("cpu")) == [1.5, 2.5]


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_gpus_flag_starts_the_ranks_itself():
    """`bench.py --gpus 2` run plainly (no torchrun) starts two ranks, which meet on 127.0.0.1 over
    gloo, exchange their timings and print ONE line with n_gpus = 2 and the slowest rank's time."""
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--host-check",
                        "--backend", "gloo", "--workload", "tiny"], env=env, capture_output=True, text=True,
                       timeout=300)
    assert r.returncode == 0, r.stderr
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2
    assert d["max_over_ranks"] == [2.0, 10.0]          # rank 1 is slower on [0], rank 0 on [1]
    assert d["config"]["workload"] == "tiny"
