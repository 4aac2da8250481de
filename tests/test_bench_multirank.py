"""The benchmark's multi-rank bookkeeping (replicas only: barrier, slowest rank's time, summed work) on CPU with gloo."""
import os
import sys

import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    dist.barrier()
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world)          # rank 1 is the slow one
    value = bench.whole_job_gflops(2_000_000_000, world, ms)
    split_value = bench.split_job_gflops(1_000_000_000 * (rank + 1), world, ms)      # slabs of unequal work
    out.put((rank, ms, value, split_value))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_summed_work():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value, split_value in results:
        assert ms == 15.0                                            # max over ranks, seen by both
        assert value == pytest.approx(2 * 2e9 / 15e-3 / 1e9)        # two replicas' work over that time
        assert split_value == pytest.approx(3e9 / 15e-3 / 1e9)      # one equation: the slabs' work summed, same time


def test_single_rank_is_a_no_op():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(7.5, 1) == 7.5
    assert bench.whole_job_gflops(10**9, 1, 1.0) == pytest.approx(1000.0)
    assert bench.split_job_gflops(10**9, 1, 1.0) == pytest.approx(1000.0)


def test_column_slab_of_the_headline_equation():
    sys.path.insert(0, ROOT)
    import numpy as np
    import bench
    import paper_2208_10391_b200 as mom
    import workloads as wl
    eq = wl.config_large_square(n=64)
    chain, add = wl.generate(eq)
    widths = 0
    for rank in range(4):
        seq, b, e = bench.column_slab_of(mom, eq, rank, 4)
        assert (b, e) == (16 * rank, 16 * rank + 16)
        assert seq.descs()[:-1] == eq.descs()[:-1] and seq.descs()[-1] == (64, 16, wl.GENERAL)
        c, a = bench.cut_columns(eq, chain, add, b, e)
        assert np.array_equal(c[-1], chain[-1][:, b:e]) and c[-1].flags["C_CONTIGUOUS"] and c[0] is chain[0]
        widths += e - b
    assert widths == bench.rd_cols(eq) == 64


@pytest.mark.parametrize("split", ["none", "columns"])
def test_bench_starts_its_own_ranks(split):
    # `python bench.py --gpus 2` (no torchrun around it) starts two ranks itself; --check-launch keeps them off the GPU:
    # gloo group, each rank plans its share, the slowest rank's time and the summed work are agreed on
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    proc = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--check-launch", "--split", split],
                          capture_output=True, text=True, timeout=600, env=env, cwd=ROOT)
    assert proc.returncode == 0, proc.stderr[-2000:]
    lines = [l for l in proc.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                         # rank 0 alone prints
    r = json.loads(lines[0])
    assert r["n_gpus"] == 2 and r["gpus_asked"] == 2 and r["ms_slowest_rank"] == 11.0
    whole = r["useful_flops_whole_equation"]
    if split == "columns":
        assert r["columns_all_ranks"] == 8192 and r["useful_flops_all_ranks"] == whole     # B is general: the cut is free
        assert r["slab_flops_over_whole"] == 1.0
        assert r["value"] == pytest.approx(whole / 11e-3 / 1e9)
    else:
        assert r["useful_flops_all_ranks"] == 2 * whole
        assert r["value"] == pytest.approx(2 * whole / 11e-3 / 1e9)


def test_launcher_command_is_one_process_per_gpu_on_the_loopback_address():
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.launcher_command(["--gpus", "4", "--steps", "7"], 4, 29876)
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29876"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "7"] and cmd[-5].endswith("bench.py")
