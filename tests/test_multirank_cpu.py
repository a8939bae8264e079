"""The N > 1 path of the benchmark on CPU: two gloo ranks.  The path shards by replica (every rank
fake-quantizes its own batch, no exchange), so what needs checking is the plumbing: each rank
draws a different batch of the same law, timing is the maximum over ranks, and the reported
value is the whole-job aggregate."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank: int, world: int, port: int, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from oracle import granq_oracle as orc
    from paper_2503_18339_b200 import workloads as wl
    spec = wl.config_tensors(1)[0]
    x = wl.make_activation(spec, block_offset=1000 * rank)          # this replica's batch
    res = orc.fused(x, 3, gy=wl.make_upstream_grad(spec, block_offset=1000 * rank))
    ms = bench.max_over_ranks(10.0 * (rank + 1), device="cpu")      # rank 1 is the slow one
    sums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(sums, torch.tensor([float(x.sum())], dtype=torch.float64))
    out[rank] = (ms, [float(s) for s in sums], float(res.hi.max()), bench.whole_job_gbs(1_000_000_000, world, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_max_time_and_distinct_batches():
    world, port = 2, 29500 + os.getpid() % 2000
    out = mp.get_context("spawn").Manager().dict()
    mp.spawn(_rank, args=(world, port, out), nprocs=world, join=True)
    (ms0, sums0, hi0, v0), (ms1, sums1, hi1, v1) = out[0], out[1]
    assert ms0 == ms1 == 20.0                                        # the slower rank's time, on both
    assert sums0 == sums1 and sums0[0] != sums0[1]                   # different batches per replica
    assert hi0 != hi1                                                # hence their own per-channel ranges
    assert v0 == v1 == 2 * 1_000_000_000 / 20e-3 / 1e9               # aggregate over both replicas


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, device="cpu") == 3.5
    assert np.isclose(bench.whole_job_gbs(16_000_000_000, 1, 4.0), 4000.0)


def test_plain_command_with_gpus_2_starts_its_own_ranks():
    """`python bench.py --gpus 2` without a torchrun environment spawns the ranks itself: here with the
    GPU-free self-test (gloo), rank 0 printing the aggregate over both ranks and the slower rank's time."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--rank-selftest"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["n_gpus"] == 2 and line["ms_per_step"] == 20.0 and line["value"] == 2 * 1e9 / 20e-3 / 1e9


def test_spawn_ranks_sets_the_torchrun_environment():
    sys.path.insert(0, ROOT)
    import bench
    code = "import os,sys; sys.exit(0 if (os.environ['WORLD_SIZE'], os.environ['MASTER_ADDR']) == ('3', '127.0.0.1') and os.environ['RANK'] == os.environ['LOCAL_RANK'] else 1)"
    assert bench.spawn_ranks(3, [sys.executable, "-c", code], timeout=60) == [0, 0, 0]
