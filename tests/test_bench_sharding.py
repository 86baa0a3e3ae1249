"""Host logic of the N > 1 benchmark path, on CPU with gloo (world_size 2): the slowest rank
sets the time, the job's value is the sum of the ranks' work over it, and the reference arm
prints on rank 0 only."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))
    val = bench.whole_job_tflops(2.0e12, world, ms)
    dist.barrier()
    if rank == 0:
        json.dump({"ms": ms, "val": val}, open(out, "w"))
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value(tmp_path):
    out = str(tmp_path / "r.json")
    mp.spawn(_worker, args=(2, 29731, out), nprocs=2, join=True)
    r = json.load(open(out))
    assert r["ms"] == 15.0                                   # the slower rank
    assert abs(r["val"] - 2 * 2.0e12 / 15e-3 / 1e12) < 1e-9  # both ranks' work over that time


def test_single_rank_helpers():
    sys.path.insert(0, ROOT)
    import bench
    import lamp_inputs as li
    assert bench.max_over_ranks(3.5) == 3.5
    cfg = li.CONFIGS[2]
    assert bench.valid_pairs(cfg) == 8192 * 8193 // 2
    assert bench.flops_of(cfg) == 4.0 * 128 * (8192 * 8193 // 2) * 4 * 32
    assert sum(bench.unit_pairs(cfg, g) for g in range(8192 // 32)) == bench.valid_pairs(cfg)
    w = 1024
    assert bench.valid_pairs(li.CONFIGS[3], window=w) == w * (w + 1) // 2 + (8192 - w) * w


def test_reference_arm_prints_on_rank0_only():
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29733", WORLD_SIZE="2")
    outs = []
    for rank in (0, 1):
        e = dict(env, RANK=str(rank), LOCAL_RANK=str(rank))
        p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                            "--config", "0", "--steps", "1", "--warmup", "0"], env=e, capture_output=True, text=True,
                           timeout=300)
        assert p.returncode == 0, p.stderr
        outs.append(p.stdout.strip())
    line = json.loads(outs[0].splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["n_gpus"] == 2
    assert outs[1] == ""
