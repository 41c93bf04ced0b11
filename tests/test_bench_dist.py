"""Multi-process path of bench.py on CPU (gloo, world size 2).

The optimiser step does not shard across GPUs (all n workers are resident on one device by construction), so
`bench.py --gpus N` runs N independent replicas; the only cross-rank logic is the barrier, the max-over-ranks
timing and the sum of launch counts, which is what this test exercises, plus the reference arm's rule that only
rank 0 works.
"""
import json
import os
import subprocess
import sys

import pytest

from conftest import ROOT

torch = pytest.importorskip("torch")


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dev = torch.device("cpu")
    dist.barrier()
    mx = bench.reduce_max(10.0 + 5.0 * rank, world, dev)        # rank 1 is the slow one
    sm = bench.reduce_sum(9.0 * (rank + 1), world, dev)
    w, r, l = bench._dist()
    dist.barrier()
    dist.destroy_process_group()
    with open(f"{out}.{rank}", "w") as f:
        json.dump({"max": mx, "sum": sm, "world": w, "rank": r, "local": l}, f)


def test_reduce_helpers_world_size_two(tmp_path):
    import torch.multiprocessing as mp
    out = str(tmp_path / "res")
    mp.spawn(_worker, args=(2, 29731, out), nprocs=2, join=True)
    res = [json.load(open(f"{out}.{r}")) for r in range(2)]
    for r, got in enumerate(res):
        assert got["max"] == 15.0 and got["sum"] == 27.0          # every rank sees the job-wide numbers
        assert (got["world"], got["rank"], got["local"]) == (2, r, r)
    # whole-job value = replicas x per-replica units / max time: two replicas at the slower rank's time
    n, d, ms = 8, 25_600_000, res[0]["max"]
    assert bench_value(2, n, d, ms) == pytest.approx(2 * n * d / (ms * 1e-3) / 1e9)


def bench_value(world, n, d, ms):
    return world * n * d / (ms * 1e-3) / 1e9


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0 and p.stdout.strip() == ""           # other ranks exit 0 without work
    env0 = dict(os.environ, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "C1", "--ref-scale", "1"], env=env0,
                       capture_output=True, text=True, timeout=300)
    assert p.returncode == 0, p.stderr
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0 and line["n_gpus"] == 2
