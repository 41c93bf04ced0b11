"""The partitioned step's driver (`PartitionedStep`) over two real processes, on CPU with gloo.

The CUDA library cannot run here, so each process drives a small CPU stand-in for the handle that takes the three
phases from the oracle's PRIMITIVES (hash family, sketch, unsketch, top-k), over its own half of the workers.  What is
under test is the exchange protocol: that the two all-reduces of the driver, with the buffer layouts the header
documents (share of the mean sketch | gradient sums on I_{t-1} in ascending order; sums of a_t at the candidates in
ascending order), turn per-process partial sums into the step the n-worker oracle takes as a whole.
"""
import json
import os
import sys

import numpy as np
import pytest

from conftest import ROOT

torch = pytest.importorskip("torch")

D, N, R, C, K, SEED, LOG2G = 6000, 4, 5, 512, 60, 11, 3
HYPER = dict(lr=0.01, beta1=0.9, beta2=0.99, eps=1e-6)
STEPS = 4


def _grads(step):
    rng = np.random.default_rng(100 + step)
    g = rng.normal(0.0, 1e-3, (N, D)).astype(np.float32)
    pos = np.random.default_rng(99).permutation(D)[:40]
    g[:, pos] += (rng.uniform(0.5, 1.0, (N, 40)) * rng.choice([-1.0, 1.0], (N, 40))).astype(np.float32)
    return g


class CpuHandle:
    """Algorithm 2 in three phases over `workers` of the N workers, from the oracle's primitives."""

    def __init__(self, workers, P):
        import oracle
        self.o, self.workers, self.P = oracle, list(workers), P
        nl = len(self.workers)
        self.idx = np.stack([oracle.hash_family(SEED, LOG2G, C, row, 0, D)[0] for row in range(R)])
        self.sgn = np.stack([oracle.hash_family(SEED, LOG2G, C, row, 0, D)[1] for row in range(R)])
        self.m = np.zeros((nl, D), np.float32)
        self.e = np.zeros((nl, D), np.float32)
        self.v = np.full(D, HYPER["eps"], np.float32)
        self.vhat = self.v.copy()
        self.I_prev = np.zeros(0, np.int64)

    def exchange_floats(self, which):
        return R * C + K if which == 1 else self.P * K

    def step_local(self, grads, exchange1):
        g = np.asarray(grads, np.float64)
        b1 = HYPER["beta1"]
        self.m = (b1 * self.m + (1 - b1) * g).astype(np.float32)
        self.e = (self.m.astype(np.float64) + self.e).astype(np.float32)          # a_t, kept in the e buffer
        x1 = exchange1.numpy()
        tables = np.stack([self.o.sketch(self.e[w], R, C, self.idx, self.sgn) for w in range(len(self.workers))])
        x1[:R * C] = (tables.astype(np.float64).sum(axis=0) / N).astype(np.float32).ravel()
        x1[R * C:] = 0.0
        x1[R * C:R * C + self.I_prev.size] = g[:, self.I_prev].sum(axis=0)
        self.g = g

    def step_select(self, exchange1, exchange2):
        x1 = exchange1.numpy()
        S = x1[:R * C].reshape(R, C).copy()
        b2 = HYPER["beta2"]
        h = np.zeros(D)
        h[self.I_prev] = x1[R * C:R * C + self.I_prev.size].astype(np.float64) / N
        self.v = (b2 * self.v + (1 - b2) * h * h).astype(np.float32)
        self.vhat = np.maximum(self.vhat, self.v)
        est = self.o.unsketch(S, D, self.idx, self.sgn, self.vhat)
        self.cand = np.sort(self.o.topk(est, self.P * K)).astype(np.int64)
        exchange2.numpy()[:] = self.e[:, self.cand].astype(np.float64).sum(axis=0)

    def step_finish(self, exchange2, x):
        exact = (exchange2.numpy().astype(np.float64) / N / np.sqrt(self.vhat[self.cand])).astype(np.float32)
        if self.P > 1:
            pos = np.sort(self.o.topk(exact, K)).astype(np.int64)
        else:
            pos = np.arange(K)
        I = self.cand[pos]
        xv = x.numpy()
        xv[I] = (xv[I].astype(np.float64) - HYPER["lr"] * exact[pos]).astype(np.float32)
        self.e[:, I] = 0.0
        self.I_prev = I


def _worker(rank, world, port, out, P):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import torch.distributed as dist
    from paper_2210_07454_b200.partitioned import PartitionedStep
    dist.init_process_group("gloo", rank=rank, world_size=world)
    per = N // world
    mine = range(rank * per, (rank + 1) * per)
    handle = CpuHandle(mine, P)
    drv = PartitionedStep(handle, "cpu")
    x = torch.zeros(D, dtype=torch.float32)
    sets = []
    for t in range(1, STEPS + 1):
        drv.step(torch.from_numpy(_grads(t)[list(mine)].copy()), x)
        sets.append(handle.I_prev.tolist())
    dist.barrier()
    dist.destroy_process_group()
    np.save(f"{out}.x{rank}.npy", x.numpy())
    np.save(f"{out}.vhat{rank}.npy", handle.vhat)
    with open(f"{out}.{rank}.json", "w") as f:
        json.dump({"I": sets, "floats": drv.floats_per_step}, f)


@pytest.mark.parametrize("P,port", [(1, 29741), (2, 29743)])
def test_two_processes_reproduce_the_n_worker_oracle(tmp_path, P, port):
    import torch.multiprocessing as mp
    import oracle
    out = str(tmp_path / "res")
    mp.spawn(_worker, args=(2, port, out, P), nprocs=2, join=True)
    ora = oracle.Oracle(D, N, R, C, K, seed=SEED, log2g=LOG2G, P=P, **HYPER)
    x_ref = np.zeros(D, np.float32)
    ref_sets = []
    for t in range(1, STEPS + 1):
        ora.step(_grads(t), x_ref)
        ref_sets.append(ora.field("I").tolist())
    res = [json.load(open(f"{out}.{r}.json")) for r in range(2)]
    xs = [np.load(f"{out}.x{r}.npy") for r in range(2)]
    vh = [np.load(f"{out}.vhat{r}.npy") for r in range(2)]
    assert res[0]["I"] == res[1]["I"] and np.array_equal(xs[0], xs[1]) and np.array_equal(vh[0], vh[1])
    assert res[0]["floats"] == oracle.comm_floats(R, C, K, P) - K     # |S| + P*k + 2k less the k sent back
    assert res[0]["I"] == ref_sets                                     # planted heavy coordinates: no near-ties
    np.testing.assert_allclose(vh[0], ora.field("vhat"), rtol=1e-5, atol=0)
    moved = np.unique(np.concatenate([np.asarray(s) for s in ref_sets]))
    np.testing.assert_allclose(xs[0][moved], x_ref[moved], rtol=1e-4, atol=1e-9)
    rest = np.setdiff1d(np.arange(D), moved)
    assert not xs[0][rest].any() and not x_ref[rest].any()
