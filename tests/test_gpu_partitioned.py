"""GPU parity of the partitioned step (workers split over processes) against the n-worker CPU oracle.

Only one GPU is needed: the processes are emulated as several handles that take each phase one after the other, and
the all-reduce between the phases is a sum of their exchange buffers in a fixed order, copied back to every one of
them (so every "process" sees the same bits, as after an NCCL all-reduce).  No kernel waits on another.
"""
import numpy as np
import pytest

import oracle
from parity import compare_step, force_state

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

PER_WORKER = ("m", "e", "tables", "vw", "vhatw")


class Ranks:
    """Several handles on one GPU, presented to the comparison helpers as one optimiser over all the workers."""

    def __init__(self, w, split, variant="ga", P=1, window_lines=None):
        from paper_2210_07454_b200 import binding
        assert sum(split) == w.n
        self.split, self.k, self.P = split, w.k, P
        self.handles = [binding.SketchedAMSGrad(w.d, nl, w.r, w.c, w.k, seed=w.seed, lr=w.lr, beta1=w.beta1,
                                                beta2=w.beta2, eps=w.eps, window_lines=window_lines, variant=variant,
                                                P=P, workers_total=w.n) for nl in split]
        self.x1 = [torch.zeros(h.exchange_floats(1), device="cuda") for h in self.handles]
        self.x2 = [torch.zeros(h.exchange_floats(2), device="cuda") for h in self.handles]
        self.first = np.concatenate([[0], np.cumsum(split)])

    @staticmethod
    def _all_reduce(bufs):
        total = bufs[0].clone()
        for b in bufs[1:]:
            total += b
        for b in bufs:
            b.copy_(total)

    def step(self, grads, xs):
        for g, h in enumerate(self.handles):
            h.step_local(grads[self.first[g]:self.first[g + 1]], self.x1[g])
        self._all_reduce(self.x1)
        for g, h in enumerate(self.handles):
            h.step_select(self.x1[g], self.x2[g])
        self._all_reduce(self.x2)
        for g, h in enumerate(self.handles):
            h.step_finish(self.x2[g], xs[g])

    def sync(self):
        for h in self.handles:
            h.sync()

    def get_option(self, key):
        return self.handles[0].get_option(key)

    def get(self, field):
        if field in PER_WORKER:
            return np.concatenate([h.get(field) for h in self.handles], axis=0)
        first = self.handles[0].get(field)
        for h in self.handles[1:]:                 # replicated state: every process must hold the same bits
            assert np.array_equal(h.get(field), first), f"replicas disagree on '{field}'"
        return first

    def set(self, field, value):
        for g, h in enumerate(self.handles):
            part = value[self.first[g]:self.first[g + 1]] if field in PER_WORKER else value
            h.set(field, np.ascontiguousarray(part))


def _workload(**over):
    from paper_2210_07454_b200 import synthetic
    w = synthetic.WORKLOADS["C1"]
    return synthetic.Workload(**{**w.__dict__, **over}) if over else w


def _exact_values(ora, e_before, variant):
    if variant == "pa":
        a = ora.field("m").astype(np.float64) / np.sqrt(ora.field("vhatw").astype(np.float64)) + e_before
        return a.mean(axis=0)
    a = ora.field("m").astype(np.float64) + e_before
    return a.mean(axis=0) / np.sqrt(ora.field("vhat").astype(np.float64))


def _run(w, split, steps, variant="ga", P=1, window_lines=None, cfg_id=None, lr_of=None, bf16=False):
    from paper_2210_07454_b200.synthetic import GradientSource
    ranks = Ranks(w, split, variant=variant, P=P, window_lines=window_lines)
    ora = oracle.Oracle(w.d, w.n, w.r, w.c, w.k, seed=w.seed, log2g=ranks.get_option("log2g"), lr=w.lr, beta1=w.beta1,
                        beta2=w.beta2, eps=w.eps, threads=8, window_lines=ranks.get_option("window_lines"),
                        variant=variant, P=P)
    src = GradientSource(w, device="cuda", cfg_id=cfg_id)
    x_ref = src.x0().cpu().numpy().copy()
    xs = [src.x0() for _ in split]
    for h in ranks.handles:
        h.set_option("grads_bf16", int(bf16))
    for t in range(1, steps + 1):
        g = src.grads(t)
        if bf16:
            g = g.to(torch.bfloat16)
        if lr_of is not None:
            ora.set_lr(lr_of(t))
            for h in ranks.handles:
                h.set_lr(lr_of(t))
        if t > 1:                                   # teacher forcing
            force_state(ranks, ora, variant)
            for x in xs:
                x.copy_(torch.from_numpy(x_ref))
        x_before = x_ref.astype(np.float64).copy()
        x_own = xs[0].cpu().numpy().copy()
        e_before = ora.field("e").astype(np.float64) if P > 1 else None
        members = ora.field("I_prev").astype(np.int64).copy()
        g_host = g.float().cpu().numpy()
        ranks.step(g, xs)
        ranks.sync()
        ora.step(g_host, x_ref)
        for x in xs[1:]:
            assert torch.equal(x, xs[0]), "the replicas of x disagree"
        compare_step(ranks, ora, xs[0].cpu().numpy(), x_ref, x_before, w.lr, x_gpu_before=x_own, variant=variant,
                     exact_ref=_exact_values(ora, e_before, variant) if P > 1 else None,
                     grads=g_host, members=members, beta2=w.beta2)
    return ranks


@pytest.mark.parametrize("split", [(4,), (2, 2), (1, 1, 1, 1), (1, 3)])
def test_c1_ten_steps(split):
    _run(_workload(), split, 10)


@pytest.mark.parametrize("P", [2, 4])
def test_c1_second_round(P):
    _run(_workload(), (2, 2), 6, P=P)


def test_c1_parameter_averaging():
    _run(_workload(), (2, 2), 6, variant="pa")
    _run(_workload(), (3, 1), 3, variant="pa", P=2)


def test_c1_sketch_of_the_local_worker_sum():
    # each process sketches the sum of its own workers once: the exchanged share of the mean sketch is the same vector
    from paper_2210_07454_b200 import synthetic  # noqa: F401
    w = _workload()
    from paper_2210_07454_b200.synthetic import GradientSource
    ranks = Ranks(w, (3, 1), P=2)
    for h in ranks.handles:
        h.set_option("sum_sketch", 1)
    ora = oracle.Oracle(w.d, w.n, w.r, w.c, w.k, seed=w.seed, log2g=ranks.get_option("log2g"), lr=w.lr, beta1=w.beta1,
                        beta2=w.beta2, eps=w.eps, threads=8, P=2, window_lines=ranks.get_option("window_lines"))
    src = GradientSource(w, device="cuda")
    x_ref = src.x0().cpu().numpy().copy()
    xs = [src.x0() for _ in ranks.handles]
    for t in range(1, 5):
        g = src.grads(t)
        if t > 1:
            force_state(ranks, ora, "ga")
            for x in xs:
                x.copy_(torch.from_numpy(x_ref))
        x_before = x_ref.astype(np.float64).copy()
        x_own = xs[0].cpu().numpy().copy()
        e_before = ora.field("e").astype(np.float64)
        members = ora.field("I_prev").astype(np.int64).copy()
        g_host = g.cpu().numpy()
        ranks.step(g, xs)
        ranks.sync()
        ora.step(g_host, x_ref)
        compare_step(ranks, ora, xs[0].cpu().numpy(), x_ref, x_before, w.lr, check_tables=False, x_gpu_before=x_own,
                     exact_ref=_exact_values(ora, e_before, "ga"), grads=g_host, members=members, beta2=w.beta2)


def test_c1_schedule_and_bf16_gradients():
    _run(_workload(), (2, 2), 6, P=2, lr_of=lambda t: float(np.float32(0.01 / np.sqrt(t))), bf16=True)


CASES = {
    "scalar_path": dict(d=10_007, n=3, r=5, c=1000, k=333, split=(2, 1)),
    "scalar_path_second_round": dict(d=10_007, n=3, r=5, c=1000, k=333, split=(1, 2), P=3),
    "k_eq_d": dict(d=2048, n=2, r=3, c=4096, k=2048, split=(1, 1)),
    "k_1": dict(d=20_000, n=4, r=5, c=1024, k=1, split=(2, 2), P=8),
    "many_rows_odd_c": dict(d=12_000, n=6, r=16, c=1001, k=120, split=(1, 2, 3)),
    "windowed_family": dict(d=40_960, n=6, r=5, c=4096, k=400, split=(4, 2), L=8),
    "more_than_one_scan_block": dict(d=1_200_000, n=2, r=3, c=8192, k=5000, split=(1, 1), P=2),
}


@pytest.mark.parametrize("case", sorted(CASES))
def test_edge_cases(case):
    cfg = dict(CASES[case])
    split, P, L = cfg.pop("split"), cfg.pop("P", 1), cfg.pop("L", None)
    w = _workload(name="E", steps=3, recipe="planted", **cfg)
    _run(w, split, 3, P=P, window_lines=L, cfg_id=7)


def test_integer_inputs_are_bit_exact_and_equal_the_unpartitioned_step():
    # integer gradients, beta1 = 0, eps = 1, n a power of two: every sum is exact whatever its order, so the
    # partitioned step must reproduce the oracle (and hence the one-call step) bit for bit
    d, n, r, c, k, P = 100_000, 4, 5, 2048, 500, 2
    from paper_2210_07454_b200 import synthetic
    w = synthetic.Workload("E", d, n, r, c, k, 1, "planted", seed=9, lr=0.5, beta1=0.0, beta2=0.5, eps=1.0)
    ranks = Ranks(w, (1, 2, 1), P=P)
    ora = oracle.Oracle(d, n, r, c, k, seed=9, log2g=ranks.get_option("log2g"), lr=0.5, beta1=0.0, beta2=0.5, eps=1.0,
                        threads=8, P=P, window_lines=ranks.get_option("window_lines"))
    gen = torch.Generator(device="cuda").manual_seed(5)
    xs = [torch.zeros(d, device="cuda") for _ in range(3)]
    x_ref = np.zeros(d, np.float32)
    for _ in range(3):
        g = torch.randint(-8, 9, (n, d), generator=gen, device="cuda").float()
        ranks.step(g, xs)
        ranks.sync()
        ora.step(g.cpu().numpy(), x_ref)
        assert np.array_equal(ranks.get("sum"), ora.field("sum"))
        assert np.array_equal(ranks.get("cand"), ora.field("cand"))
        assert np.array_equal(ranks.get("I"), ora.field("I"))
        assert np.array_equal(ranks.get("vhat"), ora.field("vhat"))
        assert np.array_equal(ranks.get("e"), ora.field("e"))
        assert np.array_equal(xs[0].cpu().numpy(), x_ref) and torch.equal(xs[0], xs[2])


def test_exchange_sizes_match_the_papers_count_and_calls_out_of_order_fail():
    from paper_2210_07454_b200 import binding
    d, n, r, c, k, P = 5000, 2, 3, 500, 40, 4
    h = binding.SketchedAMSGrad(d, n, r, c, k, P=P, workers_total=8)
    cs = (c + 31) // 32 * 32
    assert h.exchange_floats(1) == r * cs + k and h.exchange_floats(2) == P * k     # |S| + k + P*k (Section III-B)
    assert h.get_option("workers_total") == 8
    pa = binding.SketchedAMSGrad(d, n, r, c, k, variant="pa")
    assert pa.exchange_floats(1) == r * cs                                           # Algorithm 1 sends no h_t
    x1 = torch.zeros(h.exchange_floats(1), device="cuda")
    x2 = torch.zeros(h.exchange_floats(2), device="cuda")
    x = torch.zeros(d, device="cuda")
    g = torch.ones((n, d), device="cuda")
    with pytest.raises(binding.SkError):
        h.step_select(x1, x2)
    with pytest.raises(binding.SkError):
        h.step_finish(x2, x)
    h.step_local(g, x1)
    with pytest.raises(binding.SkError):
        h.step_local(g, x1)
    with pytest.raises(binding.SkError):
        h.step(g, x)                                # the one-call step may not cut into a partitioned one
    h.step_select(x1, x2)
    h.step_finish(x2, x)
    h.sync()
    with pytest.raises(binding.SkError):
        h.set_option("workers_total", 16)           # fixed after the first step
    with pytest.raises(binding.SkError):
        binding.SketchedAMSGrad(d, n, r, c, k, workers_total=1)      # fewer than the handle's own workers


def test_partitioned_driver_single_process():
    # the driver class with its default all-reduce (no process group: identity) against the one-call step
    from paper_2210_07454_b200 import binding
    from paper_2210_07454_b200.partitioned import PartitionedStep
    from paper_2210_07454_b200.synthetic import GradientSource
    w = _workload()
    a = binding.SketchedAMSGrad(w.d, w.n, w.r, w.c, w.k, seed=w.seed, lr=w.lr, eps=w.eps)
    b = binding.SketchedAMSGrad(w.d, w.n, w.r, w.c, w.k, seed=w.seed, lr=w.lr, eps=w.eps, workers_total=w.n)
    drv = PartitionedStep(b, "cuda")
    assert drv.floats_per_step == b.exchange_floats(1) + b.exchange_floats(2)
    src = GradientSource(w, device="cuda")
    xa, xb = src.x0(), src.x0()
    g = src.grads(1)
    a.step(g, xa)
    drv.step(g, xb)
    a.sync(), b.sync()
    # one process, same worker order: the same sums in the same order, hence the same bits
    assert np.array_equal(a.get("I"), b.get("I"))
    assert torch.equal(xa, xb)


def test_partitioned_driver_orders_a_side_stream_against_the_collective():
    # The handle launches on a stream of its own; the all-reduce is enqueued on torch's current stream.  Two processes
    # with identical workers are emulated: the sum over them is twice the local share (exact in fp32), and every
    # mean divides by 2n, so the result must be the bits of the n-worker one-call step.  Delays on both streams
    # widen the windows: a collective that starts before its phase has finished, or a phase that starts before the
    # collective has, would lose or repeat the doubling.
    from paper_2210_07454_b200 import binding
    from paper_2210_07454_b200.partitioned import PartitionedStep
    from paper_2210_07454_b200.synthetic import GradientSource
    w = _workload()
    side = torch.cuda.Stream()

    def doubled(t):
        torch.cuda._sleep(20_000_000)               # the collective is slow: the next phase has to wait for it
        t.mul_(2.0)

    a = binding.SketchedAMSGrad(w.d, w.n, w.r, w.c, w.k, seed=w.seed, lr=w.lr, eps=w.eps)
    b = binding.SketchedAMSGrad(w.d, w.n, w.r, w.c, w.k, seed=w.seed, lr=w.lr, eps=w.eps, workers_total=2 * w.n)
    drv = PartitionedStep(b, "cuda", all_reduce=doubled, stream=side)
    src = GradientSource(w, device="cuda")
    xa, xb, x0 = src.x0(), src.x0(), src.x0()
    for t in (1, 2):
        g = src.grads(t)
        a.step(g, xa)
        with torch.cuda.stream(side):
            torch.cuda._sleep(20_000_000)           # the handle's stream is busy: the phases start late
        drv.step(g, xb)
        torch.cuda.synchronize()
        a.sync(), b.sync()
        assert np.array_equal(a.get("I"), b.get("I")), t
        # equal up to the rounding of the gradient sums behind vhat, which both handles accumulate in arrival order;
        # a lost or repeated doubling would be off by a factor of two
        moved = float((xa - x0).abs().max())
        assert float((xa - xb).abs().max()) <= 1e-5 * moved, t
    b.set_stream(0)
