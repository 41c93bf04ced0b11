"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest

import oracle
from parity import close, compare_step, force_state, index_sets_agree

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _binding():
    from paper_2210_07454_b200 import binding
    return binding


def _source(w, device="cuda", cfg_id=None):
    from paper_2210_07454_b200.synthetic import GradientSource
    return GradientSource(w, device=device, cfg_id=cfg_id)


def _workload(base, **over):
    from paper_2210_07454_b200 import synthetic
    w = synthetic.WORKLOADS[base]
    if over:
        w = synthetic.Workload(**{**w.__dict__, **over})
    return w


def _pair(w, log2g=None, threads=8, window_lines=None, variant="ga", P=1, freeze_v=False, options=None):
    b = _binding()
    gpu = b.SketchedAMSGrad(w.d, w.n, w.r, w.c, w.k, seed=w.seed, lr=w.lr, beta1=w.beta1, beta2=w.beta2,
                            eps=w.eps, log2g=log2g, window_lines=window_lines, variant=variant, P=P)
    lg = gpu.get_option("log2g")
    ora = oracle.Oracle(w.d, w.n, w.r, w.c, w.k, seed=w.seed, log2g=lg, lr=w.lr, beta1=w.beta1, beta2=w.beta2,
                        eps=w.eps, threads=threads, window_lines=gpu.get_option("window_lines"), variant=variant, P=P, freeze_v=freeze_v)
    if freeze_v:
        gpu.set_option("freeze_v", 1)
    for key, value in (options or {}).items():
        gpu.set_option(key, value)
    return gpu, ora


# ------------------------------------------------------------------------------------------------ hash
@pytest.mark.parametrize("log2g", [0, 1, 2, 3, 4, 5])
@pytest.mark.parametrize("c", [2048, 250_000, 401])
def test_hash_bit_exact(log2g, c):
    b = _binding()
    d, r = 300_000, 7
    gpu = b.SketchedAMSGrad(d, 1, r, c, 1, seed=12345, log2g=log2g)
    L = gpu.get_option("window_lines")               # groups of 32 come with the windowed family by default
    idx = torch.empty(d, dtype=torch.int32, device="cuda")
    sgn = torch.empty(d, dtype=torch.int8, device="cuda")
    for row in range(r):
        gpu.hash(row, 0, d, idx, sgn)
        gpu.sync()
        wb, ws = oracle.hash_family(12345, log2g, c, row, 0, d, window_lines=L)
        assert np.array_equal(idx.cpu().numpy().view(np.uint32), wb)
        assert np.array_equal(sgn.cpu().numpy(), ws)
    # far end of the coordinate range
    gpu.hash(3, 2**32 - 1000, 1000, idx, sgn)
    gpu.sync()
    wb, ws = oracle.hash_family(12345, log2g, c, 3, 2**32 - 1000, 1000, window_lines=L)
    assert np.array_equal(idx[:1000].cpu().numpy().view(np.uint32), wb)
    assert np.array_equal(sgn[:1000].cpu().numpy(), ws)


# ------------------------------------------------------------------------------------------------ steps
def _exact_values(ora, e_before, variant):
    """What the second round ranks by: the preconditioned mean over the workers of a_t = (this step's m, scaled for
    Algorithm 1) + e_{t-1}, recomputed here from the oracle's state around the step."""
    if variant == "pa":
        a = ora.field("m").astype(np.float64) / np.sqrt(ora.field("vhatw").astype(np.float64)) + e_before
        return a.mean(axis=0)
    a = ora.field("m").astype(np.float64) + e_before
    return a.mean(axis=0) / np.sqrt(ora.field("vhat").astype(np.float64))


def _run_steps(w, steps, log2g=None, teacher=True, cfg_id=None, check_tables=True, window_lines=None, variant="ga",
               P=1, lr_of=None, freeze_v=False, bf16=False, options=None):
    """lr_of: step -> step size (a schedule); bf16: the GPU receives the gradients as bf16, the oracle the same
    values widened to fp32."""
    gpu, ora = _pair(w, log2g, window_lines=window_lines, variant=variant, P=P, freeze_v=freeze_v, options=options)
    if bf16:
        gpu.set_option("grads_bf16", 1)
    src = _source(w, cfg_id=cfg_id)
    x_gpu = src.x0()
    x_ref = x_gpu.cpu().numpy().copy()
    diverged_at = None
    for t in range(1, steps + 1):
        g = src.grads(t)
        if bf16:
            g = g.to(torch.bfloat16)
        g_host = g.float().cpu().numpy()
        if lr_of is not None:
            gpu.set_lr(lr_of(t))
            ora.set_lr(lr_of(t))
        if teacher and t > 1:
            force_state(gpu, ora, variant)
            x_gpu.copy_(torch.from_numpy(x_ref))
        x_before = x_ref.astype(np.float64).copy()
        x_gpu_before = x_gpu.cpu().numpy().copy()
        gpu.step(g, x_gpu)
        gpu.sync()
        e_before = ora.field("e").astype(np.float64) if P > 1 else None
        members = ora.field("I_prev").astype(np.int64).copy()
        ora.step(g_host, x_ref)
        diff = compare_step(gpu, ora, x_gpu.cpu().numpy(), x_ref, x_before, w.lr, check_tables=check_tables,
                            x_gpu_before=x_gpu_before, variant=variant,
                            exact_ref=_exact_values(ora, e_before, variant) if P > 1 else None,
                            grads=g_host, members=members, beta2=w.beta2)
        if diff.size and diverged_at is None:
            diverged_at = t
            if not teacher:
                break
    return diverged_at


def test_c1_ten_steps_teacher_forced():
    _run_steps(_workload("C1"), 10)


def test_c1_free_running():
    # without teacher forcing the trajectories may legitimately split once an in-band index flips;
    # until then every stage must agree (compare_step raises otherwise)
    _run_steps(_workload("C1"), 10, teacher=False)


@pytest.mark.parametrize("log2g", [0, 1, 2, 3, 4])
def test_c1_other_group_sizes(log2g):
    _run_steps(_workload("C1"), 3, log2g=log2g)


@pytest.mark.parametrize("L", [1, 4, 8, 16])
def test_windowed_hash_bit_exact(L):
    b = _binding()
    d, r, c = 300_000, 7, 250_000
    gpu = b.SketchedAMSGrad(d, 1, r, c, 1, seed=99, window_lines=L)
    idx = torch.empty(d, dtype=torch.int32, device="cuda")
    sgn = torch.empty(d, dtype=torch.int8, device="cuda")
    for row in (0, 3, 6):
        gpu.hash(row, 0, d, idx, sgn)
        gpu.sync()
        wb, ws = oracle.hash_family(99, 5, c, row, 0, d, window_lines=L)
        assert np.array_equal(idx.cpu().numpy().view(np.uint32), wb)
        assert np.array_equal(sgn.cpu().numpy(), ws)


def test_windowed_c1_ten_steps_teacher_forced():
    _run_steps(_workload("C1"), 10, window_lines=8)


WINDOWED = {
    "ragged_unit": dict(d=1024 * 37 + 12, n=4, r=7, c=3000, k=700, L=4),     # last unit partial, c % window != 0
    "two_launches": dict(d=40_000, n=11, r=5, c=4096, k=400, L=8),           # 8 + 3 workers
    "odd_workers": dict(d=50_000, n=5, r=5, c=4096, k=500, L=16),
    "one_window": dict(d=8192, n=2, r=3, c=300, k=80, L=8),                  # a single panel
    "many_rows": dict(d=12_000, n=2, r=16, c=2048, k=120, L=2),
    "short": dict(d=512, n=3, r=5, c=1024, k=20, L=4),                       # less than one unit
    "scalar_path": dict(d=10_007, n=3, r=5, c=1000, k=333, L=4),             # d % 4 != 0: scalar kernels, same family
}


@pytest.mark.parametrize("case", sorted(WINDOWED))
def test_windowed_edge_cases(case):
    cfg = dict(WINDOWED[case])
    L = cfg.pop("L")
    w = _workload("C1", name="E", steps=3, recipe="planted", **cfg)
    _run_steps(w, 3, cfg_id=8, window_lines=L)


@pytest.mark.parametrize("workers,worker_sum", [(1, 0), (2, 1), (3, 0), (5, 1), (8, 0)])
def test_windowed_worker_chunks_and_worker_sum(workers, worker_sum):
    # the ownership kernel runs one warp per worker: every split of the workers into launches (block sizes of
    # 32 .. 256 threads, running sums carried over launches), with and without the worker sum of a_t that the update
    # of x can read, must give the same step
    w = _workload("C1", name="E", d=1024 * 21 + 64, n=5, r=5, c=4096, k=300, steps=3, recipe="planted")
    gpu, ora = _pair(w, window_lines=8)
    gpu.set_option("window_workers", workers)
    gpu.set_option("worker_sum", worker_sum)
    src = _source(w, cfg_id=8)
    x = src.x0()
    x_ref = x.cpu().numpy().copy()
    for t in (1, 2, 3):
        g = src.grads(t)
        if t > 1:
            force_state(gpu, ora)
            x.copy_(torch.from_numpy(x_ref))
        xb = x_ref.astype(np.float64).copy()
        members = ora.field("I_prev").astype(np.int64).copy()
        g_host = g.cpu().numpy()
        gpu.step(g, x)
        gpu.sync()
        ora.step(g_host, x_ref)
        compare_step(gpu, ora, x.cpu().numpy(), x_ref, xb, w.lr, grads=g_host, members=members, beta2=w.beta2)


def test_windowed_integer_inputs_are_bit_exact():
    d, n, r, c, k = 200_000, 4, 5, 4096, 1000
    b = _binding()
    gpu = b.SketchedAMSGrad(d, n, r, c, k, seed=9, lr=0.5, beta1=0.0, beta2=0.5, eps=1.0, window_lines=8)
    ora = oracle.Oracle(d, n, r, c, k, seed=9, log2g=5, lr=0.5, beta1=0.0, beta2=0.5, eps=1.0, threads=8, window_lines=8)
    gen = torch.Generator(device="cuda").manual_seed(5)
    x = torch.zeros(d, device="cuda")
    x_ref = np.zeros(d, np.float32)
    g = torch.randint(-8, 9, (n, d), generator=gen, device="cuda").float()
    gpu.step(g, x)
    gpu.sync()
    ora.step(g.cpu().numpy(), x_ref)
    assert np.array_equal(gpu.get("tables"), ora.field("tables"))
    assert np.array_equal(gpu.get("sum"), ora.field("sum"))
    assert np.array_equal(gpu.get("I"), ora.field("I"))
    assert np.array_equal(x.cpu().numpy(), x_ref)


EDGE = {
    "k1": dict(d=4096, n=2, r=3, c=512, k=1),
    "k_eq_d": dict(d=2048, n=2, r=3, c=4096, k=2048),
    "r1_n1": dict(d=8192, n=1, r=1, c=1024, k=100),
    "d_odd": dict(d=10_007, n=3, r=5, c=1000, k=333),          # scalar kernels: d % 4 != 0, c % 32 != 0
    "c_odd": dict(d=20_000, n=3, r=5, c=401, k=200),
    "r_even": dict(d=30_000, n=2, r=10, c=2048, k=300),        # lower median
    "r16": dict(d=12_000, n=2, r=16, c=1024, k=120),           # run-time row count
    "r9": dict(d=12_000, n=2, r=9, c=1024, k=120),
    "n_odd_tail": dict(d=50_000, n=5, r=5, c=4096, k=500),     # odd worker count: the pair loop's tail
    "tiny": dict(d=4, n=1, r=1, c=32, k=2),
    "ragged_tile": dict(d=1024 * 37 + 12, n=4, r=7, c=3000, k=700),
}


@pytest.mark.parametrize("case", sorted(EDGE))
def test_edge_cases(case):
    w = _workload("C1", name="E", steps=3, recipe="planted", **EDGE[case])
    _run_steps(w, 3, cfg_id=7)


# ---------------------------------------------------------------------------- parameter averaging (Algorithm 1)
def test_pa_c1_ten_steps_teacher_forced():
    _run_steps(_workload("C1"), 10, variant="pa")


PA_CASES = {
    "scalar_path": dict(d=10_007, n=3, r=5, c=1000, k=333),
    "rows16_odd_workers": dict(d=12_000, n=5, r=16, c=1024, k=120),
    "even_rows": dict(d=30_000, n=2, r=10, c=2048, k=300),
    "k_eq_d": dict(d=2048, n=2, r=3, c=4096, k=2048),
    "windowed_family": dict(d=40_000, n=6, r=5, c=4096, k=400, L=8),   # Algorithm 1 on the windowed hash family
}


@pytest.mark.parametrize("case", sorted(PA_CASES))
def test_pa_edge_cases(case):
    cfg = dict(PA_CASES[case])
    L = cfg.pop("L", None)
    w = _workload("C1", name="E", steps=3, recipe="planted", **cfg)
    _run_steps(w, 3, cfg_id=7, variant="pa", window_lines=L)


def test_pa_state_fields_and_errors():
    b = _binding()
    ga = b.SketchedAMSGrad(1000, 2, 3, 256, 10)
    with pytest.raises(b.SkError):
        ga.get("vw")                                  # per-worker second moments exist only for Algorithm 1
    pa = b.SketchedAMSGrad(1000, 2, 3, 256, 10, variant="pa", eps=1e-3)
    assert np.all(pa.get("vw") == np.float32(1e-3)) and np.all(pa.get("vhatw") == np.float32(1e-3))
    with pytest.raises(b.SkError):
        pa.get("vhat")
    x = torch.zeros(1000, device="cuda")
    pa.step(torch.ones((2, 1000), device="cuda"), x)
    with pytest.raises(b.SkError):
        pa.set_option("variant", 0)                   # fixed after the first step
    assert pa.algorithmic_bytes() == 36 * 2 * 1000 + 8 * 2 * 3 * 256 + 4 * 3 * 256 + 8 * 2 * 10 + 8 * 10


# ------------------------------------------------------------- second round of the selection (Section III-A, P > 1)
@pytest.mark.parametrize("P", [2, 4])
def test_second_round_c1_ten_steps_teacher_forced(P):
    _run_steps(_workload("C1"), 10, P=P)


SECOND_ROUND = {
    "scalar_path": dict(d=10_007, n=3, r=5, c=1000, k=333, P=3),
    "candidates_are_everything": dict(d=4096, n=2, r=3, c=512, k=1024, P=4),       # P*k = d
    "k_1": dict(d=20_000, n=4, r=5, c=1024, k=1, P=8),
    "tiny_sketch_many_candidates": dict(d=50_000, n=4, r=3, c=256, k=500, P=16),   # estimates nearly useless
    "pa": dict(d=30_000, n=3, r=5, c=2048, k=300, P=2, variant="pa"),
    "windowed_family": dict(d=40_000, n=6, r=5, c=4096, k=400, P=2, L=8),
}


@pytest.mark.parametrize("case", sorted(SECOND_ROUND))
def test_second_round_edge_cases(case):
    cfg = dict(SECOND_ROUND[case])
    P, L, variant = cfg.pop("P"), cfg.pop("L", None), cfg.pop("variant", "ga")
    w = _workload("C1", name="E", steps=3, recipe="planted", **cfg)
    _run_steps(w, 3, cfg_id=7, variant=variant, window_lines=L, P=P)


@pytest.mark.parametrize("chunk", [0, 1, 3])
def test_second_round_integer_inputs_are_bit_exact(chunk):
    # integer gradients, beta1 = 0 and eps = 1: estimates and exact values are exact small rationals with ties
    # everywhere, so the candidates and the final set must match the oracle index for index
    d, n, r, c, k, P = 100_000, 4, 5, 2048, 500, 4
    b = _binding()
    gpu = b.SketchedAMSGrad(d, n, r, c, k, seed=9, lr=0.5, beta1=0.0, beta2=0.5, eps=1.0, P=P)
    ora = oracle.Oracle(d, n, r, c, k, seed=9, log2g=gpu.get_option("log2g"), lr=0.5, beta1=0.0, beta2=0.5, eps=1.0,
                        threads=8, P=P, window_lines=gpu.get_option("window_lines"))
    gpu.set_option("worker_chunk", chunk)            # workers in several launches: the running sums carry over
    gen = torch.Generator(device="cuda").manual_seed(5)
    x = torch.zeros(d, device="cuda")
    x_ref = np.zeros(d, np.float32)
    g = torch.randint(-8, 9, (n, d), generator=gen, device="cuda").float()
    gpu.step(g, x)
    gpu.sync()
    ora.step(g.cpu().numpy(), x_ref)
    assert np.array_equal(gpu.get("cand"), ora.field("cand"))
    assert np.array_equal(gpu.get("I"), ora.field("I"))
    assert np.array_equal(gpu.get("e"), ora.field("e"))
    assert np.array_equal(x.cpu().numpy(), x_ref)


def test_second_round_option_errors():
    b = _binding()
    with pytest.raises(b.SkError):
        b.SketchedAMSGrad(1000, 2, 3, 256, 400, P=3)          # P*k > d
    with pytest.raises(b.SkError):
        b.SketchedAMSGrad(1000, 2, 3, 256, 10, P=0)
    gpu = b.SketchedAMSGrad(1000, 2, 3, 256, 10, P=2)
    assert gpu.get_option("P") == 2 and gpu.get("cand").size == 0
    x = torch.zeros(1000, device="cuda")
    gpu.step(torch.ones((2, 1000), device="cuda"), x)
    assert gpu.get("cand").size == 20
    with pytest.raises(b.SkError):
        gpu.set_option("P", 1)                                # fixed after the first step
    with pytest.raises(b.SkError):
        gpu.select_static(torch.empty(10, dtype=torch.int32, device="cuda"))


# ------------------------------------------- step-size schedule, frozen second moments, bf16 gradients (flags)
def _inv_sqrt(t):
    return float(np.float32(0.01 / np.sqrt(t)))             # Theorem 2's alpha_t = alpha / sqrt(t)


FLAG_CASES = {
    "schedule": dict(lr_of=_inv_sqrt),
    "schedule_free_running": dict(lr_of=_inv_sqrt, teacher=False),
    "schedule_growing_steps": dict(lr_of=lambda t: 1e-3 * 2 ** (t % 3)),     # ratios below and above one
    "schedule_pa": dict(lr_of=_inv_sqrt, variant="pa"),
    "schedule_windowed": dict(lr_of=_inv_sqrt, window_lines=4),
    "schedule_second_round": dict(lr_of=_inv_sqrt, P=2),
    "frozen": dict(freeze_v=True),
    "frozen_schedule_second_round": dict(freeze_v=True, lr_of=_inv_sqrt, P=2),
    "bf16": dict(bf16=True),
    "bf16_pa": dict(bf16=True, variant="pa"),
    "bf16_windowed": dict(bf16=True, window_lines=4),
}


@pytest.mark.parametrize("case", sorted(FLAG_CASES))
def test_flags_c1_steps(case):
    _run_steps(_workload("C1"), 8, **FLAG_CASES[case])


@pytest.mark.parametrize("case", ["schedule", "bf16", "frozen"])
def test_flags_scalar_path(case):
    w = _workload("C1", name="E", steps=4, recipe="planted", d=10_007, n=3, r=5, c=1000, k=333)
    _run_steps(w, 4, cfg_id=7, **FLAG_CASES[case])


def test_frozen_second_moments_keep_v_and_its_decay_clock():
    # v and vhat must not move while frozen (not even the lazy decay), and resume exactly where they were
    w = _workload("C1", name="E", d=30_000, n=2, r=5, c=2048, k=300, steps=9)
    gpu, ora = _pair(w)
    src = _source(w, cfg_id=5)
    x = src.x0()
    x_ref = x.cpu().numpy().copy()
    for t in range(1, 10):
        frozen = 4 <= t <= 6
        gpu.set_option("freeze_v", int(frozen))
        ora.set_freeze_v(frozen)
        g = src.grads(t)
        v_before, vhat_before = gpu.get("v"), gpu.get("vhat")
        gpu.step(g, x)
        ora.step(g.cpu().numpy(), x_ref)
        if np.setxor1d(gpu.get("I"), ora.field("I")).size:
            break
        if frozen:
            assert np.array_equal(gpu.get("v"), v_before) and np.array_equal(gpu.get("vhat"), vhat_before)
        np.testing.assert_allclose(gpu.get("v"), ora.field("v"), rtol=1e-5, atol=0)
        close(gpu.get("vhat"), ora.field("vhat"), "vhat")
    else:
        return
    pytest.fail("the index sets split before the frozen window was over")


def test_flag_errors_and_bf16_host_step():
    b = _binding()
    gpu = b.SketchedAMSGrad(4000, 2, 3, 256, 20, lr=0.01)
    with pytest.raises(b.SkError):
        gpu.set_lr(float("nan"))
    with pytest.raises(b.SkError):
        gpu.set_lr(0.0)                                       # no ratio alpha_{t-1}/alpha_t with a zero step size
    pa = b.SketchedAMSGrad(4000, 2, 3, 256, 20, variant="pa")
    with pytest.raises(b.SkError):
        pa.set_option("freeze_v", 1)                          # Algorithm 2 only
    # host entry point with bf16 gradients against the device entry point
    gpu.set_option("grads_bf16", 1)
    other = b.SketchedAMSGrad(4000, 2, 3, 256, 20, lr=0.01)
    other.set_option("grads_bf16", 1)
    assert gpu.algorithmic_bytes() == other.algorithmic_bytes() == 18 * 2 * 4000 + 4 * 4000 + 8 * 2 * 3 * 256 \
        + 4 * 3 * 256 + 12 * 2 * 20 + 24 * 20
    g = (torch.randn((2, 4000), device="cuda") * 0.1).to(torch.bfloat16)
    x_dev = torch.zeros(4000, device="cuda")
    x_host = np.zeros(4000, np.float32)
    gpu.step(g, x_dev)
    other.step_host(g.cpu().view(torch.int16).numpy(), x_host)
    gpu.sync()
    assert np.array_equal(gpu.get("I"), other.get("I"))
    np.testing.assert_allclose(x_host, x_dev.cpu().numpy(), rtol=1e-6, atol=1e-9)


# -------------------------------------------- one sketch of the worker sum instead of n sketches (option sum_sketch)
SUM_SKETCH = {
    "c1": dict(),
    "c1_second_round": dict(P=2),
    "c1_pa": dict(variant="pa"),
    "c1_windowed_family": dict(window_lines=4),                 # the family, with the reduction kernel
    "c1_schedule_bf16": dict(lr_of=_inv_sqrt, bf16=True),
    "chunked_workers": dict(over=dict(d=30_000, n=7, r=16, c=1001, k=300), options={"worker_chunk": 3}),
    "chunked_workers_second_round": dict(over=dict(d=40_000, n=6, r=5, c=2048, k=400), options={"worker_chunk": 4}, P=3),
    "scalar_path": dict(over=dict(d=10_007, n=3, r=5, c=1000, k=333)),
}


@pytest.mark.parametrize("case", sorted(SUM_SKETCH))
def test_sketch_of_the_worker_sum(case):
    cfg = dict(SUM_SKETCH[case])
    over = cfg.pop("over", None)
    options = dict(cfg.pop("options", {}), sum_sketch=1)
    w = _workload("C1", name="E", steps=4, recipe="planted", **over) if over else _workload("C1")
    _run_steps(w, 4, cfg_id=7 if over else None, options=options, check_tables=False, **cfg)


def test_sketch_of_the_worker_sum_integer_inputs_bit_exact():
    d, n, r, c, k = 200_000, 4, 5, 4096, 1000
    b = _binding()
    gpu = b.SketchedAMSGrad(d, n, r, c, k, seed=9, lr=0.5, beta1=0.0, beta2=0.5, eps=1.0)
    gpu.set_option("sum_sketch", 1)
    ora = oracle.Oracle(d, n, r, c, k, seed=9, log2g=gpu.get_option("log2g"), lr=0.5, beta1=0.0, beta2=0.5, eps=1.0,
                        threads=8, window_lines=gpu.get_option("window_lines"))
    gen = torch.Generator(device="cuda").manual_seed(5)
    x = torch.zeros(d, device="cuda")
    x_ref = np.zeros(d, np.float32)
    for step in range(2):
        g = torch.randint(-8, 9, (n, d), generator=gen, device="cuda").float()
        gpu.step(g, x)
        gpu.sync()
        ora.step(g.cpu().numpy(), x_ref)
        assert np.array_equal(gpu.get("sum"), ora.field("sum"))       # n = 4: every quotient and sum is exact
        assert np.array_equal(gpu.get("I"), ora.field("I"))
        assert np.array_equal(gpu.get("e"), ora.field("e"))
        if step == 0:                                                  # vhat = 1 still: the update is exact too
            assert np.array_equal(x.cpu().numpy(), x_ref)
        x.copy_(torch.from_numpy(x_ref))
    with pytest.raises(b.SkError):
        gpu.get("tables")                                              # not formed in this mode
    assert gpu.algorithmic_bytes() == 20 * n * d + 4 * d + 8 * r * c + 12 * n * k + 24 * k


def test_worker_chunking_matches_single_pass():
    w = _workload("C1", name="E", d=40_000, n=6, r=5, c=2048, k=400)
    b = _binding()
    src = _source(w, cfg_id=6)
    outs = []
    for chunk in (0, 1, 4):
        gpu = b.SketchedAMSGrad(w.d, w.n, w.r, w.c, w.k, seed=3)
        gpu.set_option("worker_chunk", chunk)
        x = src.x0()
        for t in (1, 2):
            gpu.step(src.grads(t), x)
        gpu.sync()
        outs.append((gpu.get("tables"), gpu.get("I"), x.cpu().numpy()))
    for o in outs[1:]:
        close(o[0], outs[0][0], "tables under chunking", groups_axis=1)


def test_integer_inputs_are_bit_exact():
    # small-integer gradients and beta1 = 0 make every sum exact in fp32, whatever the order of the atomic adds:
    # a lost or doubled update would show as a wrong integer
    d, n, r, c, k = 200_000, 4, 5, 4096, 1000
    b = _binding()
    gpu = b.SketchedAMSGrad(d, n, r, c, k, seed=9, lr=0.5, beta1=0.0, beta2=0.5, eps=1.0)
    ora = oracle.Oracle(d, n, r, c, k, seed=9, log2g=gpu.get_option("log2g"), lr=0.5, beta1=0.0, beta2=0.5, eps=1.0,
                        threads=8, window_lines=gpu.get_option("window_lines"))
    gen = torch.Generator(device="cuda").manual_seed(5)
    x = torch.zeros(d, device="cuda")
    x_ref = np.zeros(d, np.float32)
    g = torch.randint(-8, 9, (n, d), generator=gen, device="cuda").float()
    gpu.step(g, x)
    gpu.sync()
    ora.step(g.cpu().numpy(), x_ref)
    assert np.array_equal(gpu.get("tables"), ora.field("tables"))
    assert np.array_equal(gpu.get("m"), ora.field("m"))
    # n = 4: the mean of four integer tables is exact too
    assert np.array_equal(gpu.get("sum"), ora.field("sum"))
    assert np.array_equal(gpu.get("est"), ora.field("est"))
    assert np.array_equal(gpu.get("I"), ora.field("I"))       # ties are everywhere here: smaller index must win
    assert np.array_equal(gpu.get("e"), ora.field("e"))
    assert np.array_equal(x.cpu().numpy(), x_ref)


@pytest.mark.parametrize("kw", [dict(), dict(window_lines=0), dict(variant="pa"), dict(P=4), dict(window_lines=0, P=2)],
                         ids=["default", "plain_family", "parameter_averaging", "second_round", "plain_second_round"])
def test_chained_and_plain_launches_give_the_same_bits(kw):
    # The step's kernels are launched chained (each may become resident while its predecessor still runs and waits
    # for it before touching global memory).  With integer gradients every sum is exact whatever the order of the
    # atomic adds, so three steps with and without chaining must agree bit for bit; a kernel that read or wrote
    # ahead of its predecessor would not.
    d, n, r, c, k = 150_016, 4, 5, 4096, 800
    b = _binding()
    gen = torch.Generator(device="cuda").manual_seed(23)
    grads = [torch.randint(-8, 9, (n, d), generator=gen, device="cuda").float() for _ in range(3)]
    results = []
    for chained in (1, 0):
        gpu = b.SketchedAMSGrad(d, n, r, c, k, seed=4, lr=0.5, beta1=0.0, beta2=0.5, eps=1.0, **kw)
        gpu.set_option("chained_launches", chained)
        assert gpu.get_option("chained_launches") == chained
        x = torch.zeros(d, device="cuda")
        for g in grads:
            gpu.step(g, x)
        gpu.sync()
        results.append({f: gpu.get(f) for f in ("tables", "sum", "m", "e", "I", "keys")} | {"x": x.cpu().numpy()})
        if kw.get("variant") != "pa":
            results[-1]["v"] = gpu.get("v")
            results[-1]["vhat"] = gpu.get("vhat")
    exact = kw.get("variant") != "pa"      # Algorithm 1 sketches m / sqrt(vhat): not integers, the add order shows
    for f, a in results[0].items():
        b_ = results[1][f]
        if exact:
            if f == "I":
                a, b_ = np.sort(a), np.sort(b_)
            assert np.array_equal(a, b_), f
        elif f in ("tables", "sum", "m"):
            assert np.allclose(a, b_, rtol=1e-5, atol=1e-5), f


def test_all_zero_gradients_select_lowest_indices():
    d, n, r, c, k = 50_000, 2, 5, 1024, 77
    b = _binding()
    gpu = b.SketchedAMSGrad(d, n, r, c, k)
    x = torch.ones(d, device="cuda")
    gpu.step(torch.zeros((n, d), device="cuda"), x)
    gpu.sync()
    assert np.array_equal(gpu.get("I"), np.arange(k, dtype=np.uint32))
    assert torch.equal(x, torch.ones(d, device="cuda"))


def test_lazy_v_decay_over_steps():
    w = _workload("C1", name="E", d=30_000, n=2, r=5, c=2048, k=300, steps=8)
    gpu, ora = _pair(w)
    src = _source(w, cfg_id=5)
    x = src.x0()
    x_ref = x.cpu().numpy().copy()
    ever = np.zeros(w.d, bool)
    for t in range(1, 9):
        g = src.grads(t)
        prev = ora.field("I_prev").copy()
        gpu.step(g, x)
        ora.step(g.cpu().numpy(), x_ref)
        if np.setxor1d(gpu.get("I"), ora.field("I")).size:
            break
        ever[prev] = True
        # a coordinate that has never been selected has only decayed: one fp32 multiply per step on both sides
        assert np.array_equal(gpu.get("v")[~ever], ora.field("v")[~ever])
        # v is a sum of non-negative terms: no cancellation, so the bound is relative to each element
        np.testing.assert_allclose(gpu.get("v"), ora.field("v"), rtol=1e-5, atol=0)
        close(gpu.get("vhat"), ora.field("vhat"), "vhat")


def test_lazy_v_after_a_long_gap_between_selections():
    # A coordinate selected at steps 1-2 and then not again until step 40 owes 37 decays when it is next updated.  The
    # hot path applies them as beta2^owed by square-and-multiply (a few ulp from the chain of single multiplies the
    # export applies): v on the re-selected coordinates must still agree with the oracle to 1e-5 of each element.
    d, n, r, c, k = 8192, 2, 5, 1024, 32
    b = _binding()
    gpu = b.SketchedAMSGrad(d, n, r, c, k, seed=3, lr=1e-3, beta1=0.0, beta2=0.99, eps=1e-2)
    ora = oracle.Oracle(d, n, r, c, k, seed=3, log2g=gpu.get_option("log2g"), lr=1e-3, beta1=0.0, beta2=0.99, eps=1e-2,
                        threads=4, window_lines=gpu.get_option("window_lines"))
    rng = np.random.default_rng(5)
    set_a = rng.choice(d, k, replace=False)
    set_b = np.setdiff1d(rng.choice(d, 3 * k, replace=False), set_a)[:k]
    x = torch.zeros(d, device="cuda")
    x_ref = np.zeros(d, np.float32)
    for t in range(1, 43):
        g = (rng.standard_normal((n, d)) * 1e-4).astype(np.float32)
        hot = set_a if t in (1, 2, 40, 41, 42) else set_b
        g[:, hot] += rng.uniform(0.5, 1.0, (n, k)).astype(np.float32)     # same sign on every worker: a large mean
        gpu.step(torch.from_numpy(g).cuda(), x)
        gpu.sync()
        ora.step(g, x_ref)
        assert np.array_equal(gpu.get("I"), ora.field("I")), t     # the planted coordinates decide the selection
    assert len(np.intersect1d(set_a, ora.field("I"))) >= k - 4     # ... up to the few the sketch loses to collisions
    np.testing.assert_allclose(gpu.get("v"), ora.field("v"), rtol=1e-5, atol=0)
    np.testing.assert_allclose(gpu.get("vhat"), ora.field("vhat"), rtol=1e-5, atol=0)


def test_checkpoint_roundtrip():
    w = _workload("C1", name="E", d=20_000, n=3, r=5, c=2048, k=200)
    b = _binding()
    src = _source(w, cfg_id=4)
    a = b.SketchedAMSGrad(w.d, w.n, w.r, w.c, w.k, seed=1)
    xa = src.x0()
    for t in (1, 2, 3):
        a.step(src.grads(t), xa)
    a.sync()
    c2 = b.SketchedAMSGrad(w.d, w.n, w.r, w.c, w.k, seed=1)
    c2.set("t", a.get("t"))
    for f in ("m", "e", "v", "vhat", "I"):
        c2.set(f, a.get(f))
    xb = xa.clone()
    a.step(src.grads(4), xa)
    c2.step(src.grads(4), xb)
    a.sync(); c2.sync()
    assert np.array_equal(a.get("I"), c2.get("I"))
    close(xb.cpu().numpy(), xa.cpu().numpy(), "x after resume")
    close(c2.get("e"), a.get("e"), "e after resume", groups_axis=0)
    # the gradient sums behind v are accumulated in arrival order (as the sketch tables are): equal to rounding
    np.testing.assert_allclose(c2.get("v"), a.get("v"), rtol=1e-6, atol=0)


def test_host_step_matches_device_step():
    w = _workload("C1", name="E", d=16_384, n=2, r=5, c=1024, k=100)
    b = _binding()
    src = _source(w, cfg_id=3)
    a = b.SketchedAMSGrad(w.d, w.n, w.r, w.c, w.k)
    h = b.SketchedAMSGrad(w.d, w.n, w.r, w.c, w.k)
    xa = src.x0()
    xh = xa.cpu().numpy().copy()
    for t in (1, 2):
        g = src.grads(t)
        a.step(g, xa)
        h.step_host(g.cpu().numpy(), xh)
    a.sync()
    assert np.array_equal(a.get("I"), h.get("I"))
    close(xh, xa.cpu().numpy(), "x via host entry point")


def test_sparse_host_step_matches_device_step():
    # parameters resident on the device, host gradients in, (index, new value) pairs out: applying the pairs to a
    # host copy of x must reproduce the device step, step after step
    w = _workload("C1", name="E", d=40_000, n=5, r=5, c=2048, k=400)
    b = _binding()
    src = _source(w, cfg_id=4)
    dev = b.SketchedAMSGrad(w.d, w.n, w.r, w.c, w.k, seed=2, lr=w.lr)
    host = b.SketchedAMSGrad(w.d, w.n, w.r, w.c, w.k, seed=2, lr=w.lr)
    x_dev = src.x0()
    x_host = x_dev.cpu().numpy().copy()
    host.set("x", x_host)
    idx = np.empty(w.k, np.uint32)
    val = np.empty(w.k, np.float32)
    for t in range(1, 5):
        g = src.grads(t)
        dev.step(g, x_dev)
        host.step_host_sparse(g.cpu().numpy(), idx, val)
        dev.sync()
        assert np.array_equal(np.sort(idx), host.get("I")) and np.array_equal(host.get("I"), dev.get("I"))
        x_host[idx] = val
        np.testing.assert_allclose(x_host, x_dev.cpu().numpy(), rtol=1e-6, atol=1e-9)
        assert np.array_equal(host.get("x"), x_host)           # the device-resident parameters are the same vector
    # the dense host step shares those parameters
    xh = x_host.copy()
    host.step_host(src.grads(5).cpu().numpy(), xh)
    assert np.array_equal(host.get("x"), xh)


def test_argument_errors():
    b = _binding()
    with pytest.raises(b.SkError):
        b.SketchedAMSGrad(100, 1, 5, 64, 101)          # k > d
    with pytest.raises(b.SkError):
        b.SketchedAMSGrad(100, 1, 17, 64, 10)          # r > 16
    with pytest.raises(b.SkError):
        b.SketchedAMSGrad(100, 1, 5, 64, 10, eps=0.0)
    s = b.SketchedAMSGrad(100, 1, 5, 64, 10)
    with pytest.raises(b.SkError):
        s.set_option("log2g", 7)
    with pytest.raises(b.SkError):
        s.get("nope")
    with pytest.raises(b.SkError):
        s.set("I", np.array([100], np.uint32))          # index >= d
    x = torch.zeros(100, device="cuda")
    s.step(torch.zeros((1, 100), device="cuda"), x)
    with pytest.raises(b.SkError):
        s.set_option("log2g", 2)                        # hash family is fixed after the first step
