"""The allocation-free selection entry point against the regular one.

sk_select_static exists for callers that cannot allocate device memory when they need a selection (a foreign
caching allocator owns the device, cudaMalloc's implicit synchronisation is not affordable, or the device is
full).  It must return exactly the index set the last sk_step selected, from the same inputs, using only the
static scratch array inside the library -- also on a second call, when that array still holds the first call's
leftovers, and for a second handle that shares the array.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _setup(d, n, r, c, k, seed, cfg_id, **kw):
    from paper_2210_07454_b200 import binding, synthetic
    w = synthetic.Workload("E", d, n, r, c, k, 3, "planted")
    src = synthetic.GradientSource(w, device="cuda", cfg_id=cfg_id)
    opt = binding.SketchedAMSGrad(d, n, r, c, k, seed=seed, **kw)
    return binding, src, opt


def _free_bytes():
    torch.cuda.synchronize()
    return torch.cuda.mem_get_info()[0]


def test_static_selection_matches_step_twice_in_a_row():
    binding, src, opt = _setup(65_536, 4, 5, 2_048, 512, seed=0, cfg_id=1)
    _, src2, opt2 = _setup(100_000, 2, 7, 4_096, 3_000, seed=5, cfg_id=2, window_lines=8)
    x, x2 = src.x0(), src2.x0()
    out = torch.full((opt.k,), -1, dtype=torch.int32, device="cuda")
    out2 = torch.full((opt2.k,), -1, dtype=torch.int32, device="cuda")
    for t in (1, 2):                                    # two calls in a row, the second on a dirty scratch array
        opt.step(src.grads(t), x)
        opt2.step(src2.grads(t), x2)
        opt.sync(); opt2.sync()
        want, want2 = opt.get("I"), opt2.get("I")
        free_before = _free_bytes()
        opt.select_static(out)
        opt.sync()                                      # calls share the scratch: never let two overlap
        opt2.select_static(out2)
        opt2.sync()
        # "allocates nothing", measured: the device's free memory is the same before and after the calls
        assert _free_bytes() == free_before
        got = np.sort(out.cpu().numpy().view(np.uint32))
        got2 = np.sort(out2.cpu().numpy().view(np.uint32))
        assert np.array_equal(got, want)                # index work: bit-exact, not a tolerance
        assert np.array_equal(got2, want2)
    # the handle's own state was only read
    assert np.array_equal(opt.get("I"), want)


@pytest.mark.parametrize("case", ["scalar_kernels", "parameter_averaging", "plain_family"])
def test_static_selection_on_the_other_kernel_paths(case):
    # d not a multiple of 4 runs the scalar kernels; Algorithm 1 ranks without vhat; window_lines = 0 is the plain
    # hash family.  Two calls in a row on each, the scratch array dirty from whatever ran before.
    kw = {"scalar_kernels": dict(d=30_001), "parameter_averaging": dict(variant="pa"), "plain_family": dict(window_lines=0)}[case]
    d = kw.pop("d", 40_000)
    binding, src, opt = _setup(d, 3, 5, 1_024, 300, seed=3, cfg_id=4, **kw)
    x = src.x0()
    out = torch.full((opt.k,), -1, dtype=torch.int32, device="cuda")
    for t in (1, 2):
        opt.step(src.grads(t), x)
        opt.sync()
        want = opt.get("I")
        free_before = _free_bytes()
        opt.select_static(out)
        opt.sync()
        assert _free_bytes() == free_before
        assert np.array_equal(np.sort(out.cpu().numpy().view(np.uint32)), want)


def test_static_selection_rejects_what_it_cannot_hold():
    binding, src, opt = _setup(binding_max_d() + 4, 1, 3, 1_024, 16, seed=1, cfg_id=3)
    out = torch.zeros(16, dtype=torch.int32, device="cuda")
    x = src.x0()
    opt.step(src.grads(1), x)
    with pytest.raises(binding.SkError, match="SK_STATIC_MAX_D"):
        opt.select_static(out)
    _, src3, fresh = _setup(4_096, 1, 3, 1_024, 16, seed=1, cfg_id=3)
    with pytest.raises(binding.SkError, match="no step"):
        fresh.select_static(out)


def binding_max_d():
    from paper_2210_07454_b200 import binding
    return binding.STATIC_MAX_D
