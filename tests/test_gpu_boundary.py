"""Boundary behaviour of the C ABI that needs a device: allocation failure, statistics, test hooks."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def test_allocation_failure_returns_null_with_a_message_and_leaks_nothing():
    from paper_2210_07454_b200 import binding
    L = binding.lib()
    torch.cuda.synchronize()
    warm = binding.SketchedAMSGrad(50_000, 2, 5, 1024, 100)          # context, module and allocator pools are up
    warm.close()
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    try:
        for nth in (0, 3, 9, 15):                                   # the first, some middle, and a late allocation
            L.sk_test_fail_allocation(nth)
            with pytest.raises(binding.SkError, match="cudaMalloc of .* bytes failed"):
                binding.SketchedAMSGrad(50_000, 2, 5, 1024, 100)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free_before, nth  # everything allocated before the failure was freed
    finally:
        L.sk_test_fail_allocation(-1)
    ok = binding.SketchedAMSGrad(50_000, 2, 5, 1024, 100)            # and the library is usable afterwards
    ok.close()


def test_statistics_of_a_step():
    from paper_2210_07454_b200 import binding, synthetic
    w = synthetic.WORKLOADS["C1"]
    src = synthetic.GradientSource(w, device="cuda")
    opt = binding.SketchedAMSGrad(w.d, w.n, w.r, w.c, w.k)
    with pytest.raises(binding.SkError, match="no step"):
        opt.stats()
    x = src.x0()
    opt.step(src.grads(1), x)
    opt.sync()
    st = opt.stats()
    assert st["emitted"] == w.k and st["status"] == 0
    assert st["floats_on_the_wire"] == w.r * w.c + w.k + 2 * w.k     # Section III-B's count with P = 1
    keys = opt.get("keys").view(np.float32)
    kth = np.sort(keys)[-w.k]                                        # the k-th largest ranking key
    assert st["threshold"] <= kth <= st["threshold"] * (1 + 2.0 ** -15)
    assert st["threshold_bin_count"] >= st["tie_group_count"] >= 1


def test_the_normal_build_has_no_device_checks_to_trigger():
    from paper_2210_07454_b200 import binding
    opt = binding.SketchedAMSGrad(4096, 1, 3, 256, 16)
    with pytest.raises(binding.SkError, match="no device-side checks"):
        opt.debug_check(1)
