"""Parity at the full benchmark sizes, in the launch configuration bench.py times (default options).

C2 and C3: two teacher-forced steps against the full oracle.  C4 and C5: the first step against the full oracle
(every stage, every element), then a second GPU step checked through properties that hold at any size.
"""
import numpy as np
import pytest

import oracle
from parity import compare_step, force_state

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _setup(name, window_lines=None, variant="ga", P=1):
    from paper_2210_07454_b200 import binding, synthetic
    w = synthetic.WORKLOADS[name]
    src = synthetic.GradientSource(w, device="cuda")
    gpu = binding.SketchedAMSGrad(w.d, w.n, w.r, w.c, w.k, seed=w.seed, lr=w.lr, beta1=w.beta1, beta2=w.beta2,
                                  eps=w.eps, window_lines=window_lines, variant=variant, P=P)
    ora = oracle.Oracle(w.d, w.n, w.r, w.c, w.k, seed=w.seed, log2g=gpu.get_option("log2g"), lr=w.lr,
                        beta1=w.beta1, beta2=w.beta2, eps=w.eps, threads=32,
                        window_lines=gpu.get_option("window_lines"), variant=variant, P=P)
    return w, src, gpu, ora


def _one_step(w, src, gpu, ora, t, x_gpu, x_ref, variant="ga"):
    g = src.grads(t)
    g_host = g.cpu().numpy()
    x_before = x_ref.astype(np.float64).copy()
    gpu.step(g, x_gpu)
    gpu.sync()
    del g
    exact = None
    if ora.P > 1:          # gradient averaging only: what the second round ranks by, mean_w(m_t + e_{t-1}) / sqrt(vhat_t)
        e_sum = ora.field("e").astype(np.float64).sum(axis=0)
    ora.step(g_host, x_ref)
    if ora.P > 1:
        exact = (ora.field("m").astype(np.float64).sum(axis=0) + e_sum) / w.n / np.sqrt(ora.field("vhat").astype(np.float64))
    return compare_step(gpu, ora, x_gpu.cpu().numpy(), x_ref, x_before, w.lr, variant=variant, exact_ref=exact)


@pytest.mark.parametrize("name", ["C2", "C3"])
def test_two_teacher_forced_steps(name):
    w, src, gpu, ora = _setup(name)
    x_gpu = src.x0()
    x_ref = x_gpu.cpu().numpy().copy()
    _one_step(w, src, gpu, ora, 1, x_gpu, x_ref)
    force_state(gpu, ora)
    x_gpu.copy_(torch.from_numpy(x_ref))
    _one_step(w, src, gpu, ora, 2, x_gpu, x_ref)


def test_c3_windowed_family_first_step():
    w, src, gpu, ora = _setup("C3", window_lines=4)
    x_gpu = src.x0()
    x_ref = x_gpu.cpu().numpy().copy()
    _one_step(w, src, gpu, ora, 1, x_gpu, x_ref)


def test_c3_parameter_averaging_two_teacher_forced_steps():
    w, src, gpu, ora = _setup("C3", variant="pa")
    x_gpu = src.x0()
    x_ref = x_gpu.cpu().numpy().copy()
    _one_step(w, src, gpu, ora, 1, x_gpu, x_ref, variant="pa")
    force_state(gpu, ora, "pa")
    x_gpu.copy_(torch.from_numpy(x_ref))
    _one_step(w, src, gpu, ora, 2, x_gpu, x_ref, variant="pa")


def test_c3_second_round_two_teacher_forced_steps():
    w, src, gpu, ora = _setup("C3", P=4)           # the candidate multiplier the paper's experiments use
    x_gpu = src.x0()
    x_ref = x_gpu.cpu().numpy().copy()
    _one_step(w, src, gpu, ora, 1, x_gpu, x_ref)
    force_state(gpu, ora)
    x_gpu.copy_(torch.from_numpy(x_ref))
    _one_step(w, src, gpu, ora, 2, x_gpu, x_ref)


@pytest.mark.parametrize("name", ["C4", "C5"])
def test_first_step_full_then_properties(name):
    w, src, gpu, ora = _setup(name)
    x_gpu = src.x0()
    x_ref = x_gpu.cpu().numpy().copy()
    _one_step(w, src, gpu, ora, 1, x_gpu, x_ref)
    ora.close()
    # second step on the GPU alone: invariants of Algorithm 2 that need no reference
    I1 = gpu.get("I")
    vhat1 = gpu.get("vhat")
    x1 = x_gpu.cpu().numpy().copy()
    g = src.grads(2)
    gpu.step(g, x_gpu)
    gpu.sync()
    I2 = gpu.get("I")
    assert len(I2) == w.k and np.all(np.diff(I2.astype(np.int64)) > 0) and I2[-1] < w.d
    vhat2 = gpu.get("vhat")
    assert np.all(vhat2 >= vhat1)                                   # vhat = max(vhat, v) never decreases
    assert np.isin(np.flatnonzero(vhat2 != vhat1), I1).all()        # and changes only on I_{t-1}
    x2 = x_gpu.cpu().numpy()
    assert np.isin(np.flatnonzero(x2 != x1), I2).all()              # x moves only on I_t
    # h_t on I_{t-1}: v there is beta2 v + (1-beta2) mean_w(g)^2, spot-checked on a sample in fp64
    sample = I1[:: max(1, len(I1) // 2000)]
    gs = g[:, torch.from_numpy(sample.astype(np.int64)).cuda()].double().mean(0).cpu().numpy()
    b2 = np.float64(np.float32(w.beta2))
    v_prev = np.float64(np.float32(w.eps)) * b2                      # after step 1: eps decayed once
    want = b2 * v_prev + (1 - b2) * gs ** 2
    np.testing.assert_allclose(gpu.get("v")[sample], want, rtol=1e-5)
    e = gpu.get("e")
    assert not e[:, I2].any()


def test_c2_hundred_free_running_steps_keep_the_invariants():
    # no reference: what must hold at every step whatever the data (Algorithm 2 and the proof of Lemma 3)
    from paper_2210_07454_b200 import binding, synthetic
    w = synthetic.WORKLOADS["C2"]
    src = synthetic.GradientSource(w, device="cuda")
    gpu = binding.SketchedAMSGrad(w.d, w.n, w.r, w.c, w.k, seed=w.seed, lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps)
    x = src.x0()
    gsets = [src.grads(t) for t in (1, 2, 3)]
    vhat_prev = gpu.get("vhat")
    I_prev = np.zeros(0, np.uint32)
    for t in range(1, 101):
        x_before = x.clone() if t % 10 == 0 else None
        gpu.step(gsets[t % 3], x)
        if t % 10:
            continue
        gpu.sync()                                            # also reads the device status word
        I = gpu.get("I")
        assert I.size == w.k and np.all(np.diff(I.astype(np.int64)) > 0) and I[-1] < w.d
        changed = torch.nonzero(x != x_before).flatten().cpu().numpy()
        assert np.isin(changed, I).all()                      # x moves on I_t only
        assert bool(torch.isfinite(x).all())
        vhat = gpu.get("vhat")
        assert np.all(vhat >= vhat_prev) and np.all(vhat >= np.float32(w.eps))
        vhat_prev = vhat
        e = gpu.get("e")
        assert not e[:, I].any() and np.isfinite(e).all()     # the residual vanishes on I_t
        I_prev = I
    assert gpu.get("t")[0] == 100
