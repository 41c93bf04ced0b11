"""Parity at the full benchmark sizes, in the launch configuration bench.py times (default options).

C2 and C3: twenty steps, compared with the full oracle at seven and six of them (teacher-forced there).  C4 and C5:
three teacher-forced steps against the full oracle (every stage, every element): from the second step on I_{t-1} is not empty, so the membership bitmap, the
gradient sums carried over the several launches these sizes need, the lazy second moments with decay owed and the
masked residual are all compared element by element.
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
    members = ora.field("I_prev").astype(np.int64).copy()
    if ora.P > 1:          # gradient averaging only: what the second round ranks by, mean_w(m_t + e_{t-1}) / sqrt(vhat_t)
        e_sum = ora.field("e").astype(np.float64).sum(axis=0)
    ora.step(g_host, x_ref)
    if ora.P > 1:
        exact = (ora.field("m").astype(np.float64).sum(axis=0) + e_sum) / w.n / np.sqrt(ora.field("vhat").astype(np.float64))
    return compare_step(gpu, ora, x_gpu.cpu().numpy(), x_ref, x_before, w.lr, variant=variant, exact_ref=exact,
                        grads=g_host, members=members, beta2=w.beta2)


@pytest.mark.parametrize("name,compared", [("C2", (1, 2, 3, 4, 5, 12, 20)), ("C3", (1, 2, 3, 4, 11, 20))])
def test_twenty_steps_teacher_forced_at_the_compared_ones(name, compared):
    # The configurations' own step count.  The oracle takes all twenty steps; the GPU takes them too and is compared
    # stage by stage at the listed ones, its state set to the oracle's just before each (in between it runs free, so
    # by step 20 the second moments have decays owed over many steps and the residuals have their long-run size).
    w, src, gpu, ora = _setup(name)
    x_gpu = src.x0()
    x_ref = x_gpu.cpu().numpy().copy()
    for t in range(1, 21):
        if t in compared:
            if t > 1:
                force_state(gpu, ora)
                x_gpu.copy_(torch.from_numpy(x_ref))
            _one_step(w, src, gpu, ora, t, x_gpu, x_ref)
        else:
            g = src.grads(t)
            gpu.step(g, x_gpu)
            ora.step(g.cpu().numpy(), x_ref)
            del g
    gpu.sync()
    ora.close()


def test_c3_plain_family_first_step():
    # the plain hash family (any group lands anywhere in its row) runs the reduction kernel: the fallback of every
    # configuration the shared-memory kernel does not cover
    w, src, gpu, ora = _setup("C3", window_lines=0)
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
def test_three_teacher_forced_steps(name):
    w, src, gpu, ora = _setup(name)
    x_gpu = src.x0()
    x_ref = x_gpu.cpu().numpy().copy()
    for t in (1, 2, 3):
        if t > 1:
            force_state(gpu, ora)
            x_gpu.copy_(torch.from_numpy(x_ref))
        _one_step(w, src, gpu, ora, t, x_gpu, x_ref)
    ora.close()


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
