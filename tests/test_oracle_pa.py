"""Pins for the oracle's parameter-averaging variant (Algorithm 1)."""
import os

import numpy as np
import pytest

import oracle
from conftest import GOLDEN

HP = dict(lr=0.1, beta1=0.9, beta2=0.99, eps=1e-2)


def _identity(d):
    return np.arange(d, dtype=np.uint32)[None, :], np.ones((1, d), np.int8)


def _golden():
    out = {}
    for line in open(os.path.join(GOLDEN, "amsgrad_pa_worked_examples.txt")):
        if line.startswith("#") or not line.strip():
            continue
        ex, t, q, j, val = line.split()
        out.setdefault(ex, []).append((int(t), q, int(j), float(val)))
    return out


EXAMPLES = {"E": dict(n=1, d=2, grads=[[1.0, 0.5]]), "F": dict(n=2, d=1, grads=[[1.0], [3.0]])}


@pytest.mark.parametrize("ex", sorted(EXAMPLES))
def test_worked_examples(ex):
    cfg = EXAMPLES[ex]
    n, d = cfg["n"], cfg["d"]
    hi, hs = _identity(d)
    o = oracle.Oracle(d, n, 1, d, 1, hash_idx=hi, hash_sgn=hs, variant="pa", **HP)
    g = np.array(cfg["grads"], np.float32)
    x = np.zeros(d, np.float32)
    checks = _golden()[ex]
    for t in range(1, max(c[0] for c in checks) + 1):
        o.step(g, x)
        for (tt, q, j, val) in checks:
            if tt != t:
                continue
            got = {"x": lambda: x[j], "I": lambda: o.field("I")[j], "e": lambda: o.field("e")[0, j],
                   "est": lambda: o.field("est")[j], "vw": lambda: o.field("vw")[0, j],
                   "vw0": lambda: o.field("vw")[0, j], "vw1": lambda: o.field("vw")[1, j]}[q]()
            assert got == pytest.approx(val, rel=2e-6, abs=1e-9), (ex, t, q, j)


def test_auxiliary_sequence_identity_and_masking():
    # Section IV-A: with x~_{t+1} = x~_t - alpha mean_w m_t^(w)/sqrt(vhat_t^(w)) one always has
    # x_t - x~_t = alpha e_{t-1} (e = mean of the workers' residuals) -- the reason e is scaled by alpha_{t-1}/alpha_t.
    d, n, k = 300, 3, 25
    hi, hs = _identity(d)
    hp = dict(lr=1e-2, beta1=0.9, beta2=0.99, eps=1e-6)
    o = oracle.Oracle(d, n, 1, d, k, hash_idx=hi, hash_sgn=hs, variant="pa", **hp)
    rng = np.random.default_rng(3)
    x = rng.standard_normal(d).astype(np.float32)
    xt = x.astype(np.float64).copy()
    lr = np.float64(np.float32(hp["lr"]))
    for t in range(10):
        g = (rng.standard_normal((n, d)) * rng.uniform(0.01, 1.0, d)).astype(np.float32)
        e_prev = o.field("e").copy()
        vhat_prev = o.field("vhatw").copy()
        o.step(g, x)
        m, vh, e, I = o.field("m"), o.field("vhatw"), o.field("e"), o.field("I")
        assert np.all(vh >= vhat_prev) and np.all(vh >= o.field("vw"))            # vhat = max(vhat, v), per worker
        xt = xt - lr * (m.astype(np.float64) / np.sqrt(vh.astype(np.float64))).mean(0)
        np.testing.assert_allclose(x.astype(np.float64) - xt, lr * e.astype(np.float64).mean(0), rtol=0, atol=5e-6)
        # error feedback is a mask of a = m/sqrt(vhat) + e_prev
        a = (m.astype(np.float64) / np.sqrt(vh.astype(np.float64)) + e_prev.astype(np.float64)).astype(np.float32)
        assert not e[:, I].any()
        rest = np.setdiff1d(np.arange(d), I)
        assert np.array_equal(e[:, rest], a[:, rest])
        # lossless sketch: the selection is the true top-k of the mean vector, by magnitude then index
        abar = a.astype(np.float64).mean(0)
        true_topk = np.sort(np.argsort(-np.abs(abar.astype(np.float32)), kind="stable")[:k])
        assert np.array_equal(I, true_topk.astype(np.uint32))


def test_auxiliary_sequence_identity_under_a_step_size_schedule():
    # Section IV-A with alpha_t = alpha / sqrt(t): x_{t+1} - x~_{t+1} = alpha_t e_t needs e_{t-1} weighted by
    # alpha_{t-1}/alpha_t in the sketched vector (Algorithm 1's sketch line)
    d, n, k = 300, 3, 25
    hi, hs = _identity(d)
    o = oracle.Oracle(d, n, 1, d, k, hash_idx=hi, hash_sgn=hs, variant="pa", lr=0.05, beta1=0.9, beta2=0.99, eps=1e-6)
    rng = np.random.default_rng(4)
    x = rng.standard_normal(d).astype(np.float32)
    xt = x.astype(np.float64).copy()
    worst = 0.0
    for t in range(1, 11):
        lr = np.float32(0.05 / np.sqrt(t))
        o.set_lr(lr)
        g = (rng.standard_normal((n, d)) * rng.uniform(0.01, 1.0, d)).astype(np.float32)
        o.step(g, x)
        m, vh = o.field("m").astype(np.float64), o.field("vhatw").astype(np.float64)
        xt = xt - np.float64(lr) * (m / np.sqrt(vh)).mean(0)
        want = np.float64(lr) * o.field("e").astype(np.float64).mean(0)
        np.testing.assert_allclose(x.astype(np.float64) - xt, want, rtol=0, atol=2e-5)
        worst = max(worst, np.abs(want).max())
    assert worst > 1e-2


def test_no_compression_averages_local_amsgrad_steps():
    # k = d and a lossless sketch: e stays 0 and x moves by the average of the workers' own AMSGrad directions
    # (Section II-A: parameter averaging is NOT AMSGrad on the averaged gradient).
    d, n = 40, 3
    hi, hs = _identity(d)
    hp = dict(lr=1e-2, beta1=0.9, beta2=0.99, eps=1e-6)
    o = oracle.Oracle(d, n, 1, d, d, hash_idx=hi, hash_sgn=hs, variant="pa", **hp)
    b1, b2, lr, eps = (np.float64(np.float32(hp[q])) for q in ("beta1", "beta2", "lr", "eps"))
    rng = np.random.default_rng(8)
    x = rng.standard_normal(d).astype(np.float32)
    xr = x.astype(np.float64).copy()
    m = np.zeros((n, d)); v = np.full((n, d), eps); vh = v.copy()
    for t in range(6):
        g = rng.standard_normal((n, d)).astype(np.float32)
        o.step(g, x)
        m = b1 * m + (1 - b1) * g; v = b2 * v + (1 - b2) * g.astype(np.float64) ** 2; vh = np.maximum(vh, v)
        xr = xr - lr * (m / np.sqrt(vh)).mean(0)
        assert not o.field("e").any()
        np.testing.assert_allclose(x, xr, rtol=1e-5, atol=1e-6)
    gavg_dir = (m.mean(0)) / np.sqrt(np.maximum(eps, v.mean(0)))
    assert not np.allclose((m / np.sqrt(vh)).mean(0), gavg_dir, rtol=1e-3)             # the two averagings differ


def test_seeded_sketch_path_matches_primitives():
    d, n, r, c, k = 2000, 2, 5, 256, 50
    o = oracle.Oracle(d, n, r, c, k, seed=4, log2g=3, variant="pa")
    rng = np.random.default_rng(0)
    x = np.zeros(d, np.float32)
    for t in range(2):
        e_prev = o.field("e").copy()
        o.step(rng.standard_normal((n, d)).astype(np.float32), x)
    idx = np.stack([oracle.hash_family(4, 3, c, j, 0, d)[0] for j in range(r)])
    sgn = np.stack([oracle.hash_family(4, 3, c, j, 0, d)[1] for j in range(r)])
    a = (o.field("m").astype(np.float64) / np.sqrt(o.field("vhatw").astype(np.float64)) + e_prev).astype(np.float32)
    for w in range(n):
        assert np.array_equal(o.field("tables")[w], oracle.sketch(a[w], r, c, idx, sgn))
    assert np.array_equal(o.field("est"), oracle.unsketch(o.field("sum"), d, idx, sgn))     # no vhat argument
    assert np.array_equal(o.field("I"), oracle.topk(o.field("est"), k))
