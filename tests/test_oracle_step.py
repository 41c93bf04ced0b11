"""Pins for the oracle's full step: Algorithm 2 (gradient averaging) with Algorithm 3's unsketch."""
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
    for line in open(os.path.join(GOLDEN, "amsgrad_ga_worked_examples.txt")):
        if line.startswith("#") or not line.strip():
            continue
        ex, t, q, j, val = line.split()
        out.setdefault(ex, []).append((int(t), q, int(j), float(val)))
    return out


EXAMPLES = {
    "A": dict(n=1, d=1, grads=[[1.0]]),
    "B": dict(n=1, d=2, grads=[[1.0, 0.5]]),
    "C": dict(n=2, d=2, grads=[[1.0, 0.5], [3.0, -0.5]]),
    "D": dict(n=1, d=1, grads=[[1.0]], v_keep=True),
    "G": dict(n=1, d=1, grads=[[1.0]], freeze_v=True),
    "H": dict(n=1, d=2, grads=[[1.0, 0.5]], freeze_v=True, lrs=[0.1, 0.05, 0.025]),
}


@pytest.mark.parametrize("ex", sorted(EXAMPLES))
def test_worked_examples(ex):
    cfg = EXAMPLES[ex]
    n, d = cfg["n"], cfg["d"]
    hi, hs = _identity(d)
    o = oracle.Oracle(d, n, 1, d, 1, hash_idx=hi, hash_sgn=hs, v_keep=cfg.get("v_keep", False),
                      freeze_v=cfg.get("freeze_v", False), **HP)
    g = np.array(cfg["grads"], np.float32)
    x = np.zeros(d, np.float32)
    checks = _golden()[ex]
    for t in range(1, max(c[0] for c in checks) + 1):
        if "lrs" in cfg:
            o.set_lr(cfg["lrs"][t - 1])
        o.step(g, x)
        for (tt, q, j, val) in checks:
            if tt != t:
                continue
            if q == "x":
                got = x[j]
            elif q == "I":
                got = o.field("I")[j]
            elif q in ("e0", "e1"):
                got = o.field("e")[int(q[1]), j]
            elif q == "e":
                got = o.field("e")[0, j]
            else:
                got = o.field(q)[j]
            assert got == pytest.approx(val, rel=2e-6, abs=1e-9), (ex, t, q, j)


def _run(d, n, r, c, k, steps, log2g, seed=0, identity=False, **kw):
    rng = np.random.default_rng(seed + 100)
    hp = dict(lr=1e-2, beta1=0.9, beta2=0.99, eps=1e-6)
    hp.update(kw)
    extra = {}
    if identity:
        hi, hs = _identity(d)
        extra = dict(hash_idx=hi, hash_sgn=hs)
        r, c = 1, d
    o = oracle.Oracle(d, n, r, c, k, seed=seed, log2g=log2g, **hp, **extra)
    x = rng.standard_normal(d).astype(np.float32)
    hist = []
    for t in range(steps):
        g = (rng.standard_normal((n, d)) * rng.uniform(0.01, 1.0, d)).astype(np.float32)
        prev = {f: o.field(f).copy() for f in ("m", "e", "v", "vhat")}
        prev["I"] = o.field("I_prev").copy()
        x0 = x.copy()
        o.step(g, x)
        hist.append(dict(g=g, prev=prev, x0=x0, x=x.copy(), I=o.field("I").copy(),
                         **{f: o.field(f).copy() for f in ("m", "e", "v", "vhat", "est", "sum", "tables")}))
    return o, hp, hist


@pytest.mark.parametrize("log2g", [0, 4])
def test_step_invariants(log2g):
    d, n, r, c, k = 3000, 3, 5, 512, 100
    o, hp, hist = _run(d, n, r, c, k, 6, log2g)
    for t, h in enumerate(hist):
        I, Iprev = h["I"], h["prev"]["I"]
        assert len(I) == k and len(np.unique(I)) == k and np.all(np.diff(I.astype(np.int64)) > 0)
        # vhat = max(vhat, v): never decreases, never below eps, changes only on I_{t-1} (proof of Lemma 3)
        assert np.all(h["vhat"] >= h["prev"]["vhat"]) and np.all(h["vhat"] >= np.float32(hp["eps"]))
        changed = np.flatnonzero(h["vhat"] != h["prev"]["vhat"])
        assert np.isin(changed, Iprev).all()
        assert np.all(h["vhat"] >= h["v"])
        # off I_{t-1}, v decays by beta2 (Algorithm 2 with h_t zero there)
        off = np.setdiff1d(np.arange(d), Iprev)
        want = (np.float64(np.float32(hp["beta2"])) * h["prev"]["v"][off].astype(np.float64)).astype(np.float32)
        assert np.array_equal(h["v"][off], want)
        # m recurrence
        b1 = np.float64(np.float32(hp["beta1"]))
        wm = (b1 * h["prev"]["m"].astype(np.float64) + (1 - b1) * h["g"].astype(np.float64)).astype(np.float32)
        assert np.array_equal(h["m"], wm)
        # error feedback is a mask: e_t = a_t off I_t, 0 on I_t, so e_t + scatter(I_t, a_t[I_t]) = a_t exactly
        a = (h["m"].astype(np.float64) + h["prev"]["e"].astype(np.float64)).astype(np.float32)
        assert not h["e"][:, I].any()
        rest = np.setdiff1d(np.arange(d), I)
        assert np.array_equal(h["e"][:, rest], a[:, rest])
        # aggregated sketch is the mean of worker sketches, and by linearity the sketch of the mean vector
        np.testing.assert_allclose(h["sum"], h["tables"].astype(np.float64).mean(0), rtol=0, atol=1e-6)
        idx = np.stack([oracle.hash_family(0, log2g, c, j, 0, d)[0] for j in range(r)])
        sgn = np.stack([oracle.hash_family(0, log2g, c, j, 0, d)[1] for j in range(r)])
        lin = oracle.sketch(a.astype(np.float64).mean(0).astype(np.float32), r, c, idx, sgn)
        np.testing.assert_allclose(h["sum"], lin, rtol=0, atol=2e-6 * np.abs(lin).max())
        # the update moves exactly the coordinates of I_t, by lr * mean_w a / sqrt(vhat)
        moved = np.flatnonzero(h["x"] != h["x0"])
        assert np.isin(moved, I).all()
        delta = a.astype(np.float64).mean(0)[I] / np.sqrt(h["vhat"][I].astype(np.float64))
        np.testing.assert_allclose(h["x"][I], h["x0"][I] - np.float64(np.float32(hp["lr"])) * delta, rtol=2e-7, atol=1e-7)
        # I_t is the top-k of the stored estimates
        assert np.array_equal(I, oracle.topk(h["est"], k))


def test_lemma3_identity_and_contraction():
    # Lemma 3: x_t - x~_t = alpha vhat_{t-1}^{-1/2} e_{t-1}, with x~_{t+1} = x~_t - alpha vhat_t^{-1/2} mean_w m_t.
    # Also, Delta_t being a restriction of Delta~_t to I_t: ||Delta~ - Delta|| <= ||Delta~||, and when I_t is the true
    # top-k of Delta~_t (lossless sketch) the bound of Lemma 2 holds: <= sqrt(1-k/d) ||Delta~||.
    d, n, k = 400, 4, 40
    o, hp, hist = _run(d, n, 1, d, k, 12, 0, identity=True)
    lr = np.float64(np.float32(hp["lr"]))
    xt = hist[0]["x0"].astype(np.float64)
    for h in hist:
        vh = h["vhat"].astype(np.float64)
        xt = xt - lr * h["m"].astype(np.float64).mean(0) / np.sqrt(vh)
        ebar = h["e"].astype(np.float64).mean(0)
        np.testing.assert_allclose(h["x"].astype(np.float64) - xt, lr * ebar / np.sqrt(vh), rtol=0, atol=5e-6)
        a = h["m"].astype(np.float64) + h["prev"]["e"].astype(np.float64)
        dtil = a.mean(0) / np.sqrt(vh)
        dsel = np.zeros(d)
        dsel[h["I"]] = dtil[h["I"]]
        assert np.linalg.norm(dtil - dsel) <= np.sqrt(1 - k / d) * np.linalg.norm(dtil) * (1 + 1e-6)
        true_topk = np.sort(np.argsort(-np.abs(dtil), kind="stable")[:k])
        assert np.array_equal(h["I"], true_topk.astype(np.uint32))


def test_lemma3_identity_under_a_step_size_schedule():
    # Lemma 3 with alpha_t = alpha / sqrt(t) (Theorem 2's choice): x_{t+1} - x~_{t+1} = alpha_t vhat_t^{-1/2} e_t with
    # x~_{t+1} = x~_t - alpha_t vhat_t^{-1/2} mean_w m_t.  It holds only because e_{t-1} enters a_t weighted by
    # alpha_{t-1}/alpha_t: with the weight dropped or inverted the two sides drift apart.
    d, n, k, steps = 300, 3, 30, 12
    hi, hs = _identity(d)
    o = oracle.Oracle(d, n, 1, d, k, hash_idx=hi, hash_sgn=hs, lr=0.05, beta1=0.9, beta2=0.99, eps=1e-6)
    rng = np.random.default_rng(21)
    x = rng.standard_normal(d).astype(np.float32)
    xt = x.astype(np.float64).copy()
    gaps = []
    for t in range(1, steps + 1):
        lr = np.float32(0.05 / np.sqrt(t))
        o.set_lr(lr)
        g = (rng.standard_normal((n, d)) * rng.uniform(0.01, 1.0, d)).astype(np.float32)
        o.step(g, x)
        vh = o.field("vhat").astype(np.float64)
        xt = xt - np.float64(lr) * o.field("m").astype(np.float64).mean(0) / np.sqrt(vh)
        want = np.float64(lr) * o.field("e").astype(np.float64).mean(0) / np.sqrt(vh)
        np.testing.assert_allclose(x.astype(np.float64) - xt, want, rtol=0, atol=2e-5)
        gaps.append(np.abs(want).max())
    assert max(gaps) > 1e-2          # the identity is not vacuous: the residual term is thousands of tolerances large


def test_constant_schedule_and_unit_weight_are_the_plain_step():
    # alpha_{t-1}/alpha_t = 1: setting the same step size before every step changes nothing, bit for bit
    d, n, r, c, k = 500, 2, 3, 64, 20
    a = oracle.Oracle(d, n, r, c, k, seed=5, log2g=2, lr=0.01)
    b = oracle.Oracle(d, n, r, c, k, seed=5, log2g=2, lr=0.01)
    rng = np.random.default_rng(2)
    xa = np.zeros(d, np.float32); xb = np.zeros(d, np.float32)
    for t in range(5):
        g = rng.standard_normal((n, d)).astype(np.float32)
        b.set_lr(0.01)
        a.step(g, xa); b.step(g, xb)
        assert np.array_equal(xa, xb) and np.array_equal(a.field("e"), b.field("e"))


def test_frozen_second_moments():
    # freeze_v (Section III-B's remark): v and vhat never change; with vhat = s^2 everywhere the estimates, and hence
    # the index sets and residuals, do not depend on s, and x moves 1/s as far (s a power of two: exactly)
    d, n, r, c, k = 800, 3, 5, 128, 40
    runs = {}
    for s2 in (1.0, 4.0):
        o = oracle.Oracle(d, n, r, c, k, seed=3, log2g=3, lr=0.25, eps=s2, freeze_v=True)
        rng = np.random.default_rng(7)
        x = np.zeros(d, np.float32)
        sets = []
        for t in range(6):
            g = rng.standard_normal((n, d)).astype(np.float32)
            o.step(g, x)
            assert np.all(o.field("vhat") == np.float32(s2)) and np.all(o.field("v") == np.float32(s2))
            sets.append(o.field("I").copy())
        runs[s2] = (sets, x.copy(), o.field("e").copy())
    for a, b in zip(runs[1.0][0], runs[4.0][0]):
        assert np.array_equal(a, b)
    assert np.array_equal(runs[1.0][2], runs[4.0][2])
    np.testing.assert_allclose(runs[4.0][1], runs[1.0][1] / 2, rtol=3e-7, atol=0)
    # and the moving-vhat run differs (the switch does something): long enough for coordinates whose vhat has grown
    # to be selected again
    xs = {}
    for frozen in (True, False):
        o = oracle.Oracle(d, n, r, c, k, seed=3, log2g=3, lr=0.25, eps=1.0, freeze_v=frozen)
        rng = np.random.default_rng(7)
        x = np.zeros(d, np.float32)
        for t in range(30):
            o.step((3.0 * rng.standard_normal((n, d))).astype(np.float32), x)     # h^2 is often above v = 1
        xs[frozen] = x
        assert (np.count_nonzero(o.field("vhat") > 1.0) > 40) == (not frozen)
    assert not np.array_equal(xs[True], xs[False])


def test_no_compression_reduces_to_distributed_amsgrad():
    # Section III-B: with no compressor (k = d, lossless sketch) Algorithm 2 is distributed AMSGrad on the mean
    # gradient -- except that v first sees the gradient at t = 2, because I_0 is empty.
    d, n = 50, 3
    o, hp, hist = _run(d, n, 1, d, d, 8, 0, identity=True)
    b1, b2, lr, eps = (np.float64(np.float32(hp[q])) for q in ("beta1", "beta2", "lr", "eps"))
    m = np.zeros(d); v = np.full(d, eps); vh = v.copy(); x = hist[0]["x0"].astype(np.float64)
    for t, h in enumerate(hist):
        gbar = h["g"].astype(np.float64).mean(0)
        m = b1 * m + (1 - b1) * gbar
        v = b2 * v + (1 - b2) * (gbar ** 2 if t > 0 else 0.0)
        vh = np.maximum(vh, v)
        x = x - lr * m / np.sqrt(vh)
        assert not h["e"].any()
        np.testing.assert_allclose(h["x"], x, rtol=1e-5, atol=1e-6)
        np.testing.assert_allclose(h["vhat"], vh, rtol=1e-5)


def test_estimates_of_seeded_sketch_match_primitives():
    # the step's on-the-fly hashing agrees with the explicit-array primitives pinned in test_oracle_sketch.py
    d, n, r, c, k = 2000, 2, 5, 256, 50
    o, hp, hist = _run(d, n, r, c, k, 2, 3, seed=4)
    h = hist[-1]
    idx = np.stack([oracle.hash_family(4, 3, c, j, 0, d)[0] for j in range(r)])
    sgn = np.stack([oracle.hash_family(4, 3, c, j, 0, d)[1] for j in range(r)])
    a = (h["m"].astype(np.float64) + h["prev"]["e"].astype(np.float64)).astype(np.float32)
    for w in range(n):
        assert np.array_equal(h["tables"][w], oracle.sketch(a[w], r, c, idx, sgn))
    assert np.array_equal(h["est"], oracle.unsketch(h["sum"], d, idx, sgn, h["vhat"]))


def test_threads_do_not_change_results():
    d, n, r, c, k = 5000, 4, 5, 512, 64
    rng = np.random.default_rng(0)
    g = rng.standard_normal((2, n, d)).astype(np.float32)
    outs = []
    for th in (1, 4):
        o = oracle.Oracle(d, n, r, c, k, seed=1, log2g=5, threads=th)
        x = np.zeros(d, np.float32)
        for t in range(2):
            o.step(g[t], x)
        outs.append((x.copy(), o.field("e").copy(), o.field("sum").copy(), o.field("I").copy()))
    for a, b in zip(*outs):
        assert np.array_equal(a, b)


# ------------------------------------------------------------------------- second round with P*k candidates
def test_second_round_selects_by_exact_values_among_candidates():
    # Section III-A: take the P*k largest estimates as candidates, fetch the exact values there, keep the k largest
    # exact magnitudes.  Checked against a brute-force restatement with numpy on a lossy sketch.
    d, n, r, c, k, P = 4000, 3, 5, 1024, 40, 4
    rng = np.random.default_rng(11)
    o = oracle.Oracle(d, n, r, c, k, seed=2, log2g=2, lr=1e-2, eps=1e-6, P=P)
    o1 = oracle.Oracle(d, n, r, c, k, seed=2, log2g=2, lr=1e-2, eps=1e-6)
    x = np.zeros(d, np.float32); x1 = x.copy()
    hits = []
    for t in range(4):
        g = (rng.standard_normal((n, d)) * rng.uniform(0.01, 1.0, d)).astype(np.float32)
        e_prev = o.field("e").copy()
        o.step(g, x)
        est, vh, I, cand = o.field("est"), o.field("vhat"), o.field("I"), o.field("cand")
        assert len(cand) == P * k and np.array_equal(cand, oracle.topk(est, P * k))
        a = (o.field("m").astype(np.float64) + e_prev.astype(np.float64)).astype(np.float32)
        exact = (a.astype(np.float64).mean(0) / np.sqrt(vh.astype(np.float64))).astype(np.float32)
        order = np.lexsort((cand, -np.abs(exact[cand])))                 # exact magnitude desc, index asc
        assert np.array_equal(I, np.sort(cand[order[:k]]))
        assert np.isin(I, cand).all()
        true_top = np.argsort(-np.abs(exact), kind="stable")[:k]
        hits.append(np.isin(true_top, I).mean())
        # error feedback still masks exactly I_t
        assert not o.field("e")[:, I].any()
    # the same run without the second round recovers fewer of the true top-k on this lossy sketch
    base = []
    rng = np.random.default_rng(11)
    for t in range(4):
        g = (rng.standard_normal((n, d)) * rng.uniform(0.01, 1.0, d)).astype(np.float32)
        e_prev = o1.field("e").copy()
        o1.step(g, x1)
        a = (o1.field("m").astype(np.float64) + e_prev.astype(np.float64)).astype(np.float32)
        exact = (a.astype(np.float64).mean(0) / np.sqrt(o1.field("vhat").astype(np.float64))).astype(np.float32)
        base.append(np.isin(np.argsort(-np.abs(exact), kind="stable")[:k], o1.field("I")).mean())
    assert hits[0] > base[0] + 0.1 and hits[0] > 0.6, (hits, base)    # first step: both start from the same state


def test_second_round_is_neutral_for_a_lossless_sketch_and_for_p1():
    d, n, k = 300, 2, 20
    hi, hs = _identity(d)
    rng = np.random.default_rng(5)
    g = rng.standard_normal((3, n, d)).astype(np.float32)
    res = []
    for P in (1, 3):
        o = oracle.Oracle(d, n, 1, d, k, hash_idx=hi, hash_sgn=hs, lr=1e-2, eps=1e-6, P=P)
        x = np.zeros(d, np.float32)
        for t in range(3):
            o.step(g[t], x)
        res.append((x.copy(), o.field("I").copy(), o.field("e").copy()))
    for a, b in zip(*res):
        assert np.array_equal(a, b)


def test_second_round_parameter_averaging():
    d, n, r, c, k, P = 3000, 2, 3, 128, 30, 4
    rng = np.random.default_rng(12)
    o = oracle.Oracle(d, n, r, c, k, seed=3, log2g=0, lr=1e-2, eps=1e-6, P=P, variant="pa")
    x = np.zeros(d, np.float32)
    for t in range(2):
        e_prev = o.field("e").copy()
        o.step(rng.standard_normal((n, d)).astype(np.float32), x)
    cand, I = o.field("cand"), o.field("I")
    a = (o.field("m").astype(np.float64) / np.sqrt(o.field("vhatw").astype(np.float64)) + e_prev).astype(np.float32)
    exact = a.astype(np.float64).mean(0).astype(np.float32)
    order = np.lexsort((cand, -np.abs(exact[cand])))
    assert np.array_equal(I, np.sort(cand[order[:k]]))
