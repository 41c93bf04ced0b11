"""Pins for the step's own on-the-fly hashing and for the choice of hash family (CPU only).

1. The oracle's step evaluates the hash family inline (`hash_at`); every branch of it (plain family with groups of 32,
   windowed family with several window sizes, ragged sizes) must reproduce what the explicit-array primitives give
   with the separately pinned `hash_family` (tests/test_oracle_hash.py checks that one against big-integer
   arithmetic).
2. Section II-C says the sketch approximately recovers the true top-k.  Grouping coordinates (g = 32) and confining
   a unit to a window must not cost recovery on the workload recipes: the fraction of the true top-k of the
   compressed vector that the selection finds is compared with the ungrouped family (g = 1) at the same r x c.
"""
import numpy as np
import pytest

import oracle
from paper_2210_07454_b200 import synthetic


@pytest.mark.parametrize("window_lines", [0, 1, 4, 8])
def test_step_hashing_matches_primitives_for_groups_of_32(window_lines):
    # d spans several units of 1024 with a ragged last one; c is not a multiple of the window or of the group
    d, n, r, c, k = 5 * 1024 + 300, 3, 5, 700, 60
    rng = np.random.default_rng(11 + window_lines)
    o = oracle.Oracle(d, n, r, c, k, seed=7, log2g=5, lr=1e-2, eps=1e-6, window_lines=window_lines)
    x = rng.standard_normal(d).astype(np.float32)
    fam = [oracle.hash_family(7, 5, c, j, 0, d, window_lines=window_lines) for j in range(r)]
    idx, sgn = np.stack([f[0] for f in fam]), np.stack([f[1] for f in fam])
    for t in range(2):
        g = (rng.standard_normal((n, d)) * rng.uniform(0.01, 1.0, d)).astype(np.float32)
        e_prev = o.field("e").astype(np.float64).copy()
        o.step(g, x)
        a = (o.field("m").astype(np.float64) + e_prev).astype(np.float32)      # what each worker sketched
        for w in range(n):
            assert np.array_equal(o.field("tables")[w], oracle.sketch(a[w], r, c, idx, sgn)), (t, w)
        assert np.array_equal(o.field("est"), oracle.unsketch(o.field("sum"), d, idx, sgn, o.field("vhat")))
        assert np.array_equal(o.field("I"), oracle.topk(o.field("est"), k))


def _recall(w, cfg_id, steps, **family):
    """Fraction of the true top-k of the compressed vector mean_w(a) / sqrt(vhat) that the step selects, and the
    share of that top-k's energy the selection captures, averaged over `steps` steps."""
    src = synthetic.GradientSource(w, device="cpu", cfg_id=cfg_id)
    o = oracle.Oracle(w.d, w.n, w.r, w.c, w.k, seed=w.seed, lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps,
                      threads=8, **family)
    x = src.x0().numpy()
    hits, energy = [], []
    for t in range(1, steps + 1):
        g = src.grads(t).numpy()
        e_prev = o.field("e").astype(np.float64).copy()
        o.step(g, x)
        exact = (o.field("m").astype(np.float64) + e_prev).mean(0) / np.sqrt(o.field("vhat").astype(np.float64))
        true = np.argsort(-np.abs(exact), kind="stable")[:w.k]
        I = o.field("I")
        hits.append(len(np.intersect1d(I, true)) / w.k)
        energy.append(float((exact[I] ** 2).sum() / (exact[true] ** 2).sum()))
    o.close()
    return float(np.mean(hits)), float(np.mean(energy))


RECIPES = {
    # name: (workload, scale, steps): the paper-shaped recipes at a size the CPU finishes in seconds
    "C1": ("C1", 1, 3),        # planted heavy coordinates, k << c: recovery is nearly complete
    "C2": ("C2", 32, 2),       # k > c: recovery is statistically poor for every family
    "C3": ("C3", 64, 2),
    "C5": ("C5", 256, 2),      # 0.1 % planted heavy coordinates
}


@pytest.mark.parametrize("name", sorted(RECIPES))
def test_recovery_does_not_depend_on_the_family(name):
    base, scale, steps = RECIPES[name]
    w = synthetic.WORKLOADS[base]
    if scale > 1:
        w = synthetic.scaled(w, scale)
    cfg = int(base[1])
    ref_hit, ref_energy = _recall(w, cfg, steps, log2g=0)
    for family in (dict(log2g=5), dict(log2g=5, window_lines=4), dict(log2g=5, window_lines=8)):
        if family.get("window_lines", 0) * 32 > w.c:
            continue
        hit, energy = _recall(w, cfg, steps, **family)
        # within noise of the ungrouped family: a few per cent of k in absolute terms
        assert hit >= ref_hit - 0.03, (name, family, hit, ref_hit)
        assert energy >= ref_energy - 0.03, (name, family, energy, ref_energy)
