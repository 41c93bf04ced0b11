"""Helpers for the GPU-vs-oracle parity tests: tolerance rule, state transfer, stage-by-stage comparison."""
from __future__ import annotations

import numpy as np

REL = 1e-5      # "within 1e-5 relative (fp32, atomic order)"


def close(got, ref, what, groups_axis=None, rel=REL, scale=None):
    """|got - ref| <= rel * max(|ref|, RMS) with RMS the root mean square of `ref` over its natural group
    (the whole array, or each slice along `groups_axis`).  A bucket or a mean is a signed sum that can cancel
    to nearly zero for any summation order, so the bound is relative to the group's scale, not to the element."""
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    if groups_axis is None:
        rms = np.sqrt(np.mean(ref * ref)) if ref.size else 0.0
    else:
        axes = tuple(a for a in range(ref.ndim) if a != groups_axis)
        rms = np.sqrt(np.mean(ref * ref, axis=axes, keepdims=True))
    bound = rel * np.maximum(np.abs(ref), rms)
    if scale is not None:                      # an additional per-element error scale inherited from an input
        bound = np.maximum(bound, rel * np.asarray(scale, np.float64))
    err = np.abs(got - ref)
    bad = err > bound
    if bad.any():
        q = np.unravel_index(np.argmax(err / np.maximum(bound, 1e-300)), err.shape)
        raise AssertionError(f"{what}: {bad.sum()} of {bad.size} outside tolerance; worst at {q}: "
                             f"got {got[q]!r} ref {ref[q]!r} err {err[q]:.3e} bound {np.broadcast_to(bound, err.shape)[q]:.3e}")


def est_scale(S_ref, vhat_ref, tables_ref=None):
    """An estimate is one bucket of the aggregated sketch divided by sqrt(vhat): it inherits the bucket's absolute
    error bound, rel * RMS(row), magnified by vhat^{-1/2}.  The aggregated bucket is the mean of the n workers'
    buckets, each formed by fp32 additions whose rounding is relative to THAT worker's partial sums: where the
    workers cancel (independent noise: the aggregate's RMS is 1/sqrt(n) of a worker's) the absolute error stays at
    the workers' scale, so the row scale is the larger of the aggregate's RMS and the workers' (tables_ref given)."""
    S = np.asarray(S_ref, np.float64)
    row_rms = np.sqrt(np.mean(S * S, axis=1)).max()
    if tables_ref is not None:
        row_rms = max(row_rms, worker_row_rms(tables_ref).max())
    return row_rms / np.sqrt(np.asarray(vhat_ref, np.float64))


def worker_row_rms(tables_ref):
    """RMS of every (worker, row) of the worker sketches, computed worker by worker in fp64: shape (n, r)."""
    return np.stack([np.sqrt(np.mean(np.asarray(t, np.float64) ** 2, axis=1)) for t in tables_ref])


LAST_INDEX_DIFFERENCE = {}     # what the last index_sets_agree call saw: {"what", "count", "worst_offset_in_bands"}


def index_sets_agree(I_gpu, I_ref, est_ref, k, what="I", rel=REL, scale=None):
    """The sets must be equal except for indices whose reference magnitude lies within the tolerance band of the
    k-th largest magnitude tau, and only a handful may differ at all (at most 0.1 % of k, at least 4): rounding can
    move a coordinate across the threshold only if it sits within a few 1e-7 of it, which few do.
    Returns the symmetric difference (to be excluded from x/e comparisons); the count and the worst offset, in
    units of the band, are printed and kept in LAST_INDEX_DIFFERENCE."""
    I_gpu = np.asarray(I_gpu, np.int64)
    I_ref = np.asarray(I_ref, np.int64)
    assert len(I_gpu) == k == len(I_ref), (what, len(I_gpu), len(I_ref), k)
    assert len(np.unique(I_gpu)) == k, f"{what}: repeated indices"
    diff = np.setxor1d(I_gpu, I_ref)
    if diff.size:
        mag = np.abs(np.asarray(est_ref, np.float64))
        tau = mag[I_ref].min()
        rms = np.sqrt(np.mean(mag * mag))
        band = rel * max(tau, rms) * np.ones(diff.size)
        if scale is not None:
            band = np.maximum(band, rel * np.asarray(scale, np.float64)[diff])
        off = np.abs(mag[diff] - tau)
        worst = float((off / band).max())
        LAST_INDEX_DIFFERENCE.update(what=what, count=int(diff.size), worst_offset_in_bands=worst)
        print(f"[parity] {what}: {diff.size} of {k} indices differ inside the band; worst offset {worst:.3f} bands "
              f"(tau = {tau:.6e})")
        # both the differing element and the threshold element carry an error of up to one band
        assert (off <= 2 * band).all(), (f"{what}: {diff.size} indices differ and {np.sum(off > 2 * band)} of them "
                                         f"are outside the band (tau={tau:.6e}, worst {off.max():.3e})")
        cap = max(4, k // 1000)
        assert diff.size <= 2 * cap, f"{what}: {diff.size} indices differ inside the band; at most {2 * cap} tolerated"
    else:
        LAST_INDEX_DIFFERENCE.update(what=what, count=0, worst_offset_in_bands=0.0)
    return diff


def force_state(gpu, ora, variant="ga"):
    """Teacher forcing: install the oracle's state (m, e, v, vhat or vw, vhatw, I_{t-1}, t) in the GPU handle."""
    t = np.array([ora.t], np.uint64)
    gpu.set("t", t)
    for f in (("m", "e", "v", "vhat") if variant == "ga" else ("m", "e", "vw", "vhatw")):
        gpu.set(f, np.ascontiguousarray(ora.field(f)))
    gpu.set("I", np.ascontiguousarray(ora.field("I_prev")))


def second_round_agree(gpu, ora, est_ref, sc, exact_ref):
    """Second round (P > 1): the candidate sets agree up to the band on the estimates; the final sets agree up to the
    band on the exact values `exact_ref` (d values, from the caller) and up to coordinates that are candidates on one
    side only (themselves inside the estimate band)."""
    k, pk = ora.k, ora.P * ora.k
    cand_gpu, cand_ref = gpu.get("cand"), ora.field("cand")
    assert np.all(np.diff(cand_gpu.astype(np.int64)) > 0)
    cdiff = index_sets_agree(cand_gpu, cand_ref, est_ref, pk, what="candidates", scale=sc)
    I_gpu, I_ref = gpu.get("I").astype(np.int64), np.asarray(ora.field("I"), np.int64)
    assert len(I_gpu) == k and np.all(np.diff(I_gpu) > 0) and np.isin(I_gpu, cand_gpu).all()
    diff = np.setxor1d(I_gpu, I_ref)
    if diff.size:
        mag = np.abs(np.asarray(exact_ref, np.float64))
        tau = mag[I_ref].min()
        band = REL * max(tau, np.sqrt(np.mean(mag[cand_ref.astype(np.int64)] ** 2)))
        ok = (np.abs(mag[diff] - tau) <= 2 * band)
        if cdiff.size:       # a candidate of one side only displaces, or is displaced by, an element at the threshold
            assert cdiff.size <= 4, "too many candidate differences to reason about"
            ok |= np.isin(diff, cdiff)
            ok |= np.abs(mag[diff] - tau) <= 2 * band + np.sort(np.abs(mag[I_ref] - tau))[min(cdiff.size, k - 1)]
        assert ok.all(), f"I after the second round: {np.sum(~ok)} of {diff.size} differing indices outside the band"
    return diff


def second_moment_bound(v_ref, grads, members, n, beta2, rel=REL):
    """Per-element bound on |v_gpu - v_ref|: `rel` relative to the element (v is a sum of non-negative terms, so
    nothing cancels inside it), plus what the rounding of the fp32 worker sum behind h_t can move it on I_{t-1}.
    h = (sum of n gradients) / n: any summation order is within (n-1) * 2^-24 * sum|g| of the exact sum, and
    v = beta2 v + (1-beta2) h^2 turns an error dh of h into at most (1-beta2) (2 |h| dh + dh^2)."""
    bound = rel * np.abs(np.asarray(v_ref, np.float64))
    if grads is not None and len(members):
        g = np.asarray(grads)[:, members].astype(np.float64)
        dh = (n - 1) * 2.0 ** -24 * np.abs(g).sum(0) / n
        h = np.abs(g.sum(0)) / n
        bound[members] += (1.0 - float(beta2)) * (2.0 * h * dh + dh * dh)
    return bound


def compare_step(gpu, ora, x_gpu, x_ref, x_before, lr, check_tables=True, x_gpu_before=None, variant="ga",
                 exact_ref=None, grads=None, members=None, beta2=None):
    """Compares every stage output of the step both sides just took from the same state and gradients.
    exact_ref: with a second round (P > 1), the d exact preconditioned worker means the second round ranks by.
    grads, members, beta2: the step's gradients (n, d), I_{t-1} and beta2, for the rounding term of the bound on v
    (without them v must agree to 1e-5 of each element outright)."""
    d, n, k = ora.d, ora.n, ora.k
    if check_tables:
        close(gpu.get("tables"), ora.field("tables"), "worker sketches", groups_axis=1)
    # the aggregate is the mean of the workers' buckets: its error scale is a worker's row, not its own (est_scale)
    tables_ref = ora.field("tables")
    close(gpu.get("sum"), ora.field("sum"), "aggregated sketch", groups_axis=0,
          scale=worker_row_rms(tables_ref).max(axis=0)[:, None])
    if variant == "ga":
        # v and vhat are sums of non-negative terms: the bound is relative to each ELEMENT, not to the array's scale
        v_ref = ora.field("v")
        vb = second_moment_bound(v_ref, grads, np.asarray([] if members is None else members, np.int64), n, beta2 or 0.0)
        for name, got, ref in (("v", gpu.get("v"), v_ref), ("vhat", gpu.get("vhat"), ora.field("vhat"))):
            err = np.abs(got.astype(np.float64) - ref.astype(np.float64))
            bad = err > vb
            assert not bad.any(), (f"{name}: {bad.sum()} of {bad.size} elements outside the element-relative bound; "
                                   f"worst ratio {np.max(err / np.maximum(vb, 1e-300)):.3f}")
        sc = est_scale(ora.field("sum"), ora.field("vhat"), tables_ref)
    else:                       # Algorithm 1: per-worker second moments (sums of non-negative terms: element-relative),
        np.testing.assert_allclose(gpu.get("vw"), ora.field("vw"), rtol=REL, atol=0)       # and a plain unsketch
        np.testing.assert_allclose(gpu.get("vhatw"), ora.field("vhatw"), rtol=REL, atol=0)
        sc = est_scale(ora.field("sum"), np.ones(d, np.float32), tables_ref)
    est_ref = ora.field("est")
    close(gpu.get("est"), est_ref, "estimates", scale=sc)
    # the keys the selection actually ran on (vector medians, hardware reciprocal square root), not the export path
    keys = gpu.get("keys").view(np.float32)
    assert np.all(keys >= 0) and np.isfinite(keys).all()
    close(keys, np.abs(est_ref), "ranking keys", scale=sc)
    I_gpu = gpu.get("I")
    assert np.all(np.diff(I_gpu.astype(np.int64)) > 0)
    if getattr(ora, "P", 1) > 1:
        diff = second_round_agree(gpu, ora, est_ref, sc, exact_ref)
    else:
        diff = index_sets_agree(I_gpu, ora.field("I"), est_ref, k, scale=sc)
    keep = np.ones(d, bool)
    keep[diff] = False
    m_gpu, m_ref = gpu.get("m"), ora.field("m")
    for w in range(n):                                   # one worker at a time: its own RMS, bounded temporaries
        close(m_gpu[w], m_ref[w], f"m[{w}]")
    del m_gpu
    e_gpu, e_ref = gpu.get("e"), ora.field("e")
    for w in range(n):
        if diff.size:
            close(e_gpu[w][keep], e_ref[w][keep], f"e[{w}]")
        else:
            close(e_gpu[w], e_ref[w], f"e[{w}]")
    assert not e_gpu[:, I_gpu].any(), "e must be zero on I_t"
    del e_gpu
    # x: compare the CHANGE against lr * RMS(Delta) scale
    dx_gpu = np.asarray(x_gpu, np.float64) - (x_before if x_gpu_before is None else np.asarray(x_gpu_before, np.float64))
    dx_ref = np.asarray(x_ref, np.float64) - x_before
    sel = np.asarray(ora.field("I"), np.int64)
    rms = np.sqrt(np.mean(dx_ref[sel] ** 2)) if sel.size else 0.0
    err = np.abs(dx_gpu - dx_ref)[keep]
    # x itself is rounded to fp32 on both sides: allow one ulp of |x| on top of the relative bound on the change
    bound = REL * np.maximum(np.abs(dx_ref[keep]), rms) + 1.2e-7 * np.abs(np.asarray(x_ref, np.float64)[keep])
    assert (err <= bound).all(), f"x: {np.sum(err > bound)} coordinates outside tolerance, worst {err.max():.3e}"
    untouched = np.setdiff1d(np.arange(d), I_gpu)
    own_before = x_before.astype(np.float32) if x_gpu_before is None else np.asarray(x_gpu_before)
    assert np.array_equal(np.asarray(x_gpu)[untouched], own_before[untouched])
    return diff
