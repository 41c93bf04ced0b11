"""Pins for the oracle's Count Sketch, median unsketch and top-k (Section II-C, Algorithm 3)."""
import numpy as np
import pytest

import oracle


def _fam(seed, log2g, c, r, d):
    idx = np.empty((r, d), np.uint32)
    sgn = np.empty((r, d), np.int8)
    for j in range(r):
        idx[j], sgn[j] = oracle.hash_family(seed, log2g, c, j, 0, d)
    return idx, sgn


@pytest.mark.parametrize("log2g", [0, 3, 5])
def test_linearity_bit_exact_on_integers(log2g):
    # Section II-C: S(alpha g1 + beta g2) = alpha S(g1) + beta S(g2).  Small integers add exactly in fp32/fp64.
    d, r, c = 5000, 5, 256
    rng = np.random.default_rng(0)
    idx, sgn = _fam(9, log2g, c, r, d)
    a = rng.integers(-50, 51, d).astype(np.float32)
    b = rng.integers(-50, 51, d).astype(np.float32)
    Sa, Sb = oracle.sketch(a, r, c, idx, sgn), oracle.sketch(b, r, c, idx, sgn)
    assert np.array_equal(oracle.sketch(3 * a - 2 * b, r, c, idx, sgn), 3 * Sa - 2 * Sb)
    assert not oracle.sketch(np.zeros(d, np.float32), r, c, idx, sgn).any()
    # every row holds each coordinate exactly once: sum of a row = sum_i s_j(i) a_i
    for j in range(r):
        assert Sa[j].sum(dtype=np.float64) == (sgn[j].astype(np.float64) * a).sum()


def test_sketch_matches_definition_by_scatter():
    # independent evaluation of S[j,h_j(i)] += s_j(i) f_i with numpy's unbuffered scatter-add in fp64
    d, r, c = 3000, 3, 97
    rng = np.random.default_rng(1)
    idx = rng.integers(0, c, (r, d)).astype(np.uint32)
    sgn = rng.choice(np.array([-1, 1], np.int8), (r, d))
    a = rng.standard_normal(d).astype(np.float32)
    want = np.zeros((r, c))
    for j in range(r):
        np.add.at(want[j], idx[j], sgn[j] * a.astype(np.float64))
    got = oracle.sketch(a, r, c, idx, sgn)
    np.testing.assert_allclose(got, want, rtol=0, atol=2e-6)
    # a transposed (row, coordinate) indexing mistake would break this single-row spot check
    j, b = 2, int(idx[2, 17])
    assert abs(got[j, b] - (sgn[j] * a.astype(np.float64))[idx[j] == b].sum()) < 2e-6


def test_identity_hash_single_row_recovers_vector_exactly():
    # r = 1, injective bucket map, c >= d  =>  U(S(a)) = a bit for bit
    d = 777
    rng = np.random.default_rng(2)
    perm = rng.permutation(1000)[:d].astype(np.uint32)[None, :]
    sgn = rng.choice(np.array([-1, 1], np.int8), (1, d))
    a = rng.standard_normal(d).astype(np.float32)
    S = oracle.sketch(a, 1, 1000, perm, sgn)
    assert np.array_equal(oracle.unsketch(S, d, perm, sgn), a)
    vhat = rng.uniform(0.1, 4.0, d).astype(np.float32)
    want = (a.astype(np.float64) / np.sqrt(vhat.astype(np.float64))).astype(np.float32)
    assert np.array_equal(oracle.unsketch(S, d, perm, sgn, vhat), want)


@pytest.mark.parametrize("log2g", [0, 5])
def test_k_sparse_vector_recovered_exactly(log2g):
    # A k-sparse vector with c >> k: a coordinate's estimate is exact when, in more than half of the rows,
    # its bucket holds no OTHER support coordinate.  That condition is checked by brute force on the indices.
    d, r, c, k = 40_000, 5, 4096, 24
    rng = np.random.default_rng(3)
    idx, sgn = _fam(21, log2g, c, r, d)
    supp = np.sort(rng.choice(d, k, replace=False))
    a = np.zeros(d, np.float32)
    a[supp] = rng.uniform(0.5, 1.0, k).astype(np.float32) * rng.choice([-1.0, 1.0], k).astype(np.float32)
    est = oracle.unsketch(oracle.sketch(a, r, c, idx, sgn), d, idx, sgn)
    clean_rows = np.zeros(d, np.int64)
    for j in range(r):
        occ = np.bincount(idx[j, supp], minlength=c)
        others = occ[idx[j]] - np.isin(np.arange(d), supp)
        clean_rows += others == 0
    good = clean_rows > r // 2
    assert good.mean() > 0.99
    assert np.array_equal(est[good], a[good])
    if good[supp].all():
        assert np.array_equal(oracle.topk(est, k), supp.astype(np.uint32))


def test_median_against_sort_all_r():
    rng = np.random.default_rng(4)
    for r in range(1, 11):
        for _ in range(200):
            q = rng.standard_normal(r).astype(np.float32)
            if rng.random() < 0.3:
                q[rng.integers(0, r)] = q[0]               # ties
            assert oracle.median(q) == np.sort(q)[(r - 1) // 2]
    assert oracle.median(np.array([3, 1, 2], np.float32)) == 2.0
    assert oracle.median(np.array([4, 1, 3, 2], np.float32)) == 2.0   # even r: LOWER median


def test_topk_against_full_sort_with_ties():
    rng = np.random.default_rng(5)
    d = 20_000
    est = rng.standard_normal(d).astype(np.float32)
    est[rng.choice(d, 4000, replace=False)] = 0.75           # a large tie class, mixed signs
    est[rng.choice(d, 2000, replace=False)] = -0.75
    order = np.lexsort((np.arange(d), -np.abs(est)))         # magnitude desc, then index asc
    for k in (1, 2, 777, 9000, d):
        want = np.sort(order[:k]).astype(np.uint32)
        assert np.array_equal(oracle.topk(est, k), want)


def test_communication_volume():
    # Section III-B: |S| + P k + 2k floats per iteration; Section V-A setting: 10 x 100,000 sketch, k = 50,000,
    # P = 8, d ~ 25 M  =>  2d / volume = 33.3 ("about 32x").
    vol = oracle.comm_floats(10, 100_000, 50_000, 8)
    assert vol == 1_000_000 + 400_000 + 100_000
    assert abs(2 * 25_000_000 / vol - 33.33) < 0.01
