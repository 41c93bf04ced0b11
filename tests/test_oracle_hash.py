"""Pins for the oracle's hash and sign family (the bucket hashes h_j and sign hashes s_j of Section II-C).

The paper names the hashes but fixes no family, so the family is this library's own definition; it is
pinned by (a) the published known-answer vector of the splitmix64 generator it is built on, (b) an
arbitrary-precision re-evaluation of the definition, (c) the structural and statistical properties a Count
Sketch needs: range, sign domain, no collision inside a group, pair collisions at rate 1/c across groups,
balanced signs, uniform buckets.
"""
import os

import numpy as np
import pytest

import oracle
from conftest import GOLDEN

M64 = (1 << 64) - 1
GOLDEN_GAMMA = 0x9E3779B97F4A7C15


def test_splitmix64_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "splitmix64_kat.txt")) if l[0] != "#"]
    assert len(rows) == 5
    for s0, t, want in rows:
        assert oracle.stream(int(s0), int(t)) == int(want)


def _mix(z):
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M64
    return z ^ (z >> 31)


def _family(seed, log2g, c, row, i):
    """The family's definition evaluated with Python integers (no fixed-width arithmetic)."""
    g = 1 << log2g
    G = c // g
    K = _mix((seed + (row + 1) * GOLDEN_GAMMA) & M64)
    q, o = divmod(i, g)
    u = _mix((K + (q + 1) * GOLDEN_GAMMA) & M64)
    hi, lo = divmod(u, 1 << 32)
    B, rem = divmod(hi * G, 1 << 32)
    p = (rem * g) >> 32                      # leading log2(g) bits of the 32-bit remainder
    return g * B + (o ^ p), (-1 if lo & 1 else 1)          # one sign per (row, group)


@pytest.mark.parametrize("log2g", [0, 1, 2, 3, 4, 5])
@pytest.mark.parametrize("c", [2048, 100_000, 250_000, 401])
def test_family_matches_bigint_definition(log2g, c):
    if c >> log2g == 0:
        pytest.skip("c < g")
    rng = np.random.default_rng(7)
    for seed in (0, 1, 0xDEADBEEFCAFEF00D):
        for row in (0, 3, 9):
            starts = [0, 1, 31, 33, int(rng.integers(0, 2**31)), 2**32 - 70]
            for i0 in starts:
                b, s = oracle.hash_family(seed, log2g, c, row, i0, 64)
                for t in range(64):
                    wb, ws = _family(seed, log2g, c, row, i0 + t)
                    assert (int(b[t]), int(s[t])) == (wb, ws)


@pytest.mark.parametrize("log2g", [0, 2, 5])
def test_range_sign_domain_determinism(log2g):
    c = 250_000
    b, s = oracle.hash_family(0, log2g, c, 1, 0, 200_000)
    b2, s2 = oracle.hash_family(0, log2g, c, 1, 0, 200_000)
    assert np.array_equal(b, b2) and np.array_equal(s, s2)
    assert b.max() < (c >> log2g) << log2g <= c
    assert set(np.unique(s)) == {-1, 1}
    # another row and another seed give different functions
    b3, _ = oracle.hash_family(0, log2g, c, 2, 0, 200_000)
    b4, _ = oracle.hash_family(1, log2g, c, 1, 0, 200_000)
    assert (b != b3).mean() > 0.99 and (b != b4).mean() > 0.99


@pytest.mark.parametrize("log2g", [1, 3, 5])
def test_group_is_a_permutation_of_one_aligned_block(log2g):
    g = 1 << log2g
    c = 100_000
    b, _ = oracle.hash_family(5, log2g, c, 0, 0, g * 4096)
    blk = b.reshape(-1, g)
    base = (blk[:, :1] // g) * g
    assert np.all(blk // g * g == base)                       # one aligned block of g buckets per group
    assert np.all(np.sort(blk - base, axis=1) == np.arange(g))  # every offset used exactly once
    # xor structure: offset(o) ^ o is constant inside a group
    x = (blk - base) ^ np.arange(g)
    assert np.all(x == x[:, :1])
    # the xor constant takes every value
    assert len(np.unique(x[:, 0])) == g


@pytest.mark.parametrize("log2g", [0, 3, 5])
def test_bucket_uniformity_chi_square(log2g):
    c, N = 2048, 2048 * 400
    b, _ = oracle.hash_family(11, log2g, c, 2, 0, N)
    cnt = np.bincount(b, minlength=c).astype(np.float64)
    chi2 = ((cnt - N / c) ** 2 / (N / c)).sum()
    # grouped buckets are filled in blocks of g, so compare at block level too; dof ~ c-1, sd ~ sqrt(2c)
    if log2g == 0:
        assert abs(chi2 - (c - 1)) < 6 * np.sqrt(2 * (c - 1))
    G = c >> log2g
    gcnt = cnt.reshape(G, -1).sum(1) / (1 << log2g)          # groups per block
    ng = N >> log2g
    chi2g = ((gcnt - ng / G) ** 2 / (ng / G)).sum()
    assert abs(chi2g - (G - 1)) < 6 * np.sqrt(2 * (G - 1))


@pytest.mark.parametrize("log2g", [0, 2, 5])
def test_pair_collision_rate_and_sign_balance(log2g):
    c, N = 4096, 60_000
    g = 1 << log2g
    b, s = oracle.hash_family(3, log2g, c, 0, 0, N)
    # one sign per (row, group): constant inside a group (whose coordinates never meet in a bucket), balanced and
    # uncorrelated across groups (whose coordinates do), and uncorrelated across rows
    sg = s[: (N // g) * g].reshape(-1, g).astype(np.float64)
    assert np.all(sg == sg[:, :1])
    n_groups = sg.shape[0]
    assert abs(sg[:, 0].mean()) < 5 / np.sqrt(n_groups)
    for lag in (1, 2, 7):
        assert abs((sg[:-lag, 0] * sg[lag:, 0]).mean()) < 5 / np.sqrt(n_groups)
    s_other = oracle.hash_family(3, log2g, c, 1, 0, N)[1][: (N // g) * g].reshape(-1, g)[:, 0].astype(np.float64)
    assert abs((sg[:, 0] * s_other).mean()) < 5 / np.sqrt(n_groups)
    # collisions: count pairs sharing a bucket
    cnt = np.bincount(b, minlength=c).astype(np.float64)
    pairs_same_bucket = (cnt * (cnt - 1) / 2).sum()
    cross_pairs = N * (N - 1) / 2 - (N // g) * g * (g - 1) / 2
    rate = pairs_same_bucket / cross_pairs
    assert abs(rate * c - 1) < 0.02
    # no two coordinates of one group share a bucket
    blk = b[: (N // g) * g].reshape(-1, g)
    assert all(len(np.unique(row)) == g for row in blk[:2000])


def test_non_divisible_c_leaves_tail_buckets_unused():
    c, log2g = 250_000, 5            # 250000 = 32*7812 + 16
    b, _ = oracle.hash_family(0, log2g, c, 0, 0, 500_000)
    assert b.max() < 7812 * 32


# ---------------------------------------------------------------------------------------------- windowed family
def _family_w(seed, L, c, row, i):
    """Windowed family (g = 32) evaluated with Python integers."""
    cw = 32 * L
    P = c // cw
    K = _mix((seed + (row + 1) * GOLDEN_GAMMA) & M64)
    q, o = divmod(i, 32)
    u = _mix((K + (q + 1) * GOLDEN_GAMMA) & M64)
    hi, lo = divmod(u, 1 << 32)
    line, rem = divmod(hi * L, 1 << 32)
    p = (rem * 32) >> 32
    return ((i // 1024) % P) * cw + 32 * line + (o ^ p), (-1 if lo & 1 else 1)


@pytest.mark.parametrize("L", [1, 4, 8, 16])
@pytest.mark.parametrize("c", [2048, 250_000, 1_000_000])
def test_windowed_family_matches_bigint_definition(L, c):
    for seed in (0, 77):
        for row in (0, 4):
            for i0 in (0, 1000, 1024 * 977 + 5, 2**32 - 70):
                b, s = oracle.hash_family(seed, 5, c, row, i0, 64, window_lines=L)
                for t in range(64):
                    assert (int(b[t]), int(s[t])) == _family_w(seed, L, c, row, i0 + t)


def test_windowed_family_structure():
    c, L, N = 250_000, 8, 1024 * 3000
    cw, P = 32 * L, 250_000 // (32 * L)
    b, s = oracle.hash_family(2, 5, c, 1, 0, N, window_lines=L)
    unit = np.arange(N) // 1024
    # every coordinate lands in the window of its unit's panel
    assert np.array_equal(b // cw, unit % P)
    assert b.max() < P * cw <= c
    # inside a group: a permutation of one aligned line
    blk = b.reshape(-1, 32)
    assert np.all(blk // 32 == blk[:, :1] // 32)
    assert np.all(np.sort(blk % 32, axis=1) == np.arange(32))
    # lines inside a window are used uniformly
    line = (blk[:, 0] % cw) // 32
    cnt = np.bincount(line, minlength=L).astype(np.float64)
    assert abs(cnt / cnt.sum() - 1 / L).max() < 0.01
    assert abs(s.astype(np.float64).mean()) < 5 / np.sqrt(N)
    # pair collisions: 1/cw between different groups of one panel, none across panels
    one = b[unit % P == 3]
    cc = np.bincount(one - 3 * cw, minlength=cw).astype(np.float64)
    pairs = (cc * (cc - 1) / 2).sum()
    n1 = one.size
    cross = n1 * (n1 - 1) / 2 - (n1 // 32) * 32 * 31 / 2
    assert abs(pairs / cross * cw - 1) < 0.05
    # the row as a whole is still filled evenly: about N/c coordinates per bucket
    tot = np.bincount(b, minlength=c)[: P * cw].astype(np.float64)
    assert abs(tot.mean() - N / (P * cw)) < 1e-9 and tot.std() / tot.mean() < 0.5
