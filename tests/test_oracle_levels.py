"""Pins of the oracle's variance-optimal level placement (Section 3 of the paper)."""
import itertools

import numpy as np
import pytest

import oracle


def direct_cost(cnt, j, m):
    """4 M^2 * sum over bins i in [j, m) of cnt_i * err(centre_i, [d_j, d_m]) by exact fractions."""
    from fractions import Fraction
    M = len(cnt)
    tot = Fraction(0)
    for i in range(j, m):
        x = Fraction(2 * i + 1, 2 * M)
        tot += int(cnt[i]) * (Fraction(m, M) - x) * (x - Fraction(j, M))
    val = tot * 4 * M * M
    assert val.denominator == 1
    return int(val)


def test_interval_cost_is_the_variance_of_the_bin_centres():
    rng = np.random.default_rng(0)
    for M in (1, 2, 5, 12):
        cnt = rng.integers(0, 50, M).astype(np.uint32)
        for j in range(M):
            for m in range(j + 1, M + 1):
                want = direct_cost(cnt, j, m)
                assert oracle.interval_cost(cnt, j, m) == want
                assert oracle.interval_cost_prefix(cnt, j, m) == want
    # no overflow at the documented limits: 10^9 points in one bin of 1024
    cnt = np.zeros(1024, np.uint32)
    cnt[1023] = 1_000_000_000
    assert oracle.interval_cost_prefix(cnt, 0, 1024) == 10 ** 9 * 1 * 2047
    assert oracle.interval_cost(cnt, 0, 1024) == 10 ** 9 * 2047


@pytest.mark.parametrize("M,s", [(4, 2), (6, 3), (9, 3), (10, 4), (14, 4), (12, 1), (7, 7), (8, 6)])
def test_dp_matches_brute_force_over_all_level_sets(M, s):
    rng = np.random.default_rng(M * 31 + s)
    for trial in range(30):
        kind = trial % 3
        if kind == 0:
            cnt = rng.integers(0, 100, M)
        elif kind == 1:
            cnt = (rng.random(M) < 0.4) * rng.integers(1, 1000, M)      # many empty bins -> ties
        else:
            cnt = np.round(1000 * np.exp(-np.arange(M))).astype(int)     # heavily skewed
        cnt = cnt.astype(np.uint32)
        idx, obj = oracle.levels_dp(cnt, s)
        bidx, bobj = oracle.levels_bruteforce(cnt, s)
        assert obj == bobj
        assert idx[0] == 0 and idx[-1] == M and (np.diff(idx) > 0).all()
        assert sum(direct_cost(cnt, idx[i], idx[i + 1]) for i in range(s)) == obj
        # python brute force, independent of both
        best = min(sum(direct_cost(cnt, e[i], e[i + 1]) for i in range(s))
                   for e in ([0, *c, M] for c in itertools.combinations(range(1, M), s - 1)))
        assert obj == best


def test_dp_never_worse_than_uniform_and_respects_symmetry():
    rng = np.random.default_rng(7)
    M, s = 64, 4
    for _ in range(10):
        cnt = rng.integers(0, 500, M).astype(np.uint32)
        idx, obj = oracle.levels_dp(cnt, s)
        uni = sum(oracle.interval_cost(cnt, i * M // s, (i + 1) * M // s) for i in range(s))
        assert obj <= uni
        _, obj_rev = oracle.levels_dp(cnt[::-1].copy(), s)
        assert obj_rev == obj
    sym = np.concatenate([np.arange(1, 33) ** 2, np.arange(32, 0, -1) ** 2]).astype(np.uint32)
    idx, _ = oracle.levels_dp(sym, 4)
    assert idx[2] == 32 and idx[1] + idx[3] == 64
    # all mass in one bin: the optimum brackets that bin as tightly as the edges allow
    one = np.zeros(32, np.uint32)
    one[10] = 1000
    idx, obj = oracle.levels_dp(one, 3)
    assert 10 in idx and 11 in idx and obj == 1000


def test_lemma_optimal_endpoints_lie_at_data_points():
    rng = np.random.default_rng(11)
    for _ in range(5):
        pts = np.sort(rng.random(7))
        s = 3
        cands = [0.0, *pts, 1.0]
        best_data = min(oracle.total_variance(pts, np.array([0.0, a, b, 1.0]))
                        for a, b in itertools.combinations(cands, 2) if a <= b)
        grid = np.linspace(0, 1, 101)
        best_grid = min(oracle.total_variance(pts, np.array([0.0, a, b, 1.0]))
                        for a, b in itertools.combinations_with_replacement(grid, 2))
        assert best_data <= best_grid + 1e-12
    # total_variance is sum (b - x)(x - a) over the cell that holds x
    assert abs(oracle.total_variance(np.array([0.25, 0.75]), np.array([0.0, 0.5, 1.0])) - 2 * 0.0625) < 1e-15
    assert abs(oracle.total_variance(np.array([0.1]), np.array([0.0, 0.4, 1.0])) - 0.3 * 0.1) < 1e-15


def test_dp_objective_equals_total_variance_for_points_at_bin_centres():
    rng = np.random.default_rng(5)
    M, s = 16, 3
    cnt = rng.integers(0, 6, M).astype(np.uint32)
    pts = np.repeat((np.arange(M) + 0.5) / M, cnt)
    idx, obj = oracle.levels_dp(cnt, s)
    tv = oracle.total_variance(pts, idx / M)
    assert abs(tv * 4 * M * M - obj) < 1e-9 * max(1, obj)


def test_discretisation_gap_within_the_theorem_bound():
    # Theorem (discretisation): MV(discrete) - MV(optimal) <= a^2 b k / (4 M^3) + a^2 b c^2 / (M k)
    rng = np.random.default_rng(2)
    N, M, k = 400, 32, 3
    pts = np.sort(rng.beta(2, 5, N))
    # exact optimum over data points (Lemma) by the same recursion on raw points, in numpy
    cands = np.concatenate([[0.0], pts, [1.0]])

    def tv(e):
        return oracle.total_variance(pts, np.asarray(e, np.float64))
    best = None
    for a_i in range(0, len(cands), 4):
        for b_i in range(a_i, len(cands), 4):
            v = tv([0.0, cands[a_i], cands[b_i], 1.0])
            if best is None or v < best[0]:
                best = (v, cands[a_i], cands[b_i])
    mv_opt_upper = best[0] / N                       # an upper bound of the true optimum is enough
    lo, hi = np.float32(0.0), np.float32(1.0)
    A = np.concatenate([[0.0], pts, [1.0]]).astype(np.float32)[:, None]
    cnt = oracle.histogram(A, M, np.array([lo]), np.array([hi]))[0]
    idx, _ = oracle.levels_dp(cnt, k)
    mv_disc = tv(idx / M) / N
    b = cnt.max() * M / (N + 2)
    widths = np.diff([0.0, best[1], best[2], 1.0])
    c = np.ceil(widths.max() * M + 1) * k / M
    bound = b * k / (4 * M ** 3) + b * c * c / (M * k)
    assert mv_disc - mv_opt_upper <= bound
    assert mv_disc <= tv(np.linspace(0, 1, k + 1)) / N + 1e-12     # and beats the uniform placement


def test_histogram_bins_and_level_values():
    A = np.array([[0.0], [1.0], [0.4999], [0.5], [0.999], [0.25]], np.float32)
    cnt = oracle.histogram(A, 4, np.array([0.0], np.float32), np.array([1.0], np.float32))[0]
    assert list(cnt) == [1, 2, 1, 2]                  # hi goes to the last bin; edges belong to the right bin
    lev = oracle.levels_from_idx(np.array([0, 3, 7, 16]), 16, np.float32(-2.0), np.float32(6.0))
    assert list(lev) == [-2.0, -0.5, 1.5, 6.0]
    const = oracle.histogram(np.full((5, 1), 3.0, np.float32), 8, np.array([3.0], np.float32),
                             np.array([3.0], np.float32))[0]
    assert list(const) == [5, 0, 0, 0, 0, 0, 0, 0]


def test_optimal_levels_end_to_end_lower_variance_than_uniform():
    rng = np.random.default_rng(9)
    m, n, bits, M = 4000, 6, 3, 256
    A = (np.exp(1.5 * rng.standard_normal((m, n))) * rng.choice([-1, 1], (m, n))).astype(np.float32)
    A /= np.abs(A).max(0, keepdims=True)
    A[:, 5] = 0.25                                   # a constant feature
    lev, obj = oracle.optimal_levels(A, bits, M)
    lo, hi = oracle.column_range(A)
    assert (lev[:, 0] == lo).all() and (lev[:, -1] == hi).all()
    assert (np.diff(lev[:5], axis=1) > 0).all() and (lev[5] == 0.25).all()
    cnt = oracle.histogram(A, M, lo, hi)
    for j in range(5):
        idx, o = oracle.levels_dp(cnt[j], 7)
        assert o == obj[j]
        assert np.array_equal(lev[j], oracle.levels_from_idx(idx, M, lo[j], hi[j]))
        x = A[:, j].astype(np.float64)
        e_opt = lev[j].astype(np.float64)
        e_uni = np.linspace(lo[j], hi[j], 8)
        assert oracle.total_variance(x, e_opt) < 0.5 * oracle.total_variance(x, e_uni)
    # quantizing onto the table stays unbiased and inside the table
    ds = oracle.quantize(A, bits, seed=3, mode=oracle.TABLE, levels=lev)
    codes = oracle.unpack_plane(ds.plane1[:50], n, bits)
    assert codes.max() <= 7
    for k in range(50):
        q = ds.dequantize(1, k)
        for j in range(n):
            c = codes[k, j]
            assert lev[j, max(c - 1, 0)] <= A[k, j] <= lev[j, min(c + 1, 7)]
            assert q[j] == lev[j, c]
