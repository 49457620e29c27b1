"""Pins of the oracle's polynomial estimator (paper Section 4.1 "Quantizing Polynomials", Section 4.2's protocol):
Q(P) = sum_i m_i prod_{j <= i} Q_j(a)^T x from d independent quantizations, and the gradient factor's plane mean.
Pinned by what the mathematics fixes: exact data give P(a^T x) itself, the estimate is unbiased (and a reused plane
is not), the extra pairs of quantizations differ from the first one exactly in the counter word the definition names."""
import numpy as np
import pytest

from oracle.build import build

build()
import oracle  # noqa: E402


def on_grid_samples(m, n, bits, seed):
    """Samples that sit on their feature's uniform grid (integers 0 .. 2^bits - 1, both ends present): every
    quantization reproduces them exactly."""
    rng = np.random.default_rng(seed)
    s = (1 << bits) - 1
    A = rng.integers(0, s + 1, size=(m, n)).astype(np.float32)
    A[0, :], A[1, :] = 0.0, float(s)
    return A


def planes_of(A, bits, seed, d, **kw):
    out, ds0 = [], None
    for q in range((d + 1) // 2):
        ds = oracle.quantize_pair(A, bits, seed, q, **kw)
        ds0 = ds0 or ds
        out += [ds.plane1, ds.plane2]
    return out[:d], ds0


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_exact_samples_give_the_polynomial_itself(bits):
    A = on_grid_samples(40, 13, bits, seed=bits)
    x = (np.random.default_rng(1).standard_normal(13) * 0.02).astype(np.float32)
    coef = [0.25, -1.0, 0.5, 2.0, -0.75]
    planes, ds = planes_of(A, bits, seed=7, d=4)
    z = A.astype(np.float64) @ x.astype(np.float64)
    want = sum(c * z ** i for i, c in enumerate(coef))
    got = oracle.poly_rows(planes, ds, x, coef)
    assert np.allclose(got, want, rtol=1e-12, atol=1e-12)
    b = np.where(np.arange(40) % 2 == 0, 1.0, -1.0).astype(np.float32)
    assert np.allclose(oracle.poly_rows(planes, ds, x, coef, scale=b), b * want, rtol=1e-12, atol=1e-12)
    # degree 0 and 1: a constant, and a line in the first plane's dot
    assert np.allclose(oracle.poly_rows([], ds, x, [3.5]), 3.5)
    assert np.allclose(oracle.poly_rows(planes[:1], ds, x, [1.0, 2.0]), 1.0 + 2.0 * z, rtol=1e-12)


def test_the_estimate_is_unbiased_and_a_reused_plane_is_not():
    rng = np.random.default_rng(3)
    m, n, bits, N = 6, 6, 2, 6000
    A = rng.uniform(-1.0, 1.0, (m, n)).astype(np.float32)
    x = rng.uniform(0.5, 1.5, n).astype(np.float32)
    coef = [0.1, 0.7, -0.4, 0.3]
    z = A.astype(np.float64) @ x.astype(np.float64)
    want = sum(c * z ** i for i, c in enumerate(coef))
    est, reused = np.zeros((N, m)), np.zeros((N, m))
    for s in range(N):
        planes, ds = planes_of(A, bits, seed=1000 + s, d=3)
        est[s] = oracle.poly_rows(planes, ds, x, coef)
        reused[s] = oracle.poly_rows([planes[0], planes[0]], ds, x, [0.0, 0.0, 1.0])        # (Q_1^T x)^2
    se = est.std(axis=0, ddof=1) / np.sqrt(N)
    assert (np.abs(est.mean(axis=0) - want) < 5 * se).all(), (est.mean(axis=0), want, se)
    assert (se > 1e-4).all()                                  # 2-bit samples: the estimate does vary
    # the square of one quantization's dot overshoots z^2 by that dot's variance: outside the error bars in every row
    se2 = reused.std(axis=0, ddof=1) / np.sqrt(N)
    assert (reused.mean(axis=0) - z ** 2 > 4 * se2).all(), ((reused.mean(axis=0) - z ** 2) / se2)


def test_further_pairs_use_the_counters_last_word():
    rng = np.random.default_rng(5)
    m, n, bits, seed = 9, 7, 4, 0x1234567890ABCDEF
    A = rng.standard_normal((m, n)).astype(np.float32)
    first = oracle.quantize(A, bits, seed)
    same = oracle.quantize_pair(A, bits, seed, 0)
    assert np.array_equal(first.plane1, same.plane1) and np.array_equal(first.plane2, same.plane2)
    lo, hi = oracle.column_range(A)
    s = (1 << bits) - 1
    for pair in (1, 2, 5):
        ds = oracle.quantize_pair(A, bits, seed, pair)
        assert np.array_equal(ds.feat_lo, first.feat_lo) and np.array_equal(ds.feat_step, first.feat_step)
        c1, c2 = oracle.unpack_plane(ds.plane1, n, bits), oracle.unpack_plane(ds.plane2, n, bits)
        for k in range(m):
            for j in range(n):
                inv = np.float32(s) / np.float32(hi[j] - lo[j])
                t = np.float32(np.float32(A[k, j] - lo[j]) * inv)
                cell = min(int(np.floor(t)), s - 1)
                p = np.float32(t - np.float32(cell))
                block = oracle.philox4x32_10((k, 0, j >> 1, pair), (seed & 0xFFFFFFFF, seed >> 32))
                for copy, codes in ((1, c1), (2, c2)):
                    u24 = block[2 * (j & 1) + copy - 1] >> 8
                    up = np.float32(u24) * np.float32(2.0 ** -24) < p
                    assert codes[k, j] == cell + int(up), (pair, k, j, copy)
        assert not np.array_equal(ds.plane1, first.plane1)


def test_weighted_plane_mean_against_exact_samples():
    A = on_grid_samples(30, 11, 4, seed=2)
    ds = oracle.quantize_pair(A, 4, 9, 1)
    c = np.random.default_rng(4).standard_normal(30)
    assert np.allclose(oracle.weighted_plane_mean(ds.plane2, ds, c), (c[:, None] * A).mean(axis=0), rtol=1e-12, atol=1e-12)
    assert np.allclose(oracle.weighted_plane_mean(ds.plane1, ds, np.ones(30)), A.astype(np.float64).mean(axis=0), rtol=1e-12)
    e = np.zeros(30)
    e[17] = 1.0
    assert np.allclose(oracle.weighted_plane_mean(ds.plane1, ds, e), A[17].astype(np.float64) / 30.0, rtol=1e-12)
