"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU needed).

Each test is chosen so that a plausible mistake in the oracle (a dropped term, a wrong sign or
index, both copies drawn from the same random word, a sum where a mean belongs) fails it.
"""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def np_unpack(plane, n, bits):
    """Independent vectorised unpack of the canonical layout (low bits first)."""
    cb = {2: 2, 3: 4, 4: 4, 8: 8}[bits]
    per = 8 // cb
    cols = np.arange(n)
    byte = plane[:, cols // per]
    return (byte >> ((cols % per) * cb).astype(np.uint8)) & ((1 << cb) - 1)


def np_dequant(ds, which):
    codes = np_unpack(ds.plane1 if which == 1 else ds.plane2, ds.n, ds.bits).astype(np.int64)
    if ds.mode == oracle.UNIFORM:
        return ds.feat_lo.astype(np.float64)[None, :] + codes * ds.feat_step.astype(np.float64)[None, :]
    return np.take_along_axis(ds.levels.astype(np.float64), codes.T, axis=1).T


# ---------------------------------------------------------------------------------------------
# Random numbers
# ---------------------------------------------------------------------------------------------
def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 3
    for r in rows:
        v = [int(t, 16) for t in r]
        out = oracle.philox4x32_10(v[0:4], v[4:6])
        assert [int(o) for o in out] == v[6:10]


def test_u24_keying_and_uniformity():
    # the four words of one block serve (feature pair) x (copy); distinct keys give distinct draws
    out = oracle.philox4x32_10([5, 0, 3, 0], [7, 0])
    assert oracle.u24_sample(7, 5, 6, 1) == int(out[0]) >> 8
    assert oracle.u24_sample(7, 5, 6, 2) == int(out[1]) >> 8
    assert oracle.u24_sample(7, 5, 7, 1) == int(out[2]) >> 8
    assert oracle.u24_sample(7, 5, 7, 2) == int(out[3]) >> 8
    assert oracle.u24_sample(7 + (1 << 32), 5, 6, 1) != oracle.u24_sample(7, 5, 6, 1)
    assert oracle.u24_sample(7, 5 + (1 << 32), 6, 1) != oracle.u24_sample(7, 5, 6, 1)
    vout = oracle.philox4x32_10([2, 11, 4, 3], [9, 1])
    assert oracle.u24_vector(9 + (1 << 32), 4, 11, 9, 3) == int(vout[1]) >> 8
    # chi-square of the top byte over a 200 x 200 block of (row, feature), both copies: df = 255
    for copy in (1, 2):
        u = np.array([[oracle.u24_sample(123, r, f, copy) for f in range(200)] for r in range(200)])
        assert u.max() < (1 << 24)
        cnt = np.bincount((u >> 16).ravel(), minlength=256)
        chi2 = ((cnt - u.size / 256) ** 2 / (u.size / 256)).sum()
        assert chi2 < 255 + 5 * np.sqrt(2 * 255)


# ---------------------------------------------------------------------------------------------
# Packing
# ---------------------------------------------------------------------------------------------
def test_pack_hand_example():
    for line in open(os.path.join(GOLDEN, "pack_example.txt")):
        if not line.strip() or line[0] == "#":
            continue
        tok = line.split()
        bits, codes, want = int(tok[0]), [int(t) for t in tok[1:8]], [int(t, 16) for t in tok[8:]]
        row = oracle.pack_codes(np.array(codes, np.uint8), bits)
        assert row.shape[0] == 16
        assert list(row[: len(want)]) == want
        assert not row[len(want):].any()


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_pack_round_trip(bits):
    rng = np.random.default_rng(bits)
    for n in (1, 3, 16, 63, 64, 65, 257, 1000):
        codes = rng.integers(0, 1 << bits, n).astype(np.uint8)
        row = oracle.pack_codes(codes, bits)
        assert row.shape[0] % 16 == 0 and row.shape[0] == oracle.row_bytes(n, bits)
        assert (oracle.unpack_codes(row, n, bits) == codes).all()
        assert (np_unpack(row[None, :], n, bits)[0] == codes).all()
    assert oracle.row_bytes(1000, 8) == 1008 and oracle.row_bytes(2048, 2) == 512
    assert oracle.row_bytes(512, 3) == 256 and oracle.row_bytes(32768, 4) == 16384


# ---------------------------------------------------------------------------------------------
# Stochastic quantization: E[Q(v)] = v, Var = (up - v)(v - low), independence of the two copies
# ---------------------------------------------------------------------------------------------
N_DRAWS = 1_000_000


def _constant_columns(values, lo, hi):
    A = np.empty((N_DRAWS + 2, len(values)), np.float32)
    A[0], A[1], A[2:] = lo, hi, np.asarray(values, np.float32)[None, :]
    return A


@pytest.mark.parametrize("bits,lo,hi", [(2, -0.3, 2.1), (4, -1.0, 1.0), (8, -3.0, 3.0), (3, 0.0, 3.5)])
def test_uniform_quantizer_unbiased_with_exact_variance(bits, lo, hi):
    s = (1 << bits) - 1
    step = (hi - lo) / s
    vals = [lo + 0.7 * step, lo + 1.001 * step, lo + (s - 0.5) * step, lo + (s - 1e-3) * step, lo + 0.25 * (hi - lo),
            lo + 2 * step]
    A = _constant_columns(vals, lo, hi)
    ds = oracle.quantize(A, bits, seed=42 + bits)
    assert np.allclose(ds.feat_lo, lo) and np.allclose(ds.feat_step, np.float32(hi - np.float32(lo)) / s, rtol=1e-6)
    zs = []
    for which in (1, 2):
        q = np_dequant(ds, which)
        assert (q[0] == ds.feat_lo).all()                          # v = lo -> code 0
        assert np.allclose(q[1], hi, atol=1e-6 * max(1, abs(hi)))  # v = hi -> top code, always
        for j, v in enumerate(np.asarray(vals, np.float32).astype(np.float64)):
            draws = q[2:, j]
            low = lo + np.floor((v - lo) / step + 1e-9) * step
            var = max((low + step - v) * (v - low), 0.0)
            sigma = np.sqrt(var / N_DRAWS)
            slack = 2e-7 * max(1, abs(hi))                         # fp32 rounding of p and of step
            # each mean within 3 sigma, except that among this many simultaneous checks one may
            # reach 4.5; the pooled z-score below is the sharp 3-sigma statement
            assert abs(draws.mean() - v) <= 4.5 * sigma + slack
            if var > 1e-4 * step * step:
                zs.append((draws.mean() - v) / sigma)
            # sample variance of a two-point law: its own deviation is <= step^2 sqrt(p(1-p)/N)
            assert abs(draws.var() - var) <= 4 * step * np.sqrt(var / N_DRAWS) + 1e-9
            assert var <= step * step / 4 + 1e-12
            assert set(np.unique(np.round((draws - low) / step))) <= {0.0, 1.0}
    zs = np.array(zs)
    assert abs(zs.sum() / np.sqrt(len(zs))) <= 3.0 + 0.05         # pooled over all values and copies
    assert (np.abs(zs) > 3).sum() <= 1
    # the two copies are independent draws
    up1 = np_unpack(ds.plane1, ds.n, bits)[2:, 0].astype(np.float64)
    up2 = np_unpack(ds.plane2, ds.n, bits)[2:, 0].astype(np.float64)
    assert abs(np.corrcoef(up1, up2)[0, 1]) < 4 / np.sqrt(N_DRAWS)


def test_paper_example_0p7_between_0_and_1():
    # Section 2.2, "Overhead of Storing Samples": 0.7 quantized to 0 or 1 -> up with probability 0.7
    A = _constant_columns([0.7], 0.0, 3.0)
    ds = oracle.quantize(A, 2, seed=1)
    codes = np_unpack(ds.plane1, 1, 2)[2:, 0]
    assert set(np.unique(codes)) == {0, 1}
    assert abs(codes.mean() - 0.7) <= 3 * np.sqrt(0.21 / N_DRAWS) + 1e-7


def test_table_quantizer_unbiased():
    lev = np.array([[-1.0, -0.5, -0.1, 0.05, 0.2, 0.4, 0.9, 1.0]], np.float32)
    vals = [-0.75, -0.100001, 0.0, 0.3, 0.95, 0.4]
    A = _constant_columns(vals, -1.0, 1.0)
    ds = oracle.quantize(A, 3, seed=5, mode=oracle.TABLE, levels=np.repeat(lev, len(vals), 0))
    levd = lev[0].astype(np.float64)
    for which in (1, 2):
        q = np_dequant(ds, which)
        assert (q[0] == -1.0).all() and (q[1] == 1.0).all()
        for j, v in enumerate(np.asarray(vals, np.float32).astype(np.float64)):
            c = max(i for i in range(7) if levd[i] <= v)
            var = (levd[c + 1] - v) * (v - levd[c])
            assert set(np.unique(q[2:, j])) <= {levd[c], levd[c + 1]}
            assert abs(q[2:, j].mean() - v) <= 3 * np.sqrt(var / N_DRAWS) + 2e-7   # 12 checks: 3 sigma each
            width = levd[c + 1] - levd[c]
            assert abs(q[2:, j].var() - var) <= 4 * width * np.sqrt(var / N_DRAWS) + 1e-9


def test_quantize_edge_cases():
    A = np.array([[1.0, 5.0, -2.0], [1.0, 7.0, 2.0], [1.0, 6.0, 0.0]], np.float32)
    ds = oracle.quantize(A, 4, seed=0)
    c1, c2 = np_unpack(ds.plane1, 3, 4), np_unpack(ds.plane2, 3, 4)
    assert (c1[:, 0] == 0).all() and (c2[:, 0] == 0).all() and ds.feat_step[0] == 0  # constant feature
    assert c1[0, 1] == 0 and c1[1, 1] == 15 and c2[0, 2] == 0 and c2[1, 2] == 15
    assert ds.plane1[:, 2:].sum() == 0                                            # padding stays zero
    bad = A.copy()
    bad[1, 1] = np.nan
    with pytest.raises(oracle.OracleError) as e:
        oracle.quantize(bad, 4, seed=0)
    assert e.value.code == oracle.ERR_NONFINITE
    for bits in (0, 9, 16):
        with pytest.raises(oracle.OracleError):
            oracle.quantize(A, bits, seed=0)
    with pytest.raises(oracle.OracleError):
        oracle.quantize(A, 8, seed=0, mode=oracle.TABLE, levels=np.zeros((3, 256), np.float32))


# ---------------------------------------------------------------------------------------------
# Row-scaled quantizer for model and gradient: unbiased, closed-form variance, the Lemma's bound
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("bits", [2, 4, 8])
def test_vector_quantizer_l2_scaled(bits):
    rng = np.random.default_rng(3)
    n, reps = 48, 20000
    v = rng.standard_normal(n).astype(np.float32)
    v[5] = 0.0
    sm = (1 << (bits - 1)) - 1
    M = float(np.float32(np.sqrt((v.astype(np.float64) ** 2).sum())))
    acc = np.zeros(n)
    acc2 = np.zeros(n)
    tv = 0.0
    for r in range(reps):
        q, codes = oracle.quantize_vector(v, bits, seed=11, epoch=r // 1000, step=r % 1000, stream=3)
        assert np.abs(codes).max() <= sm
        assert np.allclose(q, M * codes / sm, rtol=1e-6, atol=0)
        acc += q
        acc2 += q.astype(np.float64) ** 2
        tv += ((q.astype(np.float64) - v) ** 2).sum()
    t = np.abs(v.astype(np.float64)) / M * sm
    p = t - np.floor(t)
    var = (M / sm) ** 2 * p * (1 - p)
    mean = acc / reps
    assert (np.abs(mean - v) <= 4 * np.sqrt(var / reps) + 1e-6).all()
    emp_var = acc2 / reps - mean ** 2
    assert (np.abs(emp_var - var) <= 5 * (M / sm) ** 2 * np.sqrt(p * (1 - p) / reps) + 1e-9).all()
    assert mean[5] == 0.0
    bound = min(n / sm ** 2, np.sqrt(n) / sm) * float((v.astype(np.float64) ** 2).sum())
    assert tv / reps <= bound
    # different stream / step -> different draws; zero vector -> zero
    a, _ = oracle.quantize_vector(v, bits, 11, 0, 0, 3)
    b_, _ = oracle.quantize_vector(v, bits, 11, 0, 0, 4)
    assert (a != b_).any()
    z, zc = oracle.quantize_vector(np.zeros(7, np.float32), bits, 1, 0, 0, 3)
    assert not z.any() and not zc.any()


# ---------------------------------------------------------------------------------------------
# Double sampling: naive estimator biased by D_a x, double-sampled forms unbiased
# ---------------------------------------------------------------------------------------------
def test_naive_bias_closed_form_and_double_sampling_unbiased():
    bits, n = 2, 6
    rng = np.random.default_rng(0)
    a = rng.uniform(-0.9, 0.9, n).astype(np.float32)
    x = rng.standard_normal(n).astype(np.float32) * 2
    bk = np.float32(0.3)
    A = _constant_columns(a, -1.0, 1.0)
    ds = oracle.quantize(A, bits, seed=77)
    sub = oracle.Dataset(ds.plane1[2:], ds.plane2[2:], N_DRAWS, n, bits, ds.mode, ds.feat_lo, ds.feat_step, None)
    bvec = np.full(N_DRAWS, bk, np.float32)
    ad, xd = a.astype(np.float64), x.astype(np.float64)
    true = ad * (ad @ xd - float(bk))
    step = 2.0 / 3
    low = -1 + np.floor((ad + 1) / step) * step
    D = (low + step - ad) * (ad - low)
    naive = oracle.estimator_mean(sub, bvec, x, 0)
    one_sided = oracle.estimator_mean(sub, bvec, x, 1)
    sym = oracle.estimator_mean(sub, bvec, x, 2)
    tol = 8e-3
    assert np.abs(naive - (true + D * xd)).max() < tol          # Section 2.2: E = true + D_a x
    assert np.abs(naive - true).max() > 10 * tol                 # and the bias is not small here
    assert np.abs(one_sided - true).max() < tol
    assert np.abs(sym - true).max() < tol
    # the training step itself uses the symmetrised, cross-paired form (one full-batch step)
    _, g = oracle.sgd_epoch(sub, bvec, x, batch=N_DRAWS, lr=0.0, want_grad=True)
    assert np.allclose(g[0], sym, rtol=1e-5, atol=1e-6)
    assert np.abs(g[0] - true).max() < tol


def test_model_quantization_keeps_gradient_unbiased():
    rng = np.random.default_rng(1)
    m, n = 64, 12
    A = rng.integers(0, 16, (m, n)).astype(np.float32)
    A[0], A[1] = 0, 15
    x = rng.standard_normal(n).astype(np.float32)
    b = rng.standard_normal(m).astype(np.float32)
    ds = oracle.quantize(A, 4, seed=3)
    _, g0 = oracle.sgd_epoch(ds, b, x, batch=m, lr=0.0, want_grad=True)
    acc = np.zeros(n)
    reps = 4000
    for r in range(reps):
        _, g = oracle.sgd_epoch(ds, b, x, batch=m, lr=0.0, model_bits=4, seed=9, epoch=r, want_grad=True)
        acc += g[0]
    # per-draw gradient deviation is ~ |A^T A| * ||x|| / s_m / sqrt(n); 4 sigma of the mean
    dev = np.abs(acc / reps - g0[0])
    scale = np.abs(A.T @ A / m).sum(1) * np.linalg.norm(x) / 7
    assert (dev < 4 * scale / np.sqrt(reps)).all()
    assert dev.max() > 0


# ---------------------------------------------------------------------------------------------
# Mini-batch step: on-grid data reduce it to the textbook least-squares minibatch gradient
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("bits,m,n,batch", [(4, 50, 7, 16), (8, 37, 19, 5), (2, 33, 65, 33), (3, 20, 9, 64)])
def test_on_grid_data_gives_textbook_minibatch_sgd(bits, m, n, batch):
    rng = np.random.default_rng(bits * 100 + m)
    top = (1 << bits) - 1
    A = rng.integers(0, top + 1, (m, n)).astype(np.float32) - 2.0
    A[0], A[1] = -2.0, top - 2.0                       # every column spans the grid: step = 1 exactly
    b = rng.standard_normal(m).astype(np.float32)
    x0 = rng.standard_normal(n).astype(np.float32) * 0.1
    ds = oracle.quantize(A, bits, seed=4)
    assert (np_dequant(ds, 1) == A).all() and (np_dequant(ds, 2) == A).all()
    T = (m + batch - 1) // batch
    order = rng.permutation(T).astype(np.int32)
    lr = 0.01
    x_ref = x0.astype(np.float64)
    Ad, bd = A.astype(np.float64), b.astype(np.float64)
    for t in order:
        rows = slice(t * batch, min(m, (t + 1) * batch))
        g_ref = Ad[rows].T @ (Ad[rows] @ x_ref - bd[rows]) / (rows.stop - rows.start)
        x_ref = x_ref - lr * g_ref
    x1, g = oracle.sgd_epoch(ds, b, x0, batch=batch, lr=lr, batch_order=order, want_grad=True)
    assert np.allclose(x1, x_ref, rtol=2e-5, atol=2e-6)
    # last step's gradient, computed from the model just before it
    xb, _ = oracle.sgd_epoch(ds, b, x0, batch=batch, lr=lr, batch_order=order, num_steps=T - 1)
    rows = slice(order[-1] * batch, min(m, (order[-1] + 1) * batch))
    g_last = Ad[rows].T @ (Ad[rows] @ xb.astype(np.float64) - bd[rows]) / (rows.stop - rows.start)
    assert np.allclose(g[0], g_last, rtol=1e-5, atol=1e-6) and (g[0] == g[1]).all()
    # splitting an epoch into two calls changes nothing
    xa, _ = oracle.sgd_epoch(ds, b, x0, batch=batch, lr=lr, batch_order=order, first_step=0, num_steps=T // 2)
    xa, _ = oracle.sgd_epoch(ds, b, xa, batch=batch, lr=lr, batch_order=order, first_step=T // 2)
    assert (xa == x1).all()


def test_gradient_quantization_is_applied_to_the_update_only():
    rng = np.random.default_rng(8)
    m, n = 40, 10
    A = rng.uniform(-1, 1, (m, n)).astype(np.float32)
    b = rng.standard_normal(m).astype(np.float32)
    x0 = rng.standard_normal(n).astype(np.float32)
    ds = oracle.quantize(A, 4, seed=2)
    x1, g = oracle.sgd_epoch(ds, b, x0, batch=m, lr=0.1, grad_bits=8, seed=5, epoch=2, want_grad=True)
    _, g_plain = oracle.sgd_epoch(ds, b, x0, batch=m, lr=0.1, want_grad=True)
    assert (g[0] == g_plain[0]).all()
    q, _ = oracle.quantize_vector(g[0], 8, 5, 2, 0, 4)
    assert (g[1] == q).all()
    assert np.allclose(x1, x0.astype(np.float64) - 0.1 * q.astype(np.float64), rtol=1e-6, atol=1e-7)
    xm, gm = oracle.sgd_epoch(ds, b, x0, batch=m, lr=0.1, model_bits=8, seed=5, epoch=2, want_grad=True)
    xq, _ = oracle.quantize_vector(x0, 8, 5, 2, 0, 3)
    _, g_from_xq = oracle.sgd_epoch(ds, b, xq, batch=m, lr=0.1, want_grad=True)
    assert (gm[0] == g_from_xq[0]).all()
    assert np.allclose(xm, x0.astype(np.float64) - 0.1 * gm[0].astype(np.float64), rtol=1e-6, atol=1e-7)


# ---------------------------------------------------------------------------------------------
# Loss
# ---------------------------------------------------------------------------------------------
def test_loss_closed_forms():
    rng = np.random.default_rng(2)
    m, n = 500, 9
    A = rng.integers(-8, 8, (m, n)).astype(np.float32)
    A[0], A[1] = -8, 7
    x = rng.integers(-3, 4, n).astype(np.float32)
    e = rng.integers(-5, 6, m).astype(np.float32)
    b = (A @ x - e).astype(np.float32)                      # exact in fp32: residual is e
    want = float((e.astype(np.float64) ** 2).sum() / (2 * m))
    assert abs(oracle.loss_dense(A, b, x) - want) < 1e-12
    assert oracle.loss_dense(A, (A @ x).astype(np.float32), x) == 0.0
    ds = oracle.quantize(A, 4, seed=1)                       # on-grid: both planes equal A
    assert abs(oracle.loss_codes(ds, b, x) - want) < 1e-12


def test_loss_from_codes_is_unbiased():
    rng = np.random.default_rng(5)
    m, n = 2000, 8
    A = rng.uniform(-1, 1, (m, n)).astype(np.float32)
    x = rng.standard_normal(n).astype(np.float32)
    b = (A @ x + 0.3 * rng.standard_normal(m)).astype(np.float32)
    dense = oracle.loss_dense(A, b, x)
    est = np.array([oracle.loss_codes(oracle.quantize(A, 3, seed=s), b, x) for s in range(60)])
    assert abs(est.mean() - dense) < 4 * est.std() / np.sqrt(len(est))
    assert est.std() > 0


# ---------------------------------------------------------------------------------------------
# Convergence (Theorem on SGD, and the frozen-code fixed point in closed form)
# ---------------------------------------------------------------------------------------------
def test_sgd_reaches_least_squares_solution():
    rng = np.random.default_rng(10)
    m, n = 20000, 8
    A = rng.uniform(-1, 1, (m, n)).astype(np.float32)
    xs = rng.standard_normal(n)
    b = (A @ xs + 0.01 * rng.standard_normal(m)).astype(np.float32)
    x_ls = np.linalg.lstsq(A.astype(np.float64), b.astype(np.float64), rcond=None)[0]
    ds = oracle.quantize(A, 4, seed=0)
    q1, q2 = np_dequant(ds, 1), np_dequant(ds, 2)
    H = (q1.T @ q2 + q2.T @ q1) / (2 * m)
    c = (q1 + q2).T @ b.astype(np.float64) / (2 * m)
    x_fix = np.linalg.solve(H, c)
    # (ii) frozen codes, full batch: plain gradient descent on H x = c, converges to x_fix exactly
    x = np.zeros(n, np.float32)
    for _ in range(150):
        x, _ = oracle.sgd_epoch(ds, b, x, batch=m, lr=1.0)
    assert np.linalg.norm(x - x_fix) < 2e-5 * np.linalg.norm(x_fix)
    assert np.linalg.norm(x_fix - x_ls) < 10 / np.sqrt(m) * np.linalg.norm(x_ls)
    # mini-batches, diminishing step alpha/epoch (the paper's schedule): ends near the same point
    x = np.zeros(n, np.float32)
    for ep in range(1, 9):
        x, _ = oracle.sgd_epoch(ds, b, x, batch=16, lr=0.2 / ep, epoch=ep)
    assert np.linalg.norm(x - x_fix) < 0.03 * np.linalg.norm(x_fix)
    # (i) fresh codes each epoch: the iterates approach x_LS itself
    x = np.zeros(n, np.float32)
    for ep in range(1, 13):
        x, _ = oracle.sgd_epoch(oracle.quantize(A, 4, seed=100 + ep), b, x, batch=16, lr=0.2 / ep, epoch=ep)
    assert np.linalg.norm(x - x_ls) < 0.03 * np.linalg.norm(x_ls)
    assert oracle.loss_dense(A, b, x) < 5 * oracle.loss_dense(A, b, x_ls.astype(np.float32)) + 1e-3


# ---------------------------------------------------------------------------------------------
# Regularisers (Eq. (proxupdate); Supplement "Least Squares Support Vector Machines").  Frozen
# codes and full batches make the iteration deterministic proximal gradient descent on
# f(x) = 1/2 x^T H x - c^T x with H, c as in the test above, whose fixed points are known.
# ---------------------------------------------------------------------------------------------
def _frozen_quadratic(seed, m=4000, n=8, labels=None):
    rng = np.random.default_rng(seed)
    A = rng.uniform(-1, 1, (m, n)).astype(np.float32)
    xs = rng.standard_normal(n)
    xs[::3] = 0.0                                       # some coordinates the l1 term can switch off
    b = (A @ xs + 0.05 * rng.standard_normal(m)).astype(np.float32)
    if labels == "pm1":
        b = np.where(A @ xs >= 0, 1.0, -1.0).astype(np.float32)
    ds = oracle.quantize(A, 4, seed=seed)
    q1, q2 = np_dequant(ds, 1), np_dequant(ds, 2)
    H = (q1.T @ q2 + q2.T @ q1) / (2 * m)
    c = (q1 + q2).T @ b.astype(np.float64) / (2 * m)
    return ds, b, H, c, m, n


def _iterate(ds, b, m, n, steps, lr, **kw):
    x = np.zeros(n, np.float32)
    for _ in range(steps):
        x, _ = oracle.sgd_epoch(ds, b, x, batch=m, lr=lr, **kw)
    return x.astype(np.float64)


def test_one_regularised_step_against_the_operator_written_out():
    ds, b, H, c, m, n = _frozen_quadratic(21)
    x0 = (np.random.default_rng(1).standard_normal(n) * 0.3).astype(np.float32)
    lr = 0.37
    y, _ = oracle.sgd_epoch(ds, b, x0, batch=m, lr=lr)
    y = y.astype(np.float64)
    # prox of lr*c/2*||.||^2, of lr*lam*||.||_1, of the indicator of the non-negative orthant; the SVM term
    want = {(oracle.REG_L2, 0.8): y / (1 + lr * 0.8),
            (oracle.REG_L1, 0.5): np.sign(y) * np.maximum(np.abs(y) - lr * 0.5, 0.0),
            (oracle.REG_NONNEG, 0.0): np.maximum(y, 0.0),
            (oracle.REG_LSSVM, 0.8): y - lr * 0.8 * x0}
    for (reg, par), w in want.items():
        got, _ = oracle.sgd_epoch(ds, b, x0, batch=m, lr=lr, reg=reg, reg_param=par)
        assert np.allclose(got, w, rtol=1e-6, atol=1e-7), reg
    # the operator minimises 1/2 ||z - y||^2 + lr R(z): no nearby point does better (l1 case)
    z, _ = oracle.sgd_epoch(ds, b, x0, batch=m, lr=lr, reg=oracle.REG_L1, reg_param=0.5)
    obj = lambda v: 0.5 * np.sum((v - y) ** 2) + lr * 0.5 * np.sum(np.abs(v))
    rng = np.random.default_rng(2)
    assert all(obj(z.astype(np.float64)) <= obj(z + 1e-3 * rng.standard_normal(n)) + 1e-12 for _ in range(200))
    # the gradient that is reported is the data term's, with or without a regulariser
    _, g0 = oracle.sgd_epoch(ds, b, x0, batch=m, lr=lr, want_grad=True)
    _, g1 = oracle.sgd_epoch(ds, b, x0, batch=m, lr=lr, want_grad=True, reg=oracle.REG_L2, reg_param=0.8)
    assert (g0[0] == g1[0]).all()


def test_l2_and_lssvm_reach_the_ridge_solution():
    for labels in (None, "pm1"):
        ds, b, H, c, m, n = _frozen_quadratic(22, labels=labels)
        cr = 0.3
        x_ridge = np.linalg.solve(H + cr * np.eye(n), c)            # gradient of f plus cr*x vanishes
        for reg in (oracle.REG_L2, oracle.REG_LSSVM):
            x = _iterate(ds, b, m, n, 200, 1.0, reg=reg, reg_param=cr)
            assert np.linalg.norm(x - x_ridge) < 2e-5 * np.linalg.norm(x_ridge), (labels, reg)
        # and the regulariser matters: the unregularised fixed point is somewhere else
        assert np.linalg.norm(np.linalg.solve(H, c) - x_ridge) > 0.05 * np.linalg.norm(x_ridge)
    # with labels +-1 this is the least-squares SVM problem: 1/(2K) sum (1 - b a^T x)^2 = 1/(2K) sum (a^T x - b)^2


def test_l1_fixed_point_satisfies_the_lasso_optimality_conditions():
    ds, b, H, c, m, n = _frozen_quadratic(23)
    lam = 0.08
    x = _iterate(ds, b, m, n, 400, 1.0, reg=oracle.REG_L1, reg_param=lam)
    grad = H @ x - c
    on = x != 0.0
    assert on.any() and (~on).any()                                  # some coordinates survive, some are switched off
    assert np.allclose(grad[on], -lam * np.sign(x[on]), atol=2e-6)
    assert (np.abs(grad[~on]) <= lam + 2e-6).all()
    # a large enough lambda switches everything off, exactly
    x = _iterate(ds, b, m, n, 3, 1.0, reg=oracle.REG_L1, reg_param=10.0)
    assert (x == 0.0).all()


def test_nonneg_fixed_point_is_the_nonnegative_least_squares_solution():
    from scipy.optimize import nnls
    ds, b, H, c, m, n = _frozen_quadratic(24)
    c = c.copy()
    # minimise 1/2 x^T H x - c^T x over x >= 0  ==  NNLS with L^T x ~ L^-1 c for H = L L^T
    Lc = np.linalg.cholesky(H)
    x_nnls, _ = nnls(Lc.T, np.linalg.solve(Lc, c))
    x = _iterate(ds, b, m, n, 400, 1.0, reg=oracle.REG_NONNEG)
    assert (x >= 0).all() and (x_nnls == 0).any()                    # the constraint is active somewhere
    assert np.linalg.norm(x - x_nnls) < 5e-5 * np.linalg.norm(x_nnls)


def test_regulariser_arguments():
    ds, b, H, c, m, n = _frozen_quadratic(25, m=64)
    with pytest.raises(Exception):
        oracle.sgd_epoch(ds, b, np.zeros(n, np.float32), batch=m, lr=0.1, reg=7)
    with pytest.raises(Exception):
        oracle.sgd_epoch(ds, b, np.zeros(n, np.float32), batch=m, lr=0.1, reg=oracle.REG_L1, reg_param=-1.0)


@pytest.mark.parametrize("bits", [1, 5, 6, 7])
def test_the_other_bit_widths_live_in_the_next_wider_container(bits):
    """1-bit codes in 2-bit fields, 5- to 7-bit codes in bytes: same quantizer (Supplement "Randomized Quantization")
    with s = 2^bits - 1 intervals; pinned by exact samples, the code range, and the unbiased mean."""
    s = (1 << bits) - 1
    cb = {1: 2, 5: 8, 6: 8, 7: 8}[bits]
    assert oracle.container_bits(bits) == cb and oracle.row_bytes(33, bits) == (33 * cb + 7) // 8 + (-((33 * cb + 7) // 8)) % 16
    rng = np.random.default_rng(bits)
    A = rng.integers(0, s + 1, size=(20, 9)).astype(np.float32)
    A[0], A[1] = 0.0, float(s)
    ds = oracle.quantize(A, bits, seed=1)
    for plane in (ds.plane1, ds.plane2):                             # samples on the grid: the codes are the samples
        assert np.array_equal(oracle.unpack_plane(plane, 9, bits), A.astype(np.int64))
    B = rng.uniform(-1.0, 1.0, (4, 6)).astype(np.float32)
    B[0], B[1] = -1.0, 1.0
    acc, N = np.zeros((4, 6)), 3000
    for seed in range(N):
        d = oracle.quantize(B, bits, seed=seed)
        c = oracle.unpack_plane(d.plane1, 6, bits)
        assert c.max() <= s and c.min() >= 0
        acc += d.feat_lo + d.feat_step * c
    step = 2.0 / s
    assert np.abs(acc / N - B).max() < 5 * (step / 2) / np.sqrt(N) + 1e-6


def test_symmetric_grid_of_the_supplements_column_scaling():
    """Grid [-M_j, M_j] with M_j = max |value| (Supplement "Column Scaling"): lo = -M, step = 2M/s, samples on the
    grid come back exactly, the mean over seeds is the sample, and the codes differ from the range grid's."""
    rng = np.random.default_rng(11)
    bits, s = 3, 7
    A = rng.uniform(-0.4, 1.0, (12, 5)).astype(np.float32)
    M = np.abs(A).max(axis=0)
    ds = oracle.quantize_pair(A, bits, 3, 0, symmetric=True)
    assert np.array_equal(ds.feat_lo, -M) and np.allclose(ds.feat_step, 2 * M / s, rtol=1e-7)
    assert not np.array_equal(ds.plane1, oracle.quantize(A, bits, 3).plane1)
    # exact samples: integers -7, -5, ..., 7 are the eight levels of M = 7
    G = (2 * rng.integers(0, s + 1, size=(16, 4)) - s).astype(np.float32)
    G[0] = -7.0
    dg = oracle.quantize_pair(G, bits, 5, 1, symmetric=True)
    for plane in (dg.plane1, dg.plane2):
        assert np.array_equal(-7.0 + 2.0 * oracle.unpack_plane(plane, 4, bits), G)
    acc, N = np.zeros(A.shape), 4000
    for seed in range(N):
        d = oracle.quantize_pair(A, bits, seed, 0, symmetric=True)
        acc += d.feat_lo + d.feat_step * oracle.unpack_plane(d.plane2, 5, bits)
    assert np.abs(acc / N - A).max() < 5 * (2 * M.max() / s / 2) / np.sqrt(N) + 1e-6
    with pytest.raises(oracle.OracleError):
        oracle.quantize_pair(A, bits, 0, 0, mode=oracle.TABLE, levels=np.zeros((5, 8), np.float32), symmetric=True)


def test_vector_quantizer_scaled_by_the_largest_entry():
    """M(v) = max |v_i| instead of ||v||_2 (the Supplement leaves M general): the largest entry is reproduced exactly,
    nothing exceeds it, the mean over draws is v, and the variance is below the l2-scaled quantizer's."""
    rng = np.random.default_rng(8)
    v = rng.standard_normal(40).astype(np.float32)
    bits, N = 4, 4000
    big = int(np.argmax(np.abs(v)))
    acc = np.zeros(40)
    var_inf = var_l2 = 0.0
    for step in range(N):
        q, codes = oracle.quantize_vector(v, bits, 5, 1, step, 4, norm=oracle.NORM_LINF)
        assert q[big] == v[big] and abs(int(codes[big])) == 7
        assert np.abs(q).max() <= np.abs(v).max()
        acc += q
        var_inf += ((q - v) ** 2).sum()
        var_l2 += ((oracle.quantize_vector(v, bits, 5, 1, step, 4)[0] - v) ** 2).sum()
    unit = np.abs(v).max() / 7
    assert np.abs(acc / N - v).max() < 5 * (unit / 2) / np.sqrt(N) + 1e-6
    assert var_inf < 0.5 * var_l2
    # the default is the l2 scaling, unchanged
    a, _ = oracle.quantize_vector(v, bits, 5, 1, 0, 4)
    b, _ = oracle.quantize_vector(v, bits, 5, 1, 0, 4, norm=oracle.NORM_L2)
    assert np.array_equal(a, b) and np.abs(a).max() <= np.linalg.norm(v) * (1 + 1e-6)
    z, zc = oracle.quantize_vector(np.zeros(5, np.float32), bits, 0, 0, 0, 3, norm=oracle.NORM_LINF)
    assert not z.any() and not zc.any()
