"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Tolerances (from the benchmark spec): packed codes and optimal levels bit-exact; per-step
gradients <= 1e-5 relative L2; model after one epoch with the same minibatch order <= 1e-4 relative
L2; loss within 1e-3 relative (the kernels are far inside that: the tests use 1e-6).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1611_05402_b200 import binding, synth

pytestmark = pytest.mark.gpu

GRAD_TOL, MODEL_TOL, LOSS_TOL = 1e-5, 1e-4, 1e-6


@pytest.fixture(scope="module")
def ctx():
    from paper_1611_05402_b200.build import build
    build()
    c = binding.Context("cuda:0")
    yield c
    c.close()


def rel(a, b):
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def to_dev(a, ctx):
    return torch.from_numpy(np.ascontiguousarray(a)).to(ctx.device)


def dev_dataset(ods, ctx):
    """Oracle dataset -> device dataset (so that SGD parity does not depend on quantize parity)."""
    return binding.Dataset(to_dev(ods.plane1, ctx), to_dev(ods.plane2, ctx), ods.m, ods.n, ods.bits, ods.mode,
                           to_dev(ods.feat_lo, ctx), to_dev(ods.feat_step, ctx) if ods.mode == oracle.UNIFORM else None,
                           to_dev(ods.levels, ctx) if ods.levels is not None else None)


def workload(key, m, n, seed=0):
    w, A, b, xs = synth.make(key, m=m, n=n, seed=seed)
    return w, A.numpy(), b.numpy(), xs.numpy()


# ---------------------------------------------------------------------------------------------
# quantize: bit-exact planes and scales
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("key,m,n,bits", [
    ("c1", 300, 64, 4), ("c1", 257, 61, 4), ("c2", 500, 1000, 8), ("c2", 129, 1003, 8), ("c3", 200, 2048, 2),
    ("c3", 77, 2050, 2), ("c3", 5, 1, 2), ("c4u", 333, 512, 3), ("c4u", 100, 37, 3), ("c5", 40, 4100, 4),
    ("c1", 1, 5, 8), ("c2", 3000, 7, 2),
])
def test_quantize_bit_exact(ctx, key, m, n, bits):
    _, A, _, _ = workload(key, m, n, seed=bits)
    if m > 2:
        A[:, n // 2] = 0.25                                        # a constant feature
    ods = oracle.quantize(A, bits, seed=1234 + m)
    gds = ctx.zipml_quantize(to_dev(A, ctx), bits, seed=1234 + m)
    ctx.zipml_sync()
    assert (gds.feat_lo.cpu().numpy() == ods.feat_lo).all()
    assert (gds.feat_step.cpu().numpy() == ods.feat_step).all()
    assert gds.row_bytes == ods.row_bytes
    assert (gds.plane1.cpu().numpy() == ods.plane1).all()
    assert (gds.plane2.cpu().numpy() == ods.plane2).all()


def test_quantize_strided_and_unaligned_input(ctx):
    _, A, _, _ = workload("c2", 200, 101, seed=3)
    big = torch.zeros((200, 131), dtype=torch.float32, device=ctx.device)
    big[:, 3:104] = to_dev(A, ctx)
    view = big[:, 3:104]                                           # lda = 131, base not 16-byte aligned
    ods = oracle.quantize(A, 4, seed=9)
    gds = ctx.zipml_quantize(view, 4, seed=9, row_bytes=ods.row_bytes + 32)
    ctx.zipml_sync()
    assert (gds.plane1.cpu().numpy()[:, : ods.row_bytes] == ods.plane1).all()
    assert (gds.plane2.cpu().numpy()[:, : ods.row_bytes] == ods.plane2).all()
    assert not gds.plane1.cpu().numpy()[:, ods.row_bytes:].any()
    assert (gds.feat_lo.cpu().numpy() == ods.feat_lo).all()


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable(ctx):
    """The device-side waits are bounded: one that cannot succeed (a flag that nothing sets) gives up, the next
    zipml_sync returns ZIPML_ERR_TIMEOUT once, and the same context then works as before."""
    ctx.zipml_sync()
    ctx.zipml_wait_probe(50000)
    with pytest.raises(binding.ZipmlError) as e:
        ctx.zipml_sync()
    assert e.value.code == binding.ERR_TIMEOUT
    ctx.zipml_sync()                                               # reported once, then cleared
    _, A, b, _ = workload("c1", 256, 64, seed=1)
    ods = oracle.quantize(A, 4, seed=1)
    gds = ctx.zipml_quantize(to_dev(A, ctx), 4, seed=1)
    x = torch.zeros(64, device=ctx.device)
    ctx.zipml_sgd_epoch(gds, to_dev(b, ctx), x, 16, 0.01)
    ctx.zipml_sync()
    x_ref, _ = oracle.sgd_epoch(ods, b, np.zeros(64, np.float32), 16, 0.01)
    assert (gds.plane1.cpu().numpy()[:, : ods.row_bytes] == ods.plane1).all() and rel(x.cpu().numpy(), x_ref) <= MODEL_TOL
    with pytest.raises(binding.ZipmlError):
        ctx.zipml_wait_probe(0)


def test_quantize_reports_bad_input(ctx):
    A = torch.rand((64, 16), device=ctx.device)
    A[5, 3] = float("nan")
    ctx.zipml_quantize(A, 4, seed=0)
    with pytest.raises(binding.ZipmlError) as e:
        ctx.zipml_sync()
    assert e.value.code == binding.ERR_NONFINITE
    ctx.zipml_sync()                                               # the error is reported once, then cleared
    A[5, 3] = float("inf")
    ctx.zipml_quantize(A, 4, seed=0)
    with pytest.raises(binding.ZipmlError):
        ctx.zipml_sync()
    wide = torch.rand((70, 2052), device=ctx.device)               # wide rows take another range-scan kernel
    wide[69, 2049] = float("nan")                                  # in the ragged last group of four columns
    ctx.zipml_quantize(wide[:, :2050], 2, seed=0)
    with pytest.raises(binding.ZipmlError) as e:
        ctx.zipml_sync()
    assert e.value.code == binding.ERR_NONFINITE
    good = torch.rand((64, 16), device=ctx.device)
    for bits in (0, 9, 16):
        with pytest.raises(binding.ZipmlError) as e:
            ctx.zipml_quantize(good, bits, seed=0)
        assert e.value.code == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.ZipmlError) as e:
        ctx.zipml_quantize(good, 4, seed=0, row_bytes=8)
    assert e.value.code == binding.ERR_INVALID_ARG
    with pytest.raises(binding.ZipmlError) as e:
        ctx.zipml_quantize(good, 8, seed=0, level_mode=binding.LEVELS_TABLE,
                           levels=torch.zeros((16, 256), device=ctx.device))
    assert e.value.code == binding.ERR_UNSUPPORTED


# ---------------------------------------------------------------------------------------------
# optimal levels: bit-exact levels and objective; table quantization bit-exact
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("m,n,bits,bins", [(5000, 40, 3, 1024), (3000, 33, 2, 256), (2000, 16, 4, 1024), (700, 5, 3, 7),
                                           (64, 3, 4, 1000)])
def test_optimal_levels_bit_exact(ctx, m, n, bits, bins):
    _, A, _, _ = workload("c4", m, n, seed=bins)
    A[:, n - 1] = -0.5                                             # a constant feature
    lev, obj = oracle.optimal_levels(A, bits, bins)
    glev, gobj = ctx.zipml_optimal_levels(to_dev(A, ctx), bits, bins, want_objective=True)
    ctx.zipml_sync()
    assert (gobj.cpu().numpy().astype(np.uint64) == obj).all()
    assert (glev.cpu().numpy() == lev).all()
    ods = oracle.quantize(A, bits, seed=5, mode=oracle.TABLE, levels=lev)
    gds = ctx.zipml_quantize(to_dev(A, ctx), bits, seed=5, level_mode=binding.LEVELS_TABLE, levels=glev)
    ctx.zipml_sync()
    assert (gds.plane1.cpu().numpy() == ods.plane1).all() and (gds.plane2.cpu().numpy() == ods.plane2).all()
    assert (gds.feat_lo.cpu().numpy() == ods.feat_lo).all()


@pytest.mark.parametrize("distinct,bits,bins", [(3, 3, 1024), (6, 2, 1024), (40, 4, 512), (2, 3, 100)])
def test_optimal_levels_bit_exact_with_many_empty_bins(ctx, distinct, bits, bins):
    """Few distinct values: most bins are empty and many level sets cost the same, so the result hangs on the
    tie rule (smallest index) -- which the kernel's narrowed search must keep."""
    rng = np.random.default_rng(distinct)
    vals = np.sort(rng.uniform(-1.0, 1.0, distinct)).astype(np.float32)
    A = vals[rng.integers(0, distinct, size=(4000, 24))]
    A[:, 5] = vals[0]                                              # a constant feature
    A[:100, 7] = 1.5                                               # a far outlier: long empty stretch
    lev, obj = oracle.optimal_levels(A, bits, bins)
    glev, gobj = ctx.zipml_optimal_levels(to_dev(A, ctx), bits, bins, want_objective=True)
    ctx.zipml_sync()
    assert (gobj.cpu().numpy().astype(np.uint64) == obj).all()
    assert (glev.cpu().numpy() == lev).all()


# ---------------------------------------------------------------------------------------------
# SGD: per-step gradient from identical x_t, model after an epoch, both engines, several grids
# ---------------------------------------------------------------------------------------------
SGD_CASES = [
    # key, m, n, bits, batch, lr
    ("c1", 1000, 64, 4, 16, 0.01),
    ("c2", 2100, 1000, 8, 256, 1e-3),         # ragged tail: 2100 = 8*256 + 52
    ("c3", 2500, 2048, 2, 1024, 5e-4),
    ("c4u", 1500, 512, 3, 512, 1e-3),
    ("c5", 300, 4099, 4, 128, 1e-4),          # n not a multiple of anything
    ("c2", 100, 33, 8, 7, 1e-2),
    ("c1", 50, 5, 2, 64, 0.05),               # batch larger than m
]
GRIDS = [(0, 0), (1, 1), (1, 5), (2, 3), (3, 1)]


@pytest.mark.parametrize("case", SGD_CASES, ids=lambda c: f"{c[0]}-{c[1]}x{c[2]}-b{c[3]}-B{c[4]}")
@pytest.mark.parametrize("engine", [binding.ENGINE_STEPWISE, binding.ENGINE_PERSISTENT, binding.ENGINE_RING, binding.ENGINE_LEAN, binding.ENGINE_CLUSTER,
                                    binding.ENGINE_STREAM])
def test_sgd_epoch_parity(ctx, case, engine):
    key, m, n, bits, batch, lr = case
    _, A, b, _ = workload(key, m, n, seed=1)
    ods = oracle.quantize(A, bits, seed=7)
    gds = dev_dataset(ods, ctx)
    db = to_dev(b, ctx)
    T = (m + batch - 1) // batch
    order = np.random.default_rng(0).permutation(T).astype(np.int32)
    x0 = (np.random.default_rng(1).standard_normal(n) * 0.1).astype(np.float32)
    x_ref, _ = oracle.sgd_epoch(ods, b, x0, batch, lr, batch_order=order)
    # model just before the last step, for the per-step gradient check
    x_before, _ = oracle.sgd_epoch(ods, b, x0, batch, lr, batch_order=order, num_steps=T - 1)
    _, g_ref = oracle.sgd_epoch(ods, b, x_before, batch, lr, batch_order=order, first_step=T - 1, num_steps=1,
                                want_grad=True)
    for fa, fb in GRIDS:
        x = to_dev(x0, ctx)
        ctx.zipml_sgd_epoch(gds, db, x, batch, lr, batch_order=order, engine=engine, grid_feature_parts=fa,
                            grid_row_parts=fb)
        ctx.zipml_sync()
        assert rel(x.cpu().numpy(), x_ref) <= MODEL_TOL, (fa, fb)
        xb = to_dev(x_before, ctx)
        g = torch.zeros((2, n), dtype=torch.float32, device=ctx.device)
        ctx.zipml_sgd_epoch(gds, db, xb, batch, lr, batch_order=order, first_step=T - 1, num_steps=1, engine=engine,
                            grid_feature_parts=fa, grid_row_parts=fb, grad_out=g)
        ctx.zipml_sync()
        assert rel(g[0].cpu().numpy(), g_ref[0]) <= GRAD_TOL, (fa, fb)
        assert (g[0] == g[1]).all()
        assert rel(xb.cpu().numpy(), x_ref) <= MODEL_TOL


@pytest.mark.parametrize("contraction", [1, 2], ids=["fp32", "int8"])
@pytest.mark.parametrize("case", SGD_CASES[:5], ids=lambda c: f"{c[0]}-{c[1]}x{c[2]}-b{c[3]}-B{c[4]}")
def test_cluster_engine_both_contractions(ctx, case, contraction):
    """The cluster engine's fp32 and int8 tensor-core contractions, forced, against the oracle."""
    key, m, n, bits, batch, lr = case
    _, A, b, _ = workload(key, m, n, seed=3)
    ods = oracle.quantize(A, bits, seed=5)
    gds, db = dev_dataset(ods, ctx), to_dev(b, ctx)
    T = (m + batch - 1) // batch
    x0 = (np.random.default_rng(2).standard_normal(n) * 0.1).astype(np.float32)
    x_ref, _ = oracle.sgd_epoch(ods, b, x0, batch, lr)
    x_before, _ = oracle.sgd_epoch(ods, b, x0, batch, lr, num_steps=T - 1)
    _, g_ref = oracle.sgd_epoch(ods, b, x_before, batch, lr, first_step=T - 1, num_steps=1, want_grad=True)
    for fb in (0, 3, 16):
        x = to_dev(x0, ctx)
        ctx.zipml_sgd_epoch(gds, db, x, batch, lr, engine=binding.ENGINE_CLUSTER, grid_row_parts=fb,
                            cluster_contraction=contraction)
        ctx.zipml_sync()
        assert rel(x.cpu().numpy(), x_ref) <= MODEL_TOL, fb
        xb = to_dev(x_before, ctx)
        g = torch.zeros((2, n), dtype=torch.float32, device=ctx.device)
        ctx.zipml_sgd_epoch(gds, db, xb, batch, lr, first_step=T - 1, num_steps=1, engine=binding.ENGINE_CLUSTER,
                            grid_row_parts=fb, grad_out=g, cluster_contraction=contraction)
        ctx.zipml_sync()
        assert rel(g[0].cpu().numpy(), g_ref[0]) <= GRAD_TOL, fb


@pytest.mark.parametrize("case", [
    # key, m, n, bits, batch, lr: rows wide enough for many column blocks and several pass-A parts
    ("c5", 700, 20000, 4, 300, 1e-4),
    ("c2", 1300, 9001, 8, 520, 1e-3),
    ("c3", 1100, 40000, 2, 500, 5e-4),
    ("c4u", 900, 12345, 3, 333, 1e-3),
], ids=lambda c: f"{c[0]}-{c[1]}x{c[2]}-b{c[3]}-B{c[4]}")
def test_stream_engine_wide_rows(ctx, case):
    """The stream engine on shapes that give it many CTAs, from a zero and from a non-zero model, twice."""
    key, m, n, bits, batch, lr = case
    _, A, b, _ = workload(key, m, n, seed=8)
    ods = oracle.quantize(A, bits, seed=9)
    gds, db = dev_dataset(ods, ctx), to_dev(b, ctx)
    T = (m + batch - 1) // batch
    for x0 in (np.zeros(n, np.float32), (np.random.default_rng(4).standard_normal(n) * 0.05).astype(np.float32)):
        x_ref, _ = oracle.sgd_epoch(ods, b, x0, batch, lr)
        x_before, _ = oracle.sgd_epoch(ods, b, x0, batch, lr, num_steps=T - 1)
        _, g_ref = oracle.sgd_epoch(ods, b, x_before, batch, lr, first_step=T - 1, num_steps=1, want_grad=True)
        runs = []
        for fb in (0, 0, 61):
            x = to_dev(x0, ctx)
            ctx.zipml_sgd_epoch(gds, db, x, batch, lr, engine=binding.ENGINE_STREAM, grid_row_parts=fb)
            ctx.zipml_sync()
            assert ctx.zipml_last_engine() == binding.ENGINE_STREAM
            runs.append(x.cpu().numpy())
            assert rel(runs[-1], x_ref) <= MODEL_TOL, fb
        # integer sums in any order: the same bits run to run and for any grid
        assert (runs[0] == runs[1]).all() and (runs[0] == runs[2]).all()
        xb = to_dev(x_before, ctx)
        g = torch.zeros((2, n), dtype=torch.float32, device=ctx.device)
        ctx.zipml_sgd_epoch(gds, db, xb, batch, lr, first_step=T - 1, num_steps=1, engine=binding.ENGINE_STREAM, grad_out=g)
        ctx.zipml_sync()
        assert rel(g[0].cpu().numpy(), g_ref[0]) <= GRAD_TOL
    # what it does not cover is declined, not approximated
    with pytest.raises(binding.ZipmlError) as e:
        ctx.zipml_sgd_epoch(gds, db, to_dev(x0, ctx), batch, lr, engine=binding.ENGINE_STREAM, model_bits=8)
    assert e.value.code == binding.ERR_WORKSPACE


@pytest.mark.parametrize("case", [
    # key, m, n, bits, batch, lr, chunk rows (0 = automatic)
    ("c5", 700, 20000, 4, 300, 1e-4, 0),          # 79 column blocks, the last one partly past the row; ragged batches
    ("c5", 1500, 30001, 4, 640, 1e-4, 64),        # several chunks per step, n odd
    ("c2", 1300, 9001, 8, 520, 1e-3, 0),
    ("c3", 1100, 40000, 2, 500, 5e-4, 96),
    ("c4u", 900, 12345, 3, 333, 1e-3, 256),
    ("c2", 400, 300, 8, 100, 1e-3, 32),           # three CTAs only
], ids=lambda c: f"{c[0]}-{c[1]}x{c[2]}-b{c[3]}-B{c[4]}-R{c[6]}")
def test_column_engine(ctx, case):
    """The column engine (a CTA per 128-byte column block, codes read once per step): model after an epoch in a
    permuted batch order from a zero and a non-zero model, bit-identical repeats, last-step gradient, split calls."""
    key, m, n, bits, batch, lr, chunk = case
    _, A, b, _ = workload(key, m, n, seed=8)
    ods = oracle.quantize(A, bits, seed=9)
    gds, db = dev_dataset(ods, ctx), to_dev(b, ctx)
    T = (m + batch - 1) // batch
    order = np.random.default_rng(5).permutation(T).astype(np.int32)
    kw = dict(engine=binding.ENGINE_COLUMN, column_chunk_rows=chunk, batch_order=order)
    # the same planes cut into 128-byte column blocks: the layout is what a plain reshape of the oracle's planes gives
    bds = ctx.zipml_convert_layout(gds, binding.LAYOUT_COLUMN_BLOCKS)
    nblk = (ods.row_bytes + 127) // 128
    for got, plane in ((bds.plane1, ods.plane1), (bds.plane2, ods.plane2)):
        padded = np.zeros((m, nblk * 128), np.uint8)
        padded[:, : ods.row_bytes] = plane
        assert (got.cpu().numpy().reshape(nblk, m, 128) == padded.reshape(m, nblk, 128).transpose(1, 0, 2)).all()
    back = ctx.zipml_convert_layout(bds, binding.LAYOUT_ROWS)
    ctx.zipml_sync()
    assert (back.plane1.cpu().numpy() == ods.plane1).all() and (back.plane2.cpu().numpy() == ods.plane2).all()
    for x0 in (np.zeros(n, np.float32), (np.random.default_rng(4).standard_normal(n) * 0.05).astype(np.float32)):
        x_ref, _ = oracle.sgd_epoch(ods, b, x0, batch, lr, batch_order=order)
        x_before, _ = oracle.sgd_epoch(ods, b, x0, batch, lr, batch_order=order, num_steps=T - 1)
        _, g_ref = oracle.sgd_epoch(ods, b, x_before, batch, lr, batch_order=order, first_step=T - 1, num_steps=1, want_grad=True)
        runs = []
        for _ in range(2):
            x = to_dev(x0, ctx)
            ctx.zipml_sgd_epoch(gds, db, x, batch, lr, **kw)
            ctx.zipml_sync()
            assert ctx.zipml_last_engine() == binding.ENGINE_COLUMN
            runs.append(x.cpu().numpy())
            assert rel(runs[-1], x_ref) <= MODEL_TOL
        assert (runs[0] == runs[1]).all()                 # integer sums and fixed orders: the same bits run to run
        x = to_dev(x0, ctx)
        ctx.zipml_sgd_epoch(bds, db, x, batch, lr, **{**kw, "engine": binding.ENGINE_AUTO})      # from the column blocks
        ctx.zipml_sync()
        assert ctx.zipml_last_engine() == binding.ENGINE_COLUMN and (x.cpu().numpy() == runs[0]).all()
        xb = to_dev(x_before, ctx)
        g = torch.zeros((2, n), dtype=torch.float32, device=ctx.device)
        ctx.zipml_sgd_epoch(gds, db, xb, batch, lr, first_step=T - 1, num_steps=1, grad_out=g, **kw)
        ctx.zipml_sync()
        assert rel(g[0].cpu().numpy(), g_ref[0]) <= GRAD_TOL and (g[0] == g[1]).all()
        assert rel(xb.cpu().numpy(), x_ref) <= MODEL_TOL
        if T >= 3:                                        # an epoch in two calls
            x = to_dev(x0, ctx)
            ctx.zipml_sgd_epoch(gds, db, x, batch, lr, first_step=0, num_steps=2, **kw)
            ctx.zipml_sgd_epoch(gds, db, x, batch, lr, first_step=2, **kw)
            ctx.zipml_sync()
            assert rel(x.cpu().numpy(), x_ref) <= MODEL_TOL
    # what it does not cover is declined, not approximated
    for bad in (dict(model_bits=8), dict(grad_bits=8), dict(model_out=torch.zeros(n, device=ctx.device))):
        with pytest.raises(binding.ZipmlError) as e:
            ctx.zipml_sgd_epoch(gds, db, to_dev(x0, ctx), batch, lr, engine=binding.ENGINE_COLUMN, **bad)
        assert e.value.code == binding.ERR_WORKSPACE
    for engine in (binding.ENGINE_STREAM, binding.ENGINE_RING, binding.ENGINE_CLUSTER):     # the other engines read rows only
        with pytest.raises(binding.ZipmlError) as e:
            ctx.zipml_sgd_epoch(bds, db, to_dev(x0, ctx), batch, lr, engine=engine)
        assert e.value.code == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.ZipmlError) as e:
        ctx.zipml_loss(binding.LOSS_CODES, db, to_dev(x0, ctx), data=bds)
    assert e.value.code == binding.ERR_UNSUPPORTED


def test_column_engine_limits(ctx):
    """Rows narrower than one column block, rows wider than one block per SM and batches above 8,192 are declined."""
    _, A, b, _ = workload("c1", 200, 64, seed=1)
    gds, db = dev_dataset(oracle.quantize(A, 4, seed=1), ctx), to_dev(b, ctx)
    with pytest.raises(binding.ZipmlError) as e:
        ctx.zipml_sgd_epoch(gds, db, torch.zeros(64, device=ctx.device), 16, 0.01, engine=binding.ENGINE_COLUMN)
    assert e.value.code == binding.ERR_WORKSPACE
    m, n = 8300, 10240
    _, A, b, _ = workload("c5", m, n, seed=11)
    ods = oracle.quantize(A, 4, seed=12)
    gds, db = dev_dataset(ods, ctx), to_dev(b, ctx)
    x0 = np.zeros(n, np.float32)
    x_ref, _ = oracle.sgd_epoch(ods, b, x0, 8192, 1e-4)
    x = to_dev(x0, ctx)
    ctx.zipml_sgd_epoch(gds, db, x, 8192, 1e-4, engine=binding.ENGINE_COLUMN)
    ctx.zipml_sync()
    assert rel(x.cpu().numpy(), x_ref) <= MODEL_TOL
    with pytest.raises(binding.ZipmlError) as e:
        ctx.zipml_sgd_epoch(gds, db, to_dev(x0, ctx), 8193, 1e-4, engine=binding.ENGINE_COLUMN)
    assert e.value.code == binding.ERR_WORKSPACE


def test_stream_engine_batch_limits(ctx):
    """The largest batch the stream engine takes (its residual digits live in shared memory), and one row more."""
    m, n = 8300, 10240
    _, A, b, _ = workload("c5", m, n, seed=11)
    ods = oracle.quantize(A, 4, seed=12)
    gds, db = dev_dataset(ods, ctx), to_dev(b, ctx)
    x0 = np.zeros(n, np.float32)
    x_ref, _ = oracle.sgd_epoch(ods, b, x0, 8192, 1e-4)
    x = to_dev(x0, ctx)
    ctx.zipml_sgd_epoch(gds, db, x, 8192, 1e-4, engine=binding.ENGINE_STREAM)
    ctx.zipml_sync()
    assert rel(x.cpu().numpy(), x_ref) <= MODEL_TOL
    with pytest.raises(binding.ZipmlError) as e:
        ctx.zipml_sgd_epoch(gds, db, to_dev(x0, ctx), 8193, 1e-4, engine=binding.ENGINE_STREAM)
    assert e.value.code == binding.ERR_WORKSPACE
    x_ref, _ = oracle.sgd_epoch(ods, b, x0, 8193, 1e-4)
    x = to_dev(x0, ctx)
    ctx.zipml_sgd_epoch(gds, db, x, 8193, 1e-4)                                 # AUTO: another engine takes it
    ctx.zipml_sync()
    assert ctx.zipml_last_engine() != binding.ENGINE_STREAM and rel(x.cpu().numpy(), x_ref) <= MODEL_TOL


def test_sgd_engines_and_grids_agree_bitwise_where_the_reduction_order_is_the_same(ctx):
    _, A, b, _ = workload("c2", 1500, 300, seed=2)
    ods = oracle.quantize(A, 8, seed=1)
    gds, db = dev_dataset(ods, ctx), to_dev(b, ctx)
    outs = []
    for engine in (binding.ENGINE_STEPWISE, binding.ENGINE_PERSISTENT):
        x = torch.zeros(300, device=ctx.device)
        ctx.zipml_sgd_epoch(gds, db, x, 128, 1e-3, engine=engine, grid_feature_parts=2, grid_row_parts=4)
        ctx.zipml_sync()
        outs.append(x.cpu().numpy())
    assert (outs[0] == outs[1]).all()
    # and a second run is bit-identical to the first: no atomics, fixed reduction order
    x = torch.zeros(300, device=ctx.device)
    ctx.zipml_sgd_epoch(gds, db, x, 128, 1e-3, engine=binding.ENGINE_PERSISTENT, grid_feature_parts=2, grid_row_parts=4)
    ctx.zipml_sync()
    assert (x.cpu().numpy() == outs[1]).all()


def test_sgd_table_levels_parity(ctx):
    _, A, b, _ = workload("c4", 3000, 100, seed=4)
    lev, _ = oracle.optimal_levels(A, 3, 256)
    ods = oracle.quantize(A, 3, seed=3, mode=oracle.TABLE, levels=lev)
    gds, db = dev_dataset(ods, ctx), to_dev(b, ctx)
    x0 = np.zeros(100, np.float32)
    x_ref, g_ref = oracle.sgd_epoch(ods, b, x0, 512, 1e-2, want_grad=True)
    for engine in (binding.ENGINE_STEPWISE, binding.ENGINE_PERSISTENT, binding.ENGINE_RING, binding.ENGINE_LEAN, binding.ENGINE_CLUSTER):
        for fa, fb in GRIDS:
            x = to_dev(x0, ctx)
            g = torch.zeros((2, 100), dtype=torch.float32, device=ctx.device)
            ctx.zipml_sgd_epoch(gds, db, x, 512, 1e-2, engine=engine, grid_feature_parts=fa, grid_row_parts=fb,
                                grad_out=g)
            ctx.zipml_sync()
            assert rel(x.cpu().numpy(), x_ref) <= MODEL_TOL
    # per-step gradient from the same x
    _, g1 = oracle.sgd_epoch(ods, b, x_ref, 512, 1e-2, first_step=2, num_steps=1, want_grad=True)
    x = to_dev(x_ref, ctx)
    g = torch.zeros((2, 100), dtype=torch.float32, device=ctx.device)
    ctx.zipml_sgd_epoch(gds, db, x, 512, 1e-2, first_step=2, num_steps=1, grad_out=g)
    ctx.zipml_sync()
    assert rel(g[0].cpu().numpy(), g1[0]) <= GRAD_TOL


def q3_margins(x, bits, seed, epoch, step):
    """|u 2^-24 - p| of every coordinate's Q3 rounding decision (Supplement Eq. (quant2) with M = ||x||_2), from
    the oracle's own random integers; the arithmetic mirrors the quantizer's fp32 steps only to *classify*
    coordinates (which ones a sub-ulp difference in M could flip), never to produce an expected value."""
    sm = np.float32((1 << (bits - 1)) - 1)
    M = np.float32(np.sqrt(np.sum(x.astype(np.float64) ** 2)))
    t = (np.abs(x) / M).astype(np.float32) * sm
    fl = np.minimum(np.floor(t), sm - 1).astype(np.float32)
    p = (t - fl).astype(np.float32)
    u = np.array([oracle.u24_vector(seed, epoch, step, j, 3) for j in range(x.shape[0])], np.float64) * 2.0 ** -24
    return np.abs(u - p.astype(np.float64)), float(M / sm)


E2E_ENGINES = [
    # engine, cluster_contraction, id
    (binding.ENGINE_STEPWISE, 0), (binding.ENGINE_PERSISTENT, 0), (binding.ENGINE_RING, 0), (binding.ENGINE_LEAN, 0),
    (binding.ENGINE_CLUSTER, 1), (binding.ENGINE_CLUSTER, 2), (binding.ENGINE_AUTO, 0),
]


@pytest.mark.parametrize("model_bits,grad_bits", [(8, 0), (0, 8), (8, 8), (4, 4)])
@pytest.mark.parametrize("shape", [(3000, 512), (3000, 2048)], ids=["n512", "c3-n2048"])
def test_sgd_end_to_end_quantization(ctx, shape, model_bits, grad_bits):
    """Q3 / Q4 (Supplement "Quantizing the Model", "Quantizing the Gradients", "End-to-end Quantization") on 2-bit
    data with B = 1024; the second shape is config 3's own step (n = 2,048: 64 rows x 512 B per CTA, where AUTO
    runs the cluster engine's int8 contraction) and both contractions of the cluster engine are forced."""
    m, n = shape
    _, A, b, _ = workload("c3", m, n, seed=6)
    ods = oracle.quantize(A, 2, seed=2)
    gds, db = dev_dataset(ods, ctx), to_dev(b, ctx)
    x0 = (np.random.default_rng(3).standard_normal(n) * 0.05).astype(np.float32)
    seed, epoch, step = 11, 2, 1
    # what the model quantizer must produce from x0, and how close each of its decisions is to its threshold
    if model_bits:
        xq_ref, _ = oracle.quantize_vector(x0, model_bits, seed, epoch, step, 3)
        margin, unit_x = q3_margins(x0, model_bits, seed, epoch, step)
    else:
        xq_ref = x0
    for engine, contraction in E2E_ENGINES:
        x = to_dev(x0, ctx)
        g = torch.zeros((2, n), dtype=torch.float32, device=ctx.device)
        xq = torch.zeros(n, dtype=torch.float32, device=ctx.device)
        ctx.zipml_sgd_epoch(gds, db, x, 1024, 5e-4, model_bits=model_bits, grad_bits=grad_bits, seed=seed, epoch=epoch,
                            first_step=step, num_steps=1, engine=engine, grad_out=g, model_out=xq,
                            cluster_contraction=contraction)
        ctx.zipml_sync()
        if engine == binding.ENGINE_AUTO and n == 2048:
            assert ctx.zipml_last_engine() == binding.ENGINE_CLUSTER
        gg, xq = g.cpu().numpy(), xq.cpu().numpy()
        # Q3: the quantized model agrees exactly, except where a rounding sits within 1e-4 of its threshold
        # (a last-bit difference in ||x||_2 may flip those: by one quantization unit, and only a few)
        differs = xq != xq_ref
        if model_bits:
            assert not (differs & (margin >= 1e-4)).any(), (engine, contraction)
            assert differs.sum() <= 3 and (np.abs(xq - xq_ref)[differs] <= 1.001 * unit_x).all()
        else:
            assert not differs.any()
        # the gradient before Q4, held to the plain bar against the oracle run from the very model the kernel used
        _, g_ref = oracle.sgd_epoch(ods, b, xq, 1024, 5e-4, model_bits=0, grad_bits=grad_bits, seed=seed, epoch=epoch,
                                    first_step=step, num_steps=1, want_grad=True)
        assert rel(gg[0], g_ref[0]) <= GRAD_TOL, (engine, contraction)
        if grad_bits:
            sm = (1 << (grad_bits - 1)) - 1
            unit = np.linalg.norm(g_ref[0]) / sm
            flips = np.abs(gg[1] - g_ref[1]) > 0.5 * unit
            assert flips.sum() <= 3
            assert np.abs(gg[1] - g_ref[1])[~flips].max() <= 1e-5 * unit + 1e-12
        else:
            assert (gg[0] == gg[1]).all()
    # whole epoch: the trajectories stay together (a rare flipped rounding moves one coordinate by one unit)
    x_ref, _ = oracle.sgd_epoch(ods, b, x0, 1024, 5e-4, model_bits=model_bits, grad_bits=grad_bits, seed=11, epoch=2)
    for contraction in (1, 2):
        x = to_dev(x0, ctx)
        ctx.zipml_sgd_epoch(gds, db, x, 1024, 5e-4, model_bits=model_bits, grad_bits=grad_bits, seed=11, epoch=2,
                            cluster_contraction=contraction)
        ctx.zipml_sync()
        assert rel(x.cpu().numpy(), x_ref) <= 20 * MODEL_TOL


def test_ring_engine_int8_path_with_quantized_model_and_gradient(ctx):
    """The ring engine's tensor-core contraction (uniform grid, tiles of 32-row chunks) under Q3 and Q4, on a
    step too large for one cluster: 2-bit codes, n = 8,192 (2 KB rows), B = 2,048."""
    m, n, batch = 4200, 8192, 2048
    _, A, b, _ = workload("c3", m, n, seed=7)
    ods = oracle.quantize(A, 2, seed=4)
    gds, db = dev_dataset(ods, ctx), to_dev(b, ctx)
    x0 = (np.random.default_rng(5).standard_normal(n) * 0.02).astype(np.float32)
    seed, epoch, step = 21, 1, 1
    xq_ref, _ = oracle.quantize_vector(x0, 8, seed, epoch, step, 3)
    margin, unit_x = q3_margins(x0, 8, seed, epoch, step)
    for engine in (binding.ENGINE_RING, binding.ENGINE_AUTO):
        x = to_dev(x0, ctx)
        g = torch.zeros((2, n), dtype=torch.float32, device=ctx.device)
        xq = torch.zeros(n, dtype=torch.float32, device=ctx.device)
        ctx.zipml_sgd_epoch(gds, db, x, batch, 5e-4, model_bits=8, grad_bits=8, seed=seed, epoch=epoch, first_step=step,
                            num_steps=1, engine=engine, grad_out=g, model_out=xq)
        ctx.zipml_sync()
        assert ctx.zipml_last_engine() == binding.ENGINE_RING
        gg, xq = g.cpu().numpy(), xq.cpu().numpy()
        differs = xq != xq_ref
        assert not (differs & (margin >= 1e-4)).any() and differs.sum() <= 3
        _, g_ref = oracle.sgd_epoch(ods, b, xq, batch, 5e-4, model_bits=0, grad_bits=8, seed=seed, epoch=epoch,
                                    first_step=step, num_steps=1, want_grad=True)
        assert rel(gg[0], g_ref[0]) <= GRAD_TOL
        unit = np.linalg.norm(g_ref[0]) / 127
        flips = np.abs(gg[1] - g_ref[1]) > 0.5 * unit
        assert flips.sum() <= 3 and np.abs(gg[1] - g_ref[1])[~flips].max() <= 1e-5 * unit + 1e-12
    x_ref, _ = oracle.sgd_epoch(ods, b, x0, batch, 5e-4, model_bits=8, grad_bits=8, seed=seed, epoch=epoch)
    x = to_dev(x0, ctx)
    ctx.zipml_sgd_epoch(gds, db, x, batch, 5e-4, model_bits=8, grad_bits=8, seed=seed, epoch=epoch, engine=binding.ENGINE_RING)
    ctx.zipml_sync()
    assert rel(x.cpu().numpy(), x_ref) <= 20 * MODEL_TOL


def test_auto_picks_the_engine_that_fits(ctx):
    """AUTO: cluster for small steps, column (else stream) for large uniform fp32 steps on wide rows, ring where they decline."""
    _, A, b, _ = workload("c5", 700, 20000, seed=2)                 # 2 x 300 rows x 10 KB: 6 MB per step, 157 column blocks
    ods = oracle.quantize(A, 4, seed=2)
    gds, db = dev_dataset(ods, ctx), to_dev(b, ctx)
    x0 = np.zeros(20000, np.float32)
    x_ref, _ = oracle.sgd_epoch(ods, b, x0, 300, 1e-4)
    x = to_dev(x0, ctx)
    ctx.zipml_sgd_epoch(gds, db, x, 300, 1e-4)
    ctx.zipml_sync()
    assert ctx.zipml_last_engine() == binding.ENGINE_COLUMN and rel(x.cpu().numpy(), x_ref) <= MODEL_TOL
    x_small, _ = oracle.sgd_epoch(ods, b, x0, 100, 1e-4)
    x = to_dev(x0, ctx)
    ctx.zipml_sgd_epoch(gds, db, x, 100, 1e-4)                               # short steps: the stream engine's
    ctx.zipml_sync()
    assert ctx.zipml_last_engine() == binding.ENGINE_STREAM and rel(x.cpu().numpy(), x_small) <= MODEL_TOL
    x = to_dev(x0, ctx)
    ctx.zipml_sgd_epoch(gds, db, x, 300, 1e-4, grad_bits=8, seed=3)          # quantized gradient: not the stream engine's
    ctx.zipml_sync()
    assert ctx.zipml_last_engine() == binding.ENGINE_RING
    _, A, b, _ = workload("c2", 600, 1000, seed=2)
    gds, db = dev_dataset(oracle.quantize(A, 8, seed=2), ctx), to_dev(b, ctx)
    ctx.zipml_sgd_epoch(gds, db, torch.zeros(1000, device=ctx.device), 64, 1e-3)     # 0.13 MB per step
    ctx.zipml_sync()
    assert ctx.zipml_last_engine() == binding.ENGINE_CLUSTER


REGS = [(binding.REG_L2, 0.5), (binding.REG_L1, 0.02), (binding.REG_NONNEG, 0.0), (binding.REG_LSSVM, 0.5)]


@pytest.mark.parametrize("reg,param", REGS)
@pytest.mark.parametrize("case", [SGD_CASES[1], SGD_CASES[2], SGD_CASES[4]], ids=lambda c: f"{c[0]}-{c[1]}x{c[2]}-b{c[3]}-B{c[4]}")
def test_sgd_regularised_update_parity(ctx, case, reg, param):
    """Every engine applies the regulariser of Eq. (proxupdate) / the least-squares SVM term as the oracle does."""
    key, m, n, bits, batch, lr = case
    _, A, b, _ = workload(key, m, n, seed=5)
    ods = oracle.quantize(A, bits, seed=6)
    gds, db = dev_dataset(ods, ctx), to_dev(b, ctx)
    x0 = (np.random.default_rng(7).standard_normal(n) * 0.1).astype(np.float32)
    lr = lr * 5
    if reg == binding.REG_L1:
        param = 0.05 / (lr * ((m + batch - 1) // batch))            # thresholds of an epoch add up to 0.05
    x_ref, g_ref = oracle.sgd_epoch(ods, b, x0, batch, lr, reg=reg, reg_param=param, want_grad=True)
    if reg == binding.REG_L1:
        assert (x_ref == 0).any() and (x_ref != 0).any()            # the threshold bites somewhere, not everywhere
    if reg == binding.REG_NONNEG:
        assert (x_ref >= 0).all() and ((x_ref == 0).any() or key == "c5")  # (c5's large first gradients lift every coordinate)
    engines = [binding.ENGINE_STEPWISE, binding.ENGINE_PERSISTENT, binding.ENGINE_RING, binding.ENGINE_LEAN, binding.ENGINE_CLUSTER,
               binding.ENGINE_STREAM, binding.ENGINE_AUTO]
    if gds.row_bytes >= 128:
        engines.append(binding.ENGINE_COLUMN)
    for engine in engines:
        x = to_dev(x0, ctx)
        g = torch.zeros((2, n), dtype=torch.float32, device=ctx.device)
        ctx.zipml_sgd_epoch(gds, db, x, batch, lr, engine=engine, reg=reg, reg_param=param, grad_out=g)
        ctx.zipml_sync()
        got = x.cpu().numpy()
        assert rel(got, x_ref) <= MODEL_TOL, engine
        if reg in (binding.REG_L1, binding.REG_NONNEG):
            # the switched-off coordinates agree except where y sits within rounding of the threshold
            assert ((got == 0) != (x_ref == 0)).sum() <= max(1, n // 200), engine
    with pytest.raises(binding.ZipmlError) as e:
        ctx.zipml_sgd_epoch(gds, db, to_dev(x0, ctx), batch, lr, reg=9)
    assert e.value.code == binding.ERR_INVALID_ARG
    with pytest.raises(binding.ZipmlError) as e:
        ctx.zipml_sgd_epoch(gds, db, to_dev(x0, ctx), batch, lr, reg=binding.REG_L2, reg_param=-0.1)
    assert e.value.code == binding.ERR_INVALID_ARG


def test_sgd_split_calls_equal_one_call(ctx):
    _, A, b, _ = workload("c1", 640, 64, seed=9)
    ods = oracle.quantize(A, 4, seed=1)
    gds, db = dev_dataset(ods, ctx), to_dev(b, ctx)
    x_all = torch.zeros(64, device=ctx.device)
    ctx.zipml_sgd_epoch(gds, db, x_all, 16, 0.01)
    x_two = torch.zeros(64, device=ctx.device)
    ctx.zipml_sgd_epoch(gds, db, x_two, 16, 0.01, first_step=0, num_steps=13)
    ctx.zipml_sgd_epoch(gds, db, x_two, 16, 0.01, first_step=13)
    ctx.zipml_sync()
    assert (x_all == x_two).all()
    with pytest.raises(binding.ZipmlError) as e:
        ctx.zipml_sgd_epoch(gds, db, x_two, 16, 0.01, first_step=39, num_steps=5)
    assert e.value.code == binding.ERR_INVALID_ARG
    with pytest.raises(binding.ZipmlError):
        ctx.zipml_sgd_epoch(gds, db, x_two, 0, 0.01)
    with pytest.raises(binding.ZipmlError):
        ctx.zipml_sgd_epoch(gds, db, x_two, 16, 0.01, batch_order=np.full(40, 99, np.int32))


# ---------------------------------------------------------------------------------------------
# loss
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("key,m,n,bits", [("c1", 1000, 64, 4), ("c2", 700, 1001, 8), ("c3", 300, 2048, 2),
                                          ("c5", 100, 5000, 4), ("c4u", 900, 77, 3)])
def test_loss_parity(ctx, key, m, n, bits):
    _, A, b, xs = workload(key, m, n, seed=2)
    x = (xs * 0.9).astype(np.float32)
    want = oracle.loss_dense(A, b, x)
    got = ctx.zipml_loss(binding.LOSS_DENSE, to_dev(b, ctx), to_dev(x, ctx), A=to_dev(A, ctx))
    ods = oracle.quantize(A, bits, seed=3)
    want_c = oracle.loss_codes(ods, b, x)
    got_c = ctx.zipml_loss(binding.LOSS_CODES, to_dev(b, ctx), to_dev(x, ctx), data=dev_dataset(ods, ctx))
    ctx.zipml_sync()
    assert abs(got.item() - want) <= LOSS_TOL * abs(want)
    assert abs(got_c.item() - want_c) <= LOSS_TOL * max(abs(want_c), abs(want))


def test_loss_codes_with_level_table_and_strided_dense(ctx):
    _, A, b, xs = workload("c4", 2000, 60, seed=1)
    lev, _ = oracle.optimal_levels(A, 3, 128)
    ods = oracle.quantize(A, 3, seed=3, mode=oracle.TABLE, levels=lev)
    want_c = oracle.loss_codes(ods, b, xs)
    got_c = ctx.zipml_loss(binding.LOSS_CODES, to_dev(b, ctx), to_dev(xs, ctx), data=dev_dataset(ods, ctx))
    big = torch.zeros((2000, 71), device=ctx.device)
    big[:, 1:61] = to_dev(A, ctx)
    got = ctx.zipml_loss(binding.LOSS_DENSE, to_dev(b, ctx), to_dev(xs, ctx), A=big[:, 1:61])
    ctx.zipml_sync()
    assert abs(got_c.item() - want_c) <= LOSS_TOL * abs(want_c)
    assert abs(got.item() - oracle.loss_dense(A, b, xs)) <= LOSS_TOL * oracle.loss_dense(A, b, xs)


def test_loss_codes_with_a_stride_far_above_the_minimum(ctx):
    """Planes that are column slices of a wider packed matrix: the row stride, not n, sizes what the loss stages."""
    _, A, b, xs = workload("c3", 200, 100, seed=5)
    ods = oracle.quantize(A, 2, seed=6)
    want_c = oracle.loss_codes(ods, b, xs)
    stride = 80 * 1024
    wide1 = torch.zeros((200, stride), dtype=torch.uint8, device=ctx.device)
    wide2 = torch.zeros((200, stride), dtype=torch.uint8, device=ctx.device)
    wide1[:, : ods.row_bytes] = to_dev(ods.plane1, ctx)
    wide2[:, : ods.row_bytes] = to_dev(ods.plane2, ctx)
    gds = binding.Dataset(wide1, wide2, 200, 100, 2, binding.LEVELS_UNIFORM, to_dev(ods.feat_lo, ctx), to_dev(ods.feat_step, ctx), None)
    with binding.Context(ctx.device) as fresh:                     # a context whose workspace has not grown yet
        got_c = fresh.zipml_loss(binding.LOSS_CODES, to_dev(b, ctx), to_dev(xs, ctx), data=gds)
        fresh.zipml_sync()
    assert abs(got_c.item() - want_c) <= LOSS_TOL * abs(want_c)


# ---------------------------------------------------------------------------------------------
# shared-base storage of the two samples (Section 2.2, "Overhead of Storing Samples")
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("key,m,n,bits", [("c1", 300, 64, 4), ("c2", 129, 1003, 8), ("c3", 77, 2050, 2), ("c4u", 100, 37, 3),
                                          ("c5", 40, 4100, 4), ("c1", 1, 5, 8)])
def test_shared_base_planes_bit_exact(ctx, key, m, n, bits):
    _, A, b, xs = workload(key, m, n, seed=bits)
    ods = oracle.quantize(A, bits, seed=21)
    base, up1, up2 = oracle.shared_base_encode(ods)
    gds = dev_dataset(ods, ctx)
    sb = ctx.zipml_shared_base_encode(gds)
    ctx.zipml_sync()
    assert (sb.base.cpu().numpy() == base).all() and (sb.up1.cpu().numpy() == up1).all() and (sb.up2.cpu().numpy() == up2).all()
    back = ctx.zipml_shared_base_decode(sb)
    ctx.zipml_sync()
    assert (back.plane1.cpu().numpy() == ods.plane1).all() and (back.plane2.cpu().numpy() == ods.plane2).all()
    if bits > 2 and n > 256:                          # 6 instead of 8, 10 instead of 16 bits per value (2-bit codes gain nothing)
        assert sb.packed_bytes < gds.packed_bytes
    # the loss straight from the three planes is the oracle's estimate from the two
    x = (xs * 0.9).astype(np.float32)
    want = oracle.loss_codes(ods, b, x)
    got = ctx.zipml_loss_shared_base(sb, to_dev(b, ctx), to_dev(x, ctx))
    ctx.zipml_sync()
    assert abs(got.item() - want) <= LOSS_TOL * max(abs(want), oracle.loss_dense(A, b, x))


def test_shared_base_epoch_and_refusals(ctx):
    """An epoch from shared-base data gives the model of the two-plane data, bit for bit (the same planes reach the
    same engine); planes that are not two samples of one value are refused."""
    _, A, b, _ = workload("c2", 2100, 1000, seed=1)
    ods = oracle.quantize(A, 8, seed=7)
    gds, db = dev_dataset(ods, ctx), to_dev(b, ctx)
    sb = ctx.zipml_shared_base_encode(gds)
    x0 = (np.random.default_rng(1).standard_normal(1000) * 0.1).astype(np.float32)
    x_ref, g_ref = oracle.sgd_epoch(ods, b, x0, 256, 1e-3, want_grad=True)
    x1, x2 = to_dev(x0, ctx), to_dev(x0, ctx)
    g = torch.zeros((2, 1000), dtype=torch.float32, device=ctx.device)
    ctx.zipml_sgd_epoch_shared_base(sb, db, x1, 256, 1e-3, grad_out=g)
    ctx.zipml_sgd_epoch(gds, db, x2, 256, 1e-3)
    ctx.zipml_sync()
    assert rel(x1.cpu().numpy(), x_ref) <= MODEL_TOL and (x1 == x2).all()
    assert rel(g[0].cpu().numpy(), g_ref[0]) <= 10 * GRAD_TOL           # (the epoch's last step, from the kernel's own model)
    far = torch.zeros_like(gds.plane1)
    far[:, 0] = 2                                                        # plane 1 says code 2 where plane 2 says 0
    bad = binding.Dataset(far, torch.zeros_like(far), gds.m, gds.n, 8, binding.LEVELS_UNIFORM, gds.feat_lo, gds.feat_step, None)
    ctx.zipml_shared_base_encode(bad)
    with pytest.raises(binding.ZipmlError) as e:
        ctx.zipml_sync()
    assert e.value.code == binding.ERR_INVALID_ARG
    ctx.zipml_sync()


# ---------------------------------------------------------------------------------------------
# the configurations at their own step shapes (a few minibatches of rows)
# ---------------------------------------------------------------------------------------------
def test_config5_step_shape(ctx):
    """Config 5 as it runs: n = 32,768 (16 KB packed rows), 4-bit, B = 2,048; two full minibatches and a ragged one.
    Planes bit-exact, then the engine AUTO picks for this shape: model after the epoch and the last step's gradient."""
    m, n, batch, lr = 2 * 2048 + 1000, 32768, 2048, 1e-4
    _, A, b, _ = workload("c5", m, n, seed=0)
    ods = oracle.quantize(A, 4, seed=0)
    dA = to_dev(A, ctx)
    gds = ctx.zipml_quantize(dA, 4, seed=0)
    ctx.zipml_sync()
    del dA
    assert (gds.feat_lo.cpu().numpy() == ods.feat_lo).all() and (gds.feat_step.cpu().numpy() == ods.feat_step).all()
    assert (gds.plane1.cpu().numpy() == ods.plane1).all() and (gds.plane2.cpu().numpy() == ods.plane2).all()
    db = to_dev(b, ctx)
    x0 = np.zeros(n, np.float32)
    x_ref, _ = oracle.sgd_epoch(ods, b, x0, batch, lr)
    x_before, _ = oracle.sgd_epoch(ods, b, x0, batch, lr, num_steps=2)
    _, g_ref = oracle.sgd_epoch(ods, b, x_before, batch, lr, first_step=2, num_steps=1, want_grad=True)
    for engine in (binding.ENGINE_AUTO, binding.ENGINE_STREAM, binding.ENGINE_COLUMN):
        x = to_dev(x0, ctx)
        ctx.zipml_sgd_epoch(gds, db, x, batch, lr, engine=engine)
        ctx.zipml_sync()
        if engine == binding.ENGINE_AUTO:
            assert ctx.zipml_last_engine() == binding.ENGINE_COLUMN
        assert rel(x.cpu().numpy(), x_ref) <= MODEL_TOL, engine
        xb = to_dev(x_before, ctx)
        g = torch.zeros((2, n), dtype=torch.float32, device=ctx.device)
        ctx.zipml_sgd_epoch(gds, db, xb, batch, lr, first_step=2, num_steps=1, grad_out=g, engine=engine)
        ctx.zipml_sync()
        assert rel(g[0].cpu().numpy(), g_ref[0]) <= GRAD_TOL, engine
        # the full step before it too (2,048 rows)
        _, g_full = oracle.sgd_epoch(ods, b, x_before, batch, lr, first_step=1, num_steps=1, want_grad=True)
        xb = to_dev(x_before, ctx)
        ctx.zipml_sgd_epoch(gds, db, xb, batch, lr, first_step=1, num_steps=1, grad_out=g, engine=engine)
        ctx.zipml_sync()
        assert rel(g[0].cpu().numpy(), g_full[0]) <= GRAD_TOL, engine
    want = oracle.loss_codes(ods, b, x_ref)
    got = ctx.zipml_loss(binding.LOSS_CODES, db, to_dev(x_ref, ctx), data=gds)
    ctx.zipml_sync()
    assert abs(got.item() - want) <= LOSS_TOL * max(abs(want), oracle.loss_dense(A, b, x_ref))


def test_config4_step_shape_with_level_table(ctx):
    """Config 4 as it runs: n = 512, 3-bit variance-optimal levels from a 1,024-bin histogram, B = 512."""
    m, n, batch, lr = 3 * 512 + 100, 512, 512, 1e-3
    _, A, b, _ = workload("c4", m, n, seed=0)
    lev, obj = oracle.optimal_levels(A, 3, 1024)
    ods = oracle.quantize(A, 3, seed=0, mode=oracle.TABLE, levels=lev)
    dA = to_dev(A, ctx)
    glev, gobj = ctx.zipml_optimal_levels(dA, 3, 1024, want_objective=True)
    gds = ctx.zipml_quantize(dA, 3, seed=0, level_mode=binding.LEVELS_TABLE, levels=glev)
    ctx.zipml_sync()
    assert (glev.cpu().numpy() == lev).all() and (gobj.cpu().numpy().astype(np.uint64) == obj).all()
    assert (gds.plane1.cpu().numpy() == ods.plane1).all() and (gds.plane2.cpu().numpy() == ods.plane2).all()
    db = to_dev(b, ctx)
    x0 = np.zeros(n, np.float32)
    x_ref, _ = oracle.sgd_epoch(ods, b, x0, batch, lr)
    x_before, _ = oracle.sgd_epoch(ods, b, x0, batch, lr, num_steps=2)
    _, g_ref = oracle.sgd_epoch(ods, b, x_before, batch, lr, first_step=2, num_steps=1, want_grad=True)
    x = to_dev(x0, ctx)
    ctx.zipml_sgd_epoch(gds, db, x, batch, lr)
    ctx.zipml_sync()
    assert ctx.zipml_last_engine() == binding.ENGINE_CLUSTER and rel(x.cpu().numpy(), x_ref) <= MODEL_TOL
    xb = to_dev(x_before, ctx)
    g = torch.zeros((2, n), dtype=torch.float32, device=ctx.device)
    ctx.zipml_sgd_epoch(gds, db, xb, batch, lr, first_step=2, num_steps=1, grad_out=g)
    ctx.zipml_sync()
    assert rel(g[0].cpu().numpy(), g_ref[0]) <= GRAD_TOL
    want = oracle.loss_codes(ods, b, x_ref)
    got = ctx.zipml_loss(binding.LOSS_CODES, db, to_dev(x_ref, ctx), data=gds)
    ctx.zipml_sync()
    assert abs(got.item() - want) <= LOSS_TOL * max(abs(want), oracle.loss_dense(A, b, x_ref))


def test_quantize_rows_more_than_2_to_31_elements_apart(ctx):
    """A strided view whose last row starts beyond element 2^31 of its buffer: row * lda must be 64-bit arithmetic."""
    m, n, lda = 4, 300, 800_000_000
    _, A, _, _ = workload("c2", m, n, seed=4)
    big = torch.empty((m - 1) * lda + n, dtype=torch.float32, device=ctx.device)     # 9.6 GB, touched only at the rows
    view = big.as_strided((m, n), (lda, 1))
    view.copy_(to_dev(A, ctx))
    ods = oracle.quantize(A, 8, seed=77)
    gds = ctx.zipml_quantize(view, 8, seed=77)
    ctx.zipml_sync()
    assert (gds.feat_lo.cpu().numpy() == ods.feat_lo).all() and (gds.feat_step.cpu().numpy() == ods.feat_step).all()
    assert (gds.plane1.cpu().numpy() == ods.plane1).all() and (gds.plane2.cpu().numpy() == ods.plane2).all()
    lev, _ = oracle.optimal_levels(A, 2, 64)
    glev = ctx.zipml_optimal_levels(view, 2, 64)
    want = oracle.loss_dense(A, np.ones(m, np.float32), np.ones(n, np.float32))
    got = ctx.zipml_loss(binding.LOSS_DENSE, torch.ones(m, device=ctx.device), torch.ones(n, device=ctx.device), A=view)
    ctx.zipml_sync()
    assert (glev.cpu().numpy() == lev).all() and abs(got.item() - want) <= LOSS_TOL * want
    del big, view


# ---------------------------------------------------------------------------------------------
# whole path from host buffers
# ---------------------------------------------------------------------------------------------
def test_train_host_matches_oracle_pipeline(ctx):
    w, A, b, _ = workload("c1", 2048, 64, seed=0)
    x = torch.zeros(64)
    loss = ctx.zipml_train_host(torch.from_numpy(A), torch.from_numpy(b), x, bits=4, batch=16, lr=0.01, epochs=3,
                                quantize_seed=5)
    ods = oracle.quantize(A, 4, seed=5)
    xr = np.zeros(64, np.float32)
    for ep in range(3):
        xr, _ = oracle.sgd_epoch(ods, b, xr, 16, 0.01, epoch=ep)
    assert rel(x.numpy(), xr) <= MODEL_TOL
    want = oracle.loss_dense(A, b, xr)
    assert abs(loss - want) <= 1e-3 * want
    # with optimal levels and the alpha/epoch schedule
    w, A, b, _ = workload("c4", 3000, 48, seed=0)
    x = torch.zeros(48)
    loss = ctx.zipml_train_host(torch.from_numpy(A), torch.from_numpy(b), x, bits=3, batch=512, lr=0.05, epochs=2,
                                optimal_levels=True, hist_bins=256, quantize_seed=8, lr_decay=True)
    lev, _ = oracle.optimal_levels(A, 3, 256)
    ods = oracle.quantize(A, 3, seed=8, mode=oracle.TABLE, levels=lev)
    xr = np.zeros(48, np.float32)
    for ep in range(2):
        xr, _ = oracle.sgd_epoch(ods, b, xr, 512, np.float32(0.05) / np.float32(ep + 1), epoch=ep)
    assert rel(x.numpy(), xr) <= MODEL_TOL
    assert abs(loss - oracle.loss_dense(A, b, xr)) <= 1e-3 * oracle.loss_dense(A, b, xr)


@pytest.mark.parametrize("grad_bits,reg,reg_param", [(0, 0, 0.0), (6, 0, 0.0), (8, 1, 0.5), (4, 2, 0.01), (0, 3, 0.0), (5, 4, 0.3)])
def test_apply_gradient_is_the_end_of_a_step(ctx, grad_bits, reg, reg_param):
    """zipml_sgd_apply_gradient: Q4 (Supplement "Quantizing the Gradients") and the update (Eq. (proxupdate), LS-SVM
    term) on a gradient from outside, with the draws of zipml_sgd_epoch: fed the oracle's own pre-Q4 gradient of a
    step it must land on the oracle's model after that step."""
    m, n, batch, lr, seed, epoch, step = 1500, 700, 256, 0.02, 9, 3, 4
    _, A, b, _ = workload("c1", m, n, seed=8)
    ods = oracle.quantize(A, 4, seed=1)
    x0 = (np.random.default_rng(2).standard_normal(n) * 0.1).astype(np.float32)
    x1, g_ref = oracle.sgd_epoch(ods, b, x0, batch, lr, grad_bits=grad_bits, seed=seed, epoch=epoch, first_step=step,
                                 num_steps=1, want_grad=True, reg=reg, reg_param=reg_param)
    x, g = to_dev(x0, ctx), to_dev(g_ref[0], ctx)
    applied = torch.zeros(n, dtype=torch.float32, device=ctx.device)
    ctx.zipml_sgd_apply_gradient(x, g, step, lr, applied_out=applied, grad_bits=grad_bits, seed=seed, epoch=epoch, reg=reg,
                                 reg_param=reg_param)
    ctx.zipml_sync()
    got, app = x.cpu().numpy(), applied.cpu().numpy()
    if grad_bits:
        unit = np.linalg.norm(g_ref[0]) / ((1 << (grad_bits - 1)) - 1)
        flips = np.abs(app - g_ref[1]) > 0.5 * unit                # (a last-bit difference in the norm may flip a rounding)
        assert flips.sum() <= 2
        assert np.abs(app - g_ref[1])[~flips].max() <= 1e-5 * unit + 1e-12
        assert np.abs(got - x1)[~flips].max() <= 1e-6 * max(1.0, np.abs(x1).max())
    else:
        assert (app == g_ref[0]).all()
        assert np.abs(got - x1).max() <= 1e-6 * max(1.0, np.abs(x1).max())
    # refusals: nothing runs
    with pytest.raises(binding.ZipmlError):
        ctx.zipml_sgd_apply_gradient(x, g, -1, lr)
    with pytest.raises(binding.ZipmlError):
        ctx.zipml_sgd_apply_gradient(x, g, 0, lr, grad_bits=1)
    with pytest.raises(binding.ZipmlError):
        ctx.zipml_sgd_apply_gradient(x, g, 0, lr, reg=1, reg_param=-1.0)


@pytest.mark.parametrize("world", [1, 2, 4])
@pytest.mark.parametrize("case", ["plain_ragged", "q3_q4_shuffled", "wide_l2"])
def test_row_sharded_epoch_matches_the_whole_epoch(ctx, world, case):
    """The row-sharded epoch (one all-reduce of n floats per step) with its ranks run in turn on this GPU, every
    rank on its own rows and its own replica of x: all replicas end as the same bits, at the model of the
    unsharded zipml_sgd_epoch and of the oracle's epoch."""
    from paper_1611_05402_b200.sharded import ShardPlan, ShardedEpoch, take_rows
    m, n, bits, batch, mb, gb, shuffled, reg, rp = {
        "plain_ragged": (1100, 300, 4, 128, 0, 0, False, 0, 0.0),      # last batch: 76 rows: some ranks hold none of it
        "q3_q4_shuffled": (1024, 520, 2, 256, 8, 8, True, 0, 0.0),
        "wide_l2": (900, 4096, 4, 512, 0, 0, False, 1, 0.2),           # big steps: other engines serve the shares
    }[case]
    lr, seed, epoch = 0.01, 11, 2
    _, A, b, _ = workload("c1", m, n, seed=4)
    ods = oracle.quantize(A, bits, seed=3)
    gds, db = dev_dataset(ods, ctx), to_dev(b, ctx)
    T = (m + batch - 1) // batch
    order = [int(o) for o in np.random.default_rng(1).permutation(T)] if shuffled else None
    x0 = np.zeros(n, np.float32)
    kw = dict(model_bits=mb, grad_bits=gb, seed=seed, epoch=epoch, reg=reg, reg_param=rp)
    ranks = []
    for r in range(world):
        plan = ShardPlan(m, batch, r, world)
        p1, p2 = take_rows(plan, gds.plane1), take_rows(plan, gds.plane2)
        dl = binding.Dataset(p1, p2, p1.shape[0], n, bits, gds.level_mode, gds.feat_lo, gds.feat_step, gds.levels)
        ranks.append(ShardedEpoch(ctx, plan, dl, take_rows(plan, db), to_dev(x0, ctx), lr, batch_order=order, **kw))
    pos = [0]

    def all_reduce(v):                     # rank 0's share arrives; the others' are formed and added, and applied
        t = order[pos[0]] if order else pos[0]
        for other in ranks[1:]:
            v += other.share(pos[0], t, other.plan.weight(t))
        for other in ranks[1:]:
            other.apply(v.clone(), pos[0])
        pos[0] += 1

    ranks[0].run(all_reduce=all_reduce)
    ctx.zipml_sync()
    xs = [rk.x.cpu().numpy() for rk in ranks]
    for other in xs[1:]:
        assert np.array_equal(xs[0], other)
    whole = to_dev(x0, ctx)
    ctx.zipml_sgd_epoch(gds, db, whole, batch, lr, batch_order=order, **kw)
    ctx.zipml_sync()
    x_ref, _ = oracle.sgd_epoch(ods, b, x0, batch, lr, batch_order=order, **kw)
    assert np.abs(x_ref).max() > 1e-3
    tol = (20 if (mb or gb) else 1) * MODEL_TOL
    assert rel(xs[0], x_ref) <= tol
    assert rel(xs[0], whole.cpu().numpy()) <= 2 * tol


@pytest.mark.parametrize("bits,mode", [(2, "uniform"), (4, "uniform"), (8, "uniform"), (3, "table")])
def test_polynomial_estimator_over_independent_quantizations(ctx, bits, mode):
    """Section 4.1 "Quantizing Polynomials" and Section 4.2's gradient: further draws of zipml_quantize_draw are
    bit-exact against the oracle's (and differ from draw 0), Q(P) per sample and the weighted plane mean match the
    oracle from the same planes."""
    m, n, d = 1300, 333, 5
    _, A, b, _ = workload("c4" if mode == "table" else "c1", m, n, seed=9)
    dA = to_dev(A, ctx)
    kw, okw = {}, {}
    if mode == "table":
        lev, _ = oracle.optimal_levels(A, bits, 256)
        kw = dict(level_mode=binding.LEVELS_TABLE, levels=to_dev(lev, ctx))
        okw = dict(mode=oracle.TABLE, levels=lev)
    planes, oplanes, grid, ogrid = [], [], None, None
    for q in range((d + 2) // 2):                                  # d planes for Q(P), one more for the gradient
        ds = ctx.zipml_quantize(dA, bits, seed=5, draw=q, **kw)
        ods = oracle.quantize_pair(A, bits, 5, q, **okw)
        ctx.zipml_sync()
        assert np.array_equal(ds.plane1.cpu().numpy(), ods.plane1) and np.array_equal(ds.plane2.cpu().numpy(), ods.plane2)
        grid, ogrid = grid or ds, ogrid or ods
        planes += [ds.plane1, ds.plane2]
        oplanes += [ods.plane1, ods.plane2]
    assert not np.array_equal(oplanes[0], oplanes[2])
    x = (np.random.default_rng(2).standard_normal(n) * (0.3 / np.sqrt(n))).astype(np.float32)
    coef = [0.5, 0.25, -0.125, 0.3, -0.2, 0.1]
    labels = np.where(b > np.median(b), 1.0, -1.0).astype(np.float32)
    for deg in (0, 1, 3, 5):
        want = oracle.poly_rows(oplanes, ogrid, x, coef[:deg + 1], scale=labels)
        got = ctx.zipml_poly_rows(grid, planes, coef[:deg + 1], to_dev(x, ctx), scale=to_dev(labels, ctx))
        ctx.zipml_sync()
        assert np.abs(got.cpu().numpy() - want).max() <= 1e-5 * max(1.0, np.abs(want).max()), deg
    c = oracle.poly_rows(oplanes, ogrid, x, coef, scale=labels)
    g_want = oracle.weighted_plane_mean(oplanes[d], ogrid, c)
    g = ctx.zipml_weighted_plane_mean(grid, planes[d], torch.from_numpy(c).to(ctx.device))
    ctx.zipml_sync()
    assert rel(g.cpu().numpy(), g_want) <= GRAD_TOL
    with pytest.raises(binding.ZipmlError):
        ctx.zipml_poly_rows(grid, planes * 2, [1.0] * 10, to_dev(x, ctx))          # degree 9 > ZIPML_POLY_MAX_DEGREE
    with pytest.raises(binding.ZipmlError):
        ctx.zipml_poly_rows(grid, [planes[0].view(-1)[1:]], [0.0, 1.0], to_dev(x, ctx))     # a misaligned plane


@pytest.mark.parametrize("bits", [1, 5, 6, 7])
def test_bit_widths_in_wider_containers(ctx, bits):
    """1-bit codes in 2-bit fields and 5- to 7-bit codes in bytes (the paper's operating points are 5-6 bits): planes
    bit-exact, the code-plane loss, an epoch through AUTO on a small step and through the column and stream engines
    on a large one."""
    _, A, b, _ = workload("c2", 700, 200, seed=bits)
    ods = oracle.quantize(A, bits, seed=4)
    gds = ctx.zipml_quantize(to_dev(A, ctx), bits, seed=4)
    ctx.zipml_sync()
    assert np.array_equal(gds.plane1.cpu().numpy(), ods.plane1) and np.array_equal(gds.plane2.cpu().numpy(), ods.plane2)
    assert np.array_equal(gds.feat_step.cpu().numpy(), ods.feat_step)
    x0 = (np.random.default_rng(1).standard_normal(200) * 0.05).astype(np.float32)
    loss = ctx.zipml_loss(binding.LOSS_CODES, to_dev(b, ctx), to_dev(x0, ctx), data=gds)
    ctx.zipml_sync()
    want = oracle.loss_codes(ods, b, x0)
    assert abs(loss.item() - want) <= LOSS_TOL * abs(want)
    x = to_dev(x0, ctx)
    ctx.zipml_sgd_epoch(gds, to_dev(b, ctx), x, 64, 1e-3, model_bits=bits if bits > 1 else 0, grad_bits=0, seed=3)
    ctx.zipml_sync()
    x_ref, _ = oracle.sgd_epoch(ods, b, x0, 64, 1e-3, model_bits=bits if bits > 1 else 0, grad_bits=0, seed=3)
    assert rel(x.cpu().numpy(), x_ref) <= 20 * MODEL_TOL
    # a large step: 300 rows of 16 KB (1-bit: 8 KB), B = 300 -> the column engine, and the stream engine beside it
    n2 = 16384 if bits > 1 else 32768
    _, A2, b2, _ = workload("c5", 300, n2, seed=bits)
    ods2 = oracle.quantize(A2, bits, seed=6)
    gds2 = dev_dataset(ods2, ctx)
    x_ref2, _ = oracle.sgd_epoch(ods2, b2, np.zeros(n2, np.float32), 300, 1e-3)
    for engine in (binding.ENGINE_COLUMN, binding.ENGINE_STREAM):
        x2 = torch.zeros(n2, device=ctx.device)
        ctx.zipml_sgd_epoch(gds2, to_dev(b2, ctx), x2, 300, 1e-3, engine=engine)
        ctx.zipml_sync()
        assert rel(x2.cpu().numpy(), x_ref2) <= MODEL_TOL, engine
    with pytest.raises(binding.ZipmlError):
        ctx.zipml_quantize(to_dev(A, ctx), 9, seed=0)
    if bits > 4:
        with pytest.raises(binding.ZipmlError):
            ctx.zipml_quantize(to_dev(A, ctx), bits, seed=0, level_mode=binding.LEVELS_TABLE,
                               levels=torch.zeros((200, 1 << bits), device=ctx.device))


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_symmetric_grid(ctx, bits):
    """ZIPML_GRID_SYMMETRIC (Supplement "Column Scaling": levels on [-M_j, M_j]): planes, lo and step bit-exact against
    the oracle, and an epoch on such data."""
    _, A, b, _ = workload("c2", 900, 260, seed=bits)
    A = (A + 0.3).astype(np.float32)                          # ranges that are not symmetric by themselves
    ods = oracle.quantize_pair(A, bits, 7, 0, symmetric=True)
    gds = ctx.zipml_quantize(to_dev(A, ctx), bits, seed=7, grid=binding.GRID_SYMMETRIC)
    ctx.zipml_sync()
    assert np.array_equal(gds.plane1.cpu().numpy(), ods.plane1) and np.array_equal(gds.plane2.cpu().numpy(), ods.plane2)
    assert np.array_equal(gds.feat_lo.cpu().numpy(), ods.feat_lo) and np.array_equal(gds.feat_step.cpu().numpy(), ods.feat_step)
    assert np.array_equal(ods.feat_lo, -np.abs(A).max(axis=0))
    x = torch.zeros(260, device=ctx.device)
    ctx.zipml_sgd_epoch(gds, to_dev(b, ctx), x, 128, 1e-3)
    ctx.zipml_sync()
    x_ref, _ = oracle.sgd_epoch(ods, b, np.zeros(260, np.float32), 128, 1e-3)
    assert rel(x.cpu().numpy(), x_ref) <= MODEL_TOL
    with pytest.raises(binding.ZipmlError):
        ctx.zipml_quantize(to_dev(A, ctx), 3, seed=0, grid=binding.GRID_SYMMETRIC, level_mode=binding.LEVELS_TABLE,
                           levels=torch.zeros((260, 8), device=ctx.device))
    with pytest.raises(binding.ZipmlError):
        ctx.zipml_quantize(to_dev(A, ctx), bits, seed=0, grid=2)


def test_vector_scaling_by_the_largest_entry(ctx):
    """ZIPML_NORM_LINF: Q3 and Q4 scaled by max |v_i| (the Supplement leaves M(v) general).  AUTO runs the
    first-generation engine for it, the others refuse; an epoch and a single step against the oracle, and
    zipml_sgd_apply_gradient with the same option."""
    m, n, batch, lr = 2000, 300, 250, 2e-3
    _, A, b, _ = workload("c2", m, n, seed=12)
    ods = oracle.quantize(A, 4, seed=2)
    gds, db = dev_dataset(ods, ctx), to_dev(b, ctx)
    x0 = (np.random.default_rng(3).standard_normal(n) * 0.05).astype(np.float32)
    kw = dict(model_bits=6, grad_bits=6, seed=5, epoch=1)
    # one step: gradient before Q4 from the model the kernel used, then Q4's decisions
    x, g = to_dev(x0, ctx), torch.zeros((2, n), dtype=torch.float32, device=ctx.device)
    xq = torch.zeros(n, dtype=torch.float32, device=ctx.device)
    ctx.zipml_sgd_epoch(gds, db, x, batch, lr, first_step=2, num_steps=1, grad_out=g, model_out=xq, vector_norm=binding.NORM_LINF, **kw)
    ctx.zipml_sync()
    assert ctx.zipml_last_engine() in (binding.ENGINE_STEPWISE, binding.ENGINE_PERSISTENT)
    xq_ref, _ = oracle.quantize_vector(x0, 6, 5, 1, 2, 3, norm=oracle.NORM_LINF)
    assert (xq.cpu().numpy() != xq_ref).sum() <= 2
    _, g_ref = oracle.sgd_epoch(ods, b, xq.cpu().numpy(), batch, lr, model_bits=0, grad_bits=6, seed=5, epoch=1, first_step=2,
                                num_steps=1, want_grad=True, vector_norm=oracle.NORM_LINF)
    gg = g.cpu().numpy()
    assert rel(gg[0], g_ref[0]) <= GRAD_TOL
    unit = np.abs(g_ref[0]).max() / 31
    flips = np.abs(gg[1] - g_ref[1]) > 0.5 * unit
    assert flips.sum() <= 2 and np.abs(gg[1] - g_ref[1])[~flips].max() <= 1e-5 * unit + 1e-12
    assert np.abs(gg[1]).max() <= np.abs(gg[0]).max() * (1 + 1e-6)          # nothing beyond the largest entry
    # whole epoch
    x = to_dev(x0, ctx)
    ctx.zipml_sgd_epoch(gds, db, x, batch, lr, vector_norm=binding.NORM_LINF, **kw)
    ctx.zipml_sync()
    x_ref, _ = oracle.sgd_epoch(ods, b, x0, batch, lr, vector_norm=oracle.NORM_LINF, **kw)
    assert rel(x.cpu().numpy(), x_ref) <= 20 * MODEL_TOL
    x_l2, _ = oracle.sgd_epoch(ods, b, x0, batch, lr, **kw)
    assert rel(x_l2, x_ref) > 1e-3                                           # the option does change the trajectory
    # the end of a step on its own
    xa = to_dev(x0, ctx)
    ctx.zipml_sgd_apply_gradient(xa, to_dev(g_ref[0], ctx), 2, lr, grad_bits=6, seed=5, epoch=1, vector_norm=binding.NORM_LINF)
    ctx.zipml_sync()
    want = x0 - np.float32(lr) * g_ref[1]
    assert (np.abs(xa.cpu().numpy() - want) > 1e-6).sum() <= 2
    # other engines refuse; without Q3/Q4 the option means nothing and every engine runs
    for engine in (binding.ENGINE_CLUSTER, binding.ENGINE_LEAN, binding.ENGINE_RING):
        with pytest.raises(binding.ZipmlError) as e:
            ctx.zipml_sgd_epoch(gds, db, to_dev(x0, ctx), batch, lr, engine=engine, vector_norm=binding.NORM_LINF, **kw)
        assert e.value.code == binding.ERR_UNSUPPORTED
    ctx.zipml_sgd_epoch(gds, db, to_dev(x0, ctx), batch, lr, engine=binding.ENGINE_CLUSTER, vector_norm=binding.NORM_LINF)
    ctx.zipml_sync()
    with pytest.raises(binding.ZipmlError):
        ctx.zipml_sgd_epoch(gds, db, to_dev(x0, ctx), batch, lr, vector_norm=2)
