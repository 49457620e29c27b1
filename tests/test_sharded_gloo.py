"""Row-sharded epoch on CPU ranks: the partition and the step loop of paper_1611_05402_b200.sharded, driven with the
oracle's arithmetic on two gloo ranks, reproduce the single-rank oracle epoch (paper Eq. (double), symmetrised;
"End-to-end Quantization"): the gradient of a minibatch is the sum of the ranks' shares, Q3/Q4 draw from counters
that do not know the rank."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_1611_05402_b200.sharded import ShardPlan, run_steps, take_rows  # noqa: E402

CASES = {
    # name: m, n, bits, batch, model_bits, grad_bits, order, reg, reg_param
    "plain_ragged": (203, 37, 4, 16, 0, 0, False, 0, 0.0),          # last batch: 11 rows, rank 1 holds 3 of them
    "rank_without_last_batch": (197, 24, 3, 16, 0, 0, False, 0, 0.0),  # last batch: 5 rows, all on rank 0
    "q3_q4_shuffled": (192, 40, 4, 32, 6, 6, True, 0, 0.0),
    "l2_prox": (160, 16, 2, 16, 0, 0, False, 1, 0.5),
}


def _problem(m, n, seed=5):
    rng = np.random.default_rng(seed)
    A = rng.standard_normal((m, n)).astype(np.float32) * rng.uniform(0.2, 2.0, n).astype(np.float32)
    xs = rng.standard_normal(n).astype(np.float32)
    b = (A @ xs + 0.05 * rng.standard_normal(m)).astype(np.float32)
    return A, b


def _oracle_dataset_rows(oracle, ds, plan):
    p1, p2 = take_rows(plan, ds.plane1), take_rows(plan, ds.plane2)
    return oracle.Dataset(p1, p2, p1.shape[0], ds.n, ds.bits, ds.mode, ds.feat_lo, ds.feat_step, ds.levels)


def _sharded_epoch(oracle, plan, ds, b, x0, lr, model_bits, grad_bits, order, reg, reg_param, all_reduce, seed=11, epoch=2):
    dl, bl = _oracle_dataset_rows(oracle, ds, plan), take_rows(plan, b)
    x = np.array(x0, dtype=np.float32)
    T_local = plan.local_steps
    n = ds.n

    def share(pos, t, weight):
        if plan.count(t) == 0:
            return np.zeros(n, np.float32)
        lo = None
        if order is not None:
            lo = [min(int(o), T_local - 1) for o in order][:T_local]
            lo[pos] = t
        _, g = oracle.sgd_epoch(dl, bl, x, plan.local_batch, 0.0, model_bits=model_bits, grad_bits=0, seed=seed, epoch=epoch,
                                first_step=pos, num_steps=1, batch_order=lo, want_grad=True)
        return (g[0] * np.float32(weight)).astype(np.float32)

    def apply(v, pos):
        g = v
        if grad_bits:
            g, _ = oracle.quantize_vector(v, grad_bits, seed, epoch, pos, 4)
        y = x - np.float32(lr) * g
        if reg == 1:
            y = y * np.float32(1.0 / (1.0 + lr * reg_param))
        x[:] = y.astype(np.float32)

    run_steps(plan, share, all_reduce, apply, order=order)
    return x


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import oracle
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        def all_reduce(v):
            t = torch.from_numpy(v)
            dist.all_reduce(t, op=dist.ReduceOp.SUM)

        res = {}
        for name, (m, n, bits, batch, mb, gb, shuffled, reg, rp) in CASES.items():
            A, b = _problem(m, n)
            ds = oracle.quantize(A, bits, seed=3)
            plan = ShardPlan(m, batch, rank, world)
            order = list(np.random.default_rng(1).permutation(plan.steps)) if shuffled else None
            res[name] = _sharded_epoch(oracle, plan, ds, b, np.zeros(n, np.float32), 0.05, mb, gb, order, reg, rp, all_reduce)
        np.savez(f"{out}.{rank}.npz", **res)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_reproduce_the_single_rank_oracle_epoch(tmp_path):
    from oracle.build import build
    build()
    import oracle
    out = str(tmp_path / "s")
    port = 31500 + os.getpid() % 2000
    mp.spawn(_rank_main, args=(2, port, out), nprocs=2, join=True)
    r0, r1 = np.load(f"{out}.0.npz"), np.load(f"{out}.1.npz")
    for name, (m, n, bits, batch, mb, gb, shuffled, reg, rp) in CASES.items():
        A, b = _problem(m, n)
        ds = oracle.quantize(A, bits, seed=3)
        T = (m + batch - 1) // batch
        order = list(np.random.default_rng(1).permutation(T)) if shuffled else None
        want, _ = oracle.sgd_epoch(ds, b, np.zeros(n, np.float32), batch, 0.05, model_bits=mb, grad_bits=gb, seed=11, epoch=2,
                                   batch_order=order, reg=reg, reg_param=rp)
        # the replicas are the same bits on both ranks: same sums, same draws
        assert np.array_equal(r0[name], r1[name]), name
        # and the single-rank epoch up to the rounding of the shares (fp32 per rank, one fp32 sum)
        assert np.allclose(r0[name], want, rtol=2e-5, atol=2e-6), (name, np.abs(r0[name] - want).max())
        assert np.abs(want).max() > 1e-2                                  # the epoch did move x


def test_partition_covers_every_row_once():
    for m, batch, world in [(203, 16, 2), (197, 16, 2), (64, 16, 4), (1000, 24, 8), (5, 8, 2)]:
        seen = np.zeros(m, int)
        for r in range(world):
            plan = ShardPlan(m, batch, r, world)
            for a, b in plan.row_spans():
                seen[a:b] += 1
            for t in range(plan.steps):
                a, b = plan.span(t)
                assert t * batch <= a <= b <= min(m, (t + 1) * batch) and b - a <= plan.local_batch
            assert plan.local_rows == sum(plan.count(t) for t in range(plan.steps))
        assert (seen == 1).all()
        for t in range((m + batch - 1) // batch):
            assert abs(sum(ShardPlan(m, batch, r, world).weight(t) for r in range(world)) - 1.0) < 1e-12


def test_partition_refuses_what_it_cannot_split():
    with pytest.raises(ValueError):
        ShardPlan(100, 10, 0, 4)
    with pytest.raises(ValueError):
        ShardPlan(100, 16, 2, 2)
    with pytest.raises(ValueError):
        run_steps(ShardPlan(100, 16, 0, 2), None, None, None, order=[0, 1])
