"""CPU tests of the input generators (structure and determinism of the synthetic gradients) and of the
multi-process plumbing of the benchmark (world_size 2, gloo)."""
import os

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2010_16248_b200 import dist_util, workloads as wl


def test_tables_are_aligned_and_disjoint():
    for c in range(1, 6):
        t = wl.workload(c, scale=8).table
        assert np.all(t.offset % 4 == 0) and t.stride % 64 == 0
        ends = t.offset + t.sizes
        assert np.all(t.offset[1:] >= ends[:-1]) and ends[-1] <= t.stride


def test_streams_are_deterministic_and_padding_is_zero():
    for c in (1, 2, 3, 5):
        w = wl.workload(c, scale=8)
        a = wl.GradientStream(w).grads(7)
        b = wl.GradientStream(w).grads(7)
        assert torch.equal(a, b)
        assert not torch.equal(a, wl.GradientStream(w).grads(8))
        mask = torch.ones(w.table.stride, dtype=torch.bool)
        for l, sl in w.table.slices():
            mask[sl] = False
        assert float(a[:, mask].abs().max()) == 0.0 if mask.any() else True
        assert a.shape == (w.n_workers, w.table.stride) and a.dtype == torch.float32


def test_scale_jumps_double_the_norm():
    w = wl.workload(2, scale=8)
    s = wl.GradientStream(w)
    n99, n100 = s.grads(99).norm().item(), s.grads(100).norm().item()
    assert 1.8 < n100 / n99 < 2.2
    assert w.amplitude(0) == 2.0 and w.amplitude(100) == 4.0 and w.amplitude(150) == 8.0


def test_topk_workload_has_exact_ties_and_outliers():
    w = wl.workload(3, scale=4)
    g = wl.GradientStream(w).grads(0)
    l = int(np.argmax(w.table.sizes))
    off, size = int(w.table.offset[l]), int(w.table.sizes[l])
    x = g[0, off:off + size].abs().numpy()
    uniq = np.unique(x)
    assert size - len(uniq) >= size // 1500          # ~0.1 % of the coordinates duplicate a magnitude
    assert (x > 6 * np.median(x)).mean() > 0.01     # heavy-tailed support carrying the mean


def test_lstm_encoder_gradient_is_row_sparse():
    w = wl.workload(5, scale=16)
    g = wl.GradientStream(w).grads(3)
    l = w.table.names.index("encoder.weight")
    off, n, m = int(w.table.offset[l]), int(w.table.rows[l]), int(w.table.cols[l])
    for wk in (0, w.n_workers - 1):
        rows = g[wk, off:off + n * m].view(n, m)
        nz = int((rows.abs().sum(1) > 0).sum())
        assert nz == max(1, n * 2 // 100)
    assert not torch.equal(g[0, off:off + n * m], g[1, off:off + n * m])


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = dist_util.max_over_ranks(10.0 + 5.0 * rank)
        w = wl.workload(1, scale=8)
        g = wl.GradientStream(w).grads(dist_util.replica_seed_offset(rank))
        sums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(sums, g.double().sum().reshape(1))
        dist.barrier()
        out[rank] = (ms, [float(x) for x in sums])
    finally:
        dist.destroy_process_group()


def test_two_rank_replicas_gloo():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Manager().dict()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    assert out[0][0] == out[1][0] == 15.0                       # slowest rank decides
    assert out[0][1] == out[1][1] and out[0][1][0] != out[0][1][1]  # ranks drew different batches
    # whole-job throughput: both ranks' units over the slowest rank's time
    assert dist_util.whole_job_throughput(100.0, 15.0, world) == pytest.approx(2 * 100.0 / 0.015)
    assert dist_util.max_over_ranks(3.0) == 3.0                 # no process group: identity


def test_layer_groups_partition_the_table_and_keep_the_offsets():
    """Host logic of the grouped real-worker step: contiguous groups that cover every layer once, about equal in
    size, and sub-tables that keep every layer at its place in the flat buffer."""
    from paper_2010_16248_b200 import pipeline
    for config, n_groups in ((2, 4), (4, 5), (5, 3), (1, 3)):
        t = wl.workload(config, scale=4).table
        groups = pipeline._layer_groups(t, n_groups)
        assert [l for g in groups for l in g] == list(range(t.n_layers))
        assert len(groups) == min(n_groups, t.n_layers) and all(len(g) >= 1 for g in groups)
        for g in groups:
            sub = pipeline._sub_table(t, g)
            assert sub.stride == t.stride and sub.names == [t.names[l] for l in g]
            assert np.array_equal(sub.offset, t.offset[g]) and np.array_equal(sub.rows, t.rows[g])
            assert np.array_equal(sub.cols, t.cols[g]) and np.array_equal(sub.kind, t.kind[g])
    t = wl.workload(5).table  # two huge layers and small ones between them: one group each side of the middle
    sizes = [sum(int(t.sizes[l]) for l in g) for g in pipeline._layer_groups(t, 3)]
    assert max(sizes) < 0.45 * t.n_params


def _real_worker_rank_main(rank, world, port, out):
    """Two ranks with two workers each: the exchange helper over gloo, and the algebra of the real-worker split
    of the PowerSGD step (local P rows summed over ranks, Gram-Schmidt, local Q' rows summed) against the
    oracle's step over all four workers."""
    from oracle import accordion_oracle as orc
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        x = dist_util.Exchange()
        t = torch.tensor([rank + 1.0, 2.0])
        x.sum_(t)
        gathered = torch.zeros(world * 3, dtype=torch.int32)
        x.gather_into(gathered, torch.tensor([rank, 10 * rank, 7], dtype=torch.int32))
        # the split step in numpy, exchanged through the real collectives
        n, m, r, n_local = 12, 9, 2, 2
        rng = np.random.default_rng(5)
        g = rng.standard_normal((world * n_local, n * m)).astype(np.float32)
        e = (0.3 * rng.standard_normal((world * n_local, n * m))).astype(np.float32)
        q0 = rng.standard_normal((m, r)).astype(np.float32)
        mine = slice(rank * n_local, (rank + 1) * n_local)
        mbar = (g[mine].astype(np.float64) + e[mine].astype(np.float64)).mean(axis=0).reshape(n, m)
        x1 = torch.from_numpy(mbar @ q0.astype(np.float64))
        x.sum_(x1)
        p_hat = orc.gram_schmidt(x1.numpy() / world, 1e-8)
        x2 = torch.from_numpy(mbar.T @ p_hat)
        x.sum_(x2)
        q_new = x2.numpy() / world
        layers = [(0, n, m, orc.MATRIX)]
        o_out, _, o_q, o_p = orc.powersgd_step(g, e, [q0], np.ones(1, np.uint8), layers, r, r)
        ok = (np.allclose(p_hat, o_p[0], rtol=1e-10, atol=1e-12) and np.allclose(q_new, o_q[0], rtol=1e-10, atol=1e-12)
              and np.allclose((p_hat @ q_new.T).ravel(), o_out, rtol=1e-10, atol=1e-12))
        out[rank] = (t.tolist(), gathered.tolist(), x.world, x.rank, bool(ok))
    finally:
        dist.destroy_process_group()


def test_real_worker_exchange_and_split_algebra_gloo():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Manager().dict()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_real_worker_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(180)
        assert p.exitcode == 0
    for r in range(world):
        t, gathered, w, rk, ok = out[r]
        assert t == [3.0, 4.0] and gathered == [0, 0, 7, 1, 10, 7] and (w, rk) == (world, r)
        assert ok, "sum of local factor rows over ranks does not reproduce the all-worker step"
    x = dist_util.Exchange()  # no process group: one-rank identity
    a = torch.tensor([1.0, 2.0])
    assert x.world == 1 and torch.equal(x.sum_(a.clone()), a)
    assert torch.equal(x.gather_into(torch.zeros(2), a), a)
