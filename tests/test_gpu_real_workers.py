"""The real-worker path (a context per GPU holding that GPU's workers, the compressed factors exchanged between
the kernels' phases) on ONE GPU: the ranks are host threads that step through `pipeline.DistributedStep` in
lockstep and meet in an in-process stand-in for the collectives (host barriers only: no kernel ever waits for
another).  Results are compared with the oracle over all workers and with the single-context step."""
import threading

import numpy as np
import pytest
import torch

from oracle import accordion_oracle as orc
from paper_2010_16248_b200 import binding, dist_util, pipeline, workloads as wl
from tests import helpers as H
from tests.test_gpu_parity import _random_inputs, _table_mixed

pytestmark = pytest.mark.gpu


def _bits(t):
    return t.detach().cpu().numpy().view(np.uint32 if t.dtype in (torch.float32, torch.int32) else np.uint8)


class ThreadExchange:
    """Collectives between host threads of one process: every rank deposits its tensor, all meet at a barrier,
    every rank combines the deposits in rank order (so all ranks get the same bits), all meet again."""

    class Shared:
        def __init__(self, world):
            self.world = world
            self.slots = [None] * world
            self.barrier = threading.Barrier(world)

    def __init__(self, shared, rank):
        self.sh, self.rank, self.world = shared, rank, shared.world

    def _deposit(self, t):
        # ranks may run their exchanges on streams of their own: the deposit must be complete before another
        # rank's thread reads it, and what a rank read must be consumed before the slot is overwritten
        self.sh.slots[self.rank] = t.clone()
        torch.cuda.current_stream().synchronize()

    def sum_(self, t):
        self._deposit(t)
        self.sh.barrier.wait()
        total = self.sh.slots[0].clone()
        for r in range(1, self.world):
            total += self.sh.slots[r]
        t.copy_(total)
        torch.cuda.current_stream().synchronize()
        self.sh.barrier.wait()
        return t

    def gather_into(self, out, t):
        self._deposit(t)
        self.sh.barrier.wait()
        out.copy_(torch.cat([s.reshape(-1) for s in self.sh.slots]))
        torch.cuda.current_stream().synchronize()
        self.sh.barrier.wait()
        return out


def _run_ranks(world, make_step, n_iters, grads_of):
    """Runs `world` rank threads for n_iters lockstep iterations; returns the per-rank step objects."""
    shared = ThreadExchange.Shared(world)
    steps, errors = [None] * world, []

    def main(rank):
        try:
            torch.cuda.set_device(0)
            st = make_step(ThreadExchange(shared, rank))
            steps[rank] = st
            for it in range(n_iters):
                st.step(grads_of(it, rank))
            torch.cuda.synchronize()
        except Exception as e:  # surface the failure in the main thread; release the others
            errors.append(e)
            shared.barrier.abort()

    threads = [threading.Thread(target=main, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(300)
    assert not errors, errors
    return steps


@pytest.mark.parametrize("lazy", [False, True])
def test_powersgd_two_ranks_match_oracle_over_all_workers(lazy):
    table = _table_mixed()
    layers = H.layers_of(table)
    world, n_local, rl, rh = 2, 2, 3, 1
    W = world * n_local
    q0 = wl.initial_q(table, rl, seed=21)
    n_iters = 4  # check_every = 2: the level array changes on the way
    batches = [_random_inputs(table, W, 700 + it)[0] * (1.0 if it < 2 else 0.2) for it in range(n_iters)]
    x0 = torch.randn(table.stride, device="cuda")
    params = [x0.clone() for _ in range(world)]

    def make_step(exchange):
        return pipeline.DistributedStep(table, n_local, "powersgd", rank_low=rl, rank_high=rh, check_every=2,
                                        decider=3, q_init=q0, lazy_residual=lazy, exchange=exchange,
                                        optimizer={"params": params[exchange.rank], "lr": 0.1})

    steps = _run_ranks(world, make_step, n_iters, lambda it, r: batches[it][r * n_local:(r + 1) * n_local].contiguous())
    a, b = steps
    assert a.owns_decider is False and b.owns_decider is True  # global worker 3 lives on rank 1
    for name in ("out", "q", "p_hat", "level", "norm2_prev"):
        ta, tb = getattr(a, name), getattr(b, name)
        assert torch.equal(ta, tb), name  # every rank ends with the same factors, output and levels
    assert torch.equal(params[0], params[1]) and torch.equal(a.mom, b.mom)

    # the oracle over all four workers, same schedule
    err = np.zeros((W, table.stride))
    q = [None if x is None else x.cpu().numpy().astype(np.float64) for x in q0]
    level = np.ones(table.n_layers, np.uint8)
    prev = -np.ones(table.n_layers)
    delta = np.zeros(table.stride)
    ox, ou = x0.cpu().numpy().astype(np.float64), np.zeros(table.stride)
    for it in range(n_iters):
        g = batches[it].cpu().numpy()
        delta = orc.accumulate(delta, g[3], layers)
        o_out, err, q, o_p = orc.powersgd_step(g, err, q, level, layers, rl, rh, 1e-8)
        ox, ou = orc.sgd_nesterov(ox, ou, o_out, layers, 0.1, 0.9, 0.0)
        if (it + 1) % 2 == 0:
            level, prev = orc.detect_regime(orc.layer_norms2(delta, layers), prev, 0.1, 0.1, 0.5)
            delta[:] = 0.0
    assert np.array_equal(a.level.cpu().numpy(), level)
    for st in steps:
        st.flush()  # lazy mode: materialise the error memories (a no-op in eager mode)
    torch.cuda.synchronize()
    err_gpu = torch.cat([a.err, b.err]).cpu().numpy()
    out_h, x_h = a.out.cpu().numpy(), params[0].cpu().numpy()
    tol = 5e-4  # four chained steps in fp32 against fp64 (one step: 1e-4)
    for l, (off, rows, cols, kind) in enumerate(layers):
        sl = slice(off, off + rows * cols)
        assert H.rel_err(out_h[sl], o_out[sl], 1e-6 * np.linalg.norm(o_out[sl]) + 1e-12) <= tol, l
        assert H.rel_err(x_h[sl], ox[sl]) <= tol, l
        if kind == orc.MATRIX:
            floor = 1e-6 * np.linalg.norm(err[:, sl])
            assert H.rel_err(err_gpu[:, sl], err[:, sl], floor) <= tol, l


@pytest.mark.parametrize("compressor", ["powersgd", "topk"])
@pytest.mark.parametrize("lazy", [False, True])
def test_layer_groups_with_overlapped_exchange_equal_the_unsplit_step(compressor, lazy):
    """The step cut into three layer groups, whose exchanges run on a communication stream beside the next group's
    first pass, against the same step with one group: two ranks of two workers, six iterations across level
    changes, the optimiser tail included.  A layer's arithmetic does not depend on how the layers are grouped, so
    every result must be the same bits."""
    table = wl.make_table([("c0", (64, 27)), ("b0", (64,)), ("c1", (128, 576)), ("b1", (128,)), ("c2", (300, 650)),
                           ("fc", (100, 512)), ("b2", (100,))])
    world, n_local, n_iters = 2, 2, 6
    W = world * n_local
    q0 = wl.initial_q(table, 2, seed=33)
    batches = [_random_inputs(table, W, 2100 + it)[0] * (1.0 if it < 3 else 0.3) for it in range(n_iters)]
    x0 = torch.randn(table.stride, device="cuda")
    results = []
    for groups in (1, 3):
        params = [x0.clone() for _ in range(world)]

        def make_step(exchange, groups=groups, params=params):
            return pipeline.DistributedStep(table, n_local, compressor, check_every=2, decider=1, q_init=q0,
                                            lazy_residual=lazy, exchange=exchange, groups=groups,
                                            extra_flags=binding.ACC_FLAG_PIPELINE_NEVER,
                                            optimizer={"params": params[exchange.rank], "lr": 0.05})
        steps = _run_ranks(world, make_step, n_iters,
                           lambda it, r: batches[it][r * n_local:(r + 1) * n_local].contiguous())
        for st in steps:
            st.flush()
        torch.cuda.synchronize()
        results.append((steps, params))
    (one, p_one), (many, p_many) = results
    assert len(many[0].parts) == 3 and len(one[0].parts) == 1
    assert sorted(l for p in many[0].parts for l in p.ids) == list(range(table.n_layers))
    for r in range(world):
        for name in ("out", "err", "level", "norm2_prev", "mom"):
            assert torch.equal(getattr(one[r], name), getattr(many[r], name)), (r, name)
        assert torch.equal(p_one[r], p_many[r])
        if compressor == "powersgd":  # the factors, layer by layer
            c1 = one[r].ctx
            for part in many[r].parts:
                for j, l in enumerate(part.ids):
                    if table.kind[l] != wl.MATRIX:
                        continue
                    n, m = int(table.rows[l]), int(table.cols[l])
                    qa = one[r].q[c1.q_row[l]:c1.q_row[l] + m]
                    qb = part.q[part.ctx.q_row[j]:part.ctx.q_row[j] + m]
                    pa = one[r].p_hat[c1.p_row[l]:c1.p_row[l] + n]
                    pb = part.p_hat[part.ctx.p_row[j]:part.ctx.p_row[j] + n]
                    assert torch.equal(qa, qb) and torch.equal(pa, pb), (r, l)
    assert torch.equal(many[0].out, many[1].out)


def test_powersgd_one_rank_phases_equal_the_fused_step():
    """world = 1: the three phases with the identity exchange against acc_powersgd_step (same context layout)."""
    table = _table_mixed()
    W, rl, rh = 3, 2, 1
    q0 = wl.initial_q(table, rl, seed=22)
    whole = pipeline.AccordionStep(table, W, ("powersgd",), rl, rh, check_every=2, q_init=q0)
    split = pipeline.DistributedStep(table, W, "powersgd", rank_low=rl, rank_high=rh, check_every=2, q_init=q0,
                                     exchange=dist_util.Exchange())
    for it in range(4):
        g, _ = _random_inputs(table, W, 800 + it)
        whole.step(g)
        split.step(g)
    torch.cuda.synchronize()
    assert torch.equal(whole.level, split.level)
    layers = H.layers_of(table)
    for (off, rows, cols, kind) in layers:
        sl = slice(off, off + rows * cols)
        assert H.rel_err(split.out.cpu().numpy()[sl], whole.out_psgd.cpu().numpy()[sl], 1e-12) <= 1e-5
        assert H.rel_err(split.err.cpu().numpy()[:, sl], whole.err_psgd.cpu().numpy()[:, sl], 1e-12) <= 1e-5


def test_topk_two_ranks_are_bit_identical_to_the_single_gpu_step():
    table = _table_mixed()
    world, n_local = 2, 2
    W = world * n_local
    n_iters = 4
    batches = [_random_inputs(table, W, 900 + it)[0] * (1.0 if it < 2 else 0.2) for it in range(n_iters)]
    x0 = torch.randn(table.stride, device="cuda")
    params = [x0.clone() for _ in range(world)]

    def make_step(exchange):
        return pipeline.DistributedStep(table, n_local, "topk", topk_low_bp=1000, topk_high_bp=100, check_every=2,
                                        decider=2, exchange=exchange,
                                        optimizer={"params": params[exchange.rank], "lr": 0.1})

    steps = _run_ranks(world, make_step, n_iters, lambda it, r: batches[it][r * n_local:(r + 1) * n_local].contiguous())
    a, b = steps
    single_params = x0.clone()
    single = pipeline.AccordionStep(table, W, ("topk",), topk_low_bp=1000, topk_high_bp=100, check_every=2, decider=2,
                                    optimizer={"params": single_params, "lr": 0.1})
    for it in range(n_iters):
        single.step(batches[it])
    torch.cuda.synchronize()
    assert torch.equal(a.out, b.out) and torch.equal(a.level, b.level)
    # MATRIX layers: the gathered sets are added in the single-GPU step's order, so the bits agree; VECTOR layers
    # are summed per GPU first ((g0+g1)+(g2+g3) instead of ((g0+g1)+g2)+g3): equal up to fp32 rounding
    for l, sl in table.slices():
        if table.kind[l] == wl.MATRIX:
            assert np.array_equal(_bits(a.out[sl]), _bits(single.out_topk[sl])), l
            assert np.array_equal(_bits(params[0][sl]), _bits(single_params[sl])), l
        else:
            assert H.rel_err(a.out[sl].cpu().numpy(), single.out_topk[sl].cpu().numpy()) <= 1e-6, l
            assert H.rel_err(params[0][sl].cpu().numpy(), single_params[sl].cpu().numpy()) <= 1e-6, l
    assert np.array_equal(_bits(a.level), _bits(single.level))
    assert np.array_equal(_bits(torch.cat([a.err, b.err])), _bits(single.err_topk))
    assert np.array_equal(_bits(a.vals_all), _bits(single.vals)) and torch.equal(a.idx_all, single.idx)
    assert torch.equal(a.counts_all, single.counts)
    assert torch.equal(params[0], params[1])
    # communication volume of one step: what the collectives carry
    assert a.bytes_exchanged_per_step() == 4 * (2 * n_local * a.ctx.capacity + n_local * table.n_layers
                                                + max(a.ctx.vec_floats, 4))


def test_one_rank_nccl_process_group():
    """The same class over a real NCCL process group of one rank (collectives are issued, trivially)."""
    import os
    import torch.distributed as dist
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", str(33000 + os.getpid() % 2000))
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        table = _table_mixed()
        st = pipeline.DistributedStep(table, 2, "powersgd", check_every=2)
        assert st.x.on and st.world == 1
        ref = pipeline.DistributedStep(table, 2, "powersgd", check_every=2, exchange=ThreadExchange(
            ThreadExchange.Shared(1), 0))
        for it in range(2):
            g, _ = _random_inputs(table, 2, 950 + it)
            st.step(g)
            ref.step(g)
        torch.cuda.synchronize()
        assert torch.equal(st.out, ref.out) and torch.equal(st.q, ref.q)
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("shapes", [[("w", (40, 30))], [("b", (100,))], [("w0", (9, 700)), ("b", (5,)), ("w1", (700, 9))]])
@pytest.mark.parametrize("compressor", ["powersgd", "topk"])
def test_degenerate_tables_two_ranks(shapes, compressor):
    """Tables without VECTOR layers, without MATRIX layers, and with very flat / very tall matrices: two ranks of
    one worker each against the single-context step over both workers."""
    table = wl.make_table(shapes)
    world, n_local = 2, 1
    q0 = wl.initial_q(table, 2, seed=5)
    batches = [_random_inputs(table, world, 1300 + it)[0] for it in range(3)]

    def make_step(exchange):
        return pipeline.DistributedStep(table, n_local, compressor, check_every=2, q_init=q0, exchange=exchange)

    steps = _run_ranks(world, make_step, 3, lambda it, r: batches[it][r:r + 1].contiguous())
    single = pipeline.AccordionStep(table, world, (compressor,), check_every=2, q_init=q0)
    for it in range(3):
        single.step(batches[it])
    torch.cuda.synchronize()
    ref = single.out_psgd if compressor == "powersgd" else single.out_topk
    assert torch.equal(steps[0].out, steps[1].out) and torch.equal(steps[0].level, single.level)
    for l, sl in table.slices():
        got, want = steps[0].out[sl].cpu().numpy(), ref[sl].cpu().numpy()
        assert H.rel_err(got, want, 1e-7 * np.linalg.norm(want) + 1e-12) <= 1e-4, (l, compressor)


def test_topk_two_ranks_lazy_residual_equals_eager():
    table = _table_mixed()
    world, n_local, n_iters = 2, 2, 4
    batches = [_random_inputs(table, world * n_local, 1500 + it)[0] for it in range(n_iters)]
    results = []
    for lazy in (False, True):
        def make_step(exchange, lazy=lazy):
            return pipeline.DistributedStep(table, n_local, "topk", check_every=2, decider=1, lazy_residual=lazy,
                                            exchange=exchange)
        steps = _run_ranks(world, make_step, n_iters,
                           lambda it, r: batches[it][r * n_local:(r + 1) * n_local].contiguous())
        for st in steps:
            st.flush()
        torch.cuda.synchronize()
        results.append(steps)
    for a, b in zip(*results):
        for name in ("out", "err", "vals_all", "idx_all", "counts_all", "level"):
            assert torch.equal(getattr(a, name), getattr(b, name)), name
