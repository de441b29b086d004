"""Parity of the two extensions around the compression step -- the optimiser tail (Nesterov momentum) fused into
the kernels that produce the averaged gradient, and the batch-size mode of the controller -- against the CPU
oracle, through the C-ABI."""
import numpy as np
import pytest
import torch

from oracle import accordion_oracle as orc
from paper_2010_16248_b200 import binding, workloads as wl
from tests import helpers as H
from tests.test_gpu_parity import _random_inputs, _table_mixed

pytestmark = pytest.mark.gpu

TAIL_TOL = 1e-5  # fp32 fused multiply-adds against the fp64 oracle, one step from identical fp32 inputs


def _bits(t):
    return t.detach().cpu().numpy().view(np.uint32)


def _hyper(lr, mu, wd):
    return torch.tensor([lr, mu, wd], dtype=torch.float32, device="cuda")


def _check_tail_against_oracle(table, d, x0, u0, x1, u1, lr, mu, wd, tol=TAIL_TOL):
    layers = H.layers_of(table)
    ox, ou = orc.sgd_nesterov(x0.cpu().numpy(), u0.cpu().numpy(), d.cpu().numpy(), layers, lr, mu, wd)
    xh, uh = x1.cpu().numpy(), u1.cpu().numpy()
    covered = np.zeros(table.stride, bool)
    for (off, rows, cols, kind) in layers:
        sl = slice(off, off + rows * cols)
        covered[sl] = True
        assert H.rel_err(xh[sl], ox[sl]) <= tol
        assert H.rel_err(uh[sl], ou[sl]) <= tol
    # padding between layers is never touched
    assert np.array_equal(_bits(x1)[~covered], _bits(x0)[~covered])
    assert np.array_equal(_bits(u1)[~covered], _bits(u0)[~covered])


@pytest.mark.parametrize("wd", [0.0, 5e-4])
def test_sgd_nesterov_matches_oracle(wd):
    table = _table_mixed()
    ctx = binding.Context(table, 1)
    g = torch.Generator(device="cuda").manual_seed(7)
    x = torch.randn(table.stride, generator=g, device="cuda")
    u = torch.zeros(table.stride, device="cuda")
    hyper = _hyper(0.1, 0.9, wd)
    for step in range(3):
        d = torch.randn(table.stride, generator=g, device="cuda") * 0.3
        x0, u0 = x.clone(), u.clone()
        ctx.acc_sgd_nesterov(d, x, u, hyper)
        torch.cuda.synchronize()
        _check_tail_against_oracle(table, d, x0, u0, x, u, 0.1, 0.9, wd)
        hyper[0] *= 0.5  # the kernels read the learning rate from device memory
        x0, u0 = x.clone(), u.clone()
        ctx.acc_sgd_nesterov(d, x, u, hyper)
        torch.cuda.synchronize()
        _check_tail_against_oracle(table, d, x0, u0, x, u, float(hyper[0]), 0.9, wd)
        hyper[0] *= 2.0
    assert ctx.last_launch_count() == 1


@pytest.mark.parametrize("flags", [0, binding.ACC_FLAG_LAZY_RESIDUAL, binding.ACC_FLAG_PIPELINE_ALWAYS])
def test_powersgd_step_with_fused_tail(flags):
    """The fused step changes nothing but params / mom, gives the bits of plain step + stand-alone tail, and the
    parameters follow the oracle's compression step followed by the oracle's optimiser step."""
    table = _table_mixed()
    W, rl, rh = 3, 3, 1
    plain = binding.Context(table, W, rank_low=rl, rank_high=rh, flags=flags)
    fused = binding.Context(table, W, rank_low=rl, rank_high=rh, flags=flags)
    level = torch.tensor([(l * 5 + 1) % 3 != 0 for l in range(table.n_layers)], dtype=torch.uint8, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(11)
    x_a = torch.randn(table.stride, generator=g, device="cuda")
    x_b = x_a.clone()
    u_a, u_b = torch.zeros_like(x_a), torch.zeros_like(x_a)
    hyper = _hyper(0.05, 0.9, 1e-4)
    _, err_a = _random_inputs(table, W, 3)
    err_b = err_a.clone()
    q_a = plain.new_q(wl.initial_q(table, 4, seed=2))
    q_b = q_a.clone()
    p_a, p_b = plain.new_p(), fused.new_p()
    out_a, out_b = torch.zeros(table.stride, device="cuda"), torch.zeros(table.stride, device="cuda")
    delta_a, delta_b = torch.zeros(table.stride, device="cuda"), torch.zeros(table.stride, device="cuda")
    for it in range(3):
        grads, _ = _random_inputs(table, W, 40 + it)
        x0, u0 = x_b.clone(), u_b.clone()
        plain.acc_powersgd_step(grads, err_a, q_a, p_a, level, out_a, delta_a)
        plain.acc_sgd_nesterov(out_a, x_a, u_a, hyper)
        fused.acc_powersgd_step_sgd(grads, err_b, q_b, p_b, level, out_b, delta_b, x_b, u_b, hyper)
        torch.cuda.synchronize()
        for a, b in ((out_a, out_b), (err_a, err_b), (q_a, q_b), (p_a, p_b), (delta_a, delta_b), (x_a, x_b),
                     (u_a, u_b)):
            assert np.array_equal(_bits(a), _bits(b))
        # out was checked against the oracle by the plain-step tests; the tail is checked on top of it here
        _check_tail_against_oracle(table, out_b, x0, u0, x_b, u_b, 0.05, 0.9, 1e-4)
    assert fused.last_launch_count() == 6  # the plain step's five kernels + the tail of the VECTOR layers
    assert fused.acc_device_status() == 0


def test_powersgd_fused_tail_end_to_end_against_oracle():
    """Oracle compression step followed by the oracle's optimiser step, from the same inputs, two iterations."""
    table = _table_mixed()
    W, rl, rh = 2, 2, 1
    ctx = binding.Context(table, W, rank_low=rl, rank_high=rh)
    layers = H.layers_of(table)
    level = torch.ones(table.n_layers, dtype=torch.uint8, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(13)
    x = torch.randn(table.stride, generator=g, device="cuda")
    u = torch.zeros_like(x)
    hyper = _hyper(0.1, 0.9, 0.0)
    _, err = _random_inputs(table, W, 5)
    q = ctx.new_q(wl.initial_q(table, rl, seed=4))
    p = ctx.new_p()
    out = torch.zeros(table.stride, device="cuda")
    for it in range(2):
        grads, _ = _random_inputs(table, W, 60 + it)
        e0, q0, x0, u0 = err.clone(), q.clone(), x.clone(), u.clone()
        ctx.acc_powersgd_step_sgd(grads, err, q, p, level, out, None, x, u, hyper)
        torch.cuda.synchronize()
        o_out, _, _, _ = orc.powersgd_step(grads.cpu().numpy(), e0.cpu().numpy(), H.q_list_from_buffer(ctx, q0, rl),
                                           level.cpu().numpy(), layers, rl, rh, 1e-8)
        ox, ou = orc.sgd_nesterov(x0.cpu().numpy(), u0.cpu().numpy(), o_out, layers, 0.1, 0.9, 0.0)
        for (off, rows, cols, kind) in layers:
            sl = slice(off, off + rows * cols)
            assert H.rel_err(x.cpu().numpy()[sl], ox[sl]) <= H.REL_TOL
            assert H.rel_err(u.cpu().numpy()[sl], ou[sl], 1e-6 * np.linalg.norm(ou[sl]) + 1e-12) <= H.REL_TOL


@pytest.mark.parametrize("pipeline", [binding.ACC_FLAG_PIPELINE_NEVER, binding.ACC_FLAG_PIPELINE_ALWAYS])
def test_topk_step_with_fused_tail(pipeline):
    table = _table_mixed()
    W = 3
    plain = binding.Context(table, W, topk_low_bp=1000, topk_high_bp=100, flags=pipeline)
    fused = binding.Context(table, W, topk_low_bp=1000, topk_high_bp=100, flags=pipeline)
    layers = H.layers_of(table)
    level = torch.tensor([(l * 5 + 1) % 3 != 0 for l in range(table.n_layers)], dtype=torch.uint8, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(17)
    x_a = torch.randn(table.stride, generator=g, device="cuda")
    x_b = x_a.clone()
    u_a, u_b = torch.zeros_like(x_a), torch.zeros_like(x_a)
    hyper = _hyper(0.05, 0.9, 0.0)
    _, err_a = _random_inputs(table, W, 3)
    err_b = err_a.clone()
    va, ia, ca = plain.new_topk_buffers()
    vb, ib, cb = fused.new_topk_buffers()
    out_a, out_b = torch.zeros(table.stride, device="cuda"), torch.zeros(table.stride, device="cuda")
    for it in range(3):
        grads, _ = _random_inputs(table, W, 80 + it)
        e0, x0, u0 = err_b.clone(), x_b.clone(), u_b.clone()
        plain.acc_topk_step(grads, err_a, level, va, ia, ca, out_a)
        plain.acc_sgd_nesterov(out_a, x_a, u_a, hyper)
        fused.acc_topk_step_sgd(grads, err_b, level, vb, ib, cb, out_b, None, x_b, u_b, hyper)
        torch.cuda.synchronize()
        for a, b in ((out_a, out_b), (err_a, err_b), (ca, cb), (x_a, x_b), (u_a, u_b)):
            assert np.array_equal(_bits(a), _bits(b))
        H.check_topk_against_oracle(fused, table, grads, e0, level, vb, ib, cb, out_b, err_b, 1000, 100)
        _, _, _, o_out, _ = orc.topk_step(grads.cpu().numpy(), e0.cpu().numpy(), level.cpu().numpy(), layers, 1000, 100)
        ox, ou = orc.sgd_nesterov(x0.cpu().numpy(), u0.cpu().numpy(), o_out, layers, 0.05, 0.9, 0.0)
        for (off, rows, cols, kind) in layers:
            sl = slice(off, off + rows * cols)
            assert H.rel_err(x_b.cpu().numpy()[sl], ox[sl]) <= TAIL_TOL
            assert H.rel_err(u_b.cpu().numpy()[sl], ou[sl], 1e-12) <= TAIL_TOL
    assert fused.last_launch_count() == 14  # as many as the plain step: the tail rides in its last kernel


def test_tail_arguments_are_checked():
    table = _table_mixed()
    ctx = binding.Context(table, 2)
    grads, err = _random_inputs(table, 2, 1)
    q, p = ctx.new_q(wl.initial_q(table, 2, seed=1)), ctx.new_p()
    level = torch.ones(table.n_layers, dtype=torch.uint8, device="cuda")
    out = torch.zeros(table.stride, device="cuda")
    x = torch.zeros(table.stride + 4, device="cuda")
    u = torch.zeros(table.stride, device="cuda")
    hyper = _hyper(0.1, 0.9, 0.0)
    with pytest.raises(binding.AccError) as ei:
        ctx.acc_powersgd_step_sgd(grads, err, q, p, level, out, None, None, u, hyper)
    assert ei.value.status == 1  # ACC_EINVAL
    with pytest.raises(binding.AccError) as ei:
        ctx.acc_sgd_nesterov(out, x[1:table.stride + 1], u, hyper)  # 4-byte offset: not 16-byte aligned
    assert ei.value.status == 2  # ACC_EALIGN
    acc = torch.zeros(2, table.stride, device="cuda")
    with pytest.raises(binding.AccError):
        ctx.acc_batch_average(acc, 0, out)
    n2 = torch.zeros(table.n_layers, dtype=torch.float64, device="cuda")
    prev = torch.full((1,), -1.0, dtype=torch.float64, device="cuda")
    batch = torch.zeros(1, dtype=torch.int32, device="cuda")
    scale = torch.zeros(1, device="cuda")
    with pytest.raises(binding.AccError):
        ctx.acc_detect_batch(n2, prev, 0.1, 0.1, 512, 256, batch, scale)


# ------------------------------------------------------------------ batch-size mode
@pytest.mark.parametrize("W,n_accum", [(1, 1), (3, 4)])
def test_batch_accumulate_and_average_match_oracle(W, n_accum):
    table = _table_mixed()
    ctx = binding.Context(table, W)
    layers = H.layers_of(table)
    acc = torch.full((W, table.stride), 123.0, device="cuda")  # stale: the first micro-batch overwrites it
    delta = torch.zeros(table.stride, device="cuda")
    o_acc = np.zeros((W, table.stride))
    o_delta = np.zeros(table.stride)
    for j in range(n_accum):
        grads, _ = _random_inputs(table, W, 200 + j)
        ctx.acc_batch_accumulate(grads, acc, delta, first=(j == 0))
        o_acc = orc.batch_accumulate(o_acc, grads.cpu().numpy(), layers, first=(j == 0))
        o_delta = orc.accumulate(o_delta, grads[0].cpu().numpy(), layers)
    out = torch.zeros(table.stride, device="cuda")
    x = torch.randn(table.stride, device="cuda")
    u = torch.randn(table.stride, device="cuda") * 0.1
    x0, u0 = x.clone(), u.clone()
    hyper = _hyper(0.4, 0.9, 0.0)
    ctx.acc_batch_average(acc, n_accum, out, x, u, hyper)
    torch.cuda.synchronize()
    o_out = orc.batch_average(o_acc, n_accum, layers)
    for (off, rows, cols, kind) in layers:
        sl = slice(off, off + rows * cols)
        assert H.rel_err(acc.cpu().numpy()[:, sl], o_acc[:, sl]) <= 1e-6
        assert H.rel_err(delta.cpu().numpy()[sl], o_delta[sl]) <= 1e-6
        assert H.rel_err(out.cpu().numpy()[sl], o_out[sl]) <= 1e-6
    _check_tail_against_oracle(table, out, x0, u0, x, u, 0.4, 0.9, 0.0)
    # without the tail the same out, bit for bit, and params untouched
    out2 = torch.zeros(table.stride, device="cuda")
    ctx.acc_batch_average(acc, n_accum, out2)
    torch.cuda.synchronize()
    assert np.array_equal(_bits(out), _bits(out2))
    assert ctx.last_launch_count() == 1


def test_detect_batch_truth_table_and_schedule():
    table = wl.make_table([("a", (4, 4)), ("b", (9,)), ("c", (2, 8))])
    ctx = binding.Context(table, 1, eta=0.5)
    L = table.n_layers
    dev = dict(device="cuda")
    # whole-model norm 5 from exactly representable layer norms (9 + 16 + 0)
    n2 = torch.tensor([9.0, 16.0, 0.0], dtype=torch.float64, **dev)
    cases = [(10.0, 0.1, 0.1, 512), (6.0, 0.1, 0.1, 512), (4.0, 0.1, 0.1, 512), (2.0, 0.1, 0.1, 512),
             (6.0, 0.1, 0.01, 512), (10.0, 0.1, 0.1, 4096), (6.0, 0.1, 0.01, 4096), (0.0, 0.1, 0.1, 512),
             (-1.0, 0.1, 0.1, 512)]
    for a, lc, ln, bc in cases:
        prev = torch.tensor([a * a if a >= 0 else -1.0], dtype=torch.float64, **dev)
        batch = torch.tensor([bc], dtype=torch.int32, **dev)
        scale = torch.zeros(1, **dev)
        delta = torch.ones(table.stride, **dev)
        ctx.acc_detect_batch(n2, prev, lc, ln, 512, 4096, batch, scale, delta)
        torch.cuda.synchronize()
        wb, ws, wp = orc.detect_batch(n2.cpu().numpy(), a * a if a >= 0 else -1.0, lc, ln, 0.5, bc, 512, 4096)
        assert (int(batch[0]), float(scale[0]), float(prev[0])) == (wb, ws, wp), (a, lc, ln, bc)
        assert float(delta.abs().sum()) == 0.0  # new window
    # a schedule: the accumulated gradient shrinks 4x (critical), stays flat (not critical: grow), jumps (critical,
    # but the batch size never decreases)
    rng = np.random.default_rng(0)
    prev = torch.full((1,), -1.0, dtype=torch.float64, **dev)
    batch = torch.tensor([128], dtype=torch.int32, **dev)
    scale = torch.zeros(1, **dev)
    o_prev, o_batch = -1.0, 128
    n2_dev = torch.zeros(L, dtype=torch.float64, **dev)
    delta = torch.zeros(table.stride, **dev)
    got, want = [], []
    for win, amp in enumerate([1.0, 0.25, 0.25, 0.25, 4.0]):
        dl = torch.tensor(rng.standard_normal(table.stride).astype(np.float32) * amp, **dev)
        delta.copy_(dl)
        ctx.acc_layer_norms(delta, 1, n2_dev)
        ctx.acc_detect_batch(n2_dev, prev, 0.1, 0.1, 128, 1024, batch, scale, delta)
        torch.cuda.synchronize()
        o_n2 = orc.layer_norms2(dl.cpu().numpy(), H.layers_of(table))
        o_batch, o_scale, o_prev = orc.detect_batch(o_n2, o_prev, 0.1, 0.1, 0.5, o_batch, 128, 1024)
        got.append((int(batch[0]), float(scale[0])))
        want.append((o_batch, o_scale))
        assert abs(float(prev[0]) - o_prev) <= 1e-12 * o_prev
    assert got == want
    assert [b for b, _ in got] == [128, 128, 1024, 1024, 1024]


def test_batch_size_step_loop_matches_oracle():
    """The sequencing class: B_low = 2 micro-batches until the controller lets the batch grow to 4; the
    parameters follow the oracle through both phases."""
    from paper_2010_16248_b200 import pipeline
    table = _table_mixed()
    layers = H.layers_of(table)
    W = 2
    x = torch.randn(table.stride, device="cuda")
    ox, ou = x.cpu().numpy().astype(np.float64), np.zeros(table.stride)
    bs = pipeline.BatchSizeStep(table, W, b_low=64, b_high=128, micro_batch=32, eta=0.5,
                                optimizer={"params": x, "lr": 0.1, "momentum": 0.9})
    batch, o_batch, o_prev = 64, 64, -1.0
    o_delta = np.zeros(table.stride)
    seed = 300
    for window in range(3):
        for big_step in range(2):
            n_accum = batch // 32
            o_acc = np.zeros((W, table.stride))
            for j in range(n_accum):
                grads, _ = _random_inputs(table, W, seed)
                seed += 1
                bs.micro_step(grads)
                o_acc = orc.batch_accumulate(o_acc, grads.cpu().numpy(), layers, first=(j == 0))
                o_delta = orc.accumulate(o_delta, grads[0].cpu().numpy(), layers)
            out = bs.apply()
            o_out = orc.batch_average(o_acc, n_accum, layers)
            ox, ou = orc.sgd_nesterov(ox, ou, o_out, layers, 0.1, 0.9, 0.0)
            torch.cuda.synchronize()
            for (off, rows, cols, kind) in layers:
                sl = slice(off, off + rows * cols)
                assert H.rel_err(out.cpu().numpy()[sl], o_out[sl]) <= 1e-6
                assert H.rel_err(x.cpu().numpy()[sl], ox[sl]) <= H.REL_TOL
        batch = bs.check(0.1, 0.1)
        o_batch, o_scale, o_prev = orc.detect_batch(orc.layer_norms2(o_delta, layers), o_prev, 0.1, 0.1, 0.5,
                                                    o_batch, 64, 128)
        o_delta[:] = 0.0
        assert batch == o_batch and float(bs.lr_scale[0]) == o_scale
    assert batch == 128  # the windows after the first look alike: not critical, the batch grew


def test_engine_with_tail_replays_as_graph_and_follows_the_learning_rate():
    from paper_2010_16248_b200 import pipeline
    table = _table_mixed()
    W = 2
    x_a = torch.randn(table.stride, device="cuda")
    x_b = x_a.clone()
    q0 = wl.initial_q(table, 2, seed=9)
    direct = pipeline.AccordionStep(table, W, ("powersgd",), check_every=2, q_init=q0, lazy_residual=True,
                                    optimizer={"params": x_a, "lr": 0.1})
    graph = pipeline.AccordionStep(table, W, ("powersgd",), check_every=2, q_init=q0, lazy_residual=True,
                                   optimizer={"params": x_b, "lr": 0.1})
    bufs = [_random_inputs(table, W, 500 + i)[0] for i in range(2)]
    graph.capture_graphs(bufs)
    for t in range(6):
        if t == 3:
            direct.set_lr(0.01)
            graph.set_lr(0.01)
        direct.step(bufs[t % 2])
        graph.step_graph(t % 2)
    torch.cuda.synchronize()
    assert np.array_equal(_bits(x_a), _bits(x_b))
    assert np.array_equal(_bits(direct.mom), _bits(graph.mom))
    assert not np.array_equal(_bits(x_a), _bits(bufs[0][0]))
