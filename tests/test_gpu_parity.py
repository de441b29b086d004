"""Parity of the CUDA path (through the C-ABI) against the CPU oracle on the same seeded inputs.

Integer / index / byte results (TopK indices, counts, packed value bits, error-memory bits after
TopK, regime decisions) must be bit-exact; float results must match to a relative Frobenius error
of at most 1e-4 per layer."""
import numpy as np
import pytest
import torch

from oracle import accordion_oracle as orc
from paper_2010_16248_b200 import binding, pipeline, workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _table_mixed():
    # several tiles per layer (tile = 8192 elements), ragged tails, rows that are not multiples of 4,
    # rows only 8-byte aligned (cols = 650), a tiny layer (27 columns), vectors in between
    return wl.make_table([
        ("conv1.weight", (64, 27)), ("bn1.weight", (64,)), ("bn1.bias", (64,)),
        ("lstm.weight", (37, 650)), ("b0", (13,)),
        ("conv2.weight", (128, 1152)), ("wide.weight", (9, 4608)), ("b1", (8200,)),
        ("fc.weight", (100, 512)), ("odd.weight", (33, 333)), ("few.weight", (5, 7)), ("thin.weight", (300, 6)),
    ])


def _random_inputs(table, W, seed, err_scale=0.5):
    g = torch.Generator(device="cuda").manual_seed(seed)
    grads = torch.zeros(W, table.stride, device="cuda")
    err = torch.zeros(W, table.stride, device="cuda")
    for l, sl in table.slices():
        scale = 10.0 ** (-(l % 4))
        grads[:, sl] = torch.randn(W, sl.stop - sl.start, generator=g, device="cuda") * scale
        if table.kind[l] == wl.MATRIX:
            err[:, sl] = torch.randn(W, sl.stop - sl.start, generator=g, device="cuda") * scale * err_scale
    return grads, err


# ------------------------------------------------------------------ error feedback, norms, detector
@pytest.mark.parametrize("W", [1, 3])
def test_error_feedback_bit_exact(W):
    table = _table_mixed()
    ctx = binding.Context(table, W)
    grads, err = _random_inputs(table, W, 1)
    delta = torch.randn(table.stride, device="cuda")
    e0, d0 = err.clone(), delta.clone()
    ctx.acc_error_feedback(grads, err, delta)
    torch.cuda.synchronize()
    M = orc.error_feedback(grads.cpu().numpy(), e0.cpu().numpy(), H.layers_of(table), fp32=True)
    err_h, d_h = err.cpu().numpy(), delta.cpu().numpy()
    g_h, d0_h = grads.cpu().numpy(), d0.cpu().numpy()
    for l, (off, r, c, kind) in enumerate(H.layers_of(table)):
        sl = slice(off, off + r * c)
        if kind == orc.MATRIX:
            assert np.array_equal(err_h[:, sl].view(np.uint32), M[:, sl].view(np.uint32))
        else:
            assert np.array_equal(err_h[:, sl], e0.cpu().numpy()[:, sl])
        assert np.array_equal(d_h[sl], d0_h[sl] + g_h[0, sl])  # one fp32 add per element
    # no delta: err only
    err2 = e0.clone()
    ctx.acc_error_feedback(grads, err2, None)
    torch.cuda.synchronize()
    assert torch.equal(err2, err)


def test_layer_norms_match_oracle():
    table = _table_mixed()
    W = 3
    ctx = binding.Context(table, W)
    grads, _ = _random_inputs(table, W, 2)
    n2 = torch.zeros(W * table.n_layers, dtype=torch.float64, device="cuda")
    ctx.acc_layer_norms(grads, W, n2)
    n2b = torch.zeros_like(n2)
    ctx.acc_layer_norms(grads, W, n2b)
    torch.cuda.synchronize()
    assert torch.equal(n2, n2b)  # bit-reproducible
    got = n2.cpu().numpy().reshape(W, -1)
    for w in range(W):
        want = orc.layer_norms2(grads[w].cpu().numpy(), H.layers_of(table))
        assert np.allclose(got[w], want, rtol=1e-12, atol=0)
    one = torch.zeros(table.n_layers, dtype=torch.float64, device="cuda")
    ctx.acc_layer_norms(grads[1], 1, one)
    torch.cuda.synchronize()
    assert np.array_equal(one.cpu().numpy(), got[1])


def test_layer_msdr_matches_oracle():
    """Mean-to-standard-deviation ratio per layer (the second detector statistic) against the oracle: random layers
    with a mean, a constant layer (+inf), an all-zero layer (0); the second moment must be the bits acc_layer_norms
    returns, so one pass over the accumulated gradient serves both detectors."""
    table = wl.make_table([("a", (300, 70)), ("v", (33,)), ("const", (16, 16)), ("zero", (8, 8)), ("big", (129, 1000))])
    W = 2
    ctx = binding.Context(table, W)
    g = torch.Generator(device="cuda").manual_seed(4)
    buf = torch.zeros(W, table.stride, device="cuda")
    for l, sl in table.slices():
        n = sl.stop - sl.start
        if table.names[l] == "const":
            buf[:, sl] = 0.375
        elif table.names[l] != "zero":
            buf[:, sl] = torch.randn(W, n, generator=g, device="cuda") * (0.5 + l) + 0.05 * (l + 1)
    L = table.n_layers
    mom = torch.zeros(2 * W * L, dtype=torch.float64, device="cuda")
    msdr = torch.zeros(W * L, dtype=torch.float64, device="cuda")
    n2 = torch.zeros(W * L, dtype=torch.float64, device="cuda")
    ctx.acc_layer_msdr(buf, W, mom, msdr)
    ctx.acc_layer_norms(buf, W, n2)
    torch.cuda.synchronize()
    mom_h, msdr_h = mom.cpu().numpy().reshape(W, L, 2), msdr.cpu().numpy().reshape(W, L)
    assert np.array_equal(mom_h[:, :, 1].ravel(), n2.cpu().numpy())
    for w in range(W):
        want, mean, std = orc.layer_msdr(buf[w].cpu().numpy(), H.layers_of(table))
        for l in range(L):
            size = float(table.sizes[l])
            assert abs(mom_h[w, l, 0] / size - mean[l]) <= 1e-12 * max(1.0, abs(mean[l]))
            if np.isinf(want[l]):
                assert np.isinf(msdr_h[w, l]) and msdr_h[w, l] > 0, table.names[l]
            else:
                assert abs(msdr_h[w, l] - want[l]) <= 1e-9 * max(want[l], 1e-30), (table.names[l], msdr_h[w, l], want[l])
    assert msdr_h[0, table.names.index("zero")] == 0.0


def test_detect_regime_truth_table_and_random():
    L = 300
    table = wl.make_table([(f"v{i}", (4,)) for i in range(L)])
    ctx = binding.Context(table, 1, eta=0.5)
    rng = np.random.default_rng(3)
    prev = rng.uniform(0.0, 4.0, L)
    curr = rng.uniform(0.0, 4.0, L)
    # exactly representable boundary cases (a, b) -> |a-b| vs 0.5 a
    cases = [(1.0, 0.5), (1.0, 1.5), (1.0, 0.75), (1.0, 1.25), (4.0, 1.0), (0.0, 0.0), (0.0, 3.0), (2.0, 1.0), (2.0, 3.0)]
    for i, (a, b) in enumerate(cases):
        prev[i], curr[i] = a * a, b * b
    prev[20:30] = -1.0  # no previous window
    for lr_next in (0.1, 0.01):
        p = torch.tensor(prev, device="cuda"); c = torch.tensor(curr, device="cuda")
        level = torch.full((L,), 7, dtype=torch.uint8, device="cuda")
        delta = torch.ones(table.stride, device="cuda")
        ctx.acc_detect_regime(c, p, 0.1, lr_next, level, delta)
        torch.cuda.synchronize()
        want, want_prev = orc.detect_regime(curr, prev, 0.1, lr_next, np.float32(0.5))
        assert np.array_equal(level.cpu().numpy(), want)
        assert np.array_equal(p.cpu().numpy(), want_prev)
        assert float(delta.abs().max()) == 0.0
    assert list(want[:9]) == [1] * 9  # lr decay: all low
    want, _ = orc.detect_regime(curr, prev, 0.1, 0.1, 0.5)
    assert list(want[:9]) == [1, 1, 0, 0, 1, 1, 1, 1, 1]


# ------------------------------------------------------------------ PowerSGD
@pytest.mark.parametrize("pipeline", [binding.ACC_FLAG_PIPELINE_NEVER, binding.ACC_FLAG_PIPELINE_ALWAYS])
@pytest.mark.parametrize("W,rank_low,rank_high", [(1, 2, 1), (2, 2, 1), (3, 3, 2), (4, 4, 1), (8, 4, 4), (5, 1, 1)])
def test_powersgd_step_matches_oracle(W, rank_low, rank_high, pipeline):
    """Both implementations of the first pass (direct, and persistent with bulk asynchronous copies) on a
    table with ragged tiles, odd row lengths and vectors."""
    table = _table_mixed()
    ctx = binding.Context(table, W, rank_low=rank_low, rank_high=rank_high, gs_eps=1e-8, flags=pipeline)
    grads, err = _random_inputs(table, W, 10 + W)
    q = ctx.new_q(wl.initial_q(table, 4, seed=W))  # ranks beyond rank_low hold values that must survive
    p = ctx.new_p()
    p.fill_(3.25)
    level = torch.tensor([(l * 7 + W) % 3 != 0 for l in range(table.n_layers)], dtype=torch.uint8, device="cuda")
    out = torch.full((table.stride,), float("nan"), device="cuda")
    delta = torch.zeros(table.stride, device="cuda")
    for it in range(3):  # three consecutive steps: warm start, memory carried over
        e0, q0 = err.clone(), q.clone()
        ctx.acc_powersgd_step(grads, err, q, p, level, out, delta)
        torch.cuda.synchronize()
        H.check_powersgd_against_oracle(ctx, table, grads, e0, q0, level, out, err, q, p, rank_low, rank_high, 1e-8)
        grads, _ = _random_inputs(table, W, 100 + it)
    assert ctx.last_launch_count() == 5
    assert ctx.acc_device_status() == 0


def test_powersgd_invariants_and_exact_recovery():
    table = wl.make_table([("a", (48, 650)), ("v", (10,)), ("b", (200, 96))])
    W, r = 4, 2
    ctx = binding.Context(table, W, rank_low=r, rank_high=1, gs_eps=0.0)
    rng = np.random.default_rng(5)
    grads = torch.zeros(W, table.stride, device="cuda")
    for l, sl in table.slices():
        if table.kind[l] == wl.MATRIX:
            n, m = int(table.rows[l]), int(table.cols[l])
            B = rng.integers(-4, 5, (n, r)).astype(np.float64) @ rng.integers(-4, 5, (r, m)).astype(np.float64)
            grads[:, sl] = torch.tensor(B.reshape(-1), dtype=torch.float32, device="cuda")
    err = torch.zeros_like(grads)
    q = ctx.new_q(wl.initial_q(table, r))
    p = ctx.new_p()
    level = torch.ones(table.n_layers, dtype=torch.uint8, device="cuda")
    out = torch.zeros(table.stride, device="cuda")
    ctx.acc_powersgd_step(grads, err, q, p, level, out)
    torch.cuda.synchronize()
    for l, sl in table.slices():
        if table.kind[l] != wl.MATRIX:
            continue
        M = grads[0, sl]
        assert float((out[sl] - M).norm() / M.norm()) < 1e-5           # rank-r input is recovered
        assert float(err[:, sl].norm() / M.norm()) < 1e-5
        n = int(table.rows[l])
        ph = p[ctx.p_row[l]:ctx.p_row[l] + n, :r].double()
        assert torch.allclose(ph.T @ ph, torch.eye(r, device="cuda", dtype=torch.float64), atol=1e-5)
    # error-feedback invariant A + e'_w = g_w + e_w on random data
    grads2, err2 = _random_inputs(table, W, 6)
    M = grads2 + err2
    ctx.acc_powersgd_step(grads2, err2, q, p, level, out)
    torch.cuda.synchronize()
    for l, sl in table.slices():
        if table.kind[l] == wl.MATRIX:
            for w in range(W):
                assert float((out[sl] + err2[w, sl] - M[w, sl]).norm() / M[w, sl].norm()) < 1e-6


# ------------------------------------------------------------------ TopK
@pytest.mark.parametrize("pipeline", [binding.ACC_FLAG_PIPELINE_NEVER, binding.ACC_FLAG_PIPELINE_ALWAYS])
@pytest.mark.parametrize("W,low_bp,high_bp", [(1, 1000, 100), (3, 1000, 100), (4, 2500, 200), (2, 10000, 9900), (2, 1, 1)])
def test_topk_step_bit_exact(W, low_bp, high_bp, pipeline):
    table = _table_mixed()
    ctx = binding.Context(table, W, topk_low_bp=low_bp, topk_high_bp=high_bp, flags=pipeline)
    grads, err = _random_inputs(table, W, 20 + W)
    level = torch.tensor([(l * 5 + W) % 2 for l in range(table.n_layers)], dtype=torch.uint8, device="cuda")
    vals, idx, counts = ctx.new_topk_buffers()
    out = torch.full((table.stride,), float("nan"), device="cuda")
    for it in range(3):  # memory carried over: kept entries are +0.0 in the next add
        e0 = err.clone()
        ctx.acc_topk_step(grads, err, level, vals, idx, counts, out)
        torch.cuda.synchronize()
        H.check_topk_against_oracle(ctx, table, grads, e0, level, vals, idx, counts, out, err, low_bp, high_bp)
        grads, _ = _random_inputs(table, W, 200 + it)
    assert ctx.last_launch_count() == 14
    assert ctx.acc_device_status() == 0


@pytest.mark.parametrize("pipeline", [binding.ACC_FLAG_PIPELINE_NEVER, binding.ACC_FLAG_PIPELINE_ALWAYS])
def test_topk_ties_zeros_and_degenerate_layers(pipeline):
    table = wl.make_table([
        ("ties", (40, 650)),       # many exact duplicates around the threshold
        ("zeros", (30, 1000)),     # all zero: keeps the k lowest indices
        ("sparse", (500, 64)),     # row-sparse: k exceeds the non-zeros, filled with zeros by index
        ("equal", (3, 4097)),      # all equal magnitude, mixed sign
        ("small", (2, 3)), ("v", (7,)),
        ("quant", (64, 640)),      # few distinct values: ties at every level of the radix select
    ])
    W = 3
    ctx = binding.Context(table, W, topk_low_bp=1000, topk_high_bp=100, flags=pipeline)
    g = torch.Generator(device="cuda").manual_seed(7)
    grads = torch.zeros(W, table.stride, device="cuda")
    sl = {table.names[l]: s for l, s in table.slices()}
    n = sl["ties"].stop - sl["ties"].start
    base = torch.randn(W, n, generator=g, device="cuda")
    dup = torch.randint(0, n, (W, n // 3), generator=g, device="cuda")
    src = torch.randint(0, n, (W, n // 3), generator=g, device="cuda")
    sign = torch.randint(0, 2, (W, n // 3), generator=g, device="cuda").float() * 2 - 1
    base.scatter_(1, dup, torch.gather(base, 1, src).abs() * sign)
    grads[:, sl["ties"]] = base
    rows = torch.randperm(500, generator=g, device="cuda")[:10]
    sp = torch.zeros(W, 500, 64, device="cuda")
    sp[:, rows] = torch.randn(W, 10, 64, generator=g, device="cuda")
    grads[:, sl["sparse"]] = sp.reshape(W, -1)
    ne = sl["equal"].stop - sl["equal"].start
    grads[:, sl["equal"]] = (torch.randint(0, 2, (W, ne), generator=g, device="cuda").float() * 2 - 1) * 0.375
    grads[:, sl["small"]] = torch.randn(W, 6, generator=g, device="cuda")
    grads[:, sl["v"]] = torch.randn(W, 7, generator=g, device="cuda")
    nq = sl["quant"].stop - sl["quant"].start
    grads[:, sl["quant"]] = torch.randint(-3, 4, (W, nq), generator=g, device="cuda").float() * 0.25
    err = torch.zeros_like(grads)
    err[:, sl["zeros"]] = -0.0
    for level_val in (1, 0):
        level = torch.full((table.n_layers,), level_val, dtype=torch.uint8, device="cuda")
        e = err.clone()
        vals, idx, counts = ctx.new_topk_buffers()
        out = torch.zeros(table.stride, device="cuda")
        ctx.acc_topk_step(grads, e, level, vals, idx, counts, out)
        torch.cuda.synchronize()
        H.check_topk_against_oracle(ctx, table, grads, err, level, vals, idx, counts, out, e, 1000, 100)


def test_topk_is_bit_reproducible():
    table = _table_mixed()
    W = 4
    ctx = binding.Context(table, W)
    grads, err = _random_inputs(table, W, 31)
    level = torch.ones(table.n_layers, dtype=torch.uint8, device="cuda")
    res = []
    for rep in range(2):
        e = err.clone()
        vals, idx, counts = ctx.new_topk_buffers()
        out = torch.zeros(table.stride, device="cuda")
        ctx.acc_topk_step(grads, e, level, vals, idx, counts, out)
        torch.cuda.synchronize()
        res.append((e, vals, idx, counts, out))
    for a, b in zip(res[0], res[1]):
        assert torch.equal(a, b)


# ------------------------------------------------------------------ argument checks (no kernels run)
def test_bad_arguments_are_rejected():
    table = _table_mixed()
    ctx = binding.Context(table, 2)
    grads, err = _random_inputs(table, 2, 1)
    roomy = torch.zeros(grads.numel() + 8, device="cuda")
    with pytest.raises(binding.AccError) as ei:
        ctx.acc_error_feedback(roomy[1:1 + grads.numel()], err)  # long enough, but 4 bytes off a 16-byte boundary
    assert ei.value.status == 2
    with pytest.raises(ValueError):
        ctx.acc_error_feedback(grads.view(-1)[:-4], err)           # too short for the layout: refused by the binding
    with pytest.raises(ValueError):
        ctx.acc_error_feedback(grads.cpu(), err)
    with pytest.raises(binding.AccError):
        binding.Context(table, 2, rank_low=5)
    with pytest.raises(binding.AccError):
        binding.Context(table, 2, topk_low_bp=50, topk_high_bp=100)


# ------------------------------------------------------------------ PowerSGD, lazy residual
@pytest.mark.parametrize("pipeline", [binding.ACC_FLAG_PIPELINE_NEVER, binding.ACC_FLAG_PIPELINE_ALWAYS])
@pytest.mark.parametrize("W,rank_low,rank_high", [(2, 2, 1), (8, 4, 1), (3, 3, 2)])
def test_powersgd_lazy_residual_is_bit_identical_to_eager(W, rank_low, rank_high, pipeline):
    """With ACC_FLAG_LAZY_RESIDUAL err holds M_w between steps; out, q and p_hat of every step and the
    flushed error memory must equal the eager mode's bit for bit, also when the level (rank) changes
    between steps; the eager mode itself is checked against the oracle above."""
    table = _table_mixed()
    eager = binding.Context(table, W, rank_low=rank_low, rank_high=rank_high, flags=pipeline)
    lazy = binding.Context(table, W, rank_low=rank_low, rank_high=rank_high,
                           flags=binding.ACC_FLAG_LAZY_RESIDUAL | pipeline)
    grads, err0 = _random_inputs(table, W, 40 + W)
    state = []
    for ctx in (eager, lazy):
        state.append(dict(err=err0.clone(), q=ctx.new_q(wl.initial_q(table, 4, seed=3)), p=ctx.new_p(),
                          out=torch.zeros(table.stride, device="cuda"), delta=torch.zeros(table.stride, device="cuda")))
    for it in range(4):
        level = torch.tensor([(l + it) % 2 for l in range(table.n_layers)], dtype=torch.uint8, device="cuda")
        for ctx, st in zip((eager, lazy), state):
            ctx.acc_powersgd_step(grads, st["err"], st["q"], st["p"], level, st["out"], st["delta"])
        torch.cuda.synchronize()
        for name in ("out", "q", "p", "delta"):
            assert torch.equal(state[0][name], state[1][name]), f"step {it}: {name} differs"
        grads, _ = _random_inputs(table, W, 300 + it)
    lazy.acc_powersgd_flush(state[1]["err"], state[1]["q"], state[1]["p"])
    torch.cuda.synchronize()
    assert torch.equal(state[0]["err"], state[1]["err"])
    # a second flush has nothing pending and changes nothing
    before = state[1]["err"].clone()
    lazy.acc_powersgd_flush(state[1]["err"], state[1]["q"], state[1]["p"])
    torch.cuda.synchronize()
    assert torch.equal(before, state[1]["err"])
    # and the run continues identically after a flush
    for ctx, st in zip((eager, lazy), state):
        ctx.acc_powersgd_step(grads, st["err"], st["q"], st["p"], level, st["out"], None)
    lazy.acc_powersgd_flush(state[1]["err"], state[1]["q"], state[1]["p"])
    torch.cuda.synchronize()
    for name in ("out", "q", "p", "err"):
        assert torch.equal(state[0][name], state[1][name]), name
    with pytest.raises(binding.AccError):
        eager.acc_powersgd_flush(state[0]["err"], state[0]["q"], state[0]["p"])


@pytest.mark.parametrize("pipeline", [binding.ACC_FLAG_PIPELINE_NEVER, binding.ACC_FLAG_PIPELINE_ALWAYS])
def test_topk_threshold_prediction_hits_and_misses(pipeline):
    """The step predicts the threshold's bucket from the previous step at the same level.  Sequence of
    gradient scales that makes the prediction hold (same scale), miss upwards (x10: exact list path),
    miss downwards (x0.1: the histogram below the predicted band was not counted, redo path) and switch
    level in between; every step must still match the oracle bit for bit."""
    table = _table_mixed()
    W = 2
    ctx = binding.Context(table, W, flags=pipeline)
    vals, idx, counts = ctx.new_topk_buffers()
    out = torch.zeros(table.stride, device="cuda")
    base, _ = _random_inputs(table, W, 77, err_scale=0.0)
    steps = [(1.0, 1), (1.0, 1), (0.1, 1), (0.1, 1), (10.0, 1), (10.0, 0), (10.0, 0), (0.5, 0), (0.5, 1), (0.5, 1)]
    for i, (scale, lv) in enumerate(steps):
        g = torch.Generator(device="cuda").manual_seed(500 + i)
        grads = (base + 0.05 * torch.randn(base.shape, generator=g, device="cuda") * (base != 0)) * scale
        err = torch.zeros_like(grads)
        level = torch.full((table.n_layers,), lv, dtype=torch.uint8, device="cuda")
        e0 = err.clone()
        ctx.acc_topk_step(grads, err, level, vals, idx, counts, out)
        torch.cuda.synchronize()
        H.check_topk_against_oracle(ctx, table, grads, e0, level, vals, idx, counts, out, err, 1000, 100)


def test_topk_every_selection_path_is_exercised():
    """All five selection paths give the same (oracle-checked) results; this run makes sure each of them is
    actually taken: dense (a bucket too fat for a list: a layer of equal magnitudes, and a layer of zeros with a few
    denormals among them), list (first step, no prediction), predicted list (same gradients again), staged entries
    (high compression level on a layer whose kept entries stand far above the rest) and zero fill (a layer with fewer
    non-zeros than k: every non-zero plus the first zeros; an all-zero layer)."""
    table = wl.make_table([("zeros", (64, 1024)), ("noise", (256, 1024)), ("spiky", (256, 1024)),
                           ("const", (40, 1000)), ("rowsparse", (300, 650)), ("denormal", (32, 1024))])
    W = 2
    ctx = binding.Context(table, W, topk_low_bp=1000, topk_high_bp=100)
    g = torch.Generator(device="cuda").manual_seed(9)
    grads = torch.zeros(W, table.stride, device="cuda")
    sl = {table.names[l]: s for l, s in table.slices()}
    grads[:, sl["noise"]] = torch.randn(W, 256 * 1024, generator=g, device="cuda")
    spiky = 1e-3 * torch.randn(W, 256 * 1024, generator=g, device="cuda")
    hot = torch.randperm(256 * 1024, generator=g, device="cuda")[:4000]
    spiky[:, hot] = 5.0 + torch.rand(W, 4000, generator=g, device="cuda")
    grads[:, sl["spiky"]] = spiky
    sign = torch.randint(0, 2, (W, 40 * 1000), generator=g, device="cuda").float() * 2 - 1
    grads[:, sl["const"]] = 0.75 * sign                       # one magnitude: everything ties at the threshold
    rs = torch.zeros(W, 300, 650, device="cuda")
    for w in range(W):                                        # 2 % of the rows non-zero, a negative zero among the rest
        rows = torch.randperm(300, generator=g, device="cuda")[:6]
        rs[w, rows] = torch.randn(6, 650, generator=g, device="cuda")
    rs[:, 7, 3] = -0.0
    grads[:, sl["rowsparse"]] = rs.reshape(W, -1)
    den = torch.zeros(W, 32 * 1024, device="cuda")
    den[:, 5::97] = 1e-41                                     # denormals share the lowest bucket with the zeros
    den[:, 11] = 3.0
    grads[:, sl["denormal"]] = den
    vals, idx, counts = ctx.new_topk_buffers()
    out = torch.zeros(table.stride, device="cuda")
    seen = set()
    names = [n for l, n in enumerate(table.names)]
    by_layer = {}
    for lv in (1, 1, 1, 0, 0, 0, 0):
        level = torch.full((table.n_layers,), lv, dtype=torch.uint8, device="cuda")
        err = torch.zeros_like(grads)
        ctx.acc_topk_step(grads, err, level, vals, idx, counts, out)
        torch.cuda.synchronize()
        H.check_topk_against_oracle(ctx, table, grads, torch.zeros_like(grads), level, vals, idx, counts, out, err,
                                    1000, 100)
        paths = ctx.acc_topk_last_paths()
        seen.update(int(p) for p in paths.ravel())
        for j, n in enumerate(names):
            by_layer.setdefault(n, set()).update(int(p) for p in paths[:, j])
    assert seen == {0, 1, 2, 3, 4}, seen
    assert by_layer["zeros"] == {4} and 4 in by_layer["rowsparse"]      # k = 10 % of 195000 > 3900 non-zeros
    assert by_layer["const"] == {0} and by_layer["denormal"] == {0}


def test_topk_zero_fill_with_error_feedback_lazy_and_eager():
    """A row-sparse layer over several steps with error feedback: at K = 10 % the threshold is zero (all non-zeros
    and the first zeros are kept, the memory empties), at K = 1 % it lies among the non-zeros and the memory
    fills up again.  Eager and lazy residual modes must give the same bits, step by step and after the flush."""
    table = wl.make_table([("emb", (1200, 330)), ("v", (9,)), ("dense", (64, 330))])
    W = 3
    ctxs = [binding.Context(table, W), binding.Context(table, W, flags=binding.ACC_FLAG_LAZY_RESIDUAL)]
    st = [dict(zip(("vals", "idx", "counts"), c.new_topk_buffers())) for c in ctxs]
    for s_ in st:
        s_["err"] = torch.zeros(W, table.stride, device="cuda")
        s_["out"] = torch.zeros(table.stride, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(31)
    o_emb = int(table.offset[0])
    seen = set()
    for it, lv in enumerate([1, 1, 0, 0, 1, 0, 1, 1]):
        grads = torch.zeros(W, table.stride, device="cuda")
        grads[:, int(table.offset[2]):int(table.offset[2]) + 64 * 330] = torch.randn(W, 64 * 330, generator=g, device="cuda")
        grads[:, int(table.offset[1]):int(table.offset[1]) + 9] = torch.randn(W, 9, generator=g, device="cuda")
        for w in range(W):
            rows = torch.randperm(1200, generator=g, device="cuda")[:24]
            emb = torch.zeros(1200, 330, device="cuda")
            emb[rows] = torch.randn(24, 330, generator=g, device="cuda")
            grads[w, o_emb:o_emb + 1200 * 330] = emb.reshape(-1)
        level = torch.full((table.n_layers,), lv, dtype=torch.uint8, device="cuda")
        e0 = st[0]["err"].clone()
        for c, s_ in zip(ctxs, st):
            c.acc_topk_step(grads, s_["err"], level, s_["vals"], s_["idx"], s_["counts"], s_["out"])
        torch.cuda.synchronize()
        H.check_topk_against_oracle(ctxs[0], table, grads, e0, level, st[0]["vals"], st[0]["idx"], st[0]["counts"],
                                    st[0]["out"], st[0]["err"], 1000, 100)
        for name in ("vals", "idx", "counts", "out"):
            assert torch.equal(st[0][name], st[1][name]), (it, name)
        seen.update(int(p) for p in ctxs[1].acc_topk_last_paths()[:, 0])
    assert 4 in seen and len(seen) > 1, seen
    ctxs[1].acc_topk_flush(st[1]["err"])
    torch.cuda.synchronize()
    assert torch.equal(st[0]["err"], st[1]["err"])


@pytest.mark.parametrize("lazy", [0, binding.ACC_FLAG_LAZY_RESIDUAL])
def test_powersgd_tall_layers_orthonormalisation_paths(lazy):
    """Gram-Schmidt runs on a thread-block cluster for layers of 2049..49152 rows and on one block otherwise;
    a table with a layer of each kind (and one beyond the cluster's capacity) against the oracle."""
    table = wl.make_table([("tall", (3000, 40)), ("b", (7,)), ("huge", (50000, 8)), ("short", (600, 16))])
    W = 2
    ctx = binding.Context(table, W, rank_low=4, rank_high=2, flags=lazy)
    ref = binding.Context(table, W, rank_low=4, rank_high=2)  # eager twin supplies the true error memory
    grads, err = _random_inputs(table, W, 91)
    q0 = wl.initial_q(table, 4, seed=5)
    st = [dict(err=err.clone(), q=c.new_q(q0), p=c.new_p(), out=torch.zeros(table.stride, device="cuda")) for c in (ctx, ref)]
    for it in range(3):
        level = torch.tensor([(l + it) % 2 for l in range(table.n_layers)], dtype=torch.uint8, device="cuda")
        e0, qb = st[1]["err"].clone(), st[1]["q"].clone()
        for c, s_ in zip((ctx, ref), st):
            c.acc_powersgd_step(grads, s_["err"], s_["q"], s_["p"], level, s_["out"])
        torch.cuda.synchronize()
        H.check_powersgd_against_oracle(ref, table, grads, e0, qb, level, st[1]["out"], st[1]["err"], st[1]["q"],
                                        st[1]["p"], 4, 2, 1e-8)
        for name in ("out", "q", "p"):
            assert torch.equal(st[0][name], st[1][name]), name
        grads, _ = _random_inputs(table, W, 400 + it)
    assert ctx.last_launch_count() == 6 and ctx.acc_device_status() == 0


@pytest.mark.parametrize("lazy", [0, binding.ACC_FLAG_LAZY_RESIDUAL])
def test_powersgd_pipelined_pass_on_half_of_the_sms_gives_the_same_bits(lazy):
    """ACC_FLAG_SHARE_SMS only changes how many persistent blocks share the tiles of the pipelined first pass (a
    table with more tiles than SMs, so that the block count does change): every output bit stays."""
    table = wl.make_table([("big", (512, 4608)), ("v", (100,)), ("lstm", (300, 650)), ("mid", (256, 1152))])
    W = 2
    base = binding.ACC_FLAG_PIPELINE_ALWAYS | lazy
    ctxs = [binding.Context(table, W, rank_low=2, rank_high=1, flags=f) for f in (base, base | binding.ACC_FLAG_SHARE_SMS)]
    grads, err = _random_inputs(table, W, 77)
    q0 = wl.initial_q(table, 2, seed=3)
    st = [dict(err=err.clone(), q=c.new_q(q0), p=c.new_p(), out=torch.zeros(table.stride, device="cuda"),
               delta=torch.zeros(table.stride, device="cuda")) for c in ctxs]
    for it in range(3):
        level = torch.tensor([(l + it) % 2 for l in range(table.n_layers)], dtype=torch.uint8, device="cuda")
        for c, s_ in zip(ctxs, st):
            c.acc_powersgd_step(grads, s_["err"], s_["q"], s_["p"], level, s_["out"], s_["delta"])
        torch.cuda.synchronize()
        for name in ("out", "q", "p", "err", "delta"):
            assert torch.equal(st[0][name], st[1][name]), (it, name)
        grads, _ = _random_inputs(table, W, 500 + it)
    assert all(c.acc_device_status() == 0 for c in ctxs)


def test_difference_criterion_variant_matches_oracle():
    table = _table_mixed()
    ctx = binding.Context(table, 1, eta=0.5)
    layers = H.layers_of(table)
    g = torch.Generator(device="cuda").manual_seed(12)
    prev = torch.zeros(table.stride, device="cuda")
    curr = torch.zeros(table.stride, device="cuda")
    for l, sl in table.slices():
        base = torch.randn(sl.stop - sl.start, generator=g, device="cuda")
        prev[sl] = base
        # per layer a different relation: scaled copy, rotated (sign-flipped half), small perturbation
        kind = l % 3
        if kind == 0:
            curr[sl] = base * (0.4 + 0.1 * l)
        elif kind == 1:
            flipped = base.clone(); flipped[::2] *= -1.0
            curr[sl] = flipped
        else:
            curr[sl] = base + 0.1 * torch.randn(sl.stop - sl.start, generator=g, device="cuda")
    L = table.n_layers
    d2 = torch.zeros(L, dtype=torch.float64, device="cuda")
    n2c = torch.zeros(L, dtype=torch.float64, device="cuda")
    n2p = torch.zeros(L, dtype=torch.float64, device="cuda")
    ctx.acc_layer_diff_norms(prev, curr, d2)
    ctx.acc_layer_norms(curr, 1, n2c)
    ctx.acc_layer_norms(prev, 1, n2p)
    level = torch.full((L,), 9, dtype=torch.uint8, device="cuda")
    delta, delta_prev = curr.clone(), prev.clone()
    n2p_before = n2p.clone()
    ctx.acc_detect_regime_diff(d2, n2c, n2p, 0.1, 0.1, level, delta, delta_prev)
    torch.cuda.synchronize()
    ph, ch = prev.cpu().numpy(), curr.cpu().numpy()
    want_d2 = orc.layer_diff_norms2(ph, ch, layers)
    assert np.allclose(d2.cpu().numpy(), want_d2, rtol=1e-6, atol=0)   # fp32 subtraction on the device
    want, want_prev = orc.detect_regime_diff(d2.cpu().numpy(), n2c.cpu().numpy(), n2p_before.cpu().numpy(), 0.1, 0.1,
                                             np.float32(0.5))
    assert np.array_equal(level.cpu().numpy(), want) and 0 < want.sum() < L
    assert np.array_equal(n2p.cpu().numpy(), want_prev)
    assert torch.equal(delta_prev, curr) and float(delta.abs().max()) == 0.0
    # the rotated layers are critical under this variant but not under Algorithm 1
    lv1 = torch.zeros(L, dtype=torch.uint8, device="cuda")
    ctx.acc_detect_regime(n2c, n2p_before.clone(), 0.1, 0.1, lv1)
    torch.cuda.synchronize()
    assert int(level[1]) == 1 and int(lv1[1]) == 0


def test_checkpoint_resume_is_bit_identical():
    """State of the path = caller buffers (error memories, Q, P^, accumulator, norms, levels).  Running 2k
    iterations must equal k iterations + copying the state into a new context + k iterations.  In lazy mode
    what is pending inside the context is materialised (acc_powersgd_flush, acc_topk_flush) before the copy."""
    w = wl.workload(5, scale=16)
    table, W = w.table, w.n_workers
    stream = wl.GradientStream(w, device="cuda")
    names = ("level", "delta", "norm2_prev", "err_psgd", "q", "p_hat", "out_psgd", "err_topk", "out_topk")

    def engine():
        return pipeline.AccordionStep(table, W, w.compressors, w.rank_low, w.rank_high, w.topk_low_bp,
                                      w.topk_high_bp, w.eta, 1e-8, 4, lazy_residual=True)

    k = 6
    full = engine()
    for t in range(2 * k):
        full.step(stream.grads(t))
    first = engine()
    for t in range(k):
        first.step(stream.grads(t))
    first.flush()
    torch.cuda.synchronize()
    second = engine()
    for n in names:
        getattr(second, n).copy_(getattr(first, n))
    second.t = first.t
    for t in range(k, 2 * k):
        second.step(stream.grads(t))
    full.flush()
    second.flush()
    torch.cuda.synchronize()
    for n in names:
        assert torch.equal(getattr(full, n), getattr(second, n)), n


def test_two_compressors_side_by_side_equal_one_after_the_other():
    """With both compressors the engine runs the TopK step on a second stream beside the PowerSGD step; every
    result must be the bits of the sequential order, directly and as replayed CUDA graphs."""
    table = _table_mixed()
    W = 3
    q0 = wl.initial_q(table, 2, seed=31)
    engines = [pipeline.AccordionStep(table, W, ("powersgd", "topk"), check_every=2, q_init=q0, lazy_residual=True,
                                      overlap=ov) for ov in (False, True, True)]
    bufs = [_random_inputs(table, W, 1200 + i)[0] for i in range(2)]
    engines[2].capture_graphs(bufs)
    for t in range(6):
        engines[0].step(bufs[t % 2])
        engines[1].step(bufs[t % 2])
        engines[2].step_graph(t % 2)
    torch.cuda.synchronize()
    ref = engines[0]
    for e in engines[1:]:
        for name in ("out_psgd", "out_topk", "err_psgd", "err_topk", "q", "p_hat", "vals", "idx", "counts", "level",
                     "delta", "norm2_prev"):
            assert torch.equal(getattr(ref, name), getattr(e, name)), name
        assert e.launches == ref.launches


def test_topk_whole_model_selection_scope():
    """Selection over the whole model instead of per layer is the same step on a table whose single MATRIX layer
    spans all parameters: k = floor(N * K) entries are kept across what were the layers."""
    per_layer = _table_mixed()
    n = int(per_layer.stride)
    table = wl.make_table([("model", (1, n))])
    W = 2
    ctx = binding.Context(table, W, topk_low_bp=500, topk_high_bp=50)
    grads = torch.zeros(W, table.stride, device="cuda")
    g, _ = _random_inputs(per_layer, W, 77)
    grads[:, :n] = g
    err = torch.zeros_like(grads)
    vals, idx, counts = ctx.new_topk_buffers()
    out = torch.zeros(table.stride, device="cuda")
    for lv in (1, 0, 0):
        level = torch.full((1,), lv, dtype=torch.uint8, device="cuda")
        e0 = err.clone()
        ctx.acc_topk_step(grads, err, level, vals, idx, counts, out)
        torch.cuda.synchronize()
        H.check_topk_against_oracle(ctx, table, grads, e0, level, vals, idx, counts, out, err, 500, 50)
        assert int(counts[0]) == max(1, n * (500 if lv else 50) // 10000)
    # the layers with the largest scale (10^0) carry nearly all kept entries: the scope really is global
    kept = idx[:int(counts[0])].cpu().numpy()
    big = np.zeros(n, bool)
    for l, sl in per_layer.slices():
        if l % 4 == 0:
            big[sl] = True
    assert big[kept].mean() > 0.9


@pytest.mark.parametrize("pipeline_flag", [binding.ACC_FLAG_PIPELINE_NEVER, binding.ACC_FLAG_PIPELINE_ALWAYS])
def test_topk_lazy_residual_is_bit_identical_to_eager(pipeline_flag):
    """Lazy mode leaves the kept entries above the threshold in err and reads them as +0.0 on the next load: packed
    sets, outputs and -- after a flush -- the error memory are the eager mode's bits, through level switches,
    exact ties at the threshold, zero-filled selections and every selection path."""
    table = _table_mixed()
    W = 3
    eager = binding.Context(table, W, topk_low_bp=1000, topk_high_bp=100, flags=pipeline_flag)
    lazy = binding.Context(table, W, topk_low_bp=1000, topk_high_bp=100,
                           flags=pipeline_flag | binding.ACC_FLAG_LAZY_RESIDUAL)
    _, err_e = _random_inputs(table, W, 5)
    err_l = err_e.clone()
    ve, ie, ce = eager.new_topk_buffers()
    vl, il, cl = lazy.new_topk_buffers()
    out_e, out_l = torch.zeros(table.stride, device="cuda"), torch.zeros(table.stride, device="cuda")
    d_e, d_l = torch.zeros(table.stride, device="cuda"), torch.zeros(table.stride, device="cuda")
    base, _ = _random_inputs(table, W, 1400)
    for it in range(10):
        level = torch.tensor([(l + it // 3) % 2 for l in range(table.n_layers)], dtype=torch.uint8, device="cuda")
        noise, _ = _random_inputs(table, W, 1401 + it)
        grads = base + 0.05 * noise  # similar steps: the threshold predictions hold, staged and list paths run
        if it == 4:  # exact ties at and around the threshold; a worker with an all-zero gradient
            grads = torch.round(grads * 4.0) / 4.0
            grads[1].zero_()
        eager.acc_topk_step(grads, err_e, level, ve, ie, ce, out_e, d_e)
        lazy.acc_topk_step(grads, err_l, level, vl, il, cl, out_l, d_l)
        torch.cuda.synchronize()
        assert torch.equal(ie, il) and torch.equal(ce, cl) and torch.equal(out_e, out_l) and torch.equal(d_e, d_l), it
        assert torch.equal(ve.view(torch.int32), vl.view(torch.int32)), it
        if it in (2, 6):  # a flush in the middle changes nothing downstream
            lazy.acc_topk_flush(err_l)
            torch.cuda.synchronize()
            assert torch.equal(err_e.view(torch.int32), err_l.view(torch.int32)), it
    assert not torch.equal(err_e, err_l)  # something is pending: the modes differ in memory before the flush
    lazy.acc_topk_flush(err_l)
    torch.cuda.synchronize()
    assert torch.equal(err_e.view(torch.int32), err_l.view(torch.int32))
    with pytest.raises(binding.AccError):
        eager.acc_topk_flush(err_e)


@pytest.mark.parametrize("seed", [1, 2, 3, 4, 5, 6])
def test_random_tables_both_compressors(seed):
    """Seeded random layer tables (matrix shapes from 1 x 1 to a few tiles, odd row lengths, vectors in between,
    unaligned sizes), random W, ranks, fractions, levels and flags: two steps of each compressor against the
    oracle."""
    rng = np.random.default_rng(1000 + seed)
    shapes = []
    for i in range(int(rng.integers(3, 9))):
        kind = rng.integers(0, 4)
        if kind == 0:
            shapes.append((f"v{i}", (int(rng.integers(1, 9000)),)))
        elif kind == 1:
            shapes.append((f"m{i}", (int(rng.integers(1, 40)), int(rng.integers(1, 40)))))
        elif kind == 2:
            shapes.append((f"m{i}", (int(rng.integers(1, 12)), int(rng.integers(1000, 9000)))))
        else:
            shapes.append((f"m{i}", (int(rng.integers(100, 3000)), int(rng.integers(1, 24)))))
    if not any(len(s) == 2 for _, s in shapes):
        shapes.append(("m_last", (17, 19)))
    table = wl.make_table(shapes)
    W = int(rng.integers(1, 6))
    rank_low = int(rng.integers(1, 5))
    rank_high = int(rng.integers(1, rank_low + 1))
    low_bp = int(rng.integers(50, 4000))
    high_bp = int(rng.integers(1, low_bp + 1))
    flags = int(rng.choice([0, binding.ACC_FLAG_PIPELINE_ALWAYS, binding.ACC_FLAG_PIPELINE_NEVER]))
    ctx = binding.Context(table, W, rank_low=rank_low, rank_high=rank_high, topk_low_bp=low_bp, topk_high_bp=high_bp,
                          decider=int(rng.integers(0, W)), flags=flags)
    level = torch.tensor(rng.integers(0, 2, table.n_layers).astype(np.uint8), device="cuda")
    _, err_p = _random_inputs(table, W, 2000 + seed)
    err_t = err_p.clone()
    q = ctx.new_q(wl.initial_q(table, 4, seed=seed))
    p = ctx.new_p()
    vals, idx, counts = ctx.new_topk_buffers()
    out = torch.zeros(table.stride, device="cuda")
    delta = torch.zeros(table.stride, device="cuda")
    for it in range(2):
        grads, _ = _random_inputs(table, W, 2100 + 10 * seed + it)
        e0, q0 = err_p.clone(), q.clone()
        ctx.acc_powersgd_step(grads, err_p, q, p, level, out, delta)
        torch.cuda.synchronize()
        H.check_powersgd_against_oracle(ctx, table, grads, e0, q0, level, out, err_p, q, p, rank_low, rank_high, 1e-8)
        e0 = err_t.clone()
        ctx.acc_topk_step(grads, err_t, level, vals, idx, counts, out, None)
        torch.cuda.synchronize()
        H.check_topk_against_oracle(ctx, table, grads, e0, level, vals, idx, counts, out, err_t, low_bp, high_bp)
    assert ctx.acc_device_status() == 0


def test_host_fed_step_uploads_and_downloads_through_the_library():
    """Gradients in pinned host memory, uploaded by acc_upload_grads on a copy stream, outputs read back by
    acc_download_out: the host copies of the outputs equal the device-resident run's."""
    table = _table_mixed()
    W = 2
    q0 = wl.initial_q(table, 2, seed=41)
    dev_eng = pipeline.AccordionStep(table, W, ("powersgd", "topk"), check_every=2, q_init=q0)
    fed_eng = pipeline.AccordionStep(table, W, ("powersgd", "topk"), check_every=2, q_init=q0)
    fed = pipeline.HostFedStep(fed_eng)
    host = [torch.empty(W, table.stride).pin_memory() for _ in range(2)]
    for t in range(5):
        g, _ = _random_inputs(table, W, 3000 + t)
        host[t % 2].copy_(g)
        dev_eng.step(g)
        outs = fed.step(host[t % 2])
        fed.synchronize()
        torch.cuda.synchronize()
        for oh, od in zip(outs, dev_eng.outputs()):
            assert torch.equal(oh, od.cpu())
    with pytest.raises(ValueError):
        fed_eng.ctx.acc_upload_grads(torch.empty(3), fed.stage[0])


def test_many_workers():
    """W = 37 (more workers than a warp has lanes, not a multiple of the kernels' worker batches) on a small table."""
    table = wl.make_table([("w0", (50, 333)), ("b0", (77,)), ("w1", (9000, 3)), ("b1", (8195,))])
    W = 37
    ctx = binding.Context(table, W, rank_low=2, rank_high=1, topk_low_bp=700, topk_high_bp=70, decider=36)
    level = torch.tensor([1, 0, 0, 1], dtype=torch.uint8, device="cuda")
    _, err_p = _random_inputs(table, W, 3100)
    err_t = err_p.clone()
    q = ctx.new_q(wl.initial_q(table, 2, seed=3))
    p = ctx.new_p()
    vals, idx, counts = ctx.new_topk_buffers()
    out = torch.zeros(table.stride, device="cuda")
    delta = torch.zeros(table.stride, device="cuda")
    for it in range(2):
        grads, _ = _random_inputs(table, W, 3110 + it)
        e0, q0 = err_p.clone(), q.clone()
        ctx.acc_powersgd_step(grads, err_p, q, p, level, out, delta)
        torch.cuda.synchronize()
        H.check_powersgd_against_oracle(ctx, table, grads, e0, q0, level, out, err_p, q, p, 2, 1, 1e-8)
        e0 = err_t.clone()
        ctx.acc_topk_step(grads, err_t, level, vals, idx, counts, out, None)
        torch.cuda.synchronize()
        H.check_topk_against_oracle(ctx, table, grads, e0, level, vals, idx, counts, out, err_t, 700, 70)
    # the accumulator holds the deciding worker's two gradients
    want = sum(_random_inputs(table, W, 3110 + it)[0][36] for it in range(2))
    for l, sl in table.slices():
        assert torch.allclose(delta[sl], want[sl], rtol=1e-6, atol=1e-7), l


def test_topk_three_hundred_workers():
    """W = 300: more workers than the decompress pass has threads in a block (it keeps a tile's ranges for up to
    four workers per thread) and than its staging area holds at once at K = 50 % (several rounds per tile)."""
    table = wl.make_table([("w", (40, 300)), ("b", (5,)), ("tall", (2100, 4))])
    W = 300
    ctx = binding.Context(table, W, topk_low_bp=5000, topk_high_bp=100, decider=299)
    vals, idx, counts = ctx.new_topk_buffers()
    out = torch.zeros(table.stride, device="cuda")
    _, err = _random_inputs(table, W, 4100)
    for it, lv in enumerate(([1, 0, 0], [0, 0, 1])):
        level = torch.tensor(lv, dtype=torch.uint8, device="cuda")
        grads, _ = _random_inputs(table, W, 4110 + it)
        e0 = err.clone()
        ctx.acc_topk_step(grads, err, level, vals, idx, counts, out, None)
        torch.cuda.synchronize()
        H.check_topk_against_oracle(ctx, table, grads, e0, level, vals, idx, counts, out, err, 5000, 100)
    assert ctx.acc_device_status() == 0


def test_bounded_wait_reports_timeout_and_context_stays_usable():
    """Failure detection without a fault: a kernel waits, with a short poll limit, on a barrier nothing arrives at;
    the wait gives up, the status word reads ACC_ETIMEOUT, the kernel has returned normally and later calls on the
    same context work as before."""
    table = _table_mixed()
    W = 2
    ctx = binding.Context(table, W, flags=binding.ACC_FLAG_PIPELINE_ALWAYS)
    assert ctx.acc_device_status() == 0
    ctx.acc_selftest_wait_timeout()
    assert ctx.acc_device_status() == 6  # ACC_ETIMEOUT
    grads, err = _random_inputs(table, W, 3200)
    q = ctx.new_q(wl.initial_q(table, 2, seed=8))
    p = ctx.new_p()
    level = torch.ones(table.n_layers, dtype=torch.uint8, device="cuda")
    out = torch.zeros(table.stride, device="cuda")
    e0, q0 = err.clone(), q.clone()
    ctx.acc_powersgd_step(grads, err, q, p, level, out)
    torch.cuda.synchronize()
    H.check_powersgd_against_oracle(ctx, table, grads, e0, q0, level, out, err, q, p, 2, 1, 1e-8)
    assert ctx.acc_device_status() == 6  # sticky until it is reset
    ctx.acc_reset_device_status()
    assert ctx.acc_device_status() == 0
