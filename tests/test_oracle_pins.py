"""Pins of the CPU oracle against things other than itself: closed forms, invariants,
library routines on special cases, brute force on tiny inputs and the values the paper
prints (tests/golden).  A plausible mistake in the oracle (dropped term, wrong sign or
index, transposed operand) fails at least one of these."""
import itertools
import os

import numpy as np
import pytest

from oracle import accordion_oracle as orc
from paper_2010_16248_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "data_sent_tables.txt")


def _layers(table):
    return [(int(table.offset[l]), int(table.rows[l]), int(table.cols[l]), int(table.kind[l]))
            for l in range(table.n_layers)]


# ------------------------------------------------------------------ controller
def test_alg1_truth_table():
    # (prev_norm, curr_norm, lr_curr, lr_next) -> level, eta = 0.5; boundary cases are exactly representable
    cases = [
        (1.0, 0.5, 0.1, 0.1, orc.LOW),    # ratio exactly eta: ">=" -> critical
        (1.0, 1.5, 0.1, 0.1, orc.LOW),    # growth counts too (absolute value)
        (1.0, 0.75, 0.1, 0.1, orc.HIGH),
        (1.0, 1.25, 0.1, 0.1, orc.HIGH),
        (1.0, 1.0, 0.1, 0.01, orc.LOW),   # LR decay forces the low level
        (1.0, 1.0, 0.1, 0.2, orc.HIGH),   # LR increase does not
        (4.0, 1.0, 0.1, 0.1, orc.LOW),
        (0.0, 0.0, 0.1, 0.1, orc.LOW),    # ||prev|| = 0: product form, 0 >= 0
        (0.0, 3.0, 0.1, 0.1, orc.LOW),
    ]
    for a, b, lc, ln, want in cases:
        level, prev = orc.detect_regime(np.array([b * b]), np.array([a * a]), lc, ln, 0.5)
        assert level[0] == want, (a, b, lc, ln)
        assert prev[0] == b * b
    level, prev = orc.detect_regime(np.array([9.0]), np.array([-1.0]), 0.1, 0.1, 0.5)
    assert level[0] == orc.LOW and prev[0] == 9.0  # no previous window


def test_detector_scale_invariance_and_per_layer_independence():
    rng = np.random.default_rng(0)
    prev = rng.uniform(0.1, 4.0, 50)
    curr = rng.uniform(0.1, 4.0, 50)
    l1, _ = orc.detect_regime(curr, prev, 0.1, 0.1, 0.5)
    l2, _ = orc.detect_regime(curr * 64.0, prev * 64.0, 0.1, 0.1, 0.5)
    assert np.array_equal(l1, l2)
    want = (np.abs(np.sqrt(prev) - np.sqrt(curr)) / np.sqrt(prev) >= 0.5).astype(np.uint8)
    assert np.array_equal(l1, want)
    assert 0 < l1.sum() < 50


def test_difference_criterion_truth_table_and_contrast_with_algorithm1():
    """The norm-of-difference variant on hand-computed vectors; the rotated case separates the two readings:
    equal norms (Algorithm 1: not critical) but a large difference (variant: critical)."""
    table = wl.make_table([("a", (2,)), ("b", (2,)), ("c", (2,)), ("d", (2,))])
    layers = _layers(table)
    prev = np.zeros(table.stride, np.float32)
    curr = np.zeros(table.stride, np.float32)
    vec = {0: ((1, 0), (0.5, 0)),     # ||diff|| = 0.5 = eta * 1      -> LOW (>=)
           1: ((1, 0), (0.75, 0)),    # 0.25 < 0.5                    -> HIGH
           2: ((1, 0), (0, 1)),       # rotated: sqrt(2) >= 0.5       -> LOW, while the norms are equal
           3: ((0, 0), (0, 0))}       # zero previous gradient        -> LOW (0 >= 0)
    for l, (p, c) in vec.items():
        off = layers[l][0]
        prev[off:off + 2], curr[off:off + 2] = p, c
    d2 = orc.layer_diff_norms2(prev, curr, layers)
    assert np.allclose(d2, [0.25, 0.0625, 2.0, 0.0])
    n2p, n2c = orc.layer_norms2(prev, layers), orc.layer_norms2(curr, layers)
    lv, new_prev = orc.detect_regime_diff(d2, n2c, n2p, 0.1, 0.1, 0.5)
    assert list(lv) == [1, 0, 1, 1] and np.array_equal(new_prev, n2c)
    lv0, _ = orc.detect_regime(n2c, n2p, 0.1, 0.1, 0.5)
    assert list(lv0) == [1, 0, 0, 1]                      # Algorithm 1 does not see the rotation
    lv, _ = orc.detect_regime_diff(d2, n2c, -np.ones(4), 0.1, 0.1, 0.5)
    assert list(lv) == [1, 1, 1, 1]                       # no previous window
    lv, _ = orc.detect_regime_diff(d2, n2c, n2p, 0.1, 0.05, 0.5)
    assert list(lv) == [1, 1, 1, 1]                       # learning-rate decay


def test_layer_norms_closed_form_and_library():
    table = wl.make_table([("a", (3, 5)), ("b", (7,)), ("c", (4, 4))])
    layers = _layers(table)
    buf = np.zeros(table.stride, np.float32)
    buf[0:15] = 1.0                      # ||ones(15)||^2 = 15
    buf[16:23] = np.arange(1, 8)         # 1^2+..+7^2 = 140
    rng = np.random.default_rng(1)
    c = rng.standard_normal(16).astype(np.float32)
    buf[24:40] = c
    n2 = orc.layer_norms2(buf, layers)
    assert n2[0] == 15.0 and n2[1] == 140.0
    assert np.isclose(np.sqrt(n2[2]), np.linalg.norm(c.astype(np.float64)), rtol=1e-14)


def test_msdr_hand_values_library_and_invariances():
    """Mean-to-standard-deviation ratio per layer: hand-computed vectors, the library's mean / std on random
    ones, and what the definition implies (scale invariance, sign symmetry, the effect of a shift)."""
    table = wl.make_table([("a", (2, 2)), ("const", (4,)), ("zero", (1, 4)), ("sym", (4,)), ("b", (3, 5))])
    layers = _layers(table)
    buf = np.zeros(table.stride, np.float32)
    rng = np.random.default_rng(3)
    rnd = (rng.standard_normal(15) + 0.7).astype(np.float32)
    for (off, r, c, k), vals in zip(layers, ([1, 2, 3, 4], [2, 2, 2, 2], [0, 0, 0, 0], [-3, -1, 1, 3], rnd)):
        buf[off:off + r * c] = vals
    msdr, mean, std = orc.layer_msdr(buf, layers)
    # [1,2,3,4]: mean 2.5, deviations +-1.5, +-0.5 -> variance (2.25+0.25)*2/4 = 1.25
    assert mean[0] == 2.5 and abs(std[0] - np.sqrt(1.25)) < 1e-15 and abs(msdr[0] - 2.5 / np.sqrt(1.25)) < 1e-15
    assert abs(msdr[0] - np.sqrt(5.0)) < 1e-15
    assert np.isinf(msdr[1]) and mean[1] == 2.0 and std[1] == 0.0      # constant layer
    assert msdr[2] == 0.0 and msdr[3] == 0.0 and mean[3] == 0.0          # all zero; zero mean
    assert abs(std[3] - np.sqrt(5.0)) < 1e-15                            # (9+1+1+9)/4
    x = rnd.astype(np.float64)
    assert abs(msdr[4] - abs(np.mean(x)) / np.std(x)) < 1e-12 and abs(std[4] - np.std(x)) < 1e-14
    # invariances: scaling by c != 0 (also negative) leaves the ratio alone; padding is not read
    buf2 = (-3.0 * buf).astype(np.float32)
    end_b = layers[4][0] + 15
    assert end_b < table.stride
    buf2[end_b:] = 99.0
    m2, _, _ = orc.layer_msdr(buf2, layers)
    assert abs(m2[0] - msdr[0]) < 1e-6 and abs(m2[4] - msdr[4]) < 1e-6
    # a shift by s moves the mean and leaves the deviation: MSDR(x + s) = |mu + s| / sd
    off, r, c, _ = layers[4]
    shifted = buf.copy()
    shifted[off:off + 15] = (rnd.astype(np.float64) + 4.0).astype(np.float32)
    m3, mu3, sd3 = orc.layer_msdr(shifted, layers)
    xs = shifted[off:off + 15].astype(np.float64)
    assert abs(sd3[4] - np.std(xs)) < 1e-14 and abs(m3[4] - abs(np.mean(xs)) / np.std(xs)) < 1e-12
    assert abs(sd3[4] - std[4]) < 1e-6 and abs(mu3[4] - (mean[4] + 4.0)) < 1e-6


def test_accumulate_sums_decider_gradients():
    table = wl.make_table([("a", (2, 3)), ("b", (5,))])
    layers = _layers(table)
    delta = np.zeros(table.stride)
    g1 = np.arange(table.stride, dtype=np.float32)
    g2 = np.ones(table.stride, np.float32)
    orc.accumulate(delta, g1, layers)
    orc.accumulate(delta, g2, layers)
    for (off, r, c, k) in layers:
        assert np.array_equal(delta[off:off + r * c], (g1 + g2)[off:off + r * c].astype(np.float64))
    assert delta[6] == 0.0 and delta[7] == 0.0  # padding between layers untouched


def test_error_feedback_hand_values_vector_rule_and_precision_flag():
    """M = g + e on MATRIX layers, M = g on VECTOR layers (1-D tensors carry no memory), padding stays zero;
    with fp32=True the sum is ONE fp32 add, which the hand-picked operands distinguish from the fp64 sum."""
    table = wl.make_table([("a", (2, 3)), ("v", (5,))])   # matrix at 0..5, padding 6..7, vector at 8..12
    layers = _layers(table)
    assert [l[0] for l in layers] == [0, 8]
    tiny = np.float32(2.0 ** -24)                         # half an ulp of 1.0 in fp32
    g = np.zeros((2, table.stride), np.float32)
    e = np.zeros((2, table.stride), np.float32)
    g[0, 0:6] = [1.0, 2.0, -3.0, 0.5, 1.0, 1.0]
    e[0, 0:6] = [0.25, -2.0, 1.0, 0.125, tiny, 3 * tiny]
    g[1, 0:6] = [10.0, 20.0, 30.0, 40.0, 50.0, 60.0]
    e[1, 0:6] = [-1.0, -2.0, -3.0, -4.0, -5.0, -6.0]
    g[:, 8:13] = [[1.0, 2.0, 3.0, 4.0, 5.0], [6.0, 7.0, 8.0, 9.0, 10.0]]
    e[:, 8:13] = 100.0                                    # memory on a VECTOR layer must be ignored
    e[:, 6:8] = 7.0                                       # so must anything in the padding
    M64 = orc.error_feedback(g, e, layers)
    assert M64.dtype == np.float64
    assert M64[0, 0:4].tolist() == [1.25, 0.0, -2.0, 0.625]
    assert M64[0, 4] == 1.0 + 2.0 ** -24 and M64[0, 5] == 1.0 + 3 * 2.0 ** -24      # exact in fp64
    assert M64[1, 0:6].tolist() == [9.0, 18.0, 27.0, 36.0, 45.0, 54.0]
    assert M64[0, 8:13].tolist() == [1.0, 2.0, 3.0, 4.0, 5.0] and M64[1, 8:13].tolist() == [6.0, 7.0, 8.0, 9.0, 10.0]
    assert np.all(M64[:, 6:8] == 0.0) and np.all(M64[:, 13:] == 0.0)
    M32 = orc.error_feedback(g, e, layers, fp32=True)
    assert M32.dtype == np.float32
    # 1 + 2^-24 is a tie between 1 and 1 + 2^-23: round-to-even gives 1; 1 + 3*2^-24 rounds up to 1 + 2^-22
    assert M32[0, 4] == np.float32(1.0) and M32[0, 5] == np.float32(1.0 + 2.0 ** -22)
    assert float(M32[0, 4]) != M64[0, 4] and float(M32[0, 5]) != M64[0, 5]
    assert M32[0, 0:4].tolist() == [1.25, 0.0, -2.0, 0.625] and M32[0, 8:13].tolist() == [1.0, 2.0, 3.0, 4.0, 5.0]
    assert np.all(M32[:, 6:8] == 0.0)


def test_error_feedback_is_what_both_compressors_split():
    """Invariant of error feedback: what a compressor sends plus what it keeps as memory is g + e.  Ties the
    stand-alone accumulation to the two compressor steps (which were pinned independently of it)."""
    rng = np.random.default_rng(21)
    table = wl.make_table([("a", (9, 14)), ("v", (7,)), ("b", (12, 5))])
    layers = _layers(table)
    W = 3
    grads = np.zeros((W, table.stride), np.float32)
    err = np.zeros((W, table.stride), np.float32)
    for (off, r, c, k) in layers:
        grads[:, off:off + r * c] = rng.standard_normal((W, r * c))
        if k == orc.MATRIX:
            err[:, off:off + r * c] = 0.4 * rng.standard_normal((W, r * c))
    level = [1, 0, 0]
    M64 = orc.error_feedback(grads, err, layers)
    M32 = orc.error_feedback(grads, err, layers, fp32=True)
    q = [rng.standard_normal((c, 2)) if k == orc.MATRIX else None for (_, _, c, k) in layers]
    out, e_p, _, _ = orc.powersgd_step(grads, err, q, level, layers, 2, 1)
    vals, idx, counts, _, e_t = orc.topk_step(grads, err, level, layers, 1000, 100)
    for l, (off, r, c, k) in enumerate(layers):
        sl = slice(off, off + r * c)
        if k == orc.VECTOR:
            assert np.allclose(out[sl], M64[:, sl].mean(0), rtol=1e-15)   # the mean of the raw gradients
            continue
        for w in range(W):
            assert np.allclose(out[sl] + e_p[w, sl], M64[w, sl], rtol=0, atol=1e-14)
            rec = e_t[w, sl].copy()
            rec[idx[w][l]] = vals[w][l]
            assert np.array_equal(rec.view(np.uint32), M32[w, sl].view(np.uint32))   # bit for bit, fp32 add


def test_c1_schedule_known_answer():
    """Config 1: scale doubles at iteration 10, checks after iterations 4, 9, 14, 19.
    Levels: LOW before the first check and after it (no previous window), HIGH after the
    second (equal windows), LOW after the third (window norm doubled: ratio 1 >= 0.5),
    HIGH after the fourth (equal again)."""
    w = wl.workload(1, scale=4)
    layers = _layers(w.table)
    stream = wl.GradientStream(w)
    delta = np.zeros(w.table.stride)
    prev = -np.ones(1)
    levels = []
    level = np.ones(1, np.uint8)
    for t in range(w.n_iters):
        levels.append(int(level[0]))
        g = stream.grads(t).numpy()
        orc.accumulate(delta, g[0], layers)
        if (t + 1) % w.check_every == 0:
            level, prev = orc.detect_regime(orc.layer_norms2(delta, layers), prev, 0.1, 0.1, w.eta)
            delta[:] = 0
    assert levels == [1] * 5 + [1] * 5 + [0] * 5 + [1] * 5
    assert int(level[0]) == 0


# ------------------------------------------------------------------ PowerSGD
def _rand_problem(rng, n, m, W, rank_low, err_scale=0.3):
    table = wl.make_table([("w", (n, m)), ("b", (5,))])
    layers = _layers(table)
    grads = np.zeros((W, table.stride), np.float32)
    err = np.zeros((W, table.stride), np.float32)
    grads[:, :n * m] = rng.standard_normal((W, n * m))
    err[:, :n * m] = err_scale * rng.standard_normal((W, n * m))
    grads[:, layers[1][0]:layers[1][0] + 5] = rng.standard_normal((W, 5))
    q = [rng.standard_normal((m, rank_low)).astype(np.float32), None]
    return table, layers, grads, err, q


def test_powersgd_exact_recovery_of_rank_r():
    rng = np.random.default_rng(2)
    n, m, W = 12, 9, 3
    for r in (1, 2, 4):
        table, layers, grads, err, q = _rand_problem(rng, n, m, W, r)
        # small-integer factors: the product is exactly representable in fp32, so the rank is exactly r
        B = rng.integers(-4, 5, (n, r)).astype(np.float64) @ rng.integers(-4, 5, (r, m)).astype(np.float64)
        assert np.linalg.matrix_rank(B) == r
        grads[:, :n * m] = B.astype(np.float32).reshape(-1)
        err[:] = 0
        M = grads[0, :n * m].astype(np.float64).reshape(n, m)
        out, e, qn, ph = orc.powersgd_step(grads, err, q, [1, 1], layers, r, 1, gs_eps=0.0)
        assert np.allclose(out[:n * m].reshape(n, m), M, atol=1e-12 * np.abs(M).max())
        assert np.abs(e[:, :n * m]).max() < 1e-12 * np.abs(M).max()


def test_powersgd_matches_qr_and_projection():
    rng = np.random.default_rng(3)
    n, m, W, r = 10, 7, 4, 3
    table, layers, grads, err, q = _rand_problem(rng, n, m, W, r)
    out, e, qn, ph = orc.powersgd_step(grads, err, q, [1, 1], layers, r, 1, gs_eps=0.0)
    Mw = [(grads[w, :n * m].astype(np.float64) + err[w, :n * m].astype(np.float64)).reshape(n, m) for w in range(W)]
    Mbar = sum(Mw) / W
    # P^ is the thin-QR factor of Mbar Q with R's diagonal made positive (library routine)
    Qf, R = np.linalg.qr(Mbar @ q[0].astype(np.float64))
    Qf = Qf * np.sign(np.diag(R))
    assert np.allclose(ph[0], Qf, atol=1e-10)
    assert np.allclose(ph[0].T @ ph[0], np.eye(r), atol=1e-12)
    # A = P^ P^T Mbar ; Q_new = Mbar^T P^
    A = out[:n * m].reshape(n, m)
    assert np.allclose(A, Qf @ Qf.T @ Mbar, atol=1e-12)
    assert np.allclose(qn[0], Mbar.T @ Qf, atol=1e-12)
    # error-feedback invariant per worker and orthogonality of the mean residual to P^
    for w in range(W):
        assert np.allclose(A + e[w, :n * m].reshape(n, m), Mw[w], atol=1e-13)
    assert np.abs(Qf.T @ (sum(e[w, :n * m].reshape(n, m) for w in range(W)) / W)).max() < 1e-12
    # VECTOR layer: plain mean, no memory
    off = layers[1][0]
    assert np.allclose(out[off:off + 5], grads[:, off:off + 5].astype(np.float64).mean(0), atol=1e-15)
    assert np.all(e[:, off:off + 5] == 0)


def test_powersgd_rank_levels_and_untouched_columns():
    rng = np.random.default_rng(4)
    n, m, W = 8, 6, 2
    table, layers, grads, err, q = _rand_problem(rng, n, m, W, 2)
    _, _, qn_hi, ph_hi = orc.powersgd_step(grads, err, q, [0, 0], layers, 2, 1)
    assert ph_hi[0].shape == (n, 1)
    assert np.array_equal(qn_hi[0][:, 1], q[0][:, 1].astype(np.float64))  # column beyond the rank keeps its value
    _, _, qn_lo, ph_lo = orc.powersgd_step(grads, err, q, [1, 1], layers, 2, 1)
    assert ph_lo[0].shape == (n, 2)
    assert np.allclose(ph_lo[0][:, 0], ph_hi[0][:, 0])


def test_powersgd_symmetries():
    rng = np.random.default_rng(5)
    n, m, W, r = 9, 11, 3, 2
    table, layers, grads, err, q = _rand_problem(rng, n, m, W, r)
    out, e, qn, ph = orc.powersgd_step(grads, err, q, [1, 1], layers, r, 1, gs_eps=0.0)
    perm = [2, 0, 1]
    out_p, e_p, qn_p, ph_p = orc.powersgd_step(grads[perm], err[perm], q, [1, 1], layers, r, 1, gs_eps=0.0)
    assert np.allclose(out, out_p, atol=1e-13) and np.allclose(e[perm], e_p, atol=1e-13)
    c = 8.0  # power of two: exact scaling
    out_s, e_s, qn_s, ph_s = orc.powersgd_step(grads * c, err * c, q, [1, 1], layers, r, 1, gs_eps=0.0)
    assert np.allclose(out_s, c * out, rtol=1e-12, atol=1e-14)
    assert np.allclose(ph_s[0], ph[0], atol=1e-12)


@pytest.mark.parametrize("power", [1.0, 0.5])
def test_powersgd_power_iteration_reaches_best_rank_r_error(power):
    """Repeating the step on a fixed M with the memory reset is subspace iteration: the
    error converges to the optimal sqrt(sum_{i>r} s_i^2), known in closed form for the
    synthetic spectra s_i = i^-1 and i^-0.5."""
    rng = np.random.default_rng(6)
    n, m, r, rho = 40, 30, 2, 30
    U, _ = np.linalg.qr(rng.standard_normal((n, rho)))
    V, _ = np.linalg.qr(rng.standard_normal((m, rho)))
    s = np.arange(1, rho + 1, dtype=np.float64) ** (-power)
    M = (U * s) @ V.T
    table = wl.make_table([("w", (n, m))])
    layers = _layers(table)
    grads = np.zeros((1, table.stride), np.float32)
    grads[0, :n * m] = M.reshape(-1)
    M32 = grads[0, :n * m].astype(np.float64).reshape(n, m)
    s32 = np.linalg.svd(M32, compute_uv=False)
    best = np.sqrt(np.sum(s32[r:] ** 2))
    assert np.isclose(best, np.sqrt(np.sum(s[r:] ** 2)), rtol=1e-5)
    q = [rng.standard_normal((m, r)).astype(np.float32)]
    err0 = np.zeros_like(grads)
    last = None
    for it in range(400):
        out, e, q, ph = orc.powersgd_step(grads, err0, q, [1], layers, r, 1, gs_eps=0.0)
        last = np.linalg.norm(e[0, :n * m])
    assert last >= best * (1 - 1e-12)
    assert np.isclose(last, best, rtol=1e-6)


def test_gram_schmidt_zero_column_is_finite():
    P = np.zeros((5, 2))
    P[:, 0] = 1.0
    out = orc.gram_schmidt(P, 1e-8)
    assert np.all(np.isfinite(out)) and np.all(out[:, 1] == 0)


# ------------------------------------------------------------------ TopK
def _order_key(v, i):
    bits = np.float32(v).view(np.uint32) & np.uint32(0x7FFFFFFF)
    return (-int(bits), i)


def _brute_force_topk(vals, k):
    """The kept set is the unique size-k subset in which every member precedes every
    non-member in the order (larger |v| first, then lower index): enumerate subsets."""
    n = len(vals)
    found = None
    for S in itertools.combinations(range(n), k):
        rest = [i for i in range(n) if i not in S]
        worst_in = max(_order_key(vals[i], i) for i in S)
        if all(worst_in < _order_key(vals[j], j) for j in rest):
            assert found is None
            found = S
    return np.array(found)


def test_topk_brute_force_tiny():
    rng = np.random.default_rng(7)
    for trial in range(30):
        n = int(rng.integers(1, 11))
        k = int(rng.integers(1, n + 1))
        v = rng.integers(-3, 4, n).astype(np.float32) * np.float32(0.5)  # many ties, zeros, signs
        got = orc.topk_select(v, k)
        assert np.array_equal(got, _brute_force_topk(v, k)), (v, k)


def test_topk_equals_python_sort():
    rng = np.random.default_rng(8)
    v = rng.standard_normal(500).astype(np.float32)
    v[rng.integers(0, 500, 60)] = np.float32(0.75)
    v[rng.integers(0, 500, 60)] = np.float32(-0.75)
    v[rng.integers(0, 500, 20)] = np.float32(-0.0)
    for k in (1, 7, 50, 137, 499, 500):
        want = sorted(sorted(range(500), key=lambda i: _order_key(v[i], i))[:k])
        assert np.array_equal(orc.topk_select(v, k), np.array(want))


def test_topk_degenerate_inputs():
    assert np.array_equal(orc.topk_select(np.zeros(10, np.float32), 4), np.arange(4))
    assert np.array_equal(orc.topk_select(np.full(10, -2.5, np.float32), 3), np.arange(3))
    v = np.array([0.0, -0.0, 0.0, 1.0], np.float32)
    assert np.array_equal(orc.topk_select(v, 3), np.array([0, 1, 3]))  # -0.0 ties with +0.0
    assert np.array_equal(orc.topk_select(v, 4), np.arange(4))
    assert orc.topk_count(1728, 100) == 17 and orc.topk_count(50, 100) == 1 and orc.topk_count(21630700, 1000) == 2163070


def test_topk_step_invariants():
    rng = np.random.default_rng(9)
    table = wl.make_table([("a", (13, 17)), ("v", (6,)), ("b", (8, 25))])
    layers = _layers(table)
    W = 3
    grads = np.zeros((W, table.stride), np.float32)
    err = np.zeros((W, table.stride), np.float32)
    for (off, r, c, k) in layers:
        grads[:, off:off + r * c] = rng.standard_normal((W, r * c))
        if k == orc.MATRIX:
            err[:, off:off + r * c] = 0.5 * rng.standard_normal((W, r * c))
    grads[:, 3] = grads[:, 40]  # some exact ties in the gradient
    level = [1, 0, 0]
    vals, idx, counts, out, e = orc.topk_step(grads, err, level, layers, 1000, 100)
    for l, (off, r, c, kind) in enumerate(layers):
        size = r * c
        if kind == orc.VECTOR:
            assert np.allclose(out[off:off + size], grads[:, off:off + size].astype(np.float64).mean(0))
            continue
        k = max(1, size * (1000 if level[l] else 100) // 10000)
        acc = np.zeros(size)
        for w in range(W):
            M = grads[w, off:off + size] + err[w, off:off + size]   # fp32 add
            assert M.dtype == np.float32
            assert counts[w, l] == k == len(idx[w][l]) == len(vals[w][l])
            assert np.all(np.diff(idx[w][l]) > 0)
            kept = np.zeros(size, bool); kept[idx[w][l]] = True
            assert np.abs(M[kept]).min() >= np.abs(M[~kept]).max()
            # bitwise error-feedback invariant: scatter(idx, val) + e' == M
            rec = e[w, off:off + size].copy()
            assert np.all(rec[kept].view(np.uint32) == 0)           # +0.0 exactly
            rec[idx[w][l]] = vals[w][l]
            assert np.array_equal(rec.view(np.uint32), M.view(np.uint32))
            acc[idx[w][l]] += vals[w][l].astype(np.float64)
        assert np.allclose(out[off:off + size], acc / W, rtol=0, atol=1e-15)


def test_topk_tie_at_threshold_keeps_lower_indices():
    v = np.array([1, 5, 1, 1, 7, 1, 1], np.float32)
    v[2] = -1
    assert np.array_equal(orc.topk_select(v, 4), np.array([0, 1, 2, 4]))


# ------------------------------------------------------------------ tables of the paper
def _golden():
    rows, params = [], []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            t = line.split()
            if t[0] == "params":
                params.append((t[1], int(t[2]), int(t[3])))
            else:
                rows.append((t[0], int(t[1]), t[2], t[3], float(t[4]), t[5]))
    return rows, params


def _table(model, classes):
    return wl.make_table(wl.shapes_resnet18(classes) if model == "resnet18" else wl.shapes_vgg19bn(classes))


def test_parameter_totals_match_appendix_g():
    _, params = _golden()
    assert len(params) == 3
    for model, classes, total in params:
        assert _table(model, classes).n_params == total
    assert wl.make_table(wl.shapes_lstm()).n_params == 50065078
    t = _table("resnet18", 100)
    assert int((t.kind == wl.MATRIX).sum()) == 21 and int((t.kind == wl.VECTOR).sum()) == 41


def test_data_sent_matches_tables():
    rows, _ = _golden()
    assert len(rows) == 7
    iters = 300 * 98
    for model, classes, comp, setting, value, unit in rows:
        table = _table(model, classes)
        layers = _layers(table)
        L = len(layers)
        if comp == "powersgd":
            r = int(setting[4:])
            per_it = orc.floats_sent_per_iteration(layers, [1] * L, "powersgd", 4, rank_low=r, rank_high=r)
            got = per_it * iters / 1e6
            assert abs(got - value) <= 0.11, (model, setting, got, value)  # printed to 0.1 M floats
        else:
            per_it = orc.floats_sent_per_iteration(layers, [1] * L, "topk", 4, topk_low_bp=1000)
            got = per_it * iters / 1e9
            assert abs(got - value) / value < 1e-3, (got, value)


# ------------------------------------------------------------------ optimiser tail
def _toy_table():
    return wl.make_table([("w0", (6, 5)), ("b0", (7,)), ("w1", (3, 9))])


@pytest.mark.parametrize("wd", [0.0, 5e-4])
def test_sgd_nesterov_matches_library_optimiser(wd):
    import torch
    table = _toy_table()
    layers = _layers(table)
    rng = np.random.default_rng(3)
    x0 = rng.standard_normal(table.stride)
    xs, us = x0.copy(), np.zeros(table.stride)
    ts = [torch.tensor(x0[o:o + r * c].copy(), dtype=torch.float64, requires_grad=True) for (o, r, c, k) in layers]
    opt = torch.optim.SGD(ts, lr=0.1, momentum=0.9, nesterov=True, weight_decay=wd)
    for step in range(4):
        d = rng.standard_normal(table.stride)
        xs, us = orc.sgd_nesterov(xs, us, d, layers, 0.1, 0.9, wd)
        for t, (o, r, c, k) in zip(ts, layers):
            t.grad = torch.tensor(d[o:o + r * c].copy(), dtype=torch.float64)
        opt.step()
        for t, (o, r, c, k) in zip(ts, layers):
            np.testing.assert_allclose(xs[o:o + r * c], t.detach().numpy(), rtol=1e-12, atol=1e-14)
    covered = np.zeros(table.stride, bool)
    for (o, r, c, k) in layers:
        covered[o:o + r * c] = True
    assert np.array_equal(xs[~covered], x0[~covered])  # padding untouched
    assert np.all(us[~covered] == 0.0)


def test_sgd_nesterov_closed_form_constant_gradient():
    table = wl.make_table([("w", (4, 4))])
    layers = _layers(table)
    g = np.full(table.stride, 2.0)
    x, u = np.zeros(table.stride), np.zeros(table.stride)
    lr, mu = 0.25, 0.5
    want_x = 0.0
    for t in range(1, 6):
        x, u = orc.sgd_nesterov(x, u, g, layers, lr, mu)
        want_u = 2.0 * (1.0 - mu ** t) / (1.0 - mu)  # geometric sum
        want_x -= lr * (2.0 + mu * want_u)
        assert np.allclose(u[:16], want_u, rtol=1e-14)
        assert np.allclose(x[:16], want_x, rtol=1e-14)
    # momentum 0 is plain gradient descent
    x, u = orc.sgd_nesterov(np.ones(table.stride), np.zeros(table.stride), g, layers, 0.1, 0.0)
    assert np.allclose(x[:16], 1.0 - 0.2) and np.allclose(u[:16], 2.0)


# ------------------------------------------------------------------ batch-size mode
def test_batch_accumulate_and_average_equal_the_mean_over_all_micro_batches():
    table = _toy_table()
    layers = _layers(table)
    rng = np.random.default_rng(5)
    W, n_accum = 3, 4
    micro = rng.standard_normal((n_accum, W, table.stride)).astype(np.float32)
    acc = rng.standard_normal((W, table.stride))  # stale content: the first micro-batch must overwrite it
    for j in range(n_accum):
        acc = orc.batch_accumulate(acc, micro[j], layers, first=(j == 0))
    out = orc.batch_average(acc, n_accum, layers)
    want = micro.astype(np.float64).mean(axis=(0, 1))
    for (o, r, c, k) in layers:
        np.testing.assert_allclose(out[o:o + r * c], want[o:o + r * c], rtol=1e-13, atol=1e-15)
        np.testing.assert_allclose(acc[:, o:o + r * c], micro.astype(np.float64).sum(axis=0)[:, o:o + r * c],
                                   rtol=1e-13, atol=1e-15)


def test_detect_batch_truth_table():
    n2 = np.array([9.0, 16.0])  # whole-model norm 5
    # (prev norm, lr_curr, lr_next, b_curr) -> (b_next, lr_scale); eta = 0.5, B_low = 512, B_high = 4096
    cases = [
        (10.0, 0.1, 0.1, 512, 512, 1.0),    # |10-5| = 5 >= 0.5*10 exactly: critical, stay small
        (6.0, 0.1, 0.1, 512, 4096, 8.0),    # |6-5| = 1 < 3: not critical, grow; LR x8 (512 -> 4096)
        (4.0, 0.1, 0.1, 512, 4096, 8.0),    # |4-5| = 1 < 2
        (2.0, 0.1, 0.1, 512, 512, 1.0),     # |2-5| = 3 >= 1: critical (growth counts)
        (6.0, 0.1, 0.01, 512, 512, 1.0),    # LR decay declares a critical regime
        (10.0, 0.1, 0.1, 4096, 4096, 8.0),  # critical, but the batch size is never decreased
        (6.0, 0.1, 0.01, 4096, 4096, 8.0),
        (0.0, 0.1, 0.1, 512, 512, 1.0),     # ||prev|| = 0
    ]
    for a, lc, ln, bc, want_b, want_s in cases:
        b, s, prev = orc.detect_batch(n2, a * a, lc, ln, 0.5, bc, 512, 4096)
        assert (b, s) == (want_b, want_s), (a, lc, ln, bc)
        assert prev == 25.0
    b, s, prev = orc.detect_batch(n2, -1.0, 0.1, 0.1, 0.5, 512, 512, 4096)
    assert (b, s, prev) == (512, 1.0, 25.0)  # no earlier window: the early phase is critical


def test_detect_batch_uses_the_whole_model_norm_not_the_layers():
    # layer 0 collapses (per-layer test: critical) but carries little of the whole-model norm
    prev_layers = np.array([1.0, 100.0])
    curr_layers = np.array([0.01, 100.0])
    lv, _ = orc.detect_regime(curr_layers, prev_layers, 0.1, 0.1, 0.5)
    assert lv[0] == orc.LOW and lv[1] == orc.HIGH
    b, s, _ = orc.detect_batch(curr_layers, float(prev_layers.sum()), 0.1, 0.1, 0.5, 128, 128, 1024)
    assert (b, s) == (1024, 8.0)
