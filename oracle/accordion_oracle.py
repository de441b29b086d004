"""CPU oracle for the Accordion gradient-compression step.  TEST INFRASTRUCTURE ONLY.

A plain, slow, obviously-correct numpy implementation of what the hot path
computes, written from the paper's statement of the method.  Only the test
suite, the smoke check and the benchmark's ``cpu_baseline`` / reference legs
may import it; the product (CUDA) path never does, and the two share no code.

Precision: fp64 from fp32 inputs everywhere, except the TopK error-feedback add,
which is one fp32 IEEE add because the packed values and every later selection
are compared bit for bit.

Besides the compression step the file holds the two extensions that follow it in the training
loop: the optimiser tail (Nesterov momentum) and the batch-size mode of the controller.

Conventions.  ``layers`` is a sequence of ``(offset, rows, cols, kind)`` with
``kind`` 0 = MATRIX (row-major ``rows x cols`` view: convolution weights as
``out x (in*k*k)``, the view that reproduces the "Data Sent" columns of Tables
1-2) and 1 = VECTOR (1-D tensors, which the compressors leave alone, Appendix F).
``grads`` and ``err`` are ``[W, stride]`` arrays; ``level[l]`` is 1 for the low
compression level (l_low) and 0 for the high compression level (l_high).

Every function is pinned by the CPU tests against closed forms, invariants,
library routines on special cases and brute force on tiny inputs; none is
"parity unpinned".
"""
from __future__ import annotations

import numpy as np

MATRIX = 0
VECTOR = 1
LOW = 1
HIGH = 0


# --------------------------------------------------------------------------- #
# Controller (Section 4.2, Algorithm 1)
# --------------------------------------------------------------------------- #
def accumulate(delta, grads_decider, layers):
    """Gradient accumulation over the detection window (Section 4.2, "Computational
    and memory overhead"): delta += g of the deciding worker, every layer."""
    for (off, rows, cols, kind) in layers:
        sl = slice(off, off + rows * cols)
        delta[sl] += grads_decider[sl].astype(np.float64)
    return delta


def layer_norms2(buf, layers):
    """Squared L2 (Frobenius) norm of each layer of one flat buffer (Section 4.2)."""
    out = np.zeros(len(layers), np.float64)
    for l, (off, rows, cols, kind) in enumerate(layers):
        x = buf[off:off + rows * cols].astype(np.float64)
        out[l] = float(np.sum(x * x))
    return out


def detect_regime(norm2_curr, norm2_prev, lr_curr, lr_next, eta):
    """Algorithm 1, per layer.  ``norm2_*`` are squared norms; a negative
    ``norm2_prev`` means "no earlier window".  Returns (level, new norm2_prev).

    level = LOW  iff  | ||D_prev|| - ||D_curr|| | >= eta * ||D_prev||   (Section 4.2 criterion,
                      in product form so that ||D_prev|| = 0 needs no division)
                 or   lr_next < lr_curr                               (declared after LR decay)
                 or   there is no previous window (the early phase is critical, Section 4.1).
    """
    L = len(norm2_curr)
    level = np.zeros(L, np.uint8)
    for l in range(L):
        if norm2_prev[l] < 0.0:
            level[l] = LOW
            continue
        a = np.sqrt(np.float64(norm2_prev[l]))
        b = np.sqrt(np.float64(norm2_curr[l]))
        critical = abs(a - b) >= np.float64(eta) * a
        level[l] = LOW if (critical or lr_next < lr_curr) else HIGH
    return level, np.array(norm2_curr, np.float64, copy=True)


def layer_diff_norms2(a, b, layers):
    """Squared L2 norm of (a - b) per layer."""
    out = np.zeros(len(layers), np.float64)
    for l, (off, rows, cols, kind) in enumerate(layers):
        d = a[off:off + rows * cols].astype(np.float64) - b[off:off + rows * cols].astype(np.float64)
        out[l] = float(np.sum(d * d))
    return out


def detect_regime_diff(norm2_diff, norm2_curr, norm2_prev, lr_curr, lr_next, eta):
    """Variant of the criterion with the norm of the DIFFERENCE of the two accumulated gradients,
    ||D_prev - D_curr|| / ||D_prev|| >= eta (a form in which the criterion is sometimes quoted; the paper's display
    equation and Algorithm 1 use the difference of the norms, which ``detect_regime`` implements).
    It needs the previous accumulated gradient itself, not only its norm.  Otherwise as Algorithm 1."""
    L = len(norm2_curr)
    level = np.zeros(L, np.uint8)
    for l in range(L):
        if norm2_prev[l] < 0.0:
            level[l] = LOW
            continue
        critical = np.sqrt(np.float64(norm2_diff[l])) >= np.float64(eta) * np.sqrt(np.float64(norm2_prev[l]))
        level[l] = LOW if (critical or lr_next < lr_curr) else HIGH
    return level, np.array(norm2_curr, np.float64, copy=True)


def layer_msdr(buf, layers):
    """Mean-to-standard-deviation ratio of each layer of one flat buffer: the statistic of the adaptive scheme
    the paper compares itself with (Section "Comparison with Prior Work"), which lowers the compression when
    the ratio has dropped.  The paper names the statistic only; taken here over the coordinates of a layer of
    the detector's accumulated gradient:

        mu = (1/n) sum_i x_i,   sd = sqrt((1/n) sum_i (x_i - mu)^2),   MSDR = |mu| / sd

    with MSDR = 0 when mu = 0 (also for an all-zero layer) and +inf when sd = 0 but mu != 0 (a constant layer).
    Returns (msdr[L], mean[L], std[L]) in fp64."""
    L = len(layers)
    msdr, mean, std = np.zeros(L), np.zeros(L), np.zeros(L)
    for l, (off, rows, cols, kind) in enumerate(layers):
        x = buf[off:off + rows * cols].astype(np.float64)
        mu = float(np.sum(x)) / x.size
        d = x - mu
        sd = float(np.sqrt(np.sum(d * d) / x.size))
        mean[l], std[l] = mu, sd
        if mu == 0.0:
            msdr[l] = 0.0
        elif sd == 0.0:
            msdr[l] = np.inf
        else:
            msdr[l] = abs(mu) / sd
    return msdr, mean, std


# --------------------------------------------------------------------------- #
# Error feedback (the "memory term": Section "Accordion with PowerSGD", Appendix A)
# --------------------------------------------------------------------------- #
def error_feedback(grads, err, layers, fp32=False):
    """M_w = g_w + e_w on MATRIX layers (VECTOR layers carry no memory: M = g)."""
    W = grads.shape[0]
    dt = np.float32 if fp32 else np.float64
    M = np.zeros(grads.shape, dt)
    for (off, rows, cols, kind) in layers:
        sl = slice(off, off + rows * cols)
        for w in range(W):
            if kind == MATRIX:
                M[w, sl] = grads[w, sl].astype(dt) + err[w, sl].astype(dt)
            else:
                M[w, sl] = grads[w, sl].astype(dt)
    return M


# --------------------------------------------------------------------------- #
# PowerSGD rank-r with error feedback
# --------------------------------------------------------------------------- #
def gram_schmidt(P, eps):
    """Modified Gram-Schmidt on the columns of P, in column order; each projection
    is taken against the already-updated column; divide by (norm + eps)."""
    P = np.array(P, np.float64, copy=True)
    r = P.shape[1]
    for c in range(r):
        for j in range(c):
            P[:, c] -= np.dot(P[:, j], P[:, c]) * P[:, j]
        P[:, c] /= (np.sqrt(np.dot(P[:, c], P[:, c])) + eps)
    return P


def powersgd_step(grads, err, q, level, layers, rank_low, rank_high, gs_eps=1e-8):
    """One PowerSGD step with error feedback on every MATRIX layer; plain mean on
    VECTOR layers.

    q: list with, per MATRIX layer, an ``[m, rank_low]`` warm-start matrix (None
    for VECTOR layers).  Steps per layer at rank r = rank_low if level==LOW else
    rank_high:  M_w = g_w + e_w;  P = mean_w M_w Q[:, :r];  P^ = GramSchmidt(P);
    Q[:, :r] = mean_w M_w^T P^;  A = P^ Q[:, :r]^T;  out = A;  e_w = M_w - A.

    Returns (out[stride], err_new[W, stride], q_new, p_hat) in fp64.
    """
    W, stride = grads.shape
    out = np.zeros(stride, np.float64)
    err_new = np.zeros((W, stride), np.float64)
    q_new, p_hat = [], []
    for l, (off, rows, cols, kind) in enumerate(layers):
        sl = slice(off, off + rows * cols)
        if kind == VECTOR:
            acc = np.zeros(rows * cols, np.float64)
            for w in range(W):
                acc += grads[w, sl].astype(np.float64)
            out[sl] = acc / W
            q_new.append(None)
            p_hat.append(None)
            continue
        r = rank_low if level[l] == LOW else rank_high
        Q = np.array(q[l], np.float64, copy=True)
        M = [grads[w, sl].astype(np.float64).reshape(rows, cols) + err[w, sl].astype(np.float64).reshape(rows, cols)
             for w in range(W)]
        P = np.zeros((rows, r), np.float64)
        for w in range(W):
            P += M[w] @ Q[:, :r]
        P /= W
        Ph = gram_schmidt(P, gs_eps)
        Qn = np.zeros((cols, r), np.float64)
        for w in range(W):
            Qn += M[w].T @ Ph
        Qn /= W
        Q[:, :r] = Qn
        A = Ph @ Qn.T
        out[sl] = A.reshape(-1)
        for w in range(W):
            err_new[w, sl] = (M[w] - A).reshape(-1)
        q_new.append(Q)
        p_hat.append(Ph)
    return out, err_new, q_new, p_hat


# --------------------------------------------------------------------------- #
# TopK-K% with error feedback
# --------------------------------------------------------------------------- #
def topk_count(size, k_bp):
    """Entries kept from a layer of ``size`` elements at K = k_bp basis points."""
    return max(1, (int(size) * int(k_bp)) // 10000)


def topk_select(m32, k):
    """Indices (ascending) of the k entries of largest |value| of the fp32 vector
    m32.  Order: larger magnitude first, compared as the 31-bit pattern of |value|
    (so -0.0 and +0.0 tie); among equal magnitudes the lower index first."""
    key = (m32.view(np.uint32) & np.uint32(0x7FFFFFFF)).astype(np.int64)
    order = np.argsort(-key, kind="stable")  # descending key, ties by ascending index
    return np.sort(order[:k])


def topk_step(grads, err, level, layers, topk_low_bp, topk_high_bp):
    """One TopK step with error feedback per MATRIX layer and worker; plain mean on
    VECTOR layers.  Returns (vals, idx, counts, out, err_new):

    vals[w][l], idx[w][l]: kept values (fp32, bit copies of M) and layer-local
    indices (int32), ascending index;  counts[w, l] = k;  out[stride] fp64 =
    (1/W) sum_w scatter(idx_w, val_w);  err_new[W, stride] fp32 = M_w with the kept
    entries replaced by +0.0.
    """
    W, stride = grads.shape
    L = len(layers)
    out = np.zeros(stride, np.float64)
    err_new = np.zeros((W, stride), np.float32)
    vals = [[None] * L for _ in range(W)]
    idx = [[None] * L for _ in range(W)]
    counts = np.zeros((W, L), np.int32)
    for l, (off, rows, cols, kind) in enumerate(layers):
        size = rows * cols
        sl = slice(off, off + size)
        if kind == VECTOR:
            acc = np.zeros(size, np.float64)
            for w in range(W):
                acc += grads[w, sl].astype(np.float64)
            out[sl] = acc / W
            continue
        k_bp = topk_low_bp if level[l] == LOW else topk_high_bp
        k = topk_count(size, k_bp)
        acc = np.zeros(size, np.float64)
        for w in range(W):
            m32 = (grads[w, sl].astype(np.float32) + err[w, sl].astype(np.float32)).astype(np.float32)
            keep = topk_select(m32, k)
            vals[w][l] = m32[keep].copy()
            idx[w][l] = keep.astype(np.int32)
            counts[w, l] = k
            e = m32.copy()
            e[keep] = np.float32(0.0)
            err_new[w, sl] = e
            acc[keep] += m32[keep].astype(np.float64)
        out[sl] = acc / W
    return vals, idx, counts, out, err_new


# --------------------------------------------------------------------------- #
# Communication accounting ("Data Sent" columns of Tables 1-4)
# --------------------------------------------------------------------------- #
def floats_sent_per_iteration(layers, level, compressor, n_workers, rank_low=2, rank_high=1,
                              topk_low_bp=1000, topk_high_bp=100):
    """Floats one iteration communicates.  PowerSGD: r*(n+m) per MATRIX layer plus
    every VECTOR element (all-reduced once).  TopK: values + indices (2 floats per
    kept entry) gathered from every worker, plus the VECTOR elements."""
    total = 0
    for l, (off, rows, cols, kind) in enumerate(layers):
        if kind == VECTOR:
            total += rows * cols
        elif compressor == "powersgd":
            r = rank_low if level[l] == LOW else rank_high
            total += r * (rows + cols)
        elif compressor == "topk":
            k_bp = topk_low_bp if level[l] == LOW else topk_high_bp
            total += 2 * topk_count(rows * cols, k_bp) * n_workers
        else:
            raise ValueError(compressor)
    return total


# --------------------------------------------------------------------------- #
# Optimiser tail (Appendix A, Table "Hyperparameters": Nesterov momentum 0.9)
# --------------------------------------------------------------------------- #
def sgd_nesterov(params, mom, d, layers, lr, momentum, weight_decay=0.0):
    """One SGD step with Nesterov momentum on every layer, from the averaged (decompressed) gradient ``d``:

        d' = d + weight_decay * x;   u <- momentum * u + d';   x <- x - lr * (d' + momentum * u)

    (the paper names the optimiser and the momentum only; this is the usual statement of it, with no
    dampening, and weight decay -- which the paper does not list -- added to the gradient when non-zero).
    Elements outside the layers (padding) are left alone.  Returns new (params, mom) in fp64."""
    x = np.array(params, np.float64, copy=True)
    u = np.array(mom, np.float64, copy=True)
    for (off, rows, cols, kind) in layers:
        sl = slice(off, off + rows * cols)
        dd = d[sl].astype(np.float64) + np.float64(weight_decay) * x[sl]
        u[sl] = np.float64(momentum) * u[sl] + dd
        x[sl] = x[sl] - np.float64(lr) * (dd + np.float64(momentum) * u[sl])
    return x, u


# --------------------------------------------------------------------------- #
# Batch-size mode (Section 4.2, last paragraph before "Computational and memory overhead";
# Section 5.1 "Hyperparameters"; Appendix A "Additional Details for Batch Size experiment")
# --------------------------------------------------------------------------- #
def batch_accumulate(acc, grads_micro, layers, first):
    """Large batches are simulated by several backward passes whose gradients are added up before anything
    is communicated (Appendix A): acc_w <- (0 if first else acc_w) + g_w for every worker and layer."""
    W = grads_micro.shape[0]
    a = np.array(acc, np.float64, copy=True)
    for (off, rows, cols, kind) in layers:
        sl = slice(off, off + rows * cols)
        for w in range(W):
            a[w, sl] = (0.0 if first else a[w, sl]) + grads_micro[w, sl].astype(np.float64)
    return a


def batch_average(acc, n_accum, layers):
    """Uncompressed exchange of the accumulated gradients (all-reduce, Section 5.1):
    out = (1 / (W * n_accum)) * sum_w acc_w, the mean over workers of the mean over the micro-batches."""
    W, stride = acc.shape
    out = np.zeros(stride, np.float64)
    for (off, rows, cols, kind) in layers:
        sl = slice(off, off + rows * cols)
        s = np.zeros(rows * cols, np.float64)
        for w in range(W):
            s += acc[w, sl].astype(np.float64)
        out[sl] = s / (W * n_accum)
    return out


def detect_batch(norm2_layers, norm2_prev, lr_curr, lr_next, eta, b_curr, b_low, b_high):
    """Algorithm 1 at the granularity of the whole model (batch size is one setting for all layers): the
    statistic is the norm of the whole accumulated gradient, ||D||^2 = sum over layers of ||D[l]||^2; the
    small batch B_low takes the place of the low compression level and B_high of the high one.  The batch
    size is only ever increased (Appendix A), so a critical regime found while already at B_high leaves
    it there.  The learning rate scales in the same ratio as the batch size (Section 5.1).

    ``norm2_prev`` < 0 means "no earlier window".  Returns (b_next, lr_scale, new norm2_prev) where
    lr_scale = b_next / b_low multiplies the learning rate that belongs to B_low."""
    curr = float(np.sum(np.asarray(norm2_layers, np.float64)))
    if norm2_prev < 0.0:
        critical = True
    else:
        a = np.sqrt(np.float64(norm2_prev))
        b = np.sqrt(np.float64(curr))
        critical = bool(abs(a - b) >= np.float64(eta) * a) or (lr_next < lr_curr)
    want = b_low if critical else b_high
    b_next = max(int(b_curr), int(want))
    return b_next, float(b_next) / float(b_low), curr
