"""Shared helpers of the parity tests: layout conversion between the oracle's natural shapes and
the library's buffers, and the comparison rules (bit-exact integers, relative Frobenius error on
floats)."""
import numpy as np
import torch

from oracle import accordion_oracle as orc

# Float tolerance of the parity tests: relative Frobenius error per layer, fp32 kernels against the
# fp64 oracle (the target stated for this path: <= 1e-4).
REL_TOL = 1e-4


def layers_of(table):
    return [(int(table.offset[l]), int(table.rows[l]), int(table.cols[l]), int(table.kind[l]))
            for l in range(table.n_layers)]


def rel_err(got, ref, floor=0.0):
    got = np.asarray(got, np.float64).ravel()
    ref = np.asarray(ref, np.float64).ravel()
    den = max(np.linalg.norm(ref), floor)
    if den == 0.0:
        return float(np.linalg.norm(got))
    return float(np.linalg.norm(got - ref) / den)


def q_list_from_buffer(ctx, q_buf, rank_low):
    """Library q buffer [q_rows, 4] -> oracle list of [m, rank_low] fp32 arrays."""
    qh = q_buf.detach().cpu().numpy()
    out = []
    for l in range(ctx.n_layers):
        if ctx.q_row[l] < 0:
            out.append(None)
        else:
            r0, m = int(ctx.q_row[l]), int(ctx.table.cols[l])
            out.append(qh[r0:r0 + m, :rank_low].copy())
    return out


def check_powersgd_against_oracle(ctx, table, grads, err_before, q_before, level, out, err_after, q_after, p_after,
                                  rank_low, rank_high, gs_eps, tol=REL_TOL):
    """Feeds the oracle the state the GPU step started from and compares every output per layer."""
    layers = layers_of(table)
    g = grads.cpu().numpy()
    e0 = err_before.cpu().numpy()
    lv = level.cpu().numpy()
    ql = q_list_from_buffer(ctx, q_before, rank_low)
    o_out, o_err, o_q, o_p = orc.powersgd_step(g, e0, ql, lv, layers, rank_low, rank_high, gs_eps)
    out_h, err_h = out.cpu().numpy(), err_after.cpu().numpy()
    q_h, p_h = q_after.cpu().numpy(), p_after.cpu().numpy()
    q0_h = q_before.cpu().numpy()
    worst = 0.0
    for l, (off, rows, cols, kind) in enumerate(layers):
        sl = slice(off, off + rows * cols)
        if kind == orc.VECTOR:
            e = rel_err(out_h[sl], o_out[sl])
            assert e <= tol, f"layer {l} (vector) out rel err {e}"
            continue
        r = rank_low if lv[l] else rank_high
        M = g[:, sl].astype(np.float64) + e0[:, sl].astype(np.float64)
        floor = 1e-6 * np.linalg.norm(M) / np.sqrt(M.shape[0])
        errs = {
            "out": rel_err(out_h[sl], o_out[sl], floor),
            "err": max(rel_err(err_h[w, sl], o_err[w, sl], floor) for w in range(g.shape[0])),
            "q": rel_err(q_h[ctx.q_row[l]:ctx.q_row[l] + cols, :r], o_q[l][:, :r]),
            "p_hat": rel_err(p_h[ctx.p_row[l]:ctx.p_row[l] + rows, :r], o_p[l]),
        }
        for name, e in errs.items():
            assert e <= tol, f"layer {l} ({rows}x{cols}, rank {r}) {name} rel err {e}"
            worst = max(worst, e)
        # ranks beyond r keep their previous contents, bit for bit
        qa = q_h[ctx.q_row[l]:ctx.q_row[l] + cols, r:]
        qb = q0_h[ctx.q_row[l]:ctx.q_row[l] + cols, r:]
        assert np.array_equal(qa.view(np.uint32), qb.view(np.uint32)), f"layer {l}: q columns beyond the rank changed"
    return worst


def check_topk_against_oracle(ctx, table, grads, err_before, level, vals, idx, counts, out, err_after,
                              low_bp, high_bp, tol=REL_TOL, layers_subset=None, workers_subset=None):
    """Bit-exact comparison of indices, packed value bits, counts and the new error memory; float
    comparison of the averaged output.  Subsets restrict the (slow) oracle to some layers/workers."""
    layers = layers_of(table)
    W = grads.shape[0]
    ws = list(range(W)) if workers_subset is None else list(workers_subset)
    g = grads.cpu().numpy()
    e0 = err_before.cpu().numpy()
    lv = level.cpu().numpy()
    vals_h, idx_h = vals.cpu().numpy(), idx.cpu().numpy()
    counts_h = counts.cpu().numpy().reshape(W, len(layers))
    out_h, err_h = out.cpu().numpy(), err_after.cpu().numpy()
    for l, (off, rows, cols, kind) in enumerate(layers):
        if layers_subset is not None and l not in layers_subset:
            continue
        sl = slice(off, off + rows * cols)
        sub_layers = [(0, rows, cols, kind)]
        o_vals, o_idx, o_counts, o_out, o_err = orc.topk_step(g[ws][:, sl], e0[ws][:, sl], [lv[l]], sub_layers,
                                                             low_bp, high_bp)
        if kind == orc.VECTOR:
            if workers_subset is None:
                assert rel_err(out_h[sl], o_out) <= tol, f"layer {l} (vector) out"
            assert np.all(counts_h[:, l] == 0)
            continue
        for j, w in enumerate(ws):
            k = int(o_counts[j, 0])
            assert counts_h[w, l] == k, f"layer {l} worker {w}: count {counts_h[w, l]} != {k}"
            s0 = w * ctx.capacity + int(ctx.seg_offset[l])
            assert np.array_equal(idx_h[s0:s0 + k], o_idx[j][0]), f"layer {l} worker {w}: indices differ"
            assert np.array_equal(vals_h[s0:s0 + k].view(np.uint32), o_vals[j][0].view(np.uint32)), \
                f"layer {l} worker {w}: packed value bits differ"
            assert np.array_equal(err_h[w, sl].view(np.uint32), o_err[j].view(np.uint32)), \
                f"layer {l} worker {w}: error memory bits differ"
        if workers_subset is None:
            floor = 1e-30
            e = rel_err(out_h[sl], o_out, floor)
            assert e <= tol, f"layer {l} out rel err {e}"


def device_state(ctx, table, W, seed=0, err_scale=0.0):
    g = torch.Generator(device="cuda").manual_seed(seed)
    err = torch.zeros(W, table.stride, device="cuda")
    if err_scale:
        err.normal_(generator=g).mul_(err_scale)
        mask = torch.zeros(table.stride, device="cuda")
        for l, sl in table.slices():
            if table.kind[l] == 0:
                mask[sl] = 1.0
        err.mul_(mask)
    return err
