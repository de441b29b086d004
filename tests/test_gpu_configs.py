"""The five benchmark configurations on the GPU against the oracle.

Protocol.  TopK and the controller are bit-reproducible, so they run free over the iterations and must
match exactly (levels, indices, counts, packed value bits, error memory).  PowerSGD is compared per step
from synchronised state: the oracle is fed the GPU's own error memory, Q and levels from just before
the call (fp32 and fp64 trajectories may drift apart through the memory when singular values are
close).  Reduced-size versions of each configuration run many iterations across a scale jump; the
full-size versions run a few steps in the launch configuration bench.py times (lazy residual), with
the oracle restricted to sampled layers / workers where it would otherwise take minutes."""
import numpy as np
import pytest
import torch

from oracle import accordion_oracle as orc
from paper_2010_16248_b200 import binding, pipeline, workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu


class OracleController:
    """Oracle-side mirror of the detection cadence (accumulate, norms, Algorithm 1 every check_every)."""

    def __init__(self, table, check_every, eta):
        self.layers = H.layers_of(table)
        self.delta = np.zeros(table.stride)
        self.prev = -np.ones(table.n_layers)
        self.level = np.ones(table.n_layers, np.uint8)
        self.check_every, self.eta, self.t = check_every, eta, 0

    def step(self, g_decider, lr_curr=0.1, lr_next=0.1):
        orc.accumulate(self.delta, g_decider, self.layers)
        self.t += 1
        if self.t % self.check_every == 0:
            n2 = orc.layer_norms2(self.delta, self.layers)
            self.level, self.prev = orc.detect_regime(n2, self.prev, lr_curr, lr_next, np.float32(self.eta))
            self.delta[:] = 0


def _run_config(w, iters, t0=0, lazy=False, topk_layers=None, topk_workers=None, psgd_check=None, topk_check=None,
                force_level=None, paths_seen=None, extra_flags=0):
    """Runs `iters` iterations of workload `w` starting at stream iteration t0; checks every level decision
    exactly, the TopK steps listed in topk_check and the PowerSGD steps listed in psgd_check (default: all).  With
    lazy=True a second engine in lazy-residual mode (the mode bench.py times) runs in lockstep and must
    reproduce the eager engine's outputs (out, Q, P^; packed TopK sets) bit for bit at every step, and its error
    memories after a final flush.  force_level (0 / 1) starts every engine, and the oracle's controller, at that
    level instead of the initial low-compression level.  paths_seen (a set) collects the TopK selection paths the
    lazy engine (else the eager one) took.  extra_flags: further ACC_FLAG_* bits for both engines (e.g. forcing one
    implementation of the first PowerSGD pass)."""
    table, W = w.table, w.n_workers
    stream = wl.GradientStream(w, device="cuda")
    eng = pipeline.AccordionStep(table, W, w.compressors, w.rank_low, w.rank_high, w.topk_low_bp, w.topk_high_bp,
                                 w.eta, 1e-8, w.check_every, extra_flags=extra_flags)
    lz = None
    if lazy:
        lz = pipeline.AccordionStep(table, W, w.compressors, w.rank_low, w.rank_high, w.topk_low_bp, w.topk_high_bp,
                                    w.eta, 1e-8, w.check_every, lazy_residual=True, extra_flags=extra_flags)
    ctl = OracleController(table, w.check_every, w.eta)
    if force_level is not None:
        for e in (eng, lz):
            if e is not None:
                e.level.fill_(force_level)
        ctl.level[:] = force_level
    seen_levels = set()
    for i in range(iters):
        grads = stream.grads(t0 + i)
        level_before = eng.level.clone()
        assert np.array_equal(level_before.cpu().numpy(), ctl.level), f"iteration {i}: levels differ"
        seen_levels.update(int(x) for x in ctl.level[table.kind == wl.MATRIX])
        if "powersgd" in w.compressors:
            e0, q0 = eng.err_psgd.clone(), eng.q.clone()
        if "topk" in w.compressors:
            et0 = eng.err_topk.clone()
        eng.step(grads)
        if lz is not None:
            lz.step(grads)
        torch.cuda.synchronize()
        if lz is not None:
            assert torch.equal(lz.level, eng.level)
            names = (("out_psgd", "q", "p_hat") if "powersgd" in w.compressors else ()) + \
                    (("out_topk", "vals", "idx", "counts") if "topk" in w.compressors else ())
            for name in names:
                assert torch.equal(getattr(lz, name), getattr(eng, name)), f"iteration {i}: lazy {name} differs"
        if "powersgd" in w.compressors and (psgd_check is None or i in psgd_check):
            H.check_powersgd_against_oracle(eng.ctx, table, grads, e0, q0, level_before, eng.out_psgd, eng.err_psgd,
                                            eng.q, eng.p_hat, w.rank_low, w.rank_high, 1e-8)
        if "topk" in w.compressors and (topk_check is None or i in topk_check):
            H.check_topk_against_oracle(eng.ctx, table, grads, et0, level_before, eng.vals, eng.idx, eng.counts,
                                        eng.out_topk, eng.err_topk, w.topk_low_bp, w.topk_high_bp,
                                        layers_subset=topk_layers, workers_subset=topk_workers)
        if paths_seen is not None and "topk" in w.compressors:
            paths_seen.update(int(p) for p in (lz or eng).ctx.acc_topk_last_paths().ravel())
        ctl.step(grads[0].cpu().numpy())
    if lz is not None:
        lz.flush()
        torch.cuda.synchronize()
        for name in (("err_psgd",) if "powersgd" in w.compressors else ()) + \
                (("err_topk",) if "topk" in w.compressors else ()):
            assert torch.equal(getattr(lz, name), getattr(eng, name)), f"flushed lazy {name} differs from the eager one"
    return seen_levels


# ------------------------------------------------------------------ config 1, full size, all 20 iterations
def test_config1_full_run():
    w = wl.workload(1)
    levels = []
    table, W = w.table, w.n_workers
    stream = wl.GradientStream(w, device="cuda")
    eng = pipeline.AccordionStep(table, W, w.compressors, w.rank_low, w.rank_high, w.topk_low_bp, w.topk_high_bp,
                                 w.eta, 1e-8, w.check_every)
    ctl = OracleController(table, w.check_every, w.eta)
    worst = 0.0
    for t in range(w.n_iters):
        grads = stream.grads(t)
        lv = eng.level.clone()
        levels.append(int(lv[0]))
        assert np.array_equal(lv.cpu().numpy(), ctl.level)
        e0, q0, et0 = eng.err_psgd.clone(), eng.q.clone(), eng.err_topk.clone()
        eng.step(grads)
        torch.cuda.synchronize()
        worst = max(worst, H.check_powersgd_against_oracle(eng.ctx, table, grads, e0, q0, lv, eng.out_psgd,
                                                           eng.err_psgd, eng.q, eng.p_hat, w.rank_low, w.rank_high,
                                                           1e-8))
        H.check_topk_against_oracle(eng.ctx, table, grads, et0, lv, eng.vals, eng.idx, eng.counts, eng.out_topk,
                                    eng.err_topk, w.topk_low_bp, w.topk_high_bp)
        ctl.step(grads[0].cpu().numpy())
    # known answer of the schedule: the detector lags the scale jump at iteration 10 by one window
    assert levels == [1] * 10 + [0] * 5 + [1] * 5
    assert int(eng.level[0]) == 0 and worst < H.REL_TOL


# ------------------------------------------------------------------ reduced-size configs across a scale jump
@pytest.mark.parametrize("config,scale", [(2, 4), (3, 4), (4, 4), (5, 16)])
def test_reduced_configs_across_scale_jump(config, scale):
    w = wl.workload(config, scale=scale)
    # iterations 80..119 of the schedule: windows [80,90) [90,100) equal -> HIGH, jump at 100 -> LOW at 110
    seen = _run_config(w, iters=40, t0=80, psgd_check=set(range(0, 40, 3)) | {19, 20, 21, 29, 30, 31, 39})
    assert seen == {0, 1}, "both compression levels must have been exercised"


@pytest.mark.parametrize("config,scale", [(2, 4), (3, 4), (4, 4), (5, 16)])
def test_reduced_configs_second_jump_and_last_iteration(config, scale):
    """The scale jump at iteration 150 and the end of the schedule.  From iteration 140: the windows [140,150) and
    [150,160) differ by the jump (low level), [150,160) and [160,170) do not (high level from step 30).  Then the
    last 25 iterations of the configuration, which end at the high level on its final iteration."""
    w = wl.workload(config, scale=scale)
    seen = _run_config(w, iters=35, t0=140, psgd_check={0, 9, 10, 11, 19, 20, 21, 29, 30, 31, 34},
                       topk_check={0, 9, 10, 11, 19, 20, 21, 29, 30, 31, 34})
    assert seen == {0, 1}
    seen = _run_config(w, iters=25, t0=w.n_iters - 25, psgd_check={0, 19, 20, 21, 24}, topk_check={0, 19, 20, 21, 24})
    assert seen == {0, 1}


@pytest.mark.parametrize("config,scale", [(2, 4), (3, 4), (5, 16)])
def test_reduced_configs_lazy_residual(config, scale):
    w = wl.workload(config, scale=scale)
    _run_config(w, iters=25, t0=90, lazy=True, psgd_check=set(range(25)))


# ------------------------------------------------------------------ full-size configs, bench launch configuration
@pytest.mark.parametrize("config", [2, 4])
def test_full_size_powersgd(config):
    w = wl.workload(config)
    _run_config(w, iters=3, t0=0, lazy=True)


def test_full_size_config3_topk():
    w = wl.workload(3)
    big = [l for l in range(w.table.n_layers) if w.table.kind[l] == wl.MATRIX]
    # every matrix layer for worker 0, plus all workers on the first conv, the largest conv and the classifier
    _run_config(w, iters=2, t0=0, topk_workers=[0])
    sizes = w.table.sizes
    sample = [big[0], int(np.argmax(sizes)), big[-1]]
    _run_config(w, iters=3, t0=0, lazy=True, topk_layers=sample)


def test_full_size_config5_sampled():
    """LSTM set, W = 8: PowerSGD (lazy) checked on every layer for two steps; TopK checked on the row-sparse
    encoder (k exceeds its non-zeros: filled with zeros by lowest index), one gate matrix and the decoder
    for two workers."""
    w = wl.workload(5)
    names = w.table.names
    sample = [names.index("encoder.weight"), names.index("rnn.weight_hh_l1"), names.index("decoder.weight")]
    _run_config(w, iters=2, t0=0, lazy=True, topk_layers=sample, topk_workers=[0, 5])


# ------------------------------------------------------------------ full size, the steady state bench.py times
def test_full_size_config3_high_level_steady_state():
    """ResNet-18 set, TopK at K = 1 % on every layer for six steps in a row, lazy residual (what the benchmark runs for
    most of its steps): the threshold predictions engage from the second step, whole entries are staged from the
    third.  Every step must equal the eager engine's bit for bit; steps 2 and 5 are checked against the oracle on
    every MATRIX layer for one worker and on three layers for all workers."""
    w = wl.workload(3)
    mats = [l for l in range(w.table.n_layers) if w.table.kind[l] == wl.MATRIX]
    paths = set()
    _run_config(w, iters=6, t0=20, lazy=True, topk_workers=[1], topk_check={2, 5}, force_level=0, paths_seen=paths)
    assert binding.ACC_TOPK_PATH_STAGED in paths, paths  # (the predicted-list path belongs to config 5's encoder)
    sample = [mats[0], int(np.argmax(w.table.sizes)), mats[-1]]
    _run_config(w, iters=4, t0=20, lazy=True, topk_layers=sample, topk_check={3}, force_level=0)


def test_full_size_config5_high_level_steady_state():
    """LSTM set, W = 8, both compressors at the high compression level (rank 1, K = 1 %) for six steps, lazy
    residual: the pipelined first PowerSGD pass subtracts the pending rank-1 residual while loading, TopK runs on
    staged entries (gate matrices, decoder) and on the predicted list (the row-sparse encoder).  Lazy must equal
    eager at every step; PowerSGD is checked against the oracle on every layer at steps 1 and 5, TopK at step 5 on
    the encoder, a gate matrix and the decoder for two workers."""
    w = wl.workload(5)
    names = w.table.names
    sample = [names.index("encoder.weight"), names.index("rnn.weight_ih_l1"), names.index("decoder.weight")]
    paths = set()
    _run_config(w, iters=6, t0=20, lazy=True, topk_layers=sample, topk_workers=[2, 7], psgd_check={1, 5},
                topk_check={5}, force_level=0, paths_seen=paths)
    assert binding.ACC_TOPK_PATH_STAGED in paths and binding.ACC_TOPK_PATH_LIST_PREDICTED in paths, paths


@pytest.mark.parametrize("first_pass", [binding.ACC_FLAG_PIPELINE_NEVER, binding.ACC_FLAG_PIPELINE_ALWAYS])
def test_full_size_config4_high_level_pending_residual(first_pass):
    """VGG-19bn set, W = 8, rank 1 on every layer with the lazy residual pending from step to step, with the direct
    and with the pipelined first pass: the lazy engine must equal the eager one bit for bit at every step (the two
    implementations of the pass differ from each other in the last bits: they sum the partial rows of P in
    different orders); the oracle checks steps 1 and 3."""
    w = wl.workload(4)
    _run_config(w, iters=4, t0=20, lazy=True, psgd_check={1, 3}, force_level=0, extra_flags=first_pass)


def test_graph_replay_matches_direct_calls():
    """An iteration captured as CUDA graphs (one per gradient buffer, with and without the regime check)
    must leave exactly the same state as the same iterations issued call by call."""
    w = wl.workload(5, scale=16)
    table, W = w.table, w.n_workers
    stream = wl.GradientStream(w, device="cuda")
    ring = [stream.grads(t) for t in range(3)]
    engines = [pipeline.AccordionStep(table, W, w.compressors, w.rank_low, w.rank_high, w.topk_low_bp,
                                      w.topk_high_bp, w.eta, 1e-8, 4, lazy_residual=True) for _ in range(2)]
    engines[1].capture_graphs(ring)
    levels_after_decay = None
    for i in range(14):  # crosses three regime checks; the second one sees a learning-rate decay (Algorithm 1)
        lr = (0.1, 0.01) if i == 7 else (0.1, 0.1) if i < 7 else (0.01, 0.01)
        engines[0].step(ring[i % 3], *lr)
        engines[1].step_graph(i % 3, *lr)
        if i == 7:
            torch.cuda.synchronize()
            levels_after_decay = engines[1].level.clone()
    torch.cuda.synchronize()
    assert int(levels_after_decay.min()) == 1, "a learning-rate decay declares every layer critical"
    a, b = engines
    for name in ("level", "delta", "norm2_prev", "err_psgd", "q", "p_hat", "out_psgd", "err_topk", "vals", "idx",
                 "counts", "out_topk"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name
    assert a.launches == b.launches and a.ctx.acc_device_status() == 0 and b.ctx.acc_device_status() == 0
    assert set(int(x) for x in a.level.cpu()) <= {0, 1}
