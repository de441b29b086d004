"""Sequencing of the C-ABI calls for one training run: state buffers and the detection cadence.

``AccordionStep`` owns the persistent state of the path (error memories, PowerSGD factors, the
detector's accumulator and norms, the per-layer level array) as device tensors and issues, per
iteration, the compressor step(s) and -- every ``check_every`` iterations -- the norm and regime
kernels (Section 4.2: accumulate during the window, take norms at its end, Algorithm 1).  All
arithmetic happens in the library's kernels; nothing here reads results back to the host.
"""
from __future__ import annotations

from typing import Optional, Sequence

import torch

from . import binding
from . import workloads as wl


class AccordionStep:
    def __init__(self, table: wl.LayerTable, n_workers: int, compressors: Sequence[str] = ("powersgd",),
                 rank_low=2, rank_high=1, topk_low_bp=1000, topk_high_bp=100, eta=0.5, gs_eps=1e-8,
                 check_every=10, decider=0, q_init=None, device="cuda", lazy_residual=False, optimizer=None,
                 extra_flags=0, overlap=True, share_sms=False):
        """``overlap``: with two compressors, the TopK step runs on a second stream beside the PowerSGD step
        (they share only the gradients and the level array, both read-only), so that the short, latency-bound
        kernels of one hide behind the streaming kernels of the other; the results are the same bits.
        ``share_sms``: with ``overlap``, the pipelined first PowerSGD pass leaves half of the SMs to the TopK step
        (ACC_FLAG_SHARE_SMS: the whole step gets a few percent faster, that kernel alone slower).
        ``extra_flags``: further ACC_FLAG_* bits for the context (e.g. forcing one implementation of the first
        PowerSGD pass).  ``optimizer``: None, or a dict ``{"params": tensor [stride], "lr": .., "momentum": 0.9,
        "weight_decay": 0.0}``: the Nesterov update (Appendix A) is then applied to ``params`` by the kernels
        that produce the averaged gradient (one compressor only)."""
        self.table, self.W = table, n_workers
        self.compressors = tuple(compressors)
        if optimizer is not None and len(self.compressors) != 1:
            raise ValueError("the optimiser tail belongs to one compressor's output")
        self.check_every = check_every
        self.device = torch.device(device)
        self.ctx = binding.Context(table, n_workers, device=device, rank_low=rank_low, rank_high=rank_high,
                                   topk_low_bp=topk_low_bp, topk_high_bp=topk_high_bp, eta=eta, gs_eps=gs_eps,
                                   decider=decider,
                                   flags=(binding.ACC_FLAG_LAZY_RESIDUAL if lazy_residual else 0) | extra_flags |
                                   (binding.ACC_FLAG_SHARE_SMS if share_sms and overlap and len(compressors) == 2
                                    else 0))
        dev, L, stride = self.device, table.n_layers, table.stride
        self.level = torch.ones(L, dtype=torch.uint8, device=dev)  # before the first check: low compression
        self.delta = torch.zeros(stride, device=dev)
        self.norm2_curr = torch.zeros(L, dtype=torch.float64, device=dev)
        self.norm2_prev = torch.full((L,), -1.0, dtype=torch.float64, device=dev)
        self.t = 0
        self.launches = 0
        # the detector's learning-rate pair as device scalars (Algorithm 1 declares a critical regime when the rate
        # is about to decay): the captured iteration reads them, ``set_detector_lr`` rewrites them between replays
        self.lr_pair = torch.tensor([0.1, 0.1], dtype=torch.float32, device=dev)
        self._lr_pair_host = (0.1, 0.1)
        self._lr_from_device = False
        self.lazy_residual = lazy_residual
        self.overlap = overlap
        self._side = torch.cuda.Stream(device=dev)
        self._fork, self._join = torch.cuda.Event(), torch.cuda.Event()
        self.params = self.mom = self.hyper = None
        if optimizer is not None:
            self.params = optimizer["params"]
            self.mom = torch.zeros(stride, device=dev)
            self.hyper = torch.tensor([optimizer["lr"], optimizer.get("momentum", 0.9),
                                       optimizer.get("weight_decay", 0.0)], dtype=torch.float32, device=dev)
        if "powersgd" in self.compressors:
            self.err_psgd = torch.zeros(n_workers, stride, device=dev)
            self.q = self.ctx.new_q(q_init if q_init is not None else wl.initial_q(table, rank_low, device=dev))
            self.p_hat = self.ctx.new_p()
            self.out_psgd = torch.zeros(stride, device=dev)
        if "topk" in self.compressors:
            self.err_topk = torch.zeros(n_workers, stride, device=dev)
            self.vals, self.idx, self.counts = self.ctx.new_topk_buffers()
            self.out_topk = torch.zeros(stride, device=dev)

    def step(self, grads: torch.Tensor, lr_curr: float = 0.1, lr_next: float = 0.1, stream=None):
        """One iteration on device-resident gradients ``[W, stride]``."""
        c = self.ctx
        delta: Optional[torch.Tensor] = self.delta  # accumulated once per iteration, by the first compressor
        if self.overlap and len(self.compressors) == 2:
            main = stream if stream is not None else torch.cuda.current_stream(self.device)
            self._fork.record(main)
            self._side.wait_event(self._fork)
            c.acc_topk_step(grads, self.err_topk, self.level, self.vals, self.idx, self.counts, self.out_topk,
                            None, self._side)
            self.launches += c.last_launch_count()
            c.acc_powersgd_step(grads, self.err_psgd, self.q, self.p_hat, self.level, self.out_psgd, delta, main)
            self.launches += c.last_launch_count()
            self._join.record(self._side)
            main.wait_event(self._join)
            self.t += 1
            if self.t % self.check_every == 0:
                c.acc_layer_norms(self.delta, 1, self.norm2_curr, stream=main)
                self.launches += c.last_launch_count()
                self._detect(lr_curr, lr_next, main)
            return
        if "powersgd" in self.compressors:
            if self.params is not None:
                c.acc_powersgd_step_sgd(grads, self.err_psgd, self.q, self.p_hat, self.level, self.out_psgd, delta,
                                        self.params, self.mom, self.hyper, stream)
            else:
                c.acc_powersgd_step(grads, self.err_psgd, self.q, self.p_hat, self.level, self.out_psgd, delta,
                                    stream)
            self.launches += c.last_launch_count()
            delta = None
        if "topk" in self.compressors:
            if self.params is not None:
                c.acc_topk_step_sgd(grads, self.err_topk, self.level, self.vals, self.idx, self.counts,
                                    self.out_topk, delta, self.params, self.mom, self.hyper, stream)
            else:
                c.acc_topk_step(grads, self.err_topk, self.level, self.vals, self.idx, self.counts, self.out_topk,
                                delta, stream)
            self.launches += c.last_launch_count()
        self.t += 1
        if self.t % self.check_every == 0:
            c.acc_layer_norms(self.delta, 1, self.norm2_curr, stream=stream)
            self.launches += c.last_launch_count()
            self._detect(lr_curr, lr_next, stream)

    def _detect(self, lr_curr, lr_next, stream):
        if self._lr_from_device:
            self.ctx.acc_detect_regime_lr(self.norm2_curr, self.norm2_prev, self.lr_pair, self.level, self.delta, stream)
        else:
            self.ctx.acc_detect_regime(self.norm2_curr, self.norm2_prev, lr_curr, lr_next, self.level, self.delta,
                                       stream)
        self.launches += self.ctx.last_launch_count()

    def set_detector_lr(self, lr_curr: float, lr_next: float):
        """Learning rates the captured regime test will see (current iteration's and the next one's)."""
        pair = (float(lr_curr), float(lr_next))
        if pair != self._lr_pair_host:
            self.lr_pair[0:1].fill_(pair[0])
            self.lr_pair[1:2].fill_(pair[1])
            self._lr_pair_host = pair

    def flush(self, stream=None):
        """Lazy mode: materialises the error memories (what the last step compressed is removed from ``err``), so
        that the state buffers can be read, saved or copied into another engine.  A no-op in eager mode."""
        if not self.lazy_residual:
            return
        if "powersgd" in self.compressors:
            self.ctx.acc_powersgd_flush(self.err_psgd, self.q, self.p_hat, stream)
        if "topk" in self.compressors:
            self.ctx.acc_topk_flush(self.err_topk, stream)

    def set_lr(self, lr: float):
        """Learning rate of the optimiser tail: a device scalar the kernels read, so captured graphs follow it."""
        self.hyper[0:1].fill_(float(lr))

    def capture_graphs(self, grads_buffers, lr_curr: float = 0.1, lr_next: float = 0.1):
        """Captures one iteration as CUDA graphs, for each of the given fixed device gradient buffers (the
        caller refills them, or cycles through them, before every replay): one graph for an ordinary
        iteration and one for an iteration that ends a detection window (with the norm and regime kernels).
        Which rank or K a layer gets is decided on the device from ``level``, and the regime test reads its two
        learning rates from device scalars, so the same graphs serve every iteration of a schedule.
        ``step_graph(slot, lr_curr, lr_next)`` replays the right one.  Every library call is asynchronous and
        allocation-free, hence capturable."""
        torch.cuda.synchronize(self.device)
        self.set_detector_lr(lr_curr, lr_next)
        self._lr_from_device = True
        saved_t, saved_launches = self.t, self.launches
        side = torch.cuda.Stream(device=self.device)
        self._graphs, self._graph_launches = [], []
        with torch.cuda.stream(side):
            for grads in grads_buffers:
                pair, counts = [], []
                for with_check in (False, True):
                    g = torch.cuda.CUDAGraph()
                    self.t = self.check_every - 1 if with_check else 0
                    before = self.launches
                    with torch.cuda.graph(g, stream=side):
                        self.step(grads, lr_curr, lr_next, stream=side)
                    pair.append(g)
                    counts.append(self.launches - before)
                self._graphs.append(pair)
                self._graph_launches.append(counts)
        torch.cuda.synchronize(self.device)
        self._lr_from_device = False
        self.t, self.launches = saved_t, saved_launches

    def step_graph(self, slot: int = 0, lr_curr: Optional[float] = None, lr_next: Optional[float] = None):
        """Replays the captured iteration that reads gradient buffer ``slot`` (see ``capture_graphs``); the learning
        rates, when given, are what the regime test of this iteration sees (unchanged otherwise)."""
        self.t += 1
        which = 1 if self.t % self.check_every == 0 else 0
        if which and lr_curr is not None and lr_next is not None:
            self.set_detector_lr(lr_curr, lr_next)
        self._graphs[slot][which].replay()
        self.launches += self._graph_launches[slot][which]

    def outputs(self):
        outs = []
        if "powersgd" in self.compressors:
            outs.append(self.out_psgd)
        if "topk" in self.compressors:
            outs.append(self.out_topk)
        return outs


class BatchSizeStep:
    """Batch-size mode of the controller (Section 4.2, Appendix A): every backward pass adds its gradients to
    per-worker accumulators; after ``n_accum = batch / micro_batch`` passes the accumulators are averaged
    (the uncompressed exchange), optionally straight into the Nesterov update; at the end of every detection
    window the whole-model norm of the accumulated decider gradient goes through Algorithm 1, which picks
    B_low or B_high (never decreasing) and the matching learning-rate scale.  All arithmetic runs in the
    library's kernels; the host reads back one integer per window (the batch size steers its loop)."""

    def __init__(self, table: wl.LayerTable, n_workers: int, b_low: int, b_high: int, micro_batch: int, eta=0.5,
                 decider=0, device="cuda", optimizer=None):
        if b_low % micro_batch or b_high % micro_batch:
            raise ValueError("batch sizes must be multiples of the micro-batch")
        self.table, self.W = table, n_workers
        self.b_low, self.b_high, self.micro_batch = b_low, b_high, micro_batch
        self.device = dev = torch.device(device)
        self.ctx = binding.Context(table, n_workers, device=device, eta=eta, decider=decider)
        stride, L = table.stride, table.n_layers
        self.acc = torch.zeros(n_workers, stride, device=dev)
        self.delta = torch.zeros(stride, device=dev)
        self.out = torch.zeros(stride, device=dev)
        self.norm2_layers = torch.zeros(L, dtype=torch.float64, device=dev)
        self.norm2_prev = torch.full((1,), -1.0, dtype=torch.float64, device=dev)
        self.batch = torch.tensor([b_low], dtype=torch.int32, device=dev)  # the early phase is critical
        self.lr_scale = torch.ones(1, device=dev)
        self.pending = 0
        self.params = self.mom = self.hyper = None
        if optimizer is not None:
            self.params = optimizer["params"]
            self.mom = torch.zeros(stride, device=dev)
            self.hyper = torch.tensor([optimizer["lr"], optimizer.get("momentum", 0.9),
                                       optimizer.get("weight_decay", 0.0)], dtype=torch.float32, device=dev)

    def micro_step(self, grads: torch.Tensor, stream=None):
        """One backward pass worth of gradients ``[W, stride]`` (device)."""
        self.ctx.acc_batch_accumulate(grads, self.acc, self.delta, first=(self.pending == 0), stream=stream)
        self.pending += 1

    def apply(self, stream=None):
        """Ends the large batch: averages what was accumulated (and updates the parameters if asked)."""
        self.ctx.acc_batch_average(self.acc, self.pending, self.out, self.params, self.mom, self.hyper, stream)
        self.pending = 0
        return self.out

    def check(self, lr_curr: float, lr_next: float, stream=None) -> int:
        """End of a detection window; returns the batch size to use from now on."""
        self.ctx.acc_layer_norms(self.delta, 1, self.norm2_layers, stream=stream)
        self.ctx.acc_detect_batch(self.norm2_layers, self.norm2_prev, lr_curr, lr_next, self.b_low, self.b_high,
                                  self.batch, self.lr_scale, self.delta, stream)
        return int(self.batch.item())


def _layer_groups(table: wl.LayerTable, n_groups: int):
    """Contiguous runs of layers with about equal parameter counts (at least one layer each): the k-th cut falls
    at the layer boundary whose cumulative size is nearest to k / n_groups of the total."""
    sizes = [int(x) for x in table.sizes]
    L = table.n_layers
    n_groups = max(1, min(int(n_groups), L))
    cum, run = [], 0
    for sz in sizes:
        run += sz
        cum.append(run)
    cuts, lo = [], 0
    for k in range(1, n_groups):
        want = run * k / n_groups
        hi = L - (n_groups - k)  # leave a layer for each later group
        best = min(range(lo, hi), key=lambda l: abs(cum[l] - want))
        cuts.append(best + 1)
        lo = best + 1
    edges = [0] + cuts + [L]
    return [list(range(edges[i], edges[i + 1])) for i in range(n_groups)]


def _sub_table(table: wl.LayerTable, ids) -> wl.LayerTable:
    """The layers ``ids`` of ``table`` at their offsets inside the same flat per-worker buffer."""
    import numpy as np
    ids = list(ids)
    return wl.LayerTable([table.names[l] for l in ids], np.asarray(table.offset[ids], np.int64),
                         np.asarray(table.rows[ids], np.int32), np.asarray(table.cols[ids], np.int32),
                         np.asarray(table.kind[ids], np.int32), table.stride)


class _Part:
    """One layer group of a ``DistributedStep``: its own context (over the same flat buffers), factors or packed
    sets, exchange buffers and the events that order its phases against its exchanges."""

    def __init__(self, owner, ids, q_init):
        self.ids = list(ids)
        dev, n_local, world = owner.device, owner.n_local, owner.world
        self.table = owner.table if len(self.ids) == owner.table.n_layers else _sub_table(owner.table, self.ids)
        self.ctx = c = binding.Context(self.table, n_local, device=dev, **owner._cfg)
        # the group's layers are a contiguous run, so its levels are a slice of the step's level array: what the
        # regime test writes there is what the group's kernels read
        self.level = owner.level[self.ids[0]:self.ids[-1] + 1]
        if owner.compressor == "powersgd":
            ql = None if q_init is None else [q_init[l] for l in self.ids]
            self.q = c.new_q(ql if ql is not None else wl.initial_q(self.table, owner._cfg["rank_low"], device=dev))
            self.p_hat = c.new_p()
            self.x1 = torch.zeros(max(c.x1_floats, 4), device=dev)
            self.x2 = torch.zeros(max(c.x2_floats, 4), device=dev)
        else:
            self.vals, self.idx, self.counts = c.new_topk_buffers()
            self.vec = torch.zeros(max(c.vec_floats, 4), device=dev)
            self.vals_all = torch.zeros(world * self.vals.numel(), device=dev)
            self.idx_all = torch.zeros(world * self.idx.numel(), dtype=torch.int32, device=dev)
            self.counts_all = torch.zeros(world * self.counts.numel(), dtype=torch.int32, device=dev)
        self.done = [torch.cuda.Event() for _ in range(2)]       # a phase has produced an exchange buffer
        self.exchanged = [torch.cuda.Event() for _ in range(2)]  # the exchange of that buffer has finished


class DistributedStep:
    """Real workers: every rank (GPU) holds ``n_local`` workers; the compressed factors are exchanged between the
    kernels' phases (Section 5.1: all-reduce of P, then of Q, for PowerSGD; all-gather of the packed values and
    indices for TopK; the VECTOR layers ride in the first all-reduce).  Every rank ends a step with the same
    ``out``, ``q``, ``p_hat`` and ``level``: the decider's gradient is accumulated on the rank that holds it
    (global worker ``decider``), and the detector's per-layer norms are broadcast from there by a sum in which
    the other ranks contribute zeros.

    ``groups`` > 1 cuts the layers into that many contiguous groups of about equal size, each with its own
    context over the same flat buffers, and runs the exchanges on a communication stream: while group i's rows of
    P (or its packed sets) are in flight, the first pass of group i+1 runs, and likewise for Q'.  A layer's
    arithmetic does not depend on the other layers of its context, so the results are those of ``groups = 1``
    (bit for bit as long as the same implementation of the first PowerSGD pass serves both; ``extra_flags`` can
    force one).  With one group the calls and the exchanges alternate on the caller's stream."""

    def __init__(self, table: wl.LayerTable, n_local: int, compressor: str = "powersgd", rank_low=2, rank_high=1,
                 topk_low_bp=1000, topk_high_bp=100, eta=0.5, gs_eps=1e-8, check_every=10, decider=0, q_init=None,
                 device="cuda", lazy_residual=False, optimizer=None, exchange=None, groups=1, extra_flags=0):
        from . import dist_util
        if compressor not in ("powersgd", "topk"):
            raise ValueError(compressor)
        self.table, self.n_local, self.compressor = table, n_local, compressor
        self.x = exchange if exchange is not None else dist_util.Exchange()
        self.world, self.rank = self.x.world, self.x.rank
        self.lazy_residual = lazy_residual
        self.check_every = check_every
        self.device = dev = torch.device(device)
        self.owns_decider = decider // n_local == self.rank
        self._cfg = dict(rank_low=rank_low, rank_high=rank_high, topk_low_bp=topk_low_bp, topk_high_bp=topk_high_bp,
                         eta=eta, gs_eps=gs_eps, decider=decider % n_local,
                         flags=(binding.ACC_FLAG_LAZY_RESIDUAL if lazy_residual else 0) | extra_flags)
        L, stride = table.n_layers, table.stride
        self.level = torch.ones(L, dtype=torch.uint8, device=dev)
        self.delta = torch.zeros(stride, device=dev) if self.owns_decider else None
        self.norm2_curr = torch.zeros(L, dtype=torch.float64, device=dev)
        self.norm2_prev = torch.full((L,), -1.0, dtype=torch.float64, device=dev)
        self.err = torch.zeros(n_local, stride, device=dev)
        self.out = torch.zeros(stride, device=dev)
        self.t = 0
        self.params = self.mom = self.hyper = None
        if optimizer is not None:
            self.params = optimizer["params"]
            self.mom = torch.zeros(stride, device=dev)
            self.hyper = torch.tensor([optimizer["lr"], optimizer.get("momentum", 0.9),
                                       optimizer.get("weight_decay", 0.0)], dtype=torch.float32, device=dev)
        self.parts = [_Part(self, ids, q_init) for ids in _layer_groups(table, groups)]
        # the whole table's context serves the detector (norms, Algorithm 1); with one group it is that group's
        self.ctx = self.parts[0].ctx if len(self.parts) == 1 else binding.Context(table, n_local, device=dev,
                                                                                   **self._cfg)
        self._comm = torch.cuda.Stream(device=dev) if len(self.parts) > 1 else None
        one = self.parts[0]
        if len(self.parts) == 1:  # the single group's buffers under their plain names
            for name in ("q", "p_hat", "x1", "x2", "vals", "idx", "counts", "vec", "vals_all", "idx_all",
                         "counts_all"):
                if hasattr(one, name):
                    setattr(self, name, getattr(one, name))

    def flush(self, stream=None):
        """Lazy mode: materialises this rank's error memories (see ``AccordionStep.flush``)."""
        if not self.lazy_residual:
            return
        for p in self.parts:
            if self.compressor == "powersgd":
                p.ctx.acc_powersgd_flush(self.err, p.q, p.p_hat, stream)
            else:
                p.ctx.acc_topk_flush(self.err, stream)

    def bytes_exchanged_per_step(self) -> int:
        """Bytes this rank hands to the collectives in one step (the method's communication volume)."""
        if self.compressor == "powersgd":
            return 4 * sum(p.x1.numel() + p.x2.numel() for p in self.parts)
        return 4 * sum(p.vals.numel() + p.idx.numel() + p.counts.numel() + p.vec.numel() for p in self.parts)

    def _exchange(self, part, k, main, fn):
        """Runs the exchange ``fn`` of ``part``'s k-th buffer: on the caller's stream with one group, else on the
        communication stream, after the phase that filled the buffer and ahead of the phase that reads it."""
        if self._comm is None:
            with torch.cuda.stream(main):
                fn()
            return
        part.done[k].record(main)
        self._comm.wait_event(part.done[k])
        with torch.cuda.stream(self._comm):
            fn()
        part.exchanged[k].record(self._comm)

    def _await(self, part, k, main):
        if self._comm is not None:
            main.wait_event(part.exchanged[k])

    def step(self, grads: torch.Tensor, lr_curr: float = 0.1, lr_next: float = 0.1, stream=None):
        """One iteration on this rank's device-resident gradients ``[n_local, stride]``."""
        x, scale = self.x, 1.0 / self.world
        main = stream if stream is not None else torch.cuda.current_stream(self.device)
        if self.compressor == "powersgd":
            for p in self.parts:
                p.ctx.acc_powersgd_phase1(grads, self.err, p.q, p.p_hat, p.level, self.out, self.delta, p.x1, main)
                self._exchange(p, 0, main, lambda p=p: x.sum_(p.x1))
            for p in self.parts:
                self._await(p, 0, main)
                p.ctx.acc_powersgd_phase2(p.x1, scale, p.p_hat, p.level, self.out, p.x2, main)
                self._exchange(p, 1, main, lambda p=p: x.sum_(p.x2))
            for p in self.parts:
                self._await(p, 1, main)
                p.ctx.acc_powersgd_phase3(self.err, p.q, p.p_hat, p.level, p.x1, p.x2, scale, self.out, self.params,
                                          self.mom, self.hyper, main)
        else:
            def gather(p):
                x.gather_into(p.vals_all, p.vals)
                x.gather_into(p.idx_all, p.idx)
                x.gather_into(p.counts_all, p.counts)
                x.sum_(p.vec)
            for p in self.parts:
                p.ctx.acc_topk_compress(grads, self.err, p.level, p.vals, p.idx, p.counts, self.delta, p.vec, main)
                self._exchange(p, 0, main, lambda p=p: gather(p))
            for p in self.parts:
                self._await(p, 0, main)
                p.ctx.acc_topk_decompress(p.vals_all, p.idx_all, p.counts_all, self.world * self.n_local, p.vec,
                                          scale, self.out, self.params, self.mom, self.hyper, main)
        self.t += 1
        if self.t % self.check_every == 0:
            with torch.cuda.stream(main):
                if self.owns_decider:
                    self.ctx.acc_layer_norms(self.delta, 1, self.norm2_curr, stream=main)
                else:
                    self.norm2_curr.zero_()
                x.sum_(self.norm2_curr)  # a broadcast from the deciding rank (Section 3: one node decides for all)
                self.ctx.acc_detect_regime(self.norm2_curr, self.norm2_prev, lr_curr, lr_next, self.level, self.delta,
                                           main)
        return self.out


class HostFedStep:
    """Runs ``AccordionStep`` on gradients that live in pinned host memory.

    Every call copies that step's gradients to the device and the step's averaged outputs back to pinned
    host buffers (``acc_upload_grads`` / ``acc_download_out``: host pointers go straight to the library).  The copies run on their own stream with two device staging buffers, so the upload of
    step i+1 overlaps the kernels of step i; results are ordered by events, never by host synchronisation.
    """

    def __init__(self, engine: AccordionStep):
        self.eng = engine
        dev = engine.device
        shape = (engine.W, engine.table.stride)
        self.stage = [torch.empty(shape, dtype=torch.float32, device=dev) for _ in range(2)]
        self.h2d = torch.cuda.Stream(device=dev)
        self.d2h = torch.cuda.Stream(device=dev)
        self.uploaded = [torch.cuda.Event() for _ in range(2)]
        self.consumed = [torch.cuda.Event() for _ in range(2)]
        self.downloaded = torch.cuda.Event()
        self.outs_host = [torch.empty(engine.table.stride, dtype=torch.float32).pin_memory() for _ in engine.outputs()]
        self.i = 0
        self.h2d_bytes_per_step = 4 * shape[0] * shape[1]
        self.d2h_bytes_per_step = 4 * engine.table.stride * len(self.outs_host)

    def step(self, host_grads: torch.Tensor):
        """Queues upload, compute and download of one step; returns the pinned host output tensors (valid
        after ``synchronize`` or after the next call's download event)."""
        assert host_grads.is_pinned() and host_grads.dtype == torch.float32
        b = self.i & 1
        main = torch.cuda.current_stream(self.eng.device)
        with torch.cuda.stream(self.h2d):
            if self.i >= 2:
                self.h2d.wait_event(self.consumed[b])      # the step that read this staging buffer is done
            self.eng.ctx.acc_upload_grads(host_grads, self.stage[b], self.h2d)
            self.uploaded[b].record(self.h2d)
        main.wait_event(self.uploaded[b])
        if self.i >= 1:
            main.wait_event(self.downloaded)               # previous outputs are safely on the host
        self.eng.step(self.stage[b])
        self.consumed[b].record(main)
        with torch.cuda.stream(self.d2h):
            self.d2h.wait_event(self.consumed[b])
            for oh, od in zip(self.outs_host, self.eng.outputs()):
                self.eng.ctx.acc_download_out(od, oh, self.d2h)
            self.downloaded.record(self.d2h)
        self.i += 1
        return self.outs_host

    def synchronize(self):
        self.h2d.synchronize()
        self.d2h.synchronize()
        torch.cuda.current_stream(self.eng.device).synchronize()
