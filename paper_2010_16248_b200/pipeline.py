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
                 extra_flags=0, overlap=True):
        """``overlap``: with two compressors, the TopK step runs on a second stream beside the PowerSGD step
        (they share only the gradients and the level array, both read-only), so that the short, latency-bound
        kernels of one hide behind the streaming kernels of the other; the results are the same bits.
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
                                   flags=(binding.ACC_FLAG_LAZY_RESIDUAL if lazy_residual else 0) | extra_flags)
        dev, L, stride = self.device, table.n_layers, table.stride
        self.level = torch.ones(L, dtype=torch.uint8, device=dev)  # before the first check: low compression
        self.delta = torch.zeros(stride, device=dev)
        self.norm2_curr = torch.zeros(L, dtype=torch.float64, device=dev)
        self.norm2_prev = torch.full((L,), -1.0, dtype=torch.float64, device=dev)
        self.t = 0
        self.launches = 0
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
                c.acc_detect_regime(self.norm2_curr, self.norm2_prev, lr_curr, lr_next, self.level, self.delta, main)
                self.launches += c.last_launch_count()
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
            c.acc_detect_regime(self.norm2_curr, self.norm2_prev, lr_curr, lr_next, self.level, self.delta, stream)
            self.launches += c.last_launch_count()

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
        Which rank or K a layer gets is decided on the device from ``level``, so the same graphs serve every
        iteration.  ``step_graph(slot)`` replays the right one.  Every library call is asynchronous and
        allocation-free, hence capturable."""
        torch.cuda.synchronize(self.device)
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
        self.t, self.launches = saved_t, saved_launches

    def step_graph(self, slot: int = 0):
        """Replays the captured iteration that reads gradient buffer ``slot`` (see ``capture_graphs``)."""
        self.t += 1
        which = 1 if self.t % self.check_every == 0 else 0
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


class DistributedStep:
    """Real workers: every rank (GPU) holds ``n_local`` workers; the compressed factors are exchanged between the
    kernels' phases (Section 5.1: all-reduce of P, then of Q, for PowerSGD; all-gather of the packed values and
    indices for TopK; the VECTOR layers ride in the first all-reduce).  Every rank ends a step with the same
    ``out``, ``q``, ``p_hat`` and ``level``: the decider's gradient is accumulated on the rank that holds it
    (global worker ``decider``), and the detector's per-layer norms are broadcast from there by a sum in which
    the other ranks contribute zeros."""

    def __init__(self, table: wl.LayerTable, n_local: int, compressor: str = "powersgd", rank_low=2, rank_high=1,
                 topk_low_bp=1000, topk_high_bp=100, eta=0.5, gs_eps=1e-8, check_every=10, decider=0, q_init=None,
                 device="cuda", lazy_residual=False, optimizer=None, exchange=None):
        from . import dist_util
        self.table, self.n_local, self.compressor = table, n_local, compressor
        self.x = exchange if exchange is not None else dist_util.Exchange()
        self.world, self.rank = self.x.world, self.x.rank
        self.lazy_residual = lazy_residual
        self.check_every = check_every
        self.device = dev = torch.device(device)
        self.owns_decider = decider // n_local == self.rank
        self.ctx = binding.Context(table, n_local, device=device, rank_low=rank_low, rank_high=rank_high,
                                   topk_low_bp=topk_low_bp, topk_high_bp=topk_high_bp, eta=eta, gs_eps=gs_eps,
                                   decider=decider % n_local,
                                   flags=binding.ACC_FLAG_LAZY_RESIDUAL if lazy_residual else 0)
        L, stride, c = table.n_layers, table.stride, self.ctx
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
        if compressor == "powersgd":
            self.q = c.new_q(q_init if q_init is not None else wl.initial_q(table, rank_low, device=dev))
            self.p_hat = c.new_p()
            self.x1 = torch.zeros(max(c.x1_floats, 4), device=dev)
            self.x2 = torch.zeros(max(c.x2_floats, 4), device=dev)
        elif compressor == "topk":
            self.vals, self.idx, self.counts = c.new_topk_buffers()
            self.vec = torch.zeros(max(c.vec_floats, 4), device=dev)
            w = self.world
            self.vals_all = torch.zeros(w * self.vals.numel(), device=dev)
            self.idx_all = torch.zeros(w * self.idx.numel(), dtype=torch.int32, device=dev)
            self.counts_all = torch.zeros(w * self.counts.numel(), dtype=torch.int32, device=dev)
        else:
            raise ValueError(compressor)

    def flush(self, stream=None):
        """Lazy mode: materialises this rank's error memories (see ``AccordionStep.flush``)."""
        if not self.lazy_residual:
            return
        if self.compressor == "powersgd":
            self.ctx.acc_powersgd_flush(self.err, self.q, self.p_hat, stream)
        else:
            self.ctx.acc_topk_flush(self.err, stream)

    def bytes_exchanged_per_step(self) -> int:
        """Bytes this rank hands to the collectives in one step (the method's communication volume)."""
        if self.compressor == "powersgd":
            return 4 * (self.x1.numel() + self.x2.numel())
        return 4 * (self.vals.numel() + self.idx.numel() + self.counts.numel() + self.vec.numel())

    def step(self, grads: torch.Tensor, lr_curr: float = 0.1, lr_next: float = 0.1, stream=None):
        """One iteration on this rank's device-resident gradients ``[n_local, stride]``."""
        c, x, scale = self.ctx, self.x, 1.0 / self.world
        if self.compressor == "powersgd":
            c.acc_powersgd_phase1(grads, self.err, self.q, self.p_hat, self.level, self.out, self.delta, self.x1,
                                  stream)
            x.sum_(self.x1)
            c.acc_powersgd_phase2(self.x1, scale, self.p_hat, self.level, self.out, self.x2, stream)
            x.sum_(self.x2)
            c.acc_powersgd_phase3(self.err, self.q, self.p_hat, self.level, self.x1, self.x2, scale, self.out,
                                  self.params, self.mom, self.hyper, stream)
        else:
            c.acc_topk_compress(grads, self.err, self.level, self.vals, self.idx, self.counts, self.delta, self.vec,
                                stream)
            x.gather_into(self.vals_all, self.vals)
            x.gather_into(self.idx_all, self.idx)
            x.gather_into(self.counts_all, self.counts)
            x.sum_(self.vec)
            c.acc_topk_decompress(self.vals_all, self.idx_all, self.counts_all, self.world * self.n_local, self.vec,
                                  scale, self.out, self.params, self.mom, self.hyper, stream)
        self.t += 1
        if self.t % self.check_every == 0:
            if self.owns_decider:
                c.acc_layer_norms(self.delta, 1, self.norm2_curr, stream=stream)
            else:
                self.norm2_curr.zero_()
            x.sum_(self.norm2_curr)  # a broadcast from the deciding rank (Section 3: one node decides for all)
            c.acc_detect_regime(self.norm2_curr, self.norm2_prev, lr_curr, lr_next, self.level, self.delta, stream)
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
