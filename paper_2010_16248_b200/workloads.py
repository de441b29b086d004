"""Seeded synthetic gradient workloads shaped like the paper's models.

This module only *produces inputs*: layer tables (shapes, offsets) and seeded
per-iteration gradient tensors.  It contains none of the method's arithmetic
(no error feedback, no norms, no compression), so that both the CUDA path and
the CPU oracle can be fed from it without sharing any code of the method.

Shapes follow the parameter totals of the paper's Appendix G tables (ResNet-18:
11,173,962 / 11,220,132 parameters for 10 / 100 classes; VGG-19bn: 20,565,834
for 10 classes).  Convolution weights are viewed as ``out x (in*k*k)`` matrices
and 1-D tensors (biases, BatchNorm vectors) stay uncompressed, which is the
convention that reproduces the "Data Sent" columns of Tables 1-2.

The value distributions follow the qualitative structure the paper describes:
low-rank-compressible layers plus noise for PowerSGD (Section "Accordion with PowerSGD"), a fixed
sparse mean plus dense noise for TopK (Section 4.3 and Appendix A.1), and a
gradient-norm scale that changes at phase boundaries (Section 4.1).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Callable, List, Optional, Sequence, Tuple

import numpy as np
import torch

MATRIX = 0
VECTOR = 1

BASE_SEED = 20101624
ALIGN = 4  # every layer starts at a multiple of 4 floats (16 bytes)
STRIDE_ALIGN = 64  # the per-worker stride is a multiple of 64 floats (256 bytes)


# --------------------------------------------------------------------------- #
# Layer tables
# --------------------------------------------------------------------------- #
@dataclasses.dataclass
class LayerTable:
    """Offsets/shapes of all layers inside one flat per-worker buffer."""

    names: List[str]
    offset: np.ndarray  # int64 [L], in elements, multiple of ALIGN
    rows: np.ndarray  # int32 [L]  (VECTOR: rows = 1)
    cols: np.ndarray  # int32 [L]
    kind: np.ndarray  # int32 [L]  MATRIX / VECTOR
    stride: int  # elements per worker (padded)

    @property
    def n_layers(self) -> int:
        return len(self.names)

    @property
    def sizes(self) -> np.ndarray:
        return self.rows.astype(np.int64) * self.cols.astype(np.int64)

    @property
    def n_params(self) -> int:
        return int(self.sizes.sum())

    @property
    def n_matrix_params(self) -> int:
        return int(self.sizes[self.kind == MATRIX].sum())

    def slices(self):
        for l in range(self.n_layers):
            o = int(self.offset[l])
            yield l, slice(o, o + int(self.rows[l]) * int(self.cols[l]))


def make_table(shapes: Sequence[Tuple[str, Tuple[int, ...]]]) -> LayerTable:
    """Lay ``(name, shape)`` tensors out back to back, each start 16-byte aligned."""
    names, offset, rows, cols, kind = [], [], [], [], []
    cur = 0
    for name, shp in shapes:
        names.append(name)
        offset.append(cur)
        if len(shp) == 2:
            rows.append(shp[0]); cols.append(shp[1]); kind.append(MATRIX)
            size = shp[0] * shp[1]
        else:
            rows.append(1); cols.append(shp[0]); kind.append(VECTOR)
            size = shp[0]
        cur += (size + ALIGN - 1) // ALIGN * ALIGN
    stride = (cur + STRIDE_ALIGN - 1) // STRIDE_ALIGN * STRIDE_ALIGN
    return LayerTable(names, np.asarray(offset, np.int64), np.asarray(rows, np.int32),
                      np.asarray(cols, np.int32), np.asarray(kind, np.int32), max(stride, STRIDE_ALIGN))


def shapes_resnet18(num_classes: int = 100, width: int = 64):
    """ResNet-18 (CIFAR variant): 20 convolutions + classifier, 41 1-D tensors."""
    s = []

    def conv_bn(name, cout, cin, k):
        s.append((f"{name}.weight", (cout, cin * k * k)))
        s.append((f"{name}.bn.weight", (cout,)))
        s.append((f"{name}.bn.bias", (cout,)))

    conv_bn("conv1", width, 3, 3)
    cin = width
    for stage, mult in enumerate((1, 2, 4, 8)):
        cout = width * mult
        for block in range(2):
            conv_bn(f"layer{stage + 1}.{block}.conv1", cout, cin, 3)
            conv_bn(f"layer{stage + 1}.{block}.conv2", cout, cout, 3)
            if block == 0 and cin != cout:
                conv_bn(f"layer{stage + 1}.{block}.shortcut", cout, cin, 1)
            cin = cout
    s.append(("linear.weight", (num_classes, cin)))
    s.append(("linear.bias", (num_classes,)))
    return s


def shapes_vgg19bn(num_classes: int = 100, width: int = 64):
    """VGG-19 with BatchNorm: 16 3x3 convolutions (with bias) + 3 linear layers."""
    cfg = [1, 1, "M", 2, 2, "M", 4, 4, 4, 4, "M", 8, 8, 8, 8, "M", 8, 8, 8, 8, "M"]
    s = []
    cin = 3
    i = 0
    for v in cfg:
        if v == "M":
            continue
        cout = width * v
        s.append((f"features.{i}.weight", (cout, cin * 9)))
        s.append((f"features.{i}.bias", (cout,)))
        s.append((f"features.{i}.bn.weight", (cout,)))
        s.append((f"features.{i}.bn.bias", (cout,)))
        cin = cout
        i += 1
    s.append(("classifier.0.weight", (cin, cin))); s.append(("classifier.0.bias", (cin,)))
    s.append(("classifier.1.weight", (cin, cin))); s.append(("classifier.1.bias", (cin,)))
    s.append(("classifier.2.weight", (num_classes, cin))); s.append(("classifier.2.bias", (num_classes,)))
    return s


def shapes_lstm(vocab: int = 33278, hidden: int = 650):
    """2-layer LSTM language model: encoder, 4 gate matrices (4h x h), decoder."""
    s = [("encoder.weight", (vocab, hidden))]
    for layer in range(2):
        s.append((f"rnn.weight_ih_l{layer}", (4 * hidden, hidden)))
        s.append((f"rnn.weight_hh_l{layer}", (4 * hidden, hidden)))
        s.append((f"rnn.bias_l{layer}.ih", (4 * hidden,)))
        s.append((f"rnn.bias_l{layer}.hh", (4 * hidden,)))
    s.append(("decoder.weight", (vocab, hidden)))
    s.append(("decoder.bias", (vocab,)))
    return s


# --------------------------------------------------------------------------- #
# Workload descriptions (the five benchmark configurations, c1..c5)
# --------------------------------------------------------------------------- #
@dataclasses.dataclass
class Workload:
    name: str
    table: LayerTable
    n_workers: int
    n_iters: int
    check_every: int
    eta: float
    rank_low: int
    rank_high: int
    topk_low_bp: int
    topk_high_bp: int
    compressors: Tuple[str, ...]  # subset of ("powersgd", "topk")
    jumps: Tuple[int, ...]  # iterations at which the gradient scale doubles
    spectrum_power: float  # s_i = i ** -spectrum_power
    flavour: str  # "lowrank" | "sparse_mean" | "lstm"
    config_id: int

    def amplitude(self, t: int) -> float:
        return float(2.0 ** sum(1 for j in self.jumps if t >= j))


def workload(config: int, scale: int = 1) -> Workload:
    """Return benchmark configuration ``config`` (1..5).  ``scale`` > 1 shrinks widths /
    vocabulary by that factor (CPU-sized versions of the same structure)."""
    if config == 1:
        n, m = max(256 // scale, 8), max(1152 // scale, 9)
        return Workload("c1-single-256x1152", make_table([("conv.weight", (n, m))]), 2, 20, 5, 0.5,
                        2, 1, 1000, 100, ("powersgd", "topk"), (0, 10), 1.0, "lowrank", 1)
    if config == 2:
        return Workload("c2-resnet18-powersgd", make_table(shapes_resnet18(100, max(64 // scale, 4))), 4, 200, 10,
                        0.5, 2, 1, 1000, 100, ("powersgd",), (0, 100, 150), 1.0, "lowrank", 2)
    if config == 3:
        return Workload("c3-resnet18-topk", make_table(shapes_resnet18(100, max(64 // scale, 4))), 4, 200, 10,
                        0.5, 2, 1, 1000, 100, ("topk",), (0, 100, 150), 1.0, "sparse_mean", 3)
    if config == 4:
        return Workload("c4-vgg19bn-powersgd", make_table(shapes_vgg19bn(100, max(64 // scale, 4))), 8, 300, 10,
                        0.5, 4, 1, 1000, 100, ("powersgd",), (0, 100, 150), 0.5, "lowrank", 4)
    if config == 5:
        return Workload("c5-lstm-powersgd+topk",
                        make_table(shapes_lstm(max(33278 // scale, 50), max(650 // scale, 10))), 8, 300, 10,
                        0.5, 2, 1, 1000, 100, ("powersgd", "topk"), (0, 100, 150), 1.0, "lstm", 5)
    raise ValueError(f"unknown config {config}")


# --------------------------------------------------------------------------- #
# Seeded generators
# --------------------------------------------------------------------------- #
def _gen(device, *key: int) -> torch.Generator:
    seed = BASE_SEED
    for k in key:
        seed = (seed * 1000003 + int(k) * 7919 + 12345) % (2 ** 62)
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _orthonormal(n: int, r: int, gen: torch.Generator, device) -> torch.Tensor:
    a = torch.randn(n, r, generator=gen, device=device, dtype=torch.float64)
    q, _ = torch.linalg.qr(a)
    return q


class GradientStream:
    """``grads(t)`` -> fp32 tensor ``[W, stride]`` of worker gradients at iteration t.

    Everything is a deterministic function of (config, t); padding elements
    between layers are exactly zero.
    """

    def __init__(self, wl: Workload, device="cpu"):
        self.wl = wl
        self.device = torch.device(device)
        tb = wl.table
        dev = self.device
        self.signal = torch.zeros(tb.stride, device=dev, dtype=torch.float32)
        self.noise_scale = torch.zeros(tb.stride, device=dev, dtype=torch.float32)
        self.layer_scale = np.zeros(tb.n_layers)
        self._tie = None
        self._rowsparse = []  # (offset, rows, cols, weights)
        g0 = _gen(dev, wl.config_id, 0)
        tie_src, tie_dst, tie_sign = [], [], []
        for l, sl in tb.slices():
            n, m = int(tb.rows[l]), int(tb.cols[l])
            if wl.config_id == 1:
                c = 1.0
            else:
                u = torch.rand((), generator=g0, device=dev, dtype=torch.float64).item()
                c = 10.0 ** (-4.0 + 3.0 * u)  # log-uniform in [1e-4, 1e-1]
            self.layer_scale[l] = c
            if tb.kind[l] == VECTOR:
                self.noise_scale[sl] = c
                continue
            if wl.flavour == "sparse_mean":
                size = n * m
                n_sup = max(1, size * 5 // 100)
                perm = torch.randperm(size, generator=g0, device=dev)
                sup = perm[:n_sup]
                u = torch.rand(n_sup, generator=g0, device=dev, dtype=torch.float64) - 0.5
                lap = -torch.sign(u) * torch.log1p(-2.0 * u.abs())  # Laplace(0, 1)
                seg = torch.zeros(size, device=dev, dtype=torch.float64)
                seg[sup] = 10.0 * c * lap
                self.signal[sl] = seg.to(torch.float32)
                self.noise_scale[sl] = c
                n_tie = size // 1000
                if n_tie > 0 and size >= 2 * n_tie:
                    p2 = torch.randperm(size, generator=g0, device=dev)
                    tie_dst.append(p2[:n_tie] + sl.start)
                    tie_src.append(p2[n_tie:2 * n_tie] + sl.start)
                    tie_sign.append(torch.randint(0, 2, (n_tie,), generator=g0, device=dev).float() * 2 - 1)
                continue
            if wl.flavour == "lstm" and tb.names[l].startswith("encoder"):
                # row-sparse embedding gradient: Zipf(1) weights over a fixed permutation of the rows
                rank = torch.randperm(n, generator=g0, device=dev).double() + 1.0
                self._rowsparse.append((sl.start, n, m, (1.0 / rank)))
                self.noise_scale[sl] = c
                continue
            rho = min(n, m, 256)
            U = _orthonormal(n, rho, g0, dev)
            V = _orthonormal(m, rho, g0, dev)
            s = torch.arange(1, rho + 1, device=dev, dtype=torch.float64) ** (-wl.spectrum_power)
            S = (U * s) @ V.T
            if wl.config_id == 1:
                sigma = 0.01
            else:
                sigma = math.sqrt(float((s * s).sum()) / (n * m))  # noise and signal of equal Frobenius norm
            self.signal[sl] = (c * S).reshape(-1).to(torch.float32)
            self.noise_scale[sl] = c * sigma
        if tie_dst:
            self._tie = (torch.cat(tie_src), torch.cat(tie_dst), torch.cat(tie_sign))

    def grads(self, t: int, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        wl, tb, dev = self.wl, self.wl.table, self.device
        g = _gen(dev, wl.config_id, 1, t)
        W = wl.n_workers
        if out is None:
            out = torch.empty(W, tb.stride, device=dev, dtype=torch.float32)
        out.normal_(generator=g)
        out.mul_(self.noise_scale).add_(self.signal)
        for (o, n, m, wts) in self._rowsparse:
            k = max(1, n * 2 // 100)
            for w in range(W):
                rows = torch.multinomial(wts, k, replacement=False, generator=g)
                mask = torch.zeros(n, device=dev, dtype=torch.float32)
                mask[rows] = 1.0
                out[w, o:o + n * m].view(n, m).mul_(mask[:, None])
        if self._tie is not None:
            src, dst, sign = self._tie
            out[:, dst] = out[:, src].abs() * sign
        out.mul_(wl.amplitude(t))
        return out


def initial_q(table: LayerTable, rank_max: int, seed: int = BASE_SEED, device="cpu") -> List[Optional[torch.Tensor]]:
    """Warm-start matrices: per MATRIX layer an ``[m, rank_max]`` fp32 tensor of i.i.d. N(0,1)."""
    g = _gen(device, seed, 7)
    qs: List[Optional[torch.Tensor]] = []
    for l in range(table.n_layers):
        if table.kind[l] == MATRIX:
            qs.append(torch.randn(int(table.cols[l]), rank_max, generator=g, device=device, dtype=torch.float32))
        else:
            qs.append(None)
    return qs
