"""acc_sumsq_static: the entry point for callers that cannot allocate device memory or pass a
workspace (its scratch is an array built into the library).  Checked against acc_layer_norms, the
existing entry point that computes the same sums with caller-provided scratch, on two calls in a
row -- the second smaller than the first, so stale partial sums left in the shared array would show.

This file sorts last on purpose: a run that stops at the first failure has then already run every
other test."""
import numpy as np
import pytest
import torch

from paper_2010_16248_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu


def _reference_norm2(x):
    table = wl.make_table([("all", (x.numel(),))])
    ctx = binding.Context(table, 1)
    padded = torch.zeros(table.stride, device="cuda")
    padded[:x.numel()] = x
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    ctx.acc_layer_norms(padded, 1, out)
    torch.cuda.synchronize()
    return float(out.item())


def test_static_norm_matches_layer_norms_twice_in_a_row():
    g = torch.Generator(device="cuda").manual_seed(5)
    sizes = [3 * 8192 * 41 + 1237, 8192 + 5]      # many tiles with a ragged tail, then far fewer tiles
    bufs = [torch.randn(n, generator=g, device="cuda") * (10.0 ** i) for i, n in enumerate(sizes)]
    outs = [torch.full((1,), -1.0, dtype=torch.float64, device="cuda") for _ in sizes]
    for x, o in zip(bufs, outs):                  # back to back on one stream, no sync in between
        binding.acc_sumsq_static(x, x.numel(), o)
    torch.cuda.synchronize()
    for x, o in zip(bufs, outs):
        want = _reference_norm2(x)
        got = float(o.item())
        assert np.isclose(got, want, rtol=1e-12, atol=0.0), (got, want)
        assert np.isclose(got, float((x.double() ** 2).sum().item()), rtol=1e-9)


def test_static_norm_rejects_bad_sizes_without_launching():
    x = torch.ones(64, device="cuda")
    o = torch.zeros(1, dtype=torch.float64, device="cuda")
    with pytest.raises(ValueError):
        binding.acc_sumsq_static(x, (1 << 28) + 1, o)   # more elements than the tensor holds: refused by the binding
    big = torch.empty((1 << 28) + 1, device="cuda")     # 1 GiB + 4 bytes, never read
    with pytest.raises(binding.AccError) as ei:
        binding.acc_sumsq_static(big, big.numel(), o)   # beyond the built-in scratch: refused, nothing launched
    assert ei.value.status == 5 and "capacity" in str(ei.value)
    del big
    with pytest.raises(binding.AccError):
        binding.acc_sumsq_static(x, 0, o)
    with pytest.raises(binding.AccError):
        binding.acc_sumsq_static(x[1:], 8, o)           # misaligned buffer
    binding.acc_sumsq_static(x, 64, o)
    torch.cuda.synchronize()
    assert float(o.item()) == 64.0
