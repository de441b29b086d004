"""CPU-side checks of the C-ABI library: it loads, exports every symbol include/acc.h declares, and its
host-only entry points (configuration checks, workspace sizing, communication accounting) behave."""
import ctypes as C
import os
import re

import pytest

from oracle import accordion_oracle as orc
from paper_2010_16248_b200 import binding, build, workloads as wl
from tests import helpers as H

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return binding.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "acc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(acc_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = _declared()
    assert len(names) >= 13
    for n in names:
        assert hasattr(lib, n), f"{n} declared in acc.h but not exported"
    assert set(names) == set(binding.EXPORTS)


def test_workspace_sizing_and_config_validation(lib):
    table = wl.make_table(wl.shapes_resnet18(100))
    cfg = binding.make_config(table, 4)
    n = C.c_size_t()
    assert lib.acc_workspace_bytes(C.byref(cfg), C.byref(n)) == 0 and n.value > 0
    small = n.value
    cfg8 = binding.make_config(table, 8)
    assert lib.acc_workspace_bytes(C.byref(cfg8), C.byref(n)) == 0 and n.value > small
    bad = [dict(rank_low=5), dict(rank_low=1, rank_high=2), dict(topk_low_bp=0, topk_high_bp=0),
           dict(topk_low_bp=20000), dict(decider=4), dict(eta=-1.0), dict(worker_stride=table.stride // 8 * 4)]
    for kw in bad:
        c = binding.make_config(table, 4, **kw)
        assert lib.acc_workspace_bytes(C.byref(c), C.byref(n)) == 1, kw
    c = binding.make_config(table, 4, worker_stride=table.stride + 2)
    assert lib.acc_workspace_bytes(C.byref(c), C.byref(n)) == 2            # stride not a multiple of 4
    c = binding.make_config(table, 4)
    c.layers[3].offset += 1
    assert lib.acc_workspace_bytes(C.byref(c), C.byref(n)) == 2            # misaligned layer
    c = binding.make_config(table, 4)
    c.layers[5].offset = c.layers[4].offset                               # overlapping layers
    assert lib.acc_workspace_bytes(C.byref(c), C.byref(n)) == 1
    h = C.c_void_p()
    assert lib.acc_create(C.byref(cfg), None, 0, C.byref(h)) == 3          # no workspace
    assert lib.acc_strerror(3).decode().startswith("workspace")


def test_floats_sent_matches_oracle_and_tables(lib):
    for shapes, W, rl, rh in ((wl.shapes_resnet18(10), 4, 2, 1), (wl.shapes_vgg19bn(10), 4, 4, 1)):
        table = wl.make_table(shapes)
        layers = H.layers_of(table)
        cfg = binding.make_config(table, W, rank_low=rl, rank_high=rh)
        for lv in (0, 1):
            level = [lv] * table.n_layers
            for comp, name in ((binding.POWERSGD, "powersgd"), (binding.TOPK, "topk")):
                want = orc.floats_sent_per_iteration(layers, level, name, W, rl, rh, 1000, 100)
                assert binding.acc_floats_sent(cfg, level, comp) == want
    # Table 1, ResNet-18 / CIFAR-10, rank 2: 2418.4 million floats over 300 epochs x 98 iterations
    table = wl.make_table(wl.shapes_resnet18(10))
    cfg = binding.make_config(table, 4, rank_low=2, rank_high=1)
    assert abs(binding.acc_floats_sent(cfg, [1] * table.n_layers, binding.POWERSGD) * 29400 / 1e6 - 2418.4) < 0.1


def test_bench_reference_arm_prints_the_contract_line():
    """`bench.py --impl reference` (the oracle timed on the host) runs without a GPU and prints one JSON line with
    the keys the benchmark contract names."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--config", "1",
                          "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    line = json.loads(res.stdout.strip().splitlines()[-1])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
                "scaling", "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in line, key
    assert line["impl"] == "reference" and line["steps"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0


def test_bench_gpus_argument_reaches_both_arms(monkeypatch):
    """`--gpus N`: the reference arm (the oracle on the host) echoes N and prints one line whatever N is; the GPU
    arm, started without a launcher, re-executes itself under torch.distributed.run with N ranks on 127.0.0.1 and
    the same arguments."""
    import importlib
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--config", "1", "--steps", "1", "--warmup", "0"], capture_output=True, text=True,
                         timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1 and json.loads(lines[0])["n_gpus"] == 2
    cpu = json.loads(lines[0])["cpu_baseline"]
    assert cpu["value_single_thread"] > 0 and "stream" in cpu["sample"] and cpu["cores"] >= 1
    sys.path.insert(0, root)
    bench = importlib.import_module("bench")
    seen = {}
    monkeypatch.setattr(bench.subprocess, "call", lambda cmd: seen.setdefault("cmd", cmd) and 0)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "2", "--steps", "7"])
    assert bench.respawn_under_torchrun(2) == 0
    cmd = seen["cmd"]
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=2" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and int(cmd[cmd.index("--master-port") + 1]) > 0
    assert cmd[-4:] == ["--gpus", "2", "--steps", "7"] and cmd[-5].endswith("bench.py")


def _hostless_context(table, W):
    """A binding.Context with the layout fields filled in by hand and no library handle: the argument checks run
    (and must raise) before any call into the library, so they can be tested without a GPU."""
    import torch
    c = binding.Context.__new__(binding.Context)
    c.table, c.device, c._h = table, torch.device("cuda", 0), None
    c.n_workers, c.n_layers, c.stride = W, table.n_layers, table.stride
    c.extent = int(max(int(table.offset[l]) + int(table.rows[l]) * int(table.cols[l]) for l in range(table.n_layers)))
    mat = table.kind == wl.MATRIX
    c.q_rows, c.p_rows = int(table.cols[mat].sum()), int(table.rows[mat].sum())
    c.capacity = int(sum(max(1, int(s) // 10) for s in table.sizes[mat]))
    c.x1_floats, c.x2_floats, c.vec_floats = 4 * c.p_rows + 8, 4 * c.q_rows, 8
    return c


def test_binding_rejects_short_or_misplaced_tensors_before_calling_the_library():
    """The C ABI takes bare pointers, so a tensor shorter than the context's layout would become an out-of-bounds
    device access.  The binding refuses it (and wrong dtypes, non-contiguous views, CPU tensors) with ValueError."""
    import torch
    table = wl.make_table([("a", (6, 10)), ("v", (5,)), ("b", (4, 8))])
    W, L, S = 2, table.n_layers, table.stride
    c = _hostless_context(table, W)
    f = lambda n: torch.zeros(n)                                   # noqa: E731
    level = torch.zeros(L, dtype=torch.uint8)
    ok = dict(grads=f(W * S), err=f(W * S), q=f(4 * c.q_rows), p_hat=f(4 * c.p_rows), level=level, out=f(S))
    # every argument one element short, in turn: the message names it
    for name in ok:
        short = dict(ok)
        short[name] = ok[name][:-1].clone()
        with pytest.raises(ValueError, match=name):
            c.acc_powersgd_step(**short)
    with pytest.raises(ValueError, match="delta"):
        c.acc_powersgd_step(**ok, delta=f(S - 1))
    # right sizes on the CPU: refused as "not a CUDA tensor", after the size checks passed
    with pytest.raises(ValueError, match="CUDA"):
        c.acc_powersgd_step(**ok)
    with pytest.raises(ValueError, match="dtype"):
        c.acc_powersgd_step(**{**ok, "grads": torch.zeros(W * S, dtype=torch.float64)})
    with pytest.raises(ValueError, match="contiguous"):
        c.acc_powersgd_step(**{**ok, "out": torch.zeros(2 * S)[::2]})
    vals, idx = f(W * c.capacity), torch.zeros(W * c.capacity, dtype=torch.int32)
    counts = torch.zeros(W * L, dtype=torch.int32)
    with pytest.raises(ValueError, match="vals"):
        c.acc_topk_step(ok["grads"], ok["err"], level, vals[:-1].clone(), idx, counts, ok["out"])
    with pytest.raises(ValueError, match="idx"):
        c.acc_topk_step(ok["grads"], ok["err"], level, vals, idx[:-1].clone(), counts, ok["out"])
    with pytest.raises(ValueError, match="counts"):
        c.acc_topk_step(ok["grads"], ok["err"], level, vals, idx, counts[:-1].clone(), ok["out"])
    with pytest.raises(ValueError, match="level"):
        c.acc_topk_step(ok["grads"], ok["err"], level[:-1].clone(), vals, idx, counts, ok["out"])
    n2 = torch.zeros(L, dtype=torch.float64)
    with pytest.raises(ValueError, match="norm2"):
        c.acc_layer_norms(f(S), 1, n2[:-1].clone())
    with pytest.raises(ValueError, match="buf"):
        c.acc_layer_norms(f(S + c.extent - 1), 2, torch.zeros(2 * L, dtype=torch.float64))
    with pytest.raises(ValueError, match="norm2_prev"):
        c.acc_detect_regime(n2, n2[:-1].clone(), 0.1, 0.1, level)
    with pytest.raises(ValueError, match="hyper"):
        c.acc_sgd_nesterov(f(S), f(S), f(S), f(2))
    with pytest.raises(ValueError, match="together"):
        c.acc_batch_average(f(W * S), 2, f(S), params=f(S))
    with pytest.raises(ValueError, match="x1"):
        c.acc_powersgd_phase2(f(c.x1_floats - 1), 1.0, ok["p_hat"], level, ok["out"], f(c.x2_floats))
    with pytest.raises(ValueError, match="vals_all"):
        c.acc_topk_decompress(f(3 * c.capacity - 1), torch.zeros(3 * c.capacity, dtype=torch.int32),
                              torch.zeros(3 * L, dtype=torch.int32), 3, f(8), 1.0, f(S))
    # the entry point without a context: n may not exceed what the tensor holds
    with pytest.raises(ValueError, match="buf"):
        binding.acc_sumsq_static(f(64), 1000, torch.zeros(1, dtype=torch.float64))
    with pytest.raises(ValueError, match="norm2"):
        binding.acc_sumsq_static(f(64), 64, torch.zeros(0, dtype=torch.float64))
