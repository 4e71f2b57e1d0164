"""CPU-only checks of the product's host side: the C-ABI library loads and exports every symbol
declared in include/sol_attn.h, argument validation that needs no GPU, the input generator,
and the replica sharding used by multi-GPU runs (gloo, world_size 2)."""
import ctypes
import os
import re
import subprocess
import sys

import numpy as np
import pytest

from paper_2607_24027_b200 import synth
from paper_2607_24027_b200.configs import DENSITY_SWEEP, WORKLOADS, load_betas

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2607_24027_b200 import build as b
    from paper_2607_24027_b200 import binding
    b.build()
    return binding


def test_library_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "sol_attn.h")).read()
    declared = set(re.findall(r"\b(sol_attn_[a-z_]+)\s*\(", header))
    assert declared, "no declarations found"
    cdll = ctypes.CDLL(lib.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(cdll, name), f"{name} is declared in sol_attn.h but not exported"
    assert declared == set(lib.EXPORTS), (declared ^ set(lib.EXPORTS))


def test_status_strings_and_workspace_sizes(lib):
    assert lib.status_string(0) == "SOL_OK"
    assert lib.status_string(lib.SOL_ERR_DEVICE_TIMEOUT) == "SOL_ERR_DEVICE_TIMEOUT"
    assert lib.status_string(-99) == "SOL_ERR_UNKNOWN"
    small = lib.sol_attn_workspace_bytes(1, 2, 1024, 64, 64, 64)
    big = lib.sol_attn_workspace_bytes(1, 40, 75600, 128, 128, 128)
    assert 0 < small < big < 100 << 20
    assert small % 1024 == 0 and big % 1024 == 0
    # unsupported shapes have no workspace
    assert lib.sol_attn_workspace_bytes(1, 2, 1024, 96, 64, 64) == 0
    assert lib.sol_attn_workspace_bytes(1, 2, 0, 64, 64, 64) == 0
    assert lib.sol_attn_workspace_bytes(1, 2, 1024, 64, 2048, 64) == 0


def test_host_side_argument_errors_need_no_gpu(lib):
    L = lib.lib()
    # no workspace bound -> error before any CUDA call
    assert L.sol_attn_bind_workspace(None, 0, None) == lib.SOL_OK
    assert L.sol_attn_forward(16, 16, 16, 16, 1, 1, 128, 128, 128, 128, 0.5, None) == lib.SOL_ERR_WORKSPACE
    assert L.sol_attn_dense(16, 16, 16, 16, 1, 1, 128, 128, None) == lib.SOL_ERR_WORKSPACE
    assert L.sol_attn_forward_ex(None) == lib.SOL_ERR_INVALID_ARG
    # misaligned workspace pointer
    assert L.sol_attn_bind_workspace(ctypes.c_void_p(1000), 1 << 20, None) == lib.SOL_ERR_WORKSPACE
    # shape errors are reported before pointers are touched
    assert L.sol_attn_pool(None, 16, 16, 1, 1, 128, 96, 128, 128, 0.5, None) == lib.SOL_ERR_UNSUPPORTED_SHAPE
    assert L.sol_attn_pool(None, 16, 16, 1, 0, 128, 128, 128, 128, 0.5, None) == lib.SOL_ERR_INVALID_ARG
    assert L.sol_attn_launch_count() >= 0


def test_generator_is_deterministic_and_structured():
    wl = WORKLOADS["tiny"]
    a = synth.generate(wl)
    b = synth.generate(wl)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)
    q, k, v = a
    assert q.shape == (1, 2, 1024, 64) and q.dtype == np.uint16
    # a head's bits do not depend on which other heads were requested
    q1, k1, v1 = synth.generate(wl, heads=slice(1, 2))
    assert np.array_equal(q1[0], q[0, 1]) and np.array_equal(v1[0], v[0, 1])
    # bf16 rounding is round-to-nearest-even and exact on representable values
    x = np.array([1.0, 1.00390625, 1.001953125, -2.5, 3.0e38], dtype=np.float32)
    w = synth.widen(synth.f32_to_bf16_bits(x))
    assert w[0] == 1.0 and w[1] == 1.0 and w[3] == -2.5 and abs(w[2] - 1.0) < 1e-9
    # locality: same-position q/k are correlated through the shared position feature
    p = synth.position_features(wl.grid, wl.d)
    assert abs(np.mean(np.sum(p * p, axis=1)) - wl.d / 2) < 1e-3
    qf, kf = synth.widen(q[0, 0]), synth.widen(k[0, 0])
    same = np.mean(np.sum(qf * kf, axis=1))
    other = np.mean(np.sum(qf * np.roll(kf, 517, axis=0), axis=1))
    assert same > other + 5.0


def test_workloads_match_the_configured_shapes():
    assert WORKLOADS["tiny"].seq_len == 1024 and WORKLOADS["image"].seq_len == 4096
    assert WORKLOADS["video480"].seq_len == 32760 and WORKLOADS["video720"].seq_len == 75600
    assert WORKLOADS["edit"].seq_len == 65520
    assert WORKLOADS["video720"].n_blocks == 591 and WORKLOADS["edit"].n_blocks == 512
    betas = load_betas()
    for name, sweep in DENSITY_SWEEP.items():
        assert sorted(betas[name]) == sorted(sweep)
        vals = [betas[name][r] for r in sorted(sweep)]
        assert vals == sorted(vals, reverse=True), "a larger density needs a smaller beta"


def test_edit_workload_target_follows_source():
    import dataclasses
    wl = dataclasses.replace(WORKLOADS["edit"], heads=1, grid=(2, 6, 8))
    q, k, v = synth.generate(wl)
    seg = wl.seg_len
    src, tgt = synth.widen(k[0, 0, :seg]), synth.widen(k[0, 0, seg:])
    corr = np.corrcoef(src.ravel(), tgt.ravel())[0, 1]
    assert corr > 0.9


_GLOO_WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import numpy as np, torch, torch.distributed as dist
from paper_2607_24027_b200 import synth
from paper_2607_24027_b200.configs import WORKLOADS
import dataclasses
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
# the replica rule of bench.py: every rank runs the same shape with its own seed, no collective
# inside the operator; timing is max over ranks, throughput the sum
wl = WORKLOADS["tiny"]
wl_rank = dataclasses.replace(wl, seed=wl.seed + 1000 * rank) if rank else wl
q, k, v = synth.generate(wl_rank)
digest = torch.tensor([float(np.asarray(q, dtype=np.float64).sum() % 9973)])
gathered = [torch.zeros(1) for _ in range(world)]
dist.all_gather(gathered, digest)
ms = torch.tensor([10.0 + rank])
dist.all_reduce(ms, op=dist.ReduceOp.MAX)
if rank == 0:
    print(json.dumps({{"digests": [float(g.item()) for g in gathered], "ms": float(ms.item()), "world": world}}))
dist.destroy_process_group()
"""


def test_replica_sharding_over_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_GLOO_WORKER.format(root=ROOT))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29653", str(script)]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    res = json.loads(line)
    assert res["world"] == 2 and res["ms"] == 11.0
    assert res["digests"][0] != res["digests"][1], "ranks must draw different replicas"


def test_microbenchmarks_build_and_export_their_entry_points():
    """The tensor-core and softmax / hand-over probes cross-compile for sm_100a and load without a GPU."""
    from paper_2607_24027_b200 import mma_probe, softmax_probe
    mma = ctypes.CDLL(mma_probe.build())
    assert hasattr(mma, "run_probe_mma")
    soft = ctypes.CDLL(softmax_probe.build())
    assert hasattr(soft, "run_probe_softmax") and hasattr(soft, "run_probe_handover")
