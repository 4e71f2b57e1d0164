#!/usr/bin/env python
"""Benchmark of the Sol-Attn fused forward path on synthetic video-DiT-shaped inputs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload video720] [--density 0.15] [--no-sweep] [--routing fused|prepass]

One "step" is one pass of the whole hot path (pooling pre-pass, thresholds, fused kernel) over
one batch (B=1, H=40, N=75600, d=128, block 128 for the default workload).  Prints ONE JSON line.

* value / unit: dense-equivalent TFLOP/s = 4*B*H*N^2*d / time, inputs resident in HBM.
* ms_per_step: ms per call (pool + fused kernel).
* e2e: the same metric through ``sol_attn_forward_host`` with pinned HOST buffers, i.e. with
  the host->device copies of q, k, v and the device->host copy of the output inside the timed
  region.
* roofline: the fused kernel alone (``skip_pool``), computed FLOPs (exact pairs actually routed +
  the approximate outer loop) per launch / CUDA-event time, against the measured bf16 peak.
* cpu_baseline: the CPU oracle timed on a bounded sample of the same workload.
* sweep: every density of the workload's threshold sweep plus the dense-mode run; every routed point also with the
  optional routing pre-pass (``routing_prepass``).  ``--routing prepass`` takes the headline numbers that way too.

Under torchrun ONE call is sharded by heads: rank r generates and processes only its own contiguous
range of the workload's heads (heads are independent; there is no collective on the data path), timing
is max over ranks and ``value`` is the whole job's dense-equivalent throughput (``scaling``: strong).
``--replicas`` makes every rank run the whole workload instead (weak scaling).
``--impl reference`` times the CPU oracle (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2607_24027_b200 import synth  # noqa: E402
from paper_2607_24027_b200.configs import DENSITY_SWEEP, WORKLOADS, load_betas  # noqa: E402
from paper_2607_24027_b200.shard import head_partition  # noqa: E402

METRIC = "dense-equivalent attention throughput at 720p (ms/call in ms_per_step)"
UNIT = "TFLOP/s (dense-equivalent)"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"bf16_burst": p["bf16_tflops"], "bf16_sustained": p.get("bf16_tflops_sustained"),
                "hbm_gbs": p["hbm_gbs"], "source": "measured"}
    return {"bf16_burst": 1590.0, "bf16_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


def measured_traffic(kernel, wl, n_heads):
    """DRAM bytes of one launch of `kernel`, from the ncu summary committed under profiles/ (written by
    ``python -m paper_2607_24027_b200.ncu_summary``): a small-case capture scaled by the head count
    (every tensor crosses HBM once per launch, so traffic grows with the heads).  None when no summary
    covers this workload."""
    path = os.path.join(ROOT, "profiles", f"{kernel}_{wl.name}.json")
    if not os.path.exists(path):
        return None, None
    rec = json.load(open(path))
    per_head = (rec["dram_bytes_read"] + rec["dram_bytes_write"]) / float(rec["heads"])
    return per_head * n_heads, {"file": os.path.relpath(path, ROOT), "captured_heads": rec["heads"],
                                "kernel_git_hash": rec.get("kernel_git_hash")}


def dense_flops(wl):
    return 4.0 * wl.batch * wl.heads * float(wl.seq_len) ** 2 * wl.d


def computed_flops(wl, counts_sum, mode_dense=False, n_bh=None):
    """Algorithmic FLOPs of one fused-kernel launch: routed (query block, key block) pairs are
    4*b*b*d each; the approximate outer loop is a b x Nk x d pair of GEMMs per query block."""
    b, d, nk = wl.block, wl.d, wl.n_blocks
    exact = float(counts_sum) * 4.0 * b * b * d
    if mode_dense:
        return exact
    approx = (wl.batch * wl.heads if n_bh is None else n_bh) * float(nk) * 4.0 * b * nk * d
    return exact + approx


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def __exit__(self, *exc):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self):
        sm, mx, reasons = [], 0.0, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0]))
                mx = max(mx, float(f[1]))
            except ValueError:
                continue
            for n, val in zip(names, f[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx or None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------ CPU oracle arm
_HEAD0 = {}


def _head0(wl):
    if wl.name not in _HEAD0:                 # input generation is not part of the timed work
        qb, kb, vb = synth.generate(wl, heads=slice(0, 1))
        _HEAD0[wl.name] = tuple(synth.widen(x[0], np.float64) for x in (qb, kb, vb))
    return _HEAD0[wl.name]


def oracle_head_slice(wl, beta, step, n_steps):
    """Time the oracle on the pre-attention step of head 0 plus the query blocks i = step (mod n_steps)
    of that head (Algorithm 1); n_steps = 1 is the whole head.  Returns (seconds extrapolated to the
    whole head, description, achieved density)."""
    from oracle import sol_attn_oracle as orc
    q, k, v = _head0(wl)
    t0 = time.perf_counter()
    r = orc.routing(q, k, v, wl.block, wl.block, beta)
    t_route = time.perf_counter() - t0
    nq = r.mask.shape[0]
    tiles = list(range(step % n_steps, nq, n_steps))
    t0 = time.perf_counter()
    orc.sol_attn_streaming(q, k, v, r.kc, r.vc, r.tau, wl.block, wl.block, chunk=16, q_tiles=tiles)
    t_tiles = time.perf_counter() - t0
    t_head = t_route + t_tiles * nq / len(tiles)
    what = (f"head 0 of {wl.batch * wl.heads}: pooling + thresholds of all {nq} query blocks, Algorithm 1 on "
            f"{len(tiles)} of them" + ("" if n_steps == 1 else f" (every {n_steps}th, offset by the step)"))
    return t_head, what, float(r.mask.mean())


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def run_reference(args, wl, beta):
    """The reference arm of this build is the CPU oracle, as it stands, on the host cores.  A whole 720p
    call is hours of float64 numpy, so each step times a bounded sample -- the pre-attention step of head 0
    and every K-th query block of it, K = the number of steps, so that the timed steps together cover the
    head once -- and extrapolates: x (blocks / sampled blocks) to the head, x heads to the call."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_bh = wl.batch * wl.heads
    times = []
    sample = ""
    n_slices = max(1, args.steps)
    for step in range(args.warmup + args.steps):
        t_head, sample, _ = oracle_head_slice(wl, beta, step, n_slices)
        if step >= args.warmup:
            times.append(t_head * n_bh)
    t = float(np.mean(times))
    val = dense_flops(wl) / t / 1e12
    note = f"{sample}; 1 head x {n_bh}, extrapolated"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{wl.name} density {args.density}", "B": wl.batch, "H": wl.heads,
                       "N": wl.seq_len, "d": wl.d, "block": wl.block, "beta": beta,
                       "extrapolated": note},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": note},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_ablation(sb, to_dev, name="image"):
    """rel-L2 / cosine of the output against dense attention (all on the GPU, same kernel in dense
    mode), for Sol-Attn and for keep-or-drop sparsity under the same routing; per-query-block
    density percentiles from the counts output."""
    import torch
    wl = WORKLOADS[name]
    qb, kb, vb = synth.generate(wl)
    q, k, v = to_dev(qb), to_dev(kb), to_dev(vb)
    B, H, N, d = q.shape
    ws = sb.make_workspace(B, H, N, d, wl.block, wl.block)
    dense, out = torch.empty_like(q), torch.empty_like(q)
    sb.sol_attn_forward_ex(q, k, v, dense, ws, wl.block, wl.block, mode=sb.SOL_MODE_DENSE)
    ref = dense.float()
    rows = []
    for rho, beta in sorted(load_betas()[name].items()):
        rec = {"target_density": rho, "beta": beta}
        for label, mode in (("sol", sb.SOL_MODE_SOL), ("exact_only", sb.SOL_MODE_EXACT_ONLY)):
            sb.sol_attn_forward_ex(q, k, v, out, ws, wl.block, wl.block, threshold=beta, mode=mode)
            o = out.float()
            rec[label + "_rel_l2"] = float((o - ref).norm() / ref.norm())
            rec[label + "_cosine"] = float(torch.nn.functional.cosine_similarity(o.flatten(), ref.flatten(), dim=0))
        dens = ws.counts.float().flatten() / wl.n_blocks
        rec["density"] = float(dens.mean())
        rec["per_block_density_p10_p50_p90"] = [float(x) for x in torch.quantile(dens, torch.tensor([0.1, 0.5, 0.9], device=dens.device))]
        rows.append(rec)
    torch.cuda.synchronize()
    return {"workload": name, "rows": rows}


# ------------------------------------------------------------------------------------------ GPU arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="video720", choices=list(WORKLOADS))
    ap.add_argument("--density", type=float, default=0.15)
    ap.add_argument("--kernel", default="auto", choices=["auto", "tcgen05", "mma_sync"])
    ap.add_argument("--routing", default="fused", choices=["fused", "prepass"],
                    help="where Eq. (4) is decided for the headline numbers: inside the fused kernel (the paper's structure, default) or by the optional pre-pass kernel")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--heads", type=int, default=0, help="override the head count (profiling small cases)")
    ap.add_argument("--replicas", action="store_true",
                    help="multi-GPU: every rank runs the whole workload (weak scaling) instead of a head shard")
    args = ap.parse_args()

    wl = WORKLOADS[args.workload]
    if args.heads:
        import dataclasses
        wl = dataclasses.replace(wl, heads=args.heads)
    betas = load_betas()[args.workload]
    if args.density not in betas:
        raise SystemExit(f"density {args.density} not calibrated for {args.workload}: {sorted(betas)}")
    beta = betas[args.density]

    if args.impl == "reference":
        run_reference(args, wl, beta)
        return

    import torch
    import torch.distributed as dist
    from paper_2607_24027_b200 import binding as sb

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    sb.lib()   # fails loudly when the CUDA library is missing

    impl = {"auto": sb.SOL_IMPL_AUTO, "tcgen05": sb.SOL_IMPL_TCGEN05, "mma_sync": sb.SOL_IMPL_MMA_SYNC}[args.kernel]

    # inputs: generated on the host by the seeded generator, then kept resident in HBM
    import dataclasses
    if world > 1 and not args.replicas:
        # one call sharded by heads: this rank's contiguous range of (batch, head) pairs, nothing else
        mine = head_partition(wl.batch * wl.heads, world, rank)
        qb, kb, vb = (x[None] for x in synth.generate(wl, heads=mine))       # [1, n_local, N, d]
        if qb.shape[1] == 0:
            raise SystemExit(f"rank {rank} of {world} owns no head of {wl.batch * wl.heads}")
        job_flops = dense_flops(wl)                                           # the whole job, whatever N
    else:
        wl_rank = dataclasses.replace(wl, seed=wl.seed + 1000 * rank) if rank else wl
        qb, kb, vb = synth.generate(wl_rank)
        job_flops = world * dense_flops(wl)
    to_dev = lambda x: torch.from_numpy(x.view(np.int16)).cuda().view(torch.bfloat16)
    q, k, v = to_dev(qb), to_dev(kb), to_dev(vb)
    out = torch.empty_like(q)
    B, H, N, d = q.shape
    ws = sb.make_workspace(B, H, N, d, wl.block, wl.block)
    sb.sol_attn_bind_workspace(ws)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def timed(fn, steps, warmup):
        """ms per step: CUDA events on the launching stream, max over ranks."""
        for _ in range(warmup):
            fn()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        barrier()
        ms = e0.elapsed_time(e1) / steps
        if world > 1:
            t = torch.tensor([ms], device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms

    def check_status():
        st = sb.sol_attn_read_device_status()
        if st != sb.SOL_OK:
            raise SystemExit(f"device status {sb.status_string(st)}")

    def full_step(b=beta):
        if args.routing == "prepass":
            return prepass_step(b)
        sb.sol_attn_forward_ex(q, k, v, out, ws, wl.block, wl.block, threshold=b, impl=impl)

    def kernel_only(b=beta):
        if args.routing == "prepass":
            return prepass_step(b, True)
        sb.sol_attn_forward_ex(q, k, v, out, ws, wl.block, wl.block, threshold=b, impl=impl, skip_pool=True)

    mask_buf = torch.zeros(B, H, wl.n_blocks, sb.mask_words(wl.n_blocks), dtype=torch.int32, device="cuda")

    def prepass_step(b=beta, skip_pool=False):   # Eq. (4) decided by the pre-pass kernel, one bit per block pair
        sb.sol_attn_forward_ex(q, k, v, out, ws, wl.block, wl.block, threshold=b, impl=impl, skip_pool=skip_pool,
                               routing=sb.SOL_ROUTING_PREPASS, mask_out=mask_buf)

    def dense_step():
        sb.sol_attn_forward_ex(q, k, v, out, ws, wl.block, wl.block, mode=sb.SOL_MODE_DENSE, impl=impl)

    def pool_only():
        sb.sol_attn_pool(q, k, v, wl.block, wl.block, beta)

    def pool_kv_only():                      # the pooling kernel alone (no thresholds): K and V
        sb.sol_attn_pool(None, k, v, wl.block, wl.block, beta)

    dflops = 4.0 * B * H * float(N) ** 2 * d          # dense-equivalent work of THIS rank's heads
    peaks = load_peaks()

    # ---- headline: whole path, inputs resident
    launches0 = sb.sol_attn_launch_count()
    with ClockSampler(local) as clk:
        ms_step = timed(full_step, args.steps, args.warmup)
    launches = (sb.sol_attn_launch_count() - launches0) * args.steps // (args.steps + args.warmup)
    check_status()
    counts_sum = int(ws.counts.sum().item())
    density = counts_sum / float(B * H * wl.n_blocks * wl.n_blocks)

    # ---- fused kernel alone (workspace already holds the pre-attention results)
    ms_kernel = timed(kernel_only, args.steps, 1)
    cflops = computed_flops(wl, counts_sum, n_bh=B * H)
    achieved = cflops / (ms_kernel * 1e-3) / 1e12
    ms_pool = timed(pool_only, args.steps, 1)
    ms_pool_kv = timed(pool_kv_only, args.steps, 1)
    pool_bytes = 2.0 * B * H * N * d * 2 + 2.0 * B * H * wl.n_blocks * d * 4 + 2.0 * B * H * wl.n_blocks * d * 2
    check_status()

    # ---- end to end with host buffers
    hq, hk, hv = (torch.from_numpy(x.view(np.int16)).pin_memory() for x in (qb, kb, vb))
    hout = torch.empty_like(hq).pin_memory()
    dq, dk, dv, dout = (torch.empty_like(q) for _ in range(4))

    def e2e_step():
        sb.sol_attn_forward_host(hq, hk, hv, hout, dq, dk, dv, dout, wl.block, wl.block, beta)

    ms_e2e = timed(e2e_step, max(2, args.steps // 2), 1)
    check_status()
    a_host = hout.view(-1)[:65536].view(torch.bfloat16).float()
    a_dev = out.view(-1)[:65536].float().cpu()
    assert float((a_host - a_dev).abs().max()) <= 2e-2, "host path disagrees with the device path"
    del hq, hk, hv, hout, dq, dk, dv, dout

    # ---- sweep: every calibrated density + dense mode (kernel-only and whole path)
    sweep = []
    if not args.no_sweep:
        ms_dense = timed(dense_step, max(2, args.steps // 3), 1)
        dense_cf = computed_flops(wl, B * H * wl.n_blocks * wl.n_blocks, mode_dense=True)
        sweep.append({"mode": "dense", "ms_per_call": ms_dense, "dense_equiv_tflops": dflops / ms_dense / 1e9,
                      "frac_of_peak_computed": dense_cf / ms_dense / 1e9 / peaks["bf16_burst"]})
        for rho in DENSITY_SWEEP[args.workload]:
            b = betas[rho]
            ms_f = timed(lambda: full_step(b), max(3, args.steps // 2), 1)
            cs = int(ws.counts.sum().item())
            ms_k = timed(lambda: kernel_only(b), max(3, args.steps // 2), 1)
            dens = cs / float(B * H * wl.n_blocks * wl.n_blocks)
            cf = computed_flops(wl, cs, n_bh=B * H)
            entry = {"mode": "sol", "target_density": rho, "beta": b, "density": dens,
                     "ms_per_call": ms_f, "kernel_ms": ms_k, "dense_equiv_tflops": dflops / ms_f / 1e9,
                     "computed_tflops": cf / ms_k / 1e9,
                     "frac_of_peak_computed": cf / ms_k / 1e9 / peaks["bf16_burst"],
                     "speedup_vs_dense": ms_dense / ms_f, "one_over_density": 1.0 / dens}
            if impl != sb.SOL_IMPL_MMA_SYNC:
                # the optional routing pre-pass (SOL_ROUTING_PREPASS): whole call, and mask kernel + fused kernel
                ms_pf = timed(lambda: prepass_step(b), max(3, args.steps // 2), 1)
                ms_pk = timed(lambda: prepass_step(b, True), max(3, args.steps // 2), 1)
                entry["routing_prepass"] = {"ms_per_call": ms_pf, "mask_and_fused_kernel_ms": ms_pk,
                                            "frac_of_peak_computed": cf / ms_pk / 1e9 / peaks["bf16_burst"],
                                            "speedup_vs_dense": ms_dense / ms_pf}
            sweep.append(entry)
        check_status()

    # ---- routing latency: the thresholds of Eq. (4)/(5) (what the method needs before its single
    #      pass) against the materialised baselines -- proxy map written to HBM, rows sorted,
    #      top-k / top-p cut -- on the same pooled tensors
    routing = None
    if not args.no_sweep and world == 1 and wl.n_blocks <= 8192:
        nb = wl.n_blocks
        pmap = torch.empty(B, H, nb, nb, device="cuda")
        order = torch.empty(B, H, nb, nb, dtype=torch.int32, device="cuda")
        tau_b = torch.empty(B, H, nb, device="cuda")
        cnt_b = torch.empty(B, H, nb, dtype=torch.int32, device="cuda")
        k_blocks = max(1, int(round(args.density * nb)))
        ms_thr = timed(lambda: sb.sol_attn_thresholds(B, H, N, d, wl.block, wl.block, beta), args.steps, 1)
        ms_topk = timed(lambda: sb.sol_attn_route_materialized(ws.qbar, ws.kc, sb.SOL_ROUTE_TOPK, k_blocks, pmap,
                                                               tau_b, order=order, counts=cnt_b), args.steps, 1)
        ms_topp = timed(lambda: sb.sol_attn_route_materialized(ws.qbar, ws.kc, sb.SOL_ROUTE_TOPP, 0.9, pmap,
                                                               tau_b, order=order, counts=cnt_b), args.steps, 1)
        mu_s, sg_s, tau_s = (torch.empty(B, H, nb, device="cuda") for _ in range(3))
        ms_thr_static = None
        if B * H * d * (d + 1) <= sb.sol_attn_thresholds_static_max_floats():
            qbar_c, kc_c = ws.qbar.contiguous(), ws.kc.contiguous()
            ms_thr_static = timed(lambda: sb.sol_attn_thresholds_static(qbar_c, kc_c, beta, mu_s, sg_s, tau_s),
                                  args.steps, 1)
        ms_mask = timed(lambda: sb.sol_attn_route_mask(B, H, N, d, wl.block, wl.block, mask_buf), args.steps, 1)
        routing = {"thresholds_ms": ms_thr, "thresholds_static_ms": ms_thr_static, "mask_prepass_ms": ms_mask,
                   "mask_prepass_bytes": int(mask_buf.numel() * 4),
                   "topk_ms": ms_topk, "topp_ms": ms_topp,
                   "topk_over_thresholds": ms_topk / ms_thr, "topp_over_thresholds": ms_topp / ms_thr,
                   "materialised_bytes": int(pmap.numel() * 4 + order.numel() * 4),
                   "note": "thresholds: mean, covariance and tau kernels on pooled data (nothing of size Nq x Nk "
                           "exists); mask_prepass: the optional SOL_ROUTING_PREPASS kernel, one bit per block pair; baselines: "
                           "proxy map + routing indices in HBM, k = %d blocks, p = 0.9" % k_blocks}
        check_status()

    # ---- accuracy ablation on the image workload (small): error against dense attention of the
    #      full method vs keep-or-drop block-sparse attention under the SAME mask, and the spread of
    #      per-query-block densities (the counts output)
    ablation = None
    if not args.no_sweep and world == 1:
        ablation = run_ablation(sb, to_dev)

    if world > 1:
        dist.barrier()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- CPU oracle on a bounded sample (rank 0, single-GPU runs only)
    cpu = None
    if world == 1 and not args.no_cpu:
        t_head, sample, _ = oracle_head_slice(wl, beta, 0, 1)          # one whole head, timed once
        t_cpu = t_head * B * H
        cpu = {"value": dflops / t_cpu / 1e12, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
               "sample": sample + f"; {t_head:.1f} s for the head; 1 head x {B * H}, extrapolated"}

    traffic, traffic_src = measured_traffic("fwd_sm100_kernel" if args.kernel != "mma_sync" else "fwd_mma_sync_kernel",
                                            wl, B * H)
    line = {
        "metric": METRIC, "value": job_flops / (ms_step * 1e-3) / 1e12, "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step,
        "higher_is_better": True, "scaling": "weak" if args.replicas else "strong",
        "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": f"{wl.name} density {args.density}", "B": B, "H": H, "N": N, "d": d,
                   "block": wl.block, "beta": beta, "achieved_density": density, "kernel": args.kernel, "routing": args.routing,
                   "l2": "inputs (3 x %.0f MB) larger than L2" % (q.numel() * 2 / 1e6),
                   "parallelism": ("single GPU" if world == 1 else "replicas (no collective)" if args.replicas else
                                   f"one call sharded by heads: {H} of {wl.batch * wl.heads} heads on this rank, "
                                   "no collective on the data path")},
        "clocks": clk.summary(),
        "e2e": {"value": job_flops / (ms_e2e * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": ms_e2e,
                # all ranks together: every rank copies its own q, k, v in and its own output back
                "h2d_bytes_per_step": 3 * q.numel() * 2 * (world if args.replicas else 1) if world == 1 or args.replicas
                else 3 * wl.batch * wl.heads * N * d * 2,
                "d2h_bytes_per_step": q.numel() * 2 * (world if args.replicas else 1) if world == 1 or args.replicas
                else wl.batch * wl.heads * N * d * 2},
        "gpu_launches": int(launches),
        "roofline": {"bound": "tensor", "kernel": "fwd_sm100_kernel" if args.kernel != "mma_sync" else "fwd_mma_sync_kernel",
                     "achieved": achieved, "peak": peaks["bf16_burst"], "unit": "TFLOP/s",
                     "frac": achieved / peaks["bf16_burst"], "peak_source": peaks["source"] + " burst",
                     "frac_of_sustained": (achieved / peaks["bf16_sustained"]) if peaks["bf16_sustained"] else None,
                     "kernel_ms": ms_kernel, "computed_flops": cflops,
                     # dram__bytes_read + dram__bytes_write of one launch, read from the ncu summary under
                     # profiles/ (a small-case capture scaled by the head count)
                     "traffic": traffic, "traffic_source": traffic_src,
                     # the HBM-bound pre-pass: the pooling kernel alone on K and V (2 of the 3 tensors; q is
                     # pooled by the same kernel), bytes = K + V read once + their pooled copies written
                     "pool": {"bound": "hbm", "kernel": "pool_kernel", "ms": ms_pool_kv, "bytes": pool_bytes,
                              "achieved": pool_bytes / (ms_pool_kv * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                              "unit": "GB/s", "frac": pool_bytes / (ms_pool_kv * 1e-3) / 1e9 / peaks["hbm_gbs"],
                              "pre_attention_ms": ms_pool},
                     "pool_frac": pool_bytes / (ms_pool_kv * 1e-3) / 1e9 / peaks["hbm_gbs"]},
        "cpu_baseline": cpu,
        "sweep": sweep,
        "ablation": ablation,
        "routing": routing,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
