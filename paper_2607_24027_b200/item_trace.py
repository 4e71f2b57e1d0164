"""Per-work-item timeline of the fused kernel (development aid).

    python -m paper_2607_24027_b200.item_trace [--heads 16] [--density 0.05] [--workload video720]

Builds ``libsol_attn_itrace.so`` (the product sources with ``-DSOL_ITEMTRACE``: a handful of clock reads per
work item in CTA 0, nothing per tile), runs one fused-kernel launch on cuda:0 and prints, for the first
work items of CTA 0, where their cycles go: tiles, the tile loop, the end-of-item epilogue (wait for the
last value GEMM, exchange of the two groups' (m, l), merge + store), the gap to the next item's first
tile, and a least-squares fit ``cycles per item = a * tiles + b``; then how many work items every CTA
finished and when.  ``a`` is the steady cost of a tile, ``b`` the fixed cost of a work item.
"""
from __future__ import annotations

import argparse
import ctypes
import dataclasses
import os

import numpy as np

PKG = os.path.dirname(os.path.abspath(__file__))
N_ITEMS, N_SLOTS = 96, 16          # must match csrc/fwd_sm100_prof.cuh


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="video720")
    ap.add_argument("--heads", type=int, default=16)
    ap.add_argument("--density", type=float, default=0.05)
    args = ap.parse_args()

    from . import build as b
    lib_path = b._build_variant(os.path.join(PKG, "libsol_attn_itrace.so"), ["-DSOL_ITEMTRACE"], "_itrace", False)
    os.environ["SOL_ATTN_LIB"] = lib_path
    import torch
    from . import binding as sb, synth
    from .configs import WORKLOADS, load_betas

    wl = dataclasses.replace(WORKLOADS[args.workload], heads=args.heads)
    beta = load_betas()[args.workload][args.density]
    bits = synth.generate(wl)
    q, k, v = (torch.from_numpy(x.view(np.int16)).cuda().view(torch.bfloat16) for x in bits)
    out = torch.empty_like(q)
    ws = sb.make_workspace(wl.batch, wl.heads, wl.seq_len, wl.d, wl.block, wl.block)
    for it in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        sb.sol_attn_forward_ex(q, k, v, out, ws, wl.block, wl.block, threshold=beta, skip_pool=(it > 0))
        e1.record()
        torch.cuda.synchronize()
    print(f"{args.workload}, {args.heads} heads, density {args.density}: fused kernel {e0.elapsed_time(e1):.3f} ms")
    lib = sb.lib()
    buf = (ctypes.c_longlong * (N_ITEMS * N_SLOTS))()
    lib.sol_attn_debug_itemtrace(buf)
    a = np.array(buf[:], dtype=np.int64).reshape(N_ITEMS, N_SLOTS)
    rows = a[(a[:, 5] > 0) & (a[:, 9] > 0)]
    rows = rows[1:-1] if len(rows) > 4 else rows          # drop the first (cold) and the last recorded item
    nxt = a[2:len(rows) + 2, 5]
    tiles = rows[:, 10].astype(float)
    period = (nxt - rows[:, 5]).astype(float)
    print(f"CTA 0, {len(rows)} work items: tiles per item {tiles.mean():.1f}; cycles per item {period.mean():.0f} "
          f"({period.mean() / tiles.mean():.0f} per tile)")
    print(f"  tile loop (first scores seen -> last P written) {np.mean(rows[:, 6] - rows[:, 5]):.0f}")
    print(f"  epilogue {np.mean(rows[:, 9] - rows[:, 6]):.0f} = wait for the last value GEMM {np.mean(rows[:, 7] - rows[:, 6]):.0f}"
          f" + exchange of (m, l) {np.mean(rows[:, 8] - rows[:, 7]):.0f} + merge and store {np.mean(rows[:, 9] - rows[:, 8]):.0f}")
    print(f"  gap to the next item's first scores {np.mean(nxt - rows[:, 9]):.0f}")
    print(f"  router: first record {np.mean(rows[:, 1] - rows[:, 0]):.0f} cycles after it took the item, last record "
          f"{np.mean(rows[:, 2] - rows[:, 0]):.0f} (includes waiting for free records)")
    coef = np.linalg.lstsq(np.stack([tiles, np.ones_like(tiles)], 1), period, rcond=None)[0]
    print(f"  fit: cycles per item = {coef[0]:.0f} * tiles + {coef[1]:.0f}")
    cb = (ctypes.c_longlong * (256 * 4))()
    lib.sol_attn_debug_ctatrace(cb)
    c = np.array(cb[:], dtype=np.int64).reshape(256, 4)
    c = c[c[:, 3] > 0]
    t0 = c[:, 0].min()
    print(f"{len(c)} CTAs: work items per CTA min {c[:, 2].min()} median {int(np.median(c[:, 2]))} max {c[:, 2].max()}; "
          f"last tile done after {(c[:, 3].min() - t0) / 1e3:.0f}-{(c[:, 3].max() - t0) / 1e3:.0f} us")
    print("  CTAs with >= 10 % more items than the median:", np.flatnonzero(c[:, 2] >= 1.1 * np.median(c[:, 2])).tolist())


if __name__ == "__main__":
    main()
