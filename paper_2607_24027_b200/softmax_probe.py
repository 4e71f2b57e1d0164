"""Build and run the softmax-loop and barrier hand-over microbenchmarks (``csrc/probe_softmax.cu``) on cuda:0.

    python -m paper_2607_24027_b200.softmax_probe

Prints (1) SM cycles per 128 x 128 attention tile of the softmax warps' inner loop in isolation -- as the
fused kernel has it, without the exponentials, with a 3-input maximum, and with a cubic ``exp2`` on the FMA
pipes for a share of the elements -- for 8 warps (two per scheduler, the kernel's arrangement; 64 or 128
score columns per thread) and 4 warps; and (2) the cycles two threads of different warps need to pass an
mbarrier back and forth, on an idle SM and beside eight busy warps.  These are the figures the design notes
quote for the softmax-side and the hand-over cost of a tile.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)


def build() -> str:
    so = os.path.join(PKG, "libprobe_softmax.so")
    src = os.path.join(PKG, "csrc", "probe_softmax.cu")
    if not os.path.exists(so) or os.path.getmtime(so) < os.path.getmtime(src):
        nvcc = os.environ.get("NVCC") or "/usr/local/cuda/bin/nvcc"
        subprocess.run([nvcc if os.path.exists(nvcc) else "nvcc", "-std=c++17", "-O3", "-gencode",
                        "arch=compute_100a,code=sm_100a", "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(PKG, "csrc"),
                        "-I", os.path.join(ROOT, "include"), "-o", so, src], check=True)
    return so


def main():
    import torch
    lib = ctypes.CDLL(build())
    lib.run_probe_softmax.argtypes = [ctypes.c_void_p] + [ctypes.c_int] * 5
    lib.run_probe_handover.argtypes = [ctypes.c_void_p] + [ctypes.c_int] * 4
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    out = torch.zeros(sms * 16, dtype=torch.int64, device="cuda")
    variants = {0: "as in the kernel", 1: "no exp2", 2: "3-input maximum", 3: "cubic exp2 on 25 % of the pairs",
                4: "cubic exp2 on 37.5 %", 5: "cubic exp2 on 50 %", 6: "cubic exp2 on all"}
    iters = 400
    for cols, warps in ((64, 8), (128, 8), (64, 4)):
        tiles = warps * cols / 512.0                      # 128 x 128 tiles' worth of elements per pass of all warps
        for var, name in variants.items():
            for _ in range(2):
                out.zero_()
                if lib.run_probe_softmax(out.data_ptr(), var, cols, iters, sms, warps) != 0:
                    raise SystemExit("softmax probe failed")
            cyc = out.view(sms, 16)[:, :warps].float().mean().item() / iters
            print(f"softmax loop | {warps} warps x {cols:3d} columns | {name:32s}: {cyc / tiles:7.1f} cycles per tile "
                  f"({cyc / cols:5.2f} per element and warp)")
    tests = {0: "arrive -> try_wait, both ways", 1: "8 MMAs + tcgen05.commit -> try_wait; arrive back",
             2: "arrive -> test_wait spin, both ways", 3: "volatile flags, both ways"}
    rounds = 2000
    for busy in (0, 1):
        for test, name in tests.items():
            for _ in range(2):
                out.zero_()
                if lib.run_probe_handover(out.data_ptr(), test, busy, rounds, sms) != 0:
                    raise SystemExit("hand-over probe failed")
            o = out[:sms * 4].view(sms, 4).float()
            ok = int(o[:, 1].min().item())
            print(f"hand-over | {'8 busy warps' if busy else 'idle SM     '} | {name:50s}: {o[:, 0].mean().item() / rounds:7.1f} cycles per "
                  f"round trip{'' if ok else '  (a wait gave up)'}")


if __name__ == "__main__":
    main()
