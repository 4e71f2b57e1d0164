"""Build and run the tcgen05 MMA microbenchmark (``csrc/probe_mma.cu``) on cuda:0.

    python -m paper_2607_24027_b200.mma_probe

Prints SM cycles per attention tile (8 score MMAs + 8 value MMAs, 128x128x16 each) for the operand
placements the fused kernel can choose from, alone and beside bulk copies of 64 KB per tile into shared
memory, on one SM and on all of them.  These figures are the tensor-side floor quoted in the design
notes: the arithmetic alone would take 16 x 64 = 1024 cycles.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)


def build() -> str:
    so = os.path.join(PKG, "libprobe_mma.so")
    src = os.path.join(PKG, "csrc", "probe_mma.cu")
    if not os.path.exists(so) or os.path.getmtime(so) < os.path.getmtime(src):
        nvcc = os.environ.get("NVCC") or "/usr/local/cuda/bin/nvcc"
        subprocess.run([nvcc if os.path.exists(nvcc) else "nvcc", "-std=c++17", "-O3", "-gencode",
                        "arch=compute_100a,code=sm_100a", "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(PKG, "csrc"),
                        "-I", os.path.join(ROOT, "include"), "-o", so, src], check=True)
    return so


def main():
    import torch
    lib = ctypes.CDLL(build())
    lib.run_probe_mma.argtypes = [ctypes.c_void_p, ctypes.c_void_p] + [ctypes.c_int] * 4
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    src_bytes = 256 << 10                                   # per CTA; all CTAs together stay inside L2
    out = torch.zeros(sms * 4, dtype=torch.int64, device="cuda")
    src = torch.zeros(sms * src_bytes, dtype=torch.uint8, device="cuda")
    names = {0: "scores shared x shared, values TMEM x shared", 1: "  + 64 KB/tile of bulk copies",
             2: "scores TMEM x shared, values TMEM x shared", 3: "  + 64 KB/tile of bulk copies",
             8: "scores TMEM x shared in two 64-column halves", 9: "  + 64 KB/tile of bulk copies", 5: "bulk copies alone"}
    iters = 512
    for grid in (1, sms):
        for mode in (0, 1, 2, 3, 8, 9, 5):
            for _ in range(2):
                out.zero_()
                if lib.run_probe_mma(out.data_ptr(), src.data_ptr(), mode, iters, grid, src_bytes) != 0:
                    raise SystemExit("probe failed")
            o = out.view(sms, 4)[:grid].float()
            print(f"{grid:3d} CTA(s)  {names[mode]:48s} MMAs {o[:, 0].mean().item() / iters:7.1f} cycles/tile "
                  f"(issue alone {o[:, 2].mean().item() / iters:7.1f})   copies {o[:, 1].mean().item() / iters:7.1f} cycles/tile")


if __name__ == "__main__":
    main()
