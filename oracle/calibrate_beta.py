"""Calibrate the standardized cutoff beta of every workload to its target densities.

Test infrastructure: calls only the CPU oracle and the seeded input generator.  For each
workload every proxy row is standardised, z_ij = (s_ij - mu_i) / sigma_i (Eq. 4), and beta is
the (1 - rho)-quantile of z over all heads and rows, rounded to 4 decimals.  Writes
paper_2607_24027_b200/betas.json and prints the density each rounded beta achieves.

    python -m oracle.calibrate_beta [workload ...]
"""
from __future__ import annotations

import json
import os
import sys

import numpy as np

from oracle import sol_attn_oracle as orc
from paper_2607_24027_b200 import synth
from paper_2607_24027_b200.configs import DENSITY_SWEEP, WORKLOADS, _BETA_FILE


def calibrate(name: str):
    wl = WORKLOADS[name]
    zs = []
    for _b, _h, qb, kb, vb in synth.iter_heads(wl):
        r = orc.routing(synth.widen(qb, np.float64), synth.widen(kb, np.float64),
                        synth.widen(vb, np.float64), wl.block, wl.block, 0.0)
        zs.append(((r.s_hat - r.mu[:, None]) / r.sigma[:, None]).astype(np.float32).ravel())
    z = np.concatenate(zs)
    table = {}
    for rho in DENSITY_SWEEP[name]:
        beta = round(float(np.quantile(z, 1.0 - rho)), 4)
        achieved = float((z > beta).mean())
        print(f"{name}: target {rho:.2f} -> beta {beta:+.4f} (achieved {achieved:.4f}, "
              f"gaussian {orc.gaussian_density(beta):.4f})", flush=True)
        table[str(rho)] = beta
    return table


def main(argv):
    names = argv or list(WORKLOADS)
    out = {}
    if os.path.exists(_BETA_FILE):
        out = json.load(open(_BETA_FILE))
    for name in names:
        out[name] = calibrate(name)
        with open(_BETA_FILE, "w") as f:
            json.dump(out, f, indent=1, sort_keys=True)


if __name__ == "__main__":
    main(sys.argv[1:])
