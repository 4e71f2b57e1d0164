"""The five synthetic workloads and their calibrated standardized cutoffs (beta).

Shapes follow the paper's use cases: a small smoke case, an image DiT, 480p and 720p
video DiTs (81 frames -> 21 latent frames) and a video-editing sequence (source + target
concatenated).  ``BETAS`` maps workload name -> {target density: beta}; the values are
written by ``oracle/calibrate_beta.py`` (which calls only the CPU oracle and the input
generator) into ``betas.json`` next to this file.
"""
from __future__ import annotations

import json
import os

from .synth import Workload

WORKLOADS = {
    "tiny": Workload("tiny", batch=1, heads=2, d=64, grid=(4, 16, 16), block=64, seed=0),
    "image": Workload("image", batch=1, heads=24, d=128, grid=(1, 64, 64), block=128, seed=0),
    "video480": Workload("video480", batch=1, heads=40, d=128, grid=(21, 30, 52), block=128, seed=0,
                         sinks=True),
    "video720": Workload("video720", batch=1, heads=40, d=128, grid=(21, 45, 80), block=128, seed=0,
                         sinks=True),
    "edit": Workload("edit", batch=1, heads=40, d=128, grid=(21, 30, 52), block=128, seed=0,
                     sinks=True, edit=True),
}

# target densities of each workload's threshold sweep
DENSITY_SWEEP = {
    "tiny": [0.30],
    "image": [0.20, 0.30, 0.40, 0.50, 0.60],
    "video480": [0.25],
    "video720": [0.05, 0.10, 0.15, 0.25, 0.50],
    "edit": [0.10, 0.15, 0.25, 0.50],
}

_BETA_FILE = os.path.join(os.path.dirname(os.path.abspath(__file__)), "betas.json")


def load_betas():
    with open(_BETA_FILE) as f:
        raw = json.load(f)
    return {name: {float(rho): float(beta) for rho, beta in table.items()} for name, table in raw.items()}


def beta_for(name: str, density: float) -> float:
    return load_betas()[name][float(density)]
