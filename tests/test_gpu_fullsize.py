"""GPU parity at the full workload sizes, in the launch configuration bench.py times (all heads
of the workload in one call), at EVERY calibrated density of every video workload.

The oracle cannot run a whole 720p pass, so per workload the inputs are generated once and

* routing (mask, counts) is compared on ALL query blocks of ALL heads at every density -- it
  needs only the oracle's pooled tensors, computed once per head and re-thresholded per beta;
* outputs are compared on sampled query blocks of two heads per density (the heads rotate from
  density to density), always including the first block, the ragged last block, the blocks with
  the fewest / most routed keys and every block with an in-band mask flip (under both masks);
* properties that hold at any size are checked on the whole tensor: counts agree with the mask,
  the density is the calibrated one, outputs are finite and inside the per-channel range of V
  (every output row is a convex combination of value rows and block means), and the two kernel
  implementations agree with each other.

Each density prints one line: density, in-band blocks and flips over all heads, and the three
error figures of tests/helpers.py.
"""
import numpy as np
import pytest
import torch

from paper_2607_24027_b200 import synth
from paper_2607_24027_b200.configs import DENSITY_SWEEP, WORKLOADS, load_betas
from tests import helpers as hp

pytestmark = pytest.mark.gpu

sb = None


@pytest.fixture(scope="module", autouse=True)
def _lib():
    global sb
    from paper_2607_24027_b200 import binding
    sb = binding
    sb.lib()
    yield


def _sample_tiles(counts_h, n_extra, rng):
    nq = len(counts_h)
    tiles = {0, nq - 1, int(np.argmin(counts_h)), int(np.argmax(counts_h))}
    tiles.update(int(t) for t in rng.choice(nq, size=n_extra, replace=False))
    return sorted(tiles)


def _head64(bits, h):
    return tuple(synth.widen(x[0, h], np.float64) for x in bits)


def _run_workload(name, n_extra=2, cross_check_density=None):
    """All calibrated densities of one workload; returns what the dense-mode check needs."""
    wl = WORKLOADS[name]
    betas = load_betas()[name]
    bits = synth.generate(wl)
    q, k, v = (hp.to_dev(x) for x in bits)
    B, H, N, d = q.shape
    nk = wl.n_blocks
    # oracle pre-attention of every head, once (pooled tensors + proxy rows; beta comes later)
    routing = [hp.head_routing(*_head64(bits, h), wl.block) for h in range(H)]
    vmax = v.float().amax(dim=2, keepdim=True)
    vmin = v.float().amin(dim=2, keepdim=True)
    slack = 0.02 * (vmax - vmin) + 1e-2          # bf16 rounding of the output
    rng = np.random.default_rng(1)
    ws = None
    for n_density, rho in enumerate(DENSITY_SWEEP[name]):
        beta = betas[rho]
        out, counts, mask, ws = hp.run_gpu(q, k, v, wl.block, beta, ws=ws)
        counts_np = counts.cpu().numpy()
        # ---- whole-tensor properties
        assert np.array_equal(counts_np, mask.sum(axis=-1)), "counts disagree with the mask"
        density = counts_np.sum() / float(B * H * nk * nk)
        assert abs(density - rho) < 5e-3, density
        of = out.float()
        assert torch.isfinite(of).all()
        assert bool(((of <= vmax + slack) & (of >= vmin - slack)).all()), "output leaves the convex hull of V"
        if rho == cross_check_density:
            out2, counts2, mask2, _ = hp.run_gpu(q, k, v, wl.block, beta, impl=sb.SOL_IMPL_MMA_SYNC, ws=ws)
            assert np.array_equal(mask2, mask) and torch.equal(counts2, counts)
            assert float((out2.float() - of).abs().max()) <= 2 * hp.MAX_ABS
        # ---- the optional routing pre-pass in the same configuration: its decisions against the oracle on every
        #      head, its outputs bit-identical to the in-kernel router's wherever the two routed alike
        out_p, counts_p, mask_p, _ = hp.run_gpu(q, k, v, wl.block, beta, ws=ws, routing=sb.SOL_ROUTING_PREPASS)
        counts_p = counts_p.cpu().numpy()
        assert np.array_equal(counts_p, mask_p.sum(axis=-1))
        pre_flips = 0
        for h in range(H):
            _, _, tau, ref_mask = routing[h].at(beta)
            pre_flips += hp.check_mask(mask_p[0, h], counts_p[0, h], routing[h].s_hat, tau, ref_mask)["in_band_flips"]
        same = ~(mask_p != mask).any(axis=-1)[0]                                   # [H, Nq]
        rows_same = torch.from_numpy(np.repeat(same, wl.block, axis=1)[:, :N]).cuda()   # [H, N]
        assert bool((out_p.view(torch.int16)[0] == out.view(torch.int16)[0])[rows_same].all())
        pre_differ = int((~same).sum())
        del out_p
        # ---- routing of every head against the oracle
        agg = {}
        flipped_heads = []
        taus = []
        for h in range(H):
            _, _, tau, ref_mask = routing[h].at(beta)
            taus.append(tau)
            st = hp.check_mask(mask[0, h], counts_np[0, h], routing[h].s_hat, tau, ref_mask)
            if st["in_band_flips"]:
                flipped_heads.append(h)
            agg = hp.merge_stats(agg, st)
        # ---- outputs: two heads that rotate with the density, plus (up to two) heads with a flip
        heads = sorted({(7 * n_density) % H, (7 * n_density + H // 2 + 3) % H, *flipped_heads[:2]})
        for h in heads:
            qh, kh, vh = _head64(bits, h)
            tiles = _sample_tiles(counts_np[0, h], n_extra, rng)
            st = hp.check_head(qh, kh, vh, hp.dev_to_f64(out[0, h]), mask[0, h], counts_np[0, h], wl.block, beta,
                               tiles=tiles, routing=routing[h])
            st.pop("blocks"), st.pop("in_band_blocks"), st.pop("in_band_flips")   # already counted over all heads
            agg = hp.merge_stats(agg, st)
        print(f"{name} rho={rho}: density {density:.4f}; all {H} heads: in-band blocks {agg['in_band_blocks']} of "
              f"{agg['blocks']}, flips {agg['in_band_flips']}; outputs on heads {heads} ({agg['tiles']} query blocks): "
              f"max-abs {agg['max_abs']:.2e}, over |ref|<2 {agg['max_abs_ref_lt_2']:.2e}, vs bf16-rounded oracle "
              f"{agg['max_abs_vs_bf16_oracle']:.2e}, elements over 1e-2: {agg['n_over_1e-2']}, rel-L2 {agg['rel_l2']:.2e}, "
              f"max |ref| {agg['max_abs_out']:.2f}; routing pre-pass: flips {pre_flips}, query blocks routed unlike the "
              f"in-kernel router {pre_differ}, all others bit-identical")
    return wl, bits, (q, k, v), ws


def test_video480_fullsize():
    _run_workload("video480", cross_check_density=0.25)


def test_video720_fullsize_and_dense_mode():
    wl, bits, (q, k, v), ws = _run_workload("video720")
    # dense mode in the same launch configuration, sampled query blocks against Eq. (1)
    out, counts, _, _ = hp.run_gpu(q, k, v, wl.block, 0.0, mode=sb.SOL_MODE_DENSE, want_mask=False, ws=ws)
    assert (counts.cpu().numpy() == wl.n_blocks).all()
    agg = {}
    for h in (3, 39):
        qh, kh, vh = _head64(bits, h)
        for i in (0, 300, wl.n_blocks - 1):
            rows = slice(i * wl.block, min((i + 1) * wl.block, wl.seq_len))
            logits = (qh[rows] @ kh.T) / np.sqrt(wl.d)
            w = np.exp(logits - logits.max(axis=1, keepdims=True))
            ref = (w @ vh) / w.sum(axis=1, keepdims=True)
            agg = hp.merge_stats(agg, hp.error_stats(hp.dev_to_f64(out[0, h, rows]), ref))
    print(f"video720 dense mode: {agg}")


def test_edit_fullsize():
    _run_workload("edit")
