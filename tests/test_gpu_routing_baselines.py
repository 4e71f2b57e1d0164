"""Materialised top-k / top-p routing (the paper's comparison policies) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import sol_attn_oracle as orc
from paper_2607_24027_b200 import synth
from tests import helpers as hp
from tests.test_gpu_parity import _small_problem

pytestmark = pytest.mark.gpu

sb = None


@pytest.fixture(scope="module", autouse=True)
def _lib():
    global sb
    from paper_2607_24027_b200 import binding
    sb = binding
    sb.lib()
    yield


def _route(bits, block, policy, param, want_order=True):
    q, k, v = (hp.to_dev(x) for x in bits)
    B, H, N, d = q.shape
    ws = sb.make_workspace(B, H, N, d, block, block)
    sb.sol_attn_bind_workspace(ws)
    sb.sol_attn_pool(q, k, v, block, block, 0.0)
    nq, nk = ws.view.n_q_blocks, ws.view.n_k_blocks
    pmap = torch.full((B, H, nq, nk), float("nan"), device="cuda")
    tau = torch.empty(B, H, nq, device="cuda")
    order = torch.full((B, H, nq, nk), -1, dtype=torch.int32, device="cuda") if want_order else None
    counts = torch.full((B, H, nq), -1, dtype=torch.int32, device="cuda")
    sb.sol_attn_route_materialized(ws.qbar, ws.kc, policy, param, pmap, tau, order=order, counts=counts)
    torch.cuda.synchronize()
    return (q, k, v, ws), pmap.cpu().numpy(), tau, (None if order is None else order.cpu().numpy()), counts.cpu().numpy()


def _oracle_rows(bits, b, h, block):
    qh, kh, vh = (synth.widen(x[b, h], np.float64) for x in bits)
    return qh, kh, vh, orc.routing(qh, kh, vh, block, block, 0.0)


@pytest.mark.parametrize("N,d,block,k", [(1500, 128, 128, 3), (1000, 64, 64, 5), (2100, 128, 128, 0), (700, 128, 128, 99)])
def test_topk_matches_the_oracle(N, d, block, k):
    B, H = 1, 2
    bits = _small_problem(41, B, H, N, d)
    dev, pmap, tau, order, counts = _route(bits, block, sb.SOL_ROUTE_TOPK, k)
    for h in range(H):
        qh, kh, vh, r = _oracle_rows(bits, 0, h, block)
        nk = r.s_hat.shape[1]
        assert np.abs(pmap[0, h] - r.s_hat).max() < 1e-4                       # the materialised proxy map, Eq. (3)
        mask_o, order_o, tau_o = orc.route_topk(r.s_hat, k)
        assert (counts[0, h] == min(k, nk)).all()
        # rows of the routing indices are permutations sorted by the GPU's own map
        assert (np.sort(order[0, h], axis=1) == np.arange(nk)[None, :]).all()
        sorted_vals = np.take_along_axis(pmap[0, h], order[0, h], axis=1)
        assert (np.diff(sorted_vals, axis=1) <= 0).all()
        # kept set = oracle's, except blocks whose score is within the tolerance band of the cut
        mask_g = np.zeros_like(mask_o)
        for i in range(mask_g.shape[0]):
            mask_g[i, order[0, h, i, :counts[0, h, i]]] = True
        diff = mask_g != mask_o
        if 0 < k < nk:
            band = np.abs(r.s_hat - tau_o[:, None]) < hp.BAND
            assert not (diff & ~band).any()
            assert np.abs(tau[0, h].cpu().numpy() - tau_o).max() < 1e-4
        else:
            assert not diff.any()


@pytest.mark.parametrize("p", [0.0, 0.3, 0.9, 1.0])
def test_topp_matches_the_oracle(p):
    B, H, N, d, block = 1, 2, 2300, 128, 128
    bits = _small_problem(42, B, H, N, d)
    # sharpen the proxy rows so that the mass is spread over a handful of blocks
    dev, pmap, tau, order, counts = _route(bits, block, sb.SOL_ROUTE_TOPP, p)
    for h in range(H):
        qh, kh, vh, r = _oracle_rows(bits, 0, h, block)
        nk = r.s_hat.shape[1]
        mask_o, order_o, tau_o, counts_o = orc.route_topp(r.s_hat, p)
        for i in range(r.s_hat.shape[0]):
            c = int(counts[0, h, i])
            if c == counts_o[i]:
                continue
            # a different count is only legitimate on a knife edge: the oracle's own mass at the
            # GPU's count must sit within rounding of p
            row = np.sort(r.s_hat[i])[::-1]
            w = np.exp(row - row[0])
            mass = np.cumsum(w) / w.sum()
            assert abs(c - counts_o[i]) == 1
            assert abs(mass[min(c, counts_o[i]) - 1] - p) < 1e-5, (i, c, counts_o[i])
        if p == 0.0:
            assert (counts[0, h] == 0).all() and np.isposinf(tau[0, h].cpu().numpy()).all()
        if p == 1.0:
            assert (counts[0, h] >= 1).all()


def test_materialised_policy_drives_the_fused_kernel():
    """tau from the top-k baseline, fed to the fused kernel as its threshold array, routes exactly
    the k best blocks; the output equals Algorithm 1 run under the oracle's top-k mask."""
    B, H, N, d, block, k = 1, 2, 1500, 128, 128, 4
    bits = _small_problem(43, B, H, N, d)
    (q, k_, v, ws), pmap, tau, order, counts = _route(bits, block, sb.SOL_ROUTE_TOPK, k)
    for impl in (sb.SOL_IMPL_TCGEN05, sb.SOL_IMPL_MMA_SYNC):
        out, cnt, mask, _ = hp.run_gpu(q, k_, v, block, 0.0, impl=impl, tau_override=tau, ws=ws)
        assert (cnt.cpu().numpy() == k).all()
        for h in range(H):
            qh, kh, vh, r = _oracle_rows(bits, 0, h, block)
            mask_o, _, tau_o = orc.route_topk(r.s_hat, k)
            band = np.abs(r.s_hat - tau_o[:, None]) < hp.BAND
            assert not ((mask[0, h] != mask_o) & ~band).any()
            ref, _ = orc.sol_attn_streaming(qh, kh, vh, r.kc, r.vc, tau_o, block, block, mask_override=mask[0, h])
            got = hp.dev_to_f64(out)[0, h]
            assert (np.abs(got - ref) <= hp.out_bound(ref)).all()
            assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= hp.REL_L2


def test_route_arguments_are_validated():
    bits = _small_problem(44, 1, 1, 512, 128)
    q, k, v = (hp.to_dev(x) for x in bits)
    ws = sb.make_workspace(1, 1, 512, 128, 128, 128)
    sb.sol_attn_bind_workspace(ws)
    sb.sol_attn_pool(q, k, v, 128, 128, 0.0)
    pmap = torch.empty(1, 1, 4, 4, device="cuda")
    tau = torch.empty(1, 1, 4, device="cuda")
    with pytest.raises(sb.SolAttnError):
        sb.sol_attn_route_materialized(ws.qbar, ws.kc, 7, 1.0, pmap, tau)
    with pytest.raises(sb.SolAttnError):
        sb.sol_attn_route_materialized(ws.qbar, ws.kc, sb.SOL_ROUTE_TOPP, 1.5, pmap, tau)
    with pytest.raises(sb.SolAttnError):
        sb.sol_attn_route_materialized(ws.qbar, ws.kc, sb.SOL_ROUTE_TOPK, float("nan"), pmap, tau)


def test_rethreshold_without_repooling():
    """sol_attn_thresholds recomputes tau for a new beta from the pooled tensors in the workspace:
    the result is what a full pool pass with that beta leaves, and it matches Eq. (4) in the oracle."""
    B, H, N, d, block = 1, 2, 1500, 128, 128
    bits = _small_problem(45, B, H, N, d)
    q, k, v = (hp.to_dev(x) for x in bits)
    ws = sb.make_workspace(B, H, N, d, block, block)
    sb.sol_attn_bind_workspace(ws)
    sb.sol_attn_pool(q, k, v, block, block, 0.3)
    tau_a = ws.tau.clone()
    sb.sol_attn_thresholds(B, H, N, d, block, block, 1.1)
    tau_b = ws.tau.clone()
    sb.sol_attn_pool(q, k, v, block, block, 1.1)
    torch.cuda.synchronize()
    assert torch.equal(tau_b, ws.tau) and not torch.equal(tau_a, tau_b)
    for h in range(H):
        r = orc.routing(*(synth.widen(x[0, h], np.float64) for x in bits), block, block, 1.1)
        assert np.abs(tau_b[0, h].cpu().numpy() - r.tau).max() < 1e-4
    # the diagonal estimator through the same entry point
    sb.sol_attn_thresholds(B, H, N, d, block, block, 1.1, estimator=sb.SOL_EST_DIAGONAL)
    torch.cuda.synchronize()
    for h in range(H):
        r = orc.routing(*(synth.widen(x[0, h], np.float64) for x in bits), block, block, 1.1, estimator="diagonal")
        assert np.abs(ws.tau[0, h].cpu().numpy() - r.tau).max() < 1e-4
