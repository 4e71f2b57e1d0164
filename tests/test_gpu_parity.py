"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on identical seeded bits."""
import math

import numpy as np
import pytest
import torch

from oracle import sol_attn_oracle as orc
from paper_2607_24027_b200 import synth
from paper_2607_24027_b200.configs import WORKLOADS, load_betas
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


IMPLS = ["mma_sync", "auto"]
IMPLS_128 = ["mma_sync", "tcgen05"]   # shapes with d = 128 and block 128 run on both kernels


def _impl(name):
    return {"mma_sync": sb.SOL_IMPL_MMA_SYNC, "auto": sb.SOL_IMPL_AUTO, "tcgen05": sb.SOL_IMPL_TCGEN05}[name]


def _small_problem(seed, B, H, N, d, structured=True):
    wl_grid = None
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((3, B, H, N, d)).astype(np.float32)
    if structured:
        t = np.linspace(0, 6, N, dtype=np.float32)[:, None] + np.arange(d, dtype=np.float32)[None, :] * 0.37
        x[0] += 0.8 * np.sin(t)
        x[1] += 0.8 * np.sin(t)
    bits = [synth.f32_to_bf16_bits(x[i]) for i in range(3)]
    return bits


def _check_all_heads(bits, block, beta, impl, mode=None, mode_name="sol", scale=0.0, tiles=None,
                     estimator="direct", forced=None, routing=0):
    qb, kb, vb = bits
    q, k, v = (hp.to_dev(x) for x in bits)
    mode = sb.SOL_MODE_SOL if mode is None else mode
    out, counts, mask, _ = hp.run_gpu(q, k, v, block, beta, mode=mode, impl=impl, scale=scale,
                                      estimator=(1 if estimator == "diagonal" else 0), forced=forced, routing=routing)
    B, H, N, d = q.shape
    out64 = hp.dev_to_f64(out)
    agg = {}
    for b in range(B):
        for h in range(H):
            st = hp.check_head(synth.widen(qb[b, h], np.float64), synth.widen(kb[b, h], np.float64),
                               synth.widen(vb[b, h], np.float64), out64[b, h], mask[b, h],
                               counts[b, h].cpu().numpy(), block, beta, tiles=tiles,
                               scale=(scale if scale > 0 else None), mode=mode_name, estimator=estimator,
                               forced=forced)
            agg = hp.merge_stats(agg, st)
    return agg


# ----------------------------------------------------------------------------- pre-attention
@pytest.mark.parametrize("name", ["tiny", "image"])
def test_pool_and_thresholds(name):
    wl = WORKLOADS[name]
    beta = list(load_betas()[name].values())[0]
    qb, kb, vb = synth.generate(wl)
    q, k, v = hp.to_dev(qb), hp.to_dev(kb), hp.to_dev(vb)
    ws = sb.make_workspace(wl.batch, wl.heads, wl.seq_len, wl.d, wl.block, wl.block)
    sb.sol_attn_bind_workspace(ws)
    sb.sol_attn_pool(q, k, v, wl.block, wl.block, beta)
    torch.cuda.synchronize()
    for h in range(wl.heads):
        r = orc.routing(synth.widen(qb[0, h], np.float64), synth.widen(kb[0, h], np.float64),
                        synth.widen(vb[0, h], np.float64), wl.block, wl.block, beta)
        np.testing.assert_allclose(ws.qbar[0, h].cpu().numpy(), r.qbar, rtol=0, atol=2e-6)
        np.testing.assert_allclose(ws.kc[0, h].cpu().numpy(), r.kc, rtol=0, atol=2e-6)
        np.testing.assert_allclose(ws.vc[0, h].cpu().numpy(), r.vc, rtol=0, atol=2e-4)
        np.testing.assert_allclose(ws.mu[0, h].cpu().numpy(), r.mu, rtol=0, atol=2e-5)
        np.testing.assert_allclose(ws.sigma[0, h].cpu().numpy(), r.sigma, rtol=1e-4, atol=2e-5)
        np.testing.assert_allclose(ws.tau[0, h].cpu().numpy(), r.tau, rtol=0, atol=5e-5)


def test_pool_ragged_and_odd_blocks():
    bits = _small_problem(3, 2, 3, 1000, 128)
    qb, kb, vb = bits
    q, k, v = (hp.to_dev(x) for x in bits)
    for bq, bk in [(128, 128), (64, 128), (100, 36), (1000, 1)]:
        ws = sb.make_workspace(2, 3, 1000, 128, bq, bk)
        sb.sol_attn_bind_workspace(ws)
        sb.sol_attn_pool(q, k, v, bq, bk, 0.7)
        torch.cuda.synchronize()
        for b in range(2):
            for h in range(3):
                r = orc.routing(synth.widen(qb[b, h], np.float64), synth.widen(kb[b, h], np.float64),
                                synth.widen(vb[b, h], np.float64), bq, bk, 0.7)
                np.testing.assert_allclose(ws.qbar[b, h].cpu().numpy(), r.qbar, rtol=0, atol=2e-6)
                np.testing.assert_allclose(ws.kc[b, h].cpu().numpy(), r.kc, rtol=0, atol=2e-6)
                np.testing.assert_allclose(ws.vc[b, h].cpu().numpy(), r.vc, rtol=0, atol=2e-4)
                np.testing.assert_allclose(ws.tau[b, h].cpu().numpy(), r.tau, rtol=0, atol=5e-5)


# ----------------------------------------------------------------------------- fused forward
@pytest.mark.parametrize("impl", IMPLS)
def test_tiny_all_tiles(impl):
    wl = WORKLOADS["tiny"]
    beta = load_betas()["tiny"][0.3]
    agg = _check_all_heads(synth.generate(wl), wl.block, beta, _impl(impl))
    print("tiny", impl, agg)


@pytest.mark.parametrize("impl", IMPLS_128)
@pytest.mark.parametrize("rho", [0.2, 0.3, 0.4, 0.5, 0.6])
def test_image_all_tiles(impl, rho):
    wl = WORKLOADS["image"]
    beta = load_betas()["image"][rho]
    agg = _check_all_heads(synth.generate(wl), wl.block, beta, _impl(impl))
    print("image", impl, rho, agg)


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("N,d,block", [(1000, 128, 128), (520, 128, 128), (50, 128, 128), (129, 128, 128),
                                       (1000, 64, 64), (333, 128, 64), (700, 64, 128)])
def test_ragged_shapes(impl, N, d, block):
    bits = _small_problem(N + d, 2, 2, N, d)
    agg = _check_all_heads(bits, block, 0.4, _impl(impl))
    print("ragged", impl, N, d, block, agg)


@pytest.mark.parametrize("impl", IMPLS_128)
@pytest.mark.parametrize("beta", [-math.inf, math.inf])
def test_select_all_and_none(impl, beta):
    bits = _small_problem(11, 1, 2, 900, 128)
    qb, kb, vb = bits
    agg = _check_all_heads(bits, 128, beta, _impl(impl))
    # select-all must also equal dense attention; select-none the pooled-sequence closed form
    q, k, v = (hp.to_dev(x) for x in bits)
    out, counts, mask, _ = hp.run_gpu(q, k, v, 128, beta, impl=_impl(impl))
    nk = mask.shape[-1]
    assert mask.all() if beta < 0 else not mask.any()
    assert (counts.cpu().numpy() == (nk if beta < 0 else 0)).all()
    if beta < 0:
        for h in range(2):
            ref = orc.dense_attention(synth.widen(qb[0, h], np.float64), synth.widen(kb[0, h], np.float64),
                                      synth.widen(vb[0, h], np.float64))
            assert (np.abs(hp.dev_to_f64(out)[0, h] - ref) <= hp.out_bound(ref)).all()


@pytest.mark.parametrize("impl", IMPLS_128)
def test_dense_mode(impl):
    bits = _small_problem(12, 1, 3, 777, 128)
    qb, kb, vb = bits
    q, k, v = (hp.to_dev(x) for x in bits)
    out, counts, _, ws = hp.run_gpu(q, k, v, 128, 0.0, mode=sb.SOL_MODE_DENSE, impl=_impl(impl), want_mask=False)
    assert (counts.cpu().numpy() == ws.view.n_k_blocks).all()
    o = hp.dev_to_f64(out)
    for h in range(3):
        ref = orc.dense_attention(synth.widen(qb[0, h], np.float64), synth.widen(kb[0, h], np.float64),
                                  synth.widen(vb[0, h], np.float64))
        assert (np.abs(o[0, h] - ref) <= hp.out_bound(ref)).all()
        assert np.linalg.norm(o[0, h] - ref) / np.linalg.norm(ref) <= hp.REL_L2


@pytest.mark.parametrize("impl", IMPLS_128)
def test_exact_only_mode_and_scale(impl):
    bits = _small_problem(13, 1, 2, 1024, 128)
    _check_all_heads(bits, 128, 0.3, _impl(impl), mode=sb.SOL_MODE_EXACT_ONLY, mode_name="exact_only")
    _check_all_heads(bits, 128, 0.3, _impl(impl), scale=0.05)


@pytest.mark.parametrize("impl", IMPLS_128)
def test_tau_override_and_determinism(impl):
    bits = _small_problem(14, 1, 2, 1024, 128)
    q, k, v = (hp.to_dev(x) for x in bits)
    out1, c1, m1, ws = hp.run_gpu(q, k, v, 128, 0.5, impl=_impl(impl))
    tau = ws.tau.clone()
    out2, c2, m2, _ = hp.run_gpu(q, k, v, 128, 99.0, impl=_impl(impl), tau_override=tau)
    assert np.array_equal(m1, m2) and torch.equal(c1, c2)
    assert torch.equal(out1.view(torch.int16), out2.view(torch.int16))   # run-to-run bit stability


# ----------------------------------------------------------------------------- host-side errors
# ----------------------------------------------------------------------------- routing pre-pass
@pytest.mark.parametrize("N,d,block", [(1000, 128, 128), (8329, 128, 128), (129, 128, 128), (1000, 64, 64),
                                       (333, 128, 64), (2500, 64, 128)])
def test_routing_prepass_matches_the_oracle(N, d, block):
    """Eq. (4) evaluated by the pre-pass kernel: mask, counts and outputs against the oracle, like the in-kernel router."""
    bits = _small_problem(N + d + 1, 2, 2, N, d)
    agg = _check_all_heads(bits, block, 0.4, sb.SOL_IMPL_AUTO, routing=sb.SOL_ROUTING_PREPASS)
    print("prepass", N, d, block, agg)


def test_routing_prepass_agrees_with_the_fused_router():
    """Same decisions as the in-kernel router outside the rounding band, hence the same outputs there; forced
    blocks, the keep-or-drop mode and the degenerate thresholds go through the pre-pass too."""
    wl = WORKLOADS["image"]
    beta = load_betas()["image"][0.3]
    bits = synth.generate(wl)
    q, k, v = (hp.to_dev(x) for x in bits)
    out_f, counts_f, mask_f, ws = hp.run_gpu(q, k, v, wl.block, beta)
    out_p, counts_p, mask_p, _ = hp.run_gpu(q, k, v, wl.block, beta, ws=ws, routing=sb.SOL_ROUTING_PREPASS)
    differ = mask_f != mask_p
    print("prepass vs fused: differing decisions", int(differ.sum()), "of", mask_f.size)
    assert differ.sum() <= 2                               # only pairs within rounding of the threshold
    same_rows = ~differ.any(axis=-1)                       # [B, H, Nq]
    of = out_f.view(torch.int16).cpu().numpy().reshape(wl.batch, wl.heads, -1, wl.block, wl.d)
    op = out_p.view(torch.int16).cpu().numpy().reshape(wl.batch, wl.heads, -1, wl.block, wl.d)
    assert np.array_equal(of[same_rows], op[same_rows])   # bit-identical where the routing is
    assert np.array_equal(counts_p.cpu().numpy(), mask_p.sum(axis=-1))
    agg = _check_all_heads(bits, wl.block, beta, sb.SOL_IMPL_AUTO, routing=sb.SOL_ROUTING_PREPASS)
    print("prepass image", agg)
    # the pre-pass as an entry point of its own (bound workspace) writes the same bits
    sb.sol_attn_bind_workspace(ws)
    alone = torch.zeros(wl.batch, wl.heads, wl.n_blocks, sb.mask_words(wl.n_blocks), dtype=torch.int32, device="cuda")
    launches = sb.sol_attn_launch_count()
    sb.sol_attn_route_mask(wl.batch, wl.heads, wl.seq_len, wl.d, wl.block, wl.block, alone)
    torch.cuda.synchronize()
    assert sb.sol_attn_launch_count() == launches + 1
    assert np.array_equal(hp.unpack_mask(alone, wl.n_blocks), mask_p)
    with pytest.raises(sb.SolAttnError) as e:
        sb.sol_attn_route_mask(wl.batch, wl.heads, wl.seq_len, wl.d, wl.block, wl.block, None)
    assert e.value.status == sb.SOL_ERR_INVALID_ARG
    # forced blocks, keep-or-drop mode, select-all / select-none
    small = _small_problem(23, 1, 2, 1500, 128)
    forced = np.zeros(12, dtype=bool)
    forced[[0, 5, 11]] = True
    _check_all_heads(small, 128, 0.9, sb.SOL_IMPL_AUTO, forced=forced, routing=sb.SOL_ROUTING_PREPASS)
    _check_all_heads(small, 128, 0.3, sb.SOL_IMPL_AUTO, mode=sb.SOL_MODE_EXACT_ONLY, mode_name="exact_only",
                     routing=sb.SOL_ROUTING_PREPASS)
    qs, ks, vs = (hp.to_dev(x) for x in small)
    for beta_inf, want in ((-math.inf, 12), (math.inf, 0)):
        _, counts, mask, _ = hp.run_gpu(qs, ks, vs, 128, beta_inf, routing=sb.SOL_ROUTING_PREPASS)
        assert (counts.cpu().numpy() == want).all() and (mask.sum(axis=-1) == want).all()


def test_routing_prepass_argument_rules():
    bits = _small_problem(16, 1, 1, 256, 128)
    q, k, v = (hp.to_dev(x) for x in bits)
    out = torch.empty_like(q)
    ws = sb.make_workspace(1, 1, 256, 128, 128, 128)
    mask = torch.zeros(1, 1, 2, 1, dtype=torch.int32, device="cuda")
    with pytest.raises(sb.SolAttnError) as e:              # the decisions need the caller's mask buffer
        sb.sol_attn_forward_ex(q, k, v, out, ws, 128, 128, threshold=0.5, routing=sb.SOL_ROUTING_PREPASS)
    assert e.value.status == sb.SOL_ERR_INVALID_ARG
    with pytest.raises(sb.SolAttnError) as e:              # only the tcgen05 kernel reads them
        sb.sol_attn_forward_ex(q, k, v, out, ws, 128, 128, threshold=0.5, routing=sb.SOL_ROUTING_PREPASS,
                               mask_out=mask, impl=sb.SOL_IMPL_MMA_SYNC)
    assert e.value.status == sb.SOL_ERR_INVALID_ARG
    with pytest.raises(sb.SolAttnError) as e:
        sb.sol_attn_forward_ex(q, k, v, out, ws, 128, 128, threshold=0.5, routing=7, mask_out=mask)
    assert e.value.status == sb.SOL_ERR_INVALID_ARG
    # dense mode has no routing: the option is ignored, no mask needed
    sb.sol_attn_forward_ex(q, k, v, out, ws, 128, 128, mode=sb.SOL_MODE_DENSE, routing=sb.SOL_ROUTING_PREPASS)
    torch.cuda.synchronize()


def test_argument_validation():
    bits = _small_problem(15, 1, 1, 256, 128)
    q, k, v = (hp.to_dev(x) for x in bits)
    out = torch.empty_like(q)
    ws = sb.make_workspace(1, 1, 256, 128, 128, 128)
    with pytest.raises(sb.SolAttnError) as e:
        sb.sol_attn_forward_ex(q, k, v, out, ws, 128, 64)
    assert e.value.status == sb.SOL_ERR_UNSUPPORTED_SHAPE
    with pytest.raises(sb.SolAttnError) as e:
        sb.sol_attn_forward_ex(q, k, v, out, ws, 32, 32)
    assert e.value.status == sb.SOL_ERR_UNSUPPORTED_SHAPE
    with pytest.raises(sb.SolAttnError) as e:
        sb.sol_attn_forward_ex(q, k, v, out, ws, 128, 128, threshold=float("nan"))
    assert e.value.status == sb.SOL_ERR_INVALID_ARG
    small = sb.make_workspace(1, 1, 256, 128, 128, 128)
    small.buf = small.buf[:small.buf.numel() - 2048]
    with pytest.raises(sb.SolAttnError) as e:
        sb.sol_attn_forward_ex(q, k, v, out, small, 128, 128)
    assert e.value.status == sb.SOL_ERR_WORKSPACE
    sb.sol_attn_bind_workspace(None)
    with pytest.raises(sb.SolAttnError) as e:
        sb.sol_attn_forward(q, k, v, out, 128, 128, 0.5)
    assert e.value.status == sb.SOL_ERR_WORKSPACE
    # misaligned pointer
    with pytest.raises(sb.SolAttnError) as e:
        sb.sol_attn_forward_ex(q.view(-1)[1:1 + 256 * 128 - 128].view(1, 1, 255, 128), k, v, out, ws, 128, 128)
    assert e.value.status in (sb.SOL_ERR_INVALID_ARG, sb.SOL_ERR_WORKSPACE)


def test_bound_entry_points_and_host_path():
    wl = WORKLOADS["tiny"]
    beta = load_betas()["tiny"][0.3]
    qb, kb, vb = synth.generate(wl)
    q, k, v = hp.to_dev(qb), hp.to_dev(kb), hp.to_dev(vb)
    ws = sb.make_workspace(wl.batch, wl.heads, wl.seq_len, wl.d, wl.block, wl.block)
    sb.sol_attn_bind_workspace(ws)
    out = torch.empty_like(q)
    sb.sol_attn_forward(q, k, v, out, wl.block, wl.block, beta)
    torch.cuda.synchronize()
    ref, _, _, _ = hp.run_gpu(q, k, v, wl.block, beta)
    assert torch.equal(out.view(torch.int16), ref.view(torch.int16))
    # host-buffer entry point
    hq, hk, hv = (torch.from_numpy(x.view(np.int16)).pin_memory() for x in (qb, kb, vb))
    hout = torch.empty_like(hq).pin_memory()
    dq, dk, dv, dout = (torch.empty_like(q) for _ in range(4))
    sb.sol_attn_bind_workspace(ws)
    sb.sol_attn_forward_host(hq, hk, hv, hout, dq, dk, dv, dout, wl.block, wl.block, beta)
    torch.cuda.synchronize()
    assert torch.equal(hout, ref.view(torch.int16).cpu())
    dense = torch.empty_like(q)
    sb.sol_attn_dense(q, k, v, dense)
    torch.cuda.synchronize()
    for h in range(wl.heads):
        refd = orc.dense_attention(synth.widen(qb[0, h], np.float64), synth.widen(kb[0, h], np.float64),
                                   synth.widen(vb[0, h], np.float64))
        assert (np.abs(hp.dev_to_f64(dense)[0, h] - refd) <= hp.out_bound(refd)).all()


def test_host_path_pipelined_over_head_groups(monkeypatch):
    """The host-buffer entry point cut into several groups of heads (copies on their own streams,
    kernels on the caller's) returns what one device-resident call returns, counts included."""
    B, H, N, d, block = 2, 5, 700, 128, 128
    bits = _small_problem(33, B, H, N, d)
    q, k, v = (hp.to_dev(x) for x in bits)
    ref, counts_ref, _, _ = hp.run_gpu(q, k, v, block, 0.7)
    ws = sb.make_workspace(B, H, N, d, block, block)
    sb.sol_attn_bind_workspace(ws)
    hq, hk, hv = (torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).pin_memory() for x in bits)
    dq, dk, dv, dout = (torch.empty_like(q) for _ in range(4))
    for group_bytes in (N * d * 2 * 3, N * d * 2, 1 << 30):            # 3 heads, 1 head, everything at once
        monkeypatch.setenv("SOL_ATTN_HOST_GROUP_BYTES", str(group_bytes))
        hout = torch.zeros_like(hq).pin_memory()
        ws.counts.fill_(-1)
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            sb.sol_attn_forward_host(hq, hk, hv, hout, dq, dk, dv, dout, block, block, 0.7)
            side.synchronize()
        assert torch.equal(hout, ref.view(torch.int16).cpu()), group_bytes
        assert torch.equal(ws.counts, counts_ref)
        assert sb.sol_attn_read_device_status() == sb.SOL_OK


@pytest.mark.parametrize("impl", IMPLS_128)
@pytest.mark.parametrize("jump", [3.0, 6.0])
def test_reference_maximum_jumps(impl, jump):
    """Late key blocks whose logits tower over everything before them: the running maximum has to
    be raised (moderately: before the next tile; hugely: the tile is recomputed) without losing
    the earlier blocks' exact contribution.  All queries share a direction u; the keys of the last
    third of the sequence get multiples of u, growing block by block."""
    B, H, N, d = 1, 2, 1536, 128
    rng = np.random.default_rng(99)
    x = rng.standard_normal((3, B, H, N, d)).astype(np.float32)
    u = rng.standard_normal(d).astype(np.float32)
    x[0] += u                                                   # q . u is about |u|^2 = 128
    for j, blk in enumerate(range(8, 12)):                      # blocks 8..11 of 12
        x[1][:, :, blk * 128:(blk + 1) * 128] += (j + 1) * jump * u   # logits rise by ~ jump * 11.3 nats per block
    bits = [synth.f32_to_bf16_bits(x[i]) for i in range(3)]
    for beta, mode, name in [(0.0, sb.SOL_MODE_DENSE, "sol"), (-0.2, sb.SOL_MODE_SOL, "sol"), (0.8, sb.SOL_MODE_SOL, "sol")]:
        if mode == sb.SOL_MODE_DENSE:
            qb, kb, vb = bits
            q, k, v = (hp.to_dev(t) for t in bits)
            out, _, _, _ = hp.run_gpu(q, k, v, 128, 0.0, mode=mode, impl=_impl(impl), want_mask=False)
            o = hp.dev_to_f64(out)
            for h in range(H):
                ref = orc.dense_attention(synth.widen(qb[0, h], np.float64), synth.widen(kb[0, h], np.float64),
                                          synth.widen(vb[0, h], np.float64))
                assert (np.abs(o[0, h] - ref) <= hp.out_bound(ref)).all()
        else:
            _check_all_heads(bits, 128, beta, _impl(impl))


# ----------------------------------------------------------------------------- beyond the core path
@pytest.mark.parametrize("impl", IMPLS_128)
def test_diagonal_threshold_estimator(impl):
    """Eq. (appendix_diagonal_threshold): sigma from the diagonal of the pooled-key covariance."""
    bits = _small_problem(21, 1, 3, 2048, 128)
    agg = _check_all_heads(bits, 128, 0.5, _impl(impl), estimator="diagonal")
    # the two estimators really differ on these inputs (otherwise the test pins nothing)
    qb, kb, vb = bits
    r_full = orc.routing(synth.widen(qb[0, 0], np.float64), synth.widen(kb[0, 0], np.float64),
                         synth.widen(vb[0, 0], np.float64), 128, 128, 0.5)
    r_diag = orc.routing(synth.widen(qb[0, 0], np.float64), synth.widen(kb[0, 0], np.float64),
                         synth.widen(vb[0, 0], np.float64), 128, 128, 0.5, estimator="diagonal")
    assert np.abs(r_full.tau - r_diag.tau).max() > 1e-3
    print("diagonal", impl, agg)


@pytest.mark.parametrize("impl", IMPLS_128)
def test_forced_exact_key_blocks(impl):
    """Key blocks flagged as always-exact (text / sink key-value tokens) enter every S_i."""
    bits = _small_problem(22, 1, 2, 1500, 128)
    nk = 12
    forced = np.zeros(nk, dtype=bool)
    forced[[0, 5, nk - 1]] = True                     # includes the ragged last block
    q, k, v = (hp.to_dev(x) for x in bits)
    out, counts, mask, _ = hp.run_gpu(q, k, v, 128, 0.9, impl=_impl(impl), forced=forced)
    assert mask[..., forced].all()
    assert (counts.cpu().numpy() >= 3).all()
    _check_all_heads(bits, 128, 0.9, _impl(impl), forced=forced)
    # forcing every block is dense attention
    allf = np.ones(nk, dtype=bool)
    out2, counts2, _, _ = hp.run_gpu(q, k, v, 128, 0.9, impl=_impl(impl), forced=allf)
    assert (counts2.cpu().numpy() == nk).all()
    for h in range(2):
        ref = orc.dense_attention(synth.widen(bits[0][0, h], np.float64), synth.widen(bits[1][0, h], np.float64),
                                  synth.widen(bits[2][0, h], np.float64))
        assert (np.abs(hp.dev_to_f64(out2)[0, h] - ref) <= hp.out_bound(ref)).all()


@pytest.mark.parametrize("impl,N,d,block", [("mma_sync", 1000, 64, 64), ("mma_sync", 1500, 128, 128),
                                            ("tcgen05", 1500, 128, 128)])
@pytest.mark.parametrize("mode_name", ["sol", "dense"])
def test_token_major_layout(impl, N, d, block, mode_name):
    """[B, N, H, d] inputs (heads interleaved per token) give bit for bit what [B, H, N, d] gives:
    only addresses change, not the arithmetic; one head is also checked against the oracle."""
    B, H = 2, 3
    bits = _small_problem(31, B, H, N, d)
    q, k, v = (hp.to_dev(x) for x in bits)
    mode = sb.SOL_MODE_SOL if mode_name == "sol" else sb.SOL_MODE_DENSE
    out, counts, mask, _ = hp.run_gpu(q, k, v, block, 0.8, mode=mode, impl=_impl(impl))
    qt, kt, vt = (x.permute(0, 2, 1, 3).contiguous() for x in (q, k, v))
    out_t, counts_t, mask_t, _ = hp.run_gpu(qt, kt, vt, block, 0.8, mode=mode, impl=_impl(impl),
                                            layout=sb.SOL_LAYOUT_BNHD)
    assert out_t.shape == (B, N, H, d)
    assert torch.equal(out_t.permute(0, 2, 1, 3).contiguous().view(torch.int16), out.view(torch.int16))
    assert torch.equal(counts_t, counts)
    assert np.array_equal(mask_t, mask)
    if mode_name == "sol":
        b, h = 1, 2
        hp.check_head(synth.widen(bits[0][b, h], np.float64), synth.widen(bits[1][b, h], np.float64),
                      synth.widen(bits[2][b, h], np.float64),
                      hp.dev_to_f64(out_t.permute(0, 2, 1, 3).contiguous())[b, h], mask_t[b, h],
                      counts_t[b, h].cpu().numpy(), block, 0.8)


def test_layout_argument_is_validated():
    bits = _small_problem(32, 1, 1, 256, 128)
    q, k, v = (hp.to_dev(x) for x in bits)
    ws = sb.make_workspace(1, 1, 256, 128, 128, 128)
    with pytest.raises(RuntimeError):
        sb.sol_attn_forward_ex(q, k, v, torch.empty_like(q), ws, 128, 128, threshold=0.5, layout=7)


# ----------------------------------------------------------------------------- degenerate inputs
@pytest.mark.parametrize("impl", IMPLS_128)
def test_degenerate_inputs(impl):
    """Cases in which the method's statistics collapse: zero queries and keys (every logit 0, sigma = 0,
    uniform attention), keys constant within each block (the proxy term is exact, so the output is
    dense attention whatever beta selects), a single token, exactly one block."""
    rng = np.random.default_rng(7)
    d, block = 128, 128
    # (a) zero q and k: out = mean of v over all tokens, nothing NaN, counts in range
    N = 700
    z = np.zeros((1, 1, N, d), dtype=np.float32)
    vb = synth.f32_to_bf16_bits(rng.standard_normal((1, 1, N, d)).astype(np.float32))
    zb = synth.f32_to_bf16_bits(z)
    q, k, v = hp.to_dev(zb), hp.to_dev(zb), hp.to_dev(vb)
    out, counts, mask, _ = hp.run_gpu(q, k, v, block, 0.5, impl=_impl(impl))
    want = synth.widen(vb[0, 0], np.float64).mean(axis=0)
    got = hp.dev_to_f64(out)[0, 0]
    assert np.isfinite(got).all()
    assert np.abs(got - want[None, :]).max() <= 1e-2
    c = counts.cpu().numpy()
    assert (c >= 0).all() and (c <= 6).all()
    # (b) keys constant within each block: Sol-Attn equals dense attention for every beta
    N = 900
    nb = (N + block - 1) // block
    kconst = np.repeat(rng.standard_normal((nb, d)).astype(np.float32), block, axis=0)[:N]
    qf = rng.standard_normal((N, d)).astype(np.float32)
    vf = rng.standard_normal((N, d)).astype(np.float32)
    bits = [synth.f32_to_bf16_bits(x[None, None]) for x in (qf, kconst, vf)]
    ref = orc.dense_attention(*(synth.widen(x[0, 0], np.float64) for x in bits))
    for beta in (-0.5, 0.8, math.inf):
        out, _, _, _ = hp.run_gpu(*(hp.to_dev(x) for x in bits), block, beta, impl=_impl(impl))
        got = hp.dev_to_f64(out)[0, 0]
        assert (np.abs(got - ref) <= hp.out_bound(ref)).all(), beta
        assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= hp.REL_L2
    # (c) one token; exactly one full block; more (batch, head) pairs than tokens per block
    for B, H, N in ((1, 1, 1), (1, 2, 128), (3, 7, 200)):
        bits = _small_problem(50 + N, B, H, N, d)
        _check_all_heads(bits, block, 0.4, _impl(impl))


@pytest.mark.parametrize("impl", IMPLS_128)
def test_cuda_graph_capture_and_replay(impl):
    """The whole call (status reset, pooling, thresholds, fused kernel) is plain stream work: it can
    be captured into a CUDA graph and replayed, with new input values in the same buffers."""
    bits = _small_problem(61, 1, 2, 1100, 128)
    q, k, v = (hp.to_dev(x) for x in bits)
    ws = sb.make_workspace(1, 2, 1100, 128, 128, 128)
    out = torch.empty_like(q)
    eager, counts_eager, _, _ = hp.run_gpu(q, k, v, 128, 0.6, impl=_impl(impl), want_mask=False)
    sb.sol_attn_forward_ex(q, k, v, out, ws, 128, 128, threshold=0.6, impl=_impl(impl))   # warm-up outside capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        sb.sol_attn_forward_ex(q, k, v, out, ws, 128, 128, threshold=0.6, impl=_impl(impl))
    out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), eager.view(torch.int16))
    assert torch.equal(ws.counts, counts_eager)
    # new values in the same buffers: the replay recomputes everything
    bits2 = _small_problem(62, 1, 2, 1100, 128)
    for dst, src in zip((q, k, v), bits2):
        dst.copy_(hp.to_dev(src))
    graph.replay()
    torch.cuda.synchronize()
    eager2, counts2, _, _ = hp.run_gpu(q, k, v, 128, 0.6, impl=_impl(impl), want_mask=False)
    assert torch.equal(out.view(torch.int16), eager2.view(torch.int16))
    assert torch.equal(ws.counts, counts2)


# ----------------------------------------------------------------------------- device-side failure path
def test_bounded_wait_runs_out_and_the_next_call_is_clean():
    """Every wait inside the tcgen05 kernel has a limit.  With the limit shortened to about a millisecond
    and one "value GEMM finished" signal per CTA withheld (a testing hook of the library: nothing faults,
    traps or spins unbounded), the waits on that signal run out, the CTA drains its copies and MMAs,
    releases TMEM and returns; the host reads SOL_ERR_DEVICE_TIMEOUT from the status word.  The same
    workspace then serves a normal call whose result matches the oracle."""
    bits = _small_problem(71, 1, 2, 1536, 128)
    q, k, v = (hp.to_dev(x) for x in bits)
    ws = sb.make_workspace(1, 2, 1536, 128, 128, 128)
    out = torch.empty_like(q)
    sb.sol_attn_debug_set_wait(2_000_000, 1)
    try:
        sb.sol_attn_forward_ex(q, k, v, out, ws, 128, 128, threshold=0.2, impl=sb.SOL_IMPL_TCGEN05)
        torch.cuda.synchronize()
        detail = int(ws.buf[:8].view(torch.int32)[1].item())
        sb.sol_attn_bind_workspace(ws)
        st = sb.sol_attn_read_device_status()
    finally:
        sb.sol_attn_debug_set_wait(0, -1)
    assert st == sb.SOL_ERR_DEVICE_TIMEOUT, sb.status_string(st)
    assert detail != 0                                       # where the first wait gave up
    assert sb.sol_attn_read_device_status() == sb.SOL_OK      # reading the status clears it
    out2, counts, mask, _ = hp.run_gpu(q, k, v, 128, 0.2, impl=sb.SOL_IMPL_TCGEN05, ws=ws)
    o = hp.dev_to_f64(out2)
    for h in range(2):
        hp.check_head(synth.widen(bits[0][0, h], np.float64), synth.widen(bits[1][0, h], np.float64),
                      synth.widen(bits[2][0, h], np.float64), o[0, h], mask[0, h], counts[0, h].cpu().numpy(), 128, 0.2)
