"""The allocation-free threshold entry point against the regular one.

`sol_attn_thresholds_static` serves callers that may not allocate device memory (an operator
living inside another framework's memory pool, a process with all device memory reserved up
front): its intermediate pooled-key moments live in an array built into the library instead of a
caller-provided workspace.  It must reproduce the mu / sigma / tau that `sol_attn_pool` writes
into the workspace -- on two calls in a row, because every call reuses the same array and sees
whatever the previous call left there.

This file is named so that pytest collects it last.
"""
import numpy as np
import pytest
import torch

from oracle import sol_attn_oracle as orc
from paper_2607_24027_b200 import synth
from paper_2607_24027_b200.configs import WORKLOADS, load_betas
from tests import helpers as hp

pytestmark = pytest.mark.gpu


def _reference(sb, wl, beta):
    qb, kb, vb = synth.generate(wl)
    q, k, v = hp.to_dev(qb), hp.to_dev(kb), hp.to_dev(vb)
    ws = sb.make_workspace(wl.batch, wl.heads, wl.seq_len, wl.d, wl.block, wl.block)
    sb.sol_attn_bind_workspace(ws)
    sb.sol_attn_pool(q, k, v, wl.block, wl.block, beta)       # the existing entry point
    torch.cuda.synchronize()
    return ws


def _static(sb, ws, beta):
    qbar, kc = ws.qbar.contiguous(), ws.kc.contiguous()
    mu, sigma, tau = (torch.full_like(ws.tau, float("nan")) for _ in range(3))
    sb.sol_attn_thresholds_static(qbar, kc, beta, mu, sigma, tau)   # through the C ABI
    torch.cuda.synchronize()
    return mu, sigma, tau


def _close(a, b):
    # same tolerance the pre-attention parity tests use for tau
    np.testing.assert_allclose(a.cpu().numpy(), b.cpu().numpy(), rtol=1e-4, atol=5e-5)


def test_static_thresholds_match_workspace_thresholds_twice():
    from paper_2607_24027_b200 import binding as sb
    sb.lib()
    # first call: the image workload (24 heads, d = 128); second call: the tiny one (d = 64), so
    # the second call finds the first call's moments in the shared array
    for name in ("image", "tiny"):
        wl = WORKLOADS[name]
        beta = list(load_betas()[name].values())[0]
        ws = _reference(sb, wl, beta)
        mu, sigma, tau = _static(sb, ws, beta)
        _close(mu, ws.mu)
        _close(sigma, ws.sigma)
        _close(tau, ws.tau)
    # and once more on the first shape with another beta, +inf included
    wl = WORKLOADS["image"]
    for beta in (-0.3, float("inf")):
        ws = _reference(sb, wl, beta)
        mu, sigma, tau = _static(sb, ws, beta)
        _close(mu, ws.mu)
        if np.isinf(beta):
            assert torch.isinf(tau).all() and torch.isinf(ws.tau).all()
        else:
            _close(tau, ws.tau)


def test_static_thresholds_match_the_oracle_and_leave_device_memory_alone():
    """The same numbers straight against the CPU oracle (row statistics of the proxy map, Eq. 4), and
    the point of the entry point itself: a call that is not the first one on the device changes nothing
    in the device's memory accounting (the first call loads the module that holds the array)."""
    from paper_2607_24027_b200 import binding as sb
    sb.lib()
    wl = WORKLOADS["image"]
    beta = load_betas()["image"][0.3]
    ws = _reference(sb, wl, beta)
    qb, kb, vb = synth.generate(wl)
    _static(sb, ws, beta)                                   # set-up call on this device, if none came before
    qbar, kc = ws.qbar.contiguous(), ws.kc.contiguous()
    mu, sigma, tau = (torch.full_like(ws.tau, float("nan")) for _ in range(3))
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    launches_before = sb.sol_attn_launch_count()
    for _ in range(3):
        sb.sol_attn_thresholds_static(qbar, kc, beta, mu, sigma, tau)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, (free_before, free_after)
    assert sb.sol_attn_launch_count() - launches_before == 9   # three kernels per call, all counted
    for h in (0, wl.heads - 1):
        r = orc.routing(synth.widen(qb[0, h], np.float64), synth.widen(kb[0, h], np.float64),
                        synth.widen(vb[0, h], np.float64), wl.block, wl.block, beta)
        np.testing.assert_allclose(mu[0, h].cpu().numpy(), r.mu, rtol=0, atol=2e-5)
        np.testing.assert_allclose(sigma[0, h].cpu().numpy(), r.sigma, rtol=1e-4, atol=2e-5)
        np.testing.assert_allclose(tau[0, h].cpu().numpy(), r.tau, rtol=0, atol=5e-5)
    # argument checks happen before anything is launched
    with pytest.raises(sb.SolAttnError) as e:
        sb.sol_attn_thresholds_static(qbar, kc, beta, mu, sigma, tau, scale=float("inf"))
    assert e.value.status == sb.SOL_ERR_INVALID_ARG


def test_static_thresholds_reject_oversized_problems():
    from paper_2607_24027_b200 import binding as sb
    sb.lib()
    limit = sb.sol_attn_thresholds_static_max_floats()
    heads = limit // (128 * 129) + 1                      # one head too many for d = 128
    qbar = torch.zeros(1, heads, 2, 128, device="cuda")
    kc = torch.zeros(1, heads, 2, 128, device="cuda")
    out = [torch.zeros(1, heads, 2, device="cuda") for _ in range(3)]
    with pytest.raises(sb.SolAttnError) as e:
        sb.sol_attn_thresholds_static(qbar, kc, 0.5, *out)
    assert e.value.status == sb.SOL_ERR_SCRATCH_LIMIT
    assert sb.status_string(e.value.status) == "SOL_ERR_SCRATCH_LIMIT"
