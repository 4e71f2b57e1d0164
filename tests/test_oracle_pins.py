"""Pins for the CPU oracle: facts fixed by the paper and by mathematics, none of which
is the oracle's own formula retyped.

P1  beta = -inf selects every block  -> brute-force dense attention, Eq. (1)
P2  beta = +inf selects none         -> textbook softmax attention over the pooled sequence
P3  independence of chunk size and visiting order (Sec. 3.2, "C affects efficiency only")
P4  exhaustive tiny cases, every mask, against a pure-Python augmented-list evaluation
P5  keys constant inside each block  -> zeroth-order term exact -> dense for every beta (Eq. 8)
P5' block_k = 1                      -> dense for every beta
P6  constant values                  -> output equals that constant
P7  Jensen / Eq. (appendix_approximation_error) bounds
P8  Eq. (5) moments = direct row statistics; Eq. (11) column mean = Eq. (3) proxy
P9  mask invariances (q -> c q, k -> k + t)
P10 Gaussian inputs: density = 1 - Phi(beta)
P11 counts bookkeeping
P12 hand-worked example (tests/golden/hand_example.json)
"""
import itertools
import json
import math
import os

import numpy as np
import pytest
from scipy.special import softmax as scipy_softmax

from oracle import sol_attn_oracle as orc
from paper_2607_24027_b200 import synth

HERE = os.path.dirname(os.path.abspath(__file__))


def _rand(seed, L, d, structured=True):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((L, d))
    k = rng.standard_normal((L, d))
    v = rng.standard_normal((L, d))
    if structured:  # smooth component so proxies carry signal
        t = np.linspace(0, 3, L)[:, None] * np.ones((1, d))
        q += np.sin(t + np.arange(d))
        k += np.sin(t + np.arange(d))
    # round to bf16 like the real inputs
    q, k, v = (synth.widen(synth.f32_to_bf16_bits(x.astype(np.float32)), np.float64) for x in (q, k, v))
    return q, k, v


# ------------------------------------------------------------------ pure-python references
def _py_dense(q, k, v, scale):
    """Eq. (1) with python loops and math.exp only."""
    L, d = len(q), len(q[0])
    out = []
    for u in range(L):
        logits = [scale * sum(q[u][c] * k[w][c] for c in range(d)) for w in range(L)]
        mx = max(logits)
        ws = [math.exp(x - mx) for x in logits]
        z = sum(ws)
        out.append([sum(ws[w] * v[w][c] for w in range(L)) / z for c in range(d)])
    return out


def _py_augmented(q, k, v, mask, bq, bk, scale):
    """Softmax attention over the augmented key list implied by Eqs. (9)-(10): selected
    blocks contribute their tokens, unselected blocks contribute ONE entry with the mean
    key, weight n_j and the mean value.  Python loops only."""
    L, d = len(q), len(q[0])
    nk = -(-L // bk)
    out = []
    for u in range(L):
        i = u // bq
        entries = []  # (logit, weight, value)
        for j in range(nk):
            toks = list(range(j * bk, min((j + 1) * bk, L)))
            if mask[i][j]:
                for w in toks:
                    entries.append((scale * sum(q[u][c] * k[w][c] for c in range(d)), 1.0, v[w]))
            else:
                n = len(toks)
                kbar = [sum(k[w][c] for w in toks) / n for c in range(d)]
                vbar = [sum(v[w][c] for w in toks) / n for c in range(d)]
                entries.append((scale * sum(q[u][c] * kbar[c] for c in range(d)), float(n), vbar))
        mx = max(e[0] for e in entries)
        z = sum(e[1] * math.exp(e[0] - mx) for e in entries)
        out.append([sum(e[1] * math.exp(e[0] - mx) * e[2][c] for e in entries) / z for c in range(d)])
    return out


# ------------------------------------------------------------------ P1
@pytest.mark.parametrize("L,d,b", [(64, 8, 16), (100, 16, 16), (37, 4, 8)])
def test_p1_select_all_is_dense(L, d, b):
    q, k, v = _rand(1, L, d)
    r = orc.sol_attn_forward(q, k, v, b, b, -math.inf, chunk=3)
    assert r.mask.all()
    scale = 1 / math.sqrt(d)
    ref = scipy_softmax(scale * (q @ k.T), axis=1) @ v          # library routine
    np.testing.assert_allclose(r.out, ref, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(orc.dense_attention(q, k, v), ref, rtol=1e-12, atol=1e-12)
    if L <= 40:
        py = np.array(_py_dense(q.tolist(), k.tolist(), v.tolist(), scale))
        np.testing.assert_allclose(r.out, py, rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------ P2
@pytest.mark.parametrize("L,b", [(64, 16), (100, 16)])
def test_p2_select_none_is_pooled_attention(L, b):
    d = 8
    q, k, v = _rand(2, L, d)
    r = orc.sol_attn_forward(q, k, v, b, b, math.inf, chunk=2)
    assert not r.mask.any()
    nk = -(-L // b)
    n = np.array([min(b, L - j * b) for j in range(nk)], dtype=float)
    kbar = np.stack([k[j * b:(j + 1) * b].mean(0) for j in range(nk)])
    vbar = np.stack([v[j * b:(j + 1) * b].mean(0) for j in range(nk)])
    # textbook attention of Q over the pooled sequence with log-multiplicity bias
    w = scipy_softmax((q @ kbar.T) / math.sqrt(d) + np.log(n)[None, :], axis=1)
    np.testing.assert_allclose(r.out, w @ vbar, rtol=1e-12, atol=1e-12)
    if L % b == 0:  # uniform multiplicity: plain dense attention on (Q, KC, VC / b)
        np.testing.assert_allclose(r.out, orc.dense_attention(q, r.kc, r.vc / b, scale=1 / math.sqrt(d)),
                                   rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------ P3
def test_p3_chunk_and_order_invariance():
    L, d, b = 203, 8, 16
    q, k, v = _rand(3, L, d)
    base = orc.sol_attn_forward(q, k, v, b, b, 0.4, chunk=4)
    assert 0 < base.mask.mean() < 1
    np.testing.assert_allclose(base.out, orc.sol_attn_definition(q, k, v, base.mask, b, b),
                               rtol=1e-11, atol=1e-12)
    rng = np.random.default_rng(0)
    for chunk in (1, 3, 5, 13, 64):
        n_chunks = -(-base.mask.shape[1] // chunk)
        order = rng.permutation(n_chunks)
        out, mask = orc.sol_attn_streaming(q, k, v, base.kc, base.vc, base.tau, b, b, chunk=chunk,
                                           chunk_order=order, inner_reverse=True)
        assert np.array_equal(mask, base.mask)
        np.testing.assert_allclose(out, base.out, rtol=1e-11, atol=1e-12)


# ------------------------------------------------------------------ P4
@pytest.mark.parametrize("L,d,b", [(8, 2, 2), (8, 3, 4), (6, 4, 1), (7, 2, 2), (5, 1, 4)])
def test_p4_exhaustive_tiny(L, d, b):
    rng = np.random.default_rng(L * 100 + d * 10 + b)
    q = rng.integers(-2, 3, size=(L, d)).astype(float)
    k = rng.integers(-2, 3, size=(L, d)).astype(float)
    v = rng.integers(-3, 4, size=(L, d)).astype(float)
    nb = -(-L // b)
    _, kc, vc, _ = orc.pool(q, k, v, b, b)
    scale = 0.5
    rows = list(itertools.product([False, True], repeat=nb))
    for a in range(len(rows)):
        # every query block gets a (different) pattern; each block sees every one of the 2^nb patterns
        mask = np.array([rows[(a + 3 * i) % len(rows)] for i in range(nb)])
        out, m2 = orc.sol_attn_streaming(q, k, v, kc, vc, None, b, b, chunk=2, scale=scale,
                                         mask_override=mask)
        assert np.array_equal(m2, mask)
        ref = np.array(_py_augmented(q.tolist(), k.tolist(), v.tolist(), mask.tolist(), b, b, scale))
        np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(orc.sol_attn_definition(q, k, v, mask, b, b, scale=scale), ref,
                                   rtol=1e-12, atol=1e-12)


def test_p4_block_q_differs_from_block_k():
    L, d = 12, 2
    q, k, v = _rand(44, L, d)
    mask = np.array([[True, False, True, False, False, True]] * 3)
    mask[1] = ~mask[1]
    _, kc, vc, _ = orc.pool(q, k, v, 4, 2)
    out, _ = orc.sol_attn_streaming(q, k, v, kc, vc, None, 4, 2, chunk=4, scale=1.0, mask_override=mask)
    ref = np.array(_py_augmented(q.tolist(), k.tolist(), v.tolist(), mask.tolist(), 4, 2, 1.0))
    np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------ P5 / P5' / P6
@pytest.mark.parametrize("beta", [-0.5, 0.3, 1.0, math.inf])
def test_p5_blockwise_constant_keys_give_dense(beta):
    L, d, b = 96, 8, 16
    q, k, v = _rand(5, L, d)
    k = np.repeat(k[::b], b, axis=0)            # every key equals its block's first key
    r = orc.sol_attn_forward(q, k, v, b, b, beta, chunk=2)
    ref = scipy_softmax((q @ k.T) / math.sqrt(d), axis=1) @ v
    np.testing.assert_allclose(r.out, ref, rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("beta", [0.0, 0.8])
def test_p5prime_block_one_is_dense(beta):
    L, d = 40, 4
    q, k, v = _rand(6, L, d)
    r = orc.sol_attn_forward(q, k, v, 8, 1, beta, chunk=7)
    assert 0 < r.mask.mean() < 1
    ref = scipy_softmax((q @ k.T) / math.sqrt(d), axis=1) @ v
    np.testing.assert_allclose(r.out, ref, rtol=1e-11, atol=1e-12)


def test_p6_constant_values():
    L, d, b = 72, 4, 16
    q, k, _ = _rand(7, L, d)
    c = np.array([0.5, -1.25, 3.0, 0.0])
    v = np.tile(c, (L, 1))
    r = orc.sol_attn_forward(q, k, v, b, b, 0.2, chunk=2)
    np.testing.assert_allclose(r.out, v, rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------ P7
def test_p7_error_bounds():
    L, d, b = 64, 8, 16
    q, k, v = _rand(8, L, d)
    s = 1 / math.sqrt(d)
    for u in (0, 17, 63):
        for j in range(L // b):
            kj, vj = k[j * b:(j + 1) * b], v[j * b:(j + 1) * b]
            kbar = kj.mean(0)
            a = s * q[u] @ kbar
            delta = s * (kj - kbar) @ q[u]
            eta = np.abs(delta).max()
            d_exact = np.exp(s * kj @ q[u]).sum()
            d_apx = b * math.exp(a)
            assert -1e-12 <= d_exact - d_apx <= 0.5 * math.exp(a + eta) * (delta ** 2).sum() + 1e-12
            n_exact = np.exp(s * kj @ q[u]) @ vj
            n_apx = math.exp(a) * vj.sum(0)
            bound = math.exp(a + eta) * (np.abs(delta) * np.linalg.norm(vj, axis=1)).sum()
            assert np.linalg.norm(n_exact - n_apx) <= bound + 1e-12
    # consequence: with the same running max the Sol-Attn denominator never exceeds the dense one
    r = orc.sol_attn_forward(q, k, v, b, b, 0.5)
    logits = s * q @ k.T
    dense_den = np.exp(logits).sum(1)
    _, kc, _, n_k = orc.pool(q, k, v, b, b)
    for i in range(L // b):
        rows = slice(i * b, (i + 1) * b)
        den = np.zeros(b)
        for j in range(L // b):
            if r.mask[i, j]:
                den += np.exp(logits[rows, j * b:(j + 1) * b]).sum(1)
            else:
                den += n_k[j] * np.exp(s * q[rows] @ kc[j])
        assert (den <= dense_den[rows] * (1 + 1e-12)).all()


# ------------------------------------------------------------------ P8
def test_p8_moment_form_and_tile_mean():
    L, d, b = 203, 16, 16
    q, k, v = _rand(9, L, d)
    qbar, kc, _, _ = orc.pool(q, k, v, b, b)
    s = 1 / math.sqrt(d)
    s_hat = orc.proxy_scores(qbar, kc, s)
    mu, sigma, tau = orc.threshold_direct(s_hat, 0.7)
    # numpy's own statistics as the independent side
    np.testing.assert_allclose(mu, np.mean(s_hat, axis=1), rtol=1e-13)
    np.testing.assert_allclose(sigma, np.std(s_hat, axis=1), rtol=1e-12)
    mu2, sigma2, tau2 = orc.threshold_moments(qbar, kc, 0.7, s)
    np.testing.assert_allclose(mu2, mu, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(sigma2, sigma, rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(tau2, tau, rtol=1e-9, atol=1e-12)
    for i in (0, 5, qbar.shape[0] - 1):        # includes the ragged last query block
        tile_mean = orc.proxy_scores_from_tile(q[i * b:(i + 1) * b], kc, s)
        np.testing.assert_allclose(tile_mean, s_hat[i], rtol=1e-12, atol=1e-13)
    # diagonal estimator equals the full one when pooled keys are decorrelated across channels
    rng = np.random.default_rng(0)
    kc_diag = np.zeros((d * 2, d))
    amp = rng.uniform(0.5, 2.0, size=d)
    for c in range(d):                           # rows +a_c e_c and -a_c e_c: zero mean,
        kc_diag[2 * c, c] = amp[c]               # exactly diagonal covariance
        kc_diag[2 * c + 1, c] = -amp[c]
    _, sig_full, _ = orc.threshold_moments(qbar, kc_diag, 0.0, s)
    _, sig_diag, _ = orc.threshold_diagonal(qbar, kc_diag, 0.0, s)
    np.testing.assert_allclose(sig_diag, sig_full, rtol=1e-10, atol=1e-13)


# ------------------------------------------------------------------ P9
def test_p9_invariances():
    L, d, b = 160, 8, 16
    q, k, v = _rand(10, L, d)
    base = orc.sol_attn_forward(q, k, v, b, b, 0.6)
    scaled = orc.routing(4.0 * q, k, v, b, b, 0.6)
    assert np.array_equal(scaled.mask, base.mask)
    t = np.linspace(-1, 1, d)
    shifted = orc.sol_attn_forward(q, k + t, v, b, b, 0.6)
    assert np.array_equal(shifted.mask, base.mask)
    np.testing.assert_allclose(shifted.out, base.out, rtol=1e-9, atol=1e-11)
    # a different scale leaves the mask alone (standardised cutoff)
    assert np.array_equal(orc.routing(q, k, v, b, b, 0.6, scale=0.03).mask, base.mask)


# ------------------------------------------------------------------ P10
@pytest.mark.parametrize("beta,rho", [(0.5, 0.3085375387), (1.0, 0.1586552539), (1.645, 0.04998490553)])
def test_p10_gaussian_density(beta, rho):
    assert abs(orc.gaussian_density(beta) - rho) < 1e-9
    qb, kb, vb = synth.gaussian_qkv(123, 2, 4096, 32)
    dens = []
    for h in range(2):
        r = orc.routing(synth.widen(qb[h], np.float64), synth.widen(kb[h], np.float64),
                        synth.widen(vb[h], np.float64), 16, 16, beta)
        dens.append(r.mask.mean())
    n_pairs = 2 * 256 * 256
    sd = math.sqrt(rho * (1 - rho) / n_pairs)
    # rows share mu/sigma estimates, so allow a generous multiple of the binomial deviation
    assert abs(np.mean(dens) - rho) < 8 * sd + 2e-3


# ------------------------------------------------------------------ P11
def test_p11_counts_and_edges():
    L, d, b = 130, 8, 16
    q, k, v = _rand(11, L, d)
    r = orc.sol_attn_forward(q, k, v, b, b, 0.3)
    assert r.counts.sum() == np.count_nonzero(r.mask)
    assert ((0 <= r.counts) & (r.counts <= r.mask.shape[1])).all()
    assert r.out.shape == (L, d) and np.isfinite(r.out).all()
    # sigma = 0 (all proxies of a row equal) selects nothing for finite beta
    kconst = np.tile(k[0], (L, 1))
    r0 = orc.routing(q, kconst, v, b, b, 0.0)
    in_band = np.abs(r0.s_hat - r0.tau[:, None]) < 1e-9
    assert in_band.all()
    # q_tiles restricts evaluation
    sub = orc.sol_attn_forward(q, k, v, b, b, 0.3, q_tiles=[2, 8])
    np.testing.assert_array_equal(sub.out[2 * b:3 * b], r.out[2 * b:3 * b])
    np.testing.assert_array_equal(sub.out[8 * b:], r.out[8 * b:])
    assert np.isnan(sub.out[0]).all()
    # keep-or-drop variant equals masked dense attention, Eq. (2)
    eo = orc.sol_attn_forward(q, k, v, b, b, 0.3, exact_only=True)
    tok_mask = np.repeat(np.repeat(r.mask, b, axis=0), b, axis=1)[:L, :L]
    logits = np.where(tok_mask, (q @ k.T) / math.sqrt(d), -np.inf)
    rows = tok_mask.any(1)
    ref = scipy_softmax(logits[rows], axis=1) @ v
    np.testing.assert_allclose(eo.out[rows], ref, rtol=1e-11, atol=1e-12)


# ------------------------------------------------------------------ P12
def test_p12_hand_worked_example():
    g = json.load(open(os.path.join(HERE, "golden", "hand_example.json")))
    e = math.exp(1.0)
    col = lambda x: np.array(x, dtype=float)[:, None]
    q, k, v = col(g["q"]), col(g["k"]), col(g["v"])
    b = g["block"]
    r = orc.sol_attn_forward(q, k, v, b, b, g["beta"], scale=g["scale"], chunk=1)
    np.testing.assert_allclose(r.qbar[:, 0], g["qbar"], atol=1e-15)
    np.testing.assert_allclose(r.kc[:, 0], g["kc"], atol=1e-15)
    np.testing.assert_allclose(r.vc[:, 0], g["vc"], atol=1e-15)
    np.testing.assert_allclose(r.s_hat, g["s_hat"], atol=1e-15)
    np.testing.assert_allclose(r.mu, g["mu"], atol=1e-15)
    np.testing.assert_allclose(r.sigma, g["sigma"], atol=1e-15)
    np.testing.assert_allclose(r.tau, g["tau"], atol=1e-15)
    assert r.mask.tolist() == g["mask"]
    expect = [eval(x, {"e": e}) for x in g["out_natural"]]
    np.testing.assert_allclose(r.out[:, 0], expect, rtol=1e-13)
    r2 = orc.sol_attn_forward(q, k, v, b, b, g["beta"], scale=g["scale"], chunk=2,
                              mask_override=np.array(g["mask_override"]))
    expect2 = [eval(x, {"e": e}) for x in g["out_override"]]
    np.testing.assert_allclose(r2.out[:, 0], expect2, rtol=1e-13)
    # float32 mode stays within float32 rounding of the same numbers
    r32 = orc.sol_attn_forward(q, k, v, b, b, g["beta"], scale=g["scale"], dtype=np.float32)
    np.testing.assert_allclose(r32.out[:, 0], expect, rtol=2e-6)


# ------------------------------------------------------------------ forced-exact blocks, diagonal estimator
def test_forced_blocks_and_diagonal_routing():
    L, d, b = 130, 8, 16
    q, k, v = _rand(13, L, d)
    nk = -(-L // b)
    base = orc.sol_attn_forward(q, k, v, b, b, 0.7)
    forced = np.zeros(nk, dtype=bool)
    forced[[1, nk - 1]] = True
    r = orc.sol_attn_forward(q, k, v, b, b, 0.7, forced=forced)
    assert np.array_equal(r.mask, base.mask | forced[None, :])
    np.testing.assert_allclose(r.out, orc.sol_attn_definition(q, k, v, r.mask, b, b), rtol=1e-11, atol=1e-12)
    # forcing everything is dense attention whatever beta is
    rall = orc.sol_attn_forward(q, k, v, b, b, math.inf, forced=np.ones(nk, dtype=bool))
    ref = scipy_softmax((q @ k.T) / math.sqrt(d), axis=1) @ v
    np.testing.assert_allclose(rall.out, ref, rtol=1e-11, atol=1e-12)
    # the diagonal estimator changes sigma (hence tau) but not mu
    rd = orc.routing(q, k, v, b, b, 0.7, estimator="diagonal")
    np.testing.assert_allclose(rd.mu, base.mu, rtol=1e-12, atol=1e-14)
    v_k = np.var(base.kc, axis=0)                                   # numpy's own per-channel variance
    np.testing.assert_allclose(rd.sigma, np.sqrt((base.qbar ** 2) @ v_k) / math.sqrt(d), rtol=1e-10)


# ----------------------------------------------------------------------------- materialised baselines
def test_route_topk_is_the_k_largest():
    """Top-k routing (introduction, limitation L1): brute force over all subsets of a small row."""
    import itertools
    rng = np.random.default_rng(5)
    s = rng.standard_normal((6, 7))
    for k in range(0, 8):
        mask, order, tau = orc.route_topk(s, k)
        assert (mask.sum(axis=1) == min(k, 7)).all()
        for i in range(6):
            best = max(itertools.combinations(range(7), min(k, 7)), key=lambda c: s[i, list(c)].sum())
            assert set(np.flatnonzero(mask[i])) == set(best)
            assert np.array_equal(s[i] > tau[i], mask[i])            # the equivalent threshold
            assert (np.diff(s[i, order[i]]) <= 0).all()


def test_route_topp_geometric_row_closed_form():
    """Scores -j ln 2 give probabilities proportional to 2^-j: the mass of the c largest is
    (1 - 2^-c) / (1 - 2^-N), so p = 0.9 keeps 4 blocks and p = 0.5 keeps 1 (N = 10)."""
    n = 10
    s = (-np.arange(n) * np.log(2.0))[None, :]
    perm = np.random.default_rng(1).permutation(n)
    sp = s[:, perm]
    for p, want in [(0.9, 4), (0.5, 1), (0.5005, 2), (0.75, 2), (0.76, 3), (1.0, n)]:
        mask, order, tau, counts = orc.route_topp(sp, p)
        assert counts[0] == want, (p, counts)
        assert set(perm[np.flatnonzero(mask[0])]) == set(range(want))
        if want < n:
            assert np.array_equal(sp[0] > tau[0], mask[0])


def test_route_topp_uniform_row_and_budget_imbalance():
    """Equal scores: each block carries 1/N of the mass, so ceil(p N) blocks are kept (lowest indices
    first); a row dominated by one sink keeps a single block -- the budget imbalance the paper
    attributes to top-p."""
    n = 16
    mask, order, tau, counts = orc.route_topp(np.zeros((1, n)), 0.3)
    assert counts[0] == math.ceil(0.3 * n) and mask[0, :counts[0]].all()
    s = np.zeros((1, n))
    s[0, 11] = 12.0
    mask, order, tau, counts = orc.route_topp(s, 0.9)
    assert counts[0] == 1 and mask[0, 11]
