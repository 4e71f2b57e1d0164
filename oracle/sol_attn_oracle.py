"""CPU oracle for the Sol-Attn forward pass.  TEST INFRASTRUCTURE ONLY.

A plain, slow, obviously-correct numpy implementation of what the fused GPU kernel
computes, written from the paper's equations.  It shares no code with the CUDA path
and must never be imported by the product path; only the tests, the smoke check and
the benchmark's ``cpu_baseline`` / reference arm may call it.

All arithmetic is float64 by default (``dtype=np.float32`` is accepted everywhere for
same-precision experiments).  Inputs are float arrays holding exactly the bf16 values
the GPU sees.  Everything is single-(batch, head): ``q, k, v`` have shape ``[L, d]``.

What follows which passage of the paper
---------------------------------------
* ``dense_attention``            Eq. (1): ``O = Softmax(Q K^T) V`` (brute force, L x L).
* ``pool``                       Eq. (3) text: token-mean pooled ``Qbar_i``, ``Kbar_j``; the
                                 summed values ``Vhat_j`` defined just before Eq. (9).
* ``proxy_scores``               Eq. (3): ``s_ij = Qbar_i Kbar_j^T``.
* ``threshold_direct``           Eq. (4) with the row mean / population variance of
                                 Eq. (appendix_proxy_variance).
* ``threshold_moments``          Eq. (5): the same statistics from the first and second
                                 moments of the pooled keys.
* ``threshold_diagonal``         Eq. (appendix_diagonal_threshold).
* ``select_blocks``              Eq. (4): ``S_i = { j : s_ij > tau_i }`` (strict).
* ``sol_attn_definition``        Eqs. (9), (10): numerator / denominator written out row by
                                 row, no streaming.
* ``sol_attn_streaming``         Algorithm 1: chunked outer loop over pooled keys, nested
                                 exact inner loop, ONE running (m, l, acc).
* ``sol_attn_forward``           the whole path for one head: pool -> proxy -> threshold ->
                                 select -> Algorithm 1.

Readings of the paper taken here (the paper omits or leaves these open)
-----------------------------------------------------------------------
* Every logit (exact, token-to-block and block proxy) is multiplied by ``scale``
  (default ``1/sqrt(d)``); the paper "omits the scale factor".
* ``threshold`` is the standardized cutoff beta of Eq. (4); ``+inf`` selects nothing and
  ``-inf`` selects everything (no ``inf * 0`` is ever formed).
* Standard deviation is the population one (1/N), clamped at zero.
* A sequence length that is not a multiple of the block size leaves a ragged last
  block: it is pooled over its valid tokens only, its multiplicity in Eq. (9) is its
  valid token count ``n_j`` (the paper's ``B``), and row statistics weight every block
  equally.
* Algorithm 1 does not show the factor ``B`` of Eq. (9); Eq. (9) governs: an unselected
  block adds ``n_j * exp(a)`` to the denominator and ``exp(a) * Vhat_j`` (the SUM of its
  values) to the numerator.
* The proxy score is ``Qbar_i . Kbar_j`` from the pooled vectors (Eq. 3); Eq. (11)'s
  column mean of the token-to-block tile is the same number in exact arithmetic and is
  provided as ``proxy_scores_from_tile`` for cross-checking.

Parity pins: see tests/test_oracle_pins.py.  Unpinned: none of the functions above; the
paper's figure values that need real-model q/k/v (error-vs-sparsity curves, quality
tables) are "parity unpinned" and are not reproduced.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np


# --------------------------------------------------------------------------- helpers
def _nblocks(L: int, b: int) -> int:
    return -(-L // b)


def block_sizes(L: int, b: int) -> np.ndarray:
    """Valid token count of every block (``n_j``; the last one may be ragged)."""
    n = _nblocks(L, b)
    sizes = np.full(n, b, dtype=np.int64)
    sizes[-1] = L - (n - 1) * b
    return sizes


def default_scale(d: int) -> float:
    return 1.0 / math.sqrt(d)


# --------------------------------------------------------------------------- Eq. (1)
def dense_attention(q, k, v, scale: Optional[float] = None, dtype=np.float64):
    """Eq. (1): softmax(scale * Q K^T) V with the full L x L matrix formed."""
    q = np.asarray(q, dtype=dtype)
    k = np.asarray(k, dtype=dtype)
    v = np.asarray(v, dtype=dtype)
    s = default_scale(q.shape[1]) if scale is None else scale
    logits = (q @ k.T) * dtype(s)
    logits = logits - logits.max(axis=1, keepdims=True)
    w = np.exp(logits)
    return (w @ v) / w.sum(axis=1, keepdims=True)


# --------------------------------------------------------------------------- pooling, Eq. (3)
def pool(q, k, v, block_q: int, block_k: int, dtype=np.float64):
    """Token-mean pooled queries / keys and token-SUM pooled values.

    Returns ``(Qbar [N_q, d], KC [N_k, d], VC [N_k, d], n_k [N_k])`` where ``KC[j]`` is the
    mean of key block j over its valid tokens, ``VC[j]`` the sum of value block j, and
    ``n_k[j]`` the number of valid tokens in block j.
    """
    q = np.asarray(q, dtype=dtype)
    k = np.asarray(k, dtype=dtype)
    v = np.asarray(v, dtype=dtype)
    L, d = q.shape
    nq, nk = _nblocks(L, block_q), _nblocks(L, block_k)
    qbar = np.empty((nq, d), dtype=dtype)
    kc = np.empty((nk, d), dtype=dtype)
    vc = np.empty((nk, d), dtype=dtype)
    for i in range(nq):
        qbar[i] = q[i * block_q:(i + 1) * block_q].mean(axis=0)
    for j in range(nk):
        kc[j] = k[j * block_k:(j + 1) * block_k].mean(axis=0)
        vc[j] = v[j * block_k:(j + 1) * block_k].sum(axis=0)
    return qbar, kc, vc, block_sizes(L, block_k)


def proxy_scores(qbar, kc, scale: float):
    """Eq. (3): ``s_ij = scale * Qbar_i . Kbar_j`` for all (i, j)."""
    return (qbar @ kc.T) * qbar.dtype.type(scale)


def proxy_scores_from_tile(q_i, kc, scale: float):
    """Eq. (11): column mean over the query tokens of the token-to-block tile ``Q_i KC^T``."""
    tile = (q_i @ kc.T) * q_i.dtype.type(scale)
    return tile.mean(axis=0)


# --------------------------------------------------------------------------- thresholds
def _tau_from_stats(mu, sigma, beta: float):
    if math.isinf(beta):
        return np.full_like(mu, np.inf if beta > 0 else -np.inf)
    return mu + mu.dtype.type(beta) * sigma


def threshold_direct(s_hat, beta: float):
    """Eq. (4): ``tau_i = mu_i + beta sigma_i`` from the row statistics of the proxy row."""
    mu = s_hat.mean(axis=1)
    var = ((s_hat - mu[:, None]) ** 2).mean(axis=1)
    sigma = np.sqrt(np.maximum(var, 0))
    return mu, sigma, _tau_from_stats(mu, sigma, beta)


def threshold_moments(qbar, kc, beta: float, scale: float):
    """Eq. (5): the same ``mu_i``, ``sigma_i`` from pooled-key moments (no proxy row)."""
    t = qbar.dtype.type
    m_k = kc.mean(axis=0)
    M_k = (kc.T @ kc) / t(kc.shape[0])
    mu = (qbar @ m_k) * t(scale)
    second = np.einsum("id,de,ie->i", qbar, M_k, qbar) * t(scale) ** 2
    sigma = np.sqrt(np.maximum(second - mu * mu, 0))
    return mu, sigma, _tau_from_stats(mu, sigma, beta)


def threshold_diagonal(qbar, kc, beta: float, scale: float):
    """Eq. (appendix_diagonal_threshold): keep only the diagonal of the pooled-key covariance."""
    t = qbar.dtype.type
    mu_k = kc.mean(axis=0)
    v_k = (kc * kc).mean(axis=0) - mu_k * mu_k
    mu = (qbar @ mu_k) * t(scale)
    var = ((qbar * qbar) @ v_k) * t(scale) ** 2
    sigma = np.sqrt(np.maximum(var, 0))
    return mu, sigma, _tau_from_stats(mu, sigma, beta)


def route_topk(s_hat, k: int):
    """Materialised top-k routing, the first baseline of the introduction: every query block keeps
    the ``k`` key blocks with the highest proxy scores (ties go to the lower block index).

    Returns (mask [N_q, N_k] bool, order [N_q, N_k] block indices by descending score, tau [N_q]).
    ``tau`` is the threshold under which strict ``s_hat > tau`` reproduces the mask when the k-th and
    (k+1)-th scores differ: their midpoint (-inf when every block is kept, +inf when none is)."""
    s_hat = np.asarray(s_hat)
    nq, nk = s_hat.shape
    order = np.argsort(-s_hat, axis=1, kind="stable")
    k = int(min(max(k, 0), nk))
    mask = np.zeros((nq, nk), dtype=bool)
    tau = np.empty(nq, dtype=s_hat.dtype)
    for i in range(nq):
        mask[i, order[i, :k]] = True
        tau[i] = _cut_between(s_hat[i, order[i]], k)
    return mask, order, tau


def route_topp(s_hat, p: float):
    """Materialised top-p routing, the second baseline of the introduction: per query block the key
    blocks are taken in order of descending proxy score until their cumulative probability mass,
    under the softmax of that row of proxy scores, reaches ``p``.

    Returns (mask, order, tau, counts) as route_topk does; counts[i] is the number kept."""
    s_hat = np.asarray(s_hat)
    nq, nk = s_hat.shape
    order = np.argsort(-s_hat, axis=1, kind="stable")
    mask = np.zeros((nq, nk), dtype=bool)
    tau = np.empty(nq, dtype=s_hat.dtype)
    counts = np.zeros(nq, dtype=np.int64)
    for i in range(nq):
        row = s_hat[i, order[i]]
        w = np.exp(row - row[0])
        total = w.sum()
        mass = 0.0
        c = 0
        while c < nk and mass < p * total:
            mass += w[c]
            c += 1
        counts[i] = c
        mask[i, order[i, :c]] = True
        tau[i] = _cut_between(row, c)
    return mask, order, tau, counts


def _cut_between(sorted_desc, c: int):
    """A cutoff that strict ``>`` turns into 'the first c of this descending row'."""
    n = len(sorted_desc)
    if c <= 0:
        return np.inf
    if c >= n:
        return -np.inf
    return 0.5 * (sorted_desc[c - 1] + sorted_desc[c])


def select_blocks(s_hat, tau):
    """Eq. (4): boolean mask ``[N_q, N_k]``, True where ``s_ij > tau_i`` (strict)."""
    return s_hat > tau[:, None]


# --------------------------------------------------------------------------- Eqs. (9), (10)
def sol_attn_definition(q, k, v, mask, block_q: int, block_k: int,
                        scale: Optional[float] = None, dtype=np.float64,
                        q_tiles: Optional[Sequence[int]] = None):
    """Eqs. (9)-(10) evaluated row by row under a given block mask.

    For query block i with selected set S_i (``mask[i]`` True) and unselected set U_i:
      D = sum_{j in U_i} n_j exp(q Kbar_j^T) + sum_{j in S_i} sum_{v in j} exp(q k_v^T)
      N = sum_{j in U_i} exp(q Kbar_j^T) Vhat_j + sum_{j in S_i} sum_{v in j} exp(q k_v^T) v_v
      O = N / D.
    ``q_tiles`` restricts the evaluation to some query blocks; rows of other blocks are NaN.
    """
    q = np.asarray(q, dtype=dtype)
    k = np.asarray(k, dtype=dtype)
    v = np.asarray(v, dtype=dtype)
    L, d = q.shape
    s = dtype(default_scale(d) if scale is None else scale)
    _, kc, vc, n_k = pool(q, k, v, block_q, block_k, dtype=dtype)
    nq = _nblocks(L, block_q)
    out = np.full((L, d), np.nan, dtype=dtype)
    tiles = range(nq) if q_tiles is None else q_tiles
    for i in tiles:
        qi = q[i * block_q:(i + 1) * block_q]
        sel = np.flatnonzero(mask[i])
        uns = np.flatnonzero(~np.asarray(mask[i], dtype=bool))
        a = (qi @ kc[uns].T) * s                                  # token-to-block logits
        tok = np.concatenate([np.arange(j * block_k, min((j + 1) * block_k, L)) for j in sel]) \
            if len(sel) else np.zeros(0, dtype=np.int64)
        e = (qi @ k[tok].T) * s                                   # exact logits
        m = np.full(qi.shape[0], -np.inf, dtype=dtype)
        if a.shape[1]:
            m = np.maximum(m, a.max(axis=1))
        if e.shape[1]:
            m = np.maximum(m, e.max(axis=1))
        wa = np.exp(a - m[:, None])
        we = np.exp(e - m[:, None])
        den = wa @ n_k[uns].astype(dtype) + we.sum(axis=1)        # Eq. (9)
        num = wa @ vc[uns] + we @ v[tok]                          # Eq. (10)
        out[i * block_q:(i + 1) * block_q] = num / den[:, None]
    return out


# --------------------------------------------------------------------------- Algorithm 1
def _online_update(logits, weights, values, acc, l, m):
    """One online-softmax step shared by the approximate and the exact branch.

    ``logits`` [rows, cols] (``-inf`` = masked out), ``weights`` [cols] multiplicity of
    each column in the denominator, ``values`` [cols, d] what each column adds to the
    numerator per unit of exp().  Updates and returns (acc, l, m).
    """
    tile_max = logits.max(axis=1) if logits.shape[1] else np.full_like(m, -np.inf)
    m_new = np.maximum(m, tile_max)
    live = np.isfinite(m_new)                    # rows that have seen a finite logit
    if not live.any():
        return acc, l, m
    alpha = np.zeros_like(m)
    alpha[live] = np.exp(np.where(np.isfinite(m[live]), m[live] - m_new[live], -np.inf))
    p = np.zeros_like(logits)
    p[live] = np.exp(logits[live] - m_new[live, None])
    l = l * alpha + p @ weights
    acc = acc * alpha[:, None] + p @ values
    return acc, l, m_new


def sol_attn_streaming(q, k, v, kc, vc, tau, block_q: int, block_k: int, chunk: int = 16,
                       scale: Optional[float] = None, dtype=np.float64,
                       mask_override=None, chunk_order: Optional[Sequence[int]] = None,
                       inner_reverse: bool = False, q_tiles: Optional[Sequence[int]] = None,
                       exact_only: bool = False):
    """Algorithm 1 (Sol-Attn forward pass) for one head.

    For each query block the pooled keys ``KC`` are scanned in chunks of ``chunk`` blocks.
    Per chunk: the token-to-block tile ``Q_i KC_chunk^T`` is formed; a block is routed to the
    exact branch when its proxy score exceeds ``tau[i]``; the routed columns are masked out
    and the remaining columns update the running softmax with multiplicity ``n_j`` and the
    summed values ``VC``; then every routed block is processed exactly.  Both branches
    update the same (m, l, acc).

    The routing score is ``scale * Qbar_i . KC_j`` (Eq. 3) from pooled vectors in ``dtype``.
    ``mask_override`` ([N_q, N_k] bool) replaces the routing decision (used for exhaustive
    tests and for evaluating the output under another implementation's mask).
    ``chunk_order`` visits the chunks in another order and ``inner_reverse`` reverses the
    inner loop: the result must not depend on either, up to rounding.
    ``exact_only`` drops the approximate branch (keep-or-drop block-sparse attention, Eq. 2).

    Returns ``(O [L, d], mask [N_q, N_k] bool)``; rows of query blocks outside ``q_tiles``
    are NaN and their mask rows False.
    """
    q = np.asarray(q, dtype=dtype)
    k = np.asarray(k, dtype=dtype)
    v = np.asarray(v, dtype=dtype)
    kc = np.asarray(kc, dtype=dtype)
    vc = np.asarray(vc, dtype=dtype)
    L, d = q.shape
    s = dtype(default_scale(d) if scale is None else scale)
    nq, nk = _nblocks(L, block_q), _nblocks(L, block_k)
    n_k = block_sizes(L, block_k).astype(dtype)
    n_chunks = _nblocks(nk, chunk)
    order = list(range(n_chunks)) if chunk_order is None else list(chunk_order)
    assert sorted(order) == list(range(n_chunks))
    out = np.full((L, d), np.nan, dtype=dtype)
    mask_out = np.zeros((nq, nk), dtype=bool)
    tiles = range(nq) if q_tiles is None else q_tiles
    for i in tiles:
        qi = q[i * block_q:(i + 1) * block_q]
        rows = qi.shape[0]
        qbar_i = qi.mean(axis=0)
        acc = np.zeros((rows, d), dtype=dtype)
        l = np.zeros(rows, dtype=dtype)
        m = np.full(rows, -np.inf, dtype=dtype)
        for t in order:                                           # outer loop
            j0, j1 = t * chunk, min((t + 1) * chunk, nk)
            s_tile = (qi @ kc[j0:j1].T) * s                       # token-to-block tile
            if mask_override is not None:
                routed = np.asarray(mask_override[i, j0:j1], dtype=bool)
            else:
                routed = (kc[j0:j1] @ qbar_i) * s > tau[i]        # Eq. (3) proxy vs tau_i
            mask_out[i, j0:j1] = routed
            if not exact_only:
                s_ap = np.where(routed[None, :], -np.inf, s_tile)
                acc, l, m = _online_update(s_ap, n_k[j0:j1], vc[j0:j1], acc, l, m)
            inner = np.flatnonzero(routed)
            if inner_reverse:
                inner = inner[::-1]
            for r in inner:                                       # inner loop
                j = j0 + r
                kj = k[j * block_k:(j + 1) * block_k]
                vj = v[j * block_k:(j + 1) * block_k]
                s_ex = (qi @ kj.T) * s
                acc, l, m = _online_update(s_ex, np.ones(kj.shape[0], dtype=dtype), vj, acc, l, m)
        with np.errstate(invalid="ignore", divide="ignore"):
            out[i * block_q:(i + 1) * block_q] = acc / l[:, None]
    return out, mask_out


# --------------------------------------------------------------------------- whole path
@dataclass
class SolAttnResult:
    out: np.ndarray          # [L, d]
    mask: np.ndarray         # [N_q, N_k] bool, True = exact branch
    counts: np.ndarray       # [N_q] selected blocks per query block
    s_hat: np.ndarray        # [N_q, N_k] proxy scores (scaled)
    mu: np.ndarray
    sigma: np.ndarray
    tau: np.ndarray
    qbar: np.ndarray
    kc: np.ndarray
    vc: np.ndarray


def routing(q, k, v, block_q: int, block_k: int, beta: float,
            scale: Optional[float] = None, dtype=np.float64, estimator: str = "direct", forced=None):
    """Pre-attention step only: pooled tensors, proxy rows, thresholds and the block mask.

    ``estimator``: "direct" (row statistics of the proxy row, Eq. 4 -- equal to the moment form of
    Eq. 5) or "diagonal" (Eq. appendix_diagonal_threshold).  ``forced``: optional bool [N_k]; those
    key blocks are put into every S_i regardless of their score (text / sink key-value tokens that
    the paper's model integrations keep in the exact branch)."""
    q = np.asarray(q, dtype=dtype)
    d = q.shape[1]
    s = default_scale(d) if scale is None else scale
    qbar, kc, vc, _ = pool(q, k, v, block_q, block_k, dtype=dtype)
    s_hat = proxy_scores(qbar, kc, s)
    if estimator == "direct":
        mu, sigma, tau = threshold_direct(s_hat, beta)
    elif estimator == "diagonal":
        mu, sigma, tau = threshold_diagonal(qbar, kc, beta, s)
    else:
        raise ValueError(estimator)
    mask = select_blocks(s_hat, tau)
    if forced is not None:
        mask = mask | np.asarray(forced, dtype=bool)[None, :]
    return SolAttnResult(out=None, mask=mask, counts=mask.sum(axis=1), s_hat=s_hat, mu=mu,
                         sigma=sigma, tau=tau, qbar=qbar, kc=kc, vc=vc)


def sol_attn_forward(q, k, v, block_q: int, block_k: int, beta: float,
                     scale: Optional[float] = None, chunk: int = 16, dtype=np.float64,
                     q_tiles: Optional[Sequence[int]] = None, mask_override=None,
                     exact_only: bool = False, estimator: str = "direct", forced=None) -> SolAttnResult:
    """The hot path for one head: pool -> proxy row -> tau_i -> Algorithm 1."""
    r = routing(q, k, v, block_q, block_k, beta, scale=scale, dtype=dtype, estimator=estimator, forced=forced)
    if forced is not None and mask_override is None:
        mask_override = r.mask          # Algorithm 1 run under the routed-or-forced mask
    out, mask = sol_attn_streaming(q, k, v, r.kc, r.vc, r.tau, block_q, block_k, chunk=chunk,
                                   scale=scale, dtype=dtype, q_tiles=q_tiles,
                                   mask_override=mask_override, exact_only=exact_only)
    if mask_override is None and q_tiles is None:
        # chunk-wise thresholding must recover full-row thresholding (the union property of
        # Sec. 3.2); only exact ties, decided by summation order, may differ
        diff = mask != r.mask
        tie = np.abs(r.s_hat - r.tau[:, None]) <= 64 * np.finfo(dtype).eps * (1 + np.abs(r.tau[:, None]))
        assert not (diff & ~tie).any(), "chunk-wise and full-row thresholding disagree"
        r.mask = mask
        r.counts = mask.sum(axis=1)
    r.out = out
    if mask_override is not None:
        r.mask = np.asarray(mask_override, dtype=bool)
        r.counts = r.mask.sum(axis=1)
    return r


def gaussian_density(beta: float) -> float:
    """rho_G(beta) = 1 - Phi(beta): selected density under the Gaussian reference."""
    return 0.5 * math.erfc(beta / math.sqrt(2.0))
