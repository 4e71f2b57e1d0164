"""Seeded synthetic q/k/v generators for the Sol-Attn workloads.

This module only draws random numbers and lays them out; it holds none of the
method's arithmetic (no pooling, no proxies, no softmax).  Both the CPU oracle's
tests and the CUDA path's tests feed on the arrays it returns, so the two sides
always see identical bits.

Every tensor is produced as bf16: the generator rounds float32 values to bf16
with round-to-nearest-even and returns the raw 16-bit patterns (``uint16``).
``widen`` turns such patterns back into exactly-representable float32/float64.

The inputs stand in for real video-DiT activations (the paper profiles its kernel
on q/k/v captured from Wan2.1 / HunyuanVideo / LTX / Bernini, which are not
available offline).  They reproduce the structural facts the method relies on:

* locality: q, k and v of a token share a 3D sinusoidal position feature, so
  nearby tokens attend to each other more strongly (block proxies are structured
  and near-Gaussian, as in the paper's Fig. "threshold_density");
* sinks: a few high-norm key tokens per frame that every query attends to
  (the sink-dominated rows the introduction mentions);
* editing: a target sequence strongly correlated with a source sequence that is
  concatenated in front of it (the longer video-editing sequences of Sec. 4).

Recipe (frozen; the stored thresholds in ``configs.py`` depend on it):

* token order is row-major ``(t, y, x)``, ``x`` fastest;
* position feature ``p(t,y,x)`` in R^d, shared by all heads and by q, k, v:
  channels are split ``d/4 : 3d/8 : 3d/8`` over (t, y, x) (``0 : d/2 : d/2`` when
  the grid has one frame); an axis of extent A with n channels gets n/2 sin/cos
  pairs with wavelengths spaced geometrically from 2A down to 2;
* ``x = bf16(noise + 0.8 * p)`` with independent N(0,1) noise per tensor and head,
  drawn head by head in the order q, k, v from ``PCG64(seed)`` as float32;
* sinks (video workloads): with ``g_h ~ N(0, I_d)`` fixed per head (drawn from
  ``PCG64(seed + 1)``), the 4 tokens ``(t, 0, 0..3)`` of every frame get
  ``k += 4 g_h`` and every query gets ``q += 0.1 g_h``;
* editing: the source grid is generated as above, then a target copy is
  appended with ``x_tgt = bf16(x_src + 0.3 * noise')`` for q, k and v (the float32
  source values before rounding are used; ``noise'`` continues the same stream,
  drawn after the head's source q, k, v in the order q, k, v).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Iterator, Tuple

import numpy as np


# --------------------------------------------------------------------------- bf16 helpers
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round-to-nearest-even); returns uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    out = ((u + rounding) >> np.uint32(16)).astype(np.uint16)
    return out


def widen(bits: np.ndarray, dtype=np.float32) -> np.ndarray:
    """bf16 bit patterns (uint16) -> exactly equal float32 (or float64) values."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    f32 = (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return f32.astype(dtype, copy=False)


# --------------------------------------------------------------------------- workload description
@dataclass(frozen=True)
class Workload:
    """Shape and generator options of one synthetic workload.

    ``grid`` is the (T, Hh, W) token grid of ONE sequence segment; ``edit`` appends a
    correlated target copy of the segment, doubling the sequence length.
    """

    name: str
    batch: int
    heads: int
    d: int
    grid: Tuple[int, int, int]
    block: int
    seed: int = 0
    sinks: bool = False
    edit: bool = False
    pos_gain: float = 0.8

    @property
    def seg_len(self) -> int:
        t, h, w = self.grid
        return t * h * w

    @property
    def seq_len(self) -> int:
        return self.seg_len * (2 if self.edit else 1)

    @property
    def n_blocks(self) -> int:
        return -(-self.seq_len // self.block)


def _axis_features(extent: int, n_channels: int) -> np.ndarray:
    """[extent, n_channels] sin/cos features; wavelengths geometric from 2*extent to 2."""
    if n_channels == 0:
        return np.zeros((extent, 0), dtype=np.float64)
    assert n_channels % 2 == 0, "an axis needs an even number of channels"
    pairs = n_channels // 2
    if pairs == 1:
        lam = np.array([2.0 * extent])
    else:
        m = np.arange(pairs, dtype=np.float64) / (pairs - 1)
        lam = 2.0 * extent * (1.0 / extent) ** m
    pos = np.arange(extent, dtype=np.float64)[:, None]
    ang = 2.0 * np.pi * pos / lam[None, :]
    out = np.empty((extent, n_channels), dtype=np.float64)
    out[:, 0::2] = np.sin(ang)
    out[:, 1::2] = np.cos(ang)
    return out


def position_features(grid: Tuple[int, int, int], d: int) -> np.ndarray:
    """[T*Hh*W, d] float32 position feature, tokens in (t, y, x) order, x fastest."""
    t, h, w = grid
    if t == 1:
        d_t, d_y, d_x = 0, d // 2, d // 2
    else:
        d_t = d // 4
        d_y = (3 * d) // 8
        d_x = d - d_t - d_y
    ft = _axis_features(t, d_t)
    fy = _axis_features(h, d_y)
    fx = _axis_features(w, d_x)
    p = np.empty((t, h, w, d), dtype=np.float32)
    p[..., :d_t] = ft[:, None, None, :]
    p[..., d_t:d_t + d_y] = fy[None, :, None, :]
    p[..., d_t + d_y:] = fx[None, None, :, :]
    return p.reshape(t * h * w, d)


def sink_token_indices(grid: Tuple[int, int, int]) -> np.ndarray:
    """Indices (within one segment) of the tokens (t, 0, 0..3) of every frame."""
    t, h, w = grid
    per_frame = h * w
    cols = np.arange(min(4, w))
    return (np.arange(t)[:, None] * per_frame + cols[None, :]).reshape(-1)


def iter_heads(wl: Workload) -> Iterator[Tuple[int, int, np.ndarray, np.ndarray, np.ndarray]]:
    """Yield ``(b, h, q_bits, k_bits, v_bits)`` per (batch, head); arrays are [L, d] uint16."""
    rng = np.random.Generator(np.random.PCG64(wl.seed))
    rng_sink = np.random.Generator(np.random.PCG64(wl.seed + 1))
    pos = position_features(wl.grid, wl.d) * np.float32(wl.pos_gain)
    seg, d = wl.seg_len, wl.d
    sink_idx = sink_token_indices(wl.grid) if wl.sinks else None
    for b in range(wl.batch):
        for h in range(wl.heads):
            src = []
            for _name in ("q", "k", "v"):
                x = rng.standard_normal((seg, d), dtype=np.float32)
                x += pos
                src.append(x)
            if wl.sinks:
                g = rng_sink.standard_normal(d, dtype=np.float32)
                src[0] += np.float32(0.1) * g
                src[1][sink_idx] += np.float32(4.0) * g
            if wl.edit:
                full = []
                for x in src:
                    n = rng.standard_normal((seg, d), dtype=np.float32)
                    tgt = x + np.float32(0.3) * n
                    full.append(np.concatenate([x, tgt], axis=0))
                src = full
            yield b, h, f32_to_bf16_bits(src[0]), f32_to_bf16_bits(src[1]), f32_to_bf16_bits(src[2])


def generate(wl: Workload, heads: slice | None = None):
    """Materialise q, k, v as uint16 arrays of shape [B, H, L, d].

    ``heads`` (a slice over the flattened (b, h) index) keeps only part of the job in
    memory; the random stream is still advanced through the skipped heads so a head's
    bits never depend on which other heads were requested.
    """
    bh_total = wl.batch * wl.heads
    sel = range(bh_total)[heads] if heads is not None else range(bh_total)
    sel = list(sel)
    L, d = wl.seq_len, wl.d
    q = np.empty((len(sel), L, d), dtype=np.uint16)
    k = np.empty_like(q)
    v = np.empty_like(q)
    want = {bh: i for i, bh in enumerate(sel)}
    last = max(sel) if sel else -1
    for b, h, qb, kb, vb in iter_heads(wl):
        bh = b * wl.heads + h
        if bh in want:
            i = want[bh]
            q[i], k[i], v[i] = qb, kb, vb
        if bh >= last:
            break
    if heads is None:
        shape = (wl.batch, wl.heads, L, d)
        return q.reshape(shape), k.reshape(shape), v.reshape(shape)
    return q, k, v


def gaussian_qkv(seed: int, bh: int, L: int, d: int):
    """Plain iid N(0,1) bf16 q, k, v of shape [bh, L, d] (uint16 bits) for statistical tests."""
    rng = np.random.Generator(np.random.PCG64(seed))
    out = []
    for _ in range(3):
        out.append(f32_to_bf16_bits(rng.standard_normal((bh, L, d), dtype=np.float32)))
    return tuple(out)
