"""ctypes binding of the Sol-Attn C ABI (``include/sol_attn.h``).

Argument marshalling only: every step of the path runs in the CUDA library.  Tensors are
torch CUDA tensors (bf16 ``[B, H, N, d]``, contiguous); torch provides device memory and
streams, nothing else.  The functions mirror the C entry points by name.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("SOL_ATTN_LIB", os.path.join(_PKG, "libsol_attn.so"))   # override: profiling build

SOL_OK = 0
SOL_ERR_INVALID_ARG = -1
SOL_ERR_UNSUPPORTED_SHAPE = -2
SOL_ERR_UNSUPPORTED_ARCH = -3
SOL_ERR_WORKSPACE = -4
SOL_ERR_CUDA = -5
SOL_ERR_DEVICE_TIMEOUT = -6
SOL_ERR_SCRATCH_LIMIT = -7
SOL_ERR_STATIC_SCRATCH = -8

SOL_MODE_SOL, SOL_MODE_DENSE, SOL_MODE_EXACT_ONLY = 0, 1, 2
SOL_IMPL_AUTO, SOL_IMPL_TCGEN05, SOL_IMPL_MMA_SYNC = 0, 1, 2
SOL_EST_MOMENTS, SOL_EST_DIAGONAL = 0, 1
SOL_LAYOUT_BHND, SOL_LAYOUT_BNHD = 0, 1
SOL_ROUTING_FUSED, SOL_ROUTING_PREPASS = 0, 1
SOL_ROUTE_TOPK, SOL_ROUTE_TOPP = 0, 1

EXPORTS = [
    "sol_attn_status_string", "sol_attn_workspace_bytes", "sol_attn_workspace_view",
    "sol_attn_bind_workspace", "sol_attn_pool", "sol_attn_forward", "sol_attn_dense",
    "sol_attn_forward_ex", "sol_attn_forward_host", "sol_attn_read_device_status",
    "sol_attn_launch_count", "sol_attn_thresholds_static", "sol_attn_thresholds_static_max_floats",
    "sol_attn_route_materialized", "sol_attn_thresholds", "sol_attn_debug_set_wait", "sol_attn_route_mask",
]


class SolAttnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


class _WsView(ctypes.Structure):
    _fields_ = [(n, ctypes.c_size_t) for n in
                ("status", "qbar", "kc", "vc", "mu", "sigma", "tau", "total_bytes")] + \
               [("n_q_blocks", ctypes.c_int32), ("n_k_blocks", ctypes.c_int32)]


class _Args(ctypes.Structure):
    _fields_ = [
        ("q", ctypes.c_void_p), ("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("out", ctypes.c_void_p),
        ("B", ctypes.c_int32), ("H", ctypes.c_int32), ("N", ctypes.c_int32), ("d", ctypes.c_int32),
        ("block_q", ctypes.c_int32), ("block_k", ctypes.c_int32),
        ("threshold", ctypes.c_float), ("scale", ctypes.c_float),
        ("mode", ctypes.c_int32), ("impl", ctypes.c_int32), ("skip_pool", ctypes.c_int32),
        ("tau_override", ctypes.c_void_p),
        ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
        ("counts", ctypes.c_void_p), ("mask_out", ctypes.c_void_p),
        ("stream", ctypes.c_void_p),
        ("estimator", ctypes.c_int32), ("forced_blocks", ctypes.c_void_p),
        ("layout", ctypes.c_int32), ("routing", ctypes.c_int32),
    ]


_lib = None


def lib() -> ctypes.CDLL:
    """Load the CUDA library; fails loudly when it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2607_24027_b200.build` "
                          "(there is no CPU fallback)")
    L = ctypes.CDLL(LIB_PATH)
    L.sol_attn_status_string.restype = ctypes.c_char_p
    L.sol_attn_status_string.argtypes = [ctypes.c_int32]
    L.sol_attn_workspace_bytes.restype = ctypes.c_size_t
    L.sol_attn_workspace_bytes.argtypes = [ctypes.c_int] * 6
    L.sol_attn_workspace_view.restype = ctypes.c_int32
    L.sol_attn_workspace_view.argtypes = [ctypes.c_int] * 6 + [ctypes.POINTER(_WsView)]
    L.sol_attn_bind_workspace.restype = ctypes.c_int32
    L.sol_attn_bind_workspace.argtypes = [ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
    L.sol_attn_pool.restype = ctypes.c_int32
    L.sol_attn_pool.argtypes = [ctypes.c_void_p] * 3 + [ctypes.c_int] * 6 + [ctypes.c_float, ctypes.c_void_p]
    L.sol_attn_thresholds.restype = ctypes.c_int32
    L.sol_attn_thresholds.argtypes = [ctypes.c_int] * 6 + [ctypes.c_float] * 2 + [ctypes.c_int, ctypes.c_void_p]
    L.sol_attn_forward.restype = ctypes.c_int32
    L.sol_attn_forward.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int] * 6 + [ctypes.c_float, ctypes.c_void_p]
    L.sol_attn_dense.restype = ctypes.c_int32
    L.sol_attn_dense.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int] * 4 + [ctypes.c_void_p]
    L.sol_attn_forward_ex.restype = ctypes.c_int32
    L.sol_attn_forward_ex.argtypes = [ctypes.POINTER(_Args)]
    L.sol_attn_forward_host.restype = ctypes.c_int32
    L.sol_attn_forward_host.argtypes = [ctypes.c_void_p] * 8 + [ctypes.c_int] * 6 + [ctypes.c_float, ctypes.c_void_p]
    L.sol_attn_read_device_status.restype = ctypes.c_int32
    L.sol_attn_read_device_status.argtypes = [ctypes.c_void_p]
    L.sol_attn_launch_count.restype = ctypes.c_int64
    L.sol_attn_launch_count.argtypes = []
    L.sol_attn_route_mask.restype = ctypes.c_int32
    L.sol_attn_route_mask.argtypes = [ctypes.c_int] * 6 + [ctypes.c_float] + [ctypes.c_void_p] * 4
    L.sol_attn_thresholds_static.restype = ctypes.c_int32
    L.sol_attn_thresholds_static.argtypes = [ctypes.c_void_p] * 2 + [ctypes.c_int] * 5 + [ctypes.c_float] * 2 + \
                                            [ctypes.c_void_p] * 4
    L.sol_attn_thresholds_static_max_floats.restype = ctypes.c_size_t
    L.sol_attn_thresholds_static_max_floats.argtypes = []
    L.sol_attn_route_materialized.restype = ctypes.c_int32
    L.sol_attn_route_materialized.argtypes = [ctypes.c_void_p] * 2 + [ctypes.c_int] * 5 + [ctypes.c_float, ctypes.c_int,
                                                                                           ctypes.c_float] + \
                                             [ctypes.c_void_p] * 5
    L.sol_attn_debug_set_wait.restype = None
    L.sol_attn_debug_set_wait.argtypes = [ctypes.c_int64, ctypes.c_int32]
    _lib = L
    return L


def status_string(status: int) -> str:
    return lib().sol_attn_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != SOL_OK:
        raise SolAttnError(status, where)


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _dims(q: torch.Tensor):
    if q.dim() != 4 or not q.is_contiguous() or q.dtype != torch.bfloat16 or not q.is_cuda:
        raise ValueError("expected a contiguous CUDA bf16 tensor of shape [B, H, N, d]")
    return tuple(int(x) for x in q.shape)


# ----------------------------------------------------------------------------- workspace
def sol_attn_workspace_bytes(B, H, N, d, block_q, block_k) -> int:
    return int(lib().sol_attn_workspace_bytes(B, H, N, d, block_q, block_k))


@dataclass
class Workspace:
    """A device workspace plus typed views of the pre-attention results inside it."""
    buf: torch.Tensor            # uint8
    counts: torch.Tensor         # int32 [B, H, Nq]
    shape: tuple                 # (B, H, N, d, block_q, block_k)
    view: _WsView

    def _f32(self, off, *shape):
        n = 1
        for s in shape:
            n *= s
        return self.buf[off:off + 4 * n].view(torch.float32).view(*shape)

    @property
    def qbar(self):
        B, H, _, d, _, _ = self.shape
        return self._f32(self.view.qbar, B, H, self.view.n_q_blocks, d)

    @property
    def kc(self):
        B, H, _, d, _, _ = self.shape
        return self._f32(self.view.kc, B, H, self.view.n_k_blocks, d)

    @property
    def vc(self):
        B, H, _, d, _, _ = self.shape
        return self._f32(self.view.vc, B, H, self.view.n_k_blocks, d)

    def _per_q(self, off):
        B, H = self.shape[:2]
        return self._f32(off, B, H, self.view.n_q_blocks)

    @property
    def mu(self):
        return self._per_q(self.view.mu)

    @property
    def sigma(self):
        return self._per_q(self.view.sigma)

    @property
    def tau(self):
        return self._per_q(self.view.tau)


def make_workspace(B, H, N, d, block_q, block_k, device="cuda") -> Workspace:
    """Allocate (with torch) a workspace and counts array for one problem shape."""
    view = _WsView()
    _check(lib().sol_attn_workspace_view(B, H, N, d, block_q, block_k, ctypes.byref(view)), "sol_attn_workspace_view")
    buf = torch.empty(view.total_bytes + 1024, dtype=torch.uint8, device=device)
    off = (-buf.data_ptr()) % 1024
    buf = buf[off:off + view.total_bytes]
    counts = torch.zeros(B, H, view.n_q_blocks, dtype=torch.int32, device=device)
    return Workspace(buf=buf, counts=counts, shape=(B, H, N, d, block_q, block_k), view=view)


def sol_attn_bind_workspace(ws: Optional[Workspace]):
    if ws is None:
        _check(lib().sol_attn_bind_workspace(None, 0, None), "sol_attn_bind_workspace")
    else:
        _check(lib().sol_attn_bind_workspace(ws.buf.data_ptr(), ws.buf.numel(), ws.counts.data_ptr()),
               "sol_attn_bind_workspace")


# ----------------------------------------------------------------------------- entry points
def sol_attn_pool(q, k, v, block_q, block_k, threshold, stream=None):
    B, H, N, d = _dims(k)
    _check(lib().sol_attn_pool(_ptr(q), _ptr(k), _ptr(v), B, H, N, d, block_q, block_k,
                               float(threshold), _stream(stream)), "sol_attn_pool")


def sol_attn_forward(q, k, v, out, block_q, block_k, threshold, stream=None):
    B, H, N, d = _dims(q)
    _check(lib().sol_attn_forward(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, N, d, block_q, block_k,
                                  float(threshold), _stream(stream)), "sol_attn_forward")


def sol_attn_dense(q, k, v, out, stream=None):
    B, H, N, d = _dims(q)
    _check(lib().sol_attn_dense(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, N, d, _stream(stream)),
           "sol_attn_dense")


def sol_attn_forward_ex(q, k, v, out, ws: Workspace, block_q, block_k, threshold=0.0, scale=0.0,
                        mode=SOL_MODE_SOL, impl=SOL_IMPL_AUTO, skip_pool=False, tau_override=None,
                        counts=None, mask_out=None, stream=None, estimator=SOL_EST_MOMENTS, forced_blocks=None,
                        layout=SOL_LAYOUT_BHND, routing=SOL_ROUTING_FUSED):
    """``layout=SOL_LAYOUT_BNHD``: q, k, v and out are [B, N, H, d] tensors (heads interleaved)."""
    B, H, N, d = _dims(q)
    if layout == SOL_LAYOUT_BNHD:
        H, N = N, H
    a = _Args(q=_ptr(q), k=_ptr(k), v=_ptr(v), out=_ptr(out), B=B, H=H, N=N, d=d,
              block_q=block_q, block_k=block_k, threshold=float(threshold), scale=float(scale),
              mode=mode, impl=impl, skip_pool=int(skip_pool), tau_override=_ptr(tau_override),
              workspace=ws.buf.data_ptr(), workspace_bytes=ws.buf.numel(),
              counts=_ptr(counts if counts is not None else ws.counts), mask_out=_ptr(mask_out),
              stream=_stream(stream), estimator=int(estimator), forced_blocks=_ptr(forced_blocks),
              layout=int(layout), routing=int(routing))
    _check(lib().sol_attn_forward_ex(ctypes.byref(a)), "sol_attn_forward_ex")


def sol_attn_forward_host(hq, hk, hv, hout, dq, dk, dv, dout, block_q, block_k, threshold, stream=None):
    B, H, N, d = _dims(dq)
    _check(lib().sol_attn_forward_host(hq.data_ptr(), hk.data_ptr(), hv.data_ptr(), hout.data_ptr(),
                                       _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dout), B, H, N, d,
                                       block_q, block_k, float(threshold), _stream(stream)),
           "sol_attn_forward_host")


def sol_attn_thresholds_static(qbar, kc, threshold, mu, sigma, tau, scale=0.0, stream=None):
    """mu, sigma, tau (fp32 [B, H, Nq], caller-owned) from pooled queries / keys (fp32 [B, H, N*, d]) without
    any device allocation: the pooled-key moments go to an array built into the library."""
    B, H, Nq, d = (int(x) for x in qbar.shape)
    Nk = int(kc.shape[2])
    for t in (qbar, kc, mu, sigma, tau):
        if t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous():
            raise ValueError("expected contiguous CUDA fp32 tensors")
    _check(lib().sol_attn_thresholds_static(_ptr(qbar), _ptr(kc), B, H, Nq, Nk, d, float(scale), float(threshold),
                                            _ptr(mu), _ptr(sigma), _ptr(tau), _stream(stream)),
           "sol_attn_thresholds_static")


def sol_attn_thresholds(B, H, N, d, block_q, block_k, threshold, scale=0.0, estimator=SOL_EST_MOMENTS, stream=None):
    """Recompute mu, sigma, tau in the bound workspace from the pooled tensors already there."""
    _check(lib().sol_attn_thresholds(B, H, N, d, block_q, block_k, float(threshold), float(scale), int(estimator),
                                     _stream(stream)), "sol_attn_thresholds")


def sol_attn_route_mask(B, H, N, d, block_q, block_k, mask, scale=0.0, tau_override=None, forced_blocks=None, stream=None):
    """Eq. (4) decisions of the bound workspace's pooled tensors and thresholds, one bit per block pair, into ``mask``
    (int32 / uint32 [B, H, Nq, ceil(Nk / 32)])."""
    _check(lib().sol_attn_route_mask(B, H, N, d, block_q, block_k, float(scale), _ptr(tau_override), _ptr(forced_blocks),
                                     _ptr(mask), _stream(stream)), "sol_attn_route_mask")


def sol_attn_route_materialized(qbar, kc, policy, param, proxy_map, tau, order=None, counts=None, scale=0.0,
                                stream=None):
    """Top-k / top-p routing over a proxy map written to ``proxy_map`` (fp32 [B, H, Nq, Nk]); fills ``tau``
    (fp32 [B, H, Nq], usable as ``tau_override``), optionally ``order`` (int32 [B, H, Nq, Nk]) and ``counts``."""
    B, H, Nq, d = (int(x) for x in qbar.shape)
    Nk = int(kc.shape[2])
    for t in (qbar, kc, proxy_map, tau):
        if t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous():
            raise ValueError("expected contiguous CUDA fp32 tensors")
    for t in (order, counts):
        if t is not None and (t.dtype != torch.int32 or not t.is_cuda or not t.is_contiguous()):
            raise ValueError("expected contiguous CUDA int32 tensors")
    if proxy_map.numel() != B * H * Nq * Nk or tau.numel() != B * H * Nq:
        raise ValueError("proxy_map / tau have the wrong size")
    _check(lib().sol_attn_route_materialized(_ptr(qbar), _ptr(kc), B, H, Nq, Nk, d, float(scale), int(policy),
                                             float(param), _ptr(proxy_map), _ptr(order), _ptr(tau), _ptr(counts),
                                             _stream(stream)),
           "sol_attn_route_materialized")


def sol_attn_thresholds_static_max_floats() -> int:
    return int(lib().sol_attn_thresholds_static_max_floats())


def sol_attn_read_device_status(stream=None) -> int:
    return int(lib().sol_attn_read_device_status(_stream(stream)))


def sol_attn_launch_count() -> int:
    return int(lib().sol_attn_launch_count())


def sol_attn_debug_set_wait(wait_cycles: int = 0, withhold_tile: int = -1):
    """Testing hook: bound of the kernel's device-side waits (SM clocks, <= 0: default) and the tile per CTA
    whose completion signal is withheld (< 0: none)."""
    lib().sol_attn_debug_set_wait(int(wait_cycles), int(withhold_tile))


def mask_words(n_k_blocks: int) -> int:
    return (n_k_blocks + 31) // 32
