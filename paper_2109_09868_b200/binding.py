"""Thin Python binding of ``libapproxifer.so`` (declared in ``include/approxifer.h``).

Argument marshalling only: tensors are turned into device pointers and element
strides, and the C entry point of the same name is called.  Every step of the
computation runs in the library's CUDA kernels; there is no fallback of any
kind -- a missing library or a non-CUDA tensor raises.
"""
from __future__ import annotations

import ctypes
import os
import shutil
from ctypes import POINTER, c_char_p, c_float, c_int, c_int32, c_int64, c_uint32, c_void_p
from typing import Optional

import torch

from . import build as _build

OK = 0
E_NULL, E_RANGE, E_PARAM, E_CUDA, E_WORKSPACE, E_TOO_LARGE = -1, -2, -3, -4, -5, -6
STATIC_WORKSPACE_BYTES = 32 << 20
SIGN_RANK, SIGN_WORKER_INDEX = 0, 1
LOCATE_HOMOGENEOUS = 2
ONE_PASS, TWO_LAUNCHES = 4, 8
ST_NO_WORKERS, ST_FEW_WORKERS, ST_LOCATE_UNDERDETERMINED, ST_NONFINITE, ST_TIMEOUT = 1, 2, 4, 8, 16

EXPORTS = (
    "approxifer_encode",
    "approxifer_decode",
    "approxifer_locate",
    "approxifer_locate_decode",
    "approxifer_decode_rational",
    "approxifer_debug_weights",
    "approxifer_strerror",
    "approxifer_version",
    "approxifer_launch_count",
    "approxifer_debug_decode",
    "approxifer_device_wait_timeouts",
    "approxifer_reset_device_wait_timeouts",
    "approxifer_debug_locate",
    "approxifer_encode_host",
    "approxifer_decode_host",
    "approxifer_locate_host",
    "approxifer_encode_host_static",
    "approxifer_debug_fma_peak",
    "approxifer_debug_pack_rotation",
    "approxifer_encode_scatter",
    "approxifer_decode_gather",
    "approxifer_locate_gather",
    "approxifer_encode_bf16",
    "approxifer_decode_bf16",
)


class approxifer_params(ctypes.Structure):
    _fields_ = [("K", c_int32), ("W", c_int32), ("E", c_int32), ("flags", c_uint32)]


class approxifer_decode_tuning(ctypes.Structure):
    _fields_ = [("kernel", c_int32), ("stages", c_int32), ("ctas_per_sm", c_int32), ("cols", c_int32), ("split", c_int32),
                ("wait_limit", c_uint32), ("withhold_group_plus1", c_int64)]


class ApproxiferError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: %s (code %d)" % (where, strerror(code), code))


_lib = None


def library_path() -> str:
    return _build.LIB


def load() -> ctypes.CDLL:
    """Load the CUDA library, (re)building it first if nvcc is present and the
    sources are newer.  Raises if no library can be had."""
    global _lib
    if _lib is not None:
        return _lib
    have_nvcc = shutil.which("nvcc") is not None or os.path.exists("/usr/local/cuda/bin/nvcc")
    if have_nvcc and _build.is_stale():
        _build.build()
    if not os.path.exists(_build.LIB):
        raise RuntimeError(
            "libapproxifer.so is missing and cannot be built (no nvcc): run `python -m paper_2109_09868_b200.build`"
        )
    lib = ctypes.CDLL(_build.LIB)
    pf, pu, pi = POINTER(c_float), POINTER(c_uint32), POINTER(c_int32)
    pp = POINTER(approxifer_params)
    lib.approxifer_encode.argtypes = [pp, c_int64, c_int64, c_void_p, c_int64, c_int64, c_void_p, c_int64, c_int64, c_void_p]
    lib.approxifer_encode.restype = c_int
    lib.approxifer_decode.argtypes = [pp, c_int64, c_int64, c_void_p, c_int64, c_int64, c_void_p, c_void_p, c_int64,
                                      c_int64, c_void_p, c_void_p, c_void_p]
    lib.approxifer_decode.restype = c_int
    lib.approxifer_encode_bf16.argtypes = lib.approxifer_encode.argtypes
    lib.approxifer_encode_bf16.restype = c_int
    lib.approxifer_decode_bf16.argtypes = lib.approxifer_decode.argtypes
    lib.approxifer_decode_bf16.restype = c_int
    lib.approxifer_encode_scatter.argtypes = [pp, c_int64, c_int64, c_void_p, c_int64, c_int64, POINTER(c_void_p), c_int64, c_void_p]
    lib.approxifer_encode_scatter.restype = c_int
    lib.approxifer_decode_gather.argtypes = [pp, c_int64, c_int64, POINTER(c_void_p), c_int64, c_void_p, c_void_p, c_int64, c_int64,
                                             c_void_p, c_void_p, c_void_p]
    lib.approxifer_decode_gather.restype = c_int
    lib.approxifer_locate_gather.argtypes = [pp, c_int64, c_int64, POINTER(c_void_p), c_int64, c_void_p, c_void_p, c_void_p, c_void_p,
                                             c_void_p]
    lib.approxifer_locate_gather.restype = c_int
    lib.approxifer_locate.argtypes = [pp, c_int64, c_int64, c_void_p, c_int64, c_int64, c_void_p, c_void_p, c_void_p,
                                      c_void_p, c_void_p]
    lib.approxifer_locate.restype = c_int
    lib.approxifer_locate_decode.argtypes = [pp, c_int64, c_int64, c_void_p, c_int64, c_int64, c_void_p, c_void_p, c_void_p,
                                             c_void_p, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.approxifer_locate_decode.restype = c_int
    lib.approxifer_decode_rational.argtypes = [pp, c_int64, c_int64, c_void_p, c_int64, c_int64, c_void_p,
                                               c_void_p, c_int64, c_int64, c_void_p, c_void_p]
    lib.approxifer_decode_rational.restype = c_int
    lib.approxifer_debug_weights.argtypes = [pp, c_uint32, c_int, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.approxifer_debug_weights.restype = c_int
    lib.approxifer_strerror.argtypes = [c_int]
    lib.approxifer_strerror.restype = c_char_p
    lib.approxifer_version.restype = c_int
    lib.approxifer_launch_count.restype = c_int64
    lib.approxifer_debug_decode.argtypes = [pp, c_int64, c_int64, c_void_p, c_int64, c_int64, c_void_p, c_void_p, c_int64,
                                            c_int64, c_void_p, c_void_p, POINTER(approxifer_decode_tuning), c_void_p]
    lib.approxifer_debug_decode.restype = c_int
    lib.approxifer_device_wait_timeouts.restype = c_int64
    lib.approxifer_reset_device_wait_timeouts.restype = c_int
    lib.approxifer_debug_fma_peak.argtypes = [c_int, c_int, c_void_p, c_void_p]
    lib.approxifer_debug_fma_peak.restype = c_int
    lib.approxifer_debug_pack_rotation.argtypes = [ctypes.c_int32, ctypes.c_int32, c_int64, ctypes.c_int32,
                                                   POINTER(ctypes.c_int32), POINTER(ctypes.c_uint32),
                                                   POINTER(ctypes.c_int32), POINTER(ctypes.c_int32)]
    lib.approxifer_debug_pack_rotation.restype = c_int
    lib.approxifer_debug_locate.argtypes = [pp, c_int64, c_int64, c_void_p, c_int64, c_int64, c_void_p, c_void_p, c_void_p,
                                            c_void_p, c_int, c_void_p]
    lib.approxifer_debug_locate.restype = c_int
    c_size_t = ctypes.c_size_t
    lib.approxifer_encode_host.argtypes = [pp, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_size_t, POINTER(c_void_p), c_int]
    lib.approxifer_encode_host.restype = c_int
    lib.approxifer_decode_host.argtypes = [pp, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                           c_size_t, POINTER(c_void_p), c_int]
    lib.approxifer_decode_host.restype = c_int
    lib.approxifer_locate_host.argtypes = [pp, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                           c_size_t, POINTER(c_void_p), c_int]
    lib.approxifer_locate_host.restype = c_int
    lib.approxifer_encode_host_static.argtypes = [pp, c_int64, c_int64, c_void_p, c_void_p, c_void_p]
    lib.approxifer_encode_host_static.restype = c_int
    del pf, pu, pi
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load().approxifer_strerror(int(code)).decode()


def version() -> int:
    return int(load().approxifer_version())


def launch_count() -> int:
    return int(load().approxifer_launch_count())


def decode_tuning(kernel: int = 0, stages: int = 0, ctas_per_sm: int = 0, cols: int = 0, split: int = 0,
                  wait_limit: int = 0, withhold_group: int = -1) -> approxifer_decode_tuning:
    """Per-call kernel choice / launch plan for approxifer_decode(..., tuning=...) (tests and tuning only).
    wait_limit / withhold_group exercise the kernels' bounded waits (see approxifer_debug_decode)."""
    return approxifer_decode_tuning(int(kernel), int(stages), int(ctas_per_sm), int(cols), int(split), int(wait_limit),
                                    int(withhold_group) + 1)


def debug_fma_peak(iters: int, blocks: int, sink: torch.Tensor, stream=None) -> None:
    """Register-only fp32 multiply-add loop (2 * 64 * iters * 256 * blocks flop); time it with CUDA events."""
    rc = load().approxifer_debug_fma_peak(int(iters), int(blocks), sink.data_ptr(), _stream_ptr(stream))
    if rc != OK:
        raise ApproxiferError(rc, "approxifer_debug_fma_peak")


def debug_pack_rotation(K: int, W: int, C: int, mode: int = 0):
    """Host-side plan of the packed-groups decoder for a shape (no device call): (groups per work item, rotated
    groups as a bit set, modelled shared-memory passes per item without rotation, with the chosen one)."""
    gw, rot = ctypes.c_int32(0), ctypes.c_uint32(0)
    plain, chosen = ctypes.c_int32(0), ctypes.c_int32(0)
    rc = load().approxifer_debug_pack_rotation(int(K), int(W), int(C), int(mode), ctypes.byref(gw), ctypes.byref(rot),
                                               ctypes.byref(plain), ctypes.byref(chosen))
    if rc != OK:
        raise ApproxiferError(rc, "approxifer_debug_pack_rotation")
    return gw.value, rot.value, plain.value, chosen.value


def device_wait_timeouts() -> int:
    return int(load().approxifer_device_wait_timeouts())


def reset_device_wait_timeouts() -> None:
    rc = load().approxifer_reset_device_wait_timeouts()
    if rc != OK:
        raise ApproxiferError(rc, "approxifer_reset_device_wait_timeouts")


def make_params(K: int, W: int, E: int = 0, flags: int = 0) -> approxifer_params:
    return approxifer_params(int(K), int(W), int(E), int(flags))


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _payload(t: torch.Tensor, rows: int, name: str, dtype=torch.float32):
    if not t.is_cuda:
        raise ValueError("%s must be a CUDA tensor (the library has no CPU path)" % name)
    if t.dtype != dtype or t.dim() != 3 or t.shape[1] != rows:
        raise ValueError("%s must be %s [G][%d][L]" % (name, dtype, rows))
    if t.shape[2] > 1 and t.stride(2) != 1:
        raise ValueError("%s: innermost dimension must be contiguous" % name)
    return t.data_ptr(), t.stride(0), t.stride(1)


def _vec(t: Optional[torch.Tensor], dtype, n: int, name: str) -> int:
    if t is None:
        return 0
    if not t.is_cuda or t.dtype != dtype or t.numel() != n or not t.is_contiguous():
        raise ValueError("%s must be a contiguous CUDA %s tensor with %d elements" % (name, dtype, n))
    return t.data_ptr()


def approxifer_encode(params: approxifer_params, X: torch.Tensor, Xt: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """X [G][K][D] -> coded queries Xt [G][W][D] (allocated if not given)."""
    G, K, D = X.shape
    if Xt is None:
        Xt = torch.empty((G, params.W, D), device=X.device, dtype=torch.float32)
    xp, xg, xr = _payload(X, params.K, "X")
    op, og, orr = _payload(Xt, params.W, "Xt")
    if Xt.shape[0] != G or Xt.shape[2] != D:
        raise ValueError("Xt must be [G][W][D]")
    rc = load().approxifer_encode(ctypes.byref(params), G, D, xp, xg, xr, op, og, orr, _stream_ptr(stream))
    if rc != OK:
        raise ApproxiferError(rc, "approxifer_encode")
    return Xt


def approxifer_encode_bf16(params: approxifer_params, X: torch.Tensor, Xt: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """bfloat16 X [G][K][D] -> bfloat16 coded queries Xt [G][W][D] (fp32 weights and sums, one rounding)."""
    G, K, D = X.shape
    if Xt is None:
        Xt = torch.empty((G, params.W, D), device=X.device, dtype=torch.bfloat16)
    xp, xg, xr = _payload(X, params.K, "X", torch.bfloat16)
    op, og, orr = _payload(Xt, params.W, "Xt", torch.bfloat16)
    if Xt.shape[0] != G or Xt.shape[2] != D:
        raise ValueError("Xt must be [G][W][D]")
    rc = load().approxifer_encode_bf16(ctypes.byref(params), G, D, xp, xg, xr, op, og, orr, _stream_ptr(stream))
    if rc != OK:
        raise ApproxiferError(rc, "approxifer_encode_bf16")
    return Xt


def approxifer_decode_bf16(params: approxifer_params, Yt: torch.Tensor, mask: torch.Tensor, Yhat: Optional[torch.Tensor] = None,
                           n_used: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """bfloat16 Yt [G][W][C], mask [G] -> bfloat16 Yhat [G][K][C]."""
    G, W, C = Yt.shape
    if Yhat is None:
        Yhat = torch.empty((G, params.K, C), device=Yt.device, dtype=torch.bfloat16)
    yp, yg, yr = _payload(Yt, params.W, "Yt", torch.bfloat16)
    op, og, orr = _payload(Yhat, params.K, "Yhat", torch.bfloat16)
    if Yhat.shape[0] != G or Yhat.shape[2] != C:
        raise ValueError("Yhat must be [G][K][C]")
    rc = load().approxifer_decode_bf16(ctypes.byref(params), G, C, yp, yg, yr, _vec(mask, torch.int32, G, "mask"), op, og, orr,
                                       _vec(n_used, torch.int32, G, "n_used"), _vec(status, torch.int32, G, "status"),
                                       _stream_ptr(stream))
    if rc != OK:
        raise ApproxiferError(rc, "approxifer_decode_bf16")
    return Yhat


def approxifer_decode(params: approxifer_params, Yt: torch.Tensor, mask: torch.Tensor, Yhat: Optional[torch.Tensor] = None,
                      n_used: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None, stream=None,
                      tuning: Optional[approxifer_decode_tuning] = None) -> torch.Tensor:
    """Yt [G][W][C], mask [G] (int32 tensor holding the uint32 bit patterns) -> Yhat [G][K][C].
    With `tuning` the call goes through approxifer_debug_decode (same result, chosen kernel / launch plan)."""
    G, W, C = Yt.shape
    if Yhat is None:
        Yhat = torch.empty((G, params.K, C), device=Yt.device, dtype=torch.float32)
    yp, yg, yr = _payload(Yt, params.W, "Yt")
    op, og, orr = _payload(Yhat, params.K, "Yhat")
    if Yhat.shape[0] != G or Yhat.shape[2] != C:
        raise ValueError("Yhat must be [G][K][C]")
    mp = _vec(mask, torch.int32, G, "mask")
    if tuning is not None:
        rc = load().approxifer_debug_decode(ctypes.byref(params), G, C, yp, yg, yr, mp, op, og, orr,
                                            _vec(n_used, torch.int32, G, "n_used"), _vec(status, torch.int32, G, "status"),
                                            ctypes.byref(tuning), _stream_ptr(stream))
    else:
        rc = load().approxifer_decode(ctypes.byref(params), G, C, yp, yg, yr, mp, op, og, orr,
                                      _vec(n_used, torch.int32, G, "n_used"), _vec(status, torch.int32, G, "status"),
                                      _stream_ptr(stream))
    if rc != OK:
        raise ApproxiferError(rc, "approxifer_decode")
    return Yhat


def approxifer_locate(params: approxifer_params, Yt: torch.Tensor, mask: torch.Tensor, adv: Optional[torch.Tensor] = None,
                      trusted_mask: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None, stream=None,
                      force_warp_kernel: bool = False):
    """Yt [G][W][C], mask [G] -> (adv [G][E] int32, trusted_mask [G] int32 bit patterns).
    force_warp_kernel (tests): through approxifer_debug_locate, on the warp-per-group kernel."""
    G, W, C = Yt.shape
    E = max(int(params.E), 0)
    if adv is None:
        adv = torch.empty((G, E), device=Yt.device, dtype=torch.int32)
    if trusted_mask is None:
        trusted_mask = torch.empty((G,), device=Yt.device, dtype=torch.int32)
    yp, yg, yr = _payload(Yt, params.W, "Yt")
    args = (ctypes.byref(params), G, C, yp, yg, yr, _vec(mask, torch.int32, G, "mask"),
            _vec(adv, torch.int32, G * E, "adv"), _vec(trusted_mask, torch.int32, G, "trusted_mask"),
            _vec(status, torch.int32, G, "status"))
    if force_warp_kernel:
        rc = load().approxifer_debug_locate(*args, 1, _stream_ptr(stream))
    else:
        rc = load().approxifer_locate(*args, _stream_ptr(stream))
    if rc != OK:
        raise ApproxiferError(rc, "approxifer_locate")
    return adv, trusted_mask


def _row_buffers(rows, W: int, G: int, name: str):
    """W per-worker CUDA tensors [G][L] (innermost contiguous, same group stride) -> (pointer array, group stride, L)."""
    if len(rows) != W:
        raise ValueError("%s must hold one tensor per worker" % name)
    L, gs = rows[0].shape[1], rows[0].stride(0)
    for t in rows:
        if not t.is_cuda or t.dtype != torch.float32 or t.dim() != 2 or t.shape != (G, L) or t.stride(0) != gs or (L > 1 and t.stride(1) != 1):
            raise ValueError("%s: every worker's batch must be a float32 CUDA tensor [G][L] with the same group stride" % name)
    return (c_void_p * W)(*[t.data_ptr() for t in rows]), gs, L


def approxifer_encode_scatter(params: approxifer_params, X: torch.Tensor, Xt_rows, stream=None) -> None:
    """X [G][K][D] -> W per-worker batches Xt_rows[i] [G][D] (tensors of their own, possibly in peer memory)."""
    G, K, D = X.shape
    xp, xg, xr = _payload(X, params.K, "X")
    arr, gs, L = _row_buffers(Xt_rows, params.W, G, "Xt_rows")
    if L != D:
        raise ValueError("Xt_rows[i] must be [G][D]")
    rc = load().approxifer_encode_scatter(ctypes.byref(params), G, D, xp, xg, xr, arr, gs, _stream_ptr(stream))
    if rc != OK:
        raise ApproxiferError(rc, "approxifer_encode_scatter")


def approxifer_decode_gather(params: approxifer_params, Yt_rows, mask: torch.Tensor, Yhat: Optional[torch.Tensor] = None,
                             n_used: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """W per-worker prediction batches Yt_rows[i] [G][C], mask [G] -> Yhat [G][K][C]."""
    G = Yt_rows[0].shape[0]
    arr, gs, C = _row_buffers(Yt_rows, params.W, G, "Yt_rows")
    if Yhat is None:
        Yhat = torch.empty((G, params.K, C), device=Yt_rows[0].device, dtype=torch.float32)
    op, og, orr = _payload(Yhat, params.K, "Yhat")
    rc = load().approxifer_decode_gather(ctypes.byref(params), G, C, arr, gs, _vec(mask, torch.int32, G, "mask"), op, og, orr,
                                         _vec(n_used, torch.int32, G, "n_used"), _vec(status, torch.int32, G, "status"),
                                         _stream_ptr(stream))
    if rc != OK:
        raise ApproxiferError(rc, "approxifer_decode_gather")
    return Yhat


def approxifer_locate_gather(params: approxifer_params, Yt_rows, mask: torch.Tensor, status: Optional[torch.Tensor] = None, stream=None):
    """W per-worker prediction batches Yt_rows[i] [G][C], mask [G] -> (adv [G][E], trusted_mask [G])."""
    G = Yt_rows[0].shape[0]
    arr, gs, C = _row_buffers(Yt_rows, params.W, G, "Yt_rows")
    E = max(int(params.E), 0)
    adv = torch.empty((G, E), device=Yt_rows[0].device, dtype=torch.int32)
    trusted = torch.empty((G,), device=Yt_rows[0].device, dtype=torch.int32)
    rc = load().approxifer_locate_gather(ctypes.byref(params), G, C, arr, gs, _vec(mask, torch.int32, G, "mask"), adv.data_ptr(),
                                         trusted.data_ptr(), _vec(status, torch.int32, G, "status"), _stream_ptr(stream))
    if rc != OK:
        raise ApproxiferError(rc, "approxifer_locate_gather")
    return adv, trusted


def approxifer_decode_rational(params: approxifer_params, Yt: torch.Tensor, mask: torch.Tensor, Yhat: Optional[torch.Tensor] = None,
                               status: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Algorithm 3: Yhat[g][j][c] = P(alpha_j) / Q(alpha_j) with P, Q from the least-squares system of the locator."""
    G, W, C = Yt.shape
    if Yhat is None:
        Yhat = torch.empty((G, params.K, C), device=Yt.device, dtype=torch.float32)
    yp, yg, yr = _payload(Yt, params.W, "Yt")
    op, og, orr = _payload(Yhat, params.K, "Yhat")
    rc = load().approxifer_decode_rational(ctypes.byref(params), G, C, yp, yg, yr, _vec(mask, torch.int32, G, "mask"),
                                           op, og, orr, _vec(status, torch.int32, G, "status"), _stream_ptr(stream))
    if rc != OK:
        raise ApproxiferError(rc, "approxifer_decode_rational")
    return Yhat


def approxifer_locate_decode(params: approxifer_params, Yt: torch.Tensor, mask: torch.Tensor, Yhat: Optional[torch.Tensor] = None,
                             n_used: Optional[torch.Tensor] = None, locate_status: Optional[torch.Tensor] = None,
                             decode_status: Optional[torch.Tensor] = None, stream=None):
    """Locate the E Byzantine workers of every group, then decode from the remaining present workers.
    Returns (Yhat [G][K][C], adv [G][E], trusted_mask [G])."""
    G, W, C = Yt.shape
    E = max(int(params.E), 0)
    adv = torch.empty((G, E), device=Yt.device, dtype=torch.int32)
    trusted = torch.empty((G,), device=Yt.device, dtype=torch.int32)
    if Yhat is None:
        Yhat = torch.empty((G, params.K, C), device=Yt.device, dtype=torch.float32)
    yp, yg, yr = _payload(Yt, params.W, "Yt")
    op, og, orr = _payload(Yhat, params.K, "Yhat")
    rc = load().approxifer_locate_decode(ctypes.byref(params), G, C, yp, yg, yr, _vec(mask, torch.int32, G, "mask"),
                                         adv.data_ptr(), trusted.data_ptr(), op, og, orr,
                                         _vec(n_used, torch.int32, G, "n_used"),
                                         _vec(locate_status, torch.int32, G, "locate_status"),
                                         _vec(decode_status, torch.int32, G, "decode_status"), _stream_ptr(stream))
    if rc != OK:
        raise ApproxiferError(rc, "approxifer_locate_decode")
    return Yhat, adv, trusted


def approxifer_debug_weights(params: approxifer_params, mask: int = 0, which: int = 0, stream=None):
    """which=0: encoder weights [W][K]; which=1: (decoder weights [K][n], worker indices) for `mask`."""
    dev = torch.device("cuda")
    K, W = params.K, params.W
    if which == 0:
        w = torch.empty((W, K), device=dev, dtype=torch.float32)
        rc = load().approxifer_debug_weights(ctypes.byref(params), 0, 0, w.data_ptr(), 0, 0, _stream_ptr(stream))
        if rc != OK:
            raise ApproxiferError(rc, "approxifer_debug_weights")
        return w
    w = torch.empty((K, W), device=dev, dtype=torch.float32)
    idx = torch.empty((W,), device=dev, dtype=torch.int32)
    n = torch.empty((1,), device=dev, dtype=torch.int32)
    rc = load().approxifer_debug_weights(ctypes.byref(params), int(mask) & 0xFFFFFFFF, 1, w.data_ptr(), idx.data_ptr(),
                                         n.data_ptr(), _stream_ptr(stream))
    if rc != OK:
        raise ApproxiferError(rc, "approxifer_debug_weights")
    nn = int(n.item())
    return w[:, :nn], idx[:nn]


def _host(t: Optional[torch.Tensor], dtype, shape, name: str) -> int:
    if t is None:
        return 0
    if t.is_cuda or t.dtype != dtype or tuple(t.shape) != tuple(shape) or not t.is_contiguous():
        raise ValueError("%s must be a contiguous host %s tensor of shape %s" % (name, dtype, tuple(shape)))
    return t.data_ptr()


def _streams(streams):
    arr = (c_void_p * len(streams))(*[int(s.cuda_stream) for s in streams])
    return arr, len(streams)


def _workspace(workspace: torch.Tensor):
    if not workspace.is_cuda or not workspace.is_contiguous():
        raise ValueError("workspace must be a contiguous CUDA tensor")
    return workspace.data_ptr(), workspace.numel() * workspace.element_size()


def approxifer_encode_host(params: approxifer_params, hX: torch.Tensor, hXt: torch.Tensor, workspace: torch.Tensor, streams) -> None:
    """Host tensors hX [G][K][D] -> hXt [G][W][D], staged through the device `workspace` on `streams`.
    Only enqueues; synchronise the streams before touching the buffers."""
    G, K, D = hX.shape
    wp, wbytes = _workspace(workspace)
    arr, n = _streams(streams)
    rc = load().approxifer_encode_host(ctypes.byref(params), G, D, _host(hX, torch.float32, (G, params.K, D), "hX"),
                                       _host(hXt, torch.float32, (G, params.W, D), "hXt"), wp, wbytes, arr, n)
    if rc != OK:
        raise ApproxiferError(rc, "approxifer_encode_host")


def approxifer_decode_host(params: approxifer_params, hYt: torch.Tensor, hmask: torch.Tensor, hYhat: torch.Tensor,
                           workspace: torch.Tensor, streams, hn_used: Optional[torch.Tensor] = None,
                           hstatus: Optional[torch.Tensor] = None) -> None:
    G, W, C = hYt.shape
    wp, wbytes = _workspace(workspace)
    arr, n = _streams(streams)
    rc = load().approxifer_decode_host(ctypes.byref(params), G, C, _host(hYt, torch.float32, (G, params.W, C), "hYt"),
                                       _host(hmask, torch.int32, (G,), "hmask"),
                                       _host(hYhat, torch.float32, (G, params.K, C), "hYhat"),
                                       _host(hn_used, torch.int32, (G,), "hn_used"), _host(hstatus, torch.int32, (G,), "hstatus"),
                                       wp, wbytes, arr, n)
    if rc != OK:
        raise ApproxiferError(rc, "approxifer_decode_host")


def approxifer_locate_host(params: approxifer_params, hYt: torch.Tensor, hmask: torch.Tensor, hadv: torch.Tensor,
                           htrusted: torch.Tensor, workspace: torch.Tensor, streams, hstatus: Optional[torch.Tensor] = None) -> None:
    G, W, C = hYt.shape
    wp, wbytes = _workspace(workspace)
    arr, n = _streams(streams)
    rc = load().approxifer_locate_host(ctypes.byref(params), G, C, _host(hYt, torch.float32, (G, params.W, C), "hYt"),
                                       _host(hmask, torch.int32, (G,), "hmask"),
                                       _host(hadv, torch.int32, (G, max(int(params.E), 0)), "hadv"),
                                       _host(htrusted, torch.int32, (G,), "htrusted"), _host(hstatus, torch.int32, (G,), "hstatus"),
                                       wp, wbytes, arr, n)
    if rc != OK:
        raise ApproxiferError(rc, "approxifer_locate_host")


def approxifer_encode_host_static(params: approxifer_params, hX: torch.Tensor, hXt: torch.Tensor, stream=None) -> None:
    """Encoder for callers that cannot allocate device memory: host tensors hX [G][K][D] -> hXt [G][W][D],
    staged through the library's built-in device array (at most STATIC_WORKSPACE_BYTES per call).  Only
    enqueues on `stream`; synchronise it before reading hXt.  Calls that may overlap on the GPU race."""
    G, K, D = hX.shape
    rc = load().approxifer_encode_host_static(ctypes.byref(params), G, D, _host(hX, torch.float32, (G, params.K, D), "hX"),
                                              _host(hXt, torch.float32, (G, params.W, D), "hXt"), _stream_ptr(stream))
    if rc != OK:
        raise ApproxiferError(rc, "approxifer_encode_host_static")


def mask_tensor(mask_u32, device="cuda") -> torch.Tensor:
    """numpy uint32 [G] -> int32 tensor with the same bit patterns on `device`."""
    import numpy as np

    return torch.from_numpy(np.ascontiguousarray(mask_u32, dtype=np.uint32).view(np.int32).copy()).to(device)
