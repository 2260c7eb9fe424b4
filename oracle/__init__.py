"""ctypes front end of the fp64 CPU oracle (``approxifer_oracle.c``).

TEST INFRASTRUCTURE ONLY.  The oracle restates ApproxIFER's encoder, decoder
and error locator (arXiv 2109.09868, Section 3, Algorithm 2) in plain C and
fp64.  Only the tests, the smoke check and the benchmark's CPU-baseline leg may
import this package; the product never does, and the two share no code.

The shared object is compiled on first use with ``gcc -O2 -fopenmp`` (no
fast-math) next to the source.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from ctypes import POINTER, c_double, c_float, c_int, c_int32, c_int64, c_uint32

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "approxifer_oracle.c")
_SRC_BF16 = os.path.join(_HERE, "bf16_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

ST_NO_WORKERS = 1
ST_FEW_WORKERS = 2
ST_LOCATE_UNDERDETERMINED = 4
ST_NONFINITE = 8
ST_ORACLE_RANK_DEFICIENT = 0x100

FLAG_SIGN_WORKER_INDEX = 1


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than the source."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_SRC_BF16))
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, _SRC_BF16, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    pd, pf, pi, pu = POINTER(c_double), POINTER(c_float), POINTER(c_int32), POINTER(c_uint32)
    lib.oracle_set_threads.argtypes = [c_int]
    lib.oracle_get_threads.restype = c_int
    lib.oracle_alpha.argtypes = [c_int, pd]
    lib.oracle_beta.argtypes = [c_int, pd]
    lib.oracle_coincident.argtypes = [c_int, c_int, c_int, c_int]
    lib.oracle_coincident.restype = c_int
    lib.oracle_berrut.argtypes = [c_int, pd, pd, c_double]
    lib.oracle_berrut.restype = c_double
    lib.oracle_encode_weights.argtypes = [c_int, c_int, pd]
    lib.oracle_encode.argtypes = [c_int, c_int, c_int64, c_int64, pf, c_int64, c_int64, pd, c_int64, c_int64]
    lib.oracle_compact.argtypes = [c_int, c_uint32, pi]
    lib.oracle_compact.restype = c_int
    lib.oracle_decode_weights.argtypes = [c_int, c_int, c_uint32, c_uint32, pd, pi]
    lib.oracle_decode_weights.restype = c_int
    lib.oracle_decode.argtypes = [c_int, c_int, c_uint32, c_int64, c_int64, pf, c_int64, c_int64, pu,
                                  pd, c_int64, c_int64, pi, pu]
    lib.oracle_locate_class.argtypes = [c_int, c_int, pd, pd, pd, pd]
    lib.oracle_locate_class.restype = c_int
    lib.oracle_locate.argtypes = [c_int, c_int, c_int, c_int64, c_int64, pf, c_int64, c_int64, pu,
                                  pi, pu, pu, pd, pi]
    pu16 = POINTER(ctypes.c_uint16)
    lib.oracle_bf16_to_double.argtypes = [ctypes.c_uint16]
    lib.oracle_bf16_to_double.restype = c_double
    lib.oracle_double_to_bf16.argtypes = [c_double]
    lib.oracle_double_to_bf16.restype = ctypes.c_uint16
    lib.oracle_bf16_widen.argtypes = [c_int64, pu16, pf]
    lib.oracle_bf16_round.argtypes = [c_int64, pd, pu16]
    _lib = lib
    return lib


def _p(a, ct):
    return a.ctypes.data_as(POINTER(ct))


def _check_kw(K, W):
    if not (1 <= K <= 32 and 2 <= W <= 32):
        raise ValueError("oracle: need 1 <= K <= 32 and 2 <= W <= 32")


def _payload(a, rows):
    """Validate a [G][rows][L] float32 array whose last dimension is contiguous;
    return (array, group stride, row stride) in elements."""
    a = np.asarray(a)
    if a.dtype != np.float32 or a.ndim != 3 or a.shape[1] != rows:
        raise ValueError("oracle: expected float32 [G][%d][L]" % rows)
    if a.shape[2] > 1 and a.strides[2] != 4:
        a = np.ascontiguousarray(a)
    if a.strides[0] % 4 or a.strides[1] % 4:
        a = np.ascontiguousarray(a)
    return a, a.strides[0] // 4, a.strides[1] // 4


def set_threads(n: int) -> None:
    _load().oracle_set_threads(int(n))


def get_threads() -> int:
    return int(_load().oracle_get_threads())


def alpha(K: int) -> np.ndarray:
    """Chebyshev points of the first kind, alpha_j = cos((2j+1)pi/(2K))."""
    out = np.empty(K, dtype=np.float64)
    _load().oracle_alpha(K, _p(out, c_double))
    return out


def beta(W: int) -> np.ndarray:
    """Chebyshev points of the second kind, beta_i = cos(i pi/(W-1))."""
    if W < 2:
        raise ValueError("oracle: W >= 2")
    out = np.empty(W, dtype=np.float64)
    _load().oracle_beta(W, _p(out, c_double))
    return out


def coincident(K: int, W: int, j: int, i: int) -> bool:
    return bool(_load().oracle_coincident(K, W, j, i))


def berrut(nodes, values, z: float) -> float:
    """Berrut's rational interpolant (Eq. 1-2) through (nodes, values) at z."""
    x = np.ascontiguousarray(nodes, dtype=np.float64)
    f = np.ascontiguousarray(values, dtype=np.float64)
    return float(_load().oracle_berrut(len(x), _p(x, c_double), _p(f, c_double), float(z)))


def encode_weights(K: int, W: int) -> np.ndarray:
    """[W][K] matrix l_j(beta_i)."""
    _check_kw(K, W)
    e = np.empty((W, K), dtype=np.float64)
    _load().oracle_encode_weights(K, W, _p(e, c_double))
    return e


def encode(K: int, W: int, X) -> np.ndarray:
    """X float32 [G][K][D] -> coded queries float64 [G][W][D]."""
    _check_kw(K, W)
    X, gs, rs = _payload(X, K)
    G, _, D = X.shape
    out = np.empty((G, W, D), dtype=np.float64)
    _load().oracle_encode(K, W, G, D, _p(X, c_float), gs, rs, _p(out, c_double), W * D, D)
    return out


def compact(W: int, mask: int) -> list:
    F = np.empty(32, dtype=np.int32)
    n = _load().oracle_compact(W, int(mask) & 0xFFFFFFFF, _p(F, c_int32))
    return [int(v) for v in F[:n]]


def decode_weights(K: int, W: int, mask: int, flags: int = 0):
    """Returns (w [K][n] float64, F list of the n workers used, ascending)."""
    _check_kw(K, W)
    w = np.zeros((K, W), dtype=np.float64)
    F = np.empty(32, dtype=np.int32)
    n = _load().oracle_decode_weights(K, W, flags, int(mask) & 0xFFFFFFFF, _p(w, c_double), _p(F, c_int32))
    return w[:, :n].copy(), [int(v) for v in F[:n]]


def decode(K: int, W: int, Yt, mask, flags: int = 0):
    """Yt float32 [G][W][C], mask uint32 [G] -> (Yhat float64 [G][K][C], n_used, status)."""
    _check_kw(K, W)
    Yt, gs, rs = _payload(Yt, W)
    G, _, C = Yt.shape
    mask = np.ascontiguousarray(mask, dtype=np.uint32)
    assert mask.shape == (G,)
    out = np.empty((G, K, C), dtype=np.float64)
    n_used = np.empty(G, dtype=np.int32)
    status = np.empty(G, dtype=np.uint32)
    _load().oracle_decode(K, W, flags, G, C, _p(Yt, c_float), gs, rs, _p(mask, c_uint32),
                          _p(out, c_double), K * C, C, _p(n_used, c_int32), _p(status, c_uint32))
    return out, n_used, status


def locate_class(m: int, xs, y):
    """Steps 1-3 of Algorithm 2 for one class: returns (x, a, rank), x = (P_0..P_{m-1}, Q_1..Q_{m-1})."""
    xs = np.ascontiguousarray(xs, dtype=np.float64)
    y = np.ascontiguousarray(y, dtype=np.float64)
    n = len(xs)
    assert len(y) == n and n <= 32 and 2 * m - 1 <= 63
    x = np.empty(2 * m - 1, dtype=np.float64)
    a = np.empty(n, dtype=np.float64)
    rank = _load().oracle_locate_class(n, m, _p(xs, c_double), _p(y, c_double), _p(x, c_double), _p(a, c_double))
    return x, a, int(rank)


def locate(K: int, W: int, E: int, Yt, mask):
    """Algorithm 2.  Returns dict(adv [G][E] int32, trusted uint32 [G], status, min_gap, vote_margin)."""
    _check_kw(K, W)
    if E < 0:
        raise ValueError("oracle: E >= 0")
    Yt, gs, rs = _payload(Yt, W)
    G, _, C = Yt.shape
    mask = np.ascontiguousarray(mask, dtype=np.uint32)
    assert mask.shape == (G,)
    adv = np.empty((G, max(E, 0)), dtype=np.int32)
    trusted = np.empty(G, dtype=np.uint32)
    status = np.empty(G, dtype=np.uint32)
    gap = np.empty(G, dtype=np.float64)
    margin = np.empty(G, dtype=np.int32)
    _load().oracle_locate(K, W, E, G, C, _p(Yt, c_float), gs, rs, _p(mask, c_uint32), _p(adv, c_int32),
                          _p(trusted, c_uint32), _p(status, c_uint32), _p(gap, c_double), _p(margin, c_int32))
    return dict(adv=adv, trusted=trusted, status=status, min_gap=gap, vote_margin=margin)


# ---- bfloat16 storage (bf16_oracle.c): exact widening, the fp64 formulas above, one rounding to nearest-even ----

def bf16_to_double(bits: int) -> float:
    return float(_load().oracle_bf16_to_double(int(bits) & 0xFFFF))


def double_to_bf16(x: float) -> int:
    return int(_load().oracle_double_to_bf16(float(x)))


def bf16_widen(bits) -> np.ndarray:
    """uint16 bfloat16 bit patterns -> the float32 array of the same values (exact)."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(b.shape, dtype=np.float32)
    _load().oracle_bf16_widen(b.size, _p(b, ctypes.c_uint16), _p(out, c_float))
    return out


def bf16_round(x) -> np.ndarray:
    """float64 array -> uint16 bit patterns of the nearest bfloat16 (ties to even)."""
    a = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(a.shape, dtype=np.uint16)
    _load().oracle_bf16_round(a.size, _p(a, c_double), _p(out, ctypes.c_uint16))
    return out


def encode_bf16(K: int, W: int, X_bits):
    """Encoder on bfloat16 queries [G][K][D] (uint16 bit patterns): (exact fp64 coded queries, their bfloat16 roundings)."""
    exact = encode(K, W, bf16_widen(X_bits))
    return exact, bf16_round(exact)


def decode_bf16(K: int, W: int, Yt_bits, mask, flags: int = 0):
    """Decoder on bfloat16 predictions [G][W][C]: (exact fp64 result, its bfloat16 rounding, n_used, status)."""
    exact, n_used, status = decode(K, W, bf16_widen(Yt_bits), mask, flags)
    return exact, bf16_round(exact), n_used, status
