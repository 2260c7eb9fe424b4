"""Host-side checks of the C ABI that need no GPU: the library loads, exports
every symbol the header declares, and rejects bad arguments before touching
the device."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2109_09868_b200 as ap
from paper_2109_09868_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "approxifer.h")


def _declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(approxifer_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ap.load()
    names = _declared_symbols()
    assert set(binding.EXPORTS) <= set(names)
    assert len(names) >= 7
    for name in names:
        assert getattr(lib, name) is not None, name


def test_version_and_strerror():
    assert ap.version() == 100
    for code in (0, -1, -2, -3, -4, -5, -6):
        assert ap.strerror(code) and "unknown error" not in ap.strerror(code)
    assert "unknown error" in ap.strerror(-99)


def _encode_rc(K, W, G, D, x=1, xt=1, xr=None, orr=None, flags=0):
    p = ap.make_params(K, W, 0, flags)
    xr = D if xr is None else xr
    orr = D if orr is None else orr
    return ap.load().approxifer_encode(ctypes.byref(p), G, D, x, K * xr, xr, xt, W * orr, orr, None)


def test_encode_argument_errors_are_reported_on_the_host():
    assert _encode_rc(0, 5, 1, 8) == binding.E_RANGE
    assert _encode_rc(33, 5, 1, 8) == binding.E_RANGE
    assert _encode_rc(4, 1, 1, 8) == binding.E_RANGE
    assert _encode_rc(4, 33, 1, 8) == binding.E_RANGE
    assert _encode_rc(4, 5, -1, 8) == binding.E_RANGE
    assert _encode_rc(4, 5, 1, 0) == binding.E_RANGE
    assert _encode_rc(4, 5, 1, 2**31 + 4) == binding.E_RANGE
    assert _encode_rc(4, 5, 1, 8, xr=7) == binding.E_RANGE
    assert _encode_rc(4, 5, 1, 8, orr=4) == binding.E_RANGE
    assert _encode_rc(4, 5, 1, 8, x=None) == binding.E_NULL
    assert _encode_rc(4, 5, 1, 8, xt=None) == binding.E_NULL
    assert _encode_rc(4, 5, 1, 8, flags=16) == binding.E_PARAM  # unknown flag bit
    assert _encode_rc(4, 5, 0, 8, x=None, xt=None) == binding.OK  # G = 0: valid no-op
    assert ap.load().approxifer_encode(None, 1, 8, 1, 32, 8, 1, 40, 8, None) == binding.E_NULL


def test_decode_and_locate_argument_errors():
    lib = ap.load()
    p = ap.make_params(4, 5)
    assert lib.approxifer_decode(ctypes.byref(p), 1, 10, 1, 50, 10, None, 1, 40, 10, None, None, None) == binding.E_NULL
    assert lib.approxifer_decode(ctypes.byref(p), 1, 10, 1, 50, 9, 1, 1, 40, 10, None, None, None) == binding.E_RANGE
    assert lib.approxifer_decode(ctypes.byref(p), 0, 10, None, 50, 10, None, None, 40, 10, None, None, None) == binding.OK
    for (K, W, E, want) in [(8, 24, 2, binding.OK), (8, 19, 2, binding.E_PARAM), (8, 24, 0, binding.E_PARAM),
                            (8, 24, -1, binding.E_RANGE), (12, 24, 1, binding.E_PARAM)]:
        q = ap.make_params(K, W, E)
        rc = lib.approxifer_locate(ctypes.byref(q), 0, 10, None, W * 10, 10, None, None, None, None, None)
        assert rc == want, (K, W, E)
    q = ap.make_params(8, 24, 2)
    assert lib.approxifer_locate(ctypes.byref(q), 1, 10, 1, 240, 10, 1, None, 1, None, None) == binding.E_NULL
    # the homogeneous form of the locator exists for K+E <= 13
    for (K, W, E, want) in [(8, 24, 2, binding.OK), (9, 32, 2, binding.OK), (12, 32, 1, binding.OK), (12, 32, 2, binding.E_PARAM)]:
        q = ap.make_params(K, W, E, binding.LOCATE_HOMOGENEOUS)
        assert lib.approxifer_locate(ctypes.byref(q), 0, 10, None, W * 10, 10, None, None, None, None, None) == want


def test_flags_each_entry_point_ignores_or_rejects():
    """One params struct serves the whole pipeline: the decoder's sign flag and the locator's homogeneous flag
    are accepted (and ignored) by the entry points they do not concern; undefined bits are rejected everywhere."""
    lib = ap.load()
    both = binding.SIGN_WORKER_INDEX | binding.LOCATE_HOMOGENEOUS
    q = ap.make_params(8, 24, 2, both)
    bad = ap.make_params(8, 24, 2, 16)
    assert lib.approxifer_encode(ctypes.byref(q), 0, 8, None, 64, 8, None, 192, 8, None) == binding.OK
    assert lib.approxifer_encode(ctypes.byref(bad), 0, 8, None, 64, 8, None, 192, 8, None) == binding.E_PARAM
    assert lib.approxifer_decode(ctypes.byref(q), 0, 10, None, 240, 10, None, None, 80, 10, None, None, None) == binding.OK
    assert lib.approxifer_decode(ctypes.byref(bad), 0, 10, None, 240, 10, None, None, 80, 10, None, None, None) == binding.E_PARAM
    assert lib.approxifer_locate(ctypes.byref(q), 0, 10, None, 240, 10, None, None, None, None, None) == binding.OK
    assert lib.approxifer_locate(ctypes.byref(bad), 0, 10, None, 240, 10, None, None, None, None, None) == binding.E_PARAM
    assert lib.approxifer_decode_rational(ctypes.byref(q), 0, 10, None, 240, 10, None, None, 80, 10, None, None) == binding.OK
    assert lib.approxifer_decode_rational(ctypes.byref(bad), 0, 10, None, 240, 10, None, None, 80, 10, None, None) == binding.E_PARAM
    assert lib.approxifer_encode_host_static(ctypes.byref(q), 0, 8, None, None, None) == binding.OK
    assert lib.approxifer_encode_host_static(ctypes.byref(bad), 0, 8, None, None, None) == binding.E_PARAM


def test_debug_entry_points_validate_their_tuning_on_the_host():
    lib = ap.load()
    p = ap.make_params(8, 12)
    for (fields, want) in [((0, 0, 0, 0, 0), binding.OK), ((1, 0, 0, 0, 0), binding.OK), ((5, 0, 0, 0, 0), binding.E_PARAM), ((4, 0, 0, 7, 0), binding.OK),
                           ((0, 1, 0, 0, 0), binding.E_PARAM), ((0, 0, -1, 0, 0), binding.E_PARAM), ((0, 0, 0, 48, 0), binding.E_PARAM),
                           ((0, 0, 0, 0, 3), binding.E_PARAM), ((0, 4, 2, 256, 2), binding.OK)]:
        t = binding.approxifer_decode_tuning(*fields, 0, 0)
        rc = lib.approxifer_debug_decode(ctypes.byref(p), 0, 64, None, 768, 64, None, None, 512, 64, None, None, ctypes.byref(t), None)
        assert rc == want, fields
    assert lib.approxifer_debug_decode(ctypes.byref(p), 0, 64, None, 768, 64, None, None, 512, 64, None, None, None, None) == binding.OK
    # a poll limit too short for started copies to land, or a negative group, is refused
    for (limit, withhold, want) in [(65536, 5, binding.OK), (1000, 0, binding.E_PARAM), (0, -1, binding.E_PARAM)]:
        t = binding.approxifer_decode_tuning(0, 0, 0, 0, 0, limit, withhold)
        rc = lib.approxifer_debug_decode(ctypes.byref(p), 0, 64, None, 768, 64, None, None, 512, 64, None, None, ctypes.byref(t), None)
        assert rc == want, (limit, withhold)
    q = ap.make_params(8, 24, 2)
    assert lib.approxifer_debug_locate(ctypes.byref(q), 0, 10, None, 240, 10, None, None, None, None, 1, None) == binding.OK
    q = ap.make_params(8, 19, 2)
    assert lib.approxifer_debug_locate(ctypes.byref(q), 0, 10, None, 240, 10, None, None, None, None, 1, None) == binding.E_PARAM


def test_static_workspace_size_check_cannot_wrap():
    """Group counts whose byte count overflows 64 bits are refused as too large before anything is enqueued."""
    lib = ap.load()
    p = ap.make_params(8, 12)
    for G in (1 << 57, 1 << 60, (1 << 63) - 1):
        assert lib.approxifer_encode_host_static(ctypes.byref(p), G, 3072, 1, 1, None) == binding.E_TOO_LARGE
    assert lib.approxifer_encode_host_static(ctypes.byref(p), 1, 1 << 31, 1, 1, None) == binding.E_TOO_LARGE


def test_binding_refuses_cpu_tensors():
    import torch

    p = ap.make_params(4, 5)
    with pytest.raises(ValueError):
        ap.approxifer_encode(p, torch.zeros(1, 4, 8))


def test_workload_generators_are_seeded_and_shaped():
    from paper_2109_09868_b200 import workloads as wl

    for cfg in range(1, 6):
        w = wl.workload(cfg, G=64)
        m1, m2 = wl.masks(w), wl.masks(w)
        np.testing.assert_array_equal(m1, m2)
        assert m1.dtype == np.uint32 and m1.shape == (64,)
        pop = np.array([bin(int(v)).count("1") for v in m1])
        assert np.all(m1 < 2**w.W)
        if cfg == 1:
            assert np.all(pop == 4)
        elif cfg == 2:
            assert pop.min() >= 8 and pop.max() <= 12
        elif cfg == 3:
            assert pop.min() >= 12 and pop.max() <= 20
        elif cfg == 4:
            assert pop.min() >= 16 and pop.max() <= 24
        else:
            assert np.all(pop == 22)
            adv = wl.adversaries(w, m1)
            assert adv.shape == (64, 2) and np.all(adv[:, 0] < adv[:, 1])
            assert np.all((m1[:, None] >> adv.astype(np.uint32)) & 1 == 1)
    w = wl.workload(2, G=3)
    x1, x2 = wl.queries(w), wl.queries(w)
    assert x1.shape == (3, 8, 3072) and bool((x1 == x2).all()) and float(x1.min()) >= 0.0 and float(x1.max()) < 1.0
