"""approxifer_encode_host_static: the encoder for callers that cannot allocate
device memory (a front-end beside a model server that owns all device memory,
or a request path where cudaMalloc's device-wide lock and synchronisation are
not acceptable).  Its staging area is a fixed array inside the library.

The test calls it through the C ABI twice in a row, with different batches,
and compares each result with approxifer_encode (the device-pointer entry
point) on the same queries, and with the fp64 CPU checker, within the encoder
tolerance used by the other GPU tests.  The second call finds the first
call's bytes in the shared array, so it also shows that nothing stale leaks
into a result.  It also holds the entry point to its contract: a call leaves
the amount of free device memory as it found it and launches exactly one
kernel.  The file name makes pytest collect it last.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2109_09868_b200 as ap
from paper_2109_09868_b200 import binding

pytestmark = pytest.mark.gpu

ENC_TOL = 1e-5


def _encode_both_ways(K, W, G, D, seed, stream):
    g = torch.Generator().manual_seed(seed)
    hX = (torch.rand((G, K, D), generator=g) * 4 - 1).pin_memory()
    hXt = torch.full((G, W, D), float("nan")).pin_memory()
    p = ap.make_params(K, W)
    # straight through the C ABI: host pointers in, no workspace argument
    rc = ap.load().approxifer_encode_host_static(ctypes.byref(p), G, D, hX.data_ptr(), hXt.data_ptr(),
                                                 int(stream.cuda_stream))
    assert rc == binding.OK, ap.strerror(rc)
    stream.synchronize()
    ref = ap.approxifer_encode(p, hX.to("cuda:0")).cpu()
    torch.cuda.synchronize()
    err = float((hXt - ref).abs().max())
    assert err <= ENC_TOL * float(hX.abs().max()), err
    err64 = float(np.abs(hXt.numpy().astype(np.float64) - oracle.encode(K, W, hX.numpy())).max())
    assert err64 <= ENC_TOL * float(hX.abs().max()), err64
    return err


def test_static_workspace_encoder_matches_encode_on_two_calls_in_a_row():
    stream = torch.cuda.Stream()
    # a larger batch first (24 MB of staging), then a smaller, differently shaped one that reuses its bytes
    _encode_both_ways(8, 12, 100, 3072, seed=1, stream=stream)
    _encode_both_ways(3, 7, 37, 1001, seed=2, stream=stream)
    # and once more with the first shape: same answer as a fresh computation
    _encode_both_ways(8, 12, 100, 3072, seed=3, stream=stream)


def test_static_workspace_encoder_allocates_nothing_and_launches_one_kernel():
    K, W, G, D = 8, 12, 64, 3072
    p = ap.make_params(K, W)
    hX = torch.rand((G, K, D)).pin_memory()
    hXt = torch.empty((G, W, D)).pin_memory()
    stream = torch.cuda.Stream()

    def call():
        rc = ap.load().approxifer_encode_host_static(ctypes.byref(p), G, D, hX.data_ptr(), hXt.data_ptr(), int(stream.cuda_stream))
        assert rc == binding.OK, ap.strerror(rc)
        stream.synchronize()

    call()  # the first call on a device looks the array's address up
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    launches0 = ap.launch_count()
    call()
    assert ap.launch_count() == launches0 + 1
    assert torch.cuda.mem_get_info()[0] == free0


def test_static_workspace_encoder_rejects_batches_beyond_its_limit():
    p = ap.make_params(8, 12)
    G, D = 200, 3072  # 200 * 20 * 3072 * 4 = 49 MB > 32 MiB
    assert 4 * G * D * 20 > binding.STATIC_WORKSPACE_BYTES
    hX = torch.zeros((G, 8, D))
    hXt = torch.zeros((G, 12, D))
    rc = ap.load().approxifer_encode_host_static(ctypes.byref(p), G, D, hX.data_ptr(), hXt.data_ptr(), None)
    assert rc == binding.E_TOO_LARGE
    assert "staging area" in ap.strerror(rc)
    with pytest.raises(ap.ApproxiferError):
        ap.approxifer_encode_host_static(p, hX, hXt)
    # rows that are not whole 16-byte columns are padded in the staging area, and the limit counts the padding:
    # D = 1001 is staged as 1004 floats, so G = 417 fits (33,493,568 <= 33,554,432 bytes) as 4*G*D*(K+W) suggests,
    # while D = 1021 is staged as 1024 and G = 410 does not (33,587,200 bytes) although 4*G*D*(K+W) = 33,488,800 would
    for (G, D, want) in [(417, 1001, binding.OK), (410, 1021, binding.E_TOO_LARGE)]:
        assert 4 * G * D * 20 <= binding.STATIC_WORKSPACE_BYTES
        hX = torch.zeros((G, 8, D)).pin_memory()
        hXt = torch.zeros((G, 12, D)).pin_memory()
        rc = ap.load().approxifer_encode_host_static(ctypes.byref(p), G, D, hX.data_ptr(), hXt.data_ptr(), None)
        torch.cuda.synchronize()
        assert rc == want, (G, D, rc)
