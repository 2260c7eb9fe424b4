"""Host-buffer entry points (approxifer_*_host): results must equal the
device-pointer entry points bit for bit (same kernels, only the staging
differs), for any workspace size, stream count and payload length."""
import numpy as np
import pytest
import torch

import oracle
import paper_2109_09868_b200 as ap
from paper_2109_09868_b200 import binding

pytestmark = pytest.mark.gpu


def dev():
    return torch.device("cuda:0")


def sync(streams):
    for s in streams:
        s.synchronize()


@pytest.mark.parametrize("K,W,G,D,ws_mb,ns", [(8, 12, 300, 3072, 8, 3), (4, 5, 256, 784, 64, 2), (3, 7, 41, 1001, 1, 1),
                                              (12, 20, 3, 150528, 64, 4), (5, 9, 1000, 6, 1, 8)])
def test_encode_host_equals_device_entry_point(K, W, G, D, ws_mb, ns):
    g = torch.Generator().manual_seed(D)
    hX = torch.rand((G, K, D), generator=g).pin_memory()
    hXt = torch.empty((G, W, D)).pin_memory()
    ws = torch.empty(ws_mb << 20, dtype=torch.uint8, device=dev())
    streams = [torch.cuda.Stream() for _ in range(ns)]
    p = ap.make_params(K, W)
    ap.approxifer_encode_host(p, hX, hXt, ws, streams)
    sync(streams)
    ref = ap.approxifer_encode(p, hX.to(dev())).cpu()
    assert torch.equal(hXt, ref)
    assert np.abs(hXt.numpy() - oracle.encode(K, W, hX.numpy())).max() <= 1e-5


@pytest.mark.parametrize("K,W,G,C,ws_mb,ns", [(8, 12, 3000, 10, 1, 3), (16, 24, 200, 1000, 16, 2), (12, 20, 9, 1001, 2, 1)])
def test_decode_host_equals_device_entry_point(K, W, G, C, ws_mb, ns):
    rng = np.random.default_rng(C)
    hYt = torch.randn((G, W, C), generator=torch.Generator().manual_seed(C)).pin_memory()
    mask = rng.integers(0, 2**W, size=G, dtype=np.uint64).astype(np.uint32)
    mask[0] = 0
    hmask = torch.from_numpy(mask.view(np.int32).copy()).pin_memory()
    hYh = torch.empty((G, K, C)).pin_memory()
    hn = torch.empty(G, dtype=torch.int32).pin_memory()
    hst = torch.empty(G, dtype=torch.int32).pin_memory()
    ws = torch.empty(ws_mb << 20, dtype=torch.uint8, device=dev())
    streams = [torch.cuda.Stream() for _ in range(ns)]
    p = ap.make_params(K, W)
    ap.approxifer_decode_host(p, hYt, hmask, hYh, ws, streams, hn_used=hn, hstatus=hst)
    sync(streams)
    n_used = torch.empty(G, dtype=torch.int32, device=dev())
    status = torch.empty(G, dtype=torch.int32, device=dev())
    ref = ap.approxifer_decode(p, hYt.to(dev()), hmask.to(dev()), n_used=n_used, status=status).cpu()
    assert torch.equal(hYh, ref)
    assert torch.equal(hn, n_used.cpu()) and torch.equal(hst, status.cpu())
    # and against the fp64 checker, per group, at the decoder's tolerance
    want, n_ref, st_ref = oracle.decode(K, W, hYt.numpy(), mask)
    err = np.abs(hYh.numpy().astype(np.float64) - want).reshape(G, -1).max(axis=1)
    scale = np.abs(want).reshape(G, -1).max(axis=1)
    assert np.all(err <= 1e-4 * np.maximum(scale, 1e-30) + (scale == 0) * 0.0), float((err / np.maximum(scale, 1e-30)).max())
    np.testing.assert_array_equal(hn.numpy(), n_ref)
    np.testing.assert_array_equal(hst.numpy().view(np.uint32), st_ref)


def test_locate_host_equals_device_entry_point():
    K, W, E, G, C = 8, 24, 2, 500, 10
    rng = np.random.default_rng(1)
    X = rng.random((G, K, 16), dtype=np.float32)
    Y = (oracle.encode(K, W, X) @ rng.standard_normal((16, C))).astype(np.float32)
    mask = np.full(G, 2**W - 1, dtype=np.uint32)
    for g in range(G):
        Y[g, rng.choice(W, size=E, replace=False)] += 10 * rng.standard_normal((E, C)).astype(np.float32)
    hYt = torch.from_numpy(Y).pin_memory()
    hmask = torch.from_numpy(mask.view(np.int32).copy()).pin_memory()
    hadv = torch.empty((G, E), dtype=torch.int32).pin_memory()
    htr = torch.empty(G, dtype=torch.int32).pin_memory()
    hst = torch.empty(G, dtype=torch.int32).pin_memory()
    ws = torch.empty(1 << 20, dtype=torch.uint8, device=dev())
    streams = [torch.cuda.Stream() for _ in range(2)]
    p = ap.make_params(K, W, E)
    ap.approxifer_locate_host(p, hYt, hmask, hadv, htr, ws, streams, hstatus=hst)
    sync(streams)
    adv, trusted = ap.approxifer_locate(p, hYt.to(dev()), hmask.to(dev()))
    assert torch.equal(hadv, adv.cpu()) and torch.equal(htr, trusted.cpu())
    ref = oracle.locate(K, W, E, Y, mask)
    np.testing.assert_array_equal(hadv.numpy(), ref["adv"])


def test_host_entry_points_report_a_workspace_that_is_too_small():
    K, W, G, D = 8, 12, 4, 3072
    hX = torch.rand((G, K, D)).pin_memory()
    hXt = torch.empty((G, W, D)).pin_memory()
    ws = torch.empty(100_000, dtype=torch.uint8, device=dev())  # one group needs (8+12)*3072*4 = 245,760 bytes
    with pytest.raises(ap.ApproxiferError) as e:
        ap.approxifer_encode_host(ap.make_params(K, W), hX, hXt, ws, [torch.cuda.Stream()])
    assert e.value.code == binding.E_WORKSPACE
