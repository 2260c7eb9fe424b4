"""Scatter / gather entry points: every worker's batch is a buffer of its own (Section 2's architecture: coded
query i goes to worker i, its prediction comes back from it).  On one GPU the W buffers are separate allocations;
the encoder's scattered rows, the decoder's and the locator's gathered reads are checked against the oracle and
against the strided entry points on the same values (bit for bit)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2109_09868_b200 as ap

pytestmark = pytest.mark.gpu


def dev():
    return torch.device("cuda:0")


@pytest.mark.parametrize("K,W,G,D,pad", [(8, 12, 50, 3072, 0), (4, 5, 33, 784, 0), (3, 7, 9, 1001, 0), (12, 20, 3, 4096, 64), (5, 9, 21, 13, 3)])
def test_encode_scatter_writes_every_worker_batch(K, W, G, D, pad):
    g = torch.Generator().manual_seed(D)
    X = torch.rand((G, K, D), generator=g)
    p = ap.make_params(K, W)
    # one allocation per worker, each with its own guard band; `pad` extra floats between the groups of a batch
    bufs = [torch.full((G, D + pad + 8), -7.0, device=dev()) for _ in range(W)]
    rows = [b[:, :D] for b in bufs]
    ap.approxifer_encode_scatter(p, X.to(dev()), rows)
    ref = ap.approxifer_encode(p, X.to(dev()))
    want = oracle.encode(K, W, X.numpy())
    for i in range(W):
        got = rows[i].cpu()
        assert torch.equal(got, ref[:, i].cpu())
        assert np.abs(got.numpy() - want[:, i]).max() <= 1e-5
        assert bool((bufs[i][:, D:] == -7.0).all())


@pytest.mark.parametrize("K,W,G,C", [(8, 12, 200, 10), (16, 24, 40, 1000), (3, 7, 30, 9), (12, 20, 25, 36)])
def test_decode_gather_reads_every_present_worker_batch(K, W, G, C):
    rng = np.random.default_rng(C)
    Yt = torch.randn((G, W, C), generator=torch.Generator().manual_seed(C))
    mask = rng.integers(0, 2**W, size=G, dtype=np.uint64).astype(np.uint32)
    mask[0], mask[1] = 0, 2**W - 1
    rows = []
    for i in range(W):
        b = Yt[:, i].clone()
        absent = ((mask >> np.uint32(i)) & 1) == 0
        b[torch.from_numpy(absent)] = float("nan")  # an absent worker's batch entry is never read
        rows.append(b.to(dev()))
    p = ap.make_params(K, W)
    n_used = torch.empty(G, dtype=torch.int32, device=dev())
    status = torch.empty(G, dtype=torch.int32, device=dev())
    Yh = ap.approxifer_decode_gather(p, rows, ap.mask_tensor(mask), n_used=n_used, status=status)
    want, n_ref, st_ref = oracle.decode(K, W, Yt.numpy(), mask)
    got = Yh.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    err = np.abs(got - want).reshape(G, -1).max(axis=1)
    assert np.all(err <= 1e-4 * np.maximum(np.abs(want).reshape(G, -1).max(axis=1), 1e-30))
    np.testing.assert_array_equal(n_used.cpu().numpy(), n_ref)
    np.testing.assert_array_equal(status.cpu().numpy().view(np.uint32), st_ref)
    ref = ap.approxifer_decode(p, Yt.to(dev()), ap.mask_tensor(mask), tuning=ap.decode_tuning(kernel=1))
    assert torch.equal(Yh.view(torch.int32), ref.view(torch.int32))


def test_decode_gather_beyond_the_cache_takes_the_packed_groups_kernel():
    """80,000 groups of the paper's decode shape, one buffer per worker (38 MB in all): the automatic choice is the
    packed-groups kernel reading each worker's rows through the offset table.  Bit-equal to the per-column kernel on
    the same values stored group-major; a sample against the oracle."""
    K, W, C, G = 8, 12, 10, 80000
    rng = np.random.default_rng(11)
    Yt = torch.randn((G, W, C), generator=torch.Generator().manual_seed(17))
    mask = rng.integers(0, 2**W, size=G, dtype=np.uint64).astype(np.uint32)
    mask[0], mask[1] = 0, 2**W - 1
    rows = [Yt[:, i].clone().to(dev()) for i in range(W)]
    p = ap.make_params(K, W)
    n_used = torch.empty(G, dtype=torch.int32, device=dev())
    status = torch.empty(G, dtype=torch.int32, device=dev())
    launches = ap.launch_count()
    Yh = ap.approxifer_decode_gather(p, rows, ap.mask_tensor(mask), n_used=n_used, status=status)
    assert ap.launch_count() == launches + 1
    ref = ap.approxifer_decode(p, Yt.to(dev()), ap.mask_tensor(mask), tuning=ap.decode_tuning(kernel=1))
    assert torch.equal(Yh.view(torch.int32), ref.view(torch.int32))
    n = 3000
    want, n_ref, st_ref = oracle.decode(K, W, Yt[:n].numpy(), mask[:n])
    got = Yh[:n].cpu().numpy().astype(np.float64)
    scale = np.maximum(np.abs(want).reshape(n, -1).max(axis=1), 1e-30)
    ok = np.isfinite(want).reshape(n, -1).all(axis=1)
    err = np.abs(got - want).reshape(n, -1).max(axis=1)
    assert np.all(err[ok] <= 1e-4 * scale[ok])
    np.testing.assert_array_equal(n_used[:n].cpu().numpy(), n_ref)
    np.testing.assert_array_equal(status[:n].cpu().numpy().view(np.uint32), st_ref)
    assert ap.device_wait_timeouts() == 0


@pytest.mark.parametrize("K,E,S,W,C", [(8, 2, 2, 24, 10), (4, 1, 1, 12, 37), (13, 3, 0, 32, 10)])
def test_locate_gather_finds_the_same_workers(K, E, S, W, C):
    G = 120
    rng = np.random.default_rng(K + C)
    X = rng.random((G, K, 16), dtype=np.float32)
    Y = (oracle.encode(K, W, X) @ rng.standard_normal((16, C))).astype(np.float32)
    mask = np.empty(G, dtype=np.uint32)
    for g in range(G):
        present = np.sort(rng.choice(W, size=W - S, replace=False))
        mask[g] = sum(1 << int(i) for i in present)
        Y[g, rng.choice(present, size=E, replace=False)] += (10 * rng.standard_normal((E, C))).astype(np.float32)
    rows = [torch.from_numpy(np.ascontiguousarray(Y[:, i])).to(dev()) for i in range(W)]
    p = ap.make_params(K, W, E)
    adv, trusted = ap.approxifer_locate_gather(p, rows, ap.mask_tensor(mask))
    adv2, trusted2 = ap.approxifer_locate(p, torch.from_numpy(Y).to(dev()), ap.mask_tensor(mask))
    assert torch.equal(adv, adv2) and torch.equal(trusted, trusted2)
    ref = oracle.locate(K, W, E, Y, mask)
    np.testing.assert_array_equal(adv.cpu().numpy(), ref["adv"])


def test_scatter_gather_argument_errors():
    import ctypes
    lib = ap.load()
    p = ap.make_params(4, 5)
    bufs = [torch.zeros((2, 8), device=dev()) for _ in range(5)]
    arr = (ctypes.c_void_p * 5)(*[b.data_ptr() for b in bufs])
    X = torch.zeros((2, 4, 8), device=dev())
    assert lib.approxifer_encode_scatter(ctypes.byref(p), 2, 8, X.data_ptr(), 32, 8, arr, 4, None) == ap.binding.E_RANGE  # batches overlap
    arr[3] = None
    assert lib.approxifer_encode_scatter(ctypes.byref(p), 2, 8, X.data_ptr(), 32, 8, arr, 8, None) == ap.binding.E_NULL
