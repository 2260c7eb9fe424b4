"""GPU parity at the full sizes of the five workloads, in the launch
configuration the benchmark times.

The oracle cannot evaluate 10^10 outputs, so each large tensor is checked on
(a) a seeded subset of groups compared element by element and (b) a strided
sample of columns of EVERY group (encode and decode are element-wise in the
payload dimension, so a column sample of a group is itself a valid small
problem for the oracle).  Integer results (n_used, status, located sets) are
compared for every group.  Coded predictions fed to the decoder / locator come
from the oracle's encoder, never from the CUDA path.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2109_09868_b200 as ap
from paper_2109_09868_b200 import workloads as wl

pytestmark = pytest.mark.gpu

ENC_TOL = 1e-5
DEC_TOL = 1e-4


def dev():
    return torch.device("cuda:0")


def need_gb(gb):
    free, _ = torch.cuda.mem_get_info()
    if free < gb * 1e9:
        pytest.skip("needs %.0f GB of free device memory, %.0f GB available" % (gb, free / 1e9))


def sample_columns(G, L, per_group, seed):
    """int64 [G][per_group]: distinct-ish column indices per group, covering head, tail and interior."""
    rng = np.random.default_rng(seed)
    cols = rng.integers(0, L, size=(G, per_group))
    cols[:, 0] = 0
    cols[:, 1] = L - 1
    cols[:, 2] = (np.arange(G) * 7919) % L
    return cols


def gather_cols(T, cols):
    """T [G][R][L] on the GPU, cols [G][s] -> float32 numpy [G][R][s]."""
    idx = torch.as_tensor(cols, device=T.device)[:, None, :].expand(-1, T.shape[1], -1)
    return torch.gather(T, 2, idx).cpu().numpy()


def check_encode_full(w, X, Xt, seed):
    K, W = w.K, w.W
    scale = 1.0  # queries are uniform on [0, 1)
    # (a) a subset of groups, every element
    rng = np.random.default_rng(seed)
    sub = np.unique(np.concatenate([[0, w.G - 1], rng.integers(0, w.G, size=min(30, w.G))]))
    ref = oracle.encode(K, W, X[sub].cpu().numpy())
    err_a = np.abs(Xt[sub].cpu().numpy() - ref).max()
    # (b) a column sample of every group
    cols = sample_columns(w.G, w.D, 8, seed + 1)
    ref_b = oracle.encode(K, W, gather_cols(X, cols))
    err_b = np.abs(gather_cols(Xt, cols) - ref_b).max()
    assert err_a <= ENC_TOL * scale and err_b <= ENC_TOL * scale, (err_a, err_b)
    return max(err_a, err_b)


def check_decode_full(w, Yt, mask_np, Yh, n_used, status, seed, sub_groups=256):
    K, W = w.K, w.W
    rng = np.random.default_rng(seed)
    sub = np.unique(np.concatenate([[0, w.G - 1], rng.integers(0, w.G, size=min(sub_groups, w.G))]))

    def rel(got, ref):
        g = got.shape[0]
        err = np.abs(got - ref).reshape(g, -1).max(axis=1)
        sc = np.abs(ref).reshape(g, -1).max(axis=1)
        ok = (err <= DEC_TOL * sc) | ((sc == 0) & (err == 0))
        assert ok.all(), (int((~ok).sum()), float(err[~ok].max()))
        return float((err / np.maximum(sc, 1e-30)).max())

    ref, n_ref, st_ref = oracle.decode(K, W, Yt[sub].cpu().numpy(), mask_np[sub])
    worst = rel(Yh[sub].cpu().numpy(), ref)
    cols = sample_columns(w.G, w.C, min(8, w.C), seed + 1)
    ref_b, n_all, st_all = oracle.decode(K, W, gather_cols(Yt, cols), mask_np)
    got_b = gather_cols(Yh, cols)
    err = np.abs(got_b - ref_b).reshape(w.G, -1).max(axis=1)
    sc = np.abs(ref_b).reshape(w.G, -1).max(axis=1)
    ok_b = (err <= DEC_TOL * sc) | ((sc == 0) & (err == 0))
    assert ok_b.all(), (int((~ok_b).sum()), float(err[~ok_b].max()))
    np.testing.assert_array_equal(n_used.cpu().numpy(), n_all)
    np.testing.assert_array_equal(status.cpu().numpy().view(np.uint32), st_all)
    return worst


def test_workload1_end_to_end():
    w = wl.workload(1)
    X = wl.queries(w, "cpu")
    p = ap.make_params(w.K, w.W)
    Xt = ap.approxifer_encode(p, X.to(dev()))
    ref = oracle.encode(w.K, w.W, X.numpy())
    assert np.abs(Xt.cpu().numpy() - ref).max() <= ENC_TOL
    Yt = wl.apply_model(w, torch.from_numpy(ref.astype(np.float32)))  # the oracle's coded queries
    mask = wl.masks(w)
    n_used = torch.empty(w.G, dtype=torch.int32, device=dev())
    status = torch.empty(w.G, dtype=torch.int32, device=dev())
    Yh = ap.approxifer_decode(p, Yt.to(dev()), ap.mask_tensor(mask), n_used=n_used, status=status)
    ref_h, n_ref, st_ref = oracle.decode(w.K, w.W, Yt.numpy(), mask)
    err = np.abs(Yh.cpu().numpy() - ref_h).reshape(w.G, -1).max(axis=1)
    assert (err <= DEC_TOL * np.abs(ref_h).reshape(w.G, -1).max(axis=1)).all()
    np.testing.assert_array_equal(n_used.cpu().numpy(), n_ref)
    assert bool((n_used == 4).all()) and bool((status == 0).all())


def test_workload2_full_size_encode_and_decode():
    need_gb(20)
    w = wl.workload(2)
    p = ap.make_params(w.K, w.W)
    X = wl.queries(w, dev())
    Xt = ap.approxifer_encode(p, X)
    check_encode_full(w, X, Xt, seed=2)
    del X, Xt
    Yt = wl.gaussian_predictions(w, dev())
    mask = wl.masks(w)
    n_used = torch.empty(w.G, dtype=torch.int32, device=dev())
    status = torch.empty(w.G, dtype=torch.int32, device=dev())
    Yh = ap.approxifer_decode(p, Yt, ap.mask_tensor(mask), n_used=n_used, status=status)
    # C = 10: every group, every element
    ref, n_ref, st_ref = oracle.decode(w.K, w.W, Yt.cpu().numpy(), mask)
    err = np.abs(Yh.cpu().numpy() - ref).reshape(w.G, -1).max(axis=1)
    assert (err <= DEC_TOL * np.abs(ref).reshape(w.G, -1).max(axis=1)).all()
    np.testing.assert_array_equal(n_used.cpu().numpy(), n_ref)
    np.testing.assert_array_equal(status.cpu().numpy().view(np.uint32), st_ref)


def test_workload3_full_size_encode():
    need_gb(85)
    w = wl.workload(3)
    p = ap.make_params(w.K, w.W)
    X = wl.queries(w, dev())
    Xt = ap.approxifer_encode(p, X)
    check_encode_full(w, X, Xt, seed=3)


def test_workload3_full_size_decode():
    w = wl.workload(3)
    p = ap.make_params(w.K, w.W)
    Yt = wl.gaussian_predictions(w, dev())
    mask = wl.masks(w)
    n_used = torch.empty(w.G, dtype=torch.int32, device=dev())
    status = torch.empty(w.G, dtype=torch.int32, device=dev())
    Yh = ap.approxifer_decode(p, Yt, ap.mask_tensor(mask), n_used=n_used, status=status)
    check_decode_full(w, Yt, mask, Yh, n_used, status, seed=33)
    assert ap.device_wait_timeouts() == 0


def test_workload4_full_size_decode():
    need_gb(50)
    w = wl.workload(4)
    p = ap.make_params(w.K, w.W)
    # hidden queries -> the ORACLE's coded queries -> stand-in model (torch, on the GPU) -> coded predictions
    Xh = wl.queries(w, "cpu")
    Xc = torch.from_numpy(oracle.encode(w.K, w.W, Xh.numpy()).astype(np.float32)).to(dev())
    Yt = torch.empty((w.G, w.W, w.C), device=dev())
    for s in range(0, w.G, 16384):
        Yt[s:s + 16384] = wl.apply_model(w, Xc[s:s + 16384])
    del Xc
    mask = wl.masks(w)
    n_used = torch.empty(w.G, dtype=torch.int32, device=dev())
    status = torch.empty(w.G, dtype=torch.int32, device=dev())
    Yh = ap.approxifer_decode(p, Yt, ap.mask_tensor(mask), n_used=n_used, status=status)
    check_decode_full(w, Yt, mask, Yh, n_used, status, seed=4)
    assert ap.device_wait_timeouts() == 0
    assert int(n_used.min()) >= 16 and int(n_used.max()) == 24


@pytest.mark.parametrize("softmax,sigma", [(False, 10.0), (True, 10.0)])
def test_workload5_full_size_locate_then_decode(softmax, sigma):
    w = wl.workload(5)
    p = ap.make_params(w.K, w.W, w.E)
    Xh = wl.queries(w, "cpu")
    Xc = torch.from_numpy(oracle.encode(w.K, w.W, Xh.numpy()).astype(np.float32))
    Yt = wl.apply_model(w, Xc, softmax=softmax)
    mask = wl.masks(w)
    truth = wl.adversaries(w, mask)
    wl.corrupt(w, Yt, truth, sigma=sigma)
    Yd = Yt.to(dev())
    status = torch.empty(w.G, dtype=torch.int32, device=dev())
    adv, trusted = ap.approxifer_locate(p, Yd, ap.mask_tensor(mask), status=status)
    ref = oracle.locate(w.K, w.W, w.E, Yt.numpy(), mask)
    solid = (ref["min_gap"] > 1.0 + 1e-6) & (ref["vote_margin"] > 0) & ((ref["status"] & oracle.ST_ORACLE_RANK_DEFICIENT) == 0)
    got_adv = adv.cpu().numpy()
    got_tr = trusted.cpu().numpy().view(np.uint32)
    np.testing.assert_array_equal(got_adv[solid], ref["adv"][solid])
    np.testing.assert_array_equal(got_tr[solid], ref["trusted"][solid])
    np.testing.assert_array_equal(status.cpu().numpy().view(np.uint32)[solid], ref["status"][solid] & 0xFF)
    if not softmax:
        # rational honest predictions: Theorem 1 applies, no group is near-tied, every injected set is found
        assert solid.all()
        np.testing.assert_array_equal(got_adv, truth)
    else:
        assert (~solid).mean() < 0.02
    # decode from the trusted workers the oracle found (identical to the GPU's wherever solid)
    n_used = torch.empty(w.G, dtype=torch.int32, device=dev())
    st2 = torch.empty(w.G, dtype=torch.int32, device=dev())
    tr = ap.mask_tensor(ref["trusted"])
    Yh = ap.approxifer_decode(p, Yd, tr, n_used=n_used, status=st2)
    ref_h, n_ref, st_ref = oracle.decode(w.K, w.W, Yt.numpy(), ref["trusted"])
    err = np.abs(Yh.cpu().numpy() - ref_h).reshape(w.G, -1).max(axis=1)
    assert (err <= DEC_TOL * np.abs(ref_h).reshape(w.G, -1).max(axis=1)).all()
    np.testing.assert_array_equal(n_used.cpu().numpy(), n_ref)
    assert bool((n_used == 20).all())
