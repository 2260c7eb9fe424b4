"""GPU parity of approxifer_decode_rational (Algorithm 3: P/Q at the alpha nodes) against its numpy oracle,
through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from oracle import homogeneous as hom
import paper_2109_09868_b200 as ap

pytestmark = pytest.mark.gpu

TOL = 1e-4  # fp32 output, the decoder's tolerance: per group, relative to the largest value of the group


def dev():
    return torch.device("cuda:0")


def case(K, W, E, S, G, C, seed, softmax=False, sigma=10.0, d_in=12):
    rng = np.random.default_rng(seed)
    X = rng.random((G, K, d_in), dtype=np.float32)
    M = rng.standard_normal((d_in, C)) / np.sqrt(d_in)
    Y = oracle.encode(K, W, X) @ M
    if softmax:
        Y = np.exp(Y - Y.max(axis=-1, keepdims=True))
        Y /= Y.sum(axis=-1, keepdims=True)
    Y = Y.astype(np.float32)
    mask = np.empty(G, dtype=np.uint32)
    for g in range(G):
        present = np.sort(rng.choice(W, size=W - S, replace=False))
        mask[g] = sum(1 << int(i) for i in present)
        if E:
            bad = rng.choice(present, size=E, replace=False)
            Y[g, bad] += (sigma * rng.standard_normal((E, C))).astype(np.float32)
    return torch.from_numpy(Y), mask, X.astype(np.float64) @ M


def compare(K, W, E, Yt, mask, min_q=1e-6):
    G = Yt.shape[0]
    status = torch.empty(G, dtype=torch.int32, device=dev())
    Yh = ap.approxifer_decode_rational(ap.make_params(K, W, E), Yt.to(dev()), ap.mask_tensor(mask), status=status)
    torch.cuda.synchronize()
    got = Yh.cpu().numpy().astype(np.float64)
    st = status.cpu().numpy().view(np.uint32)
    ref = hom.decode_rational(K, W, E, Yt.numpy(), mask, oracle.alpha(K))
    under = (ref["status"] & oracle.ST_LOCATE_UNDERDETERMINED) != 0
    np.testing.assert_array_equal((st & oracle.ST_LOCATE_UNDERDETERMINED) != 0, under)
    assert np.all(got[under] == 0)
    # groups in which a root of Q comes close to an output node are ill-posed for any arithmetic: not compared
    ok = ~under & (ref["q_min"] > min_q)
    err = np.abs(got - ref["Yhat"]).reshape(G, -1).max(axis=1)
    scale = np.abs(ref["Yhat"]).reshape(G, -1).max(axis=1)
    assert np.all(err[ok] <= TOL * np.maximum(scale[ok], 1e-30)), float((err[ok] / np.maximum(scale[ok], 1e-30)).max())
    return got, ref, ok


@pytest.mark.parametrize("K,E,S,W", [(8, 2, 2, 24), (2, 1, 0, 6), (3, 2, 1, 12), (4, 1, 2, 12), (6, 3, 1, 20), (2, 0, 0, 4),
                                     (5, 0, 3, 13), (7, 3, 0, 32), (8, 2, 0, 20), (9, 1, 4, 24), (1, 1, 0, 4), (10, 1, 0, 22), (12, 1, 2, 28), (10, 3, 0, 26)])
def test_rational_decoder_matches_oracle_and_recovers_a_linear_model(K, E, S, W):
    G, C = 64, 10
    Yt, mask, truth = case(K, W, E, S, G, C, seed=K * 41 + E)
    got, ref, ok = compare(K, W, E, Yt, mask)
    assert ok.all()
    # the theorem after Algorithm 3: the model's own predictions come back (fp32 inputs, amplified rounding)
    assert np.abs(got - truth).max() <= (2e-4 if K + E <= 5 else (5e-2 if K + E <= 10 else 0.5)) * np.abs(truth).max()


def test_rational_decoder_softmax_model_many_classes_and_degenerate_groups():
    K, E, S, W = 4, 1, 1, 12
    for C in (1, 3, 130):
        Yt, mask, _ = case(K, W, E, S, 40, C, seed=C, softmax=True, sigma=1.0)
        mask[3] = 0x1FF  # 9 workers < 2(K+E)
        mask[4] = 0
        got, ref, ok = compare(K, W, E, Yt, mask)
        assert ok.sum() >= 30


def test_rational_decoder_strided_output_and_worker_major_input():
    K, E, S, W, G, C = 3, 1, 1, 9, 33, 7
    Yt, mask, _ = case(K, W, E, S, G, C, seed=3)
    ref = ap.approxifer_decode_rational(ap.make_params(K, W, E), Yt.to(dev()), ap.mask_tensor(mask))
    wm = Yt.to(dev()).permute(1, 0, 2).contiguous()          # [W][G][C]
    out = torch.full((G, K, C + 3), -7.0, device=dev())
    ap.approxifer_decode_rational(ap.make_params(K, W, E), wm.permute(1, 0, 2), ap.mask_tensor(mask), out[:, :, :C])
    assert torch.equal(out[:, :, :C], ref) and bool((out[:, :, C:] == -7.0).all())


def test_rational_decoder_argument_errors():
    with pytest.raises(ap.ApproxiferError):  # K+E beyond the kernel's range
        ap.approxifer_decode_rational(ap.make_params(12, 32, 2), torch.zeros((1, 32, 4), device=dev()),
                                      ap.mask_tensor(np.array([0xFFFFFFFF], dtype=np.uint32)))
    with pytest.raises(ap.ApproxiferError):  # 2(K+E) > W
        ap.approxifer_decode_rational(ap.make_params(4, 9, 1), torch.zeros((1, 9, 4), device=dev()),
                                      ap.mask_tensor(np.array([0x1FF], dtype=np.uint32)))


def test_workload5_full_size_rational_decoding():
    """The Byzantine workload at full size (65,536 groups): every group is decoded despite its two corrupted
    workers; every 64th group is compared with the oracle, and all outputs with the model's own predictions."""
    from paper_2109_09868_b200 import workloads as wl

    w = wl.workload(5)
    Xh = wl.queries(w, "cpu")
    Xc = torch.from_numpy(oracle.encode(w.K, w.W, Xh.numpy()).astype(np.float32))
    Yt = wl.apply_model(w, Xc)
    truth = wl.apply_model(w, Xh).numpy().astype(np.float64)   # the model on the uncoded queries
    mask = wl.masks(w)
    wl.corrupt(w, Yt, wl.adversaries(w, mask))
    status = torch.empty(w.G, dtype=torch.int32, device=dev())
    Yh = ap.approxifer_decode_rational(ap.make_params(w.K, w.W, w.E), Yt.to(dev()), ap.mask_tensor(mask), status=status)
    got = Yh.cpu().numpy().astype(np.float64)
    assert int(status.abs().sum()) == 0 and np.isfinite(got).all()
    sel = np.arange(0, w.G, 64)
    ref = hom.decode_rational(w.K, w.W, w.E, Yt.numpy()[sel], mask[sel], oracle.alpha(w.K))
    err = np.abs(got[sel] - ref["Yhat"]).reshape(len(sel), -1).max(axis=1)
    scale = np.abs(ref["Yhat"]).reshape(len(sel), -1).max(axis=1)
    assert np.all(err <= TOL * scale)
    # Berrut decoding from the trusted workers approximates the model; this one reproduces it (up to the amplified
    # fp32 rounding of the coded predictions)
    rel = np.abs(got - truth).reshape(w.G, -1).max(axis=1) / np.abs(truth).reshape(w.G, -1).max(axis=1)
    assert np.median(rel) < 1e-3 and np.quantile(rel, 0.999) < 0.2
