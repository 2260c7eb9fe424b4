"""GPU parity: the CUDA library, called through its C ABI, against the fp64 CPU
oracle on the same seeded inputs, element by element.

Tolerances (fp32 kernels vs fp64 oracle):
  encode : max |Xt_gpu - Xt_oracle| <= 1e-5 * max |X|  over the tensor
  decode : per group, max |Yh_gpu - Yh_oracle| <= 1e-4 * max |Yh_oracle| of that group
  mask compaction (n_used, worker lists) and the located set: bit-exact
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2109_09868_b200 as ap
from paper_2109_09868_b200 import binding
from paper_2109_09868_b200 import workloads as wl

pytestmark = pytest.mark.gpu

ENC_TOL = 1e-5
DEC_TOL = 1e-4
CANARY = 1234.5


def dev():
    return torch.device("cuda:0")


def check_encode(K, W, X_cpu, Xt_gpu):
    ref = oracle.encode(K, W, X_cpu.numpy())
    err = np.abs(Xt_gpu.cpu().numpy().astype(np.float64) - ref).max() if ref.size else 0.0
    scale = float(X_cpu.abs().max()) if X_cpu.numel() else 1.0
    assert err <= ENC_TOL * scale, (K, W, err, scale)
    return err


def check_decode(K, W, Yt_cpu, mask_np, Yh_gpu, n_used=None, status=None, flags=0):
    ref, n_ref, st_ref = oracle.decode(K, W, Yt_cpu.numpy(), mask_np, flags)
    got = Yh_gpu.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    err = np.abs(got - ref).reshape(len(mask_np), -1).max(axis=1)
    scale = np.abs(ref).reshape(len(mask_np), -1).max(axis=1)
    bad = err > DEC_TOL * np.maximum(scale, 1e-30)
    bad &= ~((scale == 0) & (err == 0))
    assert not bad.any(), (K, W, int(bad.sum()), float(err[bad].max()), float(scale[bad].min()))
    if n_used is not None:
        np.testing.assert_array_equal(n_used.cpu().numpy(), n_ref)
    if status is not None:
        np.testing.assert_array_equal(status.cpu().numpy().view(np.uint32), st_ref)
    return float((err / np.maximum(scale, 1e-30)).max())


# ------------------------------------------------------------------- encode

ENCODE_SHAPES = [
    (4, 5, 256, 784),    # workload 1
    (8, 12, 7, 3072),    # workload 2 shape
    (12, 20, 2, 150528),  # workload 3 shape, several tiles
    (16, 24, 33, 32),
    (8, 24, 65, 64),
    (3, 7, 5, 1000),     # coincident nodes: rows 1, 3, 5 copy queries 0, 1, 2
    (1, 2, 3, 8),
    (1, 9, 3, 12),
    (2, 5, 4, 16),
    (32, 32, 3, 260),
    (31, 2, 2, 4),
    (5, 32, 2, 516),
    (7, 9, 300, 4),      # D = 4: one column per group, many groups per block
    (16, 20, 5, 3072),   # rows of 768 float4 columns: whole-row CTAs of 768 threads (K <= 16)
    (3, 7, 2, 6144),     # two such CTAs per row, coincident nodes
    (20, 24, 3, 3072),   # K > 16: stays on 256-thread CTAs
]


@pytest.mark.parametrize("K,W,G,D", ENCODE_SHAPES)
def test_encode_matches_oracle(K, W, G, D):
    g = torch.Generator().manual_seed(K * 1000 + W)
    X = torch.rand((G, K, D), generator=g) * 2 - 0.5
    p = ap.make_params(K, W)
    Xt = ap.approxifer_encode(p, X.to(dev()))
    torch.cuda.synchronize()
    check_encode(K, W, X, Xt)
    if (K, W) == (3, 7):
        for (j, i) in [(0, 1), (1, 3), (2, 5)]:
            assert torch.equal(Xt[:, i].cpu(), X[:, j])
    if K == 1:
        for i in range(W):
            assert torch.equal(Xt[:, i].cpu(), X[:, 0])


@pytest.mark.parametrize("K,W,G,D", [(4, 5, 9, 783), (8, 12, 3, 3071), (3, 7, 4, 1), (12, 20, 2, 1001), (5, 6, 40, 3)])
def test_encode_odd_lengths_take_the_elementwise_path(K, W, G, D):
    g = torch.Generator().manual_seed(D)
    X = torch.rand((G, K, D), generator=g)
    Xt = ap.approxifer_encode(ap.make_params(K, W), X.to(dev()))
    check_encode(K, W, X, Xt)


def test_encode_misaligned_strided_and_guarded_buffers():
    K, W, G, D = 8, 12, 6, 260
    g = torch.Generator().manual_seed(5)
    X = torch.rand((G, K, D), generator=g)
    p = ap.make_params(K, W)
    # (a) base pointers off by one float: not 16-byte aligned
    xin = torch.zeros(G * K * D + 1, device=dev())
    xin[1:] = X.flatten().to(dev())
    out = torch.full((G * W * D + 9,), CANARY, device=dev())
    Xt = ap.approxifer_encode(p, xin[1:].view(G, K, D), out[5 : 5 + G * W * D].view(G, W, D))
    check_encode(K, W, X, Xt)
    assert bool((out[:5] == CANARY).all()) and bool((out[5 + G * W * D :] == CANARY).all())
    # (b) padded rows (row stride > D) on both sides, canaries in the padding
    pad = 12
    xin2 = torch.full((G, K, D + pad), CANARY, device=dev())
    xin2[:, :, :D] = X.to(dev())
    out2 = torch.full((G, W, D + pad), CANARY, device=dev())
    ap.approxifer_encode(p, xin2[:, :, :D], out2[:, :, :D])
    check_encode(K, W, X, out2[:, :, :D])
    assert bool((out2[:, :, D:] == CANARY).all())
    # (c) worker-major output [W][G][D]
    out3 = torch.empty((W, G, D), device=dev())
    ap.approxifer_encode(p, X.to(dev()), out3.permute(1, 0, 2))
    check_encode(K, W, X, out3.permute(1, 0, 2))
    # (d) G = 0
    ap.approxifer_encode(p, torch.empty((0, K, D), device=dev()))


def test_encode_weights_on_device_match_oracle():
    for (K, W) in [(4, 5), (8, 12), (12, 20), (16, 24), (8, 24), (3, 7), (32, 32), (1, 2), (2, 5), (4, 9)]:
        w = ap.approxifer_debug_weights(ap.make_params(K, W), which=0).cpu().numpy().astype(np.float64)
        ref = oracle.encode_weights(K, W)
        assert np.abs(w - ref).max() <= 1.2e-7 * max(1.0, np.abs(ref).max()), (K, W)
        for i in range(W):
            for j in range(K):
                if oracle.coincident(K, W, j, i):
                    assert w[i, j] == 1.0 and np.abs(w[i]).sum() == 1.0


# ------------------------------------------------------------------- decode

def random_masks(W, G, rng, min_present=0):
    m = rng.integers(0, 2**W, size=G, dtype=np.uint64)
    for g in range(G):
        while bin(int(m[g])).count("1") < min_present:
            m[g] |= np.uint64(1) << np.uint64(rng.integers(0, W))
    return m.astype(np.uint32)


DECODE_SHAPES = [
    (4, 5, 256, 10),
    (8, 12, 300, 10),
    (12, 20, 9, 1000),
    (16, 24, 21, 1000),
    (8, 24, 130, 10),
    (3, 7, 64, 36),     # coincident nodes
    (1, 2, 8, 4),
    (2, 5, 32, 8),      # alpha = +-sqrt(2)/2 coincide with beta_1, beta_3
    (4, 9, 40, 12),
    (32, 32, 5, 260),
    (5, 32, 6, 513),
    (9, 11, 50, 1),
]


@pytest.mark.parametrize("K,W,G,C", DECODE_SHAPES)
@pytest.mark.parametrize("flags", [0, 1])
def test_decode_matches_oracle(K, W, G, C, flags):
    rng = np.random.default_rng(K * 100 + W + flags)
    g = torch.Generator().manual_seed(K * 100 + W)
    Yt = torch.randn((G, W, C), generator=g)
    mask = random_masks(W, G, rng, min_present=(0 if flags == 0 else max(W - 2, 1)))
    mask[0] = 2**W - 1
    if flags == 1:
        # the literal sign (-1)^i has real poles when the used workers are not a
        # contiguous run; keep only masks whose weights stay moderate
        for gi in range(G):
            w_lit, _ = oracle.decode_weights(K, W, int(mask[gi]), 1)
            if np.abs(w_lit).sum(axis=1).max() > 30.0:
                mask[gi] = 2**W - 1
    if flags == 0 and G > 3:
        mask[1] = 0
        mask[2] = 1 << (W - 1)
        mask[3] |= np.uint32((0xFFFFFFFF << W) & 0xFFFFFFFF)  # bits beyond W must be ignored
    p = ap.make_params(K, W, 0, flags)
    n_used = torch.empty(G, dtype=torch.int32, device=dev())
    status = torch.empty(G, dtype=torch.int32, device=dev())
    Yh = ap.approxifer_decode(p, Yt.to(dev()), ap.mask_tensor(mask), n_used=n_used, status=status)
    check_decode(K, W, Yt, mask, Yh, n_used, status, flags)


@pytest.mark.parametrize("K,W", [(2, 3), (3, 6), (4, 8), (3, 7), (2, 5)])
def test_decode_all_masks_exhaustively(K, W):
    G, C = 2**W, 12
    g = torch.Generator().manual_seed(W)
    Yt = torch.randn((G, W, C), generator=g)
    mask = np.arange(G, dtype=np.uint32)
    n_used = torch.empty(G, dtype=torch.int32, device=dev())
    status = torch.empty(G, dtype=torch.int32, device=dev())
    Yh = ap.approxifer_decode(ap.make_params(K, W), Yt.to(dev()), ap.mask_tensor(mask), n_used=n_used, status=status)
    check_decode(K, W, Yt, mask, Yh, n_used, status)
    # compaction through the weight hook: worker lists are bit-exact
    for m in (1, 5, G - 1, G // 2 + 3):
        w, idx = ap.approxifer_debug_weights(ap.make_params(K, W), mask=m, which=1)
        w_ref, F = oracle.decode_weights(K, W, m)
        assert idx.cpu().tolist() == F
        assert np.abs(w.cpu().numpy() - w_ref).max() <= 2e-6 * max(1.0, np.abs(w_ref).max())


def test_decode_ignores_garbage_in_absent_rows_and_copies_at_coincident_nodes():
    K, W, G, C = 3, 7, 16, 20
    rng = np.random.default_rng(3)
    g = torch.Generator().manual_seed(3)
    Yt = torch.randn((G, W, C), generator=g)
    mask = random_masks(W, G, rng, min_present=2)
    mask[0] = 0x7F
    dirty = Yt.clone()
    for gi in range(G):
        for i in range(W):
            if not (int(mask[gi]) >> i) & 1:
                dirty[gi, i] = float("nan")
    p = ap.make_params(K, W)
    a = ap.approxifer_decode(p, Yt.to(dev()), ap.mask_tensor(mask))
    b = ap.approxifer_decode(p, dirty.to(dev()), ap.mask_tensor(mask))
    assert torch.equal(a, b)
    check_decode(K, W, Yt, mask, a)
    for (j, i) in [(0, 1), (1, 3), (2, 5)]:
        for gi in range(G):
            if (int(mask[gi]) >> i) & 1:
                assert torch.equal(a[gi, j].cpu(), Yt[gi, i])


def test_decode_misaligned_strided_and_guarded_buffers():
    K, W, G, C = 8, 12, 10, 100
    rng = np.random.default_rng(8)
    g = torch.Generator().manual_seed(8)
    Yt = torch.randn((G, W, C), generator=g)
    mask = random_masks(W, G, rng, min_present=1)
    p = ap.make_params(K, W)
    yin = torch.zeros(G * W * C + 3, device=dev())
    yin[3:] = Yt.flatten().to(dev())
    out = torch.full((G * K * C + 8,), CANARY, device=dev())
    Yh = ap.approxifer_decode(p, yin[3:].view(G, W, C), ap.mask_tensor(mask), out[2 : 2 + G * K * C].view(G, K, C))
    check_decode(K, W, Yt, mask, Yh)
    assert bool((out[:2] == CANARY).all()) and bool((out[2 + G * K * C :] == CANARY).all())
    pad = 4
    yin2 = torch.full((G, W, C + pad), float("nan"), device=dev())
    yin2[:, :, :C] = Yt.to(dev())
    out2 = torch.full((G, K, C + pad), CANARY, device=dev())
    ap.approxifer_decode(p, yin2[:, :, :C], ap.mask_tensor(mask), out2[:, :, :C])
    check_decode(K, W, Yt, mask, out2[:, :, :C])
    assert bool((out2[:, :, C:] == CANARY).all())


# ------------------------------------------------------------------- locate

def linear_case(K, W, E, S, G, C, seed, softmax=False, sigma=10.0, d_in=16):
    """Honest predictions = linear (optionally + softmax) model of the ORACLE's
    coded queries, E corrupted workers among the W-S present."""
    rng = np.random.default_rng(seed)
    X = rng.random((G, K, d_in), dtype=np.float32)
    M = rng.standard_normal((d_in, C)) / np.sqrt(d_in)
    Y = oracle.encode(K, W, X) @ M
    if softmax:
        Y = np.exp(Y - Y.max(axis=-1, keepdims=True))
        Y /= Y.sum(axis=-1, keepdims=True)
    Y = Y.astype(np.float32)
    mask = np.empty(G, dtype=np.uint32)
    truth = np.empty((G, E), dtype=np.int32)
    for g in range(G):
        present = np.sort(rng.choice(W, size=W - S, replace=False))
        mask[g] = sum(1 << int(i) for i in present)
        bad = np.sort(rng.choice(present, size=E, replace=False))
        truth[g] = bad
        Y[g, bad] += (sigma * rng.standard_normal((E, C))).astype(np.float32)
    return torch.from_numpy(Y), mask, truth


def run_locate(K, W, E, Yt, mask, force_warp_kernel=False):
    G = Yt.shape[0]
    status = torch.empty(G, dtype=torch.int32, device=dev())
    adv, trusted = ap.approxifer_locate(ap.make_params(K, W, E), Yt.to(dev()), ap.mask_tensor(mask), status=status,
                                        force_warp_kernel=force_warp_kernel)
    torch.cuda.synchronize()
    return adv.cpu().numpy(), trusted.cpu().numpy().view(np.uint32), status.cpu().numpy().view(np.uint32)


def compare_locate(K, W, E, Yt, mask, allow_fragile=False, force_warp_kernel=False):
    ref = oracle.locate(K, W, E, Yt.numpy(), mask)
    adv, trusted, status = run_locate(K, W, E, Yt, mask, force_warp_kernel=force_warp_kernel)
    solid = (ref["min_gap"] > 1.0 + 1e-6) & (ref["vote_margin"] > 0) & ((ref["status"] & oracle.ST_ORACLE_RANK_DEFICIENT) == 0)
    solid |= (ref["status"] & oracle.ST_LOCATE_UNDERDETERMINED) != 0
    if not allow_fragile:
        assert solid.all(), "workload has near-tied groups: %d" % int((~solid).sum())
    np.testing.assert_array_equal(adv[solid], ref["adv"][solid])
    np.testing.assert_array_equal(trusted[solid], ref["trusted"][solid])
    np.testing.assert_array_equal(status[solid], ref["status"][solid] & 0xFF)
    # whatever was returned is always a valid answer: E distinct present workers, ascending
    for g in range(len(mask)):
        if ref["status"][g] & oracle.ST_LOCATE_UNDERDETERMINED:
            continue
        row = adv[g]
        assert np.all(np.diff(row) > 0) and all((int(mask[g]) >> int(i)) & 1 for i in row)
        assert int(trusted[g]) == (int(mask[g]) & (2**W - 1)) & ~sum(1 << int(i) for i in row)
    return ref, adv, int((~solid).sum())


@pytest.mark.parametrize("K,E,S,W", [(8, 2, 2, 24), (2, 1, 0, 6), (3, 2, 1, 12), (4, 1, 2, 12), (12, 2, 0, 28), (12, 1, 2, 28), (10, 3, 0, 26),
                                     (6, 3, 1, 20), (1, 1, 0, 4), (13, 3, 0, 32), (8, 2, 0, 20), (2, 1, 3, 9)])
def test_locate_matches_oracle_and_finds_injected_errors(K, E, S, W):
    G, C = 96, 10
    Yt, mask, truth = linear_case(K, W, E, S, G, C, seed=K * 31 + E)
    ref, adv, _ = compare_locate(K, W, E, Yt, mask)
    if W % 2 == 0:  # no node at 0: Theorem 1 guarantees exact location for a rational model
        np.testing.assert_array_equal(adv, truth)


def test_locate_softmax_model_and_noise_scales():
    K, E, S, W = 8, 2, 2, 24
    for sigma in (1.0, 10.0, 100.0):
        Yt, mask, truth = linear_case(K, W, E, S, 256, 10, seed=int(sigma), softmax=True, sigma=sigma)
        ref, adv, fragile = compare_locate(K, W, E, Yt, mask, allow_fragile=True)
        assert fragile <= 8
        assert (adv == truth).all(axis=1).mean() > 0.9


def test_locate_many_classes_one_class_and_underdetermined_groups():
    K, E, S, W = 4, 1, 1, 12
    Yt, mask, truth = linear_case(K, W, E, S, 24, 1000, seed=77)
    compare_locate(K, W, E, Yt, mask)
    Yt1, mask1, _ = linear_case(K, W, E, S, 40, 1, seed=78)
    mask1[::4] = 0b000111111111  # 9 < 2(K+E) = 10 workers -> nothing located
    mask1[1] = 0
    ref, adv, _ = compare_locate(K, W, E, Yt1, mask1)
    assert (adv[::4] == -1).all() and adv[1, 0] == -1
    # a class whose predictions are exactly zero leaves Q = 1: the lowest workers are picked
    Z = torch.zeros((3, W, 2))
    full = np.full(3, 2**W - 1, dtype=np.uint32)
    ref, adv, _ = compare_locate(K, W, E, Z, full, allow_fragile=True)
    assert (adv == 0).all() and (ref["adv"] == 0).all()


def test_locate_then_decode_pipeline_matches_oracle():
    K, E, S, W, G, C = 8, 2, 2, 24, 200, 10
    Yt, mask, truth = linear_case(K, W, E, S, G, C, seed=5)
    p = ap.make_params(K, W, E)
    adv, trusted = ap.approxifer_locate(p, Yt.to(dev()), ap.mask_tensor(mask))
    n_used = torch.empty(G, dtype=torch.int32, device=dev())
    Yh = ap.approxifer_decode(p, Yt.to(dev()), trusted, n_used=n_used)
    ref = oracle.locate(K, W, E, Yt.numpy(), mask)
    np.testing.assert_array_equal(trusted.cpu().numpy().view(np.uint32), ref["trusted"])
    check_decode(K, W, Yt, ref["trusted"], Yh, n_used)
    assert bool((n_used == W - S - E).all())


def test_strided_predictions_for_locate():
    K, E, S, W, G, C = 3, 1, 0, 8, 20, 7
    Yt, mask, truth = linear_case(K, W, E, S, G, C, seed=9)
    big = torch.full((G, W, C + 5), float("nan"))
    big[:, :, :C] = Yt
    adv, trusted = ap.approxifer_locate(ap.make_params(K, W, E), big.to(dev())[:, :, :C], ap.mask_tensor(mask))
    ref = oracle.locate(K, W, E, Yt.numpy(), mask)
    np.testing.assert_array_equal(adv.cpu().numpy(), ref["adv"])


# ----------------------------------------------- wide-payload (staged) decoder

STAGED_SHAPES = [
    (16, 24, 300, 1000, 0),   # workload 4 shape: two column tiles per group (128 + 122 columns)
    (12, 20, 37, 4000, 0),    # eight column tiles per group, ragged last tile
    (8, 12, 200, 512, 0),     # smallest payload that takes the staged path
    (3, 7, 60, 1024, 0),      # coincident nodes
    (5, 9, 64, 2052, 1),      # literal sign: stays on the register-staged kernel
    (32, 32, 9, 1028, 0),     # largest K and W
    (7, 13, 50, 516, 0),      # odd K: the two halves own 4 and 3 queries
    (1, 2, 20, 640, 0),       # K = 1: the second half of the CTA owns nothing
    (16, 24, 90, 128, 0),     # one 32-column item per group
    (12, 20, 75, 100, 0),     # 25 of 32 columns in use (the shortest rows that take the staged path have 96 floats)
    (6, 9, 51, 96, 0),
    (8, 12, 64, 64, 0),       # the shortest rows that take the staged path: 16-column items, one compute warp
    (5, 10, 40, 80, 0),
    (8, 12, 70, 200, 0),      # 50 columns
    (12, 20, 33, 256, 0),     # exactly one 64-column item per group
    (16, 24, 40, 400, 0),     # 100 columns: 128-column items
    (8, 12, 77, 52, 0),       # K >= 8: rows of 52 .. 60 floats too (13 of 16 columns in use)
    (12, 20, 50, 60, 0),
]


@pytest.mark.parametrize("stages,ctas,cols,split", [(0, 0, 0, 0), (2, 0, 128, 2), (3, 1, 128, 4), (4, 1, 64, 2), (2, 4, 64, 4), (0, 2, 64, 4),
                                                        (0, 0, 256, 2), (2, 1, 256, 0), (0, 0, 128, 0), (0, 0, 0, 1), (0, 0, 0, 2), (0, 0, 32, 2),
                                                        (3, 0, 32, 0), (0, 0, 16, 2)])
def test_staged_decoder_matches_oracle_in_every_configuration(stages, ctas, cols, split):
    tuning = ap.decode_tuning(3, stages, ctas, cols, split)
    for (K, W, G, C, flags) in STAGED_SHAPES:
        rng = np.random.default_rng(C + K)
        g = torch.Generator().manual_seed(C)
        Yt = torch.randn((G, W, C), generator=g)
        if flags == 0:
            mask = random_masks(W, G, rng, min_present=0)
            mask[0], mask[1], mask[2] = 2**W - 1, 0, 1 << (W - 1)
        else:
            mask = np.full(G, 2**W - 1, dtype=np.uint32)
            mask[::3] = (2**W - 1) & ~1
        dirty = Yt.clone()
        for gi in range(G):
            for i in range(W):
                if not (int(mask[gi]) >> i) & 1:
                    dirty[gi, i] = float("nan")  # absent rows must never be used
        n_used = torch.empty(G, dtype=torch.int32, device=dev())
        status = torch.empty(G, dtype=torch.int32, device=dev())
        out = torch.full((G, K, C + 4), CANARY, device=dev())
        Yh = ap.approxifer_decode(ap.make_params(K, W, 0, flags), dirty.to(dev()), ap.mask_tensor(mask), out[:, :, :C],
                                  n_used=n_used, status=status, tuning=tuning)
        check_decode(K, W, Yt, mask, Yh, n_used, status, flags)
        assert bool((out[:, :, C:] == CANARY).all())
    assert ap.device_wait_timeouts() == 0


def test_staged_and_register_decoders_agree_bitwise_on_sums_order():
    """Both decoders add the same terms in the same order, so they agree to the last bit
    except for the reciprocal-multiply of the denominator (identical too)."""
    K, W, G, C = 12, 20, 64, 1000
    rng = np.random.default_rng(1)
    Yt = torch.randn((G, W, C), generator=torch.Generator().manual_seed(1)).to(dev())
    mask = ap.mask_tensor(random_masks(W, G, rng, min_present=1))
    p = ap.make_params(K, W)
    a = ap.approxifer_decode(p, Yt, mask)
    b = ap.approxifer_decode(p, Yt, mask, tuning=ap.decode_tuning(kernel=1))
    assert torch.equal(a, b)


@pytest.mark.parametrize("K,W,C,G", [(8, 12, 10, 1000), (8, 24, 10, 333), (4, 5, 10, 7), (3, 7, 9, 130), (1, 2, 1, 50),
                                     (32, 32, 32, 21), (16, 24, 31, 64), (2, 5, 2, 257), (12, 20, 17, 90), (5, 9, 4, 3),
                                     (8, 12, 100, 500), (16, 24, 128, 70), (16, 24, 256, 33), (12, 20, 36, 100), (5, 9, 64, 41),
                                     (3, 7, 20, 50), (8, 12, 500, 9), (16, 24, 508, 5), (32, 32, 64, 6), (2, 5, 102, 77)])
def test_short_payload_decoder_against_oracle_and_register_decoder(K, W, C, G):
    """Dense buffers with up to a few hundred classes take the thread-per-(query, chunk of classes) kernel
    (a few shapes here fall outside it on purpose and must still be right).  It adds the same terms in the same
    order as the thread-per-class kernel: equal to the last bit, absent rows (NaN here) never used, both sign
    rules, coincident nodes ((K, W) = (3, 7), (1, 2) and (2, 5) have them), group counts that leave a ragged last CTA."""
    rng = np.random.default_rng(K * 100 + C)
    Yt = torch.randn((G, W, C), generator=torch.Generator().manual_seed(C))
    mask = random_masks(W, G, rng, min_present=0)
    mask[0] = 0
    dirty = Yt.clone()
    for gi in range(G):
        for i in range(W):
            if not (int(mask[gi]) >> i) & 1:
                dirty[gi, i] = float("nan")
    for flags in (0, binding.SIGN_WORKER_INDEX):
        p = ap.make_params(K, W, 0, flags)
        n_used = torch.empty(G, dtype=torch.int32, device=dev())
        status = torch.empty(G, dtype=torch.int32, device=dev())
        guard = torch.full((G * K * C + 64,), CANARY, device=dev())
        Yh = guard[32: 32 + G * K * C].view(G, K, C)
        ap.approxifer_decode(p, dirty.to(dev()), ap.mask_tensor(mask), Yh, n_used=n_used, status=status,
                             tuning=ap.decode_tuning(kernel=2))
        if flags == 0:  # (the literal sign has poles: on arbitrary masks a denominator can vanish, see pin P9)
            check_decode(K, W, Yt, mask, Yh, n_used, status, flags)
        assert bool((guard[:32] == CANARY).all()) and bool((guard[32 + G * K * C:] == CANARY).all())
        ref = ap.approxifer_decode(p, dirty.to(dev()), ap.mask_tensor(mask), tuning=ap.decode_tuning(kernel=1))
        assert torch.equal(Yh.contiguous().view(torch.int32), ref.view(torch.int32))  # bit patterns: inf/NaN included


PACK_SHAPES = [
    # K, W, C, G
    (8, 12, 10, 1000),    # the paper's shape: whole-block copies, 4 queries per thread, 5 words each
    (8, 12, 10, 65),      # one full item and one group
    (4, 5, 10, 7),        # a last item that ends on an 8-byte boundary
    (5, 9, 10, 131),      # odd K: tiles of 2 queries
    (3, 7, 20, 50),       # coincident nodes (rows copied), whole-block copies
    (3, 7, 62, 50),       # coincident nodes, the longest rows this kernel takes
    (1, 2, 2, 300),       # the smallest of everything: one word per row
    (2, 5, 6, 257),
    (7, 13, 46, 77),      # 23 words per row: a ragged split (3 threads x 8 words)
    (12, 20, 36, 100),
    (16, 24, 48, 300),
    (8, 12, 64, 500),     # longer rows: other kernels (the comparison still holds)
    (16, 24, 128, 70),
    (32, 32, 20, 40),     # largest K and W: 16 lanes per group
    (32, 32, 40, 9),      # 32 lanes per group: one group per item
    (9, 24, 30, 64),
    (12, 20, 10, 999),    # six lanes per group: five groups do not start on 16-byte boundaries, four do
    (8, 24, 10, 333),
    (16, 24, 10, 1000),
    (3, 7, 10, 50),       # coincident nodes with one lane per row (where the rotated word order can apply)
    (5, 11, 10, 203),     # ... and three lanes per group, a ragged last item
    (8, 12, 8, 100),      # rows of four words, every group starting in the same banks
    (4, 8, 10, 333),      # two lanes per group, rotated because shared memory bounds it
]


@pytest.mark.parametrize("K,W,C,G", PACK_SHAPES)
def test_packed_groups_decoder_against_oracle_and_register_decoder(K, W, C, G):
    """Dense buffers with an even number of classes up to 62 take the kernel in which every warp runs its own
    pipeline over items of several groups.  It adds the same terms in the same order as the per-column kernel:
    equal to the last bit; absent rows (NaN here) never used; both sign rules; five warps per CTA, one-group items,
    and the rotated word order forced off and on as well."""
    rng = np.random.default_rng(K * 1000 + C)
    Yt = torch.randn((G, W, C), generator=torch.Generator().manual_seed(C + K))
    mask = random_masks(W, G, rng, min_present=0)
    mask[0] = 0
    mask[G - 1] = 2**W - 1
    if G > 4:
        mask[1], mask[2], mask[3] = 1, 1 << (W - 1), (2**W - 1) & ~2
    dirty = Yt.clone()
    for gi in range(G):
        for i in range(W):
            if not (int(mask[gi]) >> i) & 1:
                dirty[gi, i] = float("nan")
    dY, dm = dirty.to(dev()), ap.mask_tensor(mask)
    for flags in (0, binding.SIGN_WORKER_INDEX):
        p = ap.make_params(K, W, 0, flags)
        ref = ap.approxifer_decode(p, dY, dm, tuning=ap.decode_tuning(kernel=1))
        for tuning in (None, ap.decode_tuning(4, 2, 5, 0, 0), ap.decode_tuning(4, 4, 0, 1, 0),
                       ap.decode_tuning(4, 0, 0, 0, 1), ap.decode_tuning(4, 0, 0, 0, 2)):
            n_used = torch.empty(G, dtype=torch.int32, device=dev())
            status = torch.empty(G, dtype=torch.int32, device=dev())
            guard = torch.full((G * K * C + 64,), CANARY, device=dev())
            Yh = guard[32: 32 + G * K * C].view(G, K, C)
            ap.approxifer_decode(p, dY, dm, Yh, n_used=n_used, status=status, tuning=tuning)
            if flags == 0:  # (the literal sign has poles on arbitrary masks, see pin P9)
                check_decode(K, W, Yt, mask, Yh, n_used, status, flags)
            assert bool((guard[:32] == CANARY).all()) and bool((guard[32 + G * K * C:] == CANARY).all())
            assert torch.equal(Yh.contiguous().view(torch.int32), ref.view(torch.int32))  # bit patterns: inf/NaN included
    assert ap.device_wait_timeouts() == 0


def test_packed_groups_decoder_at_full_occupancy():
    """A problem beyond the L2 cache, where this kernel is the automatic choice and every warp goes several times
    round its ring (configs[1] shape, 160,000 groups)."""
    K, W, C, G = 8, 12, 10, 160000
    rng = np.random.default_rng(5)
    Yt = torch.randn((G, W, C), generator=torch.Generator().manual_seed(9))
    mask = random_masks(W, G, rng, min_present=8)
    n_used = torch.empty(G, dtype=torch.int32, device=dev())
    status = torch.empty(G, dtype=torch.int32, device=dev())
    p = ap.make_params(K, W)
    Yh = ap.approxifer_decode(p, Yt.to(dev()), ap.mask_tensor(mask), n_used=n_used, status=status)
    check_decode(K, W, Yt, mask, Yh, n_used, status)
    ref = ap.approxifer_decode(p, Yt.to(dev()), ap.mask_tensor(mask), tuning=ap.decode_tuning(kernel=1))
    assert torch.equal(Yh, ref)
    assert ap.device_wait_timeouts() == 0


def test_worker_major_layouts_for_decode_and_locate():
    """Coded predictions stored per worker ([W][G][C], the layout in which the workers' answers arrive) are
    addressed through the strides; both decoders and the locator must accept them."""
    K, E, S, W, G = 8, 2, 2, 24, 64
    for C in (10, 1000):
        Yt, mask, truth = linear_case(K, W, E, S, G, C, seed=C)
        wm = Yt.permute(1, 0, 2).contiguous().to(dev())          # [W][G][C]
        view = wm.permute(1, 0, 2)                                # [G][W][C] view: gstride = C, rstride = G*C
        p = ap.make_params(K, W, E)
        adv, trusted = ap.approxifer_locate(p, view, ap.mask_tensor(mask))
        ref = oracle.locate(K, W, E, Yt.numpy(), mask)
        np.testing.assert_array_equal(adv.cpu().numpy(), ref["adv"])
        out = torch.empty((K, G, C), device=dev())               # query-major output
        ap.approxifer_decode(p, view, trusted, out.permute(1, 0, 2))
        check_decode(K, W, Yt, ref["trusted"], out.permute(1, 0, 2))


@pytest.mark.parametrize("K,W,C,G", [(8, 12, 10, 1001), (8, 24, 10, 333), (16, 24, 31, 70), (3, 7, 9, 130), (12, 20, 36, 50), (4, 5, 2, 7)])
def test_short_payload_decoder_reads_worker_major_predictions(K, W, C, G):
    """Predictions stored one batch per worker ([W][G][C]) with dense results: the thread-per-(query, chunk) kernel
    gathers the W ranges of a CTA's groups itself.  Bit-equal to the per-column kernel on the same view."""
    rng = np.random.default_rng(K + C)
    Yt = torch.randn((G, W, C), generator=torch.Generator().manual_seed(C))
    mask = random_masks(W, G, rng, min_present=0)
    wm = Yt.to(dev()).permute(1, 0, 2).contiguous()           # [W][G][C]
    view = wm.permute(1, 0, 2)                                # [G][W][C] view: gstride = C, rstride = G*C
    p = ap.make_params(K, W)
    n_used = torch.empty(G, dtype=torch.int32, device=dev())
    status = torch.empty(G, dtype=torch.int32, device=dev())
    Yh = ap.approxifer_decode(p, view, ap.mask_tensor(mask), n_used=n_used, status=status)
    check_decode(K, W, Yt, mask, Yh, n_used, status)
    ref = ap.approxifer_decode(p, view, ap.mask_tensor(mask), tuning=ap.decode_tuning(kernel=1))
    assert torch.equal(Yh.view(torch.int32), ref.view(torch.int32))


@pytest.mark.parametrize("K,W,C,G", [(8, 12, 10, 1000), (8, 12, 10, 67), (4, 5, 10, 7), (5, 9, 10, 131), (3, 7, 10, 50),
                                     (16, 24, 10, 333), (8, 12, 6, 100), (3, 7, 20, 50), (12, 20, 10, 999), (2, 4, 8, 260)])
def test_packed_groups_decoder_reads_worker_major_predictions(K, W, C, G):
    """The packed-groups kernel on predictions stored one batch per worker ([W][G][C]): an item's rows arrive by one
    bulk copy per worker (by hand where a last item's pieces are not whole 16-byte columns).  Absent rows (NaN)
    never used, both sign rules, coincident nodes ((3, 7)), bit-equal to the per-column kernel on the same view."""
    rng = np.random.default_rng(K * 7 + C)
    Yt = torch.randn((G, W, C), generator=torch.Generator().manual_seed(C + 3 * K))
    mask = random_masks(W, G, rng, min_present=0)
    mask[0] = 0
    mask[G - 1] = 2**W - 1
    dirty = Yt.clone()
    for gi in range(G):
        for i in range(W):
            if not (int(mask[gi]) >> i) & 1:
                dirty[gi, i] = float("nan")
    wm = dirty.to(dev()).permute(1, 0, 2).contiguous()        # [W][G][C]
    view = wm.permute(1, 0, 2)                                # [G][W][C] view: gstride = C, rstride = G*C
    for flags in (0, binding.SIGN_WORKER_INDEX):
        p = ap.make_params(K, W, 0, flags)
        ref = ap.approxifer_decode(p, view, ap.mask_tensor(mask), tuning=ap.decode_tuning(kernel=1))
        for tuning in (ap.decode_tuning(kernel=4), ap.decode_tuning(4, 0, 5, 3, 0)):
            n_used = torch.empty(G, dtype=torch.int32, device=dev())
            status = torch.empty(G, dtype=torch.int32, device=dev())
            guard = torch.full((G * K * C + 64,), CANARY, device=dev())
            Yh = guard[32: 32 + G * K * C].view(G, K, C)
            ap.approxifer_decode(p, view, ap.mask_tensor(mask), Yh, n_used=n_used, status=status, tuning=tuning)
            if flags == 0:
                check_decode(K, W, Yt, mask, Yh, n_used, status, flags)
            assert bool((guard[:32] == CANARY).all()) and bool((guard[32 + G * K * C:] == CANARY).all())
            assert torch.equal(Yh.contiguous().view(torch.int32), ref.view(torch.int32))
    assert ap.device_wait_timeouts() == 0


@pytest.mark.parametrize("K,E,S,W,C", [(8, 2, 2, 24, 10), (3, 2, 1, 12, 37), (4, 1, 2, 12, 300), (2, 1, 0, 6, 1), (7, 3, 1, 22, 10),
                                       (10, 1, 0, 22, 10), (10, 2, 3, 27, 10), (12, 1, 0, 26, 10), (10, 3, 2, 28, 7), (11, 2, 6, 32, 10),
                                       (9, 2, 1, 23, 140), (12, 2, 0, 28, 10), (12, 3, 1, 31, 10), (13, 2, 2, 32, 5)])
def test_both_locator_kernels_return_the_same_sets(K, E, S, W, C):
    """K+E <= 15 normally takes the thread-per-class kernel (two CTAs per SM for K+E = 11..15, whose factor needs
    255 registers and, from 14 on, some local memory); the warp-per-group kernel must agree with it
    (and with the oracle) on the same inputs, including groups with too few workers."""
    G = 150
    Yt, mask, truth = linear_case(K, W, E, S, G, C, seed=K + 7 * E + C)
    mask[5] = (1 << (2 * (K + E) - 1)) - 1  # one worker short: nothing to locate
    ref, adv_rows, _ = compare_locate(K, W, E, Yt, mask)
    ref2, adv_warp, _ = compare_locate(K, W, E, Yt, mask, force_warp_kernel=True)
    np.testing.assert_array_equal(adv_rows, adv_warp)
    assert adv_rows[5, 0] == -1


def test_locate_decode_in_one_call_equals_the_two_steps():
    K, E, S, W, G, C = 8, 2, 2, 24, 300, 10
    Yt, mask, truth = linear_case(K, W, E, S, G, C, seed=21)
    mask[7] = 0x3FF  # too few workers: nothing located, decoded from all ten
    p = ap.make_params(K, W, E)
    Yd, md = Yt.to(dev()), ap.mask_tensor(mask)
    n_used = torch.empty(G, dtype=torch.int32, device=dev())
    lst = torch.empty(G, dtype=torch.int32, device=dev())
    dst = torch.empty(G, dtype=torch.int32, device=dev())
    Yh, adv, trusted = ap.approxifer_locate_decode(p, Yd, md, n_used=n_used, locate_status=lst, decode_status=dst)
    adv2, trusted2 = ap.approxifer_locate(p, Yd, md)
    Yh2 = ap.approxifer_decode(p, Yd, trusted2)
    assert torch.equal(adv, adv2) and torch.equal(trusted, trusted2) and torch.equal(Yh, Yh2)
    ref = oracle.locate(K, W, E, Yt.numpy(), mask)
    np.testing.assert_array_equal(adv.cpu().numpy(), ref["adv"])
    check_decode(K, W, Yt, ref["trusted"], Yh, n_used, dst)
    assert int(lst[7]) == 4 and int(n_used[7]) == 10


@pytest.mark.parametrize("K,E,S,W,C,G,flags", [(8, 2, 2, 24, 10, 257, 0),     # one pass: a thread per (group, class)
                                               (8, 2, 0, 20, 10, 100, 1),     # ... with the literal sign rule
                                               (1, 1, 0, 5, 10, 60, 0),       # ... alpha_0 = beta_2: a copied row
                                               (4, 1, 2, 12, 128, 40, 0),     # ... the most classes the one-pass kernel takes
                                               (4, 1, 2, 12, 129, 40, 0),     # one class more: two launches
                                               (9, 2, 1, 23, 10, 90, 0)])     # K+E = 11: two launches
def test_locate_decode_one_pass_and_two_launches_agree_with_the_two_steps(K, E, S, W, C, G, flags):
    """approxifer_locate_decode runs as one kernel where the thread-per-class locator can carry the decoding as
    its tail, else as two launches; either way the located sets, trusted masks, decoded values (bit for bit),
    worker counts and status words equal those of approxifer_locate followed by approxifer_decode."""
    Yt, mask, truth = linear_case(K, W, E, S, G, C, seed=K * 100 + C)
    mask[3] = (1 << (2 * (K + E) - 1)) - 1  # one worker short of 2(K+E): nothing located, decoded from all present
    mask[5] = 0                             # nobody answered
    p = ap.make_params(K, W, E, flags | binding.ONE_PASS)
    Yd, md = Yt.to(dev()), ap.mask_tensor(mask)
    n_used = torch.empty(G, dtype=torch.int32, device=dev())
    lst = torch.empty(G, dtype=torch.int32, device=dev())
    dst = torch.empty(G, dtype=torch.int32, device=dev())
    out = torch.full((G, K, C + 3), CANARY, device=dev())  # padded rows: element strides, canaries behind every row
    Yh, adv, trusted = ap.approxifer_locate_decode(p, Yd, md, Yhat=out[:, :, :C], n_used=n_used, locate_status=lst, decode_status=dst)
    lst2 = torch.empty(G, dtype=torch.int32, device=dev())
    adv2, trusted2 = ap.approxifer_locate(p, Yd, md, status=lst2)
    n2 = torch.empty(G, dtype=torch.int32, device=dev())
    dst2 = torch.empty(G, dtype=torch.int32, device=dev())
    Yh2 = ap.approxifer_decode(p, Yd, trusted2, n_used=n2, status=dst2, tuning=ap.decode_tuning(kernel=1))
    assert torch.equal(adv, adv2) and torch.equal(trusted, trusted2) and torch.equal(lst, lst2)
    assert torch.equal(Yh.contiguous().view(torch.int32), Yh2.view(torch.int32))
    assert torch.equal(n_used, n2) and torch.equal(dst, dst2)
    assert bool((out[:, :, C:] == CANARY).all())
    if flags == 0:
        ref = oracle.locate(K, W, E, Yt.numpy(), mask)
        solid = (ref["min_gap"] > 1.0 + 1e-6) & (ref["vote_margin"] > 0) & ((ref["status"] & oracle.ST_ORACLE_RANK_DEFICIENT) == 0)
        solid |= (ref["status"] & oracle.ST_LOCATE_UNDERDETERMINED) != 0
        np.testing.assert_array_equal(adv.cpu().numpy()[solid], ref["adv"][solid])
        check_decode(K, W, Yt, trusted.cpu().numpy().view(np.uint32), Yh, n_used, dst)
    assert int(lst[3]) == 4 and int(n_used[3]) == 2 * (K + E) - 1 and int(dst[5]) & 1


# ------------------------------------------------------------------ randomized shapes

@pytest.mark.parametrize("seed", range(24))
def test_random_shapes_strides_and_alignments(seed):
    """Seeded random (K, W, G, length, padding, base offset): every kernel path (128-bit, element-wise, staged)
    against the oracle, with canaries around and between the rows."""
    rng = np.random.default_rng(1000 + seed)
    K = int(rng.integers(1, 33))
    W = int(rng.integers(2, 33))
    G = int(rng.integers(1, 40))
    L = int(rng.choice([1, 2, 3, 5, 8, 12, 31, 64, 100, 257, 512, 516, 640, 1000, 1028, 2052]))
    pad = int(rng.choice([0, 0, 4, 8, 1, 3]))
    off = int(rng.choice([0, 0, 4, 1]))
    g = torch.Generator().manual_seed(seed)

    def guarded(rows):
        buf = torch.full((off + G * rows * (L + pad) + 7,), CANARY, device=dev())
        view = buf[off: off + G * rows * (L + pad)].view(G, rows, L + pad)[:, :, :L]
        return buf, view

    # encode
    X = torch.rand((G, K, L), generator=g) * 2 - 1
    xin_buf, xin = guarded(K)
    xin.copy_(X.to(dev()))
    out_buf, out = guarded(W)
    ap.approxifer_encode(ap.make_params(K, W), xin, out)
    check_encode(K, W, X, out)
    chk = out_buf.clone()
    chk[off: off + G * W * (L + pad)].view(G, W, L + pad)[:, :, :L] = CANARY
    assert bool((chk == CANARY).all())
    # decode
    Yt = torch.randn((G, W, L), generator=g)
    mask = random_masks(W, G, rng, min_present=0)
    yin_buf, yin = guarded(W)
    yin.copy_(Yt.to(dev()))
    for gi in range(G):  # absent rows hold NaN
        for i in range(W):
            if not (int(mask[gi]) >> i) & 1:
                yin[gi, i] = float("nan")
    yh_buf, yh = guarded(K)
    n_used = torch.empty(G, dtype=torch.int32, device=dev())
    status = torch.empty(G, dtype=torch.int32, device=dev())
    ap.approxifer_decode(ap.make_params(K, W), yin, ap.mask_tensor(mask), yh, n_used=n_used, status=status)
    check_decode(K, W, Yt, mask, yh, n_used, status)
    chk = yh_buf.clone()
    chk[off: off + G * K * (L + pad)].view(G, K, L + pad)[:, :, :L] = CANARY
    assert bool((chk == CANARY).all())
    assert ap.device_wait_timeouts() == 0


@pytest.mark.parametrize("seed", range(12))
def test_random_locator_shapes(seed):
    """Seeded random (K, E, S, C) through both locator kernels' ranges; the located set equals the oracle's on
    every group that is not near-tied, and whatever is returned is a valid answer."""
    rng = np.random.default_rng(500 + seed)
    while True:
        K = int(rng.integers(1, 14))
        E = int(rng.integers(1, 4))
        S = int(rng.integers(0, 4))
        W = 2 * (K + E) + S
        if W <= 32:
            break
    C = int(rng.choice([1, 2, 7, 10, 33, 130]))
    G = int(rng.integers(5, 60))
    Yt, mask, truth = linear_case(K, W, E, S, G, C, seed=seed, softmax=bool(seed % 3 == 0))
    mask[0] = 2**W - 1  # all workers present in one group
    compare_locate(K, W, E, Yt, mask, allow_fragile=True)
