"""bfloat16 payload variants of the encoder and the decoder against the oracle (Section 3, "ApproxIFER
Encoding" / "ApproxIFER Decoding", step 2, on bfloat16-stored values).

The oracle widens the stored values exactly, evaluates the formulas in fp64 and rounds once to the nearest
bfloat16 (ties to even).  The kernel rounds an fp32 value that is itself within the fp32 tolerance of the exact
one, so every element must satisfy
    |out - exact| <= 2^-8 |exact| + tol32 + 2^-134,
tol32 = 1e-5 max|X| for the encoder, 1e-4 max|Yhat_exact| of the group for the decoder: half a unit in the last
of bfloat16's 8 significant bits, plus the fp32 tolerance of the same operation.  Where the fp32 value is not
within fp32 rounding distance of a bfloat16 tie, the result is the oracle's rounding bit for bit: checked as a
count (almost all elements)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2109_09868_b200 as ap

pytestmark = pytest.mark.gpu


def dev():
    return torch.device("cuda:0")


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def from_bits(b: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(b.view(np.int16).copy()).view(torch.bfloat16)


def random_masks(W, G, rng, min_present):
    m = rng.integers(0, 2**W, size=G, dtype=np.uint64)
    for g in range(G):
        while bin(int(m[g])).count("1") < min_present:
            m[g] |= np.uint64(1) << np.uint64(rng.integers(0, W))
    return m.astype(np.uint32)


ENCODE_CASES = [
    (8, 12, 40, 3072),     # configs[1] shape
    (12, 20, 2, 150528),   # configs[2] shape
    (4, 5, 256, 784),      # configs[0] shape
    (16, 24, 33, 32),
    (3, 7, 5, 1000),       # coincident nodes: rows 1, 3, 5 are copies (exact in bfloat16 too)
    (5, 9, 11, 13),        # odd length: element-wise path
    (32, 32, 3, 260),
]


@pytest.mark.parametrize("K,W,G,D", ENCODE_CASES)
def test_encode_bf16_matches_oracle(K, W, G, D):
    rng = np.random.default_rng(K * 100 + D)
    Xb = oracle.bf16_round(rng.random((G, K, D)) * 4 - 1)
    exact, rounded = oracle.encode_bf16(K, W, Xb)
    out = ap.approxifer_encode_bf16(ap.make_params(K, W), from_bits(Xb).to(dev()))
    got_bits = bits_of(out)
    got = oracle.bf16_widen(got_bits).astype(np.float64)
    xmax = float(np.abs(oracle.bf16_widen(Xb)).max())
    bound = 2.0 ** -8 * np.abs(exact) + 1e-5 * xmax + 2.0 ** -134
    assert np.all(np.abs(got - exact) <= bound), float((np.abs(got - exact) - bound).max())
    assert np.mean(got_bits == rounded) > 0.995
    if (K, W) == (3, 7):
        for j, i in ((0, 1), (1, 3), (2, 5)):
            assert np.array_equal(got_bits[:, i], Xb[:, j])


def test_encode_bf16_strided_misaligned_and_guarded():
    K, W, G, D = 8, 12, 9, 100
    rng = np.random.default_rng(4)
    Xb = oracle.bf16_round(rng.standard_normal((G, K, D)))
    exact, rounded = oracle.encode_bf16(K, W, Xb)
    p = ap.make_params(K, W)
    # (a) a view that starts 2 bytes into an allocation: element-wise path; (b) padded rows; (c) worker-major output
    base = torch.zeros(G * K * D + 8, dtype=torch.bfloat16, device=dev())
    base[1: 1 + G * K * D] = from_bits(Xb).to(dev()).reshape(-1)
    x_a = base[1: 1 + G * K * D].view(G, K, D)
    canary = from_bits(np.full((G, W, D + 8), 0x7F7F, dtype=np.uint16)).to(dev())
    ap.approxifer_encode_bf16(p, x_a, canary[:, :, 4: 4 + D])
    got = bits_of(canary)
    assert np.all(got[:, :, :4] == 0x7F7F) and np.all(got[:, :, 4 + D:] == 0x7F7F)
    wide = oracle.bf16_widen(got[:, :, 4: 4 + D]).astype(np.float64)
    bound = 2.0 ** -8 * np.abs(exact) + 1e-5 * float(np.abs(oracle.bf16_widen(Xb)).max())
    assert np.all(np.abs(wide - exact) <= bound)
    wm = torch.empty((W, G, D), dtype=torch.bfloat16, device=dev())
    ap.approxifer_encode_bf16(p, from_bits(Xb).to(dev()), wm.permute(1, 0, 2))
    assert np.array_equal(bits_of(wm.permute(1, 0, 2)), got[:, :, 4: 4 + D])


DECODE_CASES = [
    (8, 12, 300, 10),      # configs[1] shape
    (12, 20, 30, 1000),    # configs[2] shape
    (16, 24, 21, 1000),    # configs[3] shape
    (8, 24, 100, 10),      # configs[4] shape
    (3, 7, 50, 36),        # coincident nodes
    (5, 9, 17, 33),        # odd length: element-wise path
    (32, 32, 5, 64),
    (8, 12, 60, 128),      # the shortest rows the bulk-copy staged kernel takes with bfloat16 payloads
    (16, 24, 9, 2056),     # several 256-column tiles per row and a ragged last one
    (12, 20, 40, 1004),    # 1004 is not a multiple of 8: per-column kernel
]


@pytest.mark.parametrize("K,W,G,C", DECODE_CASES)
def test_decode_bf16_matches_oracle(K, W, G, C):
    rng = np.random.default_rng(K * 100 + C)
    Yb = oracle.bf16_round(rng.standard_normal((G, W, C)))
    mask = random_masks(W, G, rng, min_present=0)
    mask[0], mask[1] = 0, 2**W - 1
    dirty = Yb.copy()
    for g in range(G):
        for i in range(W):
            if not (int(mask[g]) >> i) & 1:
                dirty[g, i] = 0x7FC0  # NaN: absent rows must never be used
    exact, rounded, n_ref, st_ref = oracle.decode_bf16(K, W, Yb, mask)
    n_used = torch.empty(G, dtype=torch.int32, device=dev())
    status = torch.empty(G, dtype=torch.int32, device=dev())
    out = ap.approxifer_decode_bf16(ap.make_params(K, W), from_bits(dirty).to(dev()), ap.mask_tensor(mask), n_used=n_used, status=status)
    got_bits = bits_of(out)
    got = oracle.bf16_widen(got_bits).astype(np.float64)
    assert np.isfinite(got).all()
    scale = np.abs(exact).reshape(G, -1).max(axis=1)[:, None, None]
    bound = 2.0 ** -8 * np.abs(exact) + 1e-4 * scale + 2.0 ** -134
    assert np.all(np.abs(got - exact) <= bound), float((np.abs(got - exact) - bound).max())
    assert np.mean(got_bits == rounded) > 0.99
    np.testing.assert_array_equal(n_used.cpu().numpy(), n_ref)
    np.testing.assert_array_equal(status.cpu().numpy().view(np.uint32), st_ref)


def test_decode_bf16_worker_major_and_padded_output():
    K, W, G, C = 8, 12, 40, 100
    rng = np.random.default_rng(8)
    Yb = oracle.bf16_round(rng.standard_normal((G, W, C)))
    mask = random_masks(W, G, rng, min_present=K)
    exact, rounded, _, _ = oracle.decode_bf16(K, W, Yb, mask)
    p = ap.make_params(K, W)
    dense = ap.approxifer_decode_bf16(p, from_bits(Yb).to(dev()), ap.mask_tensor(mask))
    wm = from_bits(Yb).to(dev()).permute(1, 0, 2).contiguous()  # [W][G][C]
    out = from_bits(np.full((G, K, C + 4), 0x7F7F, dtype=np.uint16)).to(dev())
    ap.approxifer_decode_bf16(p, wm.permute(1, 0, 2), ap.mask_tensor(mask), out[:, :, :C])
    got = bits_of(out)
    assert np.all(got[:, :, C:] == 0x7F7F)
    assert np.array_equal(got[:, :, :C], bits_of(dense))
    assert np.mean(got[:, :, :C] == rounded) > 0.99
