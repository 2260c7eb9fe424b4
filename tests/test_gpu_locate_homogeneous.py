"""GPU parity of the locator's homogeneous form (Algorithm 1 read as a least-squares problem with |Q| = 1,
flag APPROXIFER_LOCATE_HOMOGENEOUS) against its numpy oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from oracle import homogeneous as hom
import paper_2109_09868_b200 as ap
from paper_2109_09868_b200 import binding

pytestmark = pytest.mark.gpu


def dev():
    return torch.device("cuda:0")


def linear_case(K, W, E, S, G, C, seed, softmax=False, sigma=10.0, d_in=16):
    """Honest predictions = linear (optionally + softmax) model of the ORACLE's coded queries,
    E corrupted workers among the W-S present."""
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


def run(K, W, E, Yt, mask):
    G = Yt.shape[0]
    status = torch.empty(G, dtype=torch.int32, device=dev())
    p = ap.make_params(K, W, E, binding.LOCATE_HOMOGENEOUS)
    adv, trusted = ap.approxifer_locate(p, Yt.to(dev()), ap.mask_tensor(mask), status=status)
    torch.cuda.synchronize()
    return adv.cpu().numpy(), trusted.cpu().numpy().view(np.uint32), status.cpu().numpy().view(np.uint32)


def compare(K, W, E, Yt, mask, allow_fragile=False):
    ref = hom.locate_homogeneous(K, W, E, Yt.numpy(), mask)
    adv, trusted, status = run(K, W, E, Yt, mask)
    # groups on which the answer is decided by a clear margin: no near-tie between the E-th and (E+1)-th |a_i|,
    # no tie in the vote, and a smallest singular direction that is separated from the next one
    solid = (ref["min_gap"] > 1.0 + 1e-5) & (ref["vote_margin"] > 0) & (ref["sigma_ratio"] > 1.2)
    solid &= (ref["status"] & oracle.ST_ORACLE_RANK_DEFICIENT) == 0
    solid |= (ref["status"] & oracle.ST_LOCATE_UNDERDETERMINED) != 0
    if not allow_fragile:
        assert solid.all(), "workload has near-tied groups: %d" % int((~solid).sum())
    np.testing.assert_array_equal(adv[solid], ref["adv"][solid])
    np.testing.assert_array_equal(trusted[solid], ref["trusted"][solid])
    np.testing.assert_array_equal(status[solid], ref["status"][solid] & 0xFF)
    for g in range(len(mask)):  # whatever was returned is a valid answer: E distinct present workers, ascending
        if ref["status"][g] & oracle.ST_LOCATE_UNDERDETERMINED:
            continue
        row = adv[g]
        assert np.all(np.diff(row) > 0) and all((int(mask[g]) >> int(i)) & 1 for i in row)
        assert int(trusted[g]) == (int(mask[g]) & (2**W - 1)) & ~sum(1 << int(i) for i in row)
    return ref, adv, int((~solid).sum())


@pytest.mark.parametrize("K,E,S,W", [(8, 2, 2, 24), (2, 1, 0, 6), (3, 2, 1, 12), (4, 1, 2, 12), (6, 3, 1, 20),
                                     (1, 1, 0, 4), (7, 3, 0, 32), (8, 2, 0, 20), (2, 1, 3, 9), (3, 2, 1, 11),
                                     (5, 1, 9, 21), (10, 1, 0, 22), (12, 1, 0, 26), (10, 3, 1, 27)])
def test_homogeneous_locator_matches_oracle_and_finds_injected_errors(K, E, S, W):
    G, C = 96, 10
    Yt, mask, truth = linear_case(K, W, E, S, G, C, seed=K * 37 + E)
    ref, adv, _ = compare(K, W, E, Yt, mask)
    np.testing.assert_array_equal(adv, truth)  # Theorem 1; a node at 0 (odd W) is no obstacle for this form


def test_homogeneous_locator_softmax_model_and_noise_scales():
    K, E, S, W = 8, 2, 2, 24
    for sigma in (1.0, 10.0, 100.0):
        Yt, mask, truth = linear_case(K, W, E, S, 256, 10, seed=int(sigma), softmax=True, sigma=sigma)
        ref, adv, fragile = compare(K, W, E, Yt, mask, allow_fragile=True)
        assert fragile <= 64  # a softmax is not a rational function: some directions are poorly separated
        assert (adv == truth).all(axis=1).mean() > 0.9


def test_homogeneous_locator_underdetermined_groups_one_class_and_many_classes():
    K, E, S, W = 4, 1, 1, 12
    for C in (1, 3, 130):
        Yt, mask, truth = linear_case(K, W, E, S, 40, C, seed=C)
        mask[3] = 0x1FF  # 9 workers < 2(K+E)
        mask[4] = 0
        ref, adv, _ = compare(K, W, E, Yt, mask)
        assert adv[3, 0] == -1 and adv[4, 0] == -1


def test_a_corrupted_worker_at_node_zero_is_found():
    """W odd puts beta = 0 in the middle.  With Q_0 = 1 that worker's a_i is pinned to 1 (it can never be a root
    of Q); the homogeneous form has no such special case: there a_i is ~0 at the corrupted worker."""
    K, E, W, G, C = 3, 1, 9, 64, 6
    Yt, _, _ = linear_case(K, W, 1, 0, G, C, seed=77, sigma=0.0)
    mid = (W - 1) // 2
    rng = np.random.default_rng(3)
    Yt = Yt.clone()
    Yt[:, mid] += torch.from_numpy((5.0 * rng.standard_normal((G, C))).astype(np.float32))
    mask = np.full(G, (1 << W) - 1, dtype=np.uint32)
    ref, adv, _ = compare(K, W, E, Yt, mask)
    assert np.all(adv[:, 0] == mid)
    assert ref["min_gap"].min() > 100.0


def test_homogeneous_form_is_refused_beyond_its_range():
    p = ap.make_params(12, 32, 2, binding.LOCATE_HOMOGENEOUS)
    with pytest.raises(ap.ApproxiferError):
        ap.approxifer_locate(p, torch.zeros((1, 32, 4), device=dev()), ap.mask_tensor(np.array([0xFFFFFFFF], dtype=np.uint32)))


def test_workload5_full_size_homogeneous_form():
    """The Byzantine workload at its full size (65,536 groups, the launch configuration the benchmark times):
    every located set equals the injected one (Theorem 1: the honest predictions are a rational function), and
    a sample of every 32nd group is compared with the oracle, which is too slow for all of them."""
    from paper_2109_09868_b200 import workloads as wl

    w = wl.workload(5)
    Xh = wl.queries(w, "cpu")
    Xc = torch.from_numpy(oracle.encode(w.K, w.W, Xh.numpy()).astype(np.float32))
    Yt = wl.apply_model(w, Xc)
    mask = wl.masks(w)
    truth = wl.adversaries(w, mask)
    wl.corrupt(w, Yt, truth)
    adv, trusted, status = run(w.K, w.W, w.E, Yt, mask)
    np.testing.assert_array_equal(adv, truth)
    assert np.all(status == 0)
    sel = np.arange(0, w.G, 32)
    ref = hom.locate_homogeneous(w.K, w.W, w.E, Yt.numpy()[sel], mask[sel])
    assert ref["min_gap"].min() > 1.5 and np.all(ref["vote_margin"] > 0) and np.all(ref["status"] == 0)
    np.testing.assert_array_equal(adv[sel], ref["adv"])
    np.testing.assert_array_equal(trusted[sel], ref["trusted"])


def test_homogeneous_flag_through_the_one_call_and_host_buffer_entry_points():
    """approxifer_locate_decode and approxifer_locate_host honour the flag: same sets as approxifer_locate with
    it, and the decoded predictions equal a separate decode from those trusted workers (the decoder ignores the flag)."""
    K, E, S, W, G, C = 4, 2, 1, 13, 70, 6
    Yt, mask, truth = linear_case(K, W, E, S, G, C, seed=5)
    p = ap.make_params(K, W, E, binding.LOCATE_HOMOGENEOUS)
    Yd, md = Yt.to(dev()), ap.mask_tensor(mask)
    adv, trusted = ap.approxifer_locate(p, Yd, md)
    Yh, adv1, trusted1 = ap.approxifer_locate_decode(p, Yd, md)
    assert torch.equal(adv, adv1) and torch.equal(trusted, trusted1)
    assert torch.equal(Yh, ap.approxifer_decode(ap.make_params(K, W), Yd, trusted))
    np.testing.assert_array_equal(adv.cpu().numpy(), truth)
    hYt = Yt.pin_memory()
    hmask = torch.from_numpy(mask.view(np.int32).copy()).pin_memory()
    hadv = torch.empty((G, E), dtype=torch.int32).pin_memory()
    htr = torch.empty((G,), dtype=torch.int32).pin_memory()
    ws = torch.empty(1 << 20, dtype=torch.uint8, device=dev())
    streams = [torch.cuda.Stream() for _ in range(2)]
    ap.approxifer_locate_host(p, hYt, hmask, hadv, htr, ws, streams)
    for st in streams:
        st.synchronize()
    assert torch.equal(hadv, adv.cpu()) and torch.equal(htr, trusted.cpu())
