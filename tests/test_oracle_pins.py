"""Pins of the CPU oracle against what the paper and the mathematics fix.

No GPU needed.  Every check compares the oracle with something other than
itself: closed forms, invariants of Berrut's interpolant (Eq. 1-2), an
exact-rational evaluation of a differently written formula, an independent
least-squares routine, and Theorem 1's constructive guarantee.
"""
import itertools
import os
from fractions import Fraction

import mpmath
import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
ULP = np.finfo(np.float64).eps


# --------------------------------------------------------------------- nodes

def test_alpha_closed_forms():
    s2, s3, s6 = np.sqrt(2.0), np.sqrt(3.0), np.sqrt(6.0)
    np.testing.assert_allclose(oracle.alpha(1), [0.0], atol=0)
    np.testing.assert_allclose(oracle.alpha(2), [s2 / 2, -s2 / 2], rtol=2 * ULP)
    np.testing.assert_allclose(oracle.alpha(3), [s3 / 2, 0.0, -s3 / 2], rtol=2 * ULP)
    c1, c3 = np.sqrt(2 + s2) / 2, np.sqrt(2 - s2) / 2  # cos(pi/8), cos(3pi/8)
    np.testing.assert_allclose(oracle.alpha(4), [c1, c3, -c3, -c1], rtol=4 * ULP)
    np.testing.assert_allclose(
        oracle.alpha(6), [(s6 + s2) / 4, s2 / 2, (s6 - s2) / 4, -(s6 - s2) / 4, -s2 / 2, -(s6 + s2) / 4], rtol=4 * ULP
    )


def test_beta_closed_forms():
    s2, s3 = np.sqrt(2.0), np.sqrt(3.0)
    assert list(oracle.beta(2)) == [1.0, -1.0]
    assert list(oracle.beta(3)) == [1.0, 0.0, -1.0]
    np.testing.assert_allclose(oracle.beta(4), [1.0, 0.5, -0.5, -1.0], rtol=2 * ULP)
    np.testing.assert_allclose(oracle.beta(5), [1.0, s2 / 2, 0.0, -s2 / 2, -1.0], rtol=2 * ULP)
    np.testing.assert_allclose(oracle.beta(7), [1.0, s3 / 2, 0.5, 0.0, -0.5, -s3 / 2, -1.0], rtol=2 * ULP, atol=0)


def _cheb(n, x, kind):
    """T_n(x) (kind 1) or U_n(x) (kind 2) by the three-term recurrence, exactly."""
    x = Fraction(float(x))
    p0, p1 = Fraction(1), (x if kind == 1 else 2 * x)
    if n == 0:
        return p0
    for _ in range(n - 1):
        p0, p1 = p1, 2 * x * p1 - p0
    return p1


@pytest.mark.parametrize("n", range(1, 33))
def test_nodes_are_chebyshev_roots_and_extrema(n):
    """alpha are the K roots of T_K in decreasing order; beta are the W extrema
    of T_{W-1}, T_{W-1}(beta_i) = (-1)^i, in decreasing order."""
    a = oracle.alpha(n)
    assert np.all(np.diff(a) < 0)
    np.testing.assert_array_equal(a, -a[::-1])
    for v in a:
        t = float(_cheb(n, v, 1))
        assert abs(t) <= n * n * ULP  # |T_n'| <= n^2 on [-1,1]
    if n >= 2:
        b = oracle.beta(n)
        assert np.all(np.diff(b) < 0)
        np.testing.assert_array_equal(b, -b[::-1])
        for i, v in enumerate(b):
            t = float(_cheb(n - 1, v, 1))
            assert abs(t - (-1) ** i) <= 4 * (n * n) ** 2 * ULP
            # and it is a stationary point: U_{n-2}(beta_i) = 0 for interior nodes
            if 0 < i < n - 1:
                assert abs(float(_cheb(n - 2, v, 2))) <= 4 * n * n * ULP


def test_coincidence_is_the_integer_identity():
    for K in range(1, 33):
        for W in range(2, 33):
            a = [mpmath.cos(mpmath.pi * (2 * j + 1) / (2 * K)) for j in range(K)]
            b = [mpmath.cos(mpmath.pi * i / (W - 1)) for i in range(W)]
            for j in range(K):
                for i in range(W):
                    exact = Fraction(2 * j + 1, 2 * K) == Fraction(i, W - 1)
                    assert oracle.coincident(K, W, j, i) == exact
                    if not exact:
                        assert abs(a[j] - b[i]) > 1e-5
    # examples named in the design notes
    assert [(j, i) for j in range(3) for i in range(7) if oracle.coincident(3, 7, j, i)] == [(0, 1), (1, 3), (2, 5)]
    assert not any(oracle.coincident(K, W, j, i) for (K, W) in [(4, 5), (8, 12), (12, 20), (16, 24), (8, 24)]
                   for j in range(K) for i in range(W))


# ---------------------------------------------------- P1 partition of unity

def test_encode_weights_sum_to_one():
    for K in range(1, 33):
        for W in range(2, 33):
            e = oracle.encode_weights(K, W)
            assert np.all(np.abs(e.sum(axis=1) - 1.0) <= 64 * ULP * np.abs(e).sum(axis=1))


def test_decode_weights_sum_to_one_random_masks():
    rng = np.random.default_rng(1)
    for _ in range(2000):
        K = int(rng.integers(1, 33))
        W = int(rng.integers(2, 33))
        mask = int(rng.integers(1, 2**W))
        for flags in (0, 1):
            w, F = oracle.decode_weights(K, W, mask, flags)
            assert F == [i for i in range(W) if mask >> i & 1]
            assert w.shape == (K, len(F))
            if flags == 0:
                assert np.all(np.abs(w.sum(axis=1) - 1.0) <= 64 * ULP * np.abs(w).sum(axis=1))


def test_constants_are_reproduced():
    rng = np.random.default_rng(2)
    for (K, W) in [(1, 2), (4, 5), (8, 12), (3, 7), (12, 20), (32, 32)]:
        c = rng.standard_normal(5).astype(np.float32)
        X = np.broadcast_to(c, (3, K, 5)).copy()
        Xt = oracle.encode(K, W, X)
        np.testing.assert_allclose(Xt, np.broadcast_to(c.astype(np.float64), Xt.shape), rtol=1e-13)
        Y = np.broadcast_to(c, (3, W, 5)).copy()
        mask = rng.integers(1, 2**W, size=3).astype(np.uint32)
        Yh, n_used, status = oracle.decode(K, W, Y, mask)
        np.testing.assert_allclose(Yh, np.broadcast_to(c.astype(np.float64), Yh.shape), rtol=1e-12)


# ------------------------------------------------- P2 interpolation at nodes

def test_berrut_returns_node_values_and_stays_in_hull_for_two_nodes():
    x = np.array([1.0, 0.3, -0.2, -0.9])
    f = np.array([2.0, -1.0, 0.5, 4.0])
    for k in range(4):
        assert oracle.berrut(x, f, x[k]) == f[k]
        # approaching the node: the interpolant is continuous there
        assert abs(oracle.berrut(x, f, x[k] + 1e-9) - f[k]) < 1e-6
    # two nodes: Berrut's interpolant is the straight line through them
    for z in (-0.7, 0.0, 0.25, 0.9):
        line = f[0] + (z - x[0]) / (x[1] - x[0]) * (f[1] - f[0])
        assert abs(oracle.berrut(x[:2], f[:2], z) - line) < 1e-14


def test_encode_passes_through_queries_at_coincident_nodes():
    rng = np.random.default_rng(3)
    X = rng.random((4, 3, 9), dtype=np.float32)
    Xt = oracle.encode(3, 7, X)
    for (j, i) in [(0, 1), (1, 3), (2, 5)]:
        np.testing.assert_array_equal(Xt[:, i, :], X[:, j, :].astype(np.float64))
    # K = 1: u is the constant X_0
    X1 = rng.random((2, 1, 6), dtype=np.float32)
    for W in (2, 3, 8):
        Xt1 = oracle.encode(1, W, X1)
        for i in range(W):
            np.testing.assert_array_equal(Xt1[:, i, :], X1[:, 0, :].astype(np.float64))


def test_decode_returns_prediction_at_coincident_node_if_present():
    rng = np.random.default_rng(4)
    Y = rng.standard_normal((1, 7, 5)).astype(np.float32)
    full = np.array([0x7F], dtype=np.uint32)
    Yh, _, _ = oracle.decode(3, 7, Y, full)
    for (j, i) in [(0, 1), (1, 3), (2, 5)]:
        np.testing.assert_array_equal(Yh[0, j], Y[0, i].astype(np.float64))
    # worker 3 absent: alpha_1 = 0 is no longer a node, the value is interpolated
    part = np.array([0x7F & ~(1 << 3)], dtype=np.uint32)
    Yh2, n_used, _ = oracle.decode(3, 7, Y, part)
    assert n_used[0] == 6
    np.testing.assert_array_equal(Yh2[0, 0], Y[0, 1].astype(np.float64))
    nodes = oracle.beta(7)[[0, 1, 2, 4, 5, 6]]
    for c in range(5):
        ref = oracle.berrut(nodes, Y[0, [0, 1, 2, 4, 5, 6], c].astype(np.float64), 0.0)
        assert abs(Yh2[0, 1, c] - ref) < 1e-14


# ----------------------------------------------------- P3 closed form K = 2

def test_encode_weights_closed_form_K2_W3():
    rows = np.loadtxt(os.path.join(GOLDEN, "encode_weights_K2_W3.txt"))
    e = oracle.encode_weights(2, 3)
    np.testing.assert_allclose(e, rows[:, 1:], rtol=0, atol=4 * ULP)


def test_encode_K2_is_the_chord_through_the_two_queries():
    # l_0(z) = (z+a)/(2a), l_1(z) = (a-z)/(2a): u is the line through (a, X_0), (-a, X_1)
    a = np.sqrt(2.0) / 2
    for W in range(2, 33):
        b = oracle.beta(W)
        e = oracle.encode_weights(2, W)
        np.testing.assert_allclose(e[:, 0], (b + a) / (2 * a), atol=8 * ULP)
        np.testing.assert_allclose(e[:, 1], (a - b) / (2 * a), atol=8 * ULP)


# -------------------------------------- P4 two workers / one worker / round trip

def test_decode_from_two_workers_is_linear_interpolation():
    for (K, W) in [(2, 5), (4, 9), (8, 12), (5, 32)]:
        al, be = oracle.alpha(K), oracle.beta(W)
        for (p, q) in itertools.combinations(range(W), 2):
            w, F = oracle.decode_weights(K, W, (1 << p) | (1 << q))
            assert F == [p, q]
            for j in range(K):
                if oracle.coincident(K, W, j, p) or oracle.coincident(K, W, j, q):
                    continue
                lam = (al[j] - be[p]) / (be[q] - be[p])
                np.testing.assert_allclose(w[j], [1 - lam, lam], rtol=1e-12, atol=1e-14)


def test_literal_sign_differs_on_noncontiguous_sets():
    # workers 0 and 2 are both even: the literal sign (-1)^i gives the two terms
    # the same sign, which is not an interpolant with alternating signs any more
    w_rank, _ = oracle.decode_weights(2, 5, 0b00101, 0)
    w_lit, _ = oracle.decode_weights(2, 5, 0b00101, 1)
    assert np.max(np.abs(w_rank - w_lit)) > 0.1
    # on a contiguous run they agree
    for mask in (0b00110, 0b01110, 0b11111, 0b11100):
        a, _ = oracle.decode_weights(3, 5, mask, 0)
        b, _ = oracle.decode_weights(3, 5, mask, 1)
        np.testing.assert_allclose(a, b, rtol=1e-15)


def test_K2_round_trip_identity_model():
    rng = np.random.default_rng(5)
    X = rng.random((1, 2, 4), dtype=np.float32)
    for W in (3, 4, 6):
        Xt = oracle.encode(2, W, X)[0]  # [W][4] double; u is linear for K = 2
        for (p, q) in itertools.combinations(range(W), 2):
            w, F = oracle.decode_weights(2, W, (1 << p) | (1 << q))
            back = w @ Xt[F]
            np.testing.assert_allclose(back, X[0].astype(np.float64), rtol=1e-12, atol=1e-13)


def test_single_worker_is_copied_and_empty_mask_gives_zeros():
    rng = np.random.default_rng(6)
    Y = rng.standard_normal((3, 6, 4)).astype(np.float32)
    mask = np.array([1 << 4, 0, 0b111111], dtype=np.uint32)
    Yh, n_used, status = oracle.decode(3, 6, Y, mask)
    for j in range(3):
        np.testing.assert_array_equal(Yh[0, j], Y[0, 4].astype(np.float64))
    assert list(n_used) == [1, 0, 6]
    assert status[0] == oracle.ST_FEW_WORKERS
    assert status[1] == oracle.ST_NO_WORKERS | oracle.ST_FEW_WORKERS
    assert status[2] == 0
    assert np.all(Yh[1] == 0.0)


def test_mask_bits_beyond_W_are_ignored_and_absent_rows_untouched():
    rng = np.random.default_rng(7)
    Y = rng.standard_normal((1, 5, 3)).astype(np.float32)
    Y2 = Y.copy()
    Y2[0, 2] = np.nan  # absent worker holds garbage
    m = np.array([0b11011], dtype=np.uint32)
    a, _, _ = oracle.decode(4, 5, Y, m)
    b, n_used, _ = oracle.decode(4, 5, Y2, m | np.uint32(0xFFFFFFE0))
    assert n_used[0] == 4
    np.testing.assert_array_equal(a, b)


# --------------------------------------------------------------- P5 symmetry

def test_encode_weight_symmetry_and_K4_W5_closed_form():
    for K in range(1, 33):
        for W in (2, 5, 12, 20, 24, 31, 32):
            e = oracle.encode_weights(K, W)
            np.testing.assert_allclose(e, e[::-1, ::-1], rtol=1e-12, atol=1e-15)
    # K=4, W=5 from radicals, evaluated with 40 digits, with the polynomial form
    # of Berrut's weights (numerator prod_{l != j}(z - alpha_l), no reciprocals)
    mpmath.mp.dps = 40
    s2 = mpmath.sqrt(2)
    al = [mpmath.sqrt(2 + s2) / 2, mpmath.sqrt(2 - s2) / 2, -mpmath.sqrt(2 - s2) / 2, -mpmath.sqrt(2 + s2) / 2]
    be = [mpmath.mpf(1), s2 / 2, mpmath.mpf(0), -s2 / 2, mpmath.mpf(-1)]
    e = oracle.encode_weights(4, 5)
    for i in range(5):
        terms = [(-1) ** j * mpmath.fprod(be[i] - al[l] for l in range(4) if l != j) for j in range(4)]
        tot = mpmath.fsum(terms)
        for j in range(4):
            assert abs(e[i, j] - terms[j] / tot) < 1e-15
    assert abs(e[0, 0] - 1.120853) < 1e-6 and abs(e[2, 1] - 0.853553) < 1e-6 and e[0, 1] < 0


# -------------------------------------------------- P6 exact-rational brute force

def _exact_interpolant(nodes, signs, values, z):
    """Exact value of sum_k s_k v_k/(z-x_k) / sum_k s_k/(z-x_k) written without
    reciprocals: multiply both by prod_l (z - x_l)."""
    n = len(nodes)
    num = Fraction(0)
    den = Fraction(0)
    for k in range(n):
        prod = Fraction(1)
        for l in range(n):
            if l != k:
                prod *= z - nodes[l]
        num += signs[k] * values[k] * prod
        den += signs[k] * prod
    return num / den


def test_encode_decode_match_exact_rational_arithmetic():
    rng = np.random.default_rng(8)
    for (K, W) in [(1, 2), (2, 3), (2, 4), (3, 4), (3, 6), (4, 5), (4, 6)]:
        al = [Fraction(float(v)) for v in oracle.alpha(K)]
        be = [Fraction(float(v)) for v in oracle.beta(W)]
        X = (rng.random((1, K, 3), dtype=np.float32) * 4 - 2).astype(np.float32)
        Xt = oracle.encode(K, W, X)
        for i in range(W):
            if any(oracle.coincident(K, W, j, i) for j in range(K)):
                continue
            for d in range(3):
                ex = _exact_interpolant(al, [(-1) ** j for j in range(K)], [Fraction(float(X[0, j, d])) for j in range(K)], be[i])
                scale = max(1.0, float(np.abs(X[0, :, d]).max()))
                assert abs(float(Fraction(float(Xt[0, i, d])) - ex)) <= 64 * ULP * scale * 10
        Y = (rng.standard_normal((1, W, 3)) * 3).astype(np.float32)
        for mask in range(1, 2**W):
            F = [i for i in range(W) if mask >> i & 1]
            Yh, _, _ = oracle.decode(K, W, Y, np.array([mask], dtype=np.uint32))
            for j in range(K):
                if any(oracle.coincident(K, W, j, i) for i in F):
                    continue
                for d in range(3):
                    ex = _exact_interpolant([be[i] for i in F], [(-1) ** r for r in range(len(F))],
                                            [Fraction(float(Y[0, i, d])) for i in F], al[j])
                    wsum = float(np.abs(oracle.decode_weights(K, W, mask)[0][j]).sum())
                    scale = max(1.0, float(np.abs(Y[0, :, d]).max())) * wsum
                    assert abs(float(Fraction(float(Yh[0, j, d])) - ex)) <= 256 * ULP * scale


# ----------------------------------------------------------- P9 no real poles

def test_rank_sign_keeps_lebesgue_constant_small_literal_sign_does_not():
    worst_rank, worst_lit = 0.0, 0.0
    for (K, W) in [(4, 5), (4, 8), (6, 10), (8, 12)]:
        for mask in range(1, 2**W):
            if bin(mask).count("1") < K:
                continue
            w0, _ = oracle.decode_weights(K, W, mask, 0)
            worst_rank = max(worst_rank, np.abs(w0).sum(axis=1).max())
            if W <= 10:
                w1, _ = oracle.decode_weights(K, W, mask, 1)
                worst_lit = max(worst_lit, np.abs(w1).sum(axis=1).max())
    assert worst_rank < 20.0
    assert worst_lit > 10 * worst_rank


# ------------------------------------------------ P8 locator vs generic least squares

def _system(m, xs, y):
    V = np.vander(xs, m, increasing=True)
    return np.hstack([V, -y[:, None] * V[:, 1:]]), y.copy()


def test_locate_class_matches_numpy_lstsq():
    rng = np.random.default_rng(9)
    for (K, E, W) in [(2, 1, 6), (3, 1, 9), (4, 2, 13), (8, 2, 24), (12, 2, 32), (8, 2, 22)]:
        m = K + E
        be = oracle.beta(W)
        for _ in range(5):
            n = int(rng.integers(2 * m, W + 1))
            F = np.sort(rng.choice(W, size=n, replace=False))
            xs = be[F]
            y = rng.standard_normal(n)
            x, a, rank = oracle.locate_class(m, xs, y)
            A, b = _system(m, xs, y)
            ref, *_ = np.linalg.lstsq(A, b, rcond=None)
            assert rank == 2 * m - 1
            cond = np.linalg.cond(A)
            np.testing.assert_allclose(x, ref, rtol=0, atol=1e-13 * cond * max(1.0, np.abs(ref).max()))
            a_ref = 1.0 + np.vander(xs, m, increasing=True)[:, 1:] @ ref[m:]
            np.testing.assert_allclose(a, a_ref, rtol=0, atol=1e-12 * cond * max(1.0, np.abs(a_ref).max()))
            # residual is orthogonal to the column space (normal equations)
            r = A @ x - b
            assert np.abs(A.T @ r).max() <= 1e-10 * np.linalg.norm(A, 2) * max(1.0, np.linalg.norm(b))


def test_locate_class_solves_a_consistent_system_exactly_rational():
    """Theorem 1, tiny and exact: y_i = p(x_i)/q(x_i) with deg p, q <= K-1 except
    at one corrupted node x_e; then P = p*Lambda/q(0), Q = q*Lambda/q(0) with
    Lambda(x) = 1 - x/x_e solves every equation, and a_e = 0."""
    K, E, W = 2, 1, 6
    m = K + E
    be = [Fraction(float(v)) for v in oracle.beta(W)]
    p = [Fraction(3, 2), Fraction(-1, 3)]
    q = [Fraction(2), Fraction(1, 2)]
    e = 4
    y = [(p[0] + p[1] * x) / (q[0] + q[1] * x) for x in be]
    y[e] += Fraction(7, 3)
    lam = [Fraction(1), -1 / be[e]]
    P = [p[0] * lam[0], p[0] * lam[1] + p[1] * lam[0], p[1] * lam[1]]
    Q = [q[0] * lam[0], q[0] * lam[1] + q[1] * lam[0], q[1] * lam[1]]
    P = [c / Q[0] for c in P]
    Q = [c / Q[0] for c in Q]
    for i in range(W):  # the claimed solution satisfies P(x_i) = y_i Q(x_i) exactly
        Pv = sum(P[k] * be[i] ** k for k in range(m))
        Qv = sum(Q[k] * be[i] ** k for k in range(m))
        assert Pv == y[i] * Qv
    x, a, rank = oracle.locate_class(m, [float(v) for v in be], [float(v) for v in y])
    assert rank == 2 * m - 1
    expect = [float(c) for c in P] + [float(c) for c in Q[1:]]
    np.testing.assert_allclose(x, expect, rtol=0, atol=1e-11)
    assert abs(a[e]) < 1e-12
    assert min(abs(a[i]) for i in range(W) if i != e) > 1e-2


# ----------------------------------------------- P7 Theorem 1 through Algorithm 2

def _linear_predictions(K, W, G, C, rng, d_in=6):
    X = rng.random((G, K, d_in), dtype=np.float32)
    M = rng.standard_normal((d_in, C))
    Xt = oracle.encode(K, W, X)  # float64: f(u(beta_i)) = M^T u(beta_i) is rational of type (K-1, K-1)
    return (Xt @ M).astype(np.float32)


@pytest.mark.parametrize("K,E,S", [(2, 1, 0), (3, 2, 1), (4, 1, 2), (8, 2, 2), (12, 2, 0), (6, 3, 1)])
def test_locate_finds_injected_errors_for_a_linear_model(K, E, S):
    rng = np.random.default_rng(100 + K * 10 + E)
    W = 2 * (K + E) + S
    if W % 2 == 1:
        W += 1  # an odd W puts a node at 0, which Q(0)=1 can never flag
    G, C = 40, 5
    Y = _linear_predictions(K, W, G, C, rng)
    mask = np.empty(G, dtype=np.uint32)
    truth = np.empty((G, E), dtype=np.int32)
    for g in range(G):
        present = np.sort(rng.choice(W, size=W - S, replace=False))
        mask[g] = sum(1 << int(i) for i in present)
        bad = np.sort(rng.choice(present, size=E, replace=False))
        truth[g] = bad
        Y[g, bad] += (10.0 * rng.standard_normal((E, C))).astype(np.float32)
    out = oracle.locate(K, W, E, Y, mask)
    np.testing.assert_array_equal(out["adv"], truth)
    for g in range(G):
        assert int(out["trusted"][g]) == int(mask[g]) & ~sum(1 << int(i) for i in truth[g])
    assert np.all(out["status"] == 0)
    assert out["min_gap"].min() > 2.0
    assert np.all(out["vote_margin"] == C)


def test_locate_underdetermined_and_tie_rules():
    rng = np.random.default_rng(11)
    K, E, W, C = 2, 1, 6, 2
    Y = _linear_predictions(K, W, 3, C, rng)
    # group 0: only 5 < 2(K+E) workers -> nothing located
    # group 1: class 0 corrupted at worker 4, class 1 at worker 1 -> one vote each, lower index wins
    # group 2: both classes corrupted at worker 3
    Y[1, 4, 0] += 5.0
    Y[1, 1, 1] -= 7.0
    Y[2, 3, :] += 4.0
    mask = np.array([0b011111, 0b111111, 0xFFFFFFFF], dtype=np.uint32)
    out = oracle.locate(K, W, E, Y, mask)
    assert out["adv"][0, 0] == -1 and out["trusted"][0] == 0b011111
    assert out["status"][0] == oracle.ST_LOCATE_UNDERDETERMINED
    assert out["adv"][1, 0] == 1 and out["vote_margin"][1] == 0
    assert out["trusted"][1] == 0b111101
    assert out["adv"][2, 0] == 3 and out["vote_margin"][2] == 2
    assert out["trusted"][2] == 0b110111  # bits >= W dropped


def test_locate_then_decode_recovers_linear_predictions():
    """End to end on a rational model: after removing the located workers, the
    decoder's error is the plain approximation error of Berrut's interpolant,
    far below the injected noise."""
    rng = np.random.default_rng(12)
    K, E, S, W, G, C = 8, 2, 2, 24, 30, 10
    X = rng.random((G, K, 16), dtype=np.float32)
    M = rng.standard_normal((16, C)) / 4
    Y = (oracle.encode(K, W, X) @ M).astype(np.float32)
    clean = X.astype(np.float64) @ M
    mask = np.empty(G, dtype=np.uint32)
    for g in range(G):
        present = np.sort(rng.choice(W, size=W - S, replace=False))
        mask[g] = sum(1 << int(i) for i in present)
        bad = rng.choice(present, size=E, replace=False)
        Y[g, bad] += (10.0 * rng.standard_normal((E, C))).astype(np.float32)
    out = oracle.locate(K, W, E, Y, mask)
    Yh, n_used, _ = oracle.decode(K, W, Y, out["trusted"])
    assert np.all(n_used == W - S - E)
    assert np.abs(Yh - clean).max() < 0.5
    Yh_bad, _, _ = oracle.decode(K, W, Y, mask)
    assert np.abs(Yh_bad - clean).max() > 2.0


def test_locate_exact_ties_in_magnitude_go_to_the_lower_worker():
    """A class whose predictions are all zero leaves Q = 1, so every a_i equals 1 exactly: the tie rule
    alone decides, and it must pick the E lowest present workers (Algorithm 2 is silent; ties -> lower index)."""
    K, E, W, C = 3, 2, 12, 3
    Y = np.zeros((2, W, C), dtype=np.float32)
    mask = np.array([0xFFF, 0xFFC | 0x0], dtype=np.uint32)  # second group: workers 0 and 1 absent
    out = oracle.locate(K, W, E, Y, mask)
    assert list(out["adv"][0]) == [0, 1]
    assert list(out["adv"][1]) == [2, 3]
    assert out["min_gap"][0] == 1.0 and out["vote_margin"][0] == C
