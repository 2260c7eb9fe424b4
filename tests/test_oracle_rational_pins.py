"""Pins of the oracle for Algorithm 3 (BW-type rational interpolation in the presence of errors, Appendix A):
the theorem that follows it (the returned P/Q equals r when at most E values are wrong), exact rational
arithmetic, and plain interpolation when nothing is wrong.  No GPU needed."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import homogeneous as hom


def test_exact_rational_tiny_recovers_r_despite_an_error():
    """y = p/q of type (K-1, K-1) except at one node: P = p Lambda / c, Q = q Lambda / c solve every equation, so
    P/Q = p/q everywhere -- also at points that are not nodes."""
    K, E, W = 2, 1, 6
    m = K + E
    be = [Fraction(float(v)) for v in oracle.beta(W)]
    p = [Fraction(3, 2), Fraction(-1, 3)]
    q = [Fraction(2), Fraction(1, 2)]
    y = [(p[0] + p[1] * x) / (q[0] + q[1] * x) for x in be]
    y[4] += Fraction(7, 3)
    P, Q = hom.rational_class(m, [float(v) for v in be], [float(v) for v in y])
    for z in (0.3, -0.77, 0.0, float(oracle.alpha(K)[0])):
        r = (float(p[0]) + float(p[1]) * z) / (float(q[0]) + float(q[1]) * z)
        got = np.polyval(P[::-1], z) / np.polyval(Q[::-1], z)
        assert abs(got - r) < 1e-11
    assert Q[0] == 1.0


@pytest.mark.parametrize("K,E,S", [(2, 1, 0), (3, 2, 1), (4, 1, 2), (8, 2, 2), (5, 0, 1), (6, 3, 0)])
def test_linear_model_is_recovered_exactly_despite_errors(K, E, S):
    """The theorem after Algorithm 3 through the whole procedure: for a linear model f the honest coded
    predictions are f(u(beta_i)), a rational function of type (K-1, K-1) whose value at alpha_j is f(X_j); with at
    most E corrupted workers P/Q at alpha_j returns f(X_j) itself -- not Berrut's approximation of it."""
    rng = np.random.default_rng(500 + 10 * K + E)
    W = 2 * (K + E) + S
    if W % 2 == 1:
        W += 1  # an odd W puts a node at 0, where Q_0 = 1 forbids a root: a corrupted worker there cannot be absorbed
    G, C, d_in = 12, 3, 5
    X = rng.random((G, K, d_in), dtype=np.float32)
    M = rng.standard_normal((d_in, C))
    Y = (oracle.encode(K, W, X) @ M)
    truth = X.astype(np.float64) @ M
    mask = np.empty(G, dtype=np.uint32)
    for g in range(G):
        present = np.sort(rng.choice(W, size=W - S, replace=False))
        mask[g] = sum(1 << int(i) for i in present)
        if E:
            bad = rng.choice(present, size=E, replace=False)
            Y[g, bad] += 10.0 * rng.standard_normal((E, C))
    # in fp64 the recovery is exact to rounding ...
    al, be = oracle.alpha(K), oracle.beta(W)
    for g in range(G):
        F = oracle.compact(W, int(mask[g]))
        for c in range(C):
            P, Q = hom.rational_class(K + E, be[F], Y[g, F, c])
            r = np.polyval(P[::-1], al) / np.polyval(Q[::-1], al)
            np.testing.assert_allclose(r, truth[g, :, c], rtol=0, atol=1e-8 * np.abs(truth).max())
    # ... and through the fp32 interface the rounding of the inputs (6e-8 relative) is amplified by the solve,
    # mildly for small K+E, by up to ~1e5 at K+E = 10: the numerical fragility the paper warns about
    out = hom.decode_rational(K, W, E, Y.astype(np.float32), mask, al)
    assert np.all(out["status"] == 0)
    np.testing.assert_allclose(out["Yhat"], truth, rtol=0, atol=(2e-4 if K + E <= 5 else 2e-2) * np.abs(truth).max())


def test_without_errors_and_with_exactly_2K_workers_the_nodes_are_interpolated():
    """E = 0 and n = 2K available values of a type (K-1, K-1) function: P - y Q vanishes on all of them."""
    K, W = 3, 6
    xs = oracle.beta(W)
    y = (1.0 + 0.5 * xs - 0.25 * xs**2) / (2.0 - 0.3 * xs + 0.1 * xs**2)
    P, Q = hom.rational_class(K, xs, y)
    r = np.polyval(P[::-1], xs) / np.polyval(Q[::-1], xs)
    np.testing.assert_allclose(r, y, rtol=0, atol=1e-12)
    z = 0.123
    np.testing.assert_allclose(np.polyval(P[::-1], z) / np.polyval(Q[::-1], z),
                               (1.0 + 0.5 * z - 0.25 * z**2) / (2.0 - 0.3 * z + 0.1 * z**2), atol=1e-12)


def test_underdetermined_groups_are_flagged_and_left_at_zero():
    K, E, W, C = 2, 1, 7, 2
    Y = np.random.default_rng(0).standard_normal((2, W, C)).astype(np.float32)
    out = hom.decode_rational(K, W, E, Y, np.array([0b0011111, 0b1111111], dtype=np.uint32), oracle.alpha(K))
    assert out["status"][0] == oracle.ST_LOCATE_UNDERDETERMINED and np.all(out["Yhat"][0] == 0)
    assert out["status"][1] == 0 and np.isfinite(out["Yhat"][1]).all()
