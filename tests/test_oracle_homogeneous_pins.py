"""Pins of the homogeneous error locator (Algorithm 1, read as a least-squares problem with |Q| = 1)
against things other than itself: an eigen-decomposition of the explicitly formed Schur complement,
exact rational arithmetic, the optimality conditions, Theorem 1's constructive guarantee, and
invariances of the problem.  No GPU needed.
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import homogeneous as hom


def _objective(m, xs, y, q):
    """min over P of |V p - diag(y) V q| for a given q, by an independent least-squares call."""
    V = np.vander(xs, m, increasing=True)
    t = (y[:, None] * V) @ q
    p, *_ = np.linalg.lstsq(V, t, rcond=None)
    return np.linalg.norm(V @ p - t)


def test_solution_is_the_smallest_eigenvector_of_the_schur_complement():
    """Eliminating P from the normal equations gives S = B^T B - B^T V (V^T V)^-1 V^T B, B = diag(y) V;
    q is its eigenvector of smallest eigenvalue sigma_0^2 (formed here explicitly, a different route)."""
    rng = np.random.default_rng(4)
    for (K, E, W) in [(2, 1, 6), (3, 1, 9), (4, 2, 13), (5, 2, 16), (8, 2, 24)]:
        m = K + E
        be = oracle.beta(W)
        for _ in range(4):
            n = int(rng.integers(2 * m, W + 1))
            xs = be[np.sort(rng.choice(W, size=n, replace=False))]
            y = rng.standard_normal(n)
            p, q, a, s = hom.locate_class_homogeneous(m, xs, y)
            V = np.vander(xs, m, increasing=True)
            B = y[:, None] * V
            S = B.T @ B - B.T @ V @ np.linalg.solve(V.T @ V, V.T @ B)
            lam, vec = np.linalg.eigh((S + S.T) / 2)
            cond = np.linalg.cond(V) ** 2
            assert abs(np.linalg.norm(q) - 1.0) < 1e-14
            assert abs(lam[0] - s[0] ** 2) <= 1e-13 * cond * lam[-1]
            gap = (lam[1] - lam[0]) / lam[-1]
            assert abs(abs(vec[:, 0] @ q) - 1.0) <= 1e-12 * cond / gap
            np.testing.assert_allclose(a, V @ q, rtol=0, atol=1e-14)
            # P is the least-squares polynomial for this Q, and the residual norm is sigma_0
            assert abs(np.linalg.norm(V @ p - B @ q) - s[0]) <= 1e-12 * max(1.0, s[-1])


def test_no_unit_q_does_better():
    rng = np.random.default_rng(5)
    K, E, W = 4, 2, 14
    m = K + E
    xs = oracle.beta(W)[[0, 1, 2, 3, 5, 6, 7, 8, 9, 10, 11, 12, 13]]
    y = rng.standard_normal(len(xs))
    _, q, _, s = hom.locate_class_homogeneous(m, xs, y)
    best = _objective(m, xs, y, q)
    assert abs(best - s[0]) < 1e-12
    for _ in range(300):
        d = rng.standard_normal(m)
        for eps in (1.0, 1e-2, 1e-4):
            t = q + eps * d
            t /= np.linalg.norm(t)
            assert _objective(m, xs, y, t) >= best - 1e-13


def test_exact_rational_null_vector_tiny():
    """Theorem 1, tiny and exact: y = p/q of type (K-1, K-1) except at one node; then
    (P, Q) = (p Lambda, q Lambda), Lambda(x) = x - x_e, solves every equation exactly, so sigma_0 = 0,
    Q is parallel to q Lambda and a_e = 0."""
    K, E, W = 2, 1, 6
    m = K + E
    be = [Fraction(float(v)) for v in oracle.beta(W)]
    p = [Fraction(3, 2), Fraction(-1, 3)]
    q = [Fraction(2), Fraction(1, 2)]
    e = 4
    y = [(p[0] + p[1] * x) / (q[0] + q[1] * x) for x in be]
    y[e] += Fraction(7, 3)
    lam = [-be[e], Fraction(1)]
    P = [p[0] * lam[0], p[0] * lam[1] + p[1] * lam[0], p[1] * lam[1]]
    Q = [q[0] * lam[0], q[0] * lam[1] + q[1] * lam[0], q[1] * lam[1]]
    for i in range(W):
        assert sum(P[k] * be[i] ** k for k in range(m)) == y[i] * sum(Q[k] * be[i] ** k for k in range(m))
    pf, qf, a, s = hom.locate_class_homogeneous(m, [float(v) for v in be], [float(v) for v in y])
    Qn = np.array([float(c) for c in Q])
    Qn /= np.linalg.norm(Qn)
    assert s[0] < 1e-13 * s[-1] and s[1] > 1e-3 * s[-1]
    assert abs(abs(Qn @ qf) - 1.0) < 1e-12
    scale = (Qn @ qf) * np.linalg.norm([float(c) for c in Q])
    np.testing.assert_allclose(pf * scale, [float(c) for c in P], rtol=0, atol=1e-10)
    assert abs(a[e]) < 1e-12
    assert min(abs(a[i]) for i in range(W) if i != e) > 1e-2


def _linear_predictions(K, W, G, C, rng, d_in=6):
    X = rng.random((G, K, d_in), dtype=np.float32)
    M = rng.standard_normal((d_in, C))
    return (oracle.encode(K, W, X) @ M).astype(np.float32)


@pytest.mark.parametrize("K,E,S", [(2, 1, 0), (3, 2, 1), (4, 1, 2), (8, 2, 2), (6, 3, 1), (5, 1, 0)])
def test_locates_injected_errors_for_a_linear_model(K, E, S):
    """Theorem 1 through the whole procedure.  Unlike Algorithm 2 (Q_0 = 1, which pins a_i = 1 at a node
    equal to 0) the homogeneous form has no special node, so an odd number of workers is as good as an even one."""
    rng = np.random.default_rng(300 + K * 10 + E)
    W = 2 * (K + E) + S
    G, C = 30, 4
    Y = _linear_predictions(K, W, G, C, rng)
    mask = np.empty(G, dtype=np.uint32)
    truth = np.empty((G, E), dtype=np.int32)
    for g in range(G):
        present = np.sort(rng.choice(W, size=W - S, replace=False))
        mask[g] = sum(1 << int(i) for i in present)
        bad = np.sort(rng.choice(present, size=E, replace=False))
        if W % 2 == 1 and g == 0 and (W - 1) // 2 in present:
            bad = np.sort(np.concatenate([[(W - 1) // 2], [i for i in bad if i != (W - 1) // 2][: E - 1]]))
        truth[g] = bad
        Y[g, bad] += (10.0 * rng.standard_normal((E, C))).astype(np.float32)
    out = hom.locate_homogeneous(K, W, E, Y, mask)
    np.testing.assert_array_equal(out["adv"], truth)
    for g in range(G):
        assert int(out["trusted"][g]) == int(mask[g]) & ~sum(1 << int(i) for i in truth[g])
    assert np.all(out["status"] == 0)
    assert out["min_gap"].min() > 2.0
    assert np.all(out["vote_margin"] == C)
    assert out["sigma_ratio"].min() > 10.0


def test_invariances_scale_of_y_and_mirror_of_the_nodes():
    rng = np.random.default_rng(8)
    K, E, W = 3, 2, 12
    m = K + E
    xs = oracle.beta(W)
    y = rng.standard_normal(W)
    _, q, a, s = hom.locate_class_homogeneous(m, xs, y)
    # y -> c y: r -> c r, P -> c P, Q unchanged
    _, q2, a2, s2 = hom.locate_class_homogeneous(m, xs, -3.5 * y)
    sg = np.sign(q @ q2)
    np.testing.assert_allclose(sg * a2, a, rtol=0, atol=1e-11)
    np.testing.assert_allclose(s2, 3.5 * s, rtol=1e-11)
    # x -> -x with the same values: Q(x) -> Q(-x), so a_i is unchanged up to the common sign
    _, q3, a3, _ = hom.locate_class_homogeneous(m, -xs, y)
    alt = q3 * (-1.0) ** np.arange(m)
    sg = np.sign(q @ alt)
    np.testing.assert_allclose(sg * alt, q, rtol=0, atol=1e-10)
    np.testing.assert_allclose(sg * a3, a, rtol=0, atol=1e-10)


def test_underdetermined_groups_and_bits_beyond_w():
    K, E, W, C = 2, 1, 7, 3
    rng = np.random.default_rng(2)
    Y = rng.standard_normal((3, W, C)).astype(np.float32)
    mask = np.array([0b0011111, 0b1111111 | (1 << 20), 0], dtype=np.uint32)
    out = hom.locate_homogeneous(K, W, E, Y, mask)
    assert out["adv"][0, 0] == -1 and out["status"][0] == oracle.ST_LOCATE_UNDERDETERMINED and out["trusted"][0] == 0b0011111
    assert out["adv"][1, 0] >= 0 and out["status"][1] == 0
    assert int(out["trusted"][1]) == 0b1111111 & ~(1 << int(out["adv"][1, 0]))
    assert out["adv"][2, 0] == -1 and out["trusted"][2] == 0


def test_agrees_with_algorithm_2_when_the_errors_are_exact_roots():
    """On data that Theorem 1 covers, both normalisations (Q_0 = 1 and |Q| = 1) find the same Q up to scale,
    hence the same error locations."""
    rng = np.random.default_rng(12)
    K, E, W, G, C = 4, 2, 12, 25, 3
    Y = _linear_predictions(K, W, G, C, rng)
    mask = np.full(G, (1 << W) - 1, dtype=np.uint32)
    for g in range(G):
        bad = rng.choice(W, size=E, replace=False)
        Y[g, bad] += (5.0 * rng.standard_normal((E, C))).astype(np.float32)
    a2 = oracle.locate(K, W, E, Y, mask)
    a1 = hom.locate_homogeneous(K, W, E, Y, mask)
    np.testing.assert_array_equal(a1["adv"], a2["adv"])


def test_vote_ties_go_to_the_lower_worker():
    """Two classes, E = 1, a different worker corrupted in each: one vote each, the lower index is returned
    (the paper is silent on ties).  Exact ties between two |a_i| cannot be built in floating point for this
    form of the problem; the per-class selection uses a stable sort over the ascending worker list."""
    rng = np.random.default_rng(31)
    K, E, W, C = 3, 1, 9, 2
    Y = _linear_predictions(K, W, 2, C, rng)
    Y[0, 7, 0] += 4.0
    Y[0, 3, 1] -= 6.0
    Y[1, 2, 0] += 4.0
    Y[1, 8, 1] -= 6.0
    out = hom.locate_homogeneous(K, W, E, Y, np.full(2, (1 << W) - 1, dtype=np.uint32))
    assert list(out["adv"][:, 0]) == [3, 2]
    assert list(out["vote_margin"]) == [0, 0]
