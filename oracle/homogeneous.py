"""Algorithm 1 of ApproxIFER (arXiv 2109.09868, Section 3, "Rational Interpolation with
Erroneous Evaluations") in its homogeneous form, and Algorithm 3 (Appendix A: the rational function
itself, P / Q) at the end of the file, in numpy fp64.

TEST INFRASTRUCTURE ONLY, like the rest of this package: the product never imports it.

Step 1 of Algorithm 1 asks for polynomials P, Q of degree < K+E with P(x_i) = y_i Q(x_i) on the
available nodes -- a homogeneous system (both Q_0 and the scale are free; Algorithm 2 instead fixes
Q_0 = 1).  With more equations than the theory needs and inexact data no exact non-trivial
solution exists, so the system is read in the least-squares sense:

    minimise  sum_i (P(x_i) - y_i Q(x_i))^2   over P and over Q with  sum_k Q_k^2 = 1.

("Non-trivial" means Q != 0: Q = 0 forces P = 0 on at least K+E nodes, hence P = 0.)  For a fixed
Q the best P is the least-squares polynomial through (x_i, y_i Q(x_i)); what is left is the
smallest singular value problem of  (I - Pi) diag(y) V,  V = [x_i^k], Pi = projector on range(V).
Steps 2-3 are as printed: a_i = Q(x_i), the E smallest |a_i| are the error locations.  For
vector-valued predictions the per-class picks are combined by the vote of Algorithm 2.

Every step is a numpy / LAPACK primitive (qr, svd, lstsq); nothing here is shared with the CUDA
kernels or with approxifer_oracle.c, except the node values, which come from the latter.
"""
from __future__ import annotations

import numpy as np

from . import ST_LOCATE_UNDERDETERMINED, ST_NONFINITE, ST_ORACLE_RANK_DEFICIENT, beta, compact


def locate_class_homogeneous(m: int, xs, y):
    """Steps 1-2 of Algorithm 1 for one scalar sequence.

    xs, y: the n available nodes and values, n >= 2m.  Returns (p, q, a, sigma): coefficients of P
    and Q (each m, |q| = 1, sign arbitrary), a_i = Q(x_i), and the singular values (ascending) of
    the projected matrix -- sigma[0] is the residual norm, sigma[1]/sigma[0] tells how well q is
    determined."""
    xs = np.asarray(xs, dtype=np.float64)
    y = np.asarray(y, dtype=np.float64)
    V = np.vander(xs, m, increasing=True)          # V[i][k] = x_i^k
    YV = y[:, None] * V                            # row i of diag(y) V
    Qv, _ = np.linalg.qr(V)                        # orthonormal basis of range(V)
    Z = YV - Qv @ (Qv.T @ YV)                      # (I - Pi) diag(y) V
    _, s, Vt = np.linalg.svd(Z)
    q = Vt[m - 1]
    p, *_ = np.linalg.lstsq(V, YV @ q, rcond=None)  # the best P for this Q
    return p, q, V @ q, s[::-1].copy()


def locate_homogeneous(K: int, W: int, E: int, Yt, mask):
    """Algorithm 1 per class, the vote of Algorithm 2 over the classes.

    Yt float32 [G][W][C], mask uint32 [G].  Returns dict(adv [G][E] int32 ascending or -1,
    trusted uint32 [G], status uint32 [G], min_gap [G], vote_margin [G], sigma_ratio [G]) with
    the same meaning as oracle.locate; sigma_ratio = min over classes of sigma[1]/sigma[0]."""
    Yt = np.asarray(Yt)
    G, _, C = Yt.shape
    mask = np.asarray(mask, dtype=np.uint32)
    m = K + E
    be = beta(W)
    wmask = 0xFFFFFFFF if W >= 32 else (1 << W) - 1
    adv = np.full((G, E), -1, dtype=np.int32)
    trusted = np.empty(G, dtype=np.uint32)
    status = np.zeros(G, dtype=np.uint32)
    min_gap = np.full(G, np.inf)
    margin = np.zeros(G, dtype=np.int32)
    sigma_ratio = np.full(G, np.inf)
    for g in range(G):
        mk = int(mask[g]) & wmask
        F = compact(W, mk)
        n = len(F)
        trusted[g] = mk
        if n < 2 * m or E <= 0:
            if E > 0:
                status[g] |= ST_LOCATE_UNDERDETERMINED
            continue
        xs = be[F]
        votes = np.zeros(W, dtype=np.int64)
        for c in range(C):
            y = Yt[g, F, c].astype(np.float64)
            _, _, a, s = locate_class_homogeneous(m, xs, y)
            if not (s[m - 1] > 0.0) or s[1] <= 1e-13 * s[m - 1]:
                status[g] |= ST_ORACLE_RANK_DEFICIENT  # Q is not determined (two or more null directions)
            sigma_ratio[g] = min(sigma_ratio[g], s[1] / s[0] if s[0] > 0 else np.inf)
            mag = np.abs(a)
            bad = ~np.isfinite(a)
            if bad.any():
                status[g] |= ST_NONFINITE
                mag[bad] = np.inf
            order = np.argsort(mag, kind="stable")  # ties to the lower worker (F is ascending)
            for r in order[:E]:
                votes[F[r]] += 1
            if n > E:
                last, nxt = mag[order[E - 1]], mag[order[E]]
                min_gap[g] = min(min_gap[g], nxt / last if last > 0 else np.inf)
        cand = [i for i in F]
        cand.sort(key=lambda i: (-votes[i], i))  # most votes first, ties to the lower worker
        elected = sorted(cand[:E])
        adv[g] = elected
        margin[g] = votes[cand[E - 1]] - (votes[cand[E]] if len(cand) > E else 0)
        bits = 0
        for i in elected:
            bits |= 1 << i
        trusted[g] = mk & ~bits
    return dict(adv=adv, trusted=trusted, status=status, min_gap=min_gap, vote_margin=margin,
                sigma_ratio=sigma_ratio)


# ---------------------------------------------------------------------------------------------
# Algorithm 3 (Appendix A, "BW-type rational interpolation in presence of errors")
# ---------------------------------------------------------------------------------------------

def rational_class(m: int, xs, y):
    """Step 1 of Algorithm 3 for one scalar sequence: polynomials P, Q of degree < m with
    P(x_i) = y_i Q(x_i) on the available nodes, solved as Algorithm 2 solves the same system
    (Q_0 = 1, ordinary least squares).  Returns (P, Q) as coefficient arrays, Q[0] = 1."""
    xs = np.asarray(xs, dtype=np.float64)
    y = np.asarray(y, dtype=np.float64)
    V = np.vander(xs, m, increasing=True)
    A = np.hstack([V, -y[:, None] * V[:, 1:]])
    x, *_ = np.linalg.lstsq(A, y, rcond=None)
    return x[:m].copy(), np.concatenate([[1.0], x[m:]])


def decode_rational(K: int, W: int, E: int, Yt, mask, alpha_nodes):
    """Algorithm 3 per group and class, then Step 2: r = P / Q evaluated at the K nodes alpha_j.

    Yt float32 [G][W][C], mask uint32 [G], alpha_nodes = oracle.alpha(K).  Returns dict(Yhat float64
    [G][K][C] (0 where nothing was computed), status uint32 [G] (ST_LOCATE_UNDERDETERMINED for fewer
    than 2(K+E) workers), q_min [G] = min over classes and j of |Q(alpha_j)| / max_i |Q(beta_i)|, a
    measure of how close a pole of r comes to an output node)."""
    Yt = np.asarray(Yt)
    G, _, C = Yt.shape
    mask = np.asarray(mask, dtype=np.uint32)
    m = K + E
    be = beta(W)
    al = np.asarray(alpha_nodes, dtype=np.float64)
    Va = np.vander(al, m, increasing=True)
    wmask = 0xFFFFFFFF if W >= 32 else (1 << W) - 1
    out = np.zeros((G, K, C))
    status = np.zeros(G, dtype=np.uint32)
    q_min = np.full(G, np.inf)
    for g in range(G):
        F = compact(W, int(mask[g]) & wmask)
        if len(F) < 2 * m:
            status[g] |= ST_LOCATE_UNDERDETERMINED
            continue
        xs = be[F]
        Vb = np.vander(xs, m, increasing=True)
        for c in range(C):
            P, Q = rational_class(m, xs, Yt[g, F, c].astype(np.float64))
            qa = Va @ Q
            out[g, :, c] = (Va @ P) / qa
            q_min[g] = min(q_min[g], np.abs(qa).min() / np.abs(Vb @ Q).max())
    return dict(Yhat=out, status=status, q_min=q_min)
