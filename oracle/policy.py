"""Communication-policy generation (Algorithm 3 of arXiv 2009.05766) -- oracle side.

TEST INFRASTRUCTURE, not the product.  A step-by-step numpy statement of the paper's
policy generator: the outer search over rho, the inner search over the global average
iteration time t_bar, the row-wise linear programme (Eq. 14: minimise sum_i p_ii subject
to Eq. 10-13), the matrix Y_P = E[D^T D] (Eq. 22) and its second largest eigenvalue, and
the selection of the grid point with the smallest t_bar * ln(eps) / ln(lambda_2).

Where the paper is silent or garbled the readings are:
  * rho_k = k * U_rho / K and t_bar_r = L + r * (U - L) / R   (the printed loop bodies do
    not depend on the loop index);
  * U_rho = min(0.5/alpha, (1-1e-6) / (alpha * max_i sum_{m!=i} (d_im + d_mi))): beyond it
    the floors of Eq. 11 alone exceed a row sum of 1 (the appendix's alpha*rho <= 1/(2(M-1)));
  * L uses the sum over m != i (Eq. 25-26; Eq. 11 floors only m != i);
  * d_ii = 1 for selectability, t_ii = C_i (a self-draw is a compute-only iteration);
  * Eq. 11 is taken closed: p_im >= alpha*rho*(d_im + d_mi);
  * the LP optimum is not unique; the tie-break is the maximum-entropy optimum (an
    exponential tilt of the iteration times) when p_ii = 0 is feasible, and floors plus the
    remainder on the fastest peer(s) when it is not;
  * eps = 1e-3 (it cancels in the arg-min); grid points that are infeasible are skipped.

Numerical values of P are not printed anywhere in the paper: parity unpinned by the paper.
They are pinned instead by the constraints (Eq. 10-13), by Lemmas 1-2 / Theorem 3, by the
LP optimum value from an independent LP solver, and by an exact enumeration of E[D^T D].
"""
from __future__ import annotations

import numpy as np

ETA_CAP = 600.0
BISECT_ITERS = 100
TIE_RTOL = 1e-12


def iteration_times(link_speed_gbps: np.ndarray, d: int):
    """Iteration-time matrix from link speeds (Section II-B: t_im = max{C_i, N_im}).

    N_im = 32 d / (s_im * 1e9) seconds (a full fp32 replica over the link);
    C_i = min_{i != m} N_im / 4 for every i (communication dominates); t_ii = C_i;
    links with speed <= 0 are absent (d_im = 0).
    """
    s = np.asarray(link_speed_gbps, dtype=np.float64)
    M = s.shape[0]
    off = ~np.eye(M, dtype=bool)
    adj = ((s > 0) & off).astype(np.uint8)
    N = np.zeros((M, M))
    N[adj == 1] = 32.0 * d / (s[adj == 1] * 1e9)
    Cc = 0.25 * N[adj == 1].min()
    t = np.where(adj == 1, np.maximum(Cc, N), 0.0)
    t[np.eye(M, dtype=bool)] = Cc
    return t, adj


def tilt(times: np.ndarray, target: float) -> np.ndarray | None:
    """Weights q_m >= 0, sum 1, proportional to exp(-eta * t_m), with sum_m q_m t_m = target."""
    tmin, tmax = times.min(), times.max()
    scale = tmax - tmin
    n = times.shape[0]
    if scale <= TIE_RTOL * tmax:
        return np.full(n, 1.0 / n)
    s = (times - tmin) / scale
    sig = (target - tmin) / scale

    def mean(eta):
        w = np.exp(-eta * s)
        return float((w * s).sum() / w.sum())

    lo, hi = -ETA_CAP, ETA_CAP  # mean(lo) is the largest mean, mean(hi) the smallest
    if sig >= mean(lo):
        eta = lo
    elif sig <= mean(hi):
        eta = hi
    else:
        for _ in range(BISECT_ITERS):
            mid = 0.5 * (lo + hi)
            if mean(mid) > sig:
                lo = mid
            else:
                hi = mid
        eta = 0.5 * (lo + hi)
    w = np.exp(-eta * s)
    q = w / w.sum()
    if abs(float((q * s).sum()) - sig) > 1e-9:
        return None
    return q


def solve_row(i: int, t: np.ndarray, adj: np.ndarray, alpha: float, rho: float, T: float) -> np.ndarray | None:
    """Row i of the LP (Eq. 14): minimise p_ii s.t. sum_m p_im = 1, sum_m t_im p_im = T,
    p_im >= alpha*rho*(d_im+d_mi) for neighbours m != i, p_im = 0 for non-neighbours."""
    M = t.shape[0]
    nb = np.flatnonzero(adj[i])
    nb = nb[nb != i]
    f = alpha * rho * (adj[i, nb].astype(np.float64) + adj[nb, i].astype(np.float64))
    F = f.sum()
    if F > 1.0:
        return None
    free = 1.0 - F
    tn = t[i, nb]
    A = float((f * tn).sum())
    tmin, tmax = tn.min(), tn.max()
    lo, hi = A + free * tmin, A + free * tmax
    row = np.zeros(M)
    if T > hi * (1.0 + TIE_RTOL):
        return None
    if T >= lo * (1.0 - TIE_RTOL):
        if free <= 0.0:
            row[nb] = f
            return row
        target = min(max((T - A) / free, tmin), tmax)
        q = tilt(tn, target)
        if q is None:
            return None
        row[nb] = f + free * q
        return row
    Ci = t[i, i]
    pii = (lo - T) / (tmin - Ci)
    if pii > free * (1.0 + TIE_RTOL):
        return None
    pii = min(pii, free)
    fastest = tn <= tmin * (1.0 + TIE_RTOL)
    extra = np.where(fastest, (free - pii) / fastest.sum(), 0.0)
    row[nb] = f + extra
    row[i] = pii
    return row


def node_probabilities(P: np.ndarray, t: np.ndarray, adj: np.ndarray) -> np.ndarray:
    """Eq. 2-3: t_bar_i = sum_m t_im p_im d_im (d_ii = 1), p_i = (1/t_bar_i) / sum_m (1/t_bar_m)."""
    dd = adj.astype(np.float64) + np.eye(P.shape[0])
    tbar = (t * P * dd).sum(axis=1)
    inv = 1.0 / tbar
    return inv / inv.sum()


def y_matrix(P: np.ndarray, p_node: np.ndarray, adj: np.ndarray, alpha: float, rho: float) -> np.ndarray:
    """Eq. 22: the entries of Y_P = E[(D^k)^T D^k], with gamma_im = (d_im+d_mi) / (2 p_im)."""
    M = P.shape[0]
    dsum = adj.astype(np.float64) + adj.T.astype(np.float64)
    gamma = np.zeros((M, M))
    pos = (P > 0) & ~np.eye(M, dtype=bool)
    gamma[pos] = dsum[pos] / (2.0 * P[pos])
    a = p_node[:, None] * P * gamma        # p_i p_im gamma_im
    b = p_node[:, None] * P * gamma ** 2   # p_i p_im gamma_im^2
    Y = alpha * rho * (a + a.T) - (alpha * rho) ** 2 * (b + b.T)
    np.fill_diagonal(Y, 0.0)
    diag = 1.0 - 2.0 * alpha * rho * a.sum(axis=1) + (alpha * rho) ** 2 * (b + b.T).sum(axis=1)
    Y[np.diag_indices(M)] = diag
    return Y


def second_eigenvalue(Y: np.ndarray) -> float:
    M = Y.shape[0]
    if M <= 512:
        return float(np.linalg.eigvalsh(0.5 * (Y + Y.T))[-2])
    from scipy.sparse.linalg import eigsh
    vals = eigsh(0.5 * (Y + Y.T), k=2, which="LA", return_eigenvectors=False, tol=1e-12)
    return float(np.sort(vals)[0])


def generate_policy(t: np.ndarray, adj: np.ndarray, alpha: float, K: int, R: int, eps: float = 1e-3,
                    rho_upper: float = 0.0):
    """Algorithm 3.  Returns (P, rho, info) or raises ValueError when no grid point is feasible.

    rho_upper > 0 sets the upper end of the rho grid explicitly (0.5 / alpha is the paper's
    printed U_rho); the default caps it where the Eq. 11 floors alone fill a row."""
    t = np.asarray(t, dtype=np.float64)
    adj = np.asarray(adj, dtype=np.uint8)
    M = t.shape[0]
    dsum = adj.astype(np.float64) + adj.T.astype(np.float64)
    np.fill_diagonal(dsum, 0.0)
    U_rho = min(0.5 / alpha, (1.0 - 1e-6) / (alpha * dsum.sum(axis=1).max()))
    if rho_upper > 0.0:
        U_rho = rho_upper
    off = adj.astype(bool) & ~np.eye(M, dtype=bool)
    best = None
    for k in range(1, K + 1):
        rho = k * U_rho / K
        L = max(alpha * rho / M * float((t[i] * dsum[i]).sum()) for i in range(M))
        U = min(float(t[i][off[i]].max()) / M for i in range(M))
        if not U > L:
            continue
        delta = (U - L) / R
        for r in range(1, R + 1):
            tbar = U - (R - r) * delta
            rows = [solve_row(i, t, adj, alpha, rho, M * tbar) for i in range(M)]
            if any(row is None for row in rows):
                continue
            P = np.vstack(rows)
            lam2 = second_eigenvalue(y_matrix(P, node_probabilities(P, t, adj), adj, alpha, rho))
            if not (0.0 < lam2 < 1.0):
                continue
            t_conv = tbar * np.log(eps) / np.log(lam2)
            if best is None or t_conv < best["t_conv"] * (1.0 - 1e-12):
                best = dict(P=P, rho=rho, t_conv=float(t_conv), lam2=lam2, tbar=tbar, k=k, r=r)
    if best is None:
        raise ValueError("no feasible (rho, t_bar) grid point")
    return best["P"], best["rho"], best


# ---------------------------------------------------------------------------------------------
# Extension to pull rules with a constant weight (the paper's section "Extension to existing
# decentralized PSGD approaches"): x_i <- (1 - w)(x_i - alpha g_i) + w x_m, the update of gossip /
# AD-PSGD style averaging written as x <- D(x - alpha g) with D = I + w e_i (e_m - e_i)^T.
#
# The section prescribes two steps.  (1) Replace Eq. 11 by the condition that every entry y_im of
# E[D^T D] on a link is positive.  With a constant weight Eq. 22 becomes
#     y_im = (w - w^2)(p_i p_im + p_m p_mi),      y_ii = 1 - (2w - w^2) p_i sum_m p_im + w^2 sum_m p_m p_mi,
# so the condition reads p_im + p_mi > 0: no floor follows from it.  It is taken closed with a floor
# phi on both directions of every link, p_im >= phi d_im, and phi takes over rho's place in the outer
# search of Algorithm 3 (phi_k = k U_phi / K with U_phi where the floors alone fill a row).
# (2) Solve Eq. 8-13 again.  Row sums of Y_P are 1 + w (sum_m p_m p_mi - p_i sum_m p_im): with the
# pull weight no longer proportional to 1/p_im, Y_P is doubly stochastic (what Lemma 1 provides for
# NetMax) only if every worker is pulled from as often as it pulls; with p_i = 1/M (Eq. 10) that is
# "the columns of P sum to 1" -- an added constraint, which couples the rows of the LP.  The optimum
# is again not unique; the reading taken is p_ii = 0 and, among the feasible P, the one of maximum
# entropy above the floors: p_im = phi + exp(a_i + b_m - eta_i t_im) on links, with (a, b, eta) fixed by
# the row sums, the column sums and the rows' mean iteration time M t_bar.  The inner grid takes the
# midpoints of R cells of [L, U] (at the end points a row sits on a vertex of its simplex and the
# entropy optimum degenerates).  Grid points where no such P exists are skipped.


def y_matrix_fixed_weight(P: np.ndarray, p_node: np.ndarray, w: float) -> np.ndarray:
    """E[D^T D] for D = I + w e_i (e_m - e_i)^T drawn with probability p_i p_im (m != i)."""
    M = P.shape[0]
    off = P * (1.0 - np.eye(M))
    a = p_node[:, None] * off                      # p_i p_im
    Y = (w - w * w) * (a + a.T)
    diag = 1.0 - (2.0 * w - w * w) * a.sum(axis=1) + w * w * a.sum(axis=0)
    Y[np.diag_indices(M)] = diag
    return Y


def solve_fixed_weight(t: np.ndarray, adj: np.ndarray, phi: float, T: float, tol: float = 1e-12):
    """The maximum-entropy P above the floor phi with zero diagonal, rows and columns summing to 1
    and sum_m t_im p_im = T in every row; None if there is none.  Solved through its convex dual
    (variables a_i, b_m, eta_i) with a trust-region Newton method."""
    from scipy.optimize import minimize
    M = t.shape[0]
    link = adj.astype(bool) & ~np.eye(M, dtype=bool)
    deg = link.sum(axis=1).astype(np.float64)
    rows = 1.0 - phi * deg                          # what the residual r = p - phi has to add up to, per row
    cols = 1.0 - phi * link.sum(axis=0)
    if (rows < -1e-15).any():
        return None
    tmin, tmax = t[link].min(), t[link].max()
    if tmax - tmin <= TIE_RTOL * tmax:              # all links equally fast: the time constraint says T = t and nothing else
        if abs(T - tmin) > 1e-9 * tmax:
            return None
        scale, s, tau = 1.0, np.zeros((M, M)), np.zeros(M)
    else:
        scale = tmax - tmin
        s = np.where(link, (t - tmin) / scale, 0.0)     # iteration times mapped to [0, 1]
        tau = (T - phi * (t * link).sum(axis=1) - tmin * rows) / scale     # targets of sum_m s_im r_im
    if (rows <= 1e-15).all():                       # the floors alone fill every row
        P = phi * link
        return P if np.abs((t * P).sum(axis=1) - T).max() <= 1e-9 * tmax else None
    if (tau < -1e-12).any() or (tau > rows * (1 + 1e-12)).any():
        return None

    def unpack(z):
        return z[:M], np.concatenate([[0.0], z[M:2 * M - 1]]), z[2 * M - 1:]      # b_0 = 0 fixes the gauge

    def residual_matrix(z):
        a, b, eta = unpack(z)
        with np.errstate(over="ignore"):
            return np.where(link, np.exp(a[:, None] + b[None, :] - eta[:, None] * s), 0.0)

    def dual(z):
        a, b, eta = unpack(z)
        r = residual_matrix(z)
        f = r.sum() - a @ rows - b @ cols + eta @ tau
        g = np.concatenate([r.sum(axis=1) - rows, (r.sum(axis=0) - cols)[1:], tau - (s * r).sum(axis=1)])
        return f, g

    def hess(z):
        r = residual_matrix(z)
        sr, ssr = s * r, s * s * r
        H = np.zeros((3 * M - 1, 3 * M - 1))
        A, B, E = slice(0, M), slice(M, 2 * M - 1), slice(2 * M - 1, 3 * M - 1)
        H[A, A] = np.diag(r.sum(axis=1))
        H[A, B] = r[:, 1:]
        H[A, E] = -np.diag(sr.sum(axis=1))
        H[B, B] = np.diag(r.sum(axis=0)[1:])
        H[B, E] = -sr.T[1:, :]
        H[E, E] = np.diag(ssr.sum(axis=1))
        return H + np.triu(H, 1).T

    z0 = np.concatenate([np.log(np.maximum(rows, 1e-300) / np.maximum(deg, 1.0)), np.zeros(M - 1), np.zeros(M)])
    res = minimize(dual, z0, jac=True, hess=hess, method="trust-exact", options=dict(gtol=1e-14, maxiter=400))
    z = res.x
    for _ in range(50):     # the trust-region method stops where the dual's value no longer resolves: finish with Newton steps on the gradient
        with np.errstate(over="ignore", invalid="ignore"):
            g, H = dual(z)[1], hess(z)
        if not (np.isfinite(g).all() and np.isfinite(H).all()) or np.abs(g).max() <= 1e-14:
            break                                  # (an infeasible target drives the multipliers to infinity)
        step = np.linalg.lstsq(H, -g, rcond=None)[0]
        if not np.isfinite(step).all():
            break
        z = z + step
    r = residual_matrix(z)
    P = phi * link + r
    ok = (np.abs(P.sum(axis=1) - 1.0).max() <= 1e-9 and np.abs(P.sum(axis=0) - 1.0).max() <= 1e-9
          and np.abs((t * P).sum(axis=1) - T).max() <= 1e-9 * tmax)
    return P if ok else None


def generate_policy_fixed_weight(t: np.ndarray, adj: np.ndarray, w: float, K: int, R: int, eps: float = 1e-3,
                                 floor_upper: float = 0.0):
    """Algorithm 3 for a constant pull weight w: the floor phi in rho's place (outer loop), the
    average iteration time t_bar in the inner loop, Y_P from y_matrix_fixed_weight.  Returns
    (P, phi, info) or raises ValueError when no grid point is feasible.  floor_upper > 0 sets the
    upper end of the phi grid (default: where the floors alone fill a row)."""
    t = np.asarray(t, dtype=np.float64)
    adj = np.asarray(adj, dtype=np.uint8)
    M = t.shape[0]
    link = adj.astype(bool) & ~np.eye(M, dtype=bool)
    U_phi = floor_upper if floor_upper > 0.0 else (1.0 - 1e-6) / link.sum(axis=1).max()
    p_node = np.full(M, 1.0 / M)                        # Eq. 10 holds by construction (Lemma 1)
    best = None
    for k in range(1, K + 1):
        phi = k * U_phi / K
        L = max(phi / M * float((t[i] * link[i]).sum()) + (1.0 - phi * link[i].sum()) * float(t[i][link[i]].min()) / M
                for i in range(M))
        U = min(phi / M * float((t[i] * link[i]).sum()) + (1.0 - phi * link[i].sum()) * float(t[i][link[i]].max()) / M
                for i in range(M))
        if not U >= L:
            continue
        for r in range(1, R + 1):
            tbar = L + (r - 0.5) * (U - L) / R      # cell midpoints: at t_bar = L or U a row sits on a vertex and the entropy optimum degenerates
            P = solve_fixed_weight(t, adj, phi, M * tbar)
            if P is None:
                continue
            lam2 = second_eigenvalue(y_matrix_fixed_weight(P, p_node, w))
            if not (0.0 < lam2 < 1.0):
                continue
            t_conv = tbar * np.log(eps) / np.log(lam2)
            if best is None or t_conv < best["t_conv"] * (1.0 - 1e-12):
                best = dict(P=P, phi=phi, t_conv=float(t_conv), lam2=lam2, tbar=tbar, k=k, r=r)
    if best is None:
        raise ValueError("no feasible (phi, t_bar) grid point")
    return best["P"], best["phi"], best
