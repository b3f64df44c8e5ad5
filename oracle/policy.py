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
