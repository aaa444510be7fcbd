"""Design-time oracle in float64 numpy (test infrastructure).

Everything the paper computes once before training: the optimal structure of
Theorem 1, the closed-form sparse interval construction (Sec. III-A), recovery
of (A, w), the unbiasedness condition Eq. exp_g2_quant, the bounds of Lemma 1
and Lemma 2, the exact DP bit allocator (Eq. dp_rec), the low-complexity
allocator (Algorithm 1), the error-balance scaling eta (Sec. V-B) and the
two-track decoder v* (Sec. V-E).

Letters: n workers, k partitions (the paper writes k workers, n partitions),
bits b_i (paper z_i), residual bits r_i = b_i - 2, `dim` is the dimension l
that enters phi (the bucket size when norms are per bucket).

`bit_allocate_low_complexity`: exact agreement with the authors' allocator is
PARITY UNPINNED - the paper gives its Lagrangian step and its swap search in
one sentence each; the readings taken are written at the function.
"""
import itertools

import numpy as np


# ---------------------------------------------------------------- quantiser constants
def levels(b):
    """s_i = 2^(z_i-1) - 1 magnitude levels (Sec. II-B)."""
    return (1 << (int(b) - 1)) - 1


def phi(b, dim, eta=1.0):
    """phi(z) = l / (4 (2^(z-1)-1)^2) (Lemma 1), times the error-balance factor
    eta of Sec. V-B. b = 1 is outside the paper (z >= 2): for the two-point
    quantiser {-S,+S} the per-coordinate variance is S^2 - x^2 <= S^2, so
    phi(1) := dim."""
    b = int(b)
    if b == 1:
        return eta * float(dim)
    return eta * float(dim) / (4.0 * levels(b) ** 2)


def c_coeff(p, bits, dim, eta=1.0):
    """c_i = p_i/(1-p_i) + eta*phi(z_i)/(1-p_i) (Sec. III-A, Sec. V-B)."""
    p = np.asarray(p, np.float64)
    ph = np.array([phi(b, dim, 1.0) for b in bits], np.float64)
    return p / (1.0 - p) + eta * ph / (1.0 - p)


# ---------------------------------------------------------------- Theorem 1 + construction
def optimal_row_sums(p, bits, k_parts, dim, eta=1.0):
    """Y_i = c_i^-1 * k_parts / sum_m c_m^-1 (Theorem 1)."""
    ci = 1.0 / c_coeff(p, bits, dim, eta)
    return ci * k_parts / ci.sum()


def interval_alpha(Y, k_parts):
    """alpha_i^j = [min{R_i, j} - max{R_{i-1}, j-1}]_+ with R_i the prefix sums of Y
    and partition j <-> unit segment [j-1, j] (Sec. III-A, closed-form sparse
    construction). Returns an (n, k_parts) dense float64 matrix."""
    Y = np.asarray(Y, np.float64)
    n = len(Y)
    R = np.concatenate([[0.0], np.cumsum(Y)])
    R[-1] = float(k_parts)  # sum_i Y_i = k_parts exactly (Sec. III-A)
    alpha = np.zeros((n, k_parts), np.float64)
    for i in range(n):
        for j in range(1, k_parts + 1):
            alpha[i, j - 1] = max(min(R[i + 1], j) - max(R[i], j - 1), 0.0)
    return alpha


def physical_coefficients(alpha, p):
    """a_ij = alpha_ij / w~_i, w_i = w~_i / (1 - p_i) with the free w~_i := 1
    (Sec. III-A: any non-zero w~_i)."""
    p = np.asarray(p, np.float64)
    return np.array(alpha, np.float64), 1.0 / (1.0 - p)


def alpha_to_csr(alpha, drop=1e-12):
    """CSR of the non-zeros of alpha; entries below `drop` are removed and each
    column renormalised to sum exactly 1 (keeps Eq. exp_g2_quant exact)."""
    al = np.array(alpha, np.float64)
    al[al < drop] = 0.0
    al = al / al.sum(axis=0, keepdims=True)
    row_ptr = [0]
    col, val = [], []
    for i in range(al.shape[0]):
        nz = np.nonzero(al[i])[0]
        col.extend(nz.tolist())
        val.extend(al[i, nz].tolist())
        row_ptr.append(len(col))
    return (np.array(row_ptr, np.int32), np.array(col, np.int32), np.array(val, np.float64))


def csr_to_dense(row_ptr, col_idx, vals, k_parts):
    n = len(row_ptr) - 1
    A = np.zeros((n, k_parts), np.float64)
    for i in range(n):
        for e in range(row_ptr[i], row_ptr[i + 1]):
            A[i, col_idx[e]] += vals[e]
    return A


def unbiasedness_residual(A, w, p):
    """max_j | sum_i (1-p_i) w_i a_ij - 1 |  (Eq. exp_g2_quant)."""
    A = np.asarray(A, np.float64)
    w = np.asarray(w, np.float64)
    p = np.asarray(p, np.float64)
    return float(np.max(np.abs(((1.0 - p) * w) @ A - 1.0)))


def structure_objective(alpha, c):
    """sum_i c_i (sum_j alpha_ij)^2, the objective of (c-SP2)."""
    return float(np.sum(np.asarray(c) * np.asarray(alpha).sum(axis=1) ** 2))


def optimal_objective(c, k_parts):
    """k_parts^2 / sum_i c_i^-1: the value of (c-SP2) at the structure of
    Theorem 1 (Lemma 2 without the constant C)."""
    return float(k_parts ** 2 / np.sum(1.0 / np.asarray(c)))


def cyclic_support(n, k_parts, s):
    """Worker i holds partitions i, i+1, ..., i+s-1 (mod k_parts). Returns a list
    of sorted column lists."""
    return [sorted(((i + t) % k_parts) for t in range(s)) for i in range(n)]


def support_kkt_gap(alpha, c, support):
    """Optimality certificate for (c-SP2) restricted to a support with alpha >= 0.
    The problem is convex; alpha is optimal iff for every partition j all workers
    carrying mass in column j have the smallest marginal cost c_i*y_i among the
    workers allowed in that column (y = row sums). Returns
    (max column-sum error, max relative marginal-cost excess on active entries,
     most negative entry)."""
    alpha = np.asarray(alpha, np.float64)
    c = np.asarray(c, np.float64)
    y = alpha.sum(axis=1)
    mc = c * y
    k_parts = alpha.shape[1]
    col_err = float(np.max(np.abs(alpha.sum(axis=0) - 1.0)))
    excess = 0.0
    for j in range(k_parts):
        allowed = [i for i in range(len(support)) if j in support[i]]
        lo = min(mc[i] for i in allowed)
        for i in allowed:
            if alpha[i, j] > 1e-9:
                excess = max(excess, (mc[i] - lo) / max(lo, 1e-300))
    off = alpha.copy()
    for i, cols in enumerate(support):
        off[i, cols] = 0.0
    assert np.all(off == 0.0), "mass outside the support"
    return col_err, float(excess), float(alpha.min())


def support_restricted_alpha_reference(c, support, k_parts):
    """Reference solution of (c-SP2) on a fixed support with alpha >= 0 by a
    general-purpose constrained solver (scipy SLSQP); small problems only."""
    from scipy.optimize import minimize
    c = np.asarray(c, np.float64)
    n = len(support)
    idx = [(i, j) for i in range(n) for j in support[i]]
    nv = len(idx)
    rows = np.array([i for i, _ in idx])
    cols = np.array([j for _, j in idx])

    def fun(x):
        y = np.bincount(rows, weights=x, minlength=n)
        return float(np.sum(c * y * y))

    def jac(x):
        y = np.bincount(rows, weights=x, minlength=n)
        return 2.0 * c[rows] * y[rows]

    Aeq = np.zeros((k_parts, nv))
    Aeq[cols, np.arange(nv)] = 1.0
    deg = Aeq.sum(axis=1)
    x0 = 1.0 / deg[cols]
    res = minimize(fun, x0, jac=jac, method="SLSQP", bounds=[(0.0, None)] * nv,
                   constraints=[{"type": "eq", "fun": lambda x: Aeq @ x - 1.0, "jac": lambda x: Aeq}],
                   options={"maxiter": 2000, "ftol": 1e-15})
    alpha = np.zeros((n, k_parts))
    alpha[rows, cols] = np.maximum(res.x, 0.0)
    return alpha, float(res.fun)


# ---------------------------------------------------------------- bounds
def lemma1_bound(A, w, p, bits, dim, C=1.0, eta=1.0):
    """C * sum_i (1-p_i){p_i + phi(z_i)} w_i^2 (sum_j a_ij)^2 (Lemma 1)."""
    A = np.asarray(A, np.float64)
    w = np.asarray(w, np.float64)
    p = np.asarray(p, np.float64)
    ph = np.array([phi(b, dim, eta) for b in bits])
    return float(C * np.sum((1.0 - p) * (p + ph) * w ** 2 * A.sum(axis=1) ** 2))


def lemma2_bound(p, bits, k_parts, dim, C=1.0, eta=1.0):
    """k_parts^2 C / sum_i c_i^-1 (Lemma 2)."""
    return float(C * optimal_objective(c_coeff(p, bits, dim, eta), k_parts))


# ---------------------------------------------------------------- bit allocation
def h_utility(p_i, r, dim, eta=1.0):
    """h_i(r) = (1-p_i)/(p_i + phi(r+2)) (b-SP1)."""
    return (1.0 - p_i) / (p_i + phi(int(r) + 2, dim, eta))


def allocation_value(p, r, dim, eta=1.0):
    """F(r) = sum_i h_i(r_i)."""
    return float(sum(h_utility(pi, ri, dim, eta) for pi, ri in zip(p, r)))


def bit_allocate_dp(p, z_tot, dim, b_max=0, eta=1.0):
    """Exact optimum of (b-SP1) by the recurrence
    V[i, r] = max_{0<=a<=r} V[i-1, r-a] + h_i(a), V[0,0]=0, V[0,r>0]=-inf (Eq. dp_rec).
    b_max > 0 additionally caps a <= b_max-2 (an extension; the paper has no cap).
    Returns (bits, F)."""
    p = np.asarray(p, np.float64)
    n = len(p)
    z_res = int(z_tot) - 2 * n
    assert z_res >= 0
    cap = z_res if not b_max else min(z_res, b_max - 2)
    assert n * cap >= z_res, "budget exceeds the cap"
    V = np.full((n + 1, z_res + 1), -np.inf)
    V[0, 0] = 0.0
    arg = np.zeros((n + 1, z_res + 1), np.int64)
    for i in range(1, n + 1):
        h = np.array([h_utility(p[i - 1], a, dim, eta) for a in range(cap + 1)])
        for r in range(z_res + 1):
            a = np.arange(min(r, cap) + 1)
            cand = V[i - 1, r - a] + h[a]          # V[i-1, r-a] + h_i(a) for 0 <= a <= r
            arg[i, r] = int(np.argmax(cand))       # first maximiser
            V[i, r] = cand[arg[i, r]]
    r_alloc = np.zeros(n, np.int64)
    rem = z_res
    for i in range(n, 0, -1):
        r_alloc[i - 1] = arg[i, rem]
        rem -= arg[i, rem]
    return (r_alloc + 2).astype(np.uint8), float(V[n, z_res])


def _h_cont(p_i, r, dim, eta):
    """h_i at real-valued r (continuous relaxation)."""
    lev = 2.0 ** (r + 1.0) - 1.0
    return (1.0 - p_i) / (p_i + eta * dim / (4.0 * lev * lev))


def _dh_cont(p_i, r, dim, eta):
    """d h_i / d r at real-valued r."""
    lev = 2.0 ** (r + 1.0) - 1.0
    ph = eta * dim / (4.0 * lev * lev)
    dph = -2.0 * ph * (2.0 ** (r + 1.0)) * np.log(2.0) / lev
    return -(1.0 - p_i) * dph / (p_i + ph) ** 2


def _lagrangian_allocation(p_sel, z_res, cap, dim, eta):
    """Continuous relaxation on the selected workers, solved through its
    stationarity condition h_i'(r_i) = lambda on the concave branch of each
    sigmoidal h_i (r_i = 0 if lambda exceeds the peak slope), lambda found by
    bisection so that sum r_i = z_res; then floor + largest remainders."""
    m = len(p_sel)
    grid = np.linspace(0.0, float(cap), 2049)
    peaks, peak_slopes = [], []
    for pi in p_sel:
        dh = _dh_cont(pi, grid, dim, eta)
        t = int(np.argmax(dh))
        peaks.append(grid[t])
        peak_slopes.append(dh[t])

    p_arr = np.asarray(p_sel, np.float64)
    peaks = np.asarray(peaks)
    peak_slopes = np.asarray(peak_slopes)
    slope_at_cap = _dh_cont(p_arr, float(cap), dim, eta)

    def r_of(lam):
        # per worker: 0 if lam is above its peak slope, cap if the slope at the cap
        # still exceeds lam, else the root of h'(r) = lam right of the peak (bisection)
        lo = peaks.copy()
        hi = np.full(m, float(cap))
        for _ in range(50):
            mid = 0.5 * (lo + hi)
            above = _dh_cont(p_arr, mid, dim, eta) > lam
            lo = np.where(above, mid, lo)
            hi = np.where(above, hi, mid)
        out = 0.5 * (lo + hi)
        out = np.where(slope_at_cap >= lam, float(cap), out)
        return np.where(lam >= peak_slopes, 0.0, out)

    lo, hi = 0.0, max(peak_slopes)
    for _ in range(60):
        mid = 0.5 * (lo + hi)
        if r_of(mid).sum() > z_res:
            lo = mid
        else:
            hi = mid
    r_real = r_of(hi)
    r_int = np.floor(r_real + 1e-12).astype(np.int64)
    r_int = np.minimum(r_int, cap)
    left = z_res - int(r_int.sum())
    if left < 0:  # overshoot after flooring cannot happen, but stay safe
        order = np.argsort(-(r_int.astype(np.float64)), kind="stable")
        t = 0
        while left < 0:
            if r_int[order[t % m]] > 0:
                r_int[order[t % m]] -= 1
                left += 1
            t += 1
    frac = r_real - np.floor(r_real + 1e-12)
    while left > 0:
        order = np.argsort(-frac, kind="stable")
        progressed = False
        for t in order:
            if left == 0:
                break
            if r_int[t] < cap:
                r_int[t] += 1
                frac[t] = -1.0
                left -= 1
                progressed = True
        if not progressed:
            return None
        frac[:] = 0.0
    return r_int


def bit_allocate_low_complexity(p, z_tot, dim, b_max=0, eta=1.0):
    """Algorithm 1 (proposed low-complexity bit allocation). Readings taken where
    the paper is brief:
      - workers sorted by p ascending, ties by index; top-kappa set S_kappa;
      - EQ: z_res // kappa each, the remainder to the most reliable first;
      - LAG: `_lagrangian_allocation` on S_kappa;
      - the better of LAG / EQ by F over ALL workers (r = 0 outside S_kappa);
      - 1-bit swaps over all ordered pairs of workers, best improvement first,
        accepted while the gain exceeds 1e-12*|F|;
      - the incumbent is replaced only on strict improvement;
      - b_max > 0 caps r_i <= b_max-2 (extension).
    Returns (bits, F)."""
    p = np.asarray(p, np.float64)
    n = len(p)
    z_res = int(z_tot) - 2 * n
    assert z_res >= 0
    cap = z_res if not b_max else min(z_res, b_max - 2)
    assert n * cap >= z_res, "budget exceeds the cap"
    order = np.argsort(p, kind="stable")
    hh = np.array([[h_utility(p[i], a, dim, eta) for a in range(cap + 2)] for i in range(n)])

    def F_of(r):
        return float(sum(hh[i, r[i]] for i in range(n)))

    best_r, best_F = None, -np.inf
    if z_res == 0:
        r0 = np.zeros(n, np.int64)
        return (r0 + 2).astype(np.uint8), F_of(r0)
    for kappa in range(1, min(n, z_res) + 1):
        if kappa * cap < z_res:
            continue
        sel = order[:kappa]
        cands = []
        r_eq = np.zeros(n, np.int64)
        base, rem = divmod(z_res, kappa)
        for t, i in enumerate(sel):
            r_eq[i] = base + (1 if t < rem else 0)
        cands.append(r_eq)
        r_sel = _lagrangian_allocation(p[sel], z_res, cap, dim, eta)
        if r_sel is not None:
            r_lag = np.zeros(n, np.int64)
            r_lag[sel] = r_sel
            cands.append(r_lag)
        r = max(cands, key=F_of).copy()
        F = F_of(r)
        idx = np.arange(n)
        while True:
            # best 1-bit swap j -> i over all ordered pairs (first maximum in (i, j) order)
            up = np.where(r < cap, hh[idx, np.minimum(r + 1, cap + 1)] - hh[idx, r], -np.inf)
            down = np.where(r > 0, hh[idx, np.maximum(r - 1, 0)] - hh[idx, r], -np.inf)
            gain = up[:, None] + down[None, :]
            gain[idx, idx] = -np.inf
            flat = int(np.argmax(gain))
            best_gain = gain.flat[flat]
            if not np.isfinite(best_gain) or best_gain <= 1e-12 * abs(F):
                break
            r[flat // n] += 1
            r[flat % n] -= 1
            F = F_of(r)
        if F > best_F:
            best_F, best_r = F, r.copy()
    return (best_r + 2).astype(np.uint8), best_F


def bit_allocate_bruteforce(p, z_tot, dim, b_max=0, eta=1.0):
    """All compositions of z_res into n non-negative parts (tiny inputs only)."""
    n = len(p)
    z_res = int(z_tot) - 2 * n
    cap = z_res if not b_max else min(z_res, b_max - 2)
    best, best_r = -np.inf, None
    for r in itertools.product(range(cap + 1), repeat=n):
        if sum(r) != z_res:
            continue
        F = allocation_value(p, r, dim, eta)
        if F > best:
            best, best_r = F, r
    return (np.array(best_r) + 2).astype(np.uint8), float(best)


# ---------------------------------------------------------------- comparison allocators (Sec. VI)
# The paper's Fig. 2 sets Algorithm 1 against the exact DP and against two heuristics it names
# without printing them, "greedy" and "continuous relaxation"; these are the readings taken.
def bit_allocate_greedy(p, z_tot, dim, b_max=0, eta=1.0):
    """Greedy heuristic: from r = 0, the residual bits are handed out one at a time, each to
    the worker whose utility h_i gains most from one more bit (ties: lowest index). Exact when
    every h_i is concave on the range; trapped by the convex foot of the sigmoidal h_i otherwise.
    Returns (bits, F)."""
    p = np.asarray(p, np.float64)
    n = len(p)
    z_res = int(z_tot) - 2 * n
    assert z_res >= 0
    cap = z_res if not b_max else min(z_res, b_max - 2)
    assert n * cap >= z_res, "budget exceeds the cap"
    hh = np.array([[h_utility(p[i], a, dim, eta) for a in range(cap + 2)] for i in range(n)])
    r = np.zeros(n, np.int64)
    idx = np.arange(n)
    for _ in range(z_res):
        gain = np.where(r < cap, hh[idx, np.minimum(r + 1, cap + 1)] - hh[idx, r], -np.inf)
        r[int(np.argmax(gain))] += 1
    return (r + 2).astype(np.uint8), float(hh[idx, r].sum())


def bit_allocate_relaxation(p, z_tot, dim, b_max=0, eta=1.0):
    """Continuous-relaxation heuristic: the stationarity system of the relaxed problem over ALL
    workers (`_lagrangian_allocation` with every worker selected), rounded by floor + largest
    remainders. It is Algorithm 1's LAG candidate without the search over the top-kappa sets,
    the EQ candidate and the swap refinement. Returns (bits, F)."""
    p = np.asarray(p, np.float64)
    n = len(p)
    z_res = int(z_tot) - 2 * n
    assert z_res >= 0
    cap = z_res if not b_max else min(z_res, b_max - 2)
    assert n * cap >= z_res, "budget exceeds the cap"
    if z_res == 0:
        r = np.zeros(n, np.int64)
    else:
        r = _lagrangian_allocation(p, z_res, cap, dim, eta)
        if r is None:   # rounding could not place the bits under the cap: spread them evenly
            r = np.full(n, z_res // n, np.int64)
            r[:z_res % n] += 1
    return (r + 2).astype(np.uint8), allocation_value(p, r, dim, eta)


def allocation_upper_bound(p, z_tot, dim, b_max=0, eta=1.0):
    """An upper bound on the optimum of (b-SP1): each h_i is replaced by the upper concave
    envelope of its integer points, which makes the problem a separable concave one whose
    optimum the greedy rule over the envelope's unit slopes attains exactly. F_DP <= bound."""
    p = np.asarray(p, np.float64)
    n = len(p)
    z_res = int(z_tot) - 2 * n
    cap = z_res if not b_max else min(z_res, b_max - 2)
    slopes = []
    base = 0.0
    for i in range(n):
        h = np.array([h_utility(p[i], a, dim, eta) for a in range(cap + 1)])
        base += h[0]
        hull = [0]                                    # upper hull of the points (a, h[a])
        for a in range(1, cap + 1):
            while len(hull) >= 2:
                a0, a1 = hull[-2], hull[-1]
                if (h[a1] - h[a0]) * (a - a0) <= (h[a] - h[a0]) * (a1 - a0):
                    hull.pop()
                else:
                    break
            hull.append(a)
        for a0, a1 in zip(hull[:-1], hull[1:]):
            slopes += [(h[a1] - h[a0]) / (a1 - a0)] * (a1 - a0)
    slopes = np.sort(np.array(slopes))[::-1]
    return float(base + slopes[:z_res].sum())


def allocator_study(ns=(10, 50), multiples=(1, 2, 3, 4, 5), seeds=50, dim=512.0, b_max=0, with_eta=False,
                    probs=None):
    """Synthetic re-creation of the comparison of Fig. 2 (Sec. VI): mean objective F(r) of
    Algorithm 1, the exact DP, the greedy and the continuous-relaxation heuristics, and the
    concave-envelope upper bound, over `seeds` draws of the straggler probabilities for
    Z_res = multiple * n residual bits. `probs(n, seed)` supplies the probabilities (the
    caller passes the shifted-exponential model of Sec. V-A). with_eta applies the
    error-balance factor of Sec. V-B to every method. Returns a list of rows (dicts)."""
    rows = []
    for n in ns:
        for mult in multiples:
            z_tot = 2 * n + mult * n
            acc = {"alg1": 0.0, "dp": 0.0, "greedy": 0.0, "relaxation": 0.0, "bound": 0.0}
            worst = 1.0
            for seed in range(seeds):
                p = probs(n, seed)
                eta = eta_balance(p, z_tot, dim) if with_eta else 1.0
                f_dp = bit_allocate_dp(p, z_tot, dim, b_max, eta)[1]
                f_a = bit_allocate_low_complexity(p, z_tot, dim, b_max, eta)[1]
                acc["dp"] += f_dp
                acc["alg1"] += f_a
                acc["greedy"] += bit_allocate_greedy(p, z_tot, dim, b_max, eta)[1]
                acc["relaxation"] += bit_allocate_relaxation(p, z_tot, dim, b_max, eta)[1]
                acc["bound"] += allocation_upper_bound(p, z_tot, dim, b_max, eta)
                worst = min(worst, f_a / f_dp)
            row = {"n": n, "z_res": mult * n, "eta": bool(with_eta), "alg1_min_ratio": worst}
            row.update({k: v / seeds for k, v in acc.items()})
            rows.append(row)
    return rows


def eta_balance(p, z_tot, dim):
    """eta = mean(p) * 4 (2^(Z_tot/n - 1) - 1)^2 / l (Sec. V-B)."""
    p = np.asarray(p, np.float64)
    return float(p.mean() * 4.0 * (2.0 ** (z_tot / len(p) - 1.0) - 1.0) ** 2 / dim)


# ---------------------------------------------------------------- two-track decoder
def two_track_decoder(A, p, bits, dim, lam=1.0, eta=1.0):
    """v_i* = k_parts*Lambda / ((p_i + phi(z_i)) (sum_j a_ij) (1 + Lambda sum_m c_m^-1))
    (Sec. V-E), k_parts = number of partitions."""
    A = np.asarray(A, np.float64)
    p = np.asarray(p, np.float64)
    k_parts = A.shape[1]
    ph = np.array([phi(b, dim, eta) for b in bits])
    cinv = (1.0 - p) / (p + ph)
    return k_parts * lam / ((p + ph) * A.sum(axis=1) * (1.0 + lam * cinv.sum()))


def two_track_objective(v, A, p, bits, dim, lam=1.0, eta=1.0):
    """M(v) = Lambda*Bias(v) + Var(v) (Eq. twodec); returns (M, Bias, Var)."""
    A = np.asarray(A, np.float64)
    p = np.asarray(p, np.float64)
    v = np.asarray(v, np.float64)
    ph = np.array([phi(b, dim, eta) for b in bits])
    bias = float(np.sum(1.0 - ((1.0 - p) * v) @ A) ** 2)
    var = float(np.sum((1.0 - p) * (p + ph) * v ** 2 * A.sum(axis=1) ** 2))
    return lam * bias + var, bias, var
