// Host-side design phase: bit allocation (problem b-SP1: exact DP of Eq. dp_rec and
// the low-complexity Algorithm 1) and code construction (Theorem 1, the interval
// construction of Sec. III-A, and the same objective on a caller-given support).
// Pure C++, no CUDA.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <limits>
#include <numeric>
#include <vector>

#include "../../include/agc.h"

namespace {

inline double levels_of(int b) { return double((1 << (b - 1)) - 1); }

// phi(z) = eta * l / (4 (2^(z-1)-1)^2) (Lemma 1, Sec. V-B). z = 1 is outside the paper:
// the two-point quantiser has per-coordinate variance <= S^2, hence phi(1) = eta * l.
inline double phi_of(int b, double dim, double eta)
{
    if (b <= 1) return eta * dim;
    const double L = levels_of(b);
    return eta * dim / (4.0 * L * L);
}

// utility table h[i][r] = (1-p_i) / (p_i + phi(r+2)), r = 0..cap+1
struct Utility {
    int n, cap;
    std::vector<double> h;
    Utility(int n_, int cap_, const double *p, double dim, double eta) : n(n_), cap(cap_), h(size_t(n_) * (cap_ + 2))
    {
        for (int i = 0; i < n; ++i)
            for (int r = 0; r <= cap + 1; ++r)
                h[size_t(i) * (cap + 2) + r] = (1.0 - p[i]) / (p[i] + phi_of(r + 2, dim, eta));
    }
    double operator()(int i, int r) const { return h[size_t(i) * (cap + 2) + r]; }
    double total(const std::vector<int> &r) const
    {
        double F = 0.0;
        for (int i = 0; i < n; ++i) F += (*this)(i, r[i]);
        return F;
    }
};

int check_alloc_args(int n, const double *p, int Z_tot, int b_min, int b_max, double phi_dim,
                     double eta, const uint8_t *bits_out, int *z_res, int *cap)
{
    if (n < 1 || !p || !bits_out || b_min != 2 || !(phi_dim > 0.0) || !(eta > 0.0)) return AGC_ERR_ARG;
    if (b_max != 0 && (b_max < 2 || b_max > 255)) return AGC_ERR_ARG;
    for (int i = 0; i < n; ++i)
        if (!(p[i] >= 0.0 && p[i] < 1.0)) return AGC_ERR_PROB;
    const long long zr = (long long)Z_tot - 2LL * n;
    if (zr < 0 || zr > 253LL * n || zr > (1 << 24)) return AGC_ERR_BUDGET;
    *z_res = int(zr);
    *cap = b_max ? std::min<int>(*z_res, b_max - 2) : std::min(*z_res, 253);
    if ((long long)(*cap) * n < zr) return AGC_ERR_BUDGET;
    return AGC_OK;
}

// slope of the continuous relaxation of h_i at real r (levels 2^(r+1) - 1)
inline double h_slope(double p, double r, double dim, double eta)
{
    const double two = std::exp2(r + 1.0);
    const double lev = two - 1.0;
    const double ph = eta * dim / (4.0 * lev * lev);
    const double dph = -2.0 * ph * two * 0.6931471805599453 / lev;
    return -(1.0 - p) * dph / ((p + ph) * (p + ph));
}

// Continuous relaxation on the active workers: stationarity h_i'(r_i) = lambda on the
// concave side of each sigmoid (r_i = 0 when lambda is above the steepest slope),
// lambda by bisection to meet the budget, then floor + largest remainders.
bool lagrangian_allocation(const std::vector<double> &p, int z_res, int cap, double dim, double eta,
                           std::vector<int> &out)
{
    const int m = int(p.size());
    std::vector<double> peak(m), peak_slope(m), cap_slope(m);
    for (int t = 0; t < m; ++t) {
        double best = -1.0, at = 0.0;
        for (int g = 0; g <= 2048; ++g) {
            const double r = double(cap) * g / 2048.0;
            const double s = h_slope(p[t], r, dim, eta);
            if (s > best) { best = s; at = r; }
        }
        peak[t] = at;
        peak_slope[t] = best;
        cap_slope[t] = h_slope(p[t], double(cap), dim, eta);
    }
    auto r_of = [&](double lam, std::vector<double> &r) {
        double sum = 0.0;
        for (int t = 0; t < m; ++t) {
            double v;
            if (lam >= peak_slope[t]) v = 0.0;
            else if (cap_slope[t] >= lam) v = double(cap);
            else {
                double lo = peak[t], hi = double(cap);
                for (int it = 0; it < 50; ++it) {
                    const double mid = 0.5 * (lo + hi);
                    if (h_slope(p[t], mid, dim, eta) > lam) lo = mid; else hi = mid;
                }
                v = 0.5 * (lo + hi);
            }
            r[t] = v;
            sum += v;
        }
        return sum;
    };
    std::vector<double> rr(m);
    double lo = 0.0, hi = *std::max_element(peak_slope.begin(), peak_slope.end());
    for (int it = 0; it < 60; ++it) {
        const double mid = 0.5 * (lo + hi);
        if (r_of(mid, rr) > double(z_res)) lo = mid; else hi = mid;
    }
    r_of(hi, rr);
    out.assign(m, 0);
    std::vector<double> frac(m);
    int used = 0;
    for (int t = 0; t < m; ++t) {
        const double fl = std::floor(rr[t] + 1e-12);
        out[t] = std::min(int(fl), cap);
        frac[t] = rr[t] - fl;
        used += out[t];
    }
    int left = z_res - used;
    while (left < 0) {  // cannot happen after flooring; kept for safety
        int t = int(std::max_element(out.begin(), out.end()) - out.begin());
        --out[t]; ++left;
    }
    while (left > 0) {
        std::vector<int> order(m);
        std::iota(order.begin(), order.end(), 0);
        std::stable_sort(order.begin(), order.end(), [&](int x, int y) { return frac[x] > frac[y]; });
        bool progressed = false;
        for (int t : order) {
            if (left == 0) break;
            if (out[t] < cap) { ++out[t]; --left; progressed = true; }
        }
        if (!progressed) return false;
        std::fill(frac.begin(), frac.end(), 0.0);
    }
    return true;
}

}  // namespace

extern "C" int agc_bit_allocate_dp(int n, const double *p, int Z_tot, int b_min, int b_max,
                                   double phi_dim, double eta, uint8_t *bits_out, double *F_out)
{
    int z_res, cap;
    if (int e = check_alloc_args(n, p, Z_tot, b_min, b_max, phi_dim, eta, bits_out, &z_res, &cap)) return e;
    Utility h(n, cap, p, phi_dim, eta);
    const double NEG = -std::numeric_limits<double>::infinity();
    std::vector<double> prev(z_res + 1, NEG), cur(z_res + 1);
    std::vector<int> arg(size_t(n) * (z_res + 1));
    prev[0] = 0.0;
    for (int i = 0; i < n; ++i) {
        for (int r = 0; r <= z_res; ++r) {
            double best = NEG;
            int best_a = 0;
            for (int a = 0; a <= std::min(r, cap); ++a) {
                const double v = prev[r - a] + h(i, a);
                if (v > best) { best = v; best_a = a; }
            }
            cur[r] = best;
            arg[size_t(i) * (z_res + 1) + r] = best_a;
        }
        prev.swap(cur);
    }
    int rem = z_res;
    for (int i = n - 1; i >= 0; --i) {
        const int a = arg[size_t(i) * (z_res + 1) + rem];
        bits_out[i] = uint8_t(a + 2);
        rem -= a;
    }
    if (F_out) *F_out = prev[z_res];
    return AGC_OK;
}

extern "C" int agc_bit_allocate(int n, const double *p, int Z_tot, int b_min, int b_max,
                                double phi_dim, double eta, uint8_t *bits_out, double *F_out)
{
    int z_res, cap;
    if (int e = check_alloc_args(n, p, Z_tot, b_min, b_max, phi_dim, eta, bits_out, &z_res, &cap)) return e;
    Utility h(n, cap, p, phi_dim, eta);
    std::vector<int> order(n);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int x, int y) { return p[x] < p[y]; });

    std::vector<int> best(n, 0);
    double best_F = z_res == 0 ? h.total(best) : -std::numeric_limits<double>::infinity();
    for (int kappa = 1; kappa <= std::min(n, z_res); ++kappa) {
        if ((long long)kappa * cap < z_res) continue;
        // equal allocation on the kappa most reliable workers
        std::vector<int> r(n, 0);
        for (int t = 0; t < kappa; ++t) r[order[t]] = z_res / kappa + (t < z_res % kappa ? 1 : 0);
        double F = h.total(r);
        // Lagrangian candidate on the same set
        std::vector<double> psel(kappa);
        for (int t = 0; t < kappa; ++t) psel[t] = p[order[t]];
        std::vector<int> rsel;
        if (lagrangian_allocation(psel, z_res, cap, phi_dim, eta, rsel)) {
            std::vector<int> rl(n, 0);
            for (int t = 0; t < kappa; ++t) rl[order[t]] = rsel[t];
            const double Fl = h.total(rl);
            if (Fl > F) { F = Fl; r.swap(rl); }
        }
        // one-bit local search: best improving move of one bit from worker j to worker i
        for (;;) {
            double gain = 0.0;
            int gi = -1, gj = -1;
            for (int i = 0; i < n; ++i) {
                if (r[i] >= cap) continue;
                const double up = h(i, r[i] + 1) - h(i, r[i]);
                for (int j = 0; j < n; ++j) {
                    if (j == i || r[j] == 0) continue;
                    const double g = up + h(j, r[j] - 1) - h(j, r[j]);
                    if (g > gain) { gain = g; gi = i; gj = j; }
                }
            }
            if (gi < 0 || gain <= 1e-12 * std::fabs(F)) break;
            ++r[gi]; --r[gj];
            F = h.total(r);
        }
        if (F > best_F) { best_F = F; best = r; }
    }
    for (int i = 0; i < n; ++i) bits_out[i] = uint8_t(best[i] + 2);
    if (F_out) *F_out = best_F;
    return AGC_OK;
}

// The two heuristics the paper's Fig. 2 sets Algorithm 1 against (Sec. VI names them without
// printing them; these are the readings taken) and an upper bound on the optimum.
extern "C" int agc_bit_allocate_heuristic(int method, int n, const double *p, int Z_tot, int b_min, int b_max,
                                          double phi_dim, double eta, uint8_t *bits_out, double *F_out)
{
    int z_res, cap;
    if (method != AGC_ALLOC_GREEDY && method != AGC_ALLOC_RELAXATION) return AGC_ERR_ARG;
    if (int e = check_alloc_args(n, p, Z_tot, b_min, b_max, phi_dim, eta, bits_out, &z_res, &cap)) return e;
    Utility h(n, cap, p, phi_dim, eta);
    std::vector<int> r(n, 0);
    if (method == AGC_ALLOC_GREEDY) {
        // one bit at a time to the worker that gains most from it (ties: lowest index)
        for (int bit = 0; bit < z_res; ++bit) {
            double best = -std::numeric_limits<double>::infinity();
            int at = -1;
            for (int i = 0; i < n; ++i) {
                if (r[i] >= cap) continue;
                const double g = h(i, r[i] + 1) - h(i, r[i]);
                if (g > best) { best = g; at = i; }
            }
            ++r[at];
        }
    } else if (z_res > 0) {
        // the relaxed problem's stationarity system over all workers, rounded
        std::vector<double> pall(p, p + n);
        if (!lagrangian_allocation(pall, z_res, cap, phi_dim, eta, r)) {
            for (int i = 0; i < n; ++i) r[i] = z_res / n + (i < z_res % n ? 1 : 0);
        }
    }
    for (int i = 0; i < n; ++i) bits_out[i] = uint8_t(r[i] + 2);
    if (F_out) *F_out = h.total(r);
    return AGC_OK;
}

extern "C" int agc_allocation_upper_bound(int n, const double *p, int Z_tot, int b_min, int b_max, double phi_dim,
                                          double eta, double *bound_out)
{
    int z_res, cap;
    uint8_t dummy = 0;
    if (!bound_out) return AGC_ERR_ARG;
    if (int e = check_alloc_args(n, p, Z_tot, b_min, b_max, phi_dim, eta, &dummy, &z_res, &cap)) return e;
    Utility h(n, cap, p, phi_dim, eta);
    // upper concave envelope of each worker's integer points; the envelope's unit slopes,
    // largest first, solve the separable concave problem exactly
    std::vector<double> slopes;
    double base = 0.0;
    for (int i = 0; i < n; ++i) {
        base += h(i, 0);
        std::vector<int> hull(1, 0);
        for (int a = 1; a <= cap; ++a) {
            while (hull.size() >= 2) {
                const int a0 = hull[hull.size() - 2], a1 = hull.back();
                if ((h(i, a1) - h(i, a0)) * (a - a0) <= (h(i, a) - h(i, a0)) * (a1 - a0)) hull.pop_back();
                else break;
            }
            hull.push_back(a);
        }
        for (size_t t = 0; t + 1 < hull.size(); ++t) {
            const int a0 = hull[t], a1 = hull[t + 1];
            for (int u = a0; u < a1; ++u) slopes.push_back((h(i, a1) - h(i, a0)) / (a1 - a0));
        }
    }
    std::sort(slopes.begin(), slopes.end(), [](double x, double y) { return x > y; });
    double bound = base;
    for (int t = 0; t < z_res && t < int(slopes.size()); ++t) bound += slopes[t];
    *bound_out = bound;
    return AGC_OK;
}

extern "C" int agc_code_build(int n, int k, const double *p, const uint8_t *bits, double phi_dim,
                              double eta, int mode, const int32_t *sup_row_ptr,
                              const int32_t *sup_col_idx, int32_t nnz_cap, int32_t *row_ptr_out,
                              int32_t *col_out, float *a_out, float *w_out, double *Y_out)
{
    if (n < 1 || k < 1 || !p || !bits || !row_ptr_out || !col_out || !a_out || !w_out) return AGC_ERR_ARG;
    if (!(phi_dim > 0.0) || !(eta > 0.0)) return AGC_ERR_ARG;
    std::vector<double> c(n);
    double sum_cinv = 0.0;
    for (int i = 0; i < n; ++i) {
        if (!(p[i] >= 0.0 && p[i] < 1.0)) return AGC_ERR_PROB;
        if (bits[i] < 1 || bits[i] > 8) return AGC_ERR_BITS;
        c[i] = (p[i] + phi_of(bits[i], phi_dim, eta)) / (1.0 - p[i]);
        sum_cinv += 1.0 / c[i];
    }
    std::vector<std::vector<int>> cols(n);
    std::vector<std::vector<double>> alpha(n);

    if (mode == AGC_CODE_INTERVAL) {
        // worker i owns [R_{i-1}, R_i] on the partition axis [0, k]; partition j owns [j-1, j]
        double lo = 0.0;
        for (int i = 0; i < n; ++i) {
            const double Y = (1.0 / c[i]) * double(k) / sum_cinv;
            const double hi = (i == n - 1) ? double(k) : lo + Y;
            const int j0 = std::max(0, int(std::floor(lo)));
            const int j1 = std::min(k - 1, int(std::ceil(hi)) - 1);
            for (int j = j0; j <= j1; ++j) {
                const double ov = std::min(hi, double(j + 1)) - std::max(lo, double(j));
                if (ov > 0.0) { cols[i].push_back(j); alpha[i].push_back(ov); }
            }
            lo = hi;
        }
    } else if (mode == AGC_CODE_SUPPORT) {
        if (!sup_row_ptr || !sup_col_idx || sup_row_ptr[0] != 0) return AGC_ERR_ARG;
        std::vector<std::vector<std::pair<int, int>>> by_col(k);  // (worker, position in its row)
        for (int i = 0; i < n; ++i) {
            if (sup_row_ptr[i + 1] < sup_row_ptr[i]) return AGC_ERR_ARG;
            for (int e = sup_row_ptr[i]; e < sup_row_ptr[i + 1]; ++e) {
                const int j = sup_col_idx[e];
                if (j < 0 || j >= k || (e > sup_row_ptr[i] && j <= sup_col_idx[e - 1])) return AGC_ERR_ARG;
                by_col[j].push_back({i, int(cols[i].size())});
                cols[i].push_back(j);
                alpha[i].push_back(0.0);
            }
        }
        for (int j = 0; j < k; ++j) {
            if (by_col[j].empty()) return AGC_ERR_ARG;  // a partition nobody holds cannot be unbiased
            for (auto &wp : by_col[j]) alpha[wp.first][wp.second] = 1.0 / double(by_col[j].size());
        }
        // Block coordinate descent, one partition (column) at a time. With the other
        // columns fixed, column j solves min sum_i c_i (z_i + x_i)^2, sum x_i = 1, x >= 0,
        // whose solution is x_i = max(0, t / c_i - z_i) with t set by the budget.
        std::vector<double> y(n, 0.0);
        for (int i = 0; i < n; ++i) y[i] = std::accumulate(alpha[i].begin(), alpha[i].end(), 0.0);
        for (int sweep = 0; sweep < 20000; ++sweep) {
            double moved = 0.0;
            for (int j = 0; j < k; ++j) {
                auto &ws = by_col[j];
                const int m = int(ws.size());
                std::vector<double> z(m);
                std::vector<int> ord(m);
                for (int t = 0; t < m; ++t) { z[t] = y[ws[t].first] - alpha[ws[t].first][ws[t].second]; ord[t] = t; }
                std::sort(ord.begin(), ord.end(), [&](int a, int b) { return c[ws[a].first] * z[a] < c[ws[b].first] * z[b]; });
                double sz = 0.0, sinv = 0.0, level = 0.0;
                for (int t = 0; t < m; ++t) {
                    const int u = ord[t];
                    sz += z[u];
                    sinv += 1.0 / c[ws[u].first];
                    level = (1.0 + sz) / sinv;
                    if (t + 1 == m || level <= c[ws[ord[t + 1]].first] * z[ord[t + 1]]) break;
                }
                for (int t = 0; t < m; ++t) {
                    const int i = ws[t].first;
                    const double x = std::max(0.0, level / c[i] - z[t]);
                    moved = std::max(moved, std::fabs(x - alpha[i][ws[t].second]));
                    alpha[i][ws[t].second] = x;
                    y[i] = z[t] + x;
                }
            }
            if (moved < 1e-15) break;
        }
    } else {
        return AGC_ERR_ARG;
    }

    // drop negligible entries, renormalise every column to 1 exactly, emit CSR with w~ = 1
    std::vector<double> colsum(k, 0.0);
    for (int i = 0; i < n; ++i)
        for (size_t t = 0; t < cols[i].size(); ++t) {
            if (alpha[i][t] < 1e-12) alpha[i][t] = 0.0;
            colsum[cols[i][t]] += alpha[i][t];
        }
    for (int j = 0; j < k; ++j)
        if (!(colsum[j] > 0.0)) return AGC_ERR_UNBIASED;
    int nnz = 0;
    row_ptr_out[0] = 0;
    for (int i = 0; i < n; ++i) {
        double Y = 0.0;
        for (size_t t = 0; t < cols[i].size(); ++t) {
            if (alpha[i][t] == 0.0) continue;
            if (nnz >= nnz_cap) return AGC_ERR_ARG;
            const double v = alpha[i][t] / colsum[cols[i][t]];
            col_out[nnz] = cols[i][t];
            a_out[nnz] = float(v);
            Y += v;
            ++nnz;
        }
        row_ptr_out[i + 1] = nnz;
        w_out[i] = float(1.0 / (1.0 - p[i]));
        if (Y_out) Y_out[i] = Y;
    }
    return AGC_OK;
}

extern "C" int agc_two_track_vector(int n, int k, const double *p, const uint8_t *bits, double phi_dim,
                                    double eta, double lambda, const int32_t *row_ptr, const float *a,
                                    float *v_out)
{
    if (n < 1 || k < 1 || !p || !bits || !row_ptr || !a || !v_out || !(phi_dim > 0.0) || !(eta > 0.0) ||
        !(lambda > 0.0))
        return AGC_ERR_ARG;
    double sum_cinv = 0.0;
    for (int i = 0; i < n; ++i) {
        if (!(p[i] >= 0.0 && p[i] < 1.0)) return AGC_ERR_PROB;
        if (bits[i] < 1 || bits[i] > 8) return AGC_ERR_BITS;
        sum_cinv += (1.0 - p[i]) / (p[i] + phi_of(bits[i], phi_dim, eta));
    }
    for (int i = 0; i < n; ++i) {
        double row = 0.0;
        for (int e = row_ptr[i]; e < row_ptr[i + 1]; ++e) row += double(a[e]);
        const double den = (p[i] + phi_of(bits[i], phi_dim, eta)) * row * (1.0 + lambda * sum_cinv);
        v_out[i] = row > 0.0 ? float(double(k) * lambda / den) : 0.0f;
    }
    return AGC_OK;
}

extern "C" int agc_eta_balance(int n, const double *p, int Z_tot, double phi_dim, double *eta_out)
{
    if (n < 1 || !p || !eta_out || !(phi_dim > 0.0) || Z_tot < 2 * n) return AGC_ERR_ARG;
    double mean = 0.0;
    for (int i = 0; i < n; ++i) {
        if (!(p[i] >= 0.0 && p[i] < 1.0)) return AGC_ERR_PROB;
        mean += p[i];
    }
    mean /= double(n);
    const double lev = std::exp2(double(Z_tot) / double(n) - 1.0) - 1.0;
    *eta_out = mean * 4.0 * lev * lev / phi_dim;
    return AGC_OK;
}
