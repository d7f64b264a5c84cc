// Lloyd-Max quantiser tables for N(0,1) (EDEN, Section 3), solved on the host in
// double precision when the library is first used.
//
// The quantiser with 2^W values is symmetric, so only the M = 2^(W-1) positive values
// c_0 < ... < c_{M-1} are unknown.  They satisfy
//     c_j = E[z | t_j <= z <= t_{j+1}],  t_0 = 0,  t_j = (c_{j-1} + c_j)/2,  t_M = inf
// (value = centre of mass of its interval, Section 2.2.1; boundary = midpoint because the
// interval rule equals the nearest-value rule, Section 3).  This file solves that system
// with Newton's method on its tridiagonal Jacobian, starting from the high-resolution
// point density (proportional to the cube root of the density, i.e. quantiles of
// N(0,3)), and polishes/falls back with plain Lloyd sweeps.
#include "lloyd_max.h"

#include <cmath>
#include <vector>

namespace eden {
namespace {

const double kInvSqrt2Pi = 0.39894228040143267794;
const double kSqrt2 = 1.41421356237309504880;

double pdf(double t) { return std::isinf(t) ? 0.0 : kInvSqrt2Pi * std::exp(-0.5 * t * t); }

// P[a <= z <= b] for 0 <= a < b, tail-safe
double mass(double a, double b)
{
    double ua = 0.5 * std::erfc(a / kSqrt2);
    double ub = std::isinf(b) ? 0.0 : 0.5 * std::erfc(b / kSqrt2);
    return ua - ub;
}

// upper-tail quantile: smallest t >= 0 with P[z > t] = q  (0 < q <= 0.5), by bisection
double upper_quantile(double q)
{
    double lo = 0.0, hi = 40.0;
    for (int i = 0; i < 200; ++i) {
        double mid = 0.5 * (lo + hi);
        if (0.5 * std::erfc(mid / kSqrt2) > q) lo = mid; else hi = mid;
    }
    return 0.5 * (lo + hi);
}

struct Cell { double cm, dca, dcb; };   // centre of mass and its partials w.r.t. the ends

Cell cell(double a, double b)
{
    double P = mass(a, b);
    double fa = pdf(a), fb = pdf(b);
    Cell r;
    r.cm = (fa - fb) / P;
    r.dca = fa * (r.cm - a) / P;
    r.dcb = std::isinf(b) ? 0.0 : fb * (b - r.cm) / P;
    return r;
}

double residual(const std::vector<double>& c, std::vector<double>* F)
{
    const int M = (int)c.size();
    double worst = 0.0;
    for (int j = 0; j < M; ++j) {
        double a = j == 0 ? 0.0 : 0.5 * (c[j - 1] + c[j]);
        double b = j == M - 1 ? INFINITY : 0.5 * (c[j] + c[j + 1]);
        double f = c[j] - cell(a, b).cm;
        if (F) (*F)[j] = f;
        worst = std::fmax(worst, std::fabs(f));
    }
    return worst;
}

bool increasing_positive(const std::vector<double>& c)
{
    if (!(c[0] > 0.0)) return false;
    for (size_t j = 1; j < c.size(); ++j)
        if (!(c[j] > c[j - 1])) return false;
    return true;
}

void lloyd_sweep(std::vector<double>& c)
{
    const int M = (int)c.size();
    std::vector<double> t(M + 1);
    t[0] = 0.0;
    t[M] = INFINITY;
    for (int j = 1; j < M; ++j) t[j] = 0.5 * (c[j - 1] + c[j]);
    for (int j = 0; j < M; ++j) c[j] = cell(t[j], t[j + 1]).cm;
}

}  // namespace

void lloyd_max_half(int W, std::vector<double>& c_out)
{
    const int M = 1 << (W - 1);
    std::vector<double> c(M);
    // start: quantiles of |N(0,3)| at the cell midpoints
    for (int j = 0; j < M; ++j)
        c[j] = std::sqrt(3.0) * upper_quantile(0.5 * (1.0 - (j + 0.5) / M));
    for (int i = 0; i < 50; ++i) lloyd_sweep(c);

    std::vector<double> F(M), lo(M), di(M), up(M), delta(M);
    for (int iter = 0; iter < 100; ++iter) {
        double r = residual(c, &F);
        if (r < 1e-15) break;
        // Jacobian rows
        for (int j = 0; j < M; ++j) {
            double a = j == 0 ? 0.0 : 0.5 * (c[j - 1] + c[j]);
            double b = j == M - 1 ? INFINITY : 0.5 * (c[j] + c[j + 1]);
            Cell k = cell(a, b);
            double ga = j == 0 ? 0.0 : 0.5 * k.dca;
            double gb = j == M - 1 ? 0.0 : 0.5 * k.dcb;
            lo[j] = -ga;
            di[j] = 1.0 - ga - gb;
            up[j] = -gb;
        }
        // Thomas algorithm for J delta = -F
        std::vector<double> cp(M), dp(M);
        cp[0] = up[0] / di[0];
        dp[0] = -F[0] / di[0];
        for (int j = 1; j < M; ++j) {
            double m = di[j] - lo[j] * cp[j - 1];
            cp[j] = up[j] / m;
            dp[j] = (-F[j] - lo[j] * dp[j - 1]) / m;
        }
        delta[M - 1] = dp[M - 1];
        for (int j = M - 2; j >= 0; --j) delta[j] = dp[j] - cp[j] * delta[j + 1];
        // damped update that keeps the values ordered and the residual falling
        double step = 1.0;
        bool ok = false;
        for (int tries = 0; tries < 30 && !ok; ++tries, step *= 0.5) {
            std::vector<double> trial(c);
            for (int j = 0; j < M; ++j) trial[j] += step * delta[j];
            if (increasing_positive(trial) && residual(trial, nullptr) < r) {
                c.swap(trial);
                ok = true;
            }
        }
        if (!ok) {                     // Newton stalled at rounding level or went astray
            if (r < 1e-13) break;
            for (int i = 0; i < 200; ++i) lloyd_sweep(c);
        }
    }
    c_out = c;
}

void lloyd_max_table(int W, std::vector<double>& centroids, std::vector<double>& boundaries)
{
    std::vector<double> c;
    lloyd_max_half(W, c);
    const int M = (int)c.size(), N = 2 * M;
    centroids.assign(N, 0.0);
    boundaries.assign(N - 1, 0.0);
    for (int j = 0; j < M; ++j) {
        centroids[M + j] = c[j];
        centroids[M - 1 - j] = -c[j];
    }
    boundaries[M - 1] = 0.0;
    for (int j = 1; j < M; ++j) {
        double t = 0.5 * (c[j - 1] + c[j]);
        boundaries[M - 1 + j] = t;
        boundaries[M - 1 - j] = -t;
    }
}

}  // namespace eden
