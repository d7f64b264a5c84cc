// The uniform-interval family of EDEN, Section 4.3:
//     I_Delta = { [Delta (n - 1/2), Delta (n + 1/2)] : n integer },
// chosen so that the entropy of the interval probabilities under N(0,1) meets the bit
// budget (the message is meant for an entropy coder) while the interval of a coordinate
// is found by one rounding.  Values are centres of mass (Section 2.2.1).
#include "uniform_family.h"

#include <cmath>

namespace eden {
namespace {

const double kSqrtHalf = 0.70710678118654752440;
const double kInvSqrt2Pi = 0.39894228040143267794;

// P[z > t] for t >= 0
double upper_tail(double t) { return 0.5 * std::erfc(t * kSqrtHalf); }
double density(double t) { return kInvSqrt2Pi * std::exp(-0.5 * t * t); }

}  // namespace

double uniform_entropy(double delta)
{
    // walk outwards from the centre cell; each positive cell counts twice (its mirror)
    double edge_tail = upper_tail(0.5 * delta);          // P[z > Delta/2]
    const double centre = 1.0 - 2.0 * edge_tail;
    double bits = centre > 0.0 ? -centre * std::log2(centre) : 0.0;
    for (double edge = 0.5 * delta;; edge += delta) {
        const double next_tail = upper_tail(edge + delta);
        const double p = edge_tail - next_tail;
        if (!(p > 0.0)) break;
        bits -= 2.0 * p * std::log2(p);
        edge_tail = next_tail;
    }
    return bits;
}

double uniform_delta(double bits)
{
    // the entropy decreases with Delta: bisect on log Delta between the supported ends
    if (!(bits >= uniform_entropy(kUniformMaxDelta))) return 0.0;
    if (bits > uniform_entropy(kUniformMinDelta)) return 0.0;
    double lo = std::log(kUniformMinDelta), hi = std::log(kUniformMaxDelta);   // H(e^hi) <= bits
    for (int it = 0; it < 100; ++it) {
        const double mid = 0.5 * (lo + hi);
        if (uniform_entropy(std::exp(mid)) <= bits) hi = mid; else lo = mid;
    }
    const double delta = std::exp(hi);
    return delta < kUniformMaxDelta ? delta : 0.0;
}

void uniform_values(double delta, float* values)
{
    values[0] = 0.f;
    for (int m = 1; m < kUniformValues; ++m) {
        const double a = delta * (m - 0.5);
        const bool open = m == kUniformValues - 1;
        const double mass = upper_tail(a) - (open ? 0.0 : upper_tail(a + delta));
        // an interval so far out that its mass underflows takes its inner endpoint
        const double cm = mass > 0.0 ? (density(a) - (open ? 0.0 : density(a + delta))) / mass : a;
        values[m] = (float)cm;
    }
}

}  // namespace eden
