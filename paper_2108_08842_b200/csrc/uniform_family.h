// Host-side figures of the uniform-interval family I_Delta (EDEN, Section 4.3).
#pragma once

namespace eden {
constexpr int kUniformValues = 128;          // magnitude indices 0..127
constexpr double kUniformMinDelta = 0.0625;  // 127.5 intervals then reach ~8 standard deviations
constexpr double kUniformMaxDelta = 2.0;     // Section 4.3: the family is valid for Delta in (0, 2)

// entropy (bits per coordinate) of the interval probabilities under N(0,1)
double uniform_entropy(double delta);
// the smallest Delta whose entropy is at most `bits`; 0 if it is not in [min, max)
double uniform_delta(double bits);
// centre of mass of each interval [Delta (m - 1/2), Delta (m + 1/2)], m = 0..127; the last
// one is open-ended
void uniform_values(double delta, float* values);
}  // namespace eden
