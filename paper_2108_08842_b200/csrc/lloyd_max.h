// Host-side Lloyd-Max table solver for N(0,1) (EDEN, Section 3).
#pragma once
#include <vector>

namespace eden {
// positive half of the 2^W-value quantiser, ascending
void lloyd_max_half(int W, std::vector<double>& c_out);
// all 2^W values ascending and the 2^W - 1 boundaries between them
void lloyd_max_table(int W, std::vector<double>& centroids, std::vector<double>& boundaries);
}  // namespace eden
