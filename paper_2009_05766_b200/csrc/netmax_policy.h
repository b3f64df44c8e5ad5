// Internal glue between the C-ABI translation units.
#pragma once
#include <string>
#include <vector>

namespace netmax {
// Records the message netmax_last_error(NULL) returns on the calling thread.
void set_global_error(const std::string& msg);
// Largest eigenvalue of a symmetric tridiagonal matrix (diagonal alpha, off-diagonal beta).
double tridiagonal_top_eigenvalue(const std::vector<double>& alpha, const std::vector<double>& beta);
}  // namespace netmax
