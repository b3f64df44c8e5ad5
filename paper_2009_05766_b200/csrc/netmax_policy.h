// Internal glue between the C-ABI translation units.
#pragma once
#include <string>

namespace netmax {
// Records the message netmax_last_error(NULL) returns on the calling thread.
void set_global_error(const std::string& msg);
}  // namespace netmax
