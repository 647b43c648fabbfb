// Thread-local error message plumbing shared by the host parts of libqe.
#pragma once
#include <cstdarg>
#include <cstdint>

namespace qe {
// Records a formatted message for qe_last_error() and returns `status` unchanged.
int32_t fail(int32_t status, const char* fmt, ...);
void clear_error();
}  // namespace qe
