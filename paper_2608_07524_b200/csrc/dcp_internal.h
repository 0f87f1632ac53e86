// Internal helpers shared by the host-side translation units of libdcp (not part of the ABI).
#pragma once
#include <cstdarg>
#include <cstdio>

namespace dcp {

char* error_buffer();                       // thread-local, 512 bytes
inline int fail(int code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(error_buffer(), 512, fmt, ap);
    va_end(ap);
    return code;
}

}  // namespace dcp
