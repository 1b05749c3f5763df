#include "sw_error.h"

#include <cstdarg>
#include <cstdio>

namespace {
thread_local char g_last_error[512] = "";
}

sw_status sw_fail(sw_status status, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    std::vsnprintf(g_last_error, sizeof g_last_error, fmt, ap);
    va_end(ap);
    return status;
}

void sw_clear_error() { g_last_error[0] = '\0'; }

extern "C" const char* sw_last_error(void) { return g_last_error; }
