// Thread-local error text behind sw_last_error(); sw_fail formats it and returns the status.
#pragma once
#include "sw.h"

#if defined(__GNUC__)
#define SW_PRINTF_LIKE(a, b) __attribute__((format(printf, a, b)))
#else
#define SW_PRINTF_LIKE(a, b)
#endif

sw_status sw_fail(sw_status status, const char* fmt, ...) SW_PRINTF_LIKE(2, 3);
void sw_clear_error();
