// Host-side log of the library's decisions, switched on by the environment variable
// LGN_LOG (any value but empty or "0"), read once per process: which kernel a call takes,
// its launch shape and queue, which selection path a quantile takes, why an argument
// was refused.  One line per decision on stderr, prefixed "[lgn] "; nothing is printed,
// and nothing but one branch is executed, when the variable is not set.
#pragma once

#include <cstdarg>
#include <cstdio>
#include <cstdlib>

namespace lgn {

inline bool log_enabled() {
    static const bool on = [] {
        const char *e = std::getenv("LGN_LOG");
        return e != nullptr && e[0] != '\0' && !(e[0] == '0' && e[1] == '\0');
    }();
    return on;
}

inline void log_line(const char *fmt, ...) {
    if (!log_enabled()) return;
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    std::vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    std::fprintf(stderr, "[lgn] %s\n", buf);
}

}  // namespace lgn
