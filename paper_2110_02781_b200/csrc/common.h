// Internal helpers shared by the library's translation units.
#pragma once
#include <cstdarg>
#include <cstdio>
#include "ftpipe.h"

namespace ftp {

char* last_error_buf();                 // thread-local, 512 bytes
ftp_status fail(ftp_status s, const char* fmt, ...);

#define FTP_REQUIRE(cond, status, ...)            \
    do {                                          \
        if (!(cond)) return ::ftp::fail(status, __VA_ARGS__); \
    } while (0)

}  // namespace ftp
