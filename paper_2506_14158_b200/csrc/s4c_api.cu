// Version and error strings of the C ABI.
#include "s4c.h"

extern "C" int s4c_version(void) { return 100; }

extern "C" const char* s4c_status_string(s4c_status code) {
    switch (code) {
        case S4C_OK: return "ok";
        case S4C_ERR_NULL: return "a required pointer is NULL";
        case S4C_ERR_SHAPE: return "a size is out of range or inconsistent";
        case S4C_ERR_DTYPE: return "unknown dtype";
        case S4C_ERR_ALIGN: return "a tensor base pointer is not 16-byte aligned";
        case S4C_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case S4C_ERR_UNSUPPORTED: return "no kernel for this request";
        case S4C_ERR_CUDA: return "a CUDA runtime call failed";
    }
    return "unknown status";
}
