// Version, error strings and launch accounting of libardiff.
#include "../../include/ardiff.h"
#include "common.cuh"

namespace ardiff {
static thread_local int t_launches = 0;
void set_launch_count(int n) { t_launches = n; }
int get_launch_count() { return t_launches; }
}  // namespace ardiff

extern "C" const char* ardiff_strerror(int code) {
    switch (code) {
        case ARDIFF_OK: return "ok";
        case ARDIFF_ERR_NULL: return "a required pointer is NULL";
        case ARDIFF_ERR_SHAPE: return "a size is out of range";
        case ARDIFF_ERR_ALIGN: return "a pointer or pitch is misaligned";
        case ARDIFF_ERR_UNSUPPORTED: return "shape not supported by the kernels";
        case ARDIFF_ERR_CUDA: return "a CUDA call failed";
        case ARDIFF_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case ARDIFF_ERR_NOMEM: return "allocation failed";
        default: return "unknown ardiff error code";
    }
}

extern "C" int ardiff_version(void) { return 100; }

extern "C" int ardiff_last_launch_count(void) { return ardiff::get_launch_count(); }
