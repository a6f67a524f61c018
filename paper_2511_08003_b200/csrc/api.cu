// Version and status strings of the SharpV CUDA library.
#include "sharpv.h"

// 1xx: release build, 2xx: built with -DSHARPV_DEBUG_BOUNDS (every gather / scatter index range-checked)
#ifdef SHARPV_DEBUG_BOUNDS
extern "C" int sharpv_version(void) { return 201; }
#else
extern "C" int sharpv_version(void) { return 101; }
#endif

extern "C" const char* sharpv_status_string(sharpv_status s) {
    switch (s) {
        case SHARPV_OK: return "ok";
        case SHARPV_ERR_INVALID_ARG: return "invalid argument";
        case SHARPV_ERR_UNSUPPORTED: return "unsupported dtype, alignment or size";
        case SHARPV_ERR_WORKSPACE: return "workspace too small";
        case SHARPV_ERR_CAPACITY: return "more survivors than capacity";
        case SHARPV_ERR_CUDA: return "CUDA runtime error";
        case SHARPV_ERR_TIMEOUT: return "bounded device wait gave up";
        case SHARPV_ERR_BOUNDS: return "index out of range (debug build)";
    }
    return "unknown status";
}
