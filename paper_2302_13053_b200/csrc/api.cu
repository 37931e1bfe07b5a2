// Status strings and version of the retexo C ABI.
#include "common.cuh"

extern "C" const char* retexo_status_string(int status) {
    switch (status) {
        case RETEXO_OK: return "ok";
        case RETEXO_ERR_INVALID_ARG: return "invalid argument";
        case RETEXO_ERR_BAD_GRAPH: return "malformed CSR graph";
        case RETEXO_ERR_ALIGNMENT: return "pointer or leading dimension breaks an alignment rule";
        case RETEXO_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case RETEXO_ERR_UNSUPPORTED: return "shape not supported";
        case RETEXO_ERR_CUDA: return "CUDA runtime error or no CUDA device";
        case RETEXO_ERR_TIMEOUT: return "bounded device-side wait gave up";
        default: return "unknown status";
    }
}

extern "C" int retexo_version(void) { return 100; }
