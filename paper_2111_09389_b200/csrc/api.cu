// Version and status strings of the lpdt library.
#include "common.cuh"

extern "C" const char *lpdt_version(void) { return "lpdt 0.1 (sm_100a)"; }

extern "C" lpdt_status lpdt_fill_zero(void *p, size_t bytes, void *stream) {
    if (bytes == 0) return LPDT_OK;
    LPDT_CHECK_ARG(p != nullptr);
    LPDT_CUDA(cudaMemsetAsync(p, 0, bytes, lpdt::as_stream(stream)));
    return LPDT_OK;
}

extern "C" const char *lpdt_status_string(lpdt_status s) {
    switch (s) {
        case LPDT_OK: return "ok";
        case LPDT_ERR_INVALID_ARG: return "invalid argument";
        case LPDT_ERR_UNSUPPORTED: return "unsupported shape or mode";
        case LPDT_ERR_WORKSPACE: return "workspace missing or too small";
        case LPDT_ERR_CUDA: return "CUDA call failed";
        case LPDT_ERR_TIMEOUT: return "device-side wait timed out";
        case LPDT_ERR_OVERFLOW: return "integer overflow";
        default: return "unknown status";
    }
}
