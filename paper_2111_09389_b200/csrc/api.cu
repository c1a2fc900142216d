// Version and status strings, the status-word read-back and the message byte count of the lpdt library.
#include "common.cuh"

extern "C" const char *lpdt_version(void) { return "lpdt 0.1 (sm_100a)"; }

extern "C" const char *lpdt_last_kernel(void) { return lpdt::g_last_kernel; }
extern "C" uint64_t lpdt_launch_count(void) { return lpdt::g_launch_count; }

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

// The one call of the library that waits: everything enqueued on `stream` so far has finished when it
// returns, and the value of the status word at that moment is the result.
extern "C" lpdt_status lpdt_check_status(const int32_t *dev_status, void *stream) {
    LPDT_CHECK_ARG(dev_status != nullptr);
    int32_t host = 0;
    cudaStream_t st = lpdt::as_stream(stream);
    LPDT_CUDA(cudaMemcpyAsync(&host, dev_status, sizeof(host), cudaMemcpyDeviceToHost, st));
    LPDT_CUDA(cudaStreamSynchronize(st));
    return (host >= LPDT_OK && host <= LPDT_ERR_OVERFLOW) ? (lpdt_status)host : LPDT_ERR_CUDA;
}

// Host arithmetic only: the size of what one node hands to each neighbour in one gossip step.
extern "C" int64_t lpdt_message_bytes(int64_t d, int32_t n_segments, const int64_t *seg_offsets,
                                      const int64_t *seg_k, int32_t value_bits, int32_t index_bits) {
    if (d < 0 || n_segments < 1 || !seg_offsets || !seg_k) return -1;
    if ((value_bits != 8 && value_bits != 16 && value_bits != 32) || index_bits < 0 || index_bits > 64) return -1;
    if (seg_offsets[0] != 0 || seg_offsets[n_segments] != d) return -1;
    int64_t bits = 0;
    for (int s = 0; s < n_segments; ++s) {
        const int64_t len = seg_offsets[s + 1] - seg_offsets[s];
        if (len < 0 || seg_k[s] < 0) return -1;
        const int64_t k = seg_k[s] < len ? seg_k[s] : len;
        bits += k * value_bits;
        if (k < len) bits += k * index_bits;          // a dense segment needs no positions
        if (value_bits == 8 && k > 0) bits += 32;      // the fp32 step of the segment's 8-bit codes
    }
    return (bits + 7) / 8;
}
