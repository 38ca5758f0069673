// Version and status strings.
#include "afx.h"

extern "C" afx_status afx_version(int* major, int* minor) {
    if (major != nullptr) *major = 0;
    if (minor != nullptr) *minor = 1;
    return AFX_OK;
}

extern "C" const char* afx_status_string(afx_status s) {
    switch (s) {
        case AFX_OK: return "AFX_OK";
        case AFX_ERR_INVALID_ARG: return "AFX_ERR_INVALID_ARG";
        case AFX_ERR_ALIGNMENT: return "AFX_ERR_ALIGNMENT";
        case AFX_ERR_CAPACITY: return "AFX_ERR_CAPACITY";
        case AFX_ERR_UNSUPPORTED: return "AFX_ERR_UNSUPPORTED";
        case AFX_ERR_CUDA: return "AFX_ERR_CUDA";
        case AFX_ERR_TIMEOUT: return "AFX_ERR_TIMEOUT";
        default: return "AFX_ERR_UNKNOWN";
    }
}

#ifdef AFX_TRACE
#include <cuda_runtime.h>
__device__ long long afx_trace_buf[8 * 512 * 16];
extern "C" int afx_trace_read(long long* host_out) {
    return cudaMemcpyFromSymbol(host_out, afx_trace_buf, sizeof(long long) * 8 * 512 * 16) == cudaSuccess ? 0 : 1;
}
#endif
