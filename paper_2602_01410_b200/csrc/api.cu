// Library information, status helpers and device check.
#include <string.h>

#include "common.cuh"

namespace snip {

char *last_error_buffer()
{
    static thread_local char buf[256] = {0};
    return buf;
}

void set_last_error(const char *where, cudaError_t e)
{
    snprintf(last_error_buffer(), 256, "%s: %s (%s)", where, cudaGetErrorName(e), cudaGetErrorString(e));
}

int require_sm100()
{
    static thread_local int cached_dev = -1;
    static thread_local int cached_rc = SNIP_OK;
    int dev = 0;
    SNIP_CUDA_TRY(cudaGetDevice(&dev));
    if (dev == cached_dev) return cached_rc;
    int major = 0;
    SNIP_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    cached_dev = dev;
    cached_rc = (major == 10) ? SNIP_OK : SNIP_ERR_UNSUPPORTED;
    return cached_rc;
}

}  // namespace snip

extern "C" int snip_version(void) { return 100; /* 0.1.0 */ }

extern "C" const char *snip_status_string(int status)
{
    switch (status) {
        case SNIP_OK: return "SNIP_OK";
        case SNIP_ERR_ARG: return "SNIP_ERR_ARG";
        case SNIP_ERR_SHAPE: return "SNIP_ERR_SHAPE";
        case SNIP_ERR_ALIGN: return "SNIP_ERR_ALIGN";
        case SNIP_ERR_UNSUPPORTED: return "SNIP_ERR_UNSUPPORTED";
        case SNIP_ERR_WORKSPACE: return "SNIP_ERR_WORKSPACE";
        case SNIP_ERR_CUDA: return "SNIP_ERR_CUDA";
        case SNIP_ERR_TIMEOUT: return "SNIP_ERR_TIMEOUT";
        default: return "SNIP_ERR_UNKNOWN";
    }
}

extern "C" const char *snip_last_cuda_error(void) { return snip::last_error_buffer(); }
