// Status strings, version, per-thread error message and device capability check.
#include <stdarg.h>
#include <stdio.h>

#include "common.cuh"

namespace pa {

static thread_local char g_err[512] = "";

pa_status fail(pa_status s, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
    return s;
}

void clear_error() { g_err[0] = '\0'; }

pa_status require_sm100()
{
    int dev = 0, major = 0;
    PA_CUDA_OK(cudaGetDevice(&dev));
    PA_CUDA_OK(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    if (major != 10)
        return fail(PA_ERR_UNSUPPORTED, "device %d has compute capability %d.x; sm_100 required",
                    dev, major);
    return PA_OK;
}

}  // namespace pa

extern "C" const char *pa_status_string(pa_status s)
{
    switch (s) {
        case PA_OK: return "PA_OK";
        case PA_ERR_INVALID_ARG: return "PA_ERR_INVALID_ARG";
        case PA_ERR_SHAPE: return "PA_ERR_SHAPE";
        case PA_ERR_ALIGNMENT: return "PA_ERR_ALIGNMENT";
        case PA_ERR_LAYOUT: return "PA_ERR_LAYOUT";
        case PA_ERR_WORKSPACE: return "PA_ERR_WORKSPACE";
        case PA_ERR_UNSUPPORTED: return "PA_ERR_UNSUPPORTED";
        case PA_ERR_CUDA: return "PA_ERR_CUDA";
        case PA_ERR_TIMEOUT: return "PA_ERR_TIMEOUT";
    }
    return "PA_ERR_UNKNOWN";
}

extern "C" const char *pa_last_error_message(void) { return pa::g_err; }

extern "C" int pa_version(void) { return 100; /* 0.1.0 */ }
