// Shared host-side helpers of the library: error reporting and argument checks.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "powerattn.h"

namespace pa {

// Records a message for pa_last_error_message() and returns `s`.
pa_status fail(pa_status s, const char *fmt, ...);
void clear_error();

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// PA_OK if the current device is an sm_100 part, else PA_ERR_UNSUPPORTED / PA_ERR_CUDA.
pa_status require_sm100();

#define PA_CUDA_OK(expr)                                                                    \
    do {                                                                                    \
        cudaError_t e_ = (expr);                                                            \
        if (e_ != cudaSuccess)                                                              \
            return ::pa::fail(PA_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e_)); \
    } while (0)

}  // namespace pa
