// Shared host-side helpers of the library: error reporting, argument checks, and the small
// per-process caches (device properties, environment switches) that keep repeated calls cheap.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "powerattn.h"

namespace pa {

// Records a message for pa_last_error_message() and returns `s`.
pa_status fail(pa_status s, const char *fmt, ...);
void clear_error();

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

constexpr int kMaxDevices = 64;

// Properties of the current device, looked up once per device and process.
struct DeviceInfo {
    int device, sms, cc_major;
};
// PA_OK with *out filled in if the current device is an sm_100 part, else PA_ERR_UNSUPPORTED /
// PA_ERR_CUDA.
pa_status current_sm100_device(DeviceInfo *out);

// One-time per-device set-up steps (kernel attributes) are keyed by these slots.
enum DeviceOnce : int { ONCE_PREFILL_ATTR = 0, ONCE_DECODE_ATTR, ONCE_BACKWARD_ATTR, ONCE_BACKWARD_ATTR_64, ONCE_BACKWARD_TC_ATTR, ONCE_COUNT };
// True exactly once per (device, slot); the caller then performs the step and, if it fails, calls
// device_once_reset so that a later call tries again.
bool device_once_begin(int device, DeviceOnce slot);
void device_once_reset(int device, DeviceOnce slot);

// Environment switches (for tests and measurements).  They are read when the library first needs
// them and again on pa_reload_environment().
struct EnvSwitches {
    int decode_path;     // PA_DECODE_PATH: 0 unset, 1 splitk, 2 cluster, 3 persistent
    int decode_cluster;  // PA_DECODE_CLUSTER=1..8 chunks per row, 0 = chosen from the problem size
    int decode_stages;   // PA_DECODE_STAGES=1..8, 0 = chosen from the problem size
    int decode_ctas_per_sm;  // PA_DECODE_CTAS_PER_SM=n: size of the persistent grid (default 2 per SM)
    int validate;        // PA_VALIDATE=1
    int backward_mma;    // PA_BACKWARD_PATH=mma: the warp-level MMA kernels for head_dim 128 too
};
EnvSwitches env_switches();

// Limit of the kernels' bounded barrier waits in clock cycles as set by pa_set_wait_limit_cycles
// (0: each kernel's default).
long long wait_limit_cycles();

#define PA_CUDA_OK(expr)                                                                    \
    do {                                                                                    \
        cudaError_t e_ = (expr);                                                            \
        if (e_ != cudaSuccess)                                                              \
            return ::pa::fail(PA_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e_)); \
    } while (0)

}  // namespace pa
