// Status strings, version, per-thread error message, and the per-process caches behind the
// entry points: device properties, environment switches, encoded TMA tensor maps.
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <mutex>

#include "common.cuh"
#include "tensor_map.cuh"

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

static std::mutex g_mu;  // guards every cache below

// ---------------------------------------------------------------- devices
static DeviceInfo g_dev[kMaxDevices];
static bool g_dev_known[kMaxDevices] = {};
static bool g_once[kMaxDevices][ONCE_COUNT] = {};

pa_status current_sm100_device(DeviceInfo *out)
{
    int dev = 0;
    PA_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices)
        return fail(PA_ERR_UNSUPPORTED, "device index %d is beyond the %d devices supported", dev, kMaxDevices);
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (g_dev_known[dev]) {
            *out = g_dev[dev];
            if (out->cc_major != 10)
                return fail(PA_ERR_UNSUPPORTED, "device %d has compute capability %d.x; sm_100 required", dev,
                            out->cc_major);
            return PA_OK;
        }
    }
    DeviceInfo info;
    info.device = dev;
    PA_CUDA_OK(cudaDeviceGetAttribute(&info.cc_major, cudaDevAttrComputeCapabilityMajor, dev));
    PA_CUDA_OK(cudaDeviceGetAttribute(&info.sms, cudaDevAttrMultiProcessorCount, dev));
    {
        std::lock_guard<std::mutex> lock(g_mu);
        g_dev[dev] = info;
        g_dev_known[dev] = true;
    }
    *out = info;
    if (info.cc_major != 10)
        return fail(PA_ERR_UNSUPPORTED, "device %d has compute capability %d.x; sm_100 required", dev,
                    info.cc_major);
    return PA_OK;
}

bool device_once_begin(int device, DeviceOnce slot)
{
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_once[device][slot]) return false;
    g_once[device][slot] = true;
    return true;
}

void device_once_reset(int device, DeviceOnce slot)
{
    std::lock_guard<std::mutex> lock(g_mu);
    g_once[device][slot] = false;
}

// ---------------------------------------------------------------- environment
static EnvSwitches g_env;
static bool g_env_known = false;

static int env_int(const char *name, int lo, int hi)
{
    const char *e = getenv(name);
    const int v = e ? atoi(e) : 0;
    return v >= lo && v <= hi ? v : 0;
}

static void read_env_locked()
{
    const char *path = getenv("PA_DECODE_PATH");
    g_env.decode_path = !path ? 0 : path[0] == 's' ? 1 : path[0] == 'c' ? 2 : path[0] == 'p' ? 3 : 0;
    g_env.decode_cluster = env_int("PA_DECODE_CLUSTER", 1, 8);
    g_env.decode_stages = env_int("PA_DECODE_STAGES", 1, 8);
    g_env.decode_ctas_per_sm = env_int("PA_DECODE_CTAS_PER_SM", 1, 64);
    const char *bw = getenv("PA_BACKWARD_PATH");
    g_env.backward_mma = bw && bw[0] == 'm';
    const char *v = getenv("PA_VALIDATE");
    g_env.validate = v && v[0] == '1';
    g_env_known = true;
}

EnvSwitches env_switches()
{
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_env_known) read_env_locked();
    return g_env;
}

// ---------------------------------------------------------------- wait limit
static std::atomic<long long> g_wait_cycles{0};

long long wait_limit_cycles() { return g_wait_cycles.load(std::memory_order_relaxed); }

// ---------------------------------------------------------------- tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn g_encode = nullptr;

constexpr int kMapCacheSize = 64;
struct MapEntry {
    TensorMapKey key;
    CUtensorMap map;
    bool used;
};
static MapEntry g_maps[kMapCacheSize];
static int g_map_next = 0;

static bool same_key(const TensorMapKey &a, const TensorMapKey &b)
{
    return a.base == b.base && a.seq == b.seq && a.stride_seq == b.stride_seq && a.stride_head == b.stride_head &&
           a.stride_batch == b.stride_batch && a.device == b.device && a.head_dim == b.head_dim &&
           a.heads == b.heads && a.batch == b.batch && a.box_heads == b.box_heads && a.box_tokens == b.box_tokens;
}

pa_status get_tensor_map(const TensorMapKey &key, const char *what, CUtensorMap *out)
{
    std::lock_guard<std::mutex> lock(g_mu);
    for (int i = 0; i < kMapCacheSize; ++i)
        if (g_maps[i].used && same_key(g_maps[i].key, key)) {
            *out = g_maps[i].map;
            return PA_OK;
        }
    if (!g_encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        PA_CUDA_OK(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
        if (qres != cudaDriverEntryPointSuccess || !fn)
            return fail(PA_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
        g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    const cuuint64_t dims[4] = {(cuuint64_t)key.head_dim, (cuuint64_t)key.seq, (cuuint64_t)key.heads,
                                (cuuint64_t)key.batch};
    const cuuint64_t strides[3] = {
        (cuuint64_t)key.stride_seq * 2, (cuuint64_t)key.stride_head * 2,
        (cuuint64_t)(key.stride_batch > 0 ? key.stride_batch : key.stride_seq * key.seq) * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)key.box_tokens, (cuuint32_t)key.box_heads, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    CUtensorMap m;
    const CUresult r = g_encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(key.base), dims, strides,
                                box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return fail(PA_ERR_CUDA, "cuTensorMapEncodeTiled failed for %s (CUresult %d)", what, (int)r);
    MapEntry &e = g_maps[g_map_next];
    g_map_next = (g_map_next + 1) % kMapCacheSize;
    e.key = key;
    e.map = m;
    e.used = true;
    *out = m;
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

extern "C" int pa_version(void) { return 200; /* 0.2.0 */ }

extern "C" void pa_set_wait_limit_cycles(int64_t cycles)
{
    pa::g_wait_cycles.store(cycles > 0 ? (long long)cycles : 0, std::memory_order_relaxed);
}

extern "C" void pa_reload_environment(void)
{
    std::lock_guard<std::mutex> lock(pa::g_mu);
    pa::read_env_locked();
}
