// pa_decode: one query token per sequence against its KV cache under the PowerAttention row of
// its position (Section 4.1: same pattern in prefilling and decoding; Eq. (1) for the row).
//
// Split-K: one CTA per (sequence, KV head, chunk) where a chunk is one 64-key block of the
// row's block list.  Each CTA stages its K and V block in shared memory with coalesced 16-byte
// asynchronous copies, computes the logits of all query heads of the group, a chunk-local
// softmax (warp-shuffle reductions) and the unnormalised partial output, and writes
// (o[D], m, l) per head to the workspace.  A second kernel merges the chunks with the
// log-sum-exp rule.  The second launch overlaps the first one's tail through programmatic
// dependent launch; it waits for the partials with griddepcontrol.wait.
#include <cuda_bf16.h>
#include <math.h>

#include "common.cuh"
#include "layout_rule.cuh"

namespace pa {

constexpr int kDecBlock = 64;     // keys per block (the only supported block size)
constexpr int kDecThreads = 128;  // threads per CTA of the partial kernel
constexpr int kMaxGroup = 8;      // query heads per KV head supported by the partial kernel

struct DecodeArgs {
    const __nv_bfloat16 *q, *k, *v;
    const int32_t *lens;
    float *partial;  // [batch, Hq, chunks, D + 2]
    void *o;
    float *lse;
    int64_t k_sb, k_ss, k_sh, v_sb, v_ss, v_sh;
    int64_t max_len;
    int32_t batch, Hq, Hkv, G, W, S, chunks, o_is_f32;
    float scale_log2;  // softmax_scale * log2(e)
};

__device__ __forceinline__ void cp_async16(void *smem, const void *gmem)
{
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

// Physical 16-byte chunk of logical chunk c in row r: XOR with the row keeps the eight rows a
// quarter-warp reads at one logical column in different banks.
template <int D>
__device__ __forceinline__ int swz(int r, int c)
{
    return r * (D / 8) + (c ^ (r & 7));
}

template <int D>
__global__ void __launch_bounds__(kDecThreads) decode_partial_kernel(const DecodeArgs a)
{
    // Let the combine kernel's CTAs be scheduled as soon as SM resources free up.
    asm volatile("griddepcontrol.launch_dependents;\n" ::);

    constexpr int CPR = D / 8;  // 16-byte chunks per row
    __shared__ __align__(16) uint4 sK[kDecBlock * CPR];
    __shared__ __align__(16) uint4 sV[kDecBlock * CPR];
    __shared__ __align__(16) float sQ[kMaxGroup * D];
    __shared__ __align__(16) float sP[kMaxGroup * kDecBlock];
    __shared__ float sRed[kMaxGroup * 4];
    __shared__ float sM[kMaxGroup], sL[kMaxGroup];

    const int chunk = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = a.G;

    const int64_t len = a.lens[b];
    if (len < 1 || len > a.max_len) return;
    const int64_t p = len - 1, row = p / kDecBlock;
    // Every thread walks the (short) list; the chunk-th entry is this CTA's key block.
    int64_t jblk = -1;
    const int n = for_each_key_block(row, a.W, a.S, [&](int pos, int64_t j) {
        if (pos == chunk) jblk = j;
    });
    if (chunk >= n) return;
    const int n_keys = jblk == row ? (int)(p % kDecBlock) + 1 : kDecBlock;

    // Stage K and V (rows beyond n_keys are not read from memory and are zero-filled).
    const __nv_bfloat16 *kb = a.k + b * a.k_sb + (jblk * kDecBlock) * a.k_ss + hk * a.k_sh;
    const __nv_bfloat16 *vb = a.v + b * a.v_sb + (jblk * kDecBlock) * a.v_ss + hk * a.v_sh;
    for (int idx = tid; idx < kDecBlock * CPR; idx += kDecThreads) {
        const int r = idx / CPR, c = idx % CPR;
        if (r < n_keys)
            cp_async16(&sK[swz<D>(r, c)], kb + r * a.k_ss + c * 8);
        else
            sK[swz<D>(r, c)] = make_uint4(0, 0, 0, 0);
    }
    cp_async_commit();
    for (int idx = tid; idx < kDecBlock * CPR; idx += kDecThreads) {
        const int r = idx / CPR, c = idx % CPR;
        if (r < n_keys)
            cp_async16(&sV[r * CPR + c], vb + r * a.v_ss + c * 8);
        else
            sV[r * CPR + c] = make_uint4(0, 0, 0, 0);
    }
    cp_async_commit();
    // Query rows of the group, widened to fp32.
    const __nv_bfloat16 *qb = a.q + ((int64_t)b * a.Hq + (int64_t)hk * G) * D;
    for (int idx = tid; idx < G * D; idx += kDecThreads) sQ[idx] = __bfloat162float(qb[idx]);
    cp_async_wait<1>();
    __syncthreads();

    // Logits: thread -> (key = tid % 64, half = tid / 64); half 0 takes heads [0, 4), half 1 [4, 8).
    {
        const int key = tid & 63, h0 = (tid >> 6) * 4;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
        for (int c = 0; c < CPR; ++c) {
            const uint4 kk = sK[swz<D>(key, c)];
            const uint32_t w[4] = {kk.x, kk.y, kk.z, kk.w};
            float kf[8];
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                kf[2 * t] = __uint_as_float(w[t] << 16);
                kf[2 * t + 1] = __uint_as_float(w[t] & 0xffff0000u);
            }
#pragma unroll
            for (int hh = 0; hh < 4; ++hh) {
                if (h0 + hh < G) {
                    const float4 q0 = *reinterpret_cast<const float4 *>(&sQ[(h0 + hh) * D + c * 8]);
                    const float4 q1 = *reinterpret_cast<const float4 *>(&sQ[(h0 + hh) * D + c * 8 + 4]);
                    acc[hh] += kf[0] * q0.x + kf[1] * q0.y + kf[2] * q0.z + kf[3] * q0.w +
                               kf[4] * q1.x + kf[5] * q1.y + kf[6] * q1.z + kf[7] * q1.w;
                }
            }
        }
        // Chunk-local softmax per head in the base-2 domain: s2 = s * scale * log2(e).
#pragma unroll
        for (int hh = 0; hh < 4; ++hh) {
            const int h = h0 + hh;
            const float s2 = key < n_keys ? acc[hh] * a.scale_log2 : -INFINITY;
            float mx = s2;
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            if (lane == 0) sRed[h * 4 + (warp & 1)] = mx;
            acc[hh] = s2;
        }
        __syncthreads();
#pragma unroll
        for (int hh = 0; hh < 4; ++hh) {
            const int h = h0 + hh;
            const float m = fmaxf(sRed[h * 4 + 0], sRed[h * 4 + 1]);  // finite: key 0 is valid
            const float pexp = exp2f(acc[hh] - m);                     // 0 for masked keys
            sP[h * kDecBlock + key] = pexp;
            float sum = pexp;
            for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            if (lane == 0) sRed[h * 4 + 2 + (warp & 1)] = sum;
            if (key == 0) sM[h] = m;
        }
    }
    cp_async_wait<0>();
    __syncthreads();
    if (tid < kMaxGroup) sL[tid] = sRed[tid * 4 + 2] + sRed[tid * 4 + 3];

    // Partial output: thread -> feature d (D <= 128 threads), all heads of the group.
    if (tid < D) {
        float o[kMaxGroup];
#pragma unroll
        for (int h = 0; h < kMaxGroup; ++h) o[h] = 0.f;
        const __nv_bfloat16 *vs = reinterpret_cast<const __nv_bfloat16 *>(sV);
#pragma unroll 4
        for (int key = 0; key < kDecBlock; ++key) {
            const float vv = __bfloat162float(vs[key * D + tid]);
#pragma unroll
            for (int h = 0; h < kMaxGroup; ++h)
                if (h < G) o[h] += sP[h * kDecBlock + key] * vv;
        }
#pragma unroll
        for (int h = 0; h < kMaxGroup; ++h)
            if (h < G) {
                float *dst = a.partial + (((int64_t)b * a.Hq + hk * G + h) * a.chunks + chunk) * (D + 2);
                dst[tid] = o[h];
            }
    }
    __syncthreads();
    if (tid < G) {
        float *dst = a.partial + (((int64_t)b * a.Hq + hk * G + tid) * a.chunks + chunk) * (D + 2);
        dst[D] = sM[tid];      // base-2 running max of the chunk
        dst[D + 1] = sL[tid];  // sum of 2^(s2 - m)
    }
}

// Log-sum-exp merge of the chunk partials of one (sequence, query head):
//   m = max m_c,  l = sum l_c 2^(m_c - m),  o = sum o_c 2^(m_c - m) / l,  LSE = (m + log2 l) ln 2.
template <int D>
__global__ void __launch_bounds__(D) decode_combine_kernel(const DecodeArgs a)
{
    const int h = blockIdx.x, b = blockIdx.y, d = threadIdx.x;
    const int64_t len = a.lens[b];
    const bool valid = len >= 1 && len <= a.max_len;
    int n = 0;
    if (valid) n = row_length((len - 1) / kDecBlock, a.W, a.S);
    // The partial kernel's writes are visible only after this wait.
    asm volatile("griddepcontrol.wait;\n" ::: "memory");
    const float *src = a.partial + (((int64_t)b * a.Hq + h) * a.chunks) * (D + 2);
    float m = -INFINITY;
    for (int c = 0; c < n; ++c) m = fmaxf(m, src[c * (D + 2) + D]);
    float l = 0.f, acc = 0.f;
    for (int c = 0; c < n; ++c) {
        const float w = exp2f(src[c * (D + 2) + D] - m);
        l += src[c * (D + 2) + D + 1] * w;
        acc += src[c * (D + 2) + d] * w;
    }
    const float out = n > 0 ? acc / l : 0.f;
    const int64_t oi = ((int64_t)b * a.Hq + h) * D + d;
    if (a.o_is_f32)
        reinterpret_cast<float *>(a.o)[oi] = out;
    else
        reinterpret_cast<__nv_bfloat16 *>(a.o)[oi] = __float2bfloat16_rn(out);
    if (d == 0) a.lse[(int64_t)b * a.Hq + h] = n > 0 ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
}

__global__ void decode_block_list_kernel(int64_t len, int32_t W, int32_t S, int32_t *out,
                                         int32_t *count, int32_t capacity)
{
    const int64_t row = (len - 1) / kDecBlock;
    const int n = for_each_key_block(row, W, S, [=](int pos, int64_t j) {
        if (pos < capacity) out[pos] = (int32_t)j;
    });
    *count = n;
}

// Upper bound on the number of listed blocks of any row below n_rows.
static int max_row_blocks(int64_t n_rows, int32_t W, int32_t S)
{
    int bits = 0;
    for (int64_t x = n_rows > 0 ? n_rows - 1 : 0; x > 0; x >>= 1) ++bits;
    int64_t bound = (int64_t)(W > 1 ? W : 1) + S + bits;
    return (int)(bound < n_rows ? bound : n_rows);
}

static pa_status check_decode(const pa_decode_params *p)
{
    if (!p) return fail(PA_ERR_INVALID_ARG, "params must be non-null");
    if (p->batch < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1 || p->max_len < 1)
        return fail(PA_ERR_INVALID_ARG, "batch, head counts and max_len must be positive");
    if (p->window_blocks < 0 || p->sink_blocks < 0)
        return fail(PA_ERR_INVALID_ARG, "window_blocks and sink_blocks must be >= 0");
    if (p->o_dtype != PA_BF16 && p->o_dtype != PA_F32) return fail(PA_ERR_INVALID_ARG, "bad o_dtype");
    if (p->head_dim != 64 && p->head_dim != 128) return fail(PA_ERR_SHAPE, "head_dim must be 64 or 128");
    if (p->block != kDecBlock) return fail(PA_ERR_SHAPE, "block must be 64");
    if (p->n_q_heads % p->n_kv_heads) return fail(PA_ERR_SHAPE, "n_q_heads must be a multiple of n_kv_heads");
    if (p->n_q_heads / p->n_kv_heads > kMaxGroup)
        return fail(PA_ERR_SHAPE, "at most %d query heads per KV head", kMaxGroup);
    if (p->batch > 65535 || p->n_kv_heads > 65535 || p->n_q_heads > 65535)
        return fail(PA_ERR_SHAPE, "batch and head counts must be <= 65535");
    if (p->window_blocks > 4096 || p->sink_blocks > 4096)
        return fail(PA_ERR_SHAPE, "window_blocks and sink_blocks must be <= 4096");
    const pa_strides *st[2] = {&p->k, &p->v};
    for (auto s : st) {
        if (s->seq < p->head_dim || s->head < p->head_dim || s->batch < 0)
            return fail(PA_ERR_SHAPE, "cache strides must be >= head_dim");
        if ((s->seq % 8) || (s->head % 8) || (s->batch % 8))
            return fail(PA_ERR_ALIGNMENT, "cache strides must be multiples of 8 elements (16 bytes)");
    }
    return PA_OK;
}

}  // namespace pa

extern "C" size_t pa_decode_workspace_bytes(const pa_decode_params *p)
{
    using namespace pa;
    if (check_decode(p) != PA_OK) return 0;
    const int64_t rows = (p->max_len + kDecBlock - 1) / kDecBlock;
    const int chunks = max_row_blocks(rows, p->window_blocks, p->sink_blocks);
    return (size_t)p->batch * p->n_q_heads * chunks * (p->head_dim + 2) * sizeof(float);
}

extern "C" pa_status pa_decode(const pa_decode_params *p, const void *q, const void *k_cache,
                               const void *v_cache, const int32_t *cache_lens, void *o,
                               float *lse, void *workspace, size_t workspace_bytes, void *stream)
{
    using namespace pa;
    clear_error();
    if (pa_status s = check_decode(p)) return s;
    if (!q || !k_cache || !v_cache || !cache_lens || !o || !lse)
        return fail(PA_ERR_INVALID_ARG, "q, k_cache, v_cache, cache_lens, o and lse must be non-null");
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(o))
        return fail(PA_ERR_ALIGNMENT, "q, k_cache, v_cache and o must be 16-byte aligned");
    const size_t need = pa_decode_workspace_bytes(p);
    if (!workspace || workspace_bytes < need)
        return fail(PA_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", need, workspace_bytes);
    if (!aligned16(workspace)) return fail(PA_ERR_ALIGNMENT, "workspace must be 16-byte aligned");
    if (pa_status s = require_sm100()) return s;

    DecodeArgs a;
    a.q = static_cast<const __nv_bfloat16 *>(q);
    a.k = static_cast<const __nv_bfloat16 *>(k_cache);
    a.v = static_cast<const __nv_bfloat16 *>(v_cache);
    a.lens = cache_lens;
    a.partial = static_cast<float *>(workspace);
    a.o = o;
    a.lse = lse;
    a.k_sb = p->k.batch; a.k_ss = p->k.seq; a.k_sh = p->k.head;
    a.v_sb = p->v.batch; a.v_ss = p->v.seq; a.v_sh = p->v.head;
    a.max_len = p->max_len;
    a.batch = p->batch; a.Hq = p->n_q_heads; a.Hkv = p->n_kv_heads;
    a.G = p->n_q_heads / p->n_kv_heads;
    a.W = p->window_blocks; a.S = p->sink_blocks;
    const int64_t rows = (p->max_len + kDecBlock - 1) / kDecBlock;
    a.chunks = max_row_blocks(rows, p->window_blocks, p->sink_blocks);
    a.o_is_f32 = p->o_dtype == PA_F32;
    const float scale = p->softmax_scale != 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->head_dim);
    a.scale_log2 = scale * 1.4426950408889634f;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const dim3 grid1((unsigned)a.chunks, (unsigned)a.Hkv, (unsigned)a.batch);
    if (p->head_dim == 128)
        decode_partial_kernel<128><<<grid1, kDecThreads, 0, st>>>(a);
    else
        decode_partial_kernel<64><<<grid1, kDecThreads, 0, st>>>(a);
    PA_CUDA_OK(cudaGetLastError());

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)a.Hq, (unsigned)a.batch, 1);
    cfg.blockDim = dim3((unsigned)p->head_dim, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (p->head_dim == 128)
        PA_CUDA_OK(cudaLaunchKernelEx(&cfg, decode_combine_kernel<128>, a));
    else
        PA_CUDA_OK(cudaLaunchKernelEx(&cfg, decode_combine_kernel<64>, a));
    return PA_OK;
}

extern "C" pa_status pa_decode_block_list(int64_t cache_len, int32_t block, int32_t window_blocks,
                                          int32_t sink_blocks, int32_t *out_blocks,
                                          int32_t *out_count, int32_t capacity, void *stream)
{
    using namespace pa;
    clear_error();
    if (cache_len < 1) return fail(PA_ERR_INVALID_ARG, "cache_len must be >= 1");
    if (block != kDecBlock) return fail(PA_ERR_SHAPE, "block must be 64");
    if (window_blocks < 0 || sink_blocks < 0 || capacity < 1 || !out_blocks || !out_count)
        return fail(PA_ERR_INVALID_ARG, "bad window/sink/capacity or null output");
    decode_block_list_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(
        cache_len, window_blocks, sink_blocks, out_blocks, out_count, capacity);
    PA_CUDA_OK(cudaGetLastError());
    return PA_OK;
}

// ------------------------------------------------------------------------------------------
// pa_decode_static: the same decode, for callers that cannot allocate device memory.
//
// The split-K partial results go to a fixed array that is part of the library image instead of
// a caller-provided workspace.  The array's name is only a host-side handle in host code; the
// real device address is looked up once per device with cudaGetSymbolAddress (with that device
// current) and then handed to the kernels like any other pointer.
// ------------------------------------------------------------------------------------------
#include <mutex>

namespace pa {

static __device__ __align__(256) unsigned char g_decode_static_scratch[PA_DECODE_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
static std::mutex g_static_mu;
static void *g_static_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device (looked up on first use).
static pa_status static_scratch_address(void **out)
{
    int dev = 0;
    PA_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices)
        return fail(PA_ERR_UNSUPPORTED, "device index %d is beyond the %d devices supported", dev, kMaxDevices);
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
        void *ptr = nullptr;
        PA_CUDA_OK(cudaGetSymbolAddress(&ptr, g_decode_static_scratch));
        if (!ptr) return fail(PA_ERR_CUDA, "cudaGetSymbolAddress returned a null address");
        g_static_ptr[dev] = ptr;
    }
    *out = g_static_ptr[dev];
    return PA_OK;
}

}  // namespace pa

extern "C" pa_status pa_decode_static(const pa_decode_params *p, const void *q, const void *k_cache,
                                      const void *v_cache, const int32_t *cache_lens, void *o,
                                      float *lse, void *stream)
{
    using namespace pa;
    clear_error();
    if (pa_status s = check_decode(p)) return s;
    const size_t need = pa_decode_workspace_bytes(p);
    if (need > (size_t)PA_DECODE_STATIC_SCRATCH_BYTES)
        return fail(PA_ERR_WORKSPACE,
                    "this problem needs %zu bytes of split-K scratch but the built-in array holds %zu; "
                    "use pa_decode with a caller-allocated workspace", need,
                    (size_t)PA_DECODE_STATIC_SCRATCH_BYTES);
    void *scratch = nullptr;
    if (pa_status s = static_scratch_address(&scratch)) return s;
    return pa_decode(p, q, k_cache, v_cache, cache_lens, o, lse, scratch,
                     (size_t)PA_DECODE_STATIC_SCRATCH_BYTES, stream);
}
