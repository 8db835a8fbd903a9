// pa_decode: one query token per sequence against its KV cache under the PowerAttention row of
// its position (Section 4.1: same pattern in prefilling and decoding; Eq. (1) for the row).
//
// Two paths.  Rows with at most 32 window, power-of-two and sink candidates (every PowerAttention
// row with the default window up to millions of tokens) take decode_row_kernel: one launch, a thread-block cluster per
// (sequence, KV head), described at that kernel.  Longer rows take the split-K pair below.
//
// Split-K: one CTA per (sequence, KV head, chunk) where a chunk is one 64-key block of the
// row's block list.  Each CTA reads its K and V block with coalesced 16-byte loads and computes
// the logits of all query heads of the group, a chunk-local softmax and the unnormalised partial
// output on the warp-level tensor-core MMA.  The chunk partials (o[D], m, l) are then merged with
// the log-sum-exp rule by a second kernel, launched with programmatic dependent launch so that
// its start-up overlaps the first kernel's tail; it waits for the partials with griddepcontrol.wait.
#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <math.h>
#include <stdlib.h>

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
    int32_t stages;  // (cluster kernel) shared-memory stages of this launch
    float scale_log2;  // softmax_scale * log2(e)
};

// 16-byte read-only global load.
__device__ __forceinline__ uint4 ldg16(const void *p)
{
    uint4 r;
    asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];\n"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

// D(16x8, fp32) += A(16x16, bf16, row-major) * B(16x8, bf16, column-major), one warp.
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}

// Attention of one 64-key block for all query heads of a KV group.
//
// Logits: each of the four warps takes 16 keys; the query heads of the group are the M rows of
// the 16 x 8 x 16 MMA (rows beyond the group are zero), so one pass over K serves every head.
// K, V and Q are read straight from global memory with 16-byte loads, all issued before the
// first use.  A thread's 16-byte piece holds eight consecutive features of one row; the dot
// product does not care in which order features are paired, so the pieces are fed to the MMA
// fragments as they come (Q and K use the same pairing).  The logits go through shared memory
// once so that every warp sees the whole 64-key row and the block's softmax uses one maximum.
// Output: each warp owns 32 of the features and runs P V over all 64 keys for them (two rows of
// V are interleaved with byte permutes to form the B fragments), so no cross-warp merge is needed.
template <int D>
__global__ void __launch_bounds__(kDecThreads) decode_block_kernel(const DecodeArgs a)
{
    // Let the combine kernel's CTAs be scheduled as soon as SM resources free up.
    asm volatile("griddepcontrol.launch_dependents;\n" ::);
    constexpr int NJ = D / 32;  // 16-byte pieces per thread and row for Q and K
    __shared__ float sS[kMaxGroup][kDecBlock + 8];  // base-2 logits of the block

    const int chunk = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int G = a.G;

    const int64_t len = a.lens[b];
    const bool valid = len >= 1 && len <= a.max_len;
    const int64_t p = len - 1;
    const int32_t row = valid ? (int32_t)(p / kDecBlock) : 0;  // max_len / 64 fits in 31 bits (host check)
    // Every thread walks the (short) list; the chunk-th entry is this CTA's key block.
    int32_t jblk = -1;
    int n = 0;
    if (valid)
        n = for_each_key_block_t<int32_t>(row, a.W, a.S, [&](int pos, int32_t j) {
            if (pos == chunk) jblk = j;
        });
    if (chunk >= n) return;

    {
        const int n_keys = jblk == row ? (int)(p % kDecBlock) + 1 : kDecBlock;
        const int base = wid * 16;            // first key of this warp's logit tile
        const int vchunk = (g & 3) + 4 * wid;  // this thread's 8-feature piece of V rows
        const bool pv_warp = 4 * wid < D / 8;  // warps that own output features

        // ---- loads (keys at or beyond n_keys do not exist: zeros instead of a read)
        const __nv_bfloat16 *kb = a.k + b * a.k_sb + ((int64_t)jblk * kDecBlock) * a.k_ss + hk * a.k_sh;
        const __nv_bfloat16 *vb = a.v + b * a.v_sb + ((int64_t)jblk * kDecBlock) * a.v_ss + hk * a.v_sh;
        const uint4 zero4 = make_uint4(0, 0, 0, 0);
        uint4 kr[2][NJ], vr[4][4], qr[NJ];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            const int key = base + nt * 8 + g;
#pragma unroll
            for (int j = 0; j < NJ; ++j)
                kr[nt][j] = key < n_keys ? ldg16(kb + key * a.k_ss + 8 * (4 * j + t)) : zero4;
        }
        const __nv_bfloat16 *qb = a.q + ((int64_t)b * a.Hq + (int64_t)hk * G + g) * D;
#pragma unroll
        for (int j = 0; j < NJ; ++j) qr[j] = g < G ? ldg16(qb + 8 * (4 * j + t)) : zero4;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
#pragma unroll
            for (int kx = 0; kx < 4; ++kx) {
                const int key = 16 * ks + 2 * t + (kx & 1) + (kx >> 1) * 8;
                vr[ks][kx] = (pv_warp && key < n_keys) ? ldg16(vb + key * a.v_ss + 8 * vchunk) : zero4;
            }

        // ---- S = Q K^T: rows = heads, columns = the warp's 16 keys (two 8-key tiles)
        float sc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
            for (int j = 0; j < NJ; ++j) {
                mma_bf16(sc[nt], qr[j].x, 0u, qr[j].y, 0u, kr[nt][j].x, kr[nt][j].y);
                mma_bf16(sc[nt], qr[j].z, 0u, qr[j].w, 0u, kr[nt][j].z, kr[nt][j].w);
            }
        }
        // This thread holds head g, keys base + 8 nt + 2 t + {0, 1}: to shared memory in the
        // base-2 domain (s * scale * log2(e)); keys that do not exist become -inf.
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            const int key = base + nt * 8 + 2 * t;
            float2 v2;
            v2.x = key < n_keys ? sc[nt][0] * a.scale_log2 : -INFINITY;
            v2.y = key + 1 < n_keys ? sc[nt][1] * a.scale_log2 : -INFINITY;
            *reinterpret_cast<float2 *>(&sS[g][key]) = v2;
        }
        __syncthreads();

        // ---- block softmax: thread (g, t) takes keys 16 ks + {2t, 2t+1, 2t+8, 2t+9}, ks = 0..3
        // (exactly the positions of its P fragments); the four t lanes cover the row.
        float2 sv[4][2];
        float mrow = -INFINITY;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                sv[ks][hh] = *reinterpret_cast<const float2 *>(&sS[g][16 * ks + 8 * hh + 2 * t]);
                mrow = fmaxf(mrow, fmaxf(sv[ks][hh].x, sv[ks][hh].y));
            }
        mrow = fmaxf(mrow, __shfl_xor_sync(0xffffffffu, mrow, 1));
        mrow = fmaxf(mrow, __shfl_xor_sync(0xffffffffu, mrow, 2));  // finite: key 0 of the block exists
        uint32_t pa[4][2];
        float lrow = 0.f;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const float p0 = ex2_approx(sv[ks][hh].x - mrow), p1 = ex2_approx(sv[ks][hh].y - mrow);
                lrow += p0 + p1;
                const __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
                pa[ks][hh] = *reinterpret_cast<const uint32_t *>(&h2);
            }
        lrow += __shfl_xor_sync(0xffffffffu, lrow, 1);
        lrow += __shfl_xor_sync(0xffffffffu, lrow, 2);
        if (wid == 0 && t == 0 && g < G) {
            float *dst = a.partial + (((int64_t)b * a.Hq + hk * G + g) * a.chunks + chunk) * (D + 2);
            dst[D] = mrow;      // base-2 maximum of the block
            dst[D + 1] = lrow;  // sum of 2^(s2 - m)
        }

        // ---- O = P V for this warp's 32 features.  Lanes g and g + 4 read the same 16-byte piece
        // and take its low / high half: feature tile e covers features 8 vchunk(n) + e + 4 (n >> 2)
        // for n = 0..7.
        if (pv_warp) {
            const bool hi = (g >> 2) != 0;
            float acc[4][4];
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[e][0] = acc[e][1] = acc[e][2] = acc[e][3] = 0.f;
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                uint32_t w0[2], w1[2], w2[2], w3[2];  // the two 32-bit words this lane uses, per key
                w0[0] = hi ? vr[ks][0].z : vr[ks][0].x; w0[1] = hi ? vr[ks][0].w : vr[ks][0].y;
                w1[0] = hi ? vr[ks][1].z : vr[ks][1].x; w1[1] = hi ? vr[ks][1].w : vr[ks][1].y;
                w2[0] = hi ? vr[ks][2].z : vr[ks][2].x; w2[1] = hi ? vr[ks][2].w : vr[ks][2].y;
                w3[0] = hi ? vr[ks][3].z : vr[ks][3].x; w3[1] = hi ? vr[ks][3].w : vr[ks][3].y;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t sel = (e & 1) ? 0x7632u : 0x5410u;
                    const uint32_t b0 = __byte_perm(w0[e >> 1], w1[e >> 1], sel);
                    const uint32_t b1 = __byte_perm(w2[e >> 1], w3[e >> 1], sel);
                    mma_bf16(acc[e], pa[ks][0], 0u, pa[ks][1], 0u, b0, b1);
                }
            }
            // acc[e][x]: head g, column n = 2t + x of the tile -> feature below.
            if (g < G) {
                float *dst = a.partial + (((int64_t)b * a.Hq + hk * G + g) * a.chunks + chunk) * (D + 2);
#pragma unroll
                for (int e = 0; e < 4; ++e)
#pragma unroll
                    for (int x = 0; x < 2; ++x) {
                        const int nn = 2 * t + x;
                        dst[8 * ((nn & 3) + 4 * wid) + e + 4 * (nn >> 2)] = acc[e][x];
                    }
            }
        }
    }
}

// Log-sum-exp merge of the chunk partials of one (sequence, query head):
//   m = max m_c,  l = sum l_c 2^(m_c - m),  o = sum o_c 2^(m_c - m) / l,  LSE = (m + log2 l) ln 2.
template <int D>
__global__ void __launch_bounds__(D) decode_combine_kernel(const DecodeArgs a)
{
    __shared__ float s_red[D / 32];
    const int h = blockIdx.x, b = blockIdx.y, d = threadIdx.x;
    const int64_t len = a.lens[b];
    const bool valid = len >= 1 && len <= a.max_len;
    int n = 0;
    if (valid) n = row_length((len - 1) / kDecBlock, a.W, a.S);
    // The partial kernel's writes are visible only after this wait.
    asm volatile("griddepcontrol.wait;\n" ::: "memory");
    const float *src = a.partial + (((int64_t)b * a.Hq + h) * a.chunks) * (D + 2);
    // Global maximum: the chunks are spread over the threads (independent loads), then reduced.
    float m = -INFINITY;
    for (int c = d; c < n; c += D) m = fmaxf(m, src[c * (D + 2) + D]);
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((d & 31) == 0) s_red[d >> 5] = m;
    __syncthreads();
    m = s_red[0];
#pragma unroll
    for (int w = 1; w < D / 32; ++w) m = fmaxf(m, s_red[w]);
    // Weighted sums; the loop is unrolled so that the loads of several chunks are in flight.
    float l = 0.f, acc = 0.f;
#pragma unroll 8
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

// ------------------------------------------------------------------------------------------
// One launch per call: a thread-block cluster per (sequence, KV head).
//
// The row's key blocks are dealt round-robin to the CTAs of the cluster.  A CTA requests its K and
// V blocks with 16-byte asynchronous copies into shared memory and takes them in order as they
// land.  Two forms (kRing): a small call uses the widest cluster, so a CTA has at most four
// blocks, each with its own stage, all requested at once (lowest latency); a large call uses
// few CTAs per row, each walking its blocks through a ring of stages (one by default: six CTAs
// then share an SM, which is what fills the memory pipe).  Per block: logits and P V as in
// decode_block_kernel, with the running maximum, sum and output kept in registers across blocks
// (online softmax).  The CTAs' partial results meet in shared memory:
// after a cluster barrier CTA r merges the heads g = r, r + R, ... reading its peers' partials
// through distributed shared memory, and writes O and the LSE.  No workspace, no second launch.
// ------------------------------------------------------------------------------------------
constexpr int kRowMaxStages = 4;   // shared-memory stages (key blocks in flight) per CTA
constexpr int kRowMaxCluster = 8;  // portable cluster size limit

template <int D>
struct RowSmem {
    static constexpr int kPitch = D * 2 + 16;                  // bytes per key row (padded: no bank conflicts)
    static constexpr int kTile = kDecBlock * kPitch;           // one K or V block
    static constexpr int kBlockBytes = 2 * kTile;              // K + V of one key block
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, uint32_t src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
// Waits until at most `pending` of this thread's copy groups are still in flight.
__device__ __forceinline__ void cp_async_wait(int pending)
{
    switch (pending) {
        case 0: asm volatile("cp.async.wait_group 0;\n" ::: "memory"); break;
        case 1: asm volatile("cp.async.wait_group 1;\n" ::: "memory"); break;
        case 2: asm volatile("cp.async.wait_group 2;\n" ::: "memory"); break;
        default: asm volatile("cp.async.wait_group 3;\n" ::: "memory"); break;
    }
}
__device__ __forceinline__ uint4 lds16(uint32_t addr)
{
    uint4 r;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];\n" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr));
    return r;
}

template <int D, bool kRing>
__global__ void __launch_bounds__(kDecThreads) decode_row_kernel(const DecodeArgs a)
{
    namespace cg = cooperative_groups;
    using SM = RowSmem<D>;
    constexpr int NJ = D / 32;  // 16-byte pieces per thread and row for Q and K
    extern __shared__ __align__(16) uint8_t row_smem[];
    __shared__ float sS[kMaxGroup][kDecBlock + 8];  // base-2 logits of the current block
    __shared__ float sO[kMaxGroup][D];              // this CTA's unnormalised output
    __shared__ float sML[kMaxGroup][2];             // this CTA's running maximum and sum

    cg::cluster_group cluster = cg::this_cluster();
    const int R = (int)gridDim.x, r = (int)blockIdx.x;  // the cluster spans grid x
    const int hk = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int G = a.G;

    const int64_t len = a.lens[b];
    const bool valid = len >= 1 && len <= a.max_len;
    const int64_t p = len - 1;
    const int32_t row = valid ? (int32_t)(p / kDecBlock) : 0;
    // The row's block set, one candidate per lane (the order does not matter for Eq. (1), so the
    // set is not sorted: window distances 0 .. w-1, then the power-of-two distances >= w that do
    // not land on a sink block, then the sink blocks outside the window).  The host takes this
    // path only when window + powers + sinks fit the 32 lanes.
    int32_t cand = -1;
    if (valid) {
        const int32_t w_eff = a.W > 1 ? a.W : 1;
        const int k0 = w_eff <= 1 ? 0 : 32 - __clz(w_eff - 1);  // first k with 2^k >= w_eff
        const int kmax = row >= 1 ? 31 - __clz(row) : -1;       // last k with 2^k <= row
        const int n_pow = kmax >= k0 ? kmax - k0 + 1 : 0;
        if (lane < w_eff) {
            cand = row - lane;  // negative: before the sequence start
        } else if (lane < w_eff + n_pow) {
            const int32_t j = row - (1 << (k0 + lane - w_eff));
            if (j >= a.S) cand = j;
        } else if (lane < w_eff + n_pow + a.S) {
            const int32_t j = lane - w_eff - n_pow;
            if (row - j >= w_eff) cand = j;  // also implies j <= row
        }
    }
    const uint32_t have = __ballot_sync(0xffffffffu, cand >= 0);
    const int n = __popc(have);
    const int mine = n > r ? (n - r + R - 1) / R : 0;
    // Key block number i of this CTA: the (r + i R)-th candidate that exists.  Without the ring a
    // CTA has at most kRowMaxStages blocks and keeps their indices in registers.
    int32_t jb[kRowMaxStages];
    if constexpr (!kRing) {
#pragma unroll
        for (int i = 0; i < kRowMaxStages; ++i) {
            const int src = i < mine ? (int)__fns(have, 0, r + i * R + 1) : 0;
            jb[i] = __shfl_sync(0xffffffffu, cand, src & 31);
        }
    }
    auto block_of = [&](int i) -> int32_t {
        if constexpr (!kRing) {
            return i == 0 ? jb[0] : i == 1 ? jb[1] : i == 2 ? jb[2] : jb[3];
        } else {
            const int src = (int)__fns(have, 0, r + i * R + 1);
            return __shfl_sync(0xffffffffu, cand, src & 31);
        }
    };

    // ---- loads: one copy group per key block; a thread copies one 16-byte piece of every eighth
    // key row (rows past the sequence end are zero-filled).  Without the ring every block has its
    // own stage and all are requested here; with it, `stages` blocks are in flight at a time.
    const uint32_t smem0 = (uint32_t)__cvta_generic_to_shared(row_smem);
    const int stages = kRing ? a.stages : kRowMaxStages;
    auto issue_block = [&](int i) {
        constexpr int NP = D / 8;                       // 16-byte pieces per row
        constexpr int kRowsPerPass = kDecThreads / NP;  // key rows covered by one pass of the CTA
        const int key0 = tid / NP, pc = tid % NP;
        const int32_t j = block_of(i);
        const int n_keys = j == row ? (int)(p % kDecBlock) + 1 : kDecBlock;
        const __nv_bfloat16 *kb = a.k + b * a.k_sb + ((int64_t)j * kDecBlock + key0) * a.k_ss + hk * a.k_sh + 8 * pc;
        const __nv_bfloat16 *vb = a.v + b * a.v_sb + ((int64_t)j * kDecBlock + key0) * a.v_ss + hk * a.v_sh + 8 * pc;
        const uint32_t sk = smem0 + (i % stages) * SM::kBlockBytes + key0 * SM::kPitch + pc * 16, sv = sk + SM::kTile;
#pragma unroll
        for (int q = 0; q < kDecBlock / kRowsPerPass; ++q) {
            const uint32_t bytes = key0 + q * kRowsPerPass < n_keys ? 16u : 0u;
            cp_async16(sk + q * kRowsPerPass * SM::kPitch, kb + (int64_t)q * kRowsPerPass * a.k_ss, bytes);
            cp_async16(sv + q * kRowsPerPass * SM::kPitch, vb + (int64_t)q * kRowsPerPass * a.v_ss, bytes);
        }
        cp_async_commit();
    };
    int issued = 0;
    if constexpr (!kRing) {
#pragma unroll
        for (int i = 0; i < kRowMaxStages; ++i)
            if (i < mine) issue_block(i);
        issued = mine;
    } else {
        for (; issued < mine && issued < stages; ++issued) issue_block(issued);
    }

    uint4 qr[NJ];
    {
        const __nv_bfloat16 *qb = a.q + ((int64_t)b * a.Hq + (int64_t)hk * G + g) * D;
        const uint4 zero4 = make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int j = 0; j < NJ; ++j) qr[j] = g < G ? ldg16(qb + 8 * (4 * j + t)) : zero4;
    }

    const int base = wid * 16;             // first key of this warp's logit tile
    const int vchunk = (g & 3) + 4 * wid;  // this thread's 8-feature piece of V rows
    const bool pv_warp = 4 * wid < D / 8;  // warps that own output features
    const bool hi = (g >> 2) != 0;
    float m_run = -INFINITY, l_run = 0.f;
    float acc[4][4];
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[e][0] = acc[e][1] = acc[e][2] = acc[e][3] = 0.f;

#pragma unroll 1
    for (int i = 0; i < mine; ++i) {
        const int32_t jblk = block_of(i);
        const int n_keys = jblk == row ? (int)(p % kDecBlock) + 1 : kDecBlock;
        const uint32_t sk = smem0 + (i % stages) * SM::kBlockBytes, sv_ = sk + SM::kTile;
        if constexpr (kRing) {
            if (i >= 1) {
                __syncthreads();  // every warp has finished block i - 1: its stage is free
                if (issued < mine) {
                    issue_block(issued);  // block i - 1 + stages (block i itself when there is one stage)
                    ++issued;
                }
            }
        }
        cp_async_wait(issued - 1 - i);
        __syncthreads();  // every thread's copies of this block have landed; sS is free again

        // ---- S = Q K^T: rows = heads, columns = the warp's 16 keys (two 8-key tiles)
        float sc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            const int key = base + nt * 8 + g;
#pragma unroll
            for (int j = 0; j < NJ; ++j) {
                const uint4 kr = lds16(sk + key * SM::kPitch + 16 * (4 * j + t));
                mma_bf16(sc[nt], qr[j].x, 0u, qr[j].y, 0u, kr.x, kr.y);
                mma_bf16(sc[nt], qr[j].z, 0u, qr[j].w, 0u, kr.z, kr.w);
            }
        }
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            const int key = base + nt * 8 + 2 * t;
            float2 v2;
            v2.x = key < n_keys ? sc[nt][0] * a.scale_log2 : -INFINITY;
            v2.y = key + 1 < n_keys ? sc[nt][1] * a.scale_log2 : -INFINITY;
            *reinterpret_cast<float2 *>(&sS[g][key]) = v2;
        }
        __syncthreads();

        // ---- online softmax over the block: thread (g, t) takes keys 16 ks + {2t, 2t+1, 2t+8, 2t+9}
        float2 sv[4][2];
        float mrow = -INFINITY;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                sv[ks][hh] = *reinterpret_cast<const float2 *>(&sS[g][16 * ks + 8 * hh + 2 * t]);
                mrow = fmaxf(mrow, fmaxf(sv[ks][hh].x, sv[ks][hh].y));
            }
        mrow = fmaxf(mrow, __shfl_xor_sync(0xffffffffu, mrow, 1));
        mrow = fmaxf(mrow, __shfl_xor_sync(0xffffffffu, mrow, 2));  // finite: key 0 of the block exists
        const float m_new = fmaxf(m_run, mrow);
        const float alpha = ex2_approx(m_run - m_new);  // 0 on the first block
        uint32_t pa[4][2];
        float lrow = 0.f;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const float p0 = ex2_approx(sv[ks][hh].x - m_new), p1 = ex2_approx(sv[ks][hh].y - m_new);
                lrow += p0 + p1;
                const __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
                pa[ks][hh] = *reinterpret_cast<const uint32_t *>(&h2);
            }
        lrow += __shfl_xor_sync(0xffffffffu, lrow, 1);
        lrow += __shfl_xor_sync(0xffffffffu, lrow, 2);
        l_run = l_run * alpha + lrow;
        m_run = m_new;

        // ---- O = alpha O + P V for this warp's 32 features (see decode_block_kernel)
        if (pv_warp) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                acc[e][0] *= alpha;
                acc[e][1] *= alpha;
            }
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                uint4 vr[4];
#pragma unroll
                for (int kx = 0; kx < 4; ++kx) {
                    const int key = 16 * ks + 2 * t + (kx & 1) + (kx >> 1) * 8;
                    vr[kx] = lds16(sv_ + key * SM::kPitch + 16 * vchunk);
                }
                uint32_t w0[2], w1[2], w2[2], w3[2];
                w0[0] = hi ? vr[0].z : vr[0].x; w0[1] = hi ? vr[0].w : vr[0].y;
                w1[0] = hi ? vr[1].z : vr[1].x; w1[1] = hi ? vr[1].w : vr[1].y;
                w2[0] = hi ? vr[2].z : vr[2].x; w2[1] = hi ? vr[2].w : vr[2].y;
                w3[0] = hi ? vr[3].z : vr[3].x; w3[1] = hi ? vr[3].w : vr[3].y;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t sel = (e & 1) ? 0x7632u : 0x5410u;
                    const uint32_t b0 = __byte_perm(w0[e >> 1], w1[e >> 1], sel);
                    const uint32_t b1 = __byte_perm(w2[e >> 1], w3[e >> 1], sel);
                    mma_bf16(acc[e], pa[ks][0], 0u, pa[ks][1], 0u, b0, b1);
                }
            }
        }
    }

    // ---- this CTA's partial result to shared memory
    if (pv_warp && g < G) {
#pragma unroll
        for (int e = 0; e < 4; ++e)
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                const int nn = 2 * t + x;
                sO[g][8 * ((nn & 3) + 4 * wid) + e + 4 * (nn >> 2)] = acc[e][x];
            }
    }
    if (wid == 0 && t == 0 && g < G) {
        sML[g][0] = m_run;
        sML[g][1] = l_run;
    }
    cluster.sync();

    // ---- merge across the cluster: CTA r takes heads r, r + R, ...; thread d one feature.  All
    // remote reads of a head are issued before the first one is used (they are independent, and
    // each costs a trip through the cluster's shared-memory network).
    if (tid < D) {
        const float *peer_ml[kRowMaxCluster];
        const float *peer_o[kRowMaxCluster];
#pragma unroll
        for (int rr = 0; rr < kRowMaxCluster; ++rr) {
            const int src = rr < R ? rr : r;  // (slots beyond the cluster are given weight 0 below)
            peer_ml[rr] = cluster.map_shared_rank(&sML[0][0], src);
            peer_o[rr] = cluster.map_shared_rank(&sO[0][0], src);
        }
        for (int h = r; h < G; h += R) {
            float mr[kRowMaxCluster], lr[kRowMaxCluster], orr[kRowMaxCluster];
#pragma unroll
            for (int rr = 0; rr < kRowMaxCluster; ++rr) {
                mr[rr] = peer_ml[rr][2 * h];
                lr[rr] = peer_ml[rr][2 * h + 1];
                orr[rr] = peer_o[rr][h * D + tid];
            }
            float m = -INFINITY;
#pragma unroll
            for (int rr = 0; rr < kRowMaxCluster; ++rr)
                if (rr < R) m = fmaxf(m, mr[rr]);
            float l = 0.f, o = 0.f;
#pragma unroll
            for (int rr = 0; rr < kRowMaxCluster; ++rr) {
                const float wgt = (rr < R && mr[rr] != -INFINITY) ? exp2f(mr[rr] - m) : 0.f;
                l += lr[rr] * wgt;
                o += orr[rr] * wgt;
            }
            const float out = n > 0 ? o / l : 0.f;
            const int64_t oi = ((int64_t)b * a.Hq + (int64_t)hk * G + h) * D + tid;
            if (a.o_is_f32)
                reinterpret_cast<float *>(a.o)[oi] = out;
            else
                reinterpret_cast<__nv_bfloat16 *>(a.o)[oi] = __float2bfloat16_rn(out);
            if (tid == 0)
                a.lse[(int64_t)b * a.Hq + (int64_t)hk * G + h] = n > 0 ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
        }
    }
    cluster.sync();  // peers may still be reading this CTA's shared memory
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

// Window distances + power-of-two distances beyond the window + sink blocks that a row below
// n_rows can have, before any of them coincide or fall off the sequence start: the number of
// candidate slots the cluster kernel enumerates (one per lane, so it needs this to be <= 32).
static int64_t row_candidate_slots(int64_t n_rows, int32_t W, int32_t S)
{
    const int64_t w = W > 1 ? W : 1;
    int powers = 0;
    for (int64_t pw = 1; pw <= n_rows - 1; pw *= 2)
        if (pw >= w) ++powers;
    return w + S + powers;
}

// Upper bound on the number of listed blocks of any row below n_rows.
static int max_row_blocks(int64_t n_rows, int32_t W, int32_t S)
{
    // window distances 0 .. w-1, every power of two 2^k >= w with 2^k <= n_rows - 1, sink blocks
    const int64_t w = W > 1 ? W : 1;
    int powers = 0;
    for (int64_t pw = 1; pw <= n_rows - 1; pw *= 2)
        if (pw >= w) ++powers;
    const int64_t bound = w + S + powers;
    return (int)(bound < n_rows ? bound : n_rows);
}

// PA_DECODE_PATH=splitk forces the two-launch split-K path (tests use it to cover that path on
// workloads the cluster path would take); PA_DECODE_CLUSTER=n sets the cluster size (1..8)
// instead of the choice by batch size.
static int decode_path()
{
    const char *e = getenv("PA_DECODE_PATH");
    return e && e[0] == 's' ? 1 : 0;
}
static int decode_cluster()  // 0: chosen from the batch size
{
    const char *e = getenv("PA_DECODE_CLUSTER");
    const int v = e ? atoi(e) : 0;
    return v >= 1 && v <= kRowMaxCluster ? v : 0;
}
// PA_DECODE_STAGES=n (1..4): shared-memory stages per CTA of the cluster kernel.
static int decode_stages()  // 0: chosen from the cluster size
{
    const char *e = getenv("PA_DECODE_STAGES");
    const int v = e ? atoi(e) : 0;
    return v >= 1 && v <= kRowMaxStages ? v : 0;
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
    if (p->max_len > ((int64_t)1 << 36)) return fail(PA_ERR_SHAPE, "max_len too large");
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
    a.stages = 0;
    const float scale = p->softmax_scale != 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->head_dim);
    a.scale_log2 = scale * 1.4426950408889634f;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // Rows short enough for one cluster per (sequence, KV head) take the single-launch path.
    if (decode_path() != 1 && row_candidate_slots(rows, p->window_blocks, p->sink_blocks) <= 32) {
        // Cluster size: enough CTAs to fill the GPU about three times over at small batches (the call
        // is latency-bound there and short CTAs help), one CTA per row at large ones (no merge).
        int dev = 0, sms = 0;
        PA_CUDA_OK(cudaGetDevice(&dev));
        PA_CUDA_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        const int64_t rows_in_call = (int64_t)a.batch * a.Hkv;
        int R = decode_cluster();
        if (R == 0) {
            R = (int)((3 * (int64_t)sms + rows_in_call - 1) / rows_in_call);
            if (R > kRowMaxCluster) R = kRowMaxCluster;
            if (R < 1) R = 1;
        }
        const bool widest = R == kRowMaxCluster;  // a small call: as many CTAs per row as a cluster allows
        if (R > a.chunks) R = a.chunks;
        const int per_cta = (a.chunks + R - 1) / R;
        // Few blocks per CTA: every block gets its own stage and all copies start at once (best for
        // the latency of a small call).  Many: one stage per CTA by default, so that six CTAs share
        // an SM and keep its memory pipe full (best for throughput; measured).
        const bool ring = decode_stages() != 0 || per_cta > kRowMaxStages || !widest;
        a.stages = ring ? (decode_stages() != 0 ? decode_stages() : 1) : per_cta;
        if (a.stages > per_cta) a.stages = per_cta;
        const int smem_stages = a.stages;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)R, (unsigned)a.Hkv, (unsigned)a.batch);
        cfg.blockDim = dim3(kDecThreads, 1, 1);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)R;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        // (setting the limit is idempotent: a race between threads only repeats the call)
        static bool sized = false;
        if (!sized) {
            PA_CUDA_OK(cudaFuncSetAttribute(decode_row_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            kRowMaxStages * RowSmem<128>::kBlockBytes));
            PA_CUDA_OK(cudaFuncSetAttribute(decode_row_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            kRowMaxStages * RowSmem<128>::kBlockBytes));
            PA_CUDA_OK(cudaFuncSetAttribute(decode_row_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            kRowMaxStages * RowSmem<64>::kBlockBytes));
            PA_CUDA_OK(cudaFuncSetAttribute(decode_row_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            kRowMaxStages * RowSmem<64>::kBlockBytes));
            sized = true;
        }
        cfg.dynamicSmemBytes = (size_t)smem_stages * (p->head_dim == 128 ? RowSmem<128>::kBlockBytes : RowSmem<64>::kBlockBytes);
        if (p->head_dim == 128) {
            if (ring) PA_CUDA_OK(cudaLaunchKernelEx(&cfg, decode_row_kernel<128, true>, a));
            else PA_CUDA_OK(cudaLaunchKernelEx(&cfg, decode_row_kernel<128, false>, a));
        } else {
            if (ring) PA_CUDA_OK(cudaLaunchKernelEx(&cfg, decode_row_kernel<64, true>, a));
            else PA_CUDA_OK(cudaLaunchKernelEx(&cfg, decode_row_kernel<64, false>, a));
        }
        return PA_OK;
    }
    const dim3 grid1((unsigned)a.chunks, (unsigned)a.Hkv, (unsigned)a.batch);
    if (p->head_dim == 128)
        decode_block_kernel<128><<<grid1, kDecThreads, 0, st>>>(a);
    else
        decode_block_kernel<64><<<grid1, kDecThreads, 0, st>>>(a);
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
