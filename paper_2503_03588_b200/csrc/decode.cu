// pa_decode / pa_decode_paged: one query token per sequence against its KV cache under the
// PowerAttention row of its position (Section 4.1: same pattern in prefilling and decoding;
// Eq. (1) for the row).  The cache is either one contiguous [batch, max_len, Hkv, D] array or a
// pool of 64-token pages reached through a block table.
//
// Two paths.  Rows with at most 32 window, power-of-two and sink candidates (every PowerAttention
// row with the default window up to millions of tokens) take decode_row_kernel: one launch, a
// thread-block cluster per (sequence, KV head), described at that kernel.  Longer rows take the
// split-K pair below.
//
// Split-K: one CTA per (sequence, KV head, chunk) where a chunk is one 64-key block of the
// row's block list.  Each CTA reads its K and V block with coalesced 16-byte loads and computes
// the logits of all query heads of the group, a chunk-local softmax and the unnormalised partial
// output on the warp-level tensor-core MMA.  The chunk partials (o[D], m, l) are then merged with
// the log-sum-exp rule by a second kernel, launched with programmatic dependent launch so that
// its start-up overlaps the first kernel's tail; it waits for the partials with griddepcontrol.wait.
#include <cooperative_groups.h>
#include <cuda.h>
#include <cuda_bf16.h>
#include <math.h>
#include <stdlib.h>

#include <mutex>

#include "common.cuh"
#include "layout_rule.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace pa {

constexpr int kDecBlock = 64;     // keys per block (the only supported block size)
constexpr int kDecThreads = 128;  // threads per CTA of the partial kernel
constexpr int kMaxGroup = 8;      // query heads per KV head supported by the decode kernels
constexpr size_t kDecStatusBytes = 256;  // status block at the start of the workspace

struct DecodeArgs {
    const __nv_bfloat16 *q, *k, *v;
    const int32_t *lens;
    const int32_t *table;  // paged cache: [batch, table_stride] page numbers; null: contiguous cache
    float *partial;        // [batch, Hq, chunks, D + 2]
    int32_t *status;       // [0] error code, [1] detail
    void *o;
    float *lse;
    // Element strides.  Contiguous cache: batch, token, head.  Paged: page, token in page, head.
    int64_t k_sb, k_ss, k_sh, v_sb, v_ss, v_sh;
    int64_t max_len;
    int32_t batch, Hq, Hkv, G, W, S, chunks, o_is_f32;
    int32_t stages;        // (row kernel) shared-memory stages of this launch
    int32_t R, mode;       // (row kernel) chunks per row; what becomes of an item's result
    int32_t fixed_chunks;  // (combine kernel) > 0: every row has this many partials
    int64_t items;         // (row kernel) rows of the call x R
    int32_t table_stride, n_pages;
    float scale_log2;  // softmax_scale * log2(e)
    long long wait_cycles;  // (row kernel) limit of every barrier wait, in clock cycles
};

// Where key block j of sequence b starts: (index along the batch / page axis, first token).  A
// page number outside the pool is clamped (the result is then undefined but nothing faults).
__device__ __forceinline__ void block_origin(const DecodeArgs &a, int b, int32_t j, int64_t &outer, int64_t &tok0)
{
    if (a.table) {
        int32_t page = a.table[(int64_t)b * a.table_stride + j];
        page = page < 0 ? 0 : (page >= a.n_pages ? a.n_pages - 1 : page);
        outer = page;
        tok0 = 0;
    } else {
        outer = b;
        tok0 = (int64_t)j * kDecBlock;
    }
}

// 16-byte read-only global load.
__device__ __forceinline__ uint4 ldg16(const void *p)
{
    uint4 r;
    asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];\n"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}
__device__ __forceinline__ uint32_t ldg4(const void *p)
{
    uint32_t r;
    asm volatile("ld.global.nc.u32 %0, [%1];\n" : "=r"(r) : "l"(p));
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
    if (chunk == 0 && hk == 0 && b == 0 && tid == 0) a.status[0] = 0;  // no bounded waits on this path

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
        int64_t outer, tok0;
        block_origin(a, b, jblk, outer, tok0);
        const __nv_bfloat16 *kb = a.k + outer * a.k_sb + tok0 * a.k_ss + hk * a.k_sh;
        const __nv_bfloat16 *vb = a.v + outer * a.v_sb + tok0 * a.v_ss + hk * a.v_sh;
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
                const float p0 = ptx::ex2(sv[ks][hh].x - mrow), p1 = ptx::ex2(sv[ks][hh].y - mrow);
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
    if (valid) n = a.fixed_chunks > 0 ? a.fixed_chunks : row_length((len - 1) / kDecBlock, a.W, a.S);
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
// The row kernel: attention of (sequence, KV head) rows whose block set fits one warp's lanes.
//
// A row's key blocks are dealt round-robin to R chunks; a work item is one chunk of one row.
// Inside a CTA:
//   warp 4      producer: one elected lane walks the items' blocks and fetches each K block and
//               each V block with TMA box loads (64 keys x 64 features, 128-byte swizzle) into a
//               ring of shared-memory stages; K and V complete on separate mbarriers, so the
//               logits start as soon as K has landed.  The ring runs on across items: while the
//               consumers finish one item the next one's blocks are already on their way.
//   warps 0-3   consumers: warp w owns keys 16 w .. 16 w + 15 of every block.  Logits on the
//               warp-level MMA with the group's query heads as the M rows (K fragments by
//               ldmatrix), online softmax in registers (running maximum, sum and output kept across
//               blocks), O += P V for all D features (V fragments by transposing ldmatrix).  No
//               block-wide barrier inside the loop: a warp only waits for a stage to fill and
//               says when it has finished with it.  At the end of an item the four warps merge
//               their partial results through shared memory with the log-sum-exp rule, each
//               warp a quarter of the features.
// What happens to an item's result depends on the launch (DecodeArgs::mode):
//   kModeCluster  small calls.  One item per CTA, the R CTAs of a row form a thread-block
//                 cluster: each CTA stores its part of head h into the shared memory of CTA h % R
//                 (distributed shared memory), and after one cluster barrier that CTA merges the
//                 head and writes O and LSE.  One launch.
//   kModePartial  larger calls.  A persistent grid of two CTAs per SM strides over the items;
//                 each item's (o, m, l) goes to the workspace and decode_combine_kernel merges a
//                 row's R chunks (second launch, programmatic dependent launch).
//   kModeDirect   R = 1 in a persistent grid: O and LSE are written straight from the registers.
// Every mbarrier wait is bounded; one that runs out records PA_ERR_TIMEOUT in the status block
// and the CTA runs to its end without hanging.
// ------------------------------------------------------------------------------------------
constexpr int kRowConsumers = 4;                     // consumer warps
constexpr int kRowThreads = 32 * (kRowConsumers + 1);
constexpr int kRowMaxStages = 6;                     // shared-memory stages (key blocks in flight) per CTA
constexpr int kRowMaxCluster = 8;                    // portable cluster size limit
constexpr int kRowMaxSmem = 227 * 1024;              // dynamic shared memory a CTA may ask for
constexpr long long kRowWaitCycles = 2000000000ll;   // default limit of a barrier wait: ~1 s
enum : int32_t { kModeCluster = 0, kModePartial = 1, kModeDirect = 2 };

template <int D>
struct RowSmem {
    static constexpr uint32_t kSub = kDecBlock * 128;        // 64 keys x 64 features
    static constexpr uint32_t kTile = kSub * (D / 64);       // one K or V block
    static constexpr uint32_t kStage = 2 * kTile;            // K + V of one key block
    // Hand-over area of the end-of-item merge: per warp and head, the tiles the warp does not own
    // (three quarters of the D features) and its running maximum and sum.
    static constexpr uint32_t kPartRow = D - D / 4 + 2;
    static constexpr uint32_t kPart = kRowConsumers * kMaxGroup * kPartRow * 4;
    // (cluster form) what the row's CTAs send to the CTA that merges a head: per sending CTA and head
    // slot, o[D], m, l.  R senders x ceil(8 / R) heads of an owner is at most 14 entries (R = 7).
    static constexpr uint32_t kRecvEntries = 14;
    static constexpr uint32_t kRecv = kRecvEntries * (D + 2) * 4;
    static constexpr uint32_t kBars = 3 * kRowMaxStages * 8 + 16;
    static constexpr size_t bytes(int stages, bool cluster)
    {
        return 1024 + (size_t)stages * kStage + kPart + kBars + (cluster ? kRecv : 0);
    }
};

// The row's block set, one candidate per lane (the order does not matter for Eq. (1), so the set
// is not sorted): window distances 0 .. w-1, then the power-of-two distances >= w that do not
// land on a sink block, then the sink blocks outside the window.  Returns this lane's key block
// or -1.  The host takes the row kernel only when window + powers + sinks fit the 32 lanes.
__device__ __forceinline__ int32_t row_block_candidate(int32_t row, int32_t W, int32_t S, int lane)
{
    const int32_t w_eff = W > 1 ? W : 1;
    const int k0 = w_eff <= 1 ? 0 : 32 - __clz(w_eff - 1);  // first k with 2^k >= w_eff
    const int kmax = row >= 1 ? 31 - __clz(row) : -1;       // last k with 2^k <= row
    const int n_pow = kmax >= k0 ? kmax - k0 + 1 : 0;
    int32_t cand = -1;
    if (lane < w_eff) {
        cand = row - lane;  // negative: before the sequence start
    } else if (lane < w_eff + n_pow) {
        const int32_t j = row - (1 << (k0 + lane - w_eff));
        if (j >= S) cand = j;
    } else if (lane < w_eff + n_pow + S) {
        const int32_t j = lane - w_eff - n_pow;
        if (row - j >= w_eff) cand = j;  // also implies j <= row
    }
    return cand;
}

template <int D>
__global__ void __launch_bounds__(kRowThreads, 2) decode_row_kernel(const __grid_constant__ CUtensorMap tmK,
                                                                    const __grid_constant__ CUtensorMap tmV,
                                                                    const DecodeArgs a)
{
    namespace cg = cooperative_groups;
    using SM = RowSmem<D>;
    constexpr int DH = D / 64;  // 64-feature (128-byte) sub-tiles per key row
    extern __shared__ uint8_t row_smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(row_smem_raw) + 1023u) & ~1023u;
    uint8_t *smem = row_smem_raw + (smem_base - ptx::smem_u32(row_smem_raw));
    const int stages = a.stages;
    const uint32_t off_part = (uint32_t)stages * SM::kStage;
    float *part = reinterpret_cast<float *>(smem + off_part);  // [warp][head][kPartRow]
    // (cluster form) receive area behind the barriers: [sender][head slot][D + 2]
    float *recv = reinterpret_cast<float *>(smem + off_part + SM::kPart + SM::kBars);
    const uint32_t bars = smem_base + off_part + SM::kPart;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + off_part + SM::kPart + 3 * kRowMaxStages * 8);
    auto bar_kfull = [&](int s) { return bars + (uint32_t)s * 8u; };
    auto bar_vfull = [&](int s) { return bars + (uint32_t)(kRowMaxStages + s) * 8u; };
    auto bar_empty = [&](int s) { return bars + (uint32_t)(2 * kRowMaxStages + s) * 8u; };

    const int R = a.R;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int G = a.G;

    // (item and row counts fit 31 bits; checked on the host)
    const uint32_t n_items = (uint32_t)a.items;
    const uint32_t it0 = blockIdx.x, it_step = gridDim.x;
    // The first item's cache length is on the critical path of a small call: its load starts before
    // the barrier set-up.
    const int32_t len_first = it0 < n_items ? a.lens[(it0 / (uint32_t)R) / (uint32_t)a.Hkv] : 0;
    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            ptx::mbar_init(bar_kfull(s), 1);
            ptx::mbar_init(bar_vfull(s), 1);
            ptx::mbar_init(bar_empty(s), kRowConsumers);
        }
        *abort_flag = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async_smem();
        if (blockIdx.x == 0) a.status[0] = 0;  // a wait that gives up (much later) sets it
    }
    __syncthreads();
    // The combine kernel (kModePartial) may be scheduled as this grid's CTAs retire.
    asm volatile("griddepcontrol.launch_dependents;\n" ::);

    // Item it -> (row of the call, chunk); a row -> (sequence, KV head).
    struct Item {
        int32_t b, hk, r;        // sequence, KV head, chunk
        int32_t row, last_keys;  // the query's block row; keys of the diagonal block
        int32_t cand;            // this lane's candidate key block or -1
        int32_t rank;            // its number among the candidates that exist (lane order)
        int32_t page;            // (paged cache) its page
        uint32_t have;           // lanes whose candidate exists
        int32_t n, mine;         // blocks of the row, blocks of this chunk
    };
    auto item_len = [&](uint32_t it) -> int32_t {  // the sequence's cache length (issued early: a global load)
        return it < n_items ? a.lens[(it / (uint32_t)R) / (uint32_t)a.Hkv] : 0;
    };
    auto make_item = [&](uint32_t it, int32_t len32) {
        Item w;
        const int32_t rowid = (int32_t)(it / (uint32_t)R);
        w.r = (int32_t)(it - (uint32_t)rowid * (uint32_t)R);
        w.b = (int32_t)((uint32_t)rowid / (uint32_t)a.Hkv);
        w.hk = rowid - w.b * a.Hkv;
        const int64_t len = len32;
        const bool valid = len >= 1 && len <= a.max_len;
        const int64_t p = len - 1;
        w.row = valid ? (int32_t)(p / kDecBlock) : 0;
        w.last_keys = (int32_t)(p % kDecBlock) + 1;
        w.cand = valid ? row_block_candidate(w.row, a.W, a.S, lane) : -1;
        w.page = 0;
        if (a.table && w.cand >= 0) w.page = a.table[(int64_t)w.b * a.table_stride + w.cand];
        w.have = __ballot_sync(0xffffffffu, w.cand >= 0);
        w.rank = __popc(w.have & ((1u << lane) - 1u));
        w.n = __popc(w.have);
        w.mine = w.n > w.r ? (w.n - w.r + R - 1) / R : 0;
        return w;
    };
    // Key block number i of the item: the (r + i R)-th candidate that exists (lane that holds it).
    auto lane_of = [&](const Item &w, int i) {
        const uint32_t hit = __ballot_sync(0xffffffffu, w.cand >= 0 && w.rank == w.r + i * R);
        return (__ffs(hit) - 1) & 31;
    };

    if (wid == kRowConsumers) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            ptx::prefetch_tensormap(&tmK);
            ptx::prefetch_tensormap(&tmV);
        }
        bool ok = true;
        uint32_t ci = 0;  // blocks issued so far by this CTA (ring position)
        int32_t len_next = len_first;
        for (uint32_t it = it0; it < n_items; it += it_step) {
            const Item w = make_item(it, len_next);
            len_next = item_len(it + it_step);
            for (int i = 0; i < w.mine; ++i, ++ci) {
                const int src = lane_of(w, i);
                const int32_t j = __shfl_sync(0xffffffffu, w.cand, src);
                const int32_t page = __shfl_sync(0xffffffffu, w.page, src);
                if (lane == 0 && ok) {
                    const int s = (int)(ci % (uint32_t)stages);
                    if (ci >= (uint32_t)stages)
                        ok = ptx::mbar_wait_bounded(bar_empty(s), (ci / (uint32_t)stages - 1) & 1, abort_flag, a.status, 1,
                                                    a.wait_cycles, (int)PA_ERR_TIMEOUT);
                    if (ok) {
                        // (a page outside the pool reads as zeros)
                        const int32_t outer = a.table ? page : w.b, tok0 = a.table ? 0 : j * kDecBlock;
                        const uint32_t dst = smem_base + (uint32_t)s * SM::kStage;
                        ptx::mbar_expect_tx(bar_kfull(s), SM::kTile);
#pragma unroll
                        for (int dh = 0; dh < DH; ++dh)
                            ptx::tma_load_4d(dst + dh * SM::kSub, &tmK, bar_kfull(s), dh * 64, tok0, w.hk, outer);
                        ptx::mbar_expect_tx(bar_vfull(s), SM::kTile);
#pragma unroll
                        for (int dh = 0; dh < DH; ++dh)
                            ptx::tma_load_4d(dst + SM::kTile + dh * SM::kSub, &tmV, bar_vfull(s), dh * 64, tok0, w.hk, outer);
                    }
                }
                __syncwarp();
            }
        }
    } else {
        // ------------------------------------------------------------------ consumers
        // ldmatrix row addresses inside a tile.  K (matrices: keys 0-7 / 8-15 of the warp x two
        // 16-byte feature chunks): lane -> key 16 w + 8 (lane / 16) + lane % 8, chunk + (lane / 8) % 2.
        // V (transposed; matrices: two key halves x two feature chunks): key 16 w + 8 ((lane / 8) % 2)
        // + lane % 8, chunk + lane / 16.  A 16-byte chunk c of row `key` sits at c ^ (key % 8).
        const int k_key = 16 * wid + ((lane >> 4) << 3) + (lane & 7), k_ch = (lane >> 3) & 1;
        const int v_key = 16 * wid + (((lane >> 3) & 1) << 3) + (lane & 7), v_ch = lane >> 4;
        // Q fragments: head g is row g of the 16-row A operand (rows 8..15 are zero).  The next
        // item's are requested while the current item is worked on.
        uint32_t qn[D / 16][2];
        auto load_q = [&](uint32_t it) {
            const bool in = it < n_items && g < G;
            const int32_t rowid = in ? (int32_t)(it / (uint32_t)R) : 0;  // = b Hkv + hk, and its heads start at rowid G
            const __nv_bfloat16 *qb = a.q + ((int64_t)rowid * G + g) * D;
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                qn[ks][0] = in ? ldg4(qb + 16 * ks + 2 * t) : 0u;
                qn[ks][1] = in ? ldg4(qb + 16 * ks + 8 + 2 * t) : 0u;
            }
        };
        load_q(it0);
        bool ok = true;
        uint32_t ci = 0;
        int32_t len_next = len_first;
        for (uint32_t it = it0; it < n_items && ok; it += it_step) {
            const Item w = make_item(it, len_next);
            len_next = item_len(it + it_step);
            uint32_t qa[D / 16][2];
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                qa[ks][0] = qn[ks][0];
                qa[ks][1] = qn[ks][1];
            }
            load_q(it + it_step);
            float m_run = -INFINITY, l_run = 0.f;
            float acc[D / 8][4];
#pragma unroll
            for (int e = 0; e < D / 8; ++e) acc[e][0] = acc[e][1] = acc[e][2] = acc[e][3] = 0.f;
#pragma unroll 1
            for (int i = 0; i < w.mine && ok; ++i, ++ci) {
                const int s = (int)(ci % (uint32_t)stages);
                const uint32_t parity = (ci / (uint32_t)stages) & 1;
                const int32_t jblk = __shfl_sync(0xffffffffu, w.cand, lane_of(w, i));
                const int n_keys = jblk == w.row ? w.last_keys : kDecBlock;
                const uint32_t sk = smem_base + (uint32_t)s * SM::kStage, sv = sk + SM::kTile;
                ok = ptx::mbar_wait_bounded(bar_kfull(s), parity, abort_flag, a.status, 2, a.wait_cycles, (int)PA_ERR_TIMEOUT);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                if (16 * wid < n_keys) {  // (else none of this warp's keys exists: the diagonal block's tail)
                    // ---- S = Q K^T: rows = heads, columns = the warp's 16 keys (two 8-key tiles).  K
                    // fragments are requested four feature slices ahead of their MMAs, and each tile
                    // accumulates in two chains (even and odd slices), which halves the dependent-MMA latency.
                    float sc[2][2][4];
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                        for (int c = 0; c < 2; ++c) sc[nt][c][0] = sc[nt][c][1] = sc[nt][c][2] = sc[nt][c][3] = 0.f;
#pragma unroll
                    for (int kb = 0; kb < D / 16; kb += 4) {
                        uint32_t kf[4][4];
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            const int ch = 2 * (kb + x) + k_ch;
                            ptx::ldmatrix_x4(sk + (uint32_t)(ch >> 3) * SM::kSub + (uint32_t)k_key * 128u +
                                                 (uint32_t)(((ch & 7) ^ (k_key & 7)) << 4),
                                             kf[x][0], kf[x][1], kf[x][2], kf[x][3]);
                        }
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            mma_bf16(sc[0][x & 1], qa[kb + x][0], 0u, qa[kb + x][1], 0u, kf[x][0], kf[x][1]);
                            mma_bf16(sc[1][x & 1], qa[kb + x][0], 0u, qa[kb + x][1], 0u, kf[x][2], kf[x][3]);
                        }
                    }
                    // This thread: head g, keys 16 w + 8 nt + 2 t + {0, 1}; base-2 domain; keys that do
                    // not exist become -inf (a select, so whatever the cache holds there is ignored).
                    const int key0 = 16 * wid + 2 * t;
                    float sx[4];
                    sx[0] = key0 < n_keys ? (sc[0][0][0] + sc[0][1][0]) * a.scale_log2 : -INFINITY;
                    sx[1] = key0 + 1 < n_keys ? (sc[0][0][1] + sc[0][1][1]) * a.scale_log2 : -INFINITY;
                    sx[2] = key0 + 8 < n_keys ? (sc[1][0][0] + sc[1][1][0]) * a.scale_log2 : -INFINITY;
                    sx[3] = key0 + 9 < n_keys ? (sc[1][0][1] + sc[1][1][1]) * a.scale_log2 : -INFINITY;
                    float mx = fmaxf(fmaxf(sx[0], sx[1]), fmaxf(sx[2], sx[3]));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));  // finite: key 16 w exists
                    const float m_new = fmaxf(m_run, mx);
                    const float alpha = ptx::ex2(m_run - m_new);  // 0 on the warp's first block
                    const float p0 = ptx::ex2(sx[0] - m_new), p1 = ptx::ex2(sx[1] - m_new);
                    const float p2 = ptx::ex2(sx[2] - m_new), p3 = ptx::ex2(sx[3] - m_new);
                    float lsum = (p0 + p1) + (p2 + p3);
                    lsum += __shfl_xor_sync(0xffffffffu, lsum, 1);
                    lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
                    l_run = l_run * alpha + lsum;
                    m_run = m_new;
                    const uint32_t pa0 = ptx::cvt_bf16x2(p0, p1), pa1 = ptx::cvt_bf16x2(p2, p3);
#pragma unroll
                    for (int e = 0; e < D / 8; ++e) {
                        acc[e][0] *= alpha;
                        acc[e][1] *= alpha;
                    }
                    // V rows of keys that do not exist may hold anything (0 x NaN would poison O):
                    // they are cleared in the fragments.  Only the diagonal block has such rows.
                    uint32_t keep0 = 0xffffffffu, keep1 = 0xffffffffu;
                    if (n_keys < kDecBlock) {
                        keep0 = (key0 < n_keys ? 0x0000ffffu : 0u) | (key0 + 1 < n_keys ? 0xffff0000u : 0u);
                        keep1 = (key0 + 8 < n_keys ? 0x0000ffffu : 0u) | (key0 + 9 < n_keys ? 0xffff0000u : 0u);
                    }
                    ok = ptx::mbar_wait_bounded(bar_vfull(s), parity, abort_flag, a.status, 3, a.wait_cycles, (int)PA_ERR_TIMEOUT);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    // ---- O = alpha O + P V: rows = heads, 16 keys, all D features (8 per MMA)
#pragma unroll
                    for (int eb = 0; eb < D / 16; eb += 4) {
                        uint32_t vf[4][4];
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            const int ch = 2 * (eb + x) + v_ch;
                            ptx::ldmatrix_x4_trans(sv + (uint32_t)(ch >> 3) * SM::kSub + (uint32_t)v_key * 128u +
                                                       (uint32_t)(((ch & 7) ^ (v_key & 7)) << 4),
                                                   vf[x][0], vf[x][1], vf[x][2], vf[x][3]);
                        }
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            mma_bf16(acc[2 * (eb + x)], pa0, 0u, pa1, 0u, vf[x][0] & keep0, vf[x][1] & keep1);
                            mma_bf16(acc[2 * (eb + x) + 1], pa0, 0u, pa1, 0u, vf[x][2] & keep0, vf[x][3] & keep1);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(bar_empty(s));  // this warp has finished with the stage
            }

            // ---- the four warps' partials are merged with the log-sum-exp rule, each warp taking a
            // quarter of the features (four of the 8-feature tiles): a thread passes on the tiles it
            // does not own and picks up, for the tiles it owns, the very elements its lane holds in
            // the other three warps.
            {
                float *mine_out = part + ((size_t)wid * kMaxGroup + g) * SM::kPartRow;
#pragma unroll
                for (int e = 0; e < D / 8; ++e)
                    if (e / (D / 32) != wid)
                        *reinterpret_cast<float2 *>(mine_out + 8 * (e < wid * (D / 32) ? e : e - D / 32) + 2 * t) =
                            make_float2(acc[e][0], acc[e][1]);
                if (t == 0) {
                    mine_out[SM::kPartRow - 2] = m_run;
                    mine_out[SM::kPartRow - 1] = l_run;
                }
            }
            asm volatile("bar.sync 1, %0;\n" ::"n"(32 * kRowConsumers) : "memory");
            float m = -INFINITY, l = 0.f;
            float fin[D / 32][2];
            {
                float mw[kRowConsumers], lw[kRowConsumers], ww[kRowConsumers];
#pragma unroll
                for (int x = 0; x < kRowConsumers; ++x) {
                    const float *src = part + ((size_t)x * kMaxGroup + g) * SM::kPartRow;
                    mw[x] = x == wid ? m_run : src[SM::kPartRow - 2];
                    lw[x] = x == wid ? l_run : src[SM::kPartRow - 1];
                    m = fmaxf(m, mw[x]);
                }
#pragma unroll
                for (int x = 0; x < kRowConsumers; ++x) {
                    ww[x] = mw[x] != -INFINITY ? ptx::ex2(mw[x] - m) : 0.f;
                    l = fmaf(lw[x], ww[x], l);
                }
#pragma unroll
                for (int y = 0; y < D / 32; ++y) {
                    fin[y][0] = fin[y][1] = 0.f;
#pragma unroll
                    for (int x = 0; x < kRowConsumers; ++x) {
                        // warp x keeps this warp's tile y at slot (tile index among the tiles x does not own)
                        const int e = wid * (D / 32) + y;
                        float2 v2;
                        if (x == wid) {
                            v2 = make_float2(0.f, 0.f);  // (own tiles: taken from registers below)
                        } else {
                            const float *src = part + ((size_t)x * kMaxGroup + g) * SM::kPartRow;
                            v2 = *reinterpret_cast<const float2 *>(src + 8 * (e < x * (D / 32) ? e : e - D / 32) + 2 * t);
                        }
                        fin[y][0] = fmaf(v2.x, ww[x], fin[y][0]);
                        fin[y][1] = fmaf(v2.y, ww[x], fin[y][1]);
                    }
                }
                // own tiles out of the accumulators (the tile index depends on the warp: a uniform switch)
#pragma unroll
                for (int e = 0; e < D / 8; ++e)
                    if (e / (D / 32) == wid) {
                        fin[e % (D / 32)][0] = fmaf(acc[e][0], ww[wid], fin[e % (D / 32)][0]);
                        fin[e % (D / 32)][1] = fmaf(acc[e][1], ww[wid], fin[e % (D / 32)][1]);
                    }
            }
            // Thread (g, t) of warp w now holds head g, features (D / 4) w + 8 y + 2 t + {0, 1} of the result.
            {
                const int64_t head = ((int64_t)w.b * a.Hq + (int64_t)w.hk * G + g);
                const int f0 = wid * (D / 4) + 2 * t;
                if (a.mode == kModeCluster) {
                    // Head g is merged by CTA g % R of the cluster: this CTA's part goes straight into
                    // that CTA's receive area (a store through distributed shared memory; the area is
                    // not used for anything else, so the owner may still be busy with its blocks).
                    if (g < G) {
                        namespace cg = cooperative_groups;
                        cg::cluster_group cluster = cg::this_cluster();
                        const int owner = g % R, slot = g / R, heads_per_owner = (kMaxGroup + R - 1) / R;
                        float *dst = (R > 1 ? cluster.map_shared_rank(recv, owner) : recv) +
                                     ((size_t)w.r * heads_per_owner + slot) * (D + 2);
#pragma unroll
                        for (int y = 0; y < D / 32; ++y)
                            *reinterpret_cast<float2 *>(dst + f0 + 8 * y) = make_float2(fin[y][0], fin[y][1]);
                        if (wid == 0 && t == 0) {
                            dst[D] = m;
                            dst[D + 1] = l;
                        }
                    }
                } else if (g < G) {
                    if (a.mode == kModePartial) {
                        float *dst = a.partial + (head * R + w.r) * (D + 2);
#pragma unroll
                        for (int y = 0; y < D / 32; ++y)
                            *reinterpret_cast<float2 *>(dst + f0 + 8 * y) = make_float2(fin[y][0], fin[y][1]);
                        if (wid == 0 && t == 0) {
                            dst[D] = m;
                            dst[D + 1] = l;
                        }
                    } else {
                        const float inv = w.n > 0 ? 1.0f / l : 0.f;
                        if (a.o_is_f32) {
                            float *dst = reinterpret_cast<float *>(a.o) + head * D + f0;
#pragma unroll
                            for (int y = 0; y < D / 32; ++y)
                                *reinterpret_cast<float2 *>(dst + 8 * y) = make_float2(fin[y][0] * inv, fin[y][1] * inv);
                        } else {
                            __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(a.o) + head * D + f0;
#pragma unroll
                            for (int y = 0; y < D / 32; ++y)
                                *reinterpret_cast<uint32_t *>(dst + 8 * y) = ptx::cvt_bf16x2(fin[y][0] * inv, fin[y][1] * inv);
                        }
                        if (wid == 0 && t == 0)
                            a.lse[head] = w.n > 0 ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
                    }
                }
            }
            // The hand-over area is written again only after every warp has read it (the cluster form
            // has one item per CTA: nothing follows).
            if (a.mode != kModeCluster) asm volatile("bar.sync 1, %0;\n" ::"n"(32 * kRowConsumers) : "memory");
        }
    }

    if (a.mode == kModeCluster) {
        // ---- merge across the cluster: every CTA has pushed its parts; after one cluster barrier CTA r
        // merges heads r, r + R, ... from its own receive area (thread d one feature) and writes O
        // and LSE.  Nothing reads a peer's shared memory after the barrier, so no second one is needed.
        namespace cg = cooperative_groups;
        cg::cluster_group cluster = cg::this_cluster();
        const int r = (int)(blockIdx.x % (unsigned)R);
        const int32_t rowid = (int32_t)(blockIdx.x / (unsigned)R);
        const int heads_per_owner = (kMaxGroup + R - 1) / R;
        if (R > 1) cluster.sync();
        else __syncthreads();
        if (tid < D) {
            for (int h = r, slot = 0; h < G; h += R, ++slot) {
                float mr[kRowMaxCluster], lr[kRowMaxCluster], orr[kRowMaxCluster];
#pragma unroll
                for (int rr = 0; rr < kRowMaxCluster; ++rr) {
                    const float *src = recv + ((size_t)(rr < R ? rr : 0) * heads_per_owner + slot) * (D + 2);
                    mr[rr] = src[D];
                    lr[rr] = src[D + 1];
                    orr[rr] = src[tid];
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
                const bool any = m != -INFINITY;  // false: a cache length outside [1, max_len]
                const float out = any ? o / l : 0.f;
                const int64_t oi = ((int64_t)rowid * G + h) * D + tid;
                if (a.o_is_f32)
                    reinterpret_cast<float *>(a.o)[oi] = out;
                else
                    reinterpret_cast<__nv_bfloat16 *>(a.o)[oi] = __float2bfloat16_rn(out);
                if (tid == 0) a.lse[(int64_t)rowid * G + h] = any ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
            }
        }
    }
    __syncthreads();
    if (*abort_flag && tid == 0) {
        // A wait gave up: leave copies that may still be in flight a bounded time to land
        // before the CTA's shared memory is handed to another CTA.
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) {
        }
    }
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

// One warp: the row kernel's own enumeration, compacted in lane order.
__global__ void decode_row_block_set_kernel(int64_t len, int32_t W, int32_t S, int32_t *out, int32_t *count,
                                            int32_t capacity)
{
    const int lane = threadIdx.x;
    const int32_t row = (int32_t)((len - 1) / kDecBlock);
    const int32_t cand = row_block_candidate(row, W, S, lane);
    const uint32_t have = __ballot_sync(0xffffffffu, cand >= 0);
    const int pos = __popc(have & ((1u << lane) - 1u));
    if (cand >= 0 && pos < capacity) out[pos] = cand;
    if (lane == 0) *count = __popc(have);
}

// pa_kv_append, first kernel: the new token's K and V rows go into the page that holds position
// cache_lens[b].  One CTA per (sequence, KV head); a thread copies 16 bytes.  A sequence whose
// block table has no valid page for that position is left alone.
__global__ void kv_append_kernel(const __nv_bfloat16 *k_new, const __nv_bfloat16 *v_new, __nv_bfloat16 *k_pool,
                                 __nv_bfloat16 *v_pool, const int32_t *table, int32_t *lens, int32_t table_stride,
                                 int32_t n_pages, int32_t Hkv, int32_t D, int64_t k_sp, int64_t k_ss, int64_t k_sh,
                                 int64_t v_sp, int64_t v_ss, int64_t v_sh)
{
    const int hk = blockIdx.x, b = blockIdx.y;
    const int32_t pos = lens[b];
    const int32_t blk = pos / kDecBlock;
    bool ok = pos >= 0 && blk < table_stride;
    int32_t page = 0;
    if (ok) {
        page = table[(int64_t)b * table_stride + blk];
        ok = page >= 0 && page < n_pages;
    }
    if (ok) {
        const int slot = pos % kDecBlock;
        const int c = threadIdx.x;  // 16-byte piece of the row
        if (c < D / 8) {
            const uint4 kv = *reinterpret_cast<const uint4 *>(k_new + ((int64_t)b * Hkv + hk) * D + 8 * c);
            const uint4 vv = *reinterpret_cast<const uint4 *>(v_new + ((int64_t)b * Hkv + hk) * D + 8 * c);
            *reinterpret_cast<uint4 *>(k_pool + page * k_sp + slot * k_ss + hk * k_sh + 8 * c) = kv;
            *reinterpret_cast<uint4 *>(v_pool + page * v_sp + slot * v_ss + hk * v_sh + 8 * c) = vv;
        }
    }
}

// pa_kv_append, second kernel: every CTA of the first one has read the old lengths by now; the
// sequences that had a valid page grow by one token.
__global__ void kv_advance_kernel(const int32_t *table, int32_t *lens, int32_t batch, int32_t table_stride,
                                  int32_t n_pages)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= batch) return;
    const int32_t pos = lens[b];
    const int32_t blk = pos / kDecBlock;
    if (pos < 0 || blk >= table_stride) return;
    const int32_t page = table[(int64_t)b * table_stride + blk];
    if (page < 0 || page >= n_pages) return;
    lens[b] = pos + 1;
}

// Window distances + power-of-two distances beyond the window + sink blocks that a row below
// n_rows can have, before any of them coincide or fall off the sequence start: the number of
// candidate slots the row kernel enumerates (one per lane, so it needs this to be <= 32).
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
    const int64_t bound = row_candidate_slots(n_rows, W, S);
    return (int)(bound < n_rows ? bound : n_rows);
}

// What the checks below need to know about a decode problem, whichever cache form it uses.
struct DecodeShape {
    int32_t batch, n_q_heads, n_kv_heads, head_dim, block, window_blocks, sink_blocks;
    int64_t max_len;
    pa_strides k, v;
    pa_dtype o_dtype;
    float softmax_scale;
};

static pa_status check_decode_shape(const DecodeShape &p)
{
    if (p.batch < 1 || p.n_q_heads < 1 || p.n_kv_heads < 1 || p.max_len < 1)
        return fail(PA_ERR_INVALID_ARG, "batch, head counts and max_len must be positive");
    if (p.window_blocks < 0 || p.sink_blocks < 0)
        return fail(PA_ERR_INVALID_ARG, "window_blocks and sink_blocks must be >= 0");
    if (p.o_dtype != PA_BF16 && p.o_dtype != PA_F32) return fail(PA_ERR_INVALID_ARG, "bad o_dtype");
    if (!(p.softmax_scale >= 0.f) || isinf(p.softmax_scale))
        return fail(PA_ERR_INVALID_ARG, "softmax_scale must be finite and >= 0 (0 = default)");
    if (p.head_dim != 64 && p.head_dim != 128) return fail(PA_ERR_SHAPE, "head_dim must be 64 or 128");
    if (p.block != kDecBlock) return fail(PA_ERR_SHAPE, "block must be 64");
    if (p.n_q_heads % p.n_kv_heads) return fail(PA_ERR_SHAPE, "n_q_heads must be a multiple of n_kv_heads");
    if (p.n_q_heads / p.n_kv_heads > kMaxGroup)
        return fail(PA_ERR_SHAPE, "at most %d query heads per KV head", kMaxGroup);
    if (p.max_len > ((int64_t)1 << 30)) return fail(PA_ERR_SHAPE, "max_len too large (limit 2^30 tokens)");
    if (p.batch > 65535 || p.n_kv_heads > 65535 || p.n_q_heads > 65535)
        return fail(PA_ERR_SHAPE, "batch and head counts must be <= 65535");
    if (p.window_blocks > 4096 || p.sink_blocks > 4096)
        return fail(PA_ERR_SHAPE, "window_blocks and sink_blocks must be <= 4096");
    const pa_strides *st[2] = {&p.k, &p.v};
    for (auto s : st) {
        if (s->seq < p.head_dim || s->head < p.head_dim || s->batch < 0)
            return fail(PA_ERR_SHAPE, "cache strides must be >= head_dim");
        if ((s->seq % 8) || (s->head % 8) || (s->batch % 8))
            return fail(PA_ERR_ALIGNMENT, "cache strides must be multiples of 8 elements (16 bytes)");
        if (s->seq >= ((int64_t)1 << 38) || s->head >= ((int64_t)1 << 38) || s->batch >= ((int64_t)1 << 38))
            return fail(PA_ERR_SHAPE, "cache strides too large for a tensor map");
    }
    return PA_OK;
}

static pa_status shape_of(const pa_decode_params *p, DecodeShape *s)
{
    if (!p) return fail(PA_ERR_INVALID_ARG, "params must be non-null");
    *s = DecodeShape{p->batch, p->n_q_heads, p->n_kv_heads, p->head_dim, p->block, p->window_blocks, p->sink_blocks,
                     p->max_len, p->k, p->v, p->o_dtype, p->softmax_scale};
    return check_decode_shape(*s);
}

static pa_status shape_of(const pa_paged_params *p, DecodeShape *s)
{
    if (!p) return fail(PA_ERR_INVALID_ARG, "params must be non-null");
    if (p->n_pages < 1 || p->max_blocks_per_seq < 1)
        return fail(PA_ERR_INVALID_ARG, "n_pages and max_blocks_per_seq must be positive");
    *s = DecodeShape{p->batch, p->n_q_heads, p->n_kv_heads, p->head_dim, p->block, p->window_blocks, p->sink_blocks,
                     (int64_t)p->max_blocks_per_seq * kDecBlock, p->k, p->v, p->o_dtype, p->softmax_scale};
    if (pa_status st = check_decode_shape(*s)) return st;
    if (p->k.batch < (int64_t)kDecBlock * p->head_dim || p->v.batch < (int64_t)kDecBlock * p->head_dim)
        return fail(PA_ERR_SHAPE, "the page stride must cover a page of %d tokens", kDecBlock);
    return PA_OK;
}

static bool takes_split_k(const DecodeShape &s)
{
    const int64_t rows = (s.max_len + kDecBlock - 1) / kDecBlock;
    return env_switches().decode_path == 1 || row_candidate_slots(rows, s.window_blocks, s.sink_blocks) > 32;
}

static size_t decode_workspace_bytes(const DecodeShape &s)
{
    const int64_t rows = (s.max_len + kDecBlock - 1) / kDecBlock;
    const int chunks = max_row_blocks(rows, s.window_blocks, s.sink_blocks);
    return kDecStatusBytes + (size_t)s.batch * s.n_q_heads * chunks * (s.head_dim + 2) * sizeof(float);
}

// The launch shared by every decode entry point.  table == null: contiguous cache.
static pa_status launch_decode(const DecodeShape &p, const void *q, const void *k_cache, const void *v_cache,
                               const int32_t *table, int32_t table_stride, int32_t n_pages,
                               const int32_t *cache_lens, void *o, float *lse, void *workspace,
                               size_t workspace_bytes, void *stream)
{
    if (!q || !k_cache || !v_cache || !cache_lens || !o || !lse)
        return fail(PA_ERR_INVALID_ARG, "q, the caches, cache_lens, o and lse must be non-null");
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(o))
        return fail(PA_ERR_ALIGNMENT, "q, the caches and o must be 16-byte aligned");
    // (What this launch really touches: the status block, plus the partials on the split-K path.
    // The public entry points hold their callers to the documented size before they get here.)
    const size_t need = takes_split_k(p) ? decode_workspace_bytes(p) : kDecStatusBytes;
    if (!workspace || workspace_bytes < need)
        return fail(PA_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", need, workspace_bytes);
    if (!aligned16(workspace)) return fail(PA_ERR_ALIGNMENT, "workspace must be 16-byte aligned");
    DeviceInfo dev;
    if (pa_status s = current_sm100_device(&dev)) return s;

    DecodeArgs a;
    a.q = static_cast<const __nv_bfloat16 *>(q);
    a.k = static_cast<const __nv_bfloat16 *>(k_cache);
    a.v = static_cast<const __nv_bfloat16 *>(v_cache);
    a.lens = cache_lens;
    a.table = table;
    a.table_stride = table_stride;
    a.n_pages = n_pages;
    a.status = static_cast<int32_t *>(workspace);
    a.partial = reinterpret_cast<float *>(static_cast<uint8_t *>(workspace) + kDecStatusBytes);
    a.o = o;
    a.lse = lse;
    a.k_sb = p.k.batch; a.k_ss = p.k.seq; a.k_sh = p.k.head;
    a.v_sb = p.v.batch; a.v_ss = p.v.seq; a.v_sh = p.v.head;
    a.max_len = p.max_len;
    a.batch = p.batch; a.Hq = p.n_q_heads; a.Hkv = p.n_kv_heads;
    a.G = p.n_q_heads / p.n_kv_heads;
    a.W = p.window_blocks; a.S = p.sink_blocks;
    const int64_t rows = (p.max_len + kDecBlock - 1) / kDecBlock;
    a.chunks = max_row_blocks(rows, p.window_blocks, p.sink_blocks);
    a.o_is_f32 = p.o_dtype == PA_F32;
    a.stages = 0;
    const float scale = p.softmax_scale != 0.f ? p.softmax_scale : 1.0f / sqrtf((float)p.head_dim);
    a.scale_log2 = scale * 1.4426950408889634f;
    a.wait_cycles = wait_limit_cycles() > 0 ? wait_limit_cycles() : kRowWaitCycles;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const EnvSwitches env = env_switches();
    a.fixed_chunks = 0;
    a.R = 1;
    a.mode = kModeCluster;
    a.items = 0;
    // Rows whose block set fits one warp's lanes take the row kernel.
    if (!takes_split_k(p)) {
        const int64_t rows_in_call = (int64_t)a.batch * a.Hkv;
        const int max_R = a.chunks < kRowMaxCluster ? a.chunks : kRowMaxCluster;
        const int64_t persistent_ctas = (env.decode_ctas_per_sm ? env.decode_ctas_per_sm : 2) * (int64_t)dev.sms;
        // Small calls (latency-bound): one launch, a cluster of R CTAs per row, all resident at once.  Larger calls (bandwidth-bound): a persistent grid of
        // two CTAs per SM over (row, chunk) items.
        bool cluster = rows_in_call * kRowMaxCluster <= 2 * persistent_ctas;
        if (env.decode_path == 2) cluster = true;
        if (env.decode_path == 3) cluster = false;
        int R = env.decode_cluster;
        if (cluster) {
            if (R == 0) {
                // as many CTAs per row as still run all at once (two CTAs fit an SM): a second wave
                // of clusters doubles the call's latency (batch 16: 17.4 us with R = 8, 12.5 with R = 4)
                R = (int)(persistent_ctas / rows_in_call);
                if (R < 1) R = 1;
            }
            if (R > max_R) R = max_R;
            a.mode = kModeCluster;
        } else {
            // One chunk per row once there are enough rows for every SM; measured: finer items
            // balance the SMs better on paper but pay more per item than they gain.
            if (R == 0) R = rows_in_call >= dev.sms ? 1 : 2;
            if (R > max_R) R = max_R;
            a.mode = R == 1 ? kModeDirect : kModePartial;
        }
        a.R = R;
        a.items = rows_in_call * R;
        const int64_t grid = a.mode == kModeCluster ? a.items : (a.items < persistent_ctas ? a.items : persistent_ctas);
        if (a.items > 0x3fffffff) return fail(PA_ERR_SHAPE, "too many work items (%lld)", (long long)a.items);
        // Stages: 64 KB of blocks in flight per CTA, and no more than a CTA has blocks.
        const int64_t blocks_per_cta = ((int64_t)a.chunks * rows_in_call + grid - 1) / grid;
        // (two stages measured 1-3 % faster than three at batch 64 and 256, head_dim 128)
        const int fit = p.head_dim == 128 ? 2 : 4;
        a.stages = env.decode_stages != 0 ? env.decode_stages : fit;
        if (a.stages > kRowMaxStages) a.stages = kRowMaxStages;
        if (a.stages > blocks_per_cta) a.stages = (int)blocks_per_cta;
        if (a.stages < 1) a.stages = 1;
        while (a.stages > 1 && (p.head_dim == 128 ? RowSmem<128>::bytes(a.stages, a.mode == kModeCluster)
                                                  : RowSmem<64>::bytes(a.stages, a.mode == kModeCluster)) > (size_t)kRowMaxSmem)
            --a.stages;

        // Tensor maps over the cache: (feature, token, head, batch or page), one 64 x 64 box per copy.
        CUtensorMap tmK, tmV;
        const bool paged = table != nullptr;
        TensorMapKey kk = {k_cache, paged ? (int64_t)kDecBlock : p.max_len, p.k.seq, p.k.head, p.k.batch, dev.device,
                           p.head_dim, p.n_kv_heads, paged ? n_pages : p.batch, 1, kDecBlock};
        TensorMapKey kv = {v_cache, paged ? (int64_t)kDecBlock : p.max_len, p.v.seq, p.v.head, p.v.batch, dev.device,
                           p.head_dim, p.n_kv_heads, paged ? n_pages : p.batch, 1, kDecBlock};
        if (pa_status s = get_tensor_map(kk, "k_cache", &tmK)) return s;
        if (pa_status s = get_tensor_map(kv, "v_cache", &tmV)) return s;

        if (device_once_begin(dev.device, ONCE_DECODE_ATTR)) {
            const cudaError_t e1 = cudaFuncSetAttribute(decode_row_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                        kRowMaxSmem);
            const cudaError_t e2 = cudaFuncSetAttribute(decode_row_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                        kRowMaxSmem);
            if (e1 != cudaSuccess || e2 != cudaSuccess) {
                device_once_reset(dev.device, ONCE_DECODE_ATTR);
                return fail(PA_ERR_CUDA, "cudaFuncSetAttribute failed: %s",
                            cudaGetErrorString(e1 != cudaSuccess ? e1 : e2));
            }
        }
        if (a.mode == kModePartial) {
            a.chunks = R;  // the partials of a row are its R chunks
            a.fixed_chunks = R;
        }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)grid, 1, 1);
        cfg.blockDim = dim3(kRowThreads, 1, 1);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = a.mode == kModeCluster ? (unsigned)R : 1u;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (p.head_dim == 128) {
            cfg.dynamicSmemBytes = RowSmem<128>::bytes(a.stages, a.mode == kModeCluster);
            PA_CUDA_OK(cudaLaunchKernelEx(&cfg, decode_row_kernel<128>, tmK, tmV, a));
        } else {
            cfg.dynamicSmemBytes = RowSmem<64>::bytes(a.stages, a.mode == kModeCluster);
            PA_CUDA_OK(cudaLaunchKernelEx(&cfg, decode_row_kernel<64>, tmK, tmV, a));
        }
        if (a.mode != kModePartial) return PA_OK;
    } else {
        const dim3 grid1((unsigned)a.chunks, (unsigned)a.Hkv, (unsigned)a.batch);
        if (p.head_dim == 128)
            decode_block_kernel<128><<<grid1, kDecThreads, 0, st>>>(a);
        else
            decode_block_kernel<64><<<grid1, kDecThreads, 0, st>>>(a);
        PA_CUDA_OK(cudaGetLastError());
    }

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)a.Hq, (unsigned)a.batch, 1);
    cfg.blockDim = dim3((unsigned)p.head_dim, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (p.head_dim == 128)
        PA_CUDA_OK(cudaLaunchKernelEx(&cfg, decode_combine_kernel<128>, a));
    else
        PA_CUDA_OK(cudaLaunchKernelEx(&cfg, decode_combine_kernel<64>, a));
    return PA_OK;
}

}  // namespace pa

extern "C" size_t pa_decode_workspace_bytes(const pa_decode_params *p)
{
    using namespace pa;
    DecodeShape s;
    if (shape_of(p, &s) != PA_OK) return 0;
    return decode_workspace_bytes(s);
}

extern "C" pa_status pa_decode(const pa_decode_params *p, const void *q, const void *k_cache,
                               const void *v_cache, const int32_t *cache_lens, void *o,
                               float *lse, void *workspace, size_t workspace_bytes, void *stream)
{
    using namespace pa;
    clear_error();
    DecodeShape s;
    if (pa_status st = shape_of(p, &s)) return st;
    const size_t need = decode_workspace_bytes(s);
    if (!workspace || workspace_bytes < need)
        return fail(PA_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", need, workspace_bytes);
    return launch_decode(s, q, k_cache, v_cache, nullptr, 0, 0, cache_lens, o, lse, workspace, workspace_bytes, stream);
}

extern "C" size_t pa_decode_paged_workspace_bytes(const pa_paged_params *p)
{
    using namespace pa;
    DecodeShape s;
    if (shape_of(p, &s) != PA_OK) return 0;
    return decode_workspace_bytes(s);
}

extern "C" pa_status pa_decode_paged(const pa_paged_params *p, const void *q, const void *k_pool,
                                     const void *v_pool, const int32_t *block_table,
                                     const int32_t *cache_lens, void *o, float *lse, void *workspace,
                                     size_t workspace_bytes, void *stream)
{
    using namespace pa;
    clear_error();
    DecodeShape s;
    if (pa_status st = shape_of(p, &s)) return st;
    if (!block_table) return fail(PA_ERR_INVALID_ARG, "block_table must be non-null");
    const size_t need = decode_workspace_bytes(s);
    if (!workspace || workspace_bytes < need)
        return fail(PA_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", need, workspace_bytes);
    return launch_decode(s, q, k_pool, v_pool, block_table, p->max_blocks_per_seq, p->n_pages, cache_lens, o, lse,
                         workspace, workspace_bytes, stream);
}

extern "C" pa_status pa_kv_append(const pa_paged_params *p, const void *k_new, const void *v_new, void *k_pool,
                                  void *v_pool, const int32_t *block_table, int32_t *cache_lens, void *stream)
{
    using namespace pa;
    clear_error();
    DecodeShape s;
    if (pa_status st = shape_of(p, &s)) return st;
    if (!k_new || !v_new || !k_pool || !v_pool || !block_table || !cache_lens)
        return fail(PA_ERR_INVALID_ARG, "k_new, v_new, the pools, block_table and cache_lens must be non-null");
    if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_pool) || !aligned16(v_pool))
        return fail(PA_ERR_ALIGNMENT, "k_new, v_new and the pools must be 16-byte aligned");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    kv_append_kernel<<<dim3((unsigned)p->n_kv_heads, (unsigned)p->batch), 32, 0, st>>>(
        static_cast<const __nv_bfloat16 *>(k_new), static_cast<const __nv_bfloat16 *>(v_new),
        static_cast<__nv_bfloat16 *>(k_pool), static_cast<__nv_bfloat16 *>(v_pool), block_table, cache_lens,
        p->max_blocks_per_seq, p->n_pages, p->n_kv_heads, p->head_dim, p->k.batch, p->k.seq, p->k.head, p->v.batch,
        p->v.seq, p->v.head);
    kv_advance_kernel<<<(unsigned)((p->batch + 127) / 128), 128, 0, st>>>(block_table, cache_lens, p->batch,
                                                                          p->max_blocks_per_seq, p->n_pages);
    PA_CUDA_OK(cudaGetLastError());
    return PA_OK;
}

extern "C" pa_status pa_decode_status(const void *workspace, void *stream, int32_t *detail)
{
    using namespace pa;
    clear_error();
    if (!workspace) return fail(PA_ERR_INVALID_ARG, "workspace must be non-null");
    int32_t host[2] = {0, 0};
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    PA_CUDA_OK(cudaMemcpyAsync(host, workspace, sizeof host, cudaMemcpyDeviceToHost, st));
    PA_CUDA_OK(cudaStreamSynchronize(st));
    if (detail) *detail = host[1];
    if (host[0] == (int32_t)PA_ERR_TIMEOUT)
        return fail(PA_ERR_TIMEOUT, "a bounded wait inside the decode kernel ran out (wait id %d)", host[1]);
    if (host[0] != 0) return fail(PA_ERR_CUDA, "unexpected device status %d", host[0]);
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

extern "C" pa_status pa_decode_row_block_set(int64_t cache_len, int32_t block, int32_t window_blocks,
                                             int32_t sink_blocks, int32_t *out_blocks, int32_t *out_count,
                                             int32_t capacity, void *stream)
{
    using namespace pa;
    clear_error();
    if (cache_len < 1 || cache_len > ((int64_t)1 << 30)) return fail(PA_ERR_INVALID_ARG, "cache_len must be in [1, 2^30]");
    if (block != kDecBlock) return fail(PA_ERR_SHAPE, "block must be 64");
    if (window_blocks < 0 || sink_blocks < 0 || capacity < 32 || !out_blocks || !out_count)
        return fail(PA_ERR_INVALID_ARG, "bad window/sink, capacity < 32 or null output");
    const int64_t rows = (cache_len + kDecBlock - 1) / kDecBlock;
    if (row_candidate_slots(rows, window_blocks, sink_blocks) > 32)
        return fail(PA_ERR_SHAPE, "window + sink + power-of-two candidates exceed 32: such rows take the split-K path");
    decode_row_block_set_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(
        cache_len, window_blocks, sink_blocks, out_blocks, out_count, capacity);
    PA_CUDA_OK(cudaGetLastError());
    return PA_OK;
}

// ------------------------------------------------------------------------------------------
// pa_decode_static: the same decode, for callers that cannot allocate device memory.
//
// The workspace (status block and split-K partial results) is a fixed array that is part of the
// library image instead of a caller-provided buffer.  The array's name is only a host-side handle
// in host code; the real device address is looked up once per device with cudaGetSymbolAddress
// (with that device current) and then handed to the kernels like any other pointer.
// ------------------------------------------------------------------------------------------
namespace pa {

static __device__ __align__(256) unsigned char g_decode_static_scratch[PA_DECODE_STATIC_SCRATCH_BYTES];

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
    DecodeShape s;
    if (pa_status st = shape_of(p, &s)) return st;
    // The single-launch path keeps only its status block in the workspace; the partial results
    // of the two-kernel path are what has to fit the built-in array.
    const size_t need = takes_split_k(s) ? decode_workspace_bytes(s) : kDecStatusBytes;
    if (need > (size_t)PA_DECODE_STATIC_SCRATCH_BYTES)
        return fail(PA_ERR_WORKSPACE,
                    "this problem needs %zu bytes of split-K scratch but the built-in array holds %zu; "
                    "use pa_decode with a caller-allocated workspace", need,
                    (size_t)PA_DECODE_STATIC_SCRATCH_BYTES);
    void *scratch = nullptr;
    if (pa_status st = static_scratch_address(&scratch)) return st;
    return launch_decode(s, q, k_cache, v_cache, nullptr, 0, 0, cache_lens, o, lse, scratch,
                         (size_t)PA_DECODE_STATIC_SCRATCH_BYTES, stream);
}
