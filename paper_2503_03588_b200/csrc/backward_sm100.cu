// Backward pass of the block-sparse attention (derivatives of Eq. (1), Section 3.1, under the
// key-block lists of Algorithm 1, Section 3.3) on the sm_100a tensor cores, head_dim 128.
//
// Two kernels with the same skeleton:
//   warp 0       TMA producer (bf16 tiles, 128-byte swizzle, into rings of shared-memory stages)
//   warp 1       tcgen05 issuer of S and dP (one elected lane; the dQ kernel: of S)
//   warp 2       tensor-memory allocation (the dQ kernel: and issuer of dP)
//   warp 3       tcgen05 issuer of the second products
//   warps 4-7    compute group 0: even steps
//   warps 8-11   compute group 1: odd steps
//   warps 12-15  (dQ kernel) epilogue: the finished dQ out of tensor memory and out to global memory
// A step is one (query block, key block) pair for a pair of query heads stacked on the 64 tokens of
// the query block: a 128-row tile, as in the forward kernel.  Per step the tensor cores produce
// S = Q K^T and dP = dO V^T (128 x 64, fp32, tensor memory, two buffers: one per compute group); the
// group's threads (thread = tile row = TMEM lane) turn them into P = exp2(S scale log2e - LSE log2e)
// and dS = P (dP - delta), rounded to bf16; the second products accumulate in tensor memory.
//
//   dq_kernel   persistent; an item is a (query block, head pair): walks the row's key blocks; dS goes
//               back into tensor memory as the A operand of dQ += dS K (128 x 128 accumulator)
//   dkv_kernel  one CTA per (chunk of a key block's listing query blocks, KV head): walks the chunk
//               for every head pair of the group; P and dS go to shared memory as the B operands of
//               dV^T += dO^T P and dK^T += Q^T dS (feature x key accumulators, 128 x 64 each: the A
//               operands are the dO and Q tiles read feature-major), added into dK / dV with fp32
//               reductions because a column listed by many rows is spread over several CTAs
//
// Every barrier wait is bounded; a wait that runs out records PA_ERR_TIMEOUT in the status block,
// raises a CTA-wide abort flag, every role leaves its loop and the CTA ends after a bounded pause.
#include <cuda.h>
#include <cuda_bf16.h>
#include <math.h>

#include "backward.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

// Registers per thread by role.  A warpgroup asking for more than the pool holds would wait for ever:
// the dK / dV kernel starts 384 threads x 168, the dQ kernel (with its epilogue warps) 512 x 128.
#define PA_BWD_REG_CTRL 56
#define PA_BWD_REG_COMP 216
static_assert(4 * PA_BWD_REG_CTRL + 8 * PA_BWD_REG_COMP <= 12 * 168, "register split exceeds the CTA's registers");
#define PA_DQ_REG_COMP 144
#define PA_BWD_REG_EPI 168
static_assert(4 * PA_BWD_REG_CTRL + 8 * PA_DQ_REG_COMP + 4 * PA_BWD_REG_EPI <= 16 * 128, "register split exceeds the CTA's registers");

namespace pa {

constexpr int kTcThreads = 384;
constexpr int kDqThreads = 512;  // + four epilogue warps
constexpr uint32_t kTcTmemCols = 512;
constexpr long long kBwdWaitCycles = 4000000000ll;
constexpr uint32_t kRowTile = 128 * 128;   // 128 rows x 64 features: one 128-byte-wide half of a Q or dO tile
constexpr uint32_t kKeyTile = 64 * 128;    // 64 keys x 64 features: one half of a K or V block
// High word of every shared-memory descriptor: 1024 bytes between 8-row groups, version 1, 128-byte swizzle.
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);

// Instruction descriptor (kind::f16, bf16 operands, fp32 accumulation) with both major bits.
__host__ __device__ constexpr uint32_t idesc_bf16(int M, int N, int a_mn, int b_mn)
{
    return ptx::idesc_bf16_f32(M, N, b_mn) | ((uint32_t)a_mn << 15);
}

// ------------------------------------------------------------------------------------- dQ
// Persistent: one CTA per SM walks items (query block, head pair, batch entry), long rows first.
// Steps are numbered through the CTA's whole run, so ring positions, buffers and barrier parities do
// not care about item boundaries.  Q and dO have one buffer: the next item's tiles are requested when
// the current item's last S and dP have been issued and arrive while its last steps are computed
// and its dQ leaves tensor memory, which takes longer; the K / V ring of four stages covers a
// stage's life from request to the dQ product that reads it last.
constexpr int kDqStages = 4;  // K + V ring
constexpr uint32_t kDqOutPitch = 144;  // bytes per staged row of 32 fp32 (conflict-free 16-byte stores, 4-byte loads)
struct DqSmem {
    static constexpr uint32_t kQG = 0;                      // Q (two halves of 128 rows x 128 B), then dO
    static constexpr uint32_t kItem = 4 * kRowTile;
    static constexpr uint32_t kKV = kQG + kItem;            // stage: K (two halves), then V
    static constexpr uint32_t kStage = 4 * kKeyTile;
    static constexpr uint32_t kOut = kKV + kDqStages * kStage;  // per epilogue warp: 32 rows x 32 fp32 of dQ on their way out
    static constexpr uint32_t kBars = kOut + 4 * 32 * kDqOutPitch;
    static constexpr uint32_t kAlloc = kBars + 512 + 1024;
    static_assert(kAlloc <= 227 * 1024, "shared memory budget");
};
enum : uint32_t {
    DQ_QG_FULL = 0, DQ_QG_EMPTY = 1,
    DQ_KV_FULL = 2, DQ_KV_EMPTY = DQ_KV_FULL + kDqStages,
    DQ_SD_FULL = DQ_KV_EMPTY + kDqStages,  // [buffer]: S and dP of a step are in tensor memory
    DQ_S_TAKEN = DQ_SD_FULL + 2,            // [buffer]: the group has them in registers
    DQ_DS_FULL = DQ_S_TAKEN + 2,            // [buffer]: dS is in tensor memory
    DQ_DS_FREE = DQ_DS_FULL + 2,            // [buffer]: dQ += dS K has read it
    DQ_DONE = DQ_DS_FREE + 2,               // the item's last dQ += dS K has completed
    DQ_FREE = DQ_DONE + 1,                  // the epilogue warps have read dQ out of tensor memory
    DQ_BAR_COUNT = DQ_FREE + 1
};

struct DqItem {
    int32_t i, hk, hp, b, e0, n;
};
// Item index -> coordinates: query blocks from the last (longest row) to the first, and within a
// query block the head pairs and batch entries.
__device__ __forceinline__ DqItem dq_item(const BackwardArgs &a, uint32_t it)
{
    DqItem w;
    const uint32_t per_row = (uint32_t)(a.Hkv * a.npairs * a.batch);
    const uint32_t x = it / per_row, yz = it % per_row;
    const uint32_t hkp = yz % (uint32_t)(a.Hkv * a.npairs);
    w.i = a.nqb - 1 - (int32_t)x;
    w.b = (int32_t)(yz / (uint32_t)(a.Hkv * a.npairs));
    w.hk = (int32_t)(hkp / (uint32_t)a.npairs);
    w.hp = (int32_t)(hkp % (uint32_t)a.npairs);
    w.e0 = __ldg(a.row_ptr + w.i);
    w.n = __ldg(a.row_ptr + w.i + 1) - w.e0;
    return w;
}

__global__ void __launch_bounds__(kDqThreads, 1)
dq_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmG,
          const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const BackwardArgs a,
          const uint32_t n_items)
{
    constexpr int D = 128;
    using SM = DqSmem;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    const uint32_t bars = smem_base + SM::kBars;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + SM::kBars + DQ_BAR_COUNT * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + SM::kBars + DQ_BAR_COUNT * 8 + 8);
    auto bar = [&](uint32_t idx) { return bars + idx * 8u; };
    auto wait_bar = [&](uint32_t b_, uint32_t parity, int code) {
        return ptx::mbar_wait_bounded(b_, parity, abort_flag, a.status, code, a.wait_cycles, (int)PA_ERR_TIMEOUT);
    };
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        ptx::mbar_init(bar(DQ_QG_FULL), 1);
        ptx::mbar_init(bar(DQ_QG_EMPTY), 2);  // one commit from each of the S and dP issuers
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(bar(DQ_SD_FULL + s), 2);
            ptx::mbar_init(bar(DQ_S_TAKEN + s), 4);
            ptx::mbar_init(bar(DQ_DS_FULL + s), 4);
            ptx::mbar_init(bar(DQ_DS_FREE + s), 1);
        }
        for (int s = 0; s < kDqStages; ++s) {
            ptx::mbar_init(bar(DQ_KV_FULL + s), 1);
            ptx::mbar_init(bar(DQ_KV_EMPTY + s), 1);
        }
        ptx::mbar_init(bar(DQ_DONE), 1);
        ptx::mbar_init(bar(DQ_FREE), 4);
        *abort_flag = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async_smem();
    }
    if (warp == 2) {
        ptx::tmem_alloc(ptx::smem_u32(tmem_slot), kTcTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // Tensor memory columns: buffer b: S at 160 b, dP at 160 b + 64, dS (bf16 pairs) at 160 b + 128; dQ at 320.
    constexpr uint32_t kColDq = 320;

    if (warp < 4) ptx::setmaxnreg_dec<PA_BWD_REG_CTRL>();
    if (warp == 0) {
        // -------------------------------------------------------------- TMA producer
        if (lane == 0) {
            ptx::prefetch_tensormap(&tmQ);
            ptx::prefetch_tensormap(&tmG);
            ptx::prefetch_tensormap(&tmK);
            ptx::prefetch_tensormap(&tmV);
            uint32_t c = 0, k = 0;  // steps and (non-empty) items so far
            bool ok = true;
            for (uint32_t it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
                const DqItem w = dq_item(a, it);
                if (w.n <= 0) continue;
                if (k >= 1 && !wait_bar(bar(DQ_QG_EMPTY), (k - 1) & 1, 1)) break;
                const int h0 = w.hk * a.G + 2 * w.hp;
                const uint32_t qdst = smem_base + SM::kQG;
                ptx::mbar_expect_tx(bar(DQ_QG_FULL), SM::kItem);
                for (int dh = 0; dh < 2; ++dh) {
                    ptx::tma_load_4d(qdst + dh * kRowTile, &tmQ, bar(DQ_QG_FULL), dh * 64, w.i * kBwdBlk, h0, w.b);
                    ptx::tma_load_4d(qdst + 2 * kRowTile + dh * kRowTile, &tmG, bar(DQ_QG_FULL), dh * 64, w.i * kBwdBlk, h0, w.b);
                }
                int32_t j = __ldg(a.col_idx + w.e0);
                for (int e = 0; e < w.n; ++e, ++c) {
                    const int32_t jn = e + 1 < w.n ? __ldg(a.col_idx + w.e0 + e + 1) : 0;
                    const uint32_t st = c % kDqStages;
                    if (c >= (uint32_t)kDqStages && !wait_bar(bar(DQ_KV_EMPTY + st), (c / kDqStages - 1) & 1, 2)) {
                        ok = false;
                        break;
                    }
                    ptx::mbar_expect_tx(bar(DQ_KV_FULL + st), SM::kStage);
                    const uint32_t dst = smem_base + SM::kKV + st * SM::kStage;
                    for (int dh = 0; dh < 2; ++dh) {
                        ptx::tma_load_4d(dst + dh * kKeyTile, &tmK, bar(DQ_KV_FULL + st), dh * 64, j * kBwdBlk, w.hk, w.b);
                        ptx::tma_load_4d(dst + 2 * kKeyTile + dh * kKeyTile, &tmV, bar(DQ_KV_FULL + st), dh * 64, j * kBwdBlk, w.hk, w.b);
                    }
                    j = jn;
                }
                ++k;
            }
        }
        __syncwarp();
    } else if (warp == 1 || warp == 2) {
        // -------------------------------------------------------------- tcgen05 issuers of S (warp 1) and dP (warp 2)
        // (a warp each: issuing a step's sixteen MMAs and its three waits from one warp took longer
        // than the tensor cores need for them)
        const bool leader = ptx::elect_one();
        const bool is_dp = __shfl_sync(0xffffffffu, warp, 0) == 2;
        constexpr uint32_t idesc_s = idesc_bf16(128, 64, 0, 0);   // both operands K-major
        // A = Q (S) or dO (dP); B = the K or V half of the stage.
        const uint32_t a_lo = ((smem_base + SM::kQG + (is_dp ? 2 * kRowTile : 0u)) >> 4) | (1u << 16);
        uint32_t c = 0, k = 0;
        bool ok = true;
        for (uint32_t it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
            const int n = __shfl_sync(0xffffffffu, dq_item(a, it).n, 0);
            if (n <= 0) continue;
            for (int e = 0; e < n && ok; ++e, ++c) {
                const uint32_t bf = c & 1, st = c % kDqStages;
                if (e == 0) ok = __all_sync(0xffffffffu, wait_bar(bar(DQ_QG_FULL), k & 1, 3));
                if (ok) ok = __all_sync(0xffffffffu, wait_bar(bar(DQ_KV_FULL + st), (c / kDqStages) & 1, 4));
                if (ok && c >= 2) ok = __all_sync(0xffffffffu, wait_bar(bar(DQ_S_TAKEN + bf), ((c >> 1) - 1) & 1, 5));
                if (!ok) break;
                ptx::tc_fence_after_sync();
                if (leader) {
                    const uint32_t b_lo = ((smem_base + SM::kKV + st * SM::kStage + (is_dp ? 2 * kKeyTile : 0u)) >> 4) | (1u << 16);
                    const uint32_t t_d = tmem_base + 160 * bf + (is_dp ? 64u : 0u);
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk)
                        ptx::umma_ss_lohi(t_d, a_lo + (((kk / 4) * kRowTile + (kk % 4) * 32) >> 4), kDescHi,
                                          b_lo + (((kk / 4) * kKeyTile + (kk % 4) * 32) >> 4), kDescHi, idesc_s, kk > 0 ? 1u : 0u);
                    ptx::umma_commit(bar(DQ_SD_FULL + bf));
                    if (e == n - 1) ptx::umma_commit(bar(DQ_QG_EMPTY));  // this warp has read the item's Q (dO) tile
                }
                __syncwarp();
            }
            ++k;
        }
    } else if (warp == 3) {
        // -------------------------------------------------------------- tcgen05 issuer of dQ
        // (its own warp: a single issuer that served both kinds in order held each back behind the other's waits)
        const bool leader = ptx::elect_one();
        constexpr uint32_t idesc_dq = idesc_bf16(128, D, 0, 1);   // A = dS (tensor memory), B = K feature-contiguous
        uint32_t c = 0, k = 0;
        bool ok = true;
        for (uint32_t it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
            const int n = __shfl_sync(0xffffffffu, dq_item(a, it).n, 0);
            if (n <= 0) continue;
            for (int e = 0; e < n && ok; ++e, ++c) {
                const uint32_t bf = c & 1, st = c % kDqStages;
                ok = __all_sync(0xffffffffu, wait_bar(bar(DQ_DS_FULL + bf), (c >> 1) & 1, 6));
                // The previous item's dQ must have left tensor memory.
                if (ok && e == 0 && k > 0) ok = __all_sync(0xffffffffu, wait_bar(bar(DQ_FREE), (k - 1) & 1, 7));
                if (!ok) break;
                ptx::tc_fence_after_sync();
                if (leader) {
                    // B = the K block read feature-contiguous: 16 keys per MMA, 2048 bytes further each.
                    const uint32_t kb = ((smem_base + SM::kKV + st * SM::kStage) >> 4) | ((kKeyTile >> 4) << 16);
                    const uint32_t t_ds = tmem_base + 160 * bf + 128;
#pragma unroll
                    for (int kk = 0; kk < kBwdBlk / 16; ++kk)
                        ptx::umma_ts_lohi(tmem_base + kColDq, t_ds + kk * 8, kb + ((kk * 2048) >> 4), kDescHi, idesc_dq,
                                          (e > 0 || kk > 0) ? 1u : 0u);
                    ptx::umma_commit(bar(DQ_KV_EMPTY + st));
                    ptx::umma_commit(bar(DQ_DS_FREE + bf));
                    if (e == n - 1) ptx::umma_commit(bar(DQ_DONE));
                }
                __syncwarp();
            }
            ++k;
        }
    } else if (warp >= 4 && warp < 12) {
        // -------------------------------------------------------------- compute groups
        ptx::setmaxnreg_inc<PA_DQ_REG_COMP>();
        const int wg = (warp - 4) >> 2, quad = warp & 3;
        const int row = quad * 32 + lane, qrow = row & 63;
        const uint32_t t_lane = tmem_base + ((uint32_t)(quad * 32) << 16);
        // An item's row data for this thread: LSE (base 2), delta, whether the row ends on its diagonal
        // block.  Fetched one item ahead, so the loads are not waited for at an item's start (the item's
        // coordinates, which need the row extents, one item earlier still).
        struct RowData {
            DqItem w;
            float lse2, delta;
            bool last_is_diag;
        };
        auto fetch_item = [&](uint32_t it) {
            DqItem w = {};
            w.n = -1;
            if (it < n_items) w = dq_item(a, it);
            return w;
        };
        auto fetch = [&](uint32_t it, const DqItem &w) {
            RowData r;
            r.w = w;
            r.lse2 = INFINITY;
            r.delta = 0.f;
            r.last_is_diag = false;
            if (it >= n_items) return r;
            const int head_local = 2 * r.w.hp + (row >> 6);
            const int head = r.w.hk * a.G + head_local;
            const int64_t q = (int64_t)r.w.i * kBwdBlk + qrow;
            if (head_local < a.G && q < a.N) {
                const int64_t at = ((int64_t)r.w.b * a.Hq + head) * a.N + q;
                const float lse = __ldg(a.lse + at);
                // (a row the layout left empty has no weights: P = 0)
                r.lse2 = (lse == -INFINITY || lse == INFINITY) ? INFINITY : lse * 1.4426950408889634f;
                r.delta = __ldg(a.delta + at);
            }
            r.last_is_diag = r.w.n > 0 && __ldg(a.col_idx + r.w.e0 + r.w.n - 1) == r.w.i;
            return r;
        };
        uint32_t c = 0;
        bool ok = true;
        RowData next = fetch(blockIdx.x, fetch_item(blockIdx.x));
        DqItem item2 = fetch_item(blockIdx.x + gridDim.x);
        for (uint32_t it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
            const RowData r = next;
            next = fetch(it + gridDim.x, item2);
            item2 = fetch_item(it + 2 * gridDim.x);
            const int n = r.w.n;
            if (n <= 0) continue;
            const float lse2 = r.lse2, delta = r.delta;
            for (int e = 0; e < n; ++e, ++c) {
                if ((int)(c & 1) != wg) continue;
                ok = __all_sync(0xffffffffu, wait_bar(bar(DQ_SD_FULL + wg), (c >> 1) & 1, 8));
                if (!ok) break;
                ptx::tc_fence_after_sync();
                // Algorithm 1's causal term acts inside the diagonal pair only (the row's last block).
                const int lim = (r.last_is_diag && e == n - 1) ? qrow : 63;
                uint32_t pk[32];
                // Two halves of 32 keys, so that the logits of one half only are held at a time.
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t s[32], dp[32];
                    ptx::tmem_ld32(t_lane + 160 * wg + 32 * half, s);
                    ptx::tmem_ld32(t_lane + 160 * wg + 64 + 32 * half, dp);
                    ptx::tmem_wait_ld();
                    if (half == 1) {
                        // S and dP are in registers: their buffer may take the step after next.
                        ptx::tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(bar(DQ_S_TAKEN + wg));
                    }
#pragma unroll
                    for (int x = 0; x < 32; x += 2) {
                        float ds[2];
#pragma unroll
                        for (int y = 0; y < 2; ++y) {
                            const float p = (32 * half + x + y <= lim)
                                                ? ptx::ex2(fmaf(__uint_as_float(s[x + y]), a.scale_log2, -lse2)) : 0.f;
                            ds[y] = p * (__uint_as_float(dp[x + y]) - delta);
                        }
                        pk[16 * half + (x >> 1)] = ptx::cvt_bf16x2(ds[0], ds[1]);
                    }
                }
                if (c >= 2) {
                    ok = __all_sync(0xffffffffu, wait_bar(bar(DQ_DS_FREE + wg), ((c >> 1) - 1) & 1, 9));
                    if (!ok) break;
                }
                ptx::tmem_st32(t_lane + 160 * wg + 128, pk);
                ptx::tmem_wait_st();
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(bar(DQ_DS_FULL + wg));
            }
        }
    } else {
        // -------------------------------------------------------------- epilogue
        // dQ = scale x the accumulator, off the compute groups' path: writing an item's 64 KB out takes
        // several thousand cycles (the SM's store path), which the next item's steps run beside.  The
        // accumulator is read into registers in one go, which frees it for the next item at once.
        ptx::setmaxnreg_inc<PA_BWD_REG_EPI>();
        const int quad = warp & 3;
        const int row = quad * 32 + lane, qrow = row & 63;
        const uint32_t t_lane = tmem_base + ((uint32_t)(quad * 32) << 16);
        const uint32_t patch = smem_base + SM::kOut + (uint32_t)quad * 32u * kDqOutPitch;
        const uint8_t *patch_ptr = smem + SM::kOut + quad * 32 * kDqOutPitch;
        uint32_t k = 0;
        bool ok = true;
        for (uint32_t it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
            const DqItem w = dq_item(a, it);
            const int head_local = 2 * w.hp + (row >> 6);
            const bool head_ok = head_local < a.G;
            const int64_t q = (int64_t)w.i * kBwdBlk + qrow;
            const int64_t out = (((int64_t)w.b * a.N + q) * a.Hq + w.hk * a.G + head_local) * D;
            if (w.n <= 0) {  // empty row: zero gradient, no barrier traffic
                if (head_ok && q < a.N)
                    for (int x = 0; x < D; x += 4) *reinterpret_cast<float4 *>(a.dq + out + x) = make_float4(0.f, 0.f, 0.f, 0.f);
                continue;
            }
            ok = __all_sync(0xffffffffu, wait_bar(bar(DQ_DONE), k & 1, 10));
            if (!ok) break;
            ptx::tc_fence_after_sync();
            uint32_t acc[4][32];
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) ptx::tmem_ld32(t_lane + kColDq + 32 * ch, acc[ch]);
            ptx::tmem_wait_ld();
            // dQ is in registers: tensor memory may take the next item's first dS K.
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar(DQ_FREE));
            // A thread holds its own row: stored from here, every instruction would touch 32 rows.  The
            // warp turns 32 features at a time through its shared-memory patch, so that an instruction
            // writes one row's 128 contiguous bytes.
            const int64_t out0 = __shfl_sync(0xffffffffu, out, 0);  // lane 0's row; the warp's rows follow at Hq D
            const int64_t q0 = __shfl_sync(0xffffffffu, q, 0);
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
#pragma unroll
                for (int x = 0; x < 32; x += 4)
                    ptx::st_shared_v4(patch + (uint32_t)lane * kDqOutPitch + 4u * x, acc[ch][x], acc[ch][x + 1], acc[ch][x + 2],
                                      acc[ch][x + 3]);
                __syncwarp();
                // (all loads first: a load behind a global store would wait for it, the two might alias)
                float v[32];
#pragma unroll
                for (int rho = 0; rho < 32; ++rho) v[rho] = *reinterpret_cast<const float *>(patch_ptr + rho * kDqOutPitch + 4 * lane);
                __syncwarp();
#pragma unroll
                for (int rho = 0; rho < 32; ++rho)
                    if (head_ok && q0 + rho < a.N) a.dq[out0 + (int64_t)rho * a.Hq * D + 32 * ch + lane] = v[rho] * a.scale;
            }
            ++k;
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 2) {
        // After a wait that gave up, copies and tensor-core operations issued before it may still be
        // in flight: they finish by themselves within microseconds; a bounded two milliseconds pass
        // before the tensor memory is given back.
        if (*abort_flag) {
            const long long t0 = clock64();
            while (clock64() - t0 < 4000000ll) {
            }
        }
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTcTmemCols);
    }
}

// ------------------------------------------------------------------------------------- dK, dV
struct DkvSmem {
    static constexpr uint32_t kK = 0;                        // two halves of 64 keys x 128 B
    static constexpr uint32_t kV = kK + 2 * kKeyTile;
    static constexpr uint32_t kQG = kV + 2 * kKeyTile;       // stage: Q (two halves of 128 rows x 128 B), then dO
    static constexpr uint32_t kStage = 4 * kRowTile;
    static constexpr uint32_t kPD = kQG + 2 * kStage;        // buffer: P (128 rows x 64 keys), then dS
    static constexpr uint32_t kBuf = 2 * kRowTile;
    static constexpr uint32_t kBars = kPD + 2 * kBuf;
    static constexpr uint32_t kAlloc = kBars + 512 + 1024;
    static_assert(kAlloc <= 227 * 1024, "shared memory budget");
};
enum : uint32_t {
    KV_KV_FULL = 0,
    KV_QG_FULL = 1, KV_QG_EMPTY = 3,  // [stage]
    KV_SD_FULL = 5,                   // [buffer]: S and dP of a step are in tensor memory
    KV_S_TAKEN = 7,                   // [buffer]: the group has them in registers
    KV_PD_FULL = 9,                   // [buffer]: P and dS are in shared memory
    KV_DONE = 11,
    KV_BAR_COUNT = 12
};

__global__ void __launch_bounds__(kTcThreads, 1)
dkv_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmG,
           const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const BackwardArgs a)
{
    constexpr int D = 128;
    using SM = DkvSmem;
    const int32_t c = blockIdx.x;
    if (c >= a.chunk_ptr[a.nqb]) return;  // (the grid is an upper bound on the number of chunks)
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    const uint32_t bars = smem_base + SM::kBars;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + SM::kBars + KV_BAR_COUNT * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + SM::kBars + KV_BAR_COUNT * 8 + 8);
    auto bar = [&](uint32_t idx) { return bars + idx * 8u; };
    auto wait_bar = [&](uint32_t b_, uint32_t parity, int code) {
        return ptx::mbar_wait_bounded(b_, parity, abort_flag, a.status, code, a.wait_cycles, (int)PA_ERR_TIMEOUT);
    };
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int hk = blockIdx.y, b = blockIdx.z;
    // The column whose chunks include c: last j with chunk_ptr[j] <= c.
    int32_t lo = 0, hi = a.nqb;
    while (hi - lo > 1) {
        const int32_t mid = (lo + hi) >> 1;
        if (a.chunk_ptr[mid] <= c) lo = mid;
        else hi = mid;
    }
    const int32_t j = lo;
    const int32_t e0 = a.col_ptr[j] + (c - a.chunk_ptr[j]) * kBwdChunk;
    const int32_t e1 = e0 + kBwdChunk < a.col_ptr[j + 1] ? e0 + kBwdChunk : a.col_ptr[j + 1];
    const int n = (e1 - e0) * a.npairs;  // steps: listing query blocks x head pairs (pairs fastest); at least one

    if (threadIdx.x == 0) {
        ptx::mbar_init(bar(KV_KV_FULL), 1);
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(bar(KV_QG_FULL + s), 1);
            ptx::mbar_init(bar(KV_QG_EMPTY + s), 1);
            ptx::mbar_init(bar(KV_SD_FULL + s), 2);  // one commit from each of the S and dP issuers
            ptx::mbar_init(bar(KV_S_TAKEN + s), 4);
            ptx::mbar_init(bar(KV_PD_FULL + s), 4);
        }
        ptx::mbar_init(bar(KV_DONE), 1);
        *abort_flag = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async_smem();
    }
    if (warp == 2) {
        ptx::tmem_alloc(ptx::smem_u32(tmem_slot), kTcTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // Tensor memory columns: buffer b: S at 128 b, dP at 128 b + 64; dK^T at 256, dV^T at 320 (64 keys each).
    constexpr uint32_t kColDk = 256, kColDv = 320;

    if (warp < 4) ptx::setmaxnreg_dec<PA_BWD_REG_CTRL>();
    if (warp == 0) {
        // -------------------------------------------------------------- TMA producer
        if (lane == 0) {
            ptx::prefetch_tensormap(&tmQ);
            ptx::prefetch_tensormap(&tmG);
            ptx::prefetch_tensormap(&tmK);
            ptx::prefetch_tensormap(&tmV);
            ptx::mbar_expect_tx(bar(KV_KV_FULL), 4 * kKeyTile);
            for (int dh = 0; dh < 2; ++dh) {
                ptx::tma_load_4d(smem_base + SM::kK + dh * kKeyTile, &tmK, bar(KV_KV_FULL), dh * 64, j * kBwdBlk, hk, b);
                ptx::tma_load_4d(smem_base + SM::kV + dh * kKeyTile, &tmV, bar(KV_KV_FULL), dh * 64, j * kBwdBlk, hk, b);
            }
            int32_t i = 0;
            for (int e = 0, hp = 0; e < n; ++e) {
                if (hp == 0) i = __ldg(a.row_idx + e0 + e / a.npairs);
                const uint32_t st = e & 1;
                if (e >= 2 && !wait_bar(bar(KV_QG_EMPTY + st), ((e >> 1) - 1) & 1, 2)) break;
                ptx::mbar_expect_tx(bar(KV_QG_FULL + st), SM::kStage);
                const uint32_t dst = smem_base + SM::kQG + st * SM::kStage;
                const int h0 = hk * a.G + 2 * hp;
                for (int dh = 0; dh < 2; ++dh) {
                    ptx::tma_load_4d(dst + dh * kRowTile, &tmQ, bar(KV_QG_FULL + st), dh * 64, i * kBwdBlk, h0, b);
                    ptx::tma_load_4d(dst + 2 * kRowTile + dh * kRowTile, &tmG, bar(KV_QG_FULL + st), dh * 64, i * kBwdBlk, h0, b);
                }
                if (++hp == a.npairs) hp = 0;
            }
        }
        __syncwarp();
    } else if (warp == 1 || warp == 2) {
        // -------------------------------------------------------------- tcgen05 issuers of S (warp 1) and dP (warp 2)
        const bool leader = ptx::elect_one();
        const bool is_dp = __shfl_sync(0xffffffffu, warp, 0) == 2;
        constexpr uint32_t idesc_s = idesc_bf16(128, 64, 0, 0);    // both operands K-major
        // A = Q (S) or dO (dP) of the stage; B = the key block's K or V.
        const uint32_t b_lo = ((smem_base + (is_dp ? SM::kV : SM::kK)) >> 4) | (1u << 16);
        bool ok = __all_sync(0xffffffffu, wait_bar(bar(KV_KV_FULL), 0, 1));
        for (int e = 0; e < n && ok; ++e) {
            const uint32_t bf = e & 1;
            ok = __all_sync(0xffffffffu, wait_bar(bar(KV_QG_FULL + bf), (e >> 1) & 1, 3));
            if (ok && e >= 2) ok = __all_sync(0xffffffffu, wait_bar(bar(KV_S_TAKEN + bf), ((e >> 1) - 1) & 1, 4));
            if (!ok) break;
            ptx::tc_fence_after_sync();
            if (leader) {
                const uint32_t a_lo = ((smem_base + SM::kQG + bf * SM::kStage + (is_dp ? 2 * kRowTile : 0u)) >> 4) | (1u << 16);
                const uint32_t t_d = tmem_base + 128 * bf + (is_dp ? 64u : 0u);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk)
                    ptx::umma_ss_lohi(t_d, a_lo + (((kk / 4) * kRowTile + (kk % 4) * 32) >> 4), kDescHi,
                                      b_lo + (((kk / 4) * kKeyTile + (kk % 4) * 32) >> 4), kDescHi, idesc_s, kk > 0 ? 1u : 0u);
                ptx::umma_commit(bar(KV_SD_FULL + bf));
            }
            __syncwarp();
        }
    } else if (warp == 3) {
        // -------------------------------------------------------------- tcgen05 issuer of dV^T and dK^T
        // (its own warp: a Q / dO stage is free for the next load only when these have read it, and a
        // single in-order issuer put them behind the next step's S and dP)
        const bool leader = ptx::elect_one();
        constexpr uint32_t idesc_t = idesc_bf16(128, 64, 1, 1);    // A feature-contiguous, B key-contiguous
        bool ok = true;
        for (int e1 = 0; e1 < n && ok; ++e1) {
            {
                const uint32_t bf = e1 & 1;
                ok = __all_sync(0xffffffffu, wait_bar(bar(KV_PD_FULL + bf), (e1 >> 1) & 1, 5));
                if (!ok) break;
                ptx::tc_fence_after_sync();
                if (leader) {
                    // A = the dO (Q) tile read feature-contiguous (its two 64-feature halves are kRowTile
                    // apart), B = P (dS) read key-contiguous; 16 tile rows per MMA, 2048 bytes further each.
                    const uint32_t qa = ((smem_base + SM::kQG + bf * SM::kStage) >> 4) | ((kRowTile >> 4) << 16);
                    const uint32_t ga = qa + ((2 * kRowTile) >> 4);
                    const uint32_t pb = ((smem_base + SM::kPD + bf * SM::kBuf) >> 4) | ((kRowTile >> 4) << 16);
                    const uint32_t db = pb + (kRowTile >> 4);
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        ptx::umma_ss_lohi(tmem_base + kColDv, ga + ((kk * 2048) >> 4), kDescHi, pb + ((kk * 2048) >> 4), kDescHi,
                                          idesc_t, (e1 > 0 || kk > 0) ? 1u : 0u);
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        ptx::umma_ss_lohi(tmem_base + kColDk, qa + ((kk * 2048) >> 4), kDescHi, db + ((kk * 2048) >> 4), kDescHi,
                                          idesc_t, (e1 > 0 || kk > 0) ? 1u : 0u);
                    ptx::umma_commit(bar(KV_QG_EMPTY + bf));  // (frees the P / dS buffer as well)
                    if (e1 == n - 1) ptx::umma_commit(bar(KV_DONE));
                }
                __syncwarp();
            }
        }
    } else if (warp >= 4) {
        // -------------------------------------------------------------- compute groups
        ptx::setmaxnreg_inc<PA_BWD_REG_COMP>();
        const int wg = (warp - 4) >> 2, quad = warp & 3;
        const int row = quad * 32 + lane, qrow = row & 63;
        const uint32_t t_lane = tmem_base + ((uint32_t)(quad * 32) << 16);
        // Row statistics of a step for this thread's row: LSE and delta; +inf / 0 for a row without
        // weights (beyond the sequence, padding head, empty row): P = 0.  Nothing here uses a loaded
        // value (the thread would wait for it on the spot): the query block index is loaded two of
        // this group's steps ahead, LSE and delta one step ahead, and they are looked at when the step
        // they belong to begins.
        auto step_block = [&](int e) { return e < n ? __ldg(a.row_idx + e0 + e / a.npairs) : -1; };
        auto request_stats = [&](int e, int32_t i, float &lse, float &delta, bool &diag) {
            lse = INFINITY;
            delta = 0.f;
            diag = false;
            if (e >= n) return;
            const int head_local = 2 * (e % a.npairs) + (row >> 6);
            const int64_t q = (int64_t)i * kBwdBlk + qrow;
            diag = i == j;
            if (head_local < a.G && q < a.N) {
                const int64_t at = ((int64_t)b * a.Hq + hk * a.G + head_local) * a.N + q;
                lse = __ldg(a.lse + at);
                delta = __ldg(a.delta + at);
            }
        };
        float lse_raw, delta, lse_raw_n, delta_n;
        bool diag, diag_n;
        int32_t i_next = step_block(wg + 2);
        request_stats(wg, step_block(wg), lse_raw, delta, diag);
        const uint32_t p_row = smem_base + SM::kPD + wg * SM::kBuf + (uint32_t)row * 128u;
        bool ok = true;
        for (int e = wg; e < n; e += 2) {
            const int32_t i_next2 = step_block(e + 4);
            request_stats(e + 2, i_next, lse_raw_n, delta_n, diag_n);  // (in flight during this step)
            ok = __all_sync(0xffffffffu, wait_bar(bar(KV_SD_FULL + wg), (e >> 1) & 1, 6));
            if (!ok) break;
            ptx::tc_fence_after_sync();
            uint32_t s[64], dp[64];
            ptx::tmem_ld32(t_lane + 128 * wg, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
            ptx::tmem_ld32(t_lane + 128 * wg + 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
            ptx::tmem_ld32(t_lane + 128 * wg + 64, *reinterpret_cast<uint32_t(*)[32]>(&dp[0]));
            ptx::tmem_ld32(t_lane + 128 * wg + 96, *reinterpret_cast<uint32_t(*)[32]>(&dp[32]));
            ptx::tmem_wait_ld();
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar(KV_S_TAKEN + wg));
            // (The P / dS buffer is free: the second products of step e - 2 that read it had completed
            // before this step's Q and dO could be loaded into the stage they also read, and so before
            // the S and dP waited for above were issued.)
            // Algorithm 1's causal term acts inside the diagonal pair only.
            const int lim = diag ? qrow : 63;
            const float lse2 = (lse_raw == -INFINITY || lse_raw == INFINITY) ? INFINITY : lse_raw * 1.4426950408889634f;
#pragma unroll
            for (int ch = 0; ch < 8; ++ch) {
                uint32_t pp[4], pd[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    float p[2], ds[2];
#pragma unroll
                    for (int y = 0; y < 2; ++y) {
                        const int col = 8 * ch + 2 * x + y;
                        p[y] = (col <= lim) ? ptx::ex2(fmaf(__uint_as_float(s[col]), a.scale_log2, -lse2)) : 0.f;
                        ds[y] = p[y] * (__uint_as_float(dp[col]) - delta);
                    }
                    pp[x] = ptx::cvt_bf16x2(p[0], p[1]);
                    pd[x] = ptx::cvt_bf16x2(ds[0], ds[1]);
                }
                // 16-byte chunk ch of tile row r sits at chunk position ch ^ (r & 7) (128-byte swizzle).
                const uint32_t off = (uint32_t)((ch ^ (row & 7)) << 4);
                ptx::st_shared_v4(p_row + off, pp[0], pp[1], pp[2], pp[3]);
                ptx::st_shared_v4(p_row + kRowTile + off, pd[0], pd[1], pd[2], pd[3]);
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar(KV_PD_FULL + wg));
            lse_raw = lse_raw_n;
            delta = delta_n;
            diag = diag_n;
            i_next = i_next2;
        }
        // Group 0 adds dK^T (x scale), group 1 dV^T: thread = feature, one key per register.
        if (ok) ok = __all_sync(0xffffffffu, wait_bar(bar(KV_DONE), 0, 8));
        if (ok) {
            ptx::tc_fence_after_sync();
            float *dst = (wg == 0 ? a.dk : a.dv) + (((int64_t)b * a.N + (int64_t)j * kBwdBlk) * a.Hkv + hk) * D + row;
            const float f = wg == 0 ? a.scale : 1.0f;
#pragma unroll
            for (int ch = 0; ch < 2; ++ch) {
                uint32_t acc[32];
                ptx::tmem_ld32(t_lane + (wg == 0 ? kColDk : kColDv) + 32 * ch, acc);
                ptx::tmem_wait_ld();
#pragma unroll
                for (int x = 0; x < 32; ++x) {
                    const int key = 32 * ch + x;
                    if ((int64_t)j * kBwdBlk + key < a.N) atomicAdd(dst + (int64_t)key * a.Hkv * D, __uint_as_float(acc[x]) * f);
                }
            }
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 2) {
        if (*abort_flag) {
            const long long t0 = clock64();
            while (clock64() - t0 < 4000000ll) {
            }
        }
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTcTmemCols);
    }
}

// ---------------------------------------------------------------------------------- host side
pa_status launch_backward_sm100(const BackwardArgs &args, const pa_prefill_params *p, int64_t nnz, int device, int sms,
                                cudaStream_t st)
{
    BackwardArgs a = args;
    a.npairs = (a.G + 1) / 2;
    const long long wait_cycles = wait_limit_cycles();
    a.wait_cycles = wait_cycles > 0 ? wait_cycles : kBwdWaitCycles;
    // Tensor maps (cached per buffer and shape): a Q or dO box holds the two heads of a tile, a K or V box one head.
    CUtensorMap tmQ, tmG, tmK, tmV;
    auto map_of = [&](const void *base, int heads, const pa_strides &s, int box_heads, const char *what, CUtensorMap *m) {
        const TensorMapKey key = {base, p->seq_len, s.seq, s.head, s.batch, device, 128, heads, p->batch, box_heads, kBwdBlk};
        return get_tensor_map(key, what, m);
    };
    if (pa_status s = map_of(a.q, a.Hq, p->q, 2, "q", &tmQ)) return s;
    if (pa_status s = map_of(a.d_o, a.Hq, p->o, 2, "d_o", &tmG)) return s;
    if (pa_status s = map_of(a.k, a.Hkv, p->k, 1, "k", &tmK)) return s;
    if (pa_status s = map_of(a.v, a.Hkv, p->v, 1, "v", &tmV)) return s;
    if (device_once_begin(device, ONCE_BACKWARD_TC_ATTR)) {
        const cudaError_t e1 = cudaFuncSetAttribute(dq_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DqSmem::kAlloc);
        const cudaError_t e2 = cudaFuncSetAttribute(dkv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DkvSmem::kAlloc);
        if (e1 != cudaSuccess || e2 != cudaSuccess) {
            device_once_reset(device, ONCE_BACKWARD_TC_ATTR);
            return fail(PA_ERR_CUDA, "cudaFuncSetAttribute failed: %s", cudaGetErrorString(e1 != cudaSuccess ? e1 : e2));
        }
    }
    const int64_t n_items = (int64_t)a.nqb * a.Hkv * a.npairs * a.batch;
    if (n_items > (int64_t)0x3fffffff) return fail(PA_ERR_SHAPE, "too many work items (%lld)", (long long)n_items);
    dq_kernel<<<(unsigned)(n_items < sms ? n_items : sms), kDqThreads, DqSmem::kAlloc, st>>>(tmQ, tmG, tmK, tmV, a, (uint32_t)n_items);
    // (an upper bound on the number of chunks; CTAs beyond the real count return at once)
    const int64_t max_chunks = nnz / kBwdChunk + a.nqb;
    dkv_kernel<<<dim3((unsigned)max_chunks, (unsigned)a.Hkv, (unsigned)a.batch), kTcThreads, DkvSmem::kAlloc, st>>>(tmQ, tmG, tmK, tmV, a);
    PA_CUDA_OK(cudaGetLastError());
    return PA_OK;
}

}  // namespace pa
