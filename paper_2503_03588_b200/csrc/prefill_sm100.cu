// pa_prefill: block-sparse causal attention forward (Eq. (1), Section 3.1) over the CSR
// key-block lists of Algorithm 1 (Section 3.3), for sm_100a.
//
// One persistent CTA per SM walks work units (batch, KV head, query block, head quad).  A unit
// holds two 128-row tiles ("slots"); a tile stacks two query heads of the KV group on the 64
// tokens of the query block (the mask does not depend on the head, so they share the key list
// and the K/V tiles).  The key list is walked one 64-key block per step.  Warp roles:
//   warp 0      TMA producer: the listed K and V blocks, gathered by block index, into two rings
//               of shared-memory tiles (128-byte swizzle); the next unit's Q tiles early in
//               the current unit, into the second of two Q buffers
//   warps 1, 3  tcgen05 issuers, one per slot.  S = Q K^T of step t+1 is issued as soon as the
//               softmax warps hold S of step t in registers (one S buffer per slot), so those
//               logits are ready when step t ends, across unit boundaries too; O += P V is issued
//               when P has been handed over (P has its own two buffers in tensor memory)
//   warp 2      tensor-memory allocation
//   warps 4-7   online softmax of slot 0 (thread = tile row = TMEM lane), LSE
//   warps 8-11  online softmax of slot 1; the two slots take turns at the exponentials
//   warps 12-15 epilogue: O / l out of tensor memory into the finished unit's own Q buffer
//               (swizzled for the bulk tensor stores to global memory); runs beside the next
//               unit's first steps
// Warps 0-3 and 12-15 give registers back (setmaxnreg) and the softmax warpgroups take them.
// Every barrier wait is bounded; a wait that runs out records PA_ERR_TIMEOUT in the status
// block, raises a CTA-wide abort flag, every role leaves its loop and the CTA ends after a bounded
// pause for what is still in flight (no trap, no endless spin).
#include <cuda.h>
#include <cuda_bf16.h>
#include <math.h>
#include <stdlib.h>

#include "common.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

// Registers per thread by role: 4 control warps, 8 softmax warps, 4 epilogue warps share the
// CTA's 16 x 128.
#ifndef PA_REG_CTRL
#define PA_REG_CTRL 56
#define PA_REG_SOFT 176
#define PA_REG_EPI 104
#endif
// A warpgroup asking for more than the pool holds would wait for ever.
static_assert(4 * PA_REG_CTRL + 8 * PA_REG_SOFT + 4 * PA_REG_EPI <= 16 * 128, "register split exceeds the CTA's registers");
static_assert(PA_REG_CTRL % 8 == 0 && PA_REG_SOFT % 8 == 0 && PA_REG_EPI % 8 == 0, "setmaxnreg takes multiples of 8");

namespace pa {

constexpr int kBlk = 64;               // tokens per query / key block
constexpr int kThreads = 512;          // 16 warps: control, two softmax warpgroups, epilogue
constexpr int kKStages = 3;             // K block ring depth (a K block is needed at the start of a step)
constexpr int kVStages = 3;             // V block ring depth (a V block is needed at its end; loads take longer than two steps)
constexpr uint32_t kTmemCols = 512;    // slot s: S at columns 128 s, P buffers at 128 s + 64 + 32 b, O at 256 + s D
// A step's row sum above this limit sends the step through the exact path (new reference).
constexpr float kSumLimit = 1048576.0f;  // 2^20
constexpr int kTurnAtColumn = 16;  // column of a pass at which the other slot gets its turn (a multiple of 4 below 64)
constexpr float kRescaleThreshold = 8.0f;  // base-2 logits: rescale O only when the row max grows by more
constexpr long long kWaitCycles = 4000000000ll;  // default limit of a barrier wait: ~2 s at 2 GHz

struct PrefillArgs {
    const int32_t *row_ptr, *col_idx;
    const int32_t *cu_seqlens;  // variable-length batch: [batch + 1] token offsets of the packed sequences; else null
    void *o;
    float *lse;
    int32_t *status;  // [0] error code, [1] detail
    int64_t o_sb, o_ss, o_sh;
    int64_t lse_sb, lse_sh;  // LSE strides (batch, head); the token stride is 1
    int64_t N, n_units;     // N: sequence length (variable-length batch: the longest one, which sizes the unit grid)
    int32_t nqb, batch, Hq, Hkv, G, nsub, o_is_f32;
    uint32_t inv_nsub, inv_Hkv, inv_nqb;  // floor(2^32 / d) of the three divisors of a unit index
    float scale_log2;
    long long wait_cycles;  // limit of every barrier wait, in clock cycles
};

template <int D>
struct SmemMap {
    static constexpr uint32_t kQSub = 128 * 128;              // 128 rows x 64 features (128 B)
    static constexpr uint32_t kQSlot = kQSub * (D / 64);
    static constexpr uint32_t kQ = 0;
    static constexpr uint32_t kBlkSub = 64 * 128;             // 64 keys x 64 features
    static constexpr uint32_t kBlkTile = kBlkSub * (D / 64);  // one K or V block
    static constexpr uint32_t kQBuf = 2 * kQSlot;             // both slots' Q tiles of one unit
    static constexpr uint32_t kK = kQ + 2 * kQBuf;            // two units' worth: the next unit's Q loads early
    static constexpr uint32_t kV = kK + kKStages * kBlkTile;
    // A finished unit's output is staged in that unit's own Q buffer (its four heads x 64 tokens
    // take exactly the room of the two 128-row Q tiles), so it needs no area of its own.
    static constexpr uint32_t kOHead = 64 * D * 2;            // one head x 64 tokens of staged O
    static_assert(4 * kOHead == kQBuf, "the staged output of a unit fills its Q buffer");
    static constexpr uint32_t kStats = kV + kVStages * kBlkTile;  // [slot][row] softmax denominators
    static constexpr uint32_t kBars = kStats + 2 * 128 * 4;
    static constexpr uint32_t kTotal = kBars + 512;
    static constexpr uint32_t kAlloc = kTotal + 1024;         // slack for 1024-byte alignment
    static_assert(kAlloc <= 227 * 1024, "shared memory budget");
};

// Barrier slots inside the barrier area (8 bytes each).
enum : uint32_t {
    BAR_Q_FULL = 0, BAR_Q_EMPTY = 2,  // [unit parity]
    BAR_K_FULL = 4, BAR_K_EMPTY = BAR_K_FULL + kKStages,
    BAR_V_FULL = BAR_K_EMPTY + kKStages, BAR_V_EMPTY = BAR_V_FULL + kVStages,
    BAR_S_FULL = BAR_V_EMPTY + kVStages,  // [slot]: S of the step is in tensor memory
    BAR_S_TAKEN = BAR_S_FULL + 2,         // [slot]: the softmax warps have S in registers
    BAR_P_FULL = BAR_S_TAKEN + 2,  // [slot][step parity]: P of that step is in tensor memory
    BAR_O_DONE = BAR_P_FULL + 4,  // [slot][step parity]: P V of that step has completed
    BAR_O_FINAL = BAR_O_DONE + 4,   // [slot]: the unit's last P V has completed
    BAR_ML_READY = BAR_O_FINAL + 2,  // [slot]: the unit's row statistics are in shared memory
    BAR_O_FREE = BAR_ML_READY + 2,   // [slot]: the epilogue has read O out of tensor memory
    BAR_STAGE_FREE = BAR_O_FREE + 2,  // [unit parity]: the bulk stores have read the unit's staged output
    BAR_STAGE_FULL = BAR_STAGE_FREE + 2,  // a slot's two heads have been staged by the four epilogue warps
    BAR_TURN = BAR_STAGE_FULL + 1,  // [slot]: the other slot has finished a pass of exponentials
    BAR_COUNT = BAR_TURN + 2
};

struct Unit {
    int32_t b, hk, i, sub, rs, n;
    // Where the unit's sequence lives: batch coordinate of the tensor maps, offset of its first
    // token along their token axis, its length.  (Equal-length batch: b, 0, N.  Packed
    // variable-length batch: 0, cu_seqlens[b], cu_seqlens[b + 1] - cu_seqlens[b].)
    int32_t bt, tok0, len;
};

// u / d and u % d with inv = floor(2^32 / d) (2^32 - 1 for d = 1): the high product falls short of
// the quotient by at most one for every 32-bit u, which one compare puts right.  Every role decodes
// a unit index per unit, the softmax warps on their critical path; division by a run-time divisor
// costs some ten times as many instructions.
__device__ __forceinline__ uint32_t divmod(uint32_t u, uint32_t d, uint32_t inv, uint32_t &rem)
{
    uint32_t q = __umulhi(u, inv);
    uint32_t r = u - q * d;
    if (r >= d) {
        ++q;
        r -= d;
    }
    rem = r;
    return q;
}

// Unit index -> coordinates (the unit count fits in 30 bits; checked on the host).
__device__ __forceinline__ Unit decode_unit(const PrefillArgs &a, uint32_t u)
{
    Unit r;
    uint32_t rem;
    // Order: head quad fastest, then query block (long rows first), then KV head, then batch entry:
    // the CTAs work on one KV head at a time, whose K and V (67 MB at 128K tokens) stay in L2.
    u = divmod(u, (uint32_t)a.nsub, a.inv_nsub, rem);
    r.sub = (int32_t)rem;
    u = divmod(u, (uint32_t)a.nqb, a.inv_nqb, rem);
    r.i = a.nqb - 1 - (int32_t)rem;  // long rows first
    r.b = (int32_t)divmod(u, (uint32_t)a.Hkv, a.inv_Hkv, rem);
    r.hk = (int32_t)rem;
    r.rs = __ldg(a.row_ptr + r.i);
    r.n = __ldg(a.row_ptr + r.i + 1) - r.rs;
    if (a.cu_seqlens) {
        r.bt = 0;
        r.tok0 = __ldg(a.cu_seqlens + r.b);
        r.len = __ldg(a.cu_seqlens + r.b + 1) - r.tok0;
        if ((int64_t)r.i * kBlk >= r.len) r.n = 0;  // the sequence ends before this query block: nothing to do
    } else {
        r.bt = r.b;
        r.tok0 = 0;
        r.len = (int32_t)a.N;
    }
    return r;
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
prefill_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
               const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
               const PrefillArgs a)
{
    using SM = SmemMap<D>;
    constexpr int DH = D / 64;  // 64-feature (128-byte) sub-tiles per row
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    const uint32_t bars = smem_base + SM::kBars;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + SM::kBars + BAR_COUNT * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + SM::kBars + BAR_COUNT * 8 + 8);
    auto bar = [&](uint32_t idx) { return bars + idx * 8u; };
    // Every barrier wait is bounded by the launch's cycle limit.
    auto wait_bar = [&](uint32_t b_, uint32_t parity, volatile int *flag, int32_t *status, int code) {
        return ptx::mbar_wait_bounded(b_, parity, flag, status, code, a.wait_cycles, (int)PA_ERR_TIMEOUT);
    };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(bar(BAR_Q_FULL + s), 1);
            ptx::mbar_init(bar(BAR_Q_EMPTY + s), 2);  // (the "empty" barriers: one commit per issuing warp)
        }
        for (int s = 0; s < kKStages; ++s) {
            ptx::mbar_init(bar(BAR_K_FULL + s), 1);
            ptx::mbar_init(bar(BAR_K_EMPTY + s), 2);
        }
        for (int s = 0; s < kVStages; ++s) {
            ptx::mbar_init(bar(BAR_V_FULL + s), 1);
            ptx::mbar_init(bar(BAR_V_EMPTY + s), 2);
        }
        for (int s = 0; s < 4; ++s) ptx::mbar_init(bar(BAR_O_DONE + s), 1);
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(bar(BAR_S_FULL + s), 1);
            ptx::mbar_init(bar(BAR_S_TAKEN + s), 4);  // one arrival per softmax warp of the slot
            ptx::mbar_init(bar(BAR_P_FULL + 2 * s), 4);
            ptx::mbar_init(bar(BAR_P_FULL + 2 * s + 1), 4);
            ptx::mbar_init(bar(BAR_O_FINAL + s), 1);
            ptx::mbar_init(bar(BAR_ML_READY + s), 4);
            ptx::mbar_init(bar(BAR_O_FREE + s), 4);
        }
        ptx::mbar_init(bar(BAR_STAGE_FREE), 1);
        ptx::mbar_init(bar(BAR_STAGE_FREE + 1), 1);
        ptx::mbar_init(bar(BAR_STAGE_FULL), 4);
        ptx::mbar_init(bar(BAR_TURN), 4);
        ptx::mbar_init(bar(BAR_TURN + 1), 4);
        *abort_flag = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async_smem();
    }
    if (warp == 2) {
        ptx::tmem_alloc(ptx::smem_u32(tmem_slot), kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base_any = *tmem_slot;
    const uint32_t tmem_base = tmem_base_any;

    if (warp < 4) ptx::setmaxnreg_dec<PA_REG_CTRL>();
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            ptx::prefetch_tensormap(&tmQ);
            ptx::prefetch_tensormap(&tmK);
            ptx::prefetch_tensormap(&tmV);
            uint32_t kc = 0, ul = 0;  // key blocks and units issued so far by this CTA
            bool ok = true;
            // A unit's coordinates and its first block index are fetched while the previous unit's
            // loads are still waiting for ring space, the other block indices one block ahead.
            auto next_unit = [&](uint32_t u, Unit &w, int32_t &j0) {
                for (; u < (uint32_t)a.n_units; u += gridDim.x) {
                    w = decode_unit(a, u);
                    if (w.n > 0) {
                        j0 = __ldg(a.col_idx + w.rs);
                        break;
                    }
                }
                return u;
            };
            // Q tiles of unit number ul_q go to Q buffer ul_q & 1 once the unit two before has
            // issued its last S and its output, staged in that buffer, has left.  (Both barriers
            // complete once per two units; this thread's own wait two units ago keeps them
            // within one phase of the parity asked for.)
            auto q_buffer_free = [&](uint32_t ul_q) {
                return ul_q < 2 || ptx::mbar_test_wait(bar(BAR_STAGE_FREE + (ul_q & 1)), ((ul_q >> 1) - 1) & 1);
            };
            auto load_q = [&](const Unit &w, uint32_t ul_q) {
                const uint32_t qb = ul_q & 1;
                if (ul_q >= 2 && !wait_bar(bar(BAR_Q_EMPTY + qb), ((ul_q >> 1) - 1) & 1, abort_flag, a.status, 1)) return false;
                if (ul_q >= 2 && !wait_bar(bar(BAR_STAGE_FREE + qb), ((ul_q >> 1) - 1) & 1, abort_flag, a.status, 16)) return false;
                ptx::mbar_expect_tx(bar(BAR_Q_FULL + qb), SM::kQBuf);
                for (int s = 0; s < 2; ++s)
                    for (int dh = 0; dh < DH; ++dh)
                        ptx::tma_load_4d(smem_base + SM::kQ + qb * SM::kQBuf + s * SM::kQSlot + dh * SM::kQSub, &tmQ,
                                         bar(BAR_Q_FULL + qb), dh * 64, w.tok0 + w.i * kBlk,
                                         w.hk * a.G + w.sub * 4 + 2 * s, w.bt);
                return true;
            };
            Unit w, wn;
            int32_t j = 0, jnext = 0;
            uint32_t u = next_unit(blockIdx.x, w, j);
            if (u < (uint32_t)a.n_units) ok = load_q(w, 0);
            while (u < (uint32_t)a.n_units && ok) {
                const uint32_t un = next_unit(u + gridDim.x, wn, jnext);
                bool q_pending = un < (uint32_t)a.n_units;  // the next unit's Q tiles are still to be requested
                for (int t = 0; t < w.n; ++t, ++kc) {
                    const int32_t jn = t + 1 < w.n ? __ldg(a.col_idx + w.rs + t + 1) : 0;
                    const uint32_t ks = kc % kKStages, vs = kc % kVStages;
                    if (kc >= (uint32_t)kKStages) {
                        ok = wait_bar(bar(BAR_K_EMPTY + ks), (kc / kKStages - 1) & 1, abort_flag, a.status, 2);
                        if (!ok) break;
                    }
                    ptx::mbar_expect_tx(bar(BAR_K_FULL + ks), SM::kBlkTile);
                    for (int dh = 0; dh < DH; ++dh)
                        ptx::tma_load_4d(smem_base + SM::kK + ks * SM::kBlkTile + dh * SM::kBlkSub, &tmK,
                                         bar(BAR_K_FULL + ks), dh * 64, w.tok0 + j * kBlk, w.hk, w.bt);
                    if (kc >= (uint32_t)kVStages) {
                        ok = wait_bar(bar(BAR_V_EMPTY + vs), (kc / kVStages - 1) & 1, abort_flag, a.status, 3);
                        if (!ok) break;
                    }
                    ptx::mbar_expect_tx(bar(BAR_V_FULL + vs), SM::kBlkTile);
                    for (int dh = 0; dh < DH; ++dh)
                        ptx::tma_load_4d(smem_base + SM::kV + vs * SM::kBlkTile + dh * SM::kBlkSub, &tmV,
                                         bar(BAR_V_FULL + vs), dh * 64, w.tok0 + j * kBlk, w.hk, w.bt);
                    j = jn;
                    // The next unit's Q goes where the unit before this one kept its Q and then
                    // staged its output, which leaves during this unit's first steps: the request
                    // is made behind the first block (from the second on) that finds the buffer
                    // free, so the key blocks are not held up, and behind the last one at the latest.
                    if (q_pending && (t + 1 == w.n || (t >= 1 && q_buffer_free(ul + 1)))) {
                        ok = load_q(wn, ul + 1);
                        q_pending = false;
                        if (!ok) break;
                    }
                }
                ++ul;
                u = un;
                w = wn;
                j = jnext;
            }
        }
        __syncwarp();
    } else if (warp == 1 || warp == 3) {
        // ------------------------------------------------------------------ tcgen05 issuers
        // One issuing warp per slot (warp 1: slot 0, warp 3: slot 1): a step's waits and MMA
        // issue cost the issuing warp about a thousand cycles per slot, and one warp serving both
        // slots in turn was the longest chain of the step.  The two warps share nothing but the
        // operand tiles: a commit covers the MMAs of the committing thread only, so the barriers
        // that free a K, V or Q tile count one arrival from each.
        // The whole warp runs the (uniform) control flow and the barrier waits; one elected lane
        // issues the MMAs and commits.  Steps are numbered through the CTA's whole run (c), so ring
        // positions and buffer parities do not care about unit boundaries.  Per step c:
        //   S(c + 1) = Q K^T is issued as soon as the softmax warps have taken S(c) out of tensor
        //   memory (S has one buffer per slot; P has its own two), i.e. while they still work on
        //   step c, and it may belong to the next unit;
        //   O += P(c) V(c) is issued when P(c) has been handed over.
        // Descriptors: the high word is constant per operand kind (stride 1024 B between 8-row
        // groups, version 1, 128-byte swizzle); the low word holds the start address >> 4 (plus
        // the leading-dimension offset for the MN-major V operand).
        {
            const bool leader = ptx::elect_one();
            const int s = __shfl_sync(0xffffffffu, warp >> 1, 0);  // this warp's slot
            // Every lane holds the same values; the shuffles tell the compiler so, which lets the
            // loop bounds, ring positions and descriptors live in uniform registers.
            const uint32_t tmem_base = __shfl_sync(0xffffffffu, tmem_base_any, 0);
            constexpr uint32_t idesc_qk = ptx::idesc_bf16_f32(128, 64, 0);
            constexpr uint32_t idesc_pv = ptx::idesc_bf16_f32(128, D, 1);
            constexpr uint32_t desc_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
            const uint32_t q_lo = ((smem_base + SM::kQ) >> 4) | (1u << 16);  // + unit parity, slot
            const uint32_t k_lo = ((smem_base + SM::kK) >> 4) | (1u << 16);
            const uint32_t v_lo = ((smem_base + SM::kV) >> 4) | ((SM::kBlkSub >> 4) << 16);
            // S = Q K^T: A = Q tile (K-major), B = K block (K-major), 16 features per MMA.
            auto issue_qk = [&](uint32_t qb, uint32_t ks) {
                const uint32_t qa = q_lo + qb * (SM::kQBuf >> 4) + s * (SM::kQSlot >> 4);
                const uint32_t kb = k_lo + ks * (SM::kBlkTile >> 4);
                const uint32_t dst = tmem_base + s * 128;
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk)
                    ptx::umma_ss_lohi(dst, qa + (((kk / 4) * SM::kQSub + (kk % 4) * 32) >> 4), desc_hi,
                                      kb + (((kk / 4) * SM::kBlkSub + (kk % 4) * 32) >> 4), desc_hi, idesc_qk,
                                      kk > 0 ? 1u : 0u);
            };
            // O (+)= P V: A = P (tensor memory, bf16 pairs, buffer = step parity), B = V block
            // (MN-major: features contiguous), 16 keys per MMA.
            auto issue_pv = [&](uint32_t buf, uint32_t vs, bool acc) {
                const uint32_t vb = v_lo + vs * (SM::kBlkTile >> 4);
                const uint32_t dst = tmem_base + 256 + s * D;
                const uint32_t pa_ = tmem_base + s * 128 + 64 + buf * 32;
#pragma unroll
                for (int kk = 0; kk < kBlk / 16; ++kk)
                    ptx::umma_ts_lohi(dst, pa_ + kk * 8, vb + ((kk * 2048) >> 4), desc_hi, idesc_pv,
                                      (acc || kk > 0) ? 1u : 0u);
            };
            auto unit_blocks = [&](uint32_t u) {
                return __shfl_sync(0xffffffffu, u < (uint32_t)a.n_units ? decode_unit(a, u).n : 0, 0);
            };
            // Next non-empty unit after u.  Its block count `n` is already loaded (`ahead`); the
            // count after that is requested now, so no unit boundary waits for a load.
            auto next_unit = [&](uint32_t u, int &n, int &ahead) {
                do {
                    u += gridDim.x;
                    n = ahead;
                    ahead = unit_blocks(u + gridDim.x);
                } while (u < (uint32_t)a.n_units && n <= 0);
                return u;
            };
            bool ok = true;
            // S(c1) of this slot; `first` / `final`: c1 is the first / last step of unit number ul1.
            auto qk_step = [&](uint32_t c1, uint32_t ul1, bool first, bool final, bool wait_taken) {
                if (first) ok = __all_sync(0xffffffffu, wait_bar(bar(BAR_Q_FULL + (ul1 & 1)), (ul1 >> 1) & 1, abort_flag, a.status, 4));
                if (ok)
                    ok = __all_sync(0xffffffffu, wait_bar(bar(BAR_K_FULL + c1 % kKStages), (c1 / kKStages) & 1,
                                                          abort_flag, a.status, 5));
                if (ok && wait_taken)
                    ok = __all_sync(0xffffffffu, wait_bar(bar(BAR_S_TAKEN + s), (c1 - 1) & 1, abort_flag, a.status, 8));
                if (!ok) return;
                ptx::tc_fence_after_sync();
                if (leader) {
                    issue_qk(ul1 & 1, c1 % kKStages);
                    ptx::umma_commit(bar(BAR_S_FULL + s));
                    ptx::umma_commit(bar(BAR_K_EMPTY + c1 % kKStages));
                    if (final) ptx::umma_commit(bar(BAR_Q_EMPTY + (ul1 & 1)));
                }
                __syncwarp();
            };
            // O (+)= P(c) V(c) of this slot; t = step inside its unit (number ul) of n steps.
            auto pv_step = [&](uint32_t c, uint32_t ul, int t, int n) {
                ok = __all_sync(0xffffffffu, wait_bar(bar(BAR_V_FULL + c % kVStages), (c / kVStages) & 1,
                                                      abort_flag, a.status, 6));
                if (ok)
                    ok = __all_sync(0xffffffffu, wait_bar(bar(BAR_P_FULL + 2 * s + (c & 1)), (c >> 1) & 1, abort_flag, a.status, 7));
                // The previous unit's O must have left tensor memory.
                if (ok && t == 0 && ul > 0)
                    ok = __all_sync(0xffffffffu, wait_bar(bar(BAR_O_FREE + s), (ul - 1) & 1, abort_flag, a.status, 14));
                if (!ok) return;
                ptx::tc_fence_after_sync();
                if (leader) {
                    issue_pv(c & 1, c % kVStages, t > 0);
                    ptx::umma_commit(bar(BAR_O_DONE + 2 * s + (c & 1)));
                    if (t + 1 == n) ptx::umma_commit(bar(BAR_O_FINAL + s));
                    ptx::umma_commit(bar(BAR_V_EMPTY + c % kVStages));
                }
                __syncwarp();
            };
            uint32_t kc = 0, ul = 0;
            int n = 0, nn = 0;  // key blocks of this unit and of the next
            int ahead = unit_blocks(blockIdx.x);
            uint32_t u = next_unit(blockIdx.x - gridDim.x, n, ahead);  // (the sum wraps back to blockIdx.x)
            if (u < (uint32_t)a.n_units) qk_step(0, 0, true, n == 1, false);
            while (u < (uint32_t)a.n_units && ok) {
                const uint32_t un = next_unit(u, nn, ahead);
                const bool has_next = un < (uint32_t)a.n_units;
                for (int t = 0; t < n && ok; ++t) {
                    const uint32_t c = kc + t;
                    if (t + 1 < n) {
                        qk_step(c + 1, ul, false, t + 2 == n, true);
                        if (ok) pv_step(c, ul, t, n);
                    } else {
                        // Unit boundary: the next unit's first S goes first if its Q tile has
                        // arrived (normally long ago), else behind this unit's last P V, for which
                        // the epilogue waits.
                        const bool q_here = has_next && __all_sync(0xffffffffu, ptx::mbar_test_wait(bar(BAR_Q_FULL + ((ul + 1) & 1)), ((ul + 1) >> 1) & 1));
                        if (q_here) qk_step(c + 1, ul + 1, true, nn == 1, true);
                        if (ok) pv_step(c, ul, t, n);
                        if (ok && has_next && !q_here) qk_step(c + 1, ul + 1, true, nn == 1, true);
                    }
                }
                kc += n;
                ++ul;
                u = un;
                n = nn;
            }
        }
        __syncwarp();
    } else if (warp >= 4 && warp < 12) {
        // ------------------------------------------------------------------ online softmax
        ptx::setmaxnreg_inc<PA_REG_SOFT>();
        const int s = (warp - 4) >> 2;          // slot
        const int quad = warp & 3;              // TMEM lane quadrant this warp may access
        const int row = quad * 32 + lane;       // tile row = TMEM lane
        const int qrow = row & 63;              // token inside the query block
        const uint32_t t_s0 = tmem_base + ((uint32_t)(quad * 32) << 16) + s * 128;
        const uint32_t t_o = tmem_base + ((uint32_t)(quad * 32) << 16) + 256 + s * D;
        const float sl2 = a.scale_log2;
        const uint64_t sl2_2 = ptx::pack_f32x2(sl2, sl2);
        uint32_t kc = 0, ul = 0;
        bool ok = true;
        // Unit metadata runs ahead of its use so that no load sits between two units: the row
        // extent two units ahead, the row's last block index (needs the extent) one unit ahead.
        auto fetch_unit = [&](uint32_t u) {
            Unit r = {};
            if (u < (uint32_t)a.n_units) r = decode_unit(a, u);
            return r;
        };
        auto fetch_lastcol = [&](const Unit &r) { return r.n > 0 ? __ldg(a.col_idx + r.rs + r.n - 1) : -1; };
        Unit w_next = fetch_unit(blockIdx.x);
        Unit w_next2 = fetch_unit(blockIdx.x + gridDim.x);
        int32_t lastcol_next = fetch_lastcol(w_next);
        // Called once per unit, after the first step's hand-over (the issuer is busy with it then),
        // not between two units where the next logits are already waiting.
        auto advance_metadata = [&](uint32_t u) {
            w_next = w_next2;
            lastcol_next = fetch_lastcol(w_next);
            w_next2 = fetch_unit(u + 2 * gridDim.x);
        };
        for (uint32_t u = blockIdx.x; u < (uint32_t)a.n_units && ok; u += gridDim.x) {
            const Unit w = w_next;
            const int32_t lastcol = lastcol_next;
            const int head_local = w.sub * 4 + 2 * s + (row >> 6);
            const int head = w.hk * a.G + head_local;
            const int64_t tok = (int64_t)w.i * kBlk + qrow;
            const bool valid = head_local < a.G && tok < w.len;
            // Algorithm 1's causal term acts inside the diagonal pair (col == row) only; rows end
            // with that block.
            const bool last_is_diag = w.n > 0 && lastcol == w.i;
            float m = -INFINITY, l = 0.f;
            uint32_t sr[64];
            for (int t = 0; t < w.n; ++t, ++kc) {
                ok = wait_bar(bar(BAR_S_FULL + s), kc & 1, abort_flag, a.status, 9);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                ptx::tmem_ld32(t_s0, *reinterpret_cast<uint32_t(*)[32]>(&sr[0]));
                ptx::tmem_ld32(t_s0 + 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[32]));
                ptx::tmem_wait_ld();
                // S is in registers: its buffer may take the next step's logits.
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(bar(BAR_S_TAKEN + s));
                if (last_is_diag && t == w.n - 1) {
                    // Keys after the query's own token are masked (-inf).  A warp's 32 rows are
                    // tokens 0..31 or 32..63 of the block, so half of the columns need no compare:
                    // for the first half of the rows columns 32..63 are masked for every row, for
                    // the second half columns 0..32 for none.
                    if ((quad & 1) == 0) {
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c > lane) sr[c] = 0xff800000u;
#pragma unroll
                        for (int c = 32; c < 64; ++c) sr[c] = 0xff800000u;
                    } else {
#pragma unroll
                        for (int c = 33; c < 64; ++c)
                            if (c - 32 > lane) sr[c] = 0xff800000u;
                    }
                }
                // Fast path: p = exp2(s * scale - m) against the reference maximum m carried from
                // earlier steps (lazy rescaling: O / l at the end is exact whatever reference was
                // used, as long as nothing overflows).  Two-wide fp32 arithmetic.  The watch is the
                // step's row sum, which is needed anyway: it bounds every p of the row from above,
                // so a sum within the limit means no p came near the fp32 / bf16 range, and an
                // overflow shows up as inf.
                if (t == 0) {
                    // A unit's first step: the reference is the exact row maximum of this block
                    // (l and O are still empty, so nothing has to be rescaled), then the common pass.
                    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int c = 0; c < 64; c += 4) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) mx4[e] = fmaxf(mx4[e], __uint_as_float(sr[c + e]));
                    }
                    m = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * sl2;
                }
                const uint64_t negm_2 = ptx::pack_f32x2(-m, -m);
                uint64_t sum2[2] = {0ull, 0ull};
                uint32_t pk[32];
                // The two slots take turns at the exponentials: slot 0's pass of step kc, then slot
                // 1's, then slot 0's of step kc + 1, ...  A pass that has the exponential unit to
                // itself takes half as long, and the rest of a slot's step (loads from and stores to
                // tensor memory, barrier traffic) then runs beside the other slot's pass instead
                // of beside its own idle time.  (Turn barrier s completes once per pass of the
                // other slot, which cannot start its next pass before this slot's, so the parity
                // asked for is never more than one phase behind.)
                if (s == 1 || kc > 0) {
                    ok = wait_bar(bar(BAR_TURN + s), (kc - 1 + s) & 1, abort_flag, a.status, 18);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                }
                {
#pragma unroll
                for (int c = 0; c < 64; c += 4) {
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const uint64_t y2 = ptx::fma_f32x2(
                            ptx::pack_f32x2(__uint_as_float(sr[c + 2 * e]), __uint_as_float(sr[c + 2 * e + 1])), sl2_2,
                            negm_2);
                        float y0, y1;
                        ptx::unpack_f32x2(y2, y0, y1);
                        const float p0 = ptx::ex2(y0), p1 = ptx::ex2(y1);
                        sum2[e] = ptx::add_f32x2(sum2[e], ptx::pack_f32x2(p0, p1));
                        pk[(c >> 1) + e] = ptx::cvt_bf16x2(p0, p1);
                    }
                    // The turn is passed on a quarter of the way into the pass: the other slot needs
                    // some 350 cycles to see it (measured), which then run beside the rest of this pass.
                    if (c == kTurnAtColumn && lane == 0) ptx::mbar_arrive(bar(BAR_TURN + (s ^ 1)));
                }
                }
                float sum;
                {
                    float s0, s1, s2, s3;
                    ptx::unpack_f32x2(sum2[0], s0, s1);
                    ptx::unpack_f32x2(sum2[1], s2, s3);
                    sum = (s0 + s1) + (s2 + s3);
                }
                // !(x <= limit) also catches inf and NaN.
                const bool suspect = !(sum <= kSumLimit);
                if (__any_sync(0xffffffffu, suspect)) {
                    // Rare path: exact row maximum, new reference for the rows that need it, what
                    // was accumulated so far brought to the new reference, P recomputed from the
                    // logits still in registers.
                    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int c = 0; c < 64; c += 4) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) mx4[e] = fmaxf(mx4[e], __uint_as_float(sr[c + e]));
                    }
                    const float mx2 = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * sl2;
                    const bool grow = t == 0 || mx2 > m + kRescaleThreshold;
                    const float m_new = grow ? mx2 : m;
                    const float alpha = grow ? ptx::ex2(m - m_new) : 1.0f;  // (l and O are still empty on a first step)
                    l *= alpha;
                    m = m_new;
                    if (t > 0) {
                        // O may be rescaled only once the previous step's P V has completed.  (The
                        // completion barriers alternate by step parity; the S waited for above was issued
                        // after the P V of step kc - 2, so a barrier is never more than one phase behind.)
                        ok = wait_bar(bar(BAR_O_DONE + 2 * s + ((kc - 1) & 1)), ((kc - 1) >> 1) & 1, abort_flag, a.status, 11);
                        ok = __all_sync(0xffffffffu, ok);
                        if (!ok) break;
                        ptx::tc_fence_after_sync();
#pragma unroll 1
                        for (int ch = 0; ch < D / 32; ++ch) {
                            uint32_t orr[32];
                            ptx::tmem_ld32(t_o + ch * 32, orr);
                            ptx::tmem_wait_ld();
#pragma unroll
                            for (int c = 0; c < 32; ++c) orr[c] = __float_as_uint(__uint_as_float(orr[c]) * alpha);
                            ptx::tmem_st32(t_o + ch * 32, orr);
                        }
                    }
                    float sum4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int c = 0; c < 64; c += 4) {
                        float pv[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            pv[e] = ptx::ex2(fmaf(__uint_as_float(sr[c + e]), sl2, -m));
                            sum4[e] += pv[e];
                        }
                        pk[c >> 1] = ptx::cvt_bf16x2(pv[0], pv[1]);
                        pk[(c >> 1) + 1] = ptx::cvt_bf16x2(pv[2], pv[3]);
                    }
                    sum = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
                }
                l += sum;
                // P has two buffers (step parity).  The P V that read this one two steps ago has
                // completed: this slot's issuing thread issued it before the S of this step, whose
                // completion (which covers everything that thread issued earlier) was waited for above.
                ptx::tmem_st32(t_s0 + 64 + (kc & 1) * 32, pk);
                // (The hand-over barriers alternate by step parity like the P buffers: the S of step
                // kc + 2 is issued behind the P V of step kc, so a barrier is never more than one
                // phase ahead of the issuer, whose parity wait could not tell two from none.)
                ptx::tmem_wait_st();
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(bar(BAR_P_FULL + 2 * s + (kc & 1)));
                if (t == 0) advance_metadata(u);
                if (t + 1 == w.n) {
                    // Softmax denominators for the epilogue warps (they finish O / l).  The previous
                    // unit's must have been read: that also keeps this slot's statistics barrier at
                    // most one phase ahead of the epilogue.
                    // (With three or more steps the wait is implied: this step's S was issued
                    // behind the unit's first P V, which itself waited for that read.)
                    if (ul > 0 && w.n < 3) {
                        ok = wait_bar(bar(BAR_O_FREE + s), (ul - 1) & 1, abort_flag, a.status, 13);
                        ok = __all_sync(0xffffffffu, ok);
                        if (!ok) break;
                    }
                    reinterpret_cast<float *>(smem + SM::kStats)[s * 128 + row] = l;
                    __threadfence_block();
                    // LSE = ln sum exp(s) = (m + log2 l) ln 2.
                    if (valid) a.lse[w.b * a.lse_sb + head * a.lse_sh + w.tok0 + tok] = (m + log2f(l)) * 0.6931471805599453f;
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(bar(BAR_ML_READY + s));
                }
            }
            if (w.n > 0) ++ul;
            else advance_metadata(u);
        }
    } else if (warp >= 12) {
        // ------------------------------------------------------------------ epilogue
        // O / l for both slots, off the softmax warps' critical path.  O is read out of tensor
        // memory (which frees it for the next unit); bf16 output is staged in shared memory in
        // the 128-byte-swizzled box layout and leaves as bulk tensor stores, one per head and
        // 64-feature half (rows beyond the sequence end are clipped by the tensor map), fp32
        // output is written from registers.
        ptx::setmaxnreg_dec<PA_REG_EPI>();
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        const int qrow = row & 63;
        const bool store_thread = threadIdx.x == 12 * 32;
        uint32_t ul = 0, ns = 0;  // units and staged slots so far
        bool ok = true;
        for (uint32_t u = blockIdx.x; u < (uint32_t)a.n_units && ok; u += gridDim.x) {
            const Unit w = decode_unit(a, u);
            const int64_t tok = (int64_t)w.i * kBlk + qrow;
            // The unit's Q buffer is no longer read once its last P V has completed (every S of
            // the unit was issued before it); its output is staged there.
            const uint32_t stage = smem_base + SM::kQ + (ul & 1) * SM::kQBuf;
#pragma unroll 1
            for (int s = 0; s < 2; ++s) {
                const int head_local = w.sub * 4 + 2 * s + (row >> 6);
                const int head = w.hk * a.G + head_local;
                const bool valid = head_local < a.G && tok < w.len;
                const int64_t obase = w.bt * a.o_sb + (w.tok0 + tok) * a.o_ss + (int64_t)head * a.o_sh;
                if (w.n <= 0) {  // empty row: defined outputs, no barrier traffic
                    if (valid) {
                        for (int c = 0; c < D; ++c) {
                            if (a.o_is_f32) reinterpret_cast<float *>(a.o)[obase + c] = 0.f;
                            else reinterpret_cast<__nv_bfloat16 *>(a.o)[obase + c] = __float2bfloat16_rn(0.f);
                        }
                        a.lse[w.b * a.lse_sb + head * a.lse_sh + w.tok0 + tok] = -INFINITY;
                    }
                    continue;
                }
                ok = wait_bar(bar(BAR_ML_READY + s), ul & 1, abort_flag, a.status, 15);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const float inv = 1.0f / reinterpret_cast<const float *>(smem + SM::kStats)[s * 128 + row];
                ok = wait_bar(bar(BAR_O_FINAL + s), ul & 1, abort_flag, a.status, 10);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t t_o = tmem_base + ((uint32_t)(quad * 32) << 16) + 256 + s * D;
                if (a.o_is_f32) {
#pragma unroll
                    for (int ch = 0; ch < D / 32; ++ch) {
                        uint32_t orr[32];
                        ptx::tmem_ld32(t_o + ch * 32, orr);
                        ptx::tmem_wait_ld();
                        if (ch == D / 32 - 1) {
                            ptx::tc_fence_before_sync();
                            __syncwarp();
                            if (lane == 0) ptx::mbar_arrive(bar(BAR_O_FREE + s));
                        }
                        if (valid) {
                            float4 *dst = reinterpret_cast<float4 *>(reinterpret_cast<float *>(a.o) + obase + ch * 32);
#pragma unroll
                            for (int c = 0; c < 8; ++c)
                                dst[c] = make_float4(__uint_as_float(orr[4 * c]) * inv, __uint_as_float(orr[4 * c + 1]) * inv,
                                                     __uint_as_float(orr[4 * c + 2]) * inv, __uint_as_float(orr[4 * c + 3]) * inv);
                        }
                    }
                } else {
                    // Head 2 s + (row >> 6) of the unit: two boxes of 64 tokens x 128 bytes (one per
                    // 64-feature half); 16-byte chunk j of token t sits at chunk position j ^ (t & 7).
                    const uint32_t rbase = stage + (uint32_t)(2 * s + (row >> 6)) * SM::kOHead + (uint32_t)qrow * 128u;
                    // A packed sequence's last block may reach into the next sequence's rows, which a
                    // box store would overwrite: its rows are written one by one from the registers.
                    const bool ragged = a.cu_seqlens != nullptr && (int64_t)(w.i + 1) * kBlk > w.len;
#pragma unroll
                    for (int ch = 0; ch < D / 32; ++ch) {
                        uint32_t orr[32];
                        ptx::tmem_ld32(t_o + ch * 32, orr);
                        ptx::tmem_wait_ld();
                        if (ch == D / 32 - 1) {
                            // O is in registers: tensor memory may take the next unit's first P V.
                            ptx::tc_fence_before_sync();
                            __syncwarp();
                            if (lane == 0) ptx::mbar_arrive(bar(BAR_O_FREE + s));
                        }
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const int c = 4 * ch + k;  // 16-byte chunk of the row
                            uint32_t pk[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                pk[e] = ptx::cvt_bf16x2(__uint_as_float(orr[8 * k + 2 * e]) * inv,
                                                        __uint_as_float(orr[8 * k + 2 * e + 1]) * inv);
                            const uint32_t dst = rbase + (uint32_t)(c >> 3) * 8192u + ((uint32_t)((c & 7) ^ (qrow & 7)) << 4);
                            ptx::st_shared_v4(dst, pk[0], pk[1], pk[2], pk[3]);
                            if (ragged && valid)
                                *reinterpret_cast<uint4 *>(reinterpret_cast<__nv_bfloat16 *>(a.o) + obase + 8 * c) =
                                    make_uint4(pk[0], pk[1], pk[2], pk[3]);
                        }
                    }
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(bar(BAR_STAGE_FULL));
                    // All four warps wait (not only the storing one), so none can arrive for the
                    // next slot before this phase has completed.
                    ok = wait_bar(bar(BAR_STAGE_FULL), ns & 1, abort_flag, a.status, 17);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    ++ns;
                    if (store_thread) {
                        for (int hh = 0; hh < 2; ++hh) {
                            const int hl = w.sub * 4 + 2 * s + hh;
                            if (hl >= a.G || ragged) continue;  // the padding head of an odd group; rows already written
                            for (int dh = 0; dh < DH; ++dh)
                                ptx::tma_store_4d(&tmO, stage + (uint32_t)(2 * s + hh) * SM::kOHead + (uint32_t)dh * 8192u,
                                                  dh * 64, w.tok0 + w.i * kBlk, w.hk * a.G + hl, w.bt);
                        }
                        ptx::bulk_commit_group();
                    }
                }
            }
            if (w.n > 0 && ok) {
                // The Q buffer may be loaded again once the bulk stores have read it.
                if (store_thread) {
                    ptx::bulk_wait_read_all();
                    ptx::mbar_arrive(bar(BAR_STAGE_FREE + (ul & 1)));
                }
                ++ul;
            }
        }
        if (store_thread) ptx::bulk_wait_all();
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 2) {
        // Every role has left its loop.  After a wait that gave up, copies and tensor-core
        // operations issued before it may still be in flight: they finish by themselves within
        // microseconds (nothing they need is withheld), and the warp that owns the tensor memory
        // lets a bounded two milliseconds pass before it gives the memory back and the CTA's
        // shared memory can go to another kernel.
        if (*abort_flag) {
            const long long t0 = clock64();
            while (clock64() - t0 < 4000000ll) {
            }
        }
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ---------------------------------------------------------------------------------- host side

static pa_status check_strides(const pa_strides &s, int D, const char *what)
{
    if (s.seq < D || s.head < D || s.batch < 0)
        return fail(PA_ERR_SHAPE, "%s strides must be >= head_dim", what);
    if ((s.seq % 8) || (s.head % 8) || (s.batch % 8))
        return fail(PA_ERR_ALIGNMENT, "%s strides must be multiples of 8 elements (16 bytes)", what);
    if (s.seq >= ((int64_t)1 << 38) || s.head >= ((int64_t)1 << 38) || s.batch >= ((int64_t)1 << 38))
        return fail(PA_ERR_SHAPE, "%s strides too large for a tensor map", what);
    return PA_OK;
}

static pa_status check_prefill(const pa_prefill_params *p)
{
    if (!p) return fail(PA_ERR_INVALID_ARG, "params must be non-null");
    if (p->batch < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1 || p->seq_len < 1)
        return fail(PA_ERR_INVALID_ARG, "batch, head counts and seq_len must be positive");
    if (p->o_dtype != PA_BF16 && p->o_dtype != PA_F32) return fail(PA_ERR_INVALID_ARG, "bad o_dtype");
    if (!(p->softmax_scale >= 0.f) || isinf(p->softmax_scale))
        return fail(PA_ERR_INVALID_ARG, "softmax_scale must be finite and >= 0 (0 = default)");
    if (p->head_dim != 64 && p->head_dim != 128) return fail(PA_ERR_SHAPE, "head_dim must be 64 or 128");
    if (p->block != kBlk) return fail(PA_ERR_SHAPE, "block must be 64");
    if (p->n_q_heads % p->n_kv_heads) return fail(PA_ERR_SHAPE, "n_q_heads must be a multiple of n_kv_heads");
    if (p->n_q_heads < 2) return fail(PA_ERR_SHAPE, "n_q_heads must be >= 2");
    if (p->seq_len > ((int64_t)1 << 30)) return fail(PA_ERR_SHAPE, "seq_len too large");
    if (pa_status s = check_strides(p->q, p->head_dim, "q")) return s;
    if (pa_status s = check_strides(p->k, p->head_dim, "k")) return s;
    if (pa_status s = check_strides(p->v, p->head_dim, "v")) return s;
    if (pa_status s = check_strides(p->o, p->head_dim, "o")) return s;
    return PA_OK;
}

constexpr size_t kPrefillWorkspace = 256;

// Optional check of a caller's CSR (PA_VALIDATE=1): one thread per row.  The first violation
// found is recorded as (kind, row) in check[0..1]: 1 row_ptr does not start at 0 / end at nnz,
// 2 row extent negative or beyond nnz, 3 block index outside [0, row], 4 indices not ascending.
__global__ void validate_csr_kernel(const int32_t *row_ptr, const int32_t *col_idx, int32_t nqb, int64_t nnz,
                                    int32_t *check)
{
    const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= nqb) return;
    int kind = 0;
    const int32_t lo = row_ptr[i], hi = row_ptr[i + 1];
    if ((i == 0 && lo != 0) || (i == nqb - 1 && (int64_t)hi != nnz)) kind = 1;
    else if (lo < 0 || hi < lo || (int64_t)hi > nnz) kind = 2;
    else {
        int32_t prev = -1;
        for (int32_t e = lo; e < hi && kind == 0; ++e) {
            const int32_t j = col_idx[e];
            if (j < 0 || j > i) kind = 3;
            else if (j <= prev) kind = 4;
            prev = j;
        }
    }
    if (kind != 0 && atomicCAS(check, 0, kind) == 0) check[1] = i;
}

}  // namespace pa

extern "C" size_t pa_prefill_workspace_bytes(const pa_prefill_params *p)
{
    (void)p;
    return pa::kPrefillWorkspace;
}

namespace pa {

// The launch behind pa_prefill (cu_seqlens null) and pa_prefill_varlen (packed sequences:
// p->seq_len is the longest one, tokens run over [0, total_tokens)).
static pa_status launch_prefill(const pa_prefill_params *p, const void *q, const void *k, const void *v,
                                const int32_t *cu_seqlens, int64_t total_tokens, const int32_t *row_ptr,
                                const int32_t *col_idx, int64_t nnz, void *o, float *lse, void *workspace,
                                size_t workspace_bytes, void *stream)
{
    if (pa_status s = check_prefill(p)) return s;
    const bool varlen = cu_seqlens != nullptr;
    if (varlen && (total_tokens < 1 || total_tokens > ((int64_t)1 << 30)))
        return fail(PA_ERR_INVALID_ARG, "total_tokens must be in [1, 2^30]");
    if (!q || !k || !v || !row_ptr || !col_idx || !o || !lse)
        return fail(PA_ERR_INVALID_ARG, "q, k, v, row_ptr, col_idx, o and lse must be non-null");
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o))
        return fail(PA_ERR_ALIGNMENT, "q, k, v and o must be 16-byte aligned");
    const int64_t nqb = (p->seq_len + kBlk - 1) / kBlk;
    if (nnz < 0 || nnz > (int64_t)INT32_MAX)
        return fail(PA_ERR_LAYOUT, "nnz %lld is outside [0, 2^31)", (long long)nnz);
    if (!workspace || workspace_bytes < kPrefillWorkspace)
        return fail(PA_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", kPrefillWorkspace, workspace_bytes);
    if (!aligned16(workspace)) return fail(PA_ERR_ALIGNMENT, "workspace must be 16-byte aligned");
    DeviceInfo dev;
    if (pa_status s = current_sm100_device(&dev)) return s;

    // Tensor maps (cached per buffer and shape): a Q box holds the two heads of a tile, K, V and O
    // boxes one head.
    CUtensorMap tmQ, tmK, tmV, tmO;
    const int D = p->head_dim;
    auto map_of = [&](const void *base, int heads, const pa_strides &st, int box_heads, const char *what, CUtensorMap *m) {
        // (packed sequences: one "batch" entry of total_tokens tokens)
        const TensorMapKey key = {base, varlen ? total_tokens : p->seq_len, st.seq, st.head, varlen ? 0 : st.batch, dev.device, D,
                                  heads, varlen ? 1 : p->batch, box_heads, kBlk};
        return get_tensor_map(key, what, m);
    };
    if (pa_status s = map_of(q, p->n_q_heads, p->q, 2, "q", &tmQ)) return s;
    if (pa_status s = map_of(k, p->n_kv_heads, p->k, 1, "k", &tmK)) return s;
    if (pa_status s = map_of(v, p->n_kv_heads, p->v, 1, "v", &tmV)) return s;
    if (p->o_dtype == PA_BF16) {
        if (pa_status s = map_of(o, p->n_q_heads, p->o, 1, "o", &tmO)) return s;
    } else {
        tmO = tmQ;  // fp32 output is written from registers; the map is not used
    }

    PrefillArgs a;
    a.row_ptr = row_ptr;
    a.col_idx = col_idx;
    a.cu_seqlens = cu_seqlens;
    a.o = o;
    a.lse = lse;
    a.status = static_cast<int32_t *>(workspace);
    a.o_sb = p->o.batch; a.o_ss = p->o.seq; a.o_sh = p->o.head;
    // LSE: [batch, Hq, seq_len], or [Hq, total_tokens] for packed sequences.
    a.lse_sb = varlen ? 0 : (int64_t)p->n_q_heads * p->seq_len;
    a.lse_sh = varlen ? total_tokens : p->seq_len;
    a.N = p->seq_len;
    a.nqb = (int32_t)nqb;
    a.batch = p->batch; a.Hq = p->n_q_heads; a.Hkv = p->n_kv_heads;
    a.G = p->n_q_heads / p->n_kv_heads;
    a.nsub = (a.G + 3) / 4;
    a.n_units = (int64_t)p->batch * nqb * a.Hkv * a.nsub;
    auto inv32 = [](int32_t d) { return d == 1 ? 0xffffffffu : (uint32_t)((1ull << 32) / (uint64_t)d); };
    a.inv_nsub = inv32(a.nsub); a.inv_Hkv = inv32(a.Hkv); a.inv_nqb = inv32(a.nqb);
    if (a.n_units > (int64_t)0x3fffffff) return fail(PA_ERR_SHAPE, "too many work units (%lld)", (long long)a.n_units);
    a.o_is_f32 = p->o_dtype == PA_F32;
    const float scale = p->softmax_scale != 0.f ? p->softmax_scale : 1.0f / sqrtf((float)D);
    a.scale_log2 = scale * 1.4426950408889634f;

    const long long wait_cycles = wait_limit_cycles();
    a.wait_cycles = wait_cycles > 0 ? wait_cycles : kWaitCycles;
    const unsigned grid = (unsigned)(a.n_units < dev.sms ? a.n_units : dev.sms);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    PA_CUDA_OK(cudaMemsetAsync(workspace, 0, kPrefillWorkspace, st));
    {
        // PA_VALIDATE=1: check the CSR on the device before the attention kernel is enqueued.  This
        // synchronises the stream (so not during stream capture) and is meant for bring-up: a CSR
        // whose extents point outside col_idx would otherwise be read out of bounds.
        if (env_switches().validate) {
            int32_t *check = static_cast<int32_t *>(workspace) + 32;
            validate_csr_kernel<<<(unsigned)((nqb + 127) / 128), 128, 0, st>>>(row_ptr, col_idx, (int32_t)nqb, nnz, check);
            PA_CUDA_OK(cudaGetLastError());
            int32_t found[2] = {0, 0};
            PA_CUDA_OK(cudaMemcpyAsync(found, check, sizeof(found), cudaMemcpyDeviceToHost, st));
            PA_CUDA_OK(cudaStreamSynchronize(st));
            static const char *const what[] = {"", "row_ptr must start at 0 and end at nnz", "row extent negative or beyond nnz",
                                               "block index outside [0, row]", "block indices of a row must ascend"};
            if (found[0] >= 1 && found[0] <= 4)
                return fail(PA_ERR_LAYOUT, "CSR check: %s (row %d)", what[found[0]], (int)found[1]);
        }
    }
    if (device_once_begin(dev.device, ONCE_PREFILL_ATTR)) {
        const cudaError_t e1 = cudaFuncSetAttribute(prefill_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                    (int)SmemMap<128>::kAlloc);
        const cudaError_t e2 = cudaFuncSetAttribute(prefill_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                    (int)SmemMap<64>::kAlloc);
        if (e1 != cudaSuccess || e2 != cudaSuccess) {
            device_once_reset(dev.device, ONCE_PREFILL_ATTR);
            return fail(PA_ERR_CUDA, "cudaFuncSetAttribute failed: %s", cudaGetErrorString(e1 != cudaSuccess ? e1 : e2));
        }
    }
    if (D == 128)
        prefill_kernel<128><<<grid, kThreads, SmemMap<128>::kAlloc, st>>>(tmQ, tmK, tmV, tmO, a);
    else
        prefill_kernel<64><<<grid, kThreads, SmemMap<64>::kAlloc, st>>>(tmQ, tmK, tmV, tmO, a);
    PA_CUDA_OK(cudaGetLastError());
    return PA_OK;
}

}  // namespace pa

extern "C" pa_status pa_prefill(const pa_prefill_params *p, const void *q, const void *k,
                                const void *v, const int32_t *row_ptr, const int32_t *col_idx,
                                int64_t nnz, void *o, float *lse, void *workspace,
                                size_t workspace_bytes, void *stream)
{
    pa::clear_error();
    return pa::launch_prefill(p, q, k, v, nullptr, 0, row_ptr, col_idx, nnz, o, lse, workspace, workspace_bytes, stream);
}

extern "C" pa_status pa_prefill_varlen(const pa_prefill_params *p, const void *q, const void *k, const void *v,
                                       const int32_t *cu_seqlens, int64_t total_tokens, const int32_t *row_ptr,
                                       const int32_t *col_idx, int64_t nnz, void *o, float *lse, void *workspace,
                                       size_t workspace_bytes, void *stream)
{
    pa::clear_error();
    if (!cu_seqlens) return pa::fail(PA_ERR_INVALID_ARG, "cu_seqlens must be non-null");
    return pa::launch_prefill(p, q, k, v, cu_seqlens, total_tokens, row_ptr, col_idx, nnz, o, lse, workspace,
                              workspace_bytes, stream);
}

extern "C" pa_status pa_prefill_status(const void *workspace, void *stream, int32_t *detail)
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
        return fail(PA_ERR_TIMEOUT, "a bounded wait inside the prefill kernel ran out (wait id %d)", host[1]);
    if (host[0] != 0) return fail(PA_ERR_CUDA, "unexpected device status %d", host[0]);
    return PA_OK;
}
