// pa_prefill_backward: gradients of the block-sparse attention forward (Eq. (1), Section 3.1, under
// the key-block lists of Algorithm 1, Section 3.3; the paper trains with the mask, Section 4.1).
//
// With P_ij = exp(scale <q_i, k_j> - LSE_i) for the attended pairs and an upstream gradient dO:
//     delta_i = <dO_i, O_i>                      dV_j = sum_i P_ij dO_i
//     dS_ij = P_ij (<dO_i, v_j> - delta_i)       dQ_i = scale sum_j dS_ij k_j
//                                                dK_j = scale sum_i dS_ij q_i
// (dK and dV also sum over the query heads that share the KV head).  This file holds the entry
// point, the kernels common to every head size (delta, the transposed layout) and the attention kernels
// for head_dim 64; head_dim 128 takes the tcgen05 kernels of the sibling file for the two attention
// kernels.  The kernels here:
//   backward_delta_kernel    delta = rowsum(dO * O)
//   csc_count / csc_fill     the CSR transposed: for every key block the query blocks that list it
//                            (a column walks the rows below it with a binary search each, so the lists
//                            come out ascending without atomics), and the columns cut into chunks
//   backward_dq_kernel       one CTA per (query block, query head): walks the row's key blocks
//   backward_dkv_kernel      one CTA per (key block, chunk of its query blocks, KV head): walks the
//                            chunk for every query head of the group; a column listed by many rows
//                            (the sink block is listed by all of them) is spread over many CTAs,
//                            which add their parts into dK / dV with fp32 atomics
// Both attention kernels of this file recompute S and P tile by tile (64 queries x 64 keys) on the warp-level
// tensor-core MMA from bf16 tiles staged in padded shared memory; P and dS go back into the MMA as
// bf16, accumulation is fp32.  Outputs are fp32.
#include <cuda_bf16.h>
#include <math.h>

#include "backward.cuh"
#include "common.cuh"
#include "scan.cuh"
#include "sm100_ptx.cuh"

namespace pa {

constexpr int kBwdThreads = 128;  // four warps, 16 rows of the tile each

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// delta[b, h, t] = sum_d dO[b, t, h, d] O[b, t, h, d]; D / 8 lanes per (token, head) row, 16 bytes per lane.
template <int D>
__global__ void backward_delta_kernel(const BackwardArgs a)
{
    constexpr int kLanes = D / 8;              // lanes that share a row
    constexpr int kRowsPerWarp = 32 / kLanes;
    const int lane = threadIdx.x & 31, sub = lane % kLanes;
    const int64_t row = ((int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * kRowsPerWarp + lane / kLanes;
    const int64_t rows = (int64_t)a.batch * a.N * a.Hq;
    float acc = 0.f;
    int h = 0;
    int64_t t = 0, b = 0;
    if (row < rows) {
        h = (int)(row % a.Hq);
        t = (row / a.Hq) % a.N;
        b = row / ((int64_t)a.Hq * a.N);
        const int64_t off = b * a.o_sb + t * a.o_ss + (int64_t)h * a.o_sh + 8 * sub;
        const uint4 x = *reinterpret_cast<const uint4 *>(a.o + off);
        const uint4 y = *reinterpret_cast<const uint4 *>(a.d_o + off);
        const uint32_t xs[4] = {x.x, x.y, x.z, x.w}, ys[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 xf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&xs[e]));
            const float2 yf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&ys[e]));
            acc += xf.x * yf.x + xf.y * yf.y;
        }
    }
#pragma unroll
    for (int o = kLanes / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (row < rows && sub == 0) a.delta[(b * a.Hq + h) * a.N + t] = acc;
}

// Does row i of the CSR list block j?  (rows are ascending: binary search)
__device__ __forceinline__ bool row_lists(const int32_t *row_ptr, const int32_t *col_idx, int32_t i, int32_t j)
{
    int32_t lo = row_ptr[i], hi = row_ptr[i + 1];
    while (lo < hi) {
        const int32_t mid = (lo + hi) >> 1;
        const int32_t c = col_idx[mid];
        if (c == j) return true;
        if (c < j) lo = mid + 1;
        else hi = mid;
    }
    return false;
}

// One warp per key block j: counts the query blocks i >= j that list it.  col_ptr[j + 1] = count
// (scanned afterwards), chunk_ptr[j + 1] = ceil(count / kBwdChunk).
__global__ void csc_count_kernel(const BackwardArgs a)
{
    const int32_t j = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (j >= a.nqb) return;
    int32_t cnt = 0;
    for (int32_t i = j + lane; i < a.nqb; i += 32) cnt += row_lists(a.row_ptr, a.col_idx, i, j) ? 1 : 0;
    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    if (lane == 0) {
        if (j == 0) a.col_ptr[0] = a.chunk_ptr[0] = 0;
        a.col_ptr[j + 1] = cnt;
        a.chunk_ptr[j + 1] = (cnt + kBwdChunk - 1) / kBwdChunk;
    }
}

// One warp per key block j: writes its listers in ascending order.
__global__ void csc_fill_kernel(const BackwardArgs a)
{
    const int32_t j = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (j >= a.nqb) return;
    int32_t pos = a.col_ptr[j];
    for (int32_t base = j; base < a.nqb; base += 32) {
        const int32_t i = base + lane;
        const bool on = i < a.nqb && row_lists(a.row_ptr, a.col_idx, i, j);
        const uint32_t m = __ballot_sync(0xffffffffu, on);
        if (on) a.row_idx[pos + __popc(m & ((1u << lane) - 1u))] = i;
        pos += __popc(m);
    }
}

// ---------------------------------------------------------------- tiles in shared memory
// A tile is 64 rows of D bf16 at a pitch of 2 D + 16 bytes (rows 16-byte aligned, eight
// consecutive rows on different banks for ldmatrix).
template <int D>
struct BwdTile {
    static constexpr uint32_t kPitch = D * 2 + 16;
    static constexpr uint32_t kBytes = kBwdBlk * kPitch;
};

__device__ __forceinline__ void bwd_cp_async16(uint32_t dst, const void *src, uint32_t src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}

// Copies rows [tok0, tok0 + 64) of one head into a tile; rows at or beyond N are zero-filled.
template <int D>
__device__ __forceinline__ void load_tile(uint32_t dst, const __nv_bfloat16 *base, int64_t stride_tok, int64_t tok0,
                                          int64_t N, int tid)
{
    constexpr int NP = D / 8, kRows = kBwdThreads / NP;
    const int r0 = tid / NP, pc = tid % NP;
#pragma unroll
    for (int r = r0; r < kBwdBlk; r += kRows) {
        const bool in = tok0 + r < N;
        bwd_cp_async16(dst + (uint32_t)r * BwdTile<D>::kPitch + (uint32_t)pc * 16u,
                       base + (in ? (tok0 + r) * stride_tok : 0) + 8 * pc, in ? 16u : 0u);
    }
}

// A fragment (16 rows x 16 k) of a [row][k] tile.
template <int D>
__device__ __forceinline__ void frag_a(uint32_t tile, int r0, int ks, int lane, uint32_t (&f)[4])
{
    const int row = r0 + (lane & 7) + ((lane >> 3) & 1) * 8, ch = 2 * ks + (lane >> 4);
    ptx::ldmatrix_x4(tile + (uint32_t)row * BwdTile<D>::kPitch + (uint32_t)ch * 16u, f[0], f[1], f[2], f[3]);
}
// B fragments of two 8-column tiles (columns n0 .. n0 + 15) from a [n][k] tile (B = tile^T).
template <int D>
__device__ __forceinline__ void frag_b_nk(uint32_t tile, int n0, int ks, int lane, uint32_t (&f)[4])
{
    const int row = n0 + (lane & 7) + (lane >> 4) * 8, ch = 2 * ks + ((lane >> 3) & 1);
    ptx::ldmatrix_x4(tile + (uint32_t)row * BwdTile<D>::kPitch + (uint32_t)ch * 16u, f[0], f[1], f[2], f[3]);
}
// B fragments of two 8-column tiles (16-byte column chunks c, c + 1) from a [k][n] tile, k rows k0 .. k0 + 15.
template <int D>
__device__ __forceinline__ void frag_b_kn(uint32_t tile, int k0, int c, int lane, uint32_t (&f)[4])
{
    const int row = k0 + (lane & 7) + ((lane >> 3) & 1) * 8, ch = c + (lane >> 4);
    ptx::ldmatrix_x4_trans(tile + (uint32_t)row * BwdTile<D>::kPitch + (uint32_t)ch * 16u, f[0], f[1], f[2], f[3]);
}

// acc[nt] (16 x 8 each, nt = 0..7) = A-tile rows r0..r0+15 times B-tile^T (64 columns), over D.
template <int D>
__device__ __forceinline__ void tile_product(uint32_t a_tile, int r0, uint32_t b_tile, int lane, float (&acc)[8][4])
{
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
        uint32_t fa[4];
        frag_a<D>(a_tile, r0, ks, lane, fa);
#pragma unroll
        for (int np = 0; np < 4; ++np) {
            uint32_t fb[4];
            frag_b_nk<D>(b_tile, 16 * np, ks, lane, fb);
            mma_bf16_16816(acc[2 * np], fa[0], fa[1], fa[2], fa[3], fb[0], fb[1]);
            mma_bf16_16816(acc[2 * np + 1], fa[0], fa[1], fa[2], fa[3], fb[2], fb[3]);
        }
    }
}

// out[e] (16 x 8 each, e = 0 .. D/8 - 1) += W (16 x 64, given as four k-steps of A fragments) times a
// [k = 64 rows][D] tile.
template <int D>
__device__ __forceinline__ void tile_accumulate(const uint32_t (&w)[4][4], uint32_t b_tile, int lane, float (&out)[D / 8][4])
{
#pragma unroll
    for (int kk = 0; kk < 4; ++kk)
#pragma unroll
        for (int c = 0; c < D / 8; c += 2) {
            uint32_t fb[4];
            frag_b_kn<D>(b_tile, 16 * kk, c, lane, fb);
            mma_bf16_16816(out[c], w[kk][0], w[kk][1], w[kk][2], w[kk][3], fb[0], fb[1]);
            mma_bf16_16816(out[c + 1], w[kk][0], w[kk][1], w[kk][2], w[kk][3], fb[2], fb[3]);
        }
}

// The two rows (g and g + 8 of the warp's 16) a thread holds in an accumulator tile.
struct RowStat {
    float lse2[2], delta[2];
};

// dS (or P) as the A operand of the next MMA: accumulator tiles 2 kk, 2 kk + 1 are k-step kk.
__device__ __forceinline__ void pack_a(const float (&x)[8][4], uint32_t (&w)[4][4])
{
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
        w[kk][0] = ptx::cvt_bf16x2(x[2 * kk][0], x[2 * kk][1]);
        w[kk][1] = ptx::cvt_bf16x2(x[2 * kk][2], x[2 * kk][3]);
        w[kk][2] = ptx::cvt_bf16x2(x[2 * kk + 1][0], x[2 * kk + 1][1]);
        w[kk][3] = ptx::cvt_bf16x2(x[2 * kk + 1][2], x[2 * kk + 1][3]);
    }
}

// dQ: one CTA per (query block, query head); warp w owns query rows 16 w .. 16 w + 15.
template <int D>
__global__ void __launch_bounds__(kBwdThreads, 3) backward_dq_kernel(const BackwardArgs a)
{
    using T = BwdTile<D>;
    extern __shared__ __align__(16) uint8_t bwd_smem[];
    const uint32_t sQ = ptx::smem_u32(bwd_smem), sG = sQ + T::kBytes, sK = sG + T::kBytes, sV = sK + T::kBytes;
    const int i = a.nqb - 1 - (int)blockIdx.x, h = blockIdx.y, b = blockIdx.z, hk = h / a.G;  // long rows first
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, g = lane >> 2, t = lane & 3;
    const int r0 = 16 * wid;
    const int32_t e0 = a.row_ptr[i], e1 = a.row_ptr[i + 1];

    load_tile<D>(sQ, a.q + b * a.q_sb + (int64_t)h * a.q_sh, a.q_ss, (int64_t)i * kBwdBlk, a.N, tid);
    load_tile<D>(sG, a.d_o + b * a.o_sb + (int64_t)h * a.o_sh, a.o_ss, (int64_t)i * kBwdBlk, a.N, tid);
    RowStat st;
#pragma unroll
    for (int x = 0; x < 2; ++x) {
        const int64_t q = (int64_t)i * kBwdBlk + r0 + g + 8 * x;
        const float lse = q < a.N ? a.lse[((int64_t)b * a.Hq + h) * a.N + q] : INFINITY;
        // (a row beyond the sequence, or one the layout left empty, has no weights: P = 0)
        st.lse2[x] = (lse == -INFINITY || lse == INFINITY) ? INFINITY : lse * 1.4426950408889634f;
        st.delta[x] = q < a.N ? a.delta[((int64_t)b * a.Hq + h) * a.N + q] : 0.f;
    }
    float dq[D / 8][4];
#pragma unroll
    for (int e = 0; e < D / 8; ++e) dq[e][0] = dq[e][1] = dq[e][2] = dq[e][3] = 0.f;

    const __nv_bfloat16 *kbase = a.k + b * a.k_sb + (int64_t)hk * a.k_sh;
    const __nv_bfloat16 *vbase = a.v + b * a.v_sb + (int64_t)hk * a.v_sh;
    for (int32_t e = e0; e < e1; ++e) {
        const int32_t j = a.col_idx[e];
        __syncthreads();  // every warp has finished with the previous K and V tiles
        load_tile<D>(sK, kbase, a.k_ss, (int64_t)j * kBwdBlk, a.N, tid);
        load_tile<D>(sV, vbase, a.v_ss, (int64_t)j * kBwdBlk, a.N, tid);
        asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;\n" ::: "memory");
        __syncthreads();
        float s[8][4], dp[8][4];
        tile_product<D>(sQ, r0, sK, lane, s);   // S = Q K^T
        tile_product<D>(sG, r0, sV, lane, dp);  // dP = dO V^T
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const int64_t kv = (int64_t)j * kBwdBlk + 8 * nt + 2 * t + (x & 1);
                const int64_t q = (int64_t)i * kBwdBlk + r0 + g + 8 * (x >> 1);
                const bool keep = kv < a.N && (j != i || kv <= q);  // Algorithm 1's causal term on the diagonal pair
                const float p = keep ? ptx::ex2(s[nt][x] * a.scale_log2 - st.lse2[x >> 1]) : 0.f;
                s[nt][x] = p * (dp[nt][x] - st.delta[x >> 1]);  // dS
            }
        uint32_t w[4][4];
        pack_a(s, w);
        tile_accumulate<D>(w, sK, lane, dq);  // dQ += dS K
    }
#pragma unroll
    for (int x = 0; x < 2; ++x) {
        const int64_t q = (int64_t)i * kBwdBlk + r0 + g + 8 * x;
        if (q >= a.N) continue;
        float *dst = a.dq + (((int64_t)b * a.N + q) * a.Hq + h) * D + 2 * t;
#pragma unroll
        for (int e = 0; e < D / 8; ++e)
            *reinterpret_cast<float2 *>(dst + 8 * e) = make_float2(dq[e][2 * x] * a.scale, dq[e][2 * x + 1] * a.scale);
    }
}

// dK, dV: one CTA per (chunk of a key block's query blocks, KV head); warp w owns key rows
// 16 w .. 16 w + 15 and walks the chunk once per query head of the group.
template <int D>
__global__ void __launch_bounds__(kBwdThreads) backward_dkv_kernel(const BackwardArgs a)
{
    using T = BwdTile<D>;
    extern __shared__ __align__(16) uint8_t bwd_smem[];
    const uint32_t sK = ptx::smem_u32(bwd_smem), sV = sK + T::kBytes, sQ = sV + T::kBytes, sG = sQ + T::kBytes;
    float *s_lse2 = reinterpret_cast<float *>(bwd_smem + 4 * T::kBytes);  // [64] per query of the tile
    float *s_delta = s_lse2 + kBwdBlk;
    const int32_t c = blockIdx.x;
    const int hk = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, g = lane >> 2, t = lane & 3;
    const int r0 = 16 * wid;
    if (c >= a.chunk_ptr[a.nqb]) return;
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

    load_tile<D>(sK, a.k + b * a.k_sb + (int64_t)hk * a.k_sh, a.k_ss, (int64_t)j * kBwdBlk, a.N, tid);
    load_tile<D>(sV, a.v + b * a.v_sb + (int64_t)hk * a.v_sh, a.v_ss, (int64_t)j * kBwdBlk, a.N, tid);
    float dk[D / 8][4], dv[D / 8][4];
#pragma unroll
    for (int e = 0; e < D / 8; ++e) {
        dk[e][0] = dk[e][1] = dk[e][2] = dk[e][3] = 0.f;
        dv[e][0] = dv[e][1] = dv[e][2] = dv[e][3] = 0.f;
    }
    for (int h = hk * a.G; h < (hk + 1) * a.G; ++h) {
        const __nv_bfloat16 *qbase = a.q + b * a.q_sb + (int64_t)h * a.q_sh;
        const __nv_bfloat16 *gbase = a.d_o + b * a.o_sb + (int64_t)h * a.o_sh;
        for (int32_t e = e0; e < e1; ++e) {
            const int32_t i = a.row_idx[e];
            __syncthreads();  // every warp has finished with the previous Q and dO tiles
            load_tile<D>(sQ, qbase, a.q_ss, (int64_t)i * kBwdBlk, a.N, tid);
            load_tile<D>(sG, gbase, a.o_ss, (int64_t)i * kBwdBlk, a.N, tid);
            if (tid < kBwdBlk) {
                const int64_t q = (int64_t)i * kBwdBlk + tid;
                const float lse = q < a.N ? a.lse[((int64_t)b * a.Hq + h) * a.N + q] : INFINITY;
                s_lse2[tid] = (lse == -INFINITY || lse == INFINITY) ? INFINITY : lse * 1.4426950408889634f;
                s_delta[tid] = q < a.N ? a.delta[((int64_t)b * a.Hq + h) * a.N + q] : 0.f;
            }
            asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;\n" ::: "memory");
            __syncthreads();
            float s[8][4], dp[8][4];
            tile_product<D>(sK, r0, sQ, lane, s);   // S^T = K Q^T: rows = keys, columns = queries
            tile_product<D>(sV, r0, sG, lane, dp);  // dP^T = V dO^T
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    const int col = 8 * nt + 2 * t + (x & 1);
                    const int64_t q = (int64_t)i * kBwdBlk + col;
                    const int64_t kv = (int64_t)j * kBwdBlk + r0 + g + 8 * (x >> 1);
                    const bool keep = i != j || kv <= q;  // (queries beyond the sequence carry lse2 = inf: P = 0)
                    const float p = keep ? ptx::ex2(s[nt][x] * a.scale_log2 - s_lse2[col]) : 0.f;
                    s[nt][x] = p;                                   // P^T
                    dp[nt][x] = p * (dp[nt][x] - s_delta[col]);     // dS^T
                }
            uint32_t wp[4][4], wd[4][4];
            pack_a(s, wp);
            pack_a(dp, wd);
            tile_accumulate<D>(wp, sG, lane, dv);  // dV += P^T dO
            tile_accumulate<D>(wd, sQ, lane, dk);  // dK += dS^T Q
        }
    }
    // A column that many rows list is spread over several CTAs: the parts are added up in memory.
#pragma unroll
    for (int x = 0; x < 2; ++x) {
        const int64_t kv = (int64_t)j * kBwdBlk + r0 + g + 8 * x;
        if (kv >= a.N) continue;
        const int64_t off = (((int64_t)b * a.N + kv) * a.Hkv + hk) * D + 2 * t;
#pragma unroll
        for (int e = 0; e < D / 8; ++e) {
            atomicAdd(a.dk + off + 8 * e, dk[e][2 * x] * a.scale);
            atomicAdd(a.dk + off + 8 * e + 1, dk[e][2 * x + 1] * a.scale);
            atomicAdd(a.dv + off + 8 * e, dv[e][2 * x]);
            atomicAdd(a.dv + off + 8 * e + 1, dv[e][2 * x + 1]);
        }
    }
}

}  // namespace pa

namespace pa {

// Workspace: status block (256 bytes), delta [batch, Hq, N] fp32, then col_ptr [nqb + 1], chunk_ptr [nqb + 1],
// row_idx [nnz] int32.
static size_t backward_workspace_bytes(const pa_prefill_params *p, int64_t nnz)
{
    const int64_t nqb = (p->seq_len + kBwdBlk - 1) / kBwdBlk;
    size_t bytes = kBwdStatusBytes + (size_t)p->batch * p->n_q_heads * p->seq_len * sizeof(float);
    bytes = (bytes + 255) & ~(size_t)255;
    bytes += (size_t)(2 * (nqb + 1) + nnz) * sizeof(int32_t);
    return (bytes + 255) & ~(size_t)255;
}

static pa_status check_backward(const pa_prefill_params *p, int64_t nnz)
{
    if (!p) return fail(PA_ERR_INVALID_ARG, "params must be non-null");
    if (p->batch < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1 || p->seq_len < 1)
        return fail(PA_ERR_INVALID_ARG, "batch, head counts and seq_len must be positive");
    if (!(p->softmax_scale >= 0.f) || isinf(p->softmax_scale))
        return fail(PA_ERR_INVALID_ARG, "softmax_scale must be finite and >= 0 (0 = default)");
    if (p->head_dim != 64 && p->head_dim != 128) return fail(PA_ERR_SHAPE, "head_dim must be 64 or 128");
    if (p->block != kBwdBlk) return fail(PA_ERR_SHAPE, "block must be 64");
    if (p->n_q_heads % p->n_kv_heads) return fail(PA_ERR_SHAPE, "n_q_heads must be a multiple of n_kv_heads");
    if (p->n_q_heads < 2) return fail(PA_ERR_SHAPE, "n_q_heads must be >= 2");  // (as in pa_prefill: tiles stack two heads)
    if (p->o_dtype != PA_BF16) return fail(PA_ERR_SHAPE, "the backward pass reads O and dO as bfloat16");
    if (p->seq_len > ((int64_t)1 << 30)) return fail(PA_ERR_SHAPE, "seq_len too large");
    if (p->batch > 65535 || p->n_q_heads > 65535) return fail(PA_ERR_SHAPE, "batch and head counts must be <= 65535");
    if (nnz < 0 || nnz > (int64_t)INT32_MAX) return fail(PA_ERR_LAYOUT, "nnz %lld is outside [0, 2^31)", (long long)nnz);
    const pa_strides *st[4] = {&p->q, &p->k, &p->v, &p->o};
    for (auto s : st) {
        if (s->seq < p->head_dim || s->head < p->head_dim || s->batch < 0)
            return fail(PA_ERR_SHAPE, "strides must be >= head_dim");
        if ((s->seq % 8) || (s->head % 8) || (s->batch % 8))
            return fail(PA_ERR_ALIGNMENT, "strides must be multiples of 8 elements (16 bytes)");
    }
    return PA_OK;
}

template <int D>
static pa_status launch_backward(const BackwardArgs &a, const pa_prefill_params *p, int64_t nnz, int device, int sms,
                                 cudaStream_t st)
{
    constexpr int kSmemDq = 4 * BwdTile<D>::kBytes, kSmemDkv = 4 * BwdTile<D>::kBytes + 2 * kBwdBlk * 4;
    if (device_once_begin(device, D == 128 ? ONCE_BACKWARD_ATTR : ONCE_BACKWARD_ATTR_64)) {
        const cudaError_t e1 = cudaFuncSetAttribute(backward_dq_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemDq);
        const cudaError_t e2 = cudaFuncSetAttribute(backward_dkv_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemDkv);
        if (e1 != cudaSuccess || e2 != cudaSuccess) {
            device_once_reset(device, D == 128 ? ONCE_BACKWARD_ATTR : ONCE_BACKWARD_ATTR_64);
            return fail(PA_ERR_CUDA, "cudaFuncSetAttribute failed: %s", cudaGetErrorString(e1 != cudaSuccess ? e1 : e2));
        }
    }
    const int64_t rows = (int64_t)a.batch * a.N * a.Hq;
    constexpr int kDeltaRowsPerBlock = 8 * (32 / (D / 8));  // eight warps, each 32 / (D / 8) rows
    backward_delta_kernel<D><<<(unsigned)((rows + kDeltaRowsPerBlock - 1) / kDeltaRowsPerBlock), 256, 0, st>>>(a);
    const unsigned col_blocks = (unsigned)((a.nqb + 7) / 8);
    csc_count_kernel<<<col_blocks, 256, 0, st>>>(a);
    layout_scan_kernel<<<1, 1024, 0, st>>>(a.nqb, a.col_ptr);
    layout_scan_kernel<<<1, 1024, 0, st>>>(a.nqb, a.chunk_ptr);
    csc_fill_kernel<<<col_blocks, 256, 0, st>>>(a);
    // head_dim 128: dQ, dK and dV on the tcgen05 tensor cores (PA_BACKWARD_PATH=mma keeps the warp-level kernels).
    if (D == 128 && !env_switches().backward_mma) {
        PA_CUDA_OK(cudaGetLastError());
        return launch_backward_sm100(a, p, nnz, device, sms, st);
    }
    backward_dq_kernel<D><<<dim3((unsigned)a.nqb, (unsigned)a.Hq, (unsigned)a.batch), kBwdThreads, kSmemDq, st>>>(a);
    // (an upper bound on the number of chunks; CTAs beyond the real count return at once)
    const int64_t max_chunks = nnz / kBwdChunk + a.nqb;
    backward_dkv_kernel<D><<<dim3((unsigned)max_chunks, (unsigned)a.Hkv, (unsigned)a.batch), kBwdThreads, kSmemDkv, st>>>(a);
    PA_CUDA_OK(cudaGetLastError());
    return PA_OK;
}

}  // namespace pa

extern "C" size_t pa_prefill_backward_workspace_bytes(const pa_prefill_params *p, int64_t nnz)
{
    using namespace pa;
    if (check_backward(p, nnz) != PA_OK) return 0;
    return backward_workspace_bytes(p, nnz);
}

extern "C" pa_status pa_prefill_backward(const pa_prefill_params *p, const void *q, const void *k, const void *v,
                                         const void *o, const float *lse, const void *d_o, const int32_t *row_ptr,
                                         const int32_t *col_idx, int64_t nnz, float *dq, float *dk, float *dv,
                                         void *workspace, size_t workspace_bytes, void *stream)
{
    using namespace pa;
    clear_error();
    if (pa_status s = check_backward(p, nnz)) return s;
    if (!q || !k || !v || !o || !lse || !d_o || !row_ptr || !col_idx || !dq || !dk || !dv)
        return fail(PA_ERR_INVALID_ARG, "q, k, v, o, lse, d_o, row_ptr, col_idx, dq, dk and dv must be non-null");
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(d_o) || !aligned16(dq) ||
        !aligned16(dk) || !aligned16(dv))
        return fail(PA_ERR_ALIGNMENT, "tensors must be 16-byte aligned");
    const size_t need = backward_workspace_bytes(p, nnz);
    if (!workspace || workspace_bytes < need)
        return fail(PA_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", need, workspace_bytes);
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return fail(PA_ERR_ALIGNMENT, "workspace must be 256-byte aligned");
    DeviceInfo dev;
    if (pa_status s = current_sm100_device(&dev)) return s;

    BackwardArgs a;
    a.q = static_cast<const __nv_bfloat16 *>(q);
    a.k = static_cast<const __nv_bfloat16 *>(k);
    a.v = static_cast<const __nv_bfloat16 *>(v);
    a.o = static_cast<const __nv_bfloat16 *>(o);
    a.d_o = static_cast<const __nv_bfloat16 *>(d_o);
    a.lse = lse;
    a.row_ptr = row_ptr;
    a.col_idx = col_idx;
    const int64_t nqb = (p->seq_len + kBwdBlk - 1) / kBwdBlk;
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    a.status = reinterpret_cast<int32_t *>(ws);
    a.delta = reinterpret_cast<float *>(ws + kBwdStatusBytes);
    size_t off = (kBwdStatusBytes + (size_t)p->batch * p->n_q_heads * p->seq_len * sizeof(float) + 255) & ~(size_t)255;
    a.col_ptr = reinterpret_cast<int32_t *>(ws + off);
    a.chunk_ptr = a.col_ptr + (nqb + 1);
    a.row_idx = a.chunk_ptr + (nqb + 1);
    a.dq = dq; a.dk = dk; a.dv = dv;
    a.q_sb = p->q.batch; a.q_ss = p->q.seq; a.q_sh = p->q.head;
    a.k_sb = p->k.batch; a.k_ss = p->k.seq; a.k_sh = p->k.head;
    a.v_sb = p->v.batch; a.v_ss = p->v.seq; a.v_sh = p->v.head;
    a.o_sb = p->o.batch; a.o_ss = p->o.seq; a.o_sh = p->o.head;
    a.N = p->seq_len;
    a.nqb = (int32_t)nqb;
    a.batch = p->batch; a.Hq = p->n_q_heads; a.Hkv = p->n_kv_heads;
    a.G = p->n_q_heads / p->n_kv_heads;
    a.scale = p->softmax_scale != 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->head_dim);
    a.scale_log2 = a.scale * 1.4426950408889634f;
    a.npairs = (a.G + 1) / 2;
    a.wait_cycles = 0;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t kv_bytes = (size_t)p->batch * p->seq_len * p->n_kv_heads * p->head_dim * sizeof(float);
    PA_CUDA_OK(cudaMemsetAsync(workspace, 0, kBwdStatusBytes, st));
    PA_CUDA_OK(cudaMemsetAsync(dk, 0, kv_bytes, st));
    PA_CUDA_OK(cudaMemsetAsync(dv, 0, kv_bytes, st));
    return p->head_dim == 128 ? launch_backward<128>(a, p, nnz, dev.device, dev.sms, st) : launch_backward<64>(a, p, nnz, dev.device, dev.sms, st);
}
