// pa_layout_size / pa_build_layout: the block-sparse CSR of Algorithm 1 (Section 3.3).
#include <vector>

#include "common.cuh"
#include "layout_rule.cuh"
#include "scan.cuh"

namespace pa {

__global__ void layout_count_kernel(int32_t nqb, int32_t W, int32_t S, int32_t *row_ptr, bool power)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) row_ptr[0] = 0;
    if (i < nqb) row_ptr[i + 1] = row_length(i, W, S, power);
}

struct StoreCols {
    int32_t *out;
    __device__ void operator()(int pos, int64_t j) const { out[pos] = (int32_t)j; }
};

__global__ void layout_fill_kernel(int32_t nqb, int32_t W, int32_t S, const int32_t *row_ptr,
                                   int32_t *col_idx, bool power)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= nqb) return;
    for_each_key_block(i, W, S, StoreCols{col_idx + row_ptr[i]}, power);
}

// Tile layouts: the mask's block holds r tiles of the attention kernel.  Algorithm 1's window,
// power and sink terms see the blocks only, so every listed block j < i contributes its r tiles;
// its causal term cuts the diagonal block i down to the tiles i r .. ti.
__host__ __device__ inline int64_t tile_row_length(int64_t ti, int32_t r, int32_t W, int32_t S)
{
    const int64_t i = ti / r;
    return (int64_t)r * (row_length(i, W, S) - 1) + (ti - i * r + 1);
}

__global__ void tile_layout_count_kernel(int32_t nqt, int32_t r, int32_t W, int32_t S, int32_t *row_ptr)
{
    const int64_t ti = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (ti == 0) row_ptr[0] = 0;
    if (ti < nqt) row_ptr[ti + 1] = (int32_t)tile_row_length(ti, r, W, S);
}

struct StoreTileCols {
    int32_t *out;
    int64_t i, ti;
    int32_t r;
    __device__ void operator()(int pos, int64_t j) const
    {
        // (The diagonal block is the last one listed, so every block before it is whole.)
        const int64_t last = j == i ? ti : j * r + r - 1;
        int32_t *dst = out + (int64_t)pos * r;
        for (int64_t tj = j * r; tj <= last; ++tj) *dst++ = (int32_t)tj;
    }
};

__global__ void tile_layout_fill_kernel(int32_t nqt, int32_t r, int32_t W, int32_t S, const int32_t *row_ptr,
                                        int32_t *col_idx)
{
    const int64_t ti = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (ti >= nqt) return;
    const int64_t i = ti / r;
    for_each_key_block(i, W, S, StoreTileCols{col_idx + row_ptr[ti], i, ti, r});
}

static pa_status check_layout_args(int64_t seq_len, int32_t block, int32_t W, int32_t S)
{
    if (seq_len < 1) return fail(PA_ERR_INVALID_ARG, "seq_len must be >= 1 (got %lld)", (long long)seq_len);
    if (block < 1) return fail(PA_ERR_INVALID_ARG, "block must be >= 1 (got %d)", block);
    if (W < 0 || S < 0) return fail(PA_ERR_INVALID_ARG, "window_blocks and sink_blocks must be >= 0");
    return PA_OK;
}

}  // namespace pa

namespace pa {

static pa_status layout_size(int64_t seq_len, int32_t block, int32_t W, int32_t S, bool power, int32_t *n_qblocks,
                             int64_t *nnz)
{
    if (pa_status s = check_layout_args(seq_len, block, W, S)) return s;
    if (!power && W < 1)
        return fail(PA_ERR_INVALID_ARG, "a sliding-window layout needs window_blocks >= 1 (the diagonal block)");
    if (!n_qblocks || !nnz) return fail(PA_ERR_INVALID_ARG, "n_qblocks and nnz must be non-null");
    const int64_t nqb = (seq_len + block - 1) / block;
    if (nqb >= INT32_MAX) return fail(PA_ERR_SHAPE, "n_qblocks %lld does not fit in int32", (long long)nqb);
    int64_t total = 0;
    for (int64_t i = 0; i < nqb; ++i) total += row_length(i, W, S, power);
    if (total > INT32_MAX) return fail(PA_ERR_SHAPE, "nnz %lld does not fit in int32", (long long)total);
    *n_qblocks = (int32_t)nqb;
    *nnz = total;
    return PA_OK;
}

static pa_status build_layout(int64_t seq_len, int32_t block, int32_t W, int32_t S, bool power, int32_t *row_ptr,
                              int32_t *col_idx, int64_t col_capacity, void *stream)
{
    int32_t nqb = 0;
    int64_t nnz = 0;
    if (pa_status s = layout_size(seq_len, block, W, S, power, &nqb, &nnz)) return s;
    if (!row_ptr || !col_idx) return fail(PA_ERR_INVALID_ARG, "row_ptr and col_idx must be non-null");
    if (col_capacity < nnz)
        return fail(PA_ERR_LAYOUT, "col_capacity %lld < nnz %lld", (long long)col_capacity, (long long)nnz);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int threads = 256;
    const unsigned blocks = (unsigned)((nqb + threads - 1) / threads);
    layout_count_kernel<<<blocks, threads, 0, st>>>(nqb, W, S, row_ptr, power);
    layout_scan_kernel<<<1, 1024, 0, st>>>(nqb, row_ptr);
    layout_fill_kernel<<<blocks, threads, 0, st>>>(nqb, W, S, row_ptr, col_idx, power);
    PA_CUDA_OK(cudaGetLastError());
    return PA_OK;
}

}  // namespace pa

extern "C" pa_status pa_layout_size(int64_t seq_len, int32_t block, int32_t window_blocks,
                                    int32_t sink_blocks, int32_t *n_qblocks, int64_t *nnz)
{
    pa::clear_error();
    return pa::layout_size(seq_len, block, window_blocks, sink_blocks, true, n_qblocks, nnz);
}

extern "C" pa_status pa_build_layout(int64_t seq_len, int32_t block, int32_t window_blocks,
                                     int32_t sink_blocks, int32_t *row_ptr, int32_t *col_idx,
                                     int64_t col_capacity, void *stream)
{
    pa::clear_error();
    return pa::build_layout(seq_len, block, window_blocks, sink_blocks, true, row_ptr, col_idx, col_capacity, stream);
}

extern "C" pa_status pa_window_layout_size(int64_t seq_len, int32_t block, int32_t window_blocks,
                                           int32_t sink_blocks, int32_t *n_qblocks, int64_t *nnz)
{
    pa::clear_error();
    return pa::layout_size(seq_len, block, window_blocks, sink_blocks, false, n_qblocks, nnz);
}

extern "C" pa_status pa_build_window_layout(int64_t seq_len, int32_t block, int32_t window_blocks,
                                            int32_t sink_blocks, int32_t *row_ptr, int32_t *col_idx,
                                            int64_t col_capacity, void *stream)
{
    pa::clear_error();
    return pa::build_layout(seq_len, block, window_blocks, sink_blocks, false, row_ptr, col_idx, col_capacity, stream);
}

extern "C" pa_status pa_reach_counts(const int32_t *row_ptr, const int32_t *col_idx, int32_t n_blocks,
                                     int32_t start, int32_t max_steps, int64_t *counts)
{
    using namespace pa;
    clear_error();
    if (!row_ptr || !col_idx || !counts) return fail(PA_ERR_INVALID_ARG, "row_ptr, col_idx and counts must be non-null");
    if (n_blocks < 1 || start < 0 || start >= n_blocks || max_steps < 1)
        return fail(PA_ERR_INVALID_ARG, "need n_blocks >= 1, 0 <= start < n_blocks, max_steps >= 1");
    // Breadth-first search from `start` over the edges block -> listed key block, level by level.
    std::vector<int32_t> depth((size_t)n_blocks, -1), frontier{start}, next;
    depth[(size_t)start] = 0;
    int64_t reached = 1;
    for (int32_t k = 1; k <= max_steps; ++k) {
        next.clear();
        for (int32_t u : frontier) {
            const int32_t lo = row_ptr[u], hi = row_ptr[u + 1];
            if (lo < 0 || hi < lo) return fail(PA_ERR_LAYOUT, "row %d has a negative extent", u);
            for (int32_t e = lo; e < hi; ++e) {
                const int32_t v = col_idx[e];
                if (v < 0 || v >= n_blocks) return fail(PA_ERR_LAYOUT, "row %d lists block %d outside [0, %d)", u, v, n_blocks);
                if (depth[(size_t)v] < 0) {
                    depth[(size_t)v] = k;
                    next.push_back(v);
                    ++reached;
                }
            }
        }
        counts[k - 1] = reached;
        frontier.swap(next);
    }
    return PA_OK;
}

extern "C" pa_status pa_tile_layout_size(int64_t seq_len, int32_t block, int32_t window_blocks,
                                         int32_t sink_blocks, int32_t tile, int32_t *n_qtiles, int64_t *nnz)
{
    using namespace pa;
    clear_error();
    if (pa_status s = check_layout_args(seq_len, block, window_blocks, sink_blocks)) return s;
    if (tile < 1) return fail(PA_ERR_INVALID_ARG, "tile must be >= 1 (got %d)", tile);
    if (block % tile != 0) return fail(PA_ERR_SHAPE, "block %d is not a multiple of tile %d", block, tile);
    if (!n_qtiles || !nnz) return fail(PA_ERR_INVALID_ARG, "n_qtiles and nnz must be non-null");
    const int32_t r = block / tile;
    const int64_t nqt = (seq_len + tile - 1) / tile;
    if (nqt >= INT32_MAX) return fail(PA_ERR_SHAPE, "n_qtiles %lld does not fit in int32", (long long)nqt);
    // Tiles of one block share the block's row length; their diagonal parts are 1, 2, ..., r.
    int64_t total = 0;
    for (int64_t i = 0; i * r < nqt; ++i) {
        const int64_t tiles = nqt - i * r < r ? nqt - i * r : r;  // the last block may be cut short
        total += tiles * r * (int64_t)(row_length(i, window_blocks, sink_blocks) - 1) + tiles * (tiles + 1) / 2;
    }
    if (total > INT32_MAX) return fail(PA_ERR_SHAPE, "nnz %lld does not fit in int32", (long long)total);
    *n_qtiles = (int32_t)nqt;
    *nnz = total;
    return PA_OK;
}

extern "C" pa_status pa_build_tile_layout(int64_t seq_len, int32_t block, int32_t window_blocks,
                                          int32_t sink_blocks, int32_t tile, int32_t *row_ptr,
                                          int32_t *col_idx, int64_t col_capacity, void *stream)
{
    using namespace pa;
    clear_error();
    int32_t nqt = 0;
    int64_t nnz = 0;
    if (pa_status s = pa_tile_layout_size(seq_len, block, window_blocks, sink_blocks, tile, &nqt, &nnz)) return s;
    if (!row_ptr || !col_idx) return fail(PA_ERR_INVALID_ARG, "row_ptr and col_idx must be non-null");
    if (col_capacity < nnz)
        return fail(PA_ERR_LAYOUT, "col_capacity %lld < nnz %lld", (long long)col_capacity, (long long)nnz);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int threads = 256;
    const unsigned blocks = (unsigned)((nqt + threads - 1) / threads);
    const int32_t r = block / tile;
    tile_layout_count_kernel<<<blocks, threads, 0, st>>>(nqt, r, window_blocks, sink_blocks, row_ptr);
    layout_scan_kernel<<<1, 1024, 0, st>>>(nqt, row_ptr);
    tile_layout_fill_kernel<<<blocks, threads, 0, st>>>(nqt, r, window_blocks, sink_blocks, row_ptr, col_idx);
    PA_CUDA_OK(cudaGetLastError());
    return PA_OK;
}
