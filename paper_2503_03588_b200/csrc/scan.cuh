// One-block prefix sum used by the layout writers and the backward pass's transposed layout.
#pragma once

#include <stdint.h>

namespace pa {

// In-place inclusive scan of row_ptr[1 .. nqb] by one block, tile by tile with a running carry.
static __global__ void layout_scan_kernel(int32_t nqb, int32_t *row_ptr)
{
    __shared__ int32_t warp_sums[32];
    __shared__ int32_t carry_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) carry_s = 0;
    __syncthreads();
    for (int64_t base = 0; base < nqb; base += blockDim.x) {
        const int64_t idx = base + tid;
        int32_t v = idx < nqb ? row_ptr[idx + 1] : 0;
        for (int o = 1; o < 32; o <<= 1) {
            int32_t t = __shfl_up_sync(0xffffffffu, v, o);
            if (lane >= o) v += t;
        }
        if (lane == 31) warp_sums[warp] = v;
        __syncthreads();
        if (warp == 0) {
            int32_t s = lane < (int)(blockDim.x >> 5) ? warp_sums[lane] : 0;
            for (int o = 1; o < 32; o <<= 1) {
                int32_t t = __shfl_up_sync(0xffffffffu, s, o);
                if (lane >= o) s += t;
            }
            warp_sums[lane] = s;
        }
        __syncthreads();
        const int32_t carry = carry_s;
        const int32_t before = warp > 0 ? warp_sums[warp - 1] : 0;
        if (idx < nqb) row_ptr[idx + 1] = carry + before + v;
        __syncthreads();
        if (tid == (int)blockDim.x - 1) carry_s = carry + before + v;
        __syncthreads();
    }
}

}  // namespace pa
