// Shared between the backward pass's two translation units: the argument block of its kernels and
// the entry of the tensor-core (tcgen05) kernels for head_dim 128.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"

namespace pa {

constexpr int kBwdBlk = 64;       // tokens per block
constexpr int kBwdChunk = 32;     // query blocks per CTA of the dK / dV kernels
constexpr size_t kBwdStatusBytes = 256;  // status block at the head of the workspace ([0] error code, [1] detail)

struct BackwardArgs {
    const __nv_bfloat16 *q, *k, *v, *o, *d_o;
    const float *lse;          // [batch, Hq, N]
    const int32_t *row_ptr, *col_idx;
    int32_t *status;           // [0] error code, [1] detail (bounded waits of the tensor-core kernels)
    float *delta;              // [batch, Hq, N]
    int32_t *col_ptr;          // [nqb + 1]: extents of the transposed lists
    int32_t *row_idx;          // [nnz]: query blocks that list each key block, ascending
    int32_t *chunk_ptr;        // [nqb + 1]: first chunk of each column
    float *dq, *dk, *dv;       // fp32, contiguous [batch, N, H, D]
    int64_t q_sb, q_ss, q_sh, k_sb, k_ss, k_sh, v_sb, v_ss, v_sh, o_sb, o_ss, o_sh;
    int64_t N;
    int32_t nqb, batch, Hq, Hkv, G;
    int32_t npairs;            // head pairs per KV group: ceil(G / 2)
    float scale, scale_log2;
    long long wait_cycles;     // limit of every barrier wait of the tensor-core kernels
};

// dQ, dK, dV for head_dim 128 on tcgen05 (delta and the transposed lists are already in the workspace).
pa_status launch_backward_sm100(const BackwardArgs &a, const pa_prefill_params *p, int64_t nnz, int device, int sms,
                                cudaStream_t st);

}  // namespace pa
