// Host side of the TMA tensor maps used by the prefill and decode kernels.
//
// Every tensor the kernels fetch by TMA is a bf16 [batch, seq, head, D] array given by element
// strides (D contiguous).  Its map orders the dimensions (feature, token, head, batch) so that a
// box of `box_heads` heads x 64 tokens x 64 features lands in shared memory as rows
// head * 64 + token of 128 bytes each, 128-byte swizzled.  Encoding a map costs a driver call of
// a microsecond or two, and a serving loop calls with the same buffers over and over, so encoded
// maps are kept in a small per-process cache keyed by everything that goes into them.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace pa {

struct TensorMapKey {
    const void *base;
    int64_t seq, stride_seq, stride_head, stride_batch;
    int32_t device, head_dim, heads, batch, box_heads, box_tokens;
};

// Encoded map for `key` (from the cache, or encoded now and cached).  Thread-safe.
pa_status get_tensor_map(const TensorMapKey &key, const char *what, CUtensorMap *out);

}  // namespace pa
