// Algorithm 1 (Section 3.3) on block indices: the ascending list of key blocks of one query
// block.  With equal, aligned query and key blocks the window and power-of-two terms depend on
// the block distance d = i - j only, the sink term on j, and causality on j <= i.  The listed
// set is the union of three ascending runs, merged here without duplicates:
//   sink    j = 0 .. min(S, i+1) - 1
//   power   j = i - 2^k for every 2^k <= i, k descending   (d = 0 is covered by the window run)
//   window  j = max(0, i - max(W,1) + 1) .. i              (d = 0 always passes: 0 & -1 == 0)
#pragma once

#include <stdint.h>

namespace pa {

// Calls emit(pos, j) for every listed key block j of query block i in ascending order and
// returns the row length.  i >= 0, W >= 0, S >= 0.  Index is int64_t, or int32_t where the block
// indices are known to fit (the decode kernel: a cheaper walk on its critical path).
// `power` false drops the power-of-two run: the sliding-window pattern (local window plus sink
// blocks, Section 3.2 / Section 4.1 "Baseline"), for which W >= 1 keeps the diagonal block listed.
template <typename Index, typename Emit>
__host__ __device__ inline int for_each_key_block_t(Index i, int32_t W, int32_t S, Emit emit, bool power = true)
{
    const Index w_eff = W > 1 ? (Index)W : (Index)1;
    const Index sink_end = (Index)S < i + 1 ? (Index)S : i + 1;  // sink run [0, sink_end)
    Index js = 0;                                                // sink cursor
    Index jw = i - w_eff + 1 > 0 ? i - w_eff + 1 : 0;            // window cursor .. i
    Index pw = 0;                                                // current power distance
    if (power && i >= 1) {
        pw = 1;
        while (pw <= i / 2) pw *= 2;                             // largest 2^k <= i
    }
    const Index kNone = sizeof(Index) == 8 ? (Index)INT64_MAX : (Index)INT32_MAX;
    int n = 0;
    while (true) {
        const Index a = js < sink_end ? js : kNone;
        const Index b = pw >= 1 ? i - pw : kNone;
        const Index c = jw <= i ? jw : kNone;
        Index j = a < b ? a : b;
        j = j < c ? j : c;
        if (j == kNone) break;
        emit(n, j);
        ++n;
        if (a == j) ++js;
        if (b == j) pw >>= 1;  // 2^k -> 2^(k-1) -> ... -> 1 -> 0 (exhausted)
        if (c == j) ++jw;
    }
    return n;
}

template <typename Emit>
__host__ __device__ inline int for_each_key_block(int64_t i, int32_t W, int32_t S, Emit emit, bool power = true)
{
    return for_each_key_block_t<int64_t>(i, W, S, emit, power);
}

struct NoEmit {
    __host__ __device__ void operator()(int, int64_t) const {}
};

__host__ __device__ inline int row_length(int64_t i, int32_t W, int32_t S, bool power = true)
{
    return for_each_key_block(i, W, S, NoEmit(), power);
}

}  // namespace pa
