/*
 * powerattn.h -- C ABI of the PowerAttention block-sparse attention library for NVIDIA B200
 * (sm_100a).
 *
 * The library computes causal block-sparse attention under the static mask of PowerAttention
 * (arXiv 2503.03588): every query block attends to the key blocks at power-of-two block
 * distances, to a local window of recent blocks and to the first ("sink") blocks.
 *
 * General conventions
 *   - Every buffer is owned by the caller.  No entry point allocates or frees device memory
 *     unless its comment says otherwise; scratch is passed in as `workspace`.
 *   - "device" pointers are CUDA device pointers valid on the current device; "host" pointers
 *     are ordinary process memory.  Each argument says which it is.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls
 *     only enqueue work on it; none synchronises unless its comment says so.
 *   - Tensors are bfloat16 unless stated; strides are in ELEMENTS; the head_dim axis is
 *     contiguous (stride 1) and every row start must be 16-byte aligned.
 *   - Grouped-query attention: query head h reads KV head floor(h / (n_q_heads / n_kv_heads)).
 *   - Failures are returned as a pa_status; nothing aborts and no kernel traps.  Argument
 *     checks run before any launch.  pa_last_error_message() gives a host-side description of
 *     the calling thread's most recent failure.
 */
#ifndef POWERATTN_H_
#define POWERATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PA_OK = 0,
    PA_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, bad enum                    */
    PA_ERR_SHAPE = 2,       /* unsupported head_dim / block / head grouping / strides       */
    PA_ERR_ALIGNMENT = 3,   /* a pointer or stride breaks the 16-byte rule                  */
    PA_ERR_LAYOUT = 4,      /* CSR arrays inconsistent with the problem (capacity, nnz)     */
    PA_ERR_WORKSPACE = 5,   /* workspace missing or smaller than the *_workspace_bytes size */
    PA_ERR_UNSUPPORTED = 6, /* the device is not an sm_100 GPU                              */
    PA_ERR_CUDA = 7,        /* a CUDA runtime / driver call failed                          */
    PA_ERR_TIMEOUT = 8      /* a bounded device-side wait gave up (see pa_prefill_status)   */
} pa_status;

const char *pa_status_string(pa_status s);
/* Host string describing the calling thread's last failing call ("" if none). */
const char *pa_last_error_message(void);
/* major * 10000 + minor * 100 + patch */
int pa_version(void);

/* Environment switches (PA_VALIDATE, PA_DECODE_PATH, PA_DECODE_CLUSTER, PA_DECODE_STAGES,
 * PA_DECODE_CTAS_PER_SM, PA_BACKWARD_PATH; each is
 * described at the call it affects) are read once, when a call first needs them.  This re-reads
 * them; tests and measurement scripts call it after changing the environment. */
void pa_reload_environment(void);

/* Limit, in GPU clock cycles, of every bounded barrier wait inside the prefill, backward and decode kernels
 * (a wait that runs out ends the kernel with PA_ERR_TIMEOUT in its status block, see
 * pa_prefill_status and pa_decode_status).  cycles <= 0 restores the defaults of one to two
 * seconds.  Process-wide; applies to calls made after it returns. */
void pa_set_wait_limit_cycles(int64_t cycles);

/* ------------------------------------------------------------------------------------------
 * Layout: Algorithm 1 (Section 3.3) evaluated on blocks.
 *
 * With equal, aligned query and key blocks of `block` tokens, key block j is listed for query
 * block i exactly when j <= i and ( i - j < window_blocks  or  (i - j) & (i - j - 1) == 0  or
 * j < sink_blocks ).  The paper's sink is one block (kv_idx < B); `sink_blocks` generalises it.
 * Distance 0 passes the power-of-two test, so the diagonal block is always listed and no row
 * is empty.  n_qblocks = ceil(seq_len / block).  Rows are ascending without duplicates; the
 * arrays are CSR: row i owns col_idx[row_ptr[i] .. row_ptr[i+1]).
 * ------------------------------------------------------------------------------------------ */

/* Host-only closed-form sizes.  n_qblocks, nnz: host pointers, written on success.
 * Errors: PA_ERR_INVALID_ARG (seq_len < 1, block < 1, window/sink < 0, null outputs),
 * PA_ERR_SHAPE (n_qblocks or nnz would not fit in int32). */
pa_status pa_layout_size(int64_t seq_len, int32_t block, int32_t window_blocks,
                         int32_t sink_blocks, int32_t *n_qblocks, int64_t *nnz);

/* Writes the CSR on the device.  row_ptr: device int32[n_qblocks + 1]; col_idx: device
 * int32[col_capacity], col_capacity >= nnz from pa_layout_size (else PA_ERR_LAYOUT, nothing
 * launched).  Three small kernels are enqueued on `stream`; no scratch memory is used. */
pa_status pa_build_layout(int64_t seq_len, int32_t block, int32_t window_blocks,
                          int32_t sink_blocks, int32_t *row_ptr, int32_t *col_idx,
                          int64_t col_capacity, void *stream);

/* The sliding-window comparison pattern of Section 3.2 / Section 4.1 ("Baseline": a local window
 * plus initial sink tokens; the paper's setting is a 9-block window and 1 sink block): Algorithm 1
 * without its power-of-two term, i.e. key block j is listed for query block i exactly when j <= i
 * and ( i - j < window_blocks  or  j < sink_blocks ).  window_blocks >= 1 is required so that the
 * diagonal block is listed (PA_ERR_INVALID_ARG otherwise); everything else as pa_layout_size /
 * pa_build_layout.  The CSR runs through pa_prefill like any other causal layout. */
pa_status pa_window_layout_size(int64_t seq_len, int32_t block, int32_t window_blocks,
                                int32_t sink_blocks, int32_t *n_qblocks, int64_t *nnz);
pa_status pa_build_window_layout(int64_t seq_len, int32_t block, int32_t window_blocks,
                                 int32_t sink_blocks, int32_t *row_ptr, int32_t *col_idx,
                                 int64_t col_capacity, void *stream);

/* Receptive field of a layout seen as a directed graph over blocks (Section 3.1; Appendix A):
 * counts[k-1] = |B_k|, the number of blocks that block `start` reaches within k steps along the
 * edges block -> listed key block, itself included, for k = 1 .. max_steps.  Appendix A's
 * theoretical accuracy is |B_k| / n_blocks with start = the last block (10/128 for the sliding
 * window of its worked example).  Host only: row_ptr [n_blocks + 1], col_idx and counts
 * [max_steps] are HOST pointers; nothing is launched.  Errors: PA_ERR_INVALID_ARG, PA_ERR_LAYOUT
 * (an index outside [0, n_blocks) or a negative row extent). */
pa_status pa_reach_counts(const int32_t *row_ptr, const int32_t *col_idx, int32_t n_blocks,
                          int32_t start, int32_t max_steps, int64_t *counts);

/* Tile layouts: the same mask listed at the granularity of the attention kernel.
 *
 * The paper's efficiency runs use 256-token blocks (Section 4.1, "Implementation"), the kernels
 * here walk 64-token tiles.  For `block` a multiple of `tile`, query tile ti (tokens
 * [ti tile, ti tile + tile)) lists key tile tj exactly when some token pair of the two tiles
 * passes Algorithm 1 evaluated with `block`: with i = ti tile / block and j = tj tile / block,
 * that is tj <= ti and block j is listed for block i.  Every listed block before the diagonal
 * one contributes all its tiles, the diagonal block its tiles up to ti.  The CSR has
 * n_qtiles = ceil(seq_len / tile) ascending rows and can be given to pa_prefill with
 * block = tile: the only pair that the kernel masks by token is tj == ti, which is the only
 * partial one here as well.  With tile == block this is pa_layout_size / pa_build_layout. */

/* Host-only closed-form sizes.  n_qtiles, nnz: host pointers, written on success.
 * Errors: as pa_layout_size, and PA_ERR_INVALID_ARG (tile < 1), PA_ERR_SHAPE (block is not a
 * multiple of tile). */
pa_status pa_tile_layout_size(int64_t seq_len, int32_t block, int32_t window_blocks,
                              int32_t sink_blocks, int32_t tile, int32_t *n_qtiles, int64_t *nnz);

/* Writes the tile CSR on the device.  row_ptr: device int32[n_qtiles + 1]; col_idx: device
 * int32[col_capacity], col_capacity >= nnz from pa_tile_layout_size (else PA_ERR_LAYOUT, nothing
 * launched).  Three small kernels are enqueued on `stream`; no scratch memory is used. */
pa_status pa_build_tile_layout(int64_t seq_len, int32_t block, int32_t window_blocks,
                               int32_t sink_blocks, int32_t tile, int32_t *row_ptr,
                               int32_t *col_idx, int64_t col_capacity, void *stream);

/* ------------------------------------------------------------------------------------------
 * Prefill: Eq. (1) (Section 3.1) over the listed key blocks of each query block.
 *
 *   s_kv = softmax_scale * <Q[b,q,h,:], K[b,kv,hk,:]>          for kv in the listed blocks,
 *   kv <= q inside the diagonal block (Algorithm 1's causal term), kv < seq_len;
 *   LSE[b,h,q] = ln sum_kv exp(s_kv);   O[b,q,h,:] = sum_kv exp(s_kv - LSE) V[b,kv,hk,:].
 *
 * The kernel accepts ANY causal CSR whose rows are ascending and hold only cols <= row: the
 * PowerAttention layout, dense causal, sliding window.  It applies token-level causality to the
 * diagonal pair (col == row, which if listed is the row's last entry) and the seq_len bound
 * itself.  A row may be empty: its query tokens get O = 0 and LSE = -inf.
 * Arithmetic: bf16 operands, fp32 accumulation (tensor cores), fp32 softmax; O rounded to
 * bf16 or kept fp32; LSE fp32.
 * ------------------------------------------------------------------------------------------ */

typedef enum { PA_BF16 = 0, PA_F32 = 1 } pa_dtype;

/* Element strides of a [batch, seq, head, head_dim] tensor; head_dim stride is 1. */
typedef struct {
    int64_t batch, seq, head;
} pa_strides;

typedef struct {
    int32_t batch, n_q_heads, n_kv_heads, head_dim; /* head_dim in {64, 128}              */
    int64_t seq_len;                                /* same for queries and keys          */
    int32_t block;                                  /* tokens per block; must be 64       */
    float softmax_scale;                            /* 0 => 1 / sqrt(head_dim)            */
    pa_strides q, k, v, o;
    pa_dtype o_dtype;
} pa_prefill_params;

/* Bytes of device scratch pa_prefill needs (a status block; 16-byte aligned start). */
size_t pa_prefill_workspace_bytes(const pa_prefill_params *p);

/* q, k, v: device bf16, read-only.  row_ptr [ceil(seq_len/block) + 1], col_idx [nnz]: device
 * int32 CSR, shared by every batch entry and head (the mask does not depend on them).
 * o: device, o_dtype, strides p->o.  lse: device fp32 [batch, n_q_heads, seq_len] contiguous.
 * workspace: device, >= pa_prefill_workspace_bytes(p); cleared by the call itself.
 * Enqueues one memset and one kernel.  Errors: PA_ERR_INVALID_ARG, PA_ERR_SHAPE,
 * PA_ERR_ALIGNMENT, PA_ERR_LAYOUT (nnz outside [0, 2^31)), PA_ERR_WORKSPACE, PA_ERR_UNSUPPORTED,
 * PA_ERR_CUDA.  Outputs are undefined after a failure.  The CSR is trusted: extents that point
 * outside col_idx would be read out of bounds.  With PA_VALIDATE=1 in the environment (see
 * pa_reload_environment) the call
 * first checks it on the device (row_ptr from 0 to nnz, extents inside col_idx, every index in
 * [0, row] and ascending within its row), synchronises the stream, and returns PA_ERR_LAYOUT with
 * the first offending row in pa_last_error_message() instead of enqueuing the kernel; do not
 * use that switch while capturing the stream. */
pa_status pa_prefill(const pa_prefill_params *p, const void *q, const void *k, const void *v,
                     const int32_t *row_ptr, const int32_t *col_idx, int64_t nnz, void *o,
                     float *lse, void *workspace, size_t workspace_bytes, void *stream);

/* Variable-length batch: the sequences are packed one after the other along the token axis
 * (Algorithm 1's mask takes no batch argument: every sequence uses the same layout, cut off at
 * its own length).  q [total_tokens, n_q_heads, head_dim], k, v [total_tokens, n_kv_heads,
 * head_dim] by the .seq and .head strides of p (the .batch strides are ignored); cu_seqlens:
 * device int32 [p->batch + 1], ascending, cu_seqlens[0] = 0, cu_seqlens[batch] = total_tokens:
 * sequence b owns tokens [cu_seqlens[b], cu_seqlens[b+1]).  p->seq_len is the length of the longest
 * sequence (an upper bound is fine; query tokens of a sequence beyond it get no output), and the
 * CSR has at least ceil(p->seq_len / block) rows: row i serves query block i of every sequence.
 * o as q (n_q_heads heads); lse: device fp32 [n_q_heads, total_tokens].  A sequence's last block is
 * written row by row so that the next sequence's rows stay untouched; empty sequences are allowed.
 * Everything else as pa_prefill. */
pa_status pa_prefill_varlen(const pa_prefill_params *p, const void *q, const void *k, const void *v,
                            const int32_t *cu_seqlens, int64_t total_tokens, const int32_t *row_ptr,
                            const int32_t *col_idx, int64_t nnz, void *o, float *lse, void *workspace,
                            size_t workspace_bytes, void *stream);

/* Synchronises `stream` and reads back the status block a pa_prefill call left in `workspace`.
 * Returns PA_OK, PA_ERR_TIMEOUT (a bounded barrier wait inside the kernel ran out; *detail, a
 * host pointer that may be NULL, receives a code naming the wait) or PA_ERR_CUDA. */
pa_status pa_prefill_status(const void *workspace, void *stream, int32_t *detail);

/* ------------------------------------------------------------------------------------------
 * Backward of the prefill (the paper trains with its mask, Section 4.1 "Implementation"; it prints no
 * gradient formulas: these are the derivatives of Eq. (1)).  With P = exp(s - LSE) on the attended
 * pairs and dO the gradient of the output:
 *   delta_q = <dO_q, O_q>;   dV_kv = sum_q P dO_q;   dS = P (<dO_q, V_kv> - delta_q);
 *   dQ_q = softmax_scale sum_kv dS K_kv;   dK_kv = softmax_scale sum_q dS Q_q,
 * dK and dV summed over the query heads of the KV head's group as well.
 *
 * p, q, k, v, row_ptr, col_idx, nnz: as given to pa_prefill (o_dtype must be PA_BF16); o, lse: what
 * pa_prefill returned; d_o: device bf16 with the strides of o.  dq: device fp32 [batch, seq_len,
 * n_q_heads, head_dim] contiguous; dk, dv: device fp32 [batch, seq_len, n_kv_heads, head_dim]
 * contiguous (cleared by the call).  workspace: device, 256-byte aligned,
 * >= pa_prefill_backward_workspace_bytes(p, nnz) (a status block, the row sums delta and the
 * transposed layout).  Three memsets and seven kernels are enqueued.  S and P are recomputed tile by
 * tile on the tensor cores (bf16 operands, fp32 accumulation): head_dim 128 on tcgen05 with
 * accumulators in tensor memory, head_dim 64 (and head_dim 128 under PA_BACKWARD_PATH=mma) on the
 * warp-level MMA.  A key block that many query blocks list (a sink block is listed by all) is spread
 * over several CTAs that add their parts with fp32 atomics, so dk and dv of such blocks may differ
 * in the last bits from run to run.
 * Errors: as pa_prefill.  The tcgen05 kernels bound their barrier waits like the prefill kernel;
 * pa_prefill_status(workspace, ...) on the backward workspace reports a wait that ran out.
 * ------------------------------------------------------------------------------------------ */
size_t pa_prefill_backward_workspace_bytes(const pa_prefill_params *p, int64_t nnz);
pa_status pa_prefill_backward(const pa_prefill_params *p, const void *q, const void *k, const void *v,
                              const void *o, const float *lse, const void *d_o, const int32_t *row_ptr,
                              const int32_t *col_idx, int64_t nnz, float *dq, float *dk, float *dv,
                              void *workspace, size_t workspace_bytes, void *stream);

/* ------------------------------------------------------------------------------------------
 * Decode: one query token per sequence against its KV cache (Section 4.1: the same pattern in
 * prefilling and decoding).  cache_lens[b] counts the cached keys INCLUDING the current token,
 * so the query sits at position p = cache_lens[b] - 1, attends to itself, and its key blocks
 * are row floor(p / block) of the layout; the last block holds (p mod block) + 1 keys.
 * The block list is derived in closed form inside the kernel (no CSR is read).
 * ------------------------------------------------------------------------------------------ */

typedef struct {
    int32_t batch, n_q_heads, n_kv_heads, head_dim; /* head_dim in {64, 128}; group <= 8   */
    int32_t block, window_blocks, sink_blocks;      /* block must be 64                    */
    int64_t max_len;                                /* cache capacity in tokens            */
    float softmax_scale;                            /* 0 => 1 / sqrt(head_dim)             */
    pa_strides k, v;                                /* cache [batch, max_len, n_kv_heads, D] */
    pa_dtype o_dtype;
} pa_decode_params;

/* Bytes of device scratch: a 256-byte status block, then the split-K partial results (m, l,
 * o[head_dim] per query head and chunk of the block list). */
size_t pa_decode_workspace_bytes(const pa_decode_params *p);

/* q: device bf16 [batch, n_q_heads, head_dim] contiguous.  k_cache, v_cache: device bf16 by
 * strides.  cache_lens: device int32 [batch], each in [1, max_len] (a length outside that
 * range makes the sequence's outputs zero and its LSE -inf; nothing faults).
 * o: device [batch, n_q_heads, head_dim] contiguous, o_dtype.  lse: device fp32
 * [batch, n_q_heads].  When a row's window, power-of-two and sink candidates number at most 32
 * (window_blocks + sink_blocks + log2 of the row count: any default-window row up to millions of
 * tokens) the row kernel runs: a row's key blocks are dealt to R chunks; in each CTA a producer
 * warp fetches the blocks of its chunk by TMA into a ring of shared-memory stages and four warps
 * run an online softmax over them.  Small calls (batch x n_kv_heads up to about 70) are one
 * launch in which the R CTAs of a row form a thread-block cluster and merge their results through
 * distributed shared memory with the log-sum-exp rule
 * m = max m_c, l = sum l_c e^(m_c - m), o = sum o_c e^(m_c - m) / l.  Larger calls run a
 * persistent grid (two CTAs per SM) over the (row, chunk) items and, unless R is 1, a second small
 * kernel that merges each row's R partial results from the workspace.  Rows with more candidates
 * take two kernels: partial attention per (sequence, KV head, block) into the workspace, then
 * the same merge.  The workspace (>= pa_decode_workspace_bytes(p), 16-byte aligned) must always
 * be given; its first word is a status block (see pa_decode_status).
 * Calls that share a workspace must not overlap on the GPU.  Environment switches (for tests and
 * measurements, see pa_reload_environment): PA_DECODE_PATH=splitk forces the two-kernel path,
 * =cluster / =persist the two forms of the row kernel; PA_DECODE_CLUSTER=n (1..8) sets R (default:
 * for small calls as many CTAs per row as run all at once, for large ones one chunk per row once
 * there are as many rows as SMs, else two); PA_DECODE_STAGES=n (1..6) the number of key blocks a CTA keeps
 * in flight; PA_DECODE_CTAS_PER_SM=n the size of the persistent grid (default 2 per SM). */
pa_status pa_decode(const pa_decode_params *p, const void *q, const void *k_cache,
                    const void *v_cache, const int32_t *cache_lens, void *o, float *lse,
                    void *workspace, size_t workspace_bytes, void *stream);

/* Synchronises `stream` and reads back the status block a decode call (pa_decode, pa_decode_paged)
 * left in `workspace`.  Returns PA_OK, PA_ERR_TIMEOUT (a bounded barrier wait inside the kernel
 * ran out; *detail, a host pointer that may be NULL, receives a code naming the wait) or
 * PA_ERR_CUDA. */
pa_status pa_decode_status(const void *workspace, void *stream, int32_t *detail);

/* The key-block list of one cache length as the two-kernel path derives it (ascending), written
 * on the device by the device function that path uses: out_blocks device int32[capacity],
 * out_count device int32[1].  Equals row floor((cache_len-1)/block) of pa_build_layout(cache_len,
 * ...).  capacity >= 64 + window_blocks + sink_blocks is always enough. */
pa_status pa_decode_block_list(int64_t cache_len, int32_t block, int32_t window_blocks,
                               int32_t sink_blocks, int32_t *out_blocks, int32_t *out_count,
                               int32_t capacity, void *stream);

/* The key-block SET of one cache length as the single-launch kernel derives it: that kernel
 * enumerates window, power-of-two and sink candidates one per lane and does not sort them (the
 * order of the keys does not matter for Eq. (1)).  Written by the kernel's own device function in
 * lane order: out_blocks device int32[capacity >= 32], out_count device int32[1].  As a set it
 * equals row floor((cache_len-1)/block) of pa_build_layout(cache_len, ...), without duplicates.
 * PA_ERR_SHAPE when the candidates number more than 32 (such rows take the two-kernel path). */
pa_status pa_decode_row_block_set(int64_t cache_len, int32_t block, int32_t window_blocks,
                                  int32_t sink_blocks, int32_t *out_blocks, int32_t *out_count,
                                  int32_t capacity, void *stream);

/* ------------------------------------------------------------------------------------------
 * Decode against a paged KV cache (Section 4.5 measures 16K-128K-token inputs followed by 1024
 * decoding steps; Section 4.1: the same pattern in both phases).  Keys and values live in a pool
 * of pages of `block` (= 64) tokens, [n_pages, block, n_kv_heads, head_dim] by strides
 * (k.batch / v.batch is the PAGE stride, .seq the token stride inside a page, .head the head
 * stride).  block_table[b, j] (device int32 [batch, max_blocks_per_seq]) is the page that holds
 * tokens [64 j, 64 j + 64) of sequence b, so a key block of the mask is exactly one page.  The
 * caller owns the pool and the table and decides which pages a sequence gets; the library
 * allocates nothing.
 * ------------------------------------------------------------------------------------------ */
typedef struct {
    int32_t batch, n_q_heads, n_kv_heads, head_dim; /* head_dim in {64, 128}; group <= 8    */
    int32_t block, window_blocks, sink_blocks;      /* block = page size, must be 64        */
    int32_t n_pages;                                /* pages in the pool                    */
    int32_t max_blocks_per_seq;                     /* row length of block_table            */
    float softmax_scale;                            /* 0 => 1 / sqrt(head_dim)              */
    pa_strides k, v;                                /* pool strides: page, token, head      */
    pa_dtype o_dtype;
} pa_paged_params;

size_t pa_decode_paged_workspace_bytes(const pa_paged_params *p);

/* As pa_decode, with the key blocks fetched through block_table.  cache_lens[b] in
 * [1, 64 * max_blocks_per_seq].  A table entry outside [0, n_pages) does not fault: on the
 * single-launch path that page reads as zeros, on the two-kernel path it is clamped into the
 * pool; the sequence's result is then meaningless. */
pa_status pa_decode_paged(const pa_paged_params *p, const void *q, const void *k_pool,
                          const void *v_pool, const int32_t *block_table,
                          const int32_t *cache_lens, void *o, float *lse, void *workspace,
                          size_t workspace_bytes, void *stream);

/* Appends one token per sequence: k_new, v_new (device bf16 [batch, n_kv_heads, head_dim]
 * contiguous) are written at position cache_lens[b] (the page block_table[b, cache_lens[b] / 64],
 * slot cache_lens[b] mod 64) and cache_lens[b] (device int32, read and written) grows by one.
 * A sequence whose table has no page for that position (position beyond 64 * max_blocks_per_seq,
 * or an entry outside [0, n_pages)) is left unchanged: nothing written, length kept.  Two small
 * kernels are enqueued on `stream`. */
pa_status pa_kv_append(const pa_paged_params *p, const void *k_new, const void *v_new,
                       void *k_pool, void *v_pool, const int32_t *block_table,
                       int32_t *cache_lens, void *stream);

/* ------------------------------------------------------------------------------------------
 * Decode without any allocation.  (The paper has no counterpart to this entry point; it exists
 * for integration reasons only.)
 *
 * Some hosts of this library are not allowed to obtain device memory at the moment they need to
 * decode: code that runs inside a memory-pool or allocator callback, plug-ins whose embedding
 * runtime owns every byte of the device and hands out none, and real-time serving loops in which
 * an allocation (which may synchronise the device or fail) is forbidden once warm-up is over.
 * pa_decode asks such callers for a workspace they have no means to provide.  pa_decode_static
 * computes exactly what pa_decode computes, but keeps the workspace (the status block and, on the
 * two-kernel path, the split-K partial results) in an array of PA_DECODE_STATIC_SCRATCH_BYTES
 * bytes that is part of the library image.  Every GPU on which the library's code gets loaded
 * carries that array until the process exits.
 *
 * Arguments q, k_cache, v_cache, cache_lens, o, lse and stream: as for pa_decode.
 *   - Limit: a problem that takes the two-kernel path (long windows, or PA_DECODE_PATH=splitk)
 *     needs pa_decode_workspace_bytes(p) bytes of the array; beyond
 *     PA_DECODE_STATIC_SCRATCH_BYTES the call returns PA_ERR_WORKSPACE (with a message giving both
 *     numbers) and launches nothing.  The batch-8, 28-head, head_dim-128, 128K-token workload
 *     would need about 2 MB there.  A problem that takes the single-launch path uses only the
 *     256-byte status block, whatever its size.
 *   - The call itself performs no device allocation or free, and calls no library that does.
 *   - The first call on each device looks up the array's device address (a one-time set-up that
 *     loads the library's device code if it is not loaded yet).  Make that first call during
 *     start-up, outside any stream capture.
 *   - All calls on one device share the one array, and it still holds the previous call's
 *     status and partial results when the next call starts.  The status word is cleared by the
 *     kernels themselves at their start; nothing else has to start at zero: each call overwrites
 *     every entry it later reads.  Because the array is shared, two calls that run
 *     on the GPU at the same time (different streams, or different host threads) overwrite each
 *     other's partial results; issue them on one stream or order them yourself.
 * ------------------------------------------------------------------------------------------ */
#define PA_DECODE_STATIC_SCRATCH_BYTES (4u << 20)

pa_status pa_decode_static(const pa_decode_params *p, const void *q, const void *k_cache,
                           const void *v_cache, const int32_t *cache_lens, void *o, float *lse,
                           void *stream);

#ifdef __cplusplus
}
#endif
#endif /* POWERATTN_H_ */
