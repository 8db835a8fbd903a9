"""GPU: pa_prefill against the fp64 oracle -- element by element on sizes the oracle finishes in
seconds, on sampled rows at the full workload sizes, plus closed-form checks at any size."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from util import compare

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pa():
    import paper_2503_03588_b200 as pa_

    return pa_


def _gpu_prefill(pa, Q, K, V, W, S, scale=0.0, o_dtype=torch.bfloat16, layout=None):
    N = Q.shape[1]
    rp, ci = layout if layout is not None else pa.pa_build_layout(N, 64, W, S)
    o, lse, ws = pa.pa_prefill(Q.cuda(), K.cuda(), V.cuda(), rp, ci, softmax_scale=scale, o_dtype=o_dtype)
    pa.pa_prefill_status(ws)   # synchronises; raises on a device-side timeout
    return o, lse


def _full_compare(pa, oracle, Q, K, V, W, S, scale=0.0, o_dtype=torch.bfloat16, what=""):
    o, lse = _gpu_prefill(pa, Q, K, V, W, S, scale, o_dtype)
    o_ref, lse_ref, _ = oracle.prefill(Q, K, V, 64, W, S, scale=scale if scale else None)
    return compare(o, lse, o_ref, lse_ref, what)


def test_tiny_config(pa, oracle):
    """Batch 1, 2/2 heads, seq 2048, head_dim 64, window 1, sink 1, scale 1/sqrt(64)."""
    w = si.TINY_PREFILL
    Q, K, V = si.prefill_inputs(w)
    st = _full_compare(pa, oracle, Q, K, V, w.window_blocks, w.sink_blocks, what=w.name)
    print(w.name, st)


@pytest.mark.parametrize("N,Hq,Hkv,D,W,S", [
    (64, 2, 2, 64, 5, 1),        # one block
    (1, 2, 1, 128, 5, 1),        # one token
    (200, 4, 2, 128, 5, 1),      # ragged tail
    (1000, 7, 1, 128, 5, 1),     # one full 7-head group, ragged
    (1536, 28, 4, 128, 5, 1),    # the 7B-like head shape
    (777, 8, 2, 64, 0, 0),       # pure power-of-two pattern
    (900, 6, 2, 128, 30, 2),     # window covers everything: dense causal
    (1300, 16, 2, 64, 3, 3),     # group of 8 (two full quads)
])
def test_small_shapes(pa, oracle, N, Hq, Hkv, D, W, S):
    Q = si.bf16_randn((2, N, Hq, D), 100 + N)
    K = si.bf16_randn((2, N, Hkv, D), 200 + N)
    V = si.bf16_randn((2, N, Hkv, D), 300 + N)
    _full_compare(pa, oracle, Q, K, V, W, S, what=f"N={N} Hq={Hq} Hkv={Hkv} D={D} W={W} S={S}")


def test_peaky_logits_fp32_output_and_custom_scale(pa, oracle):
    N, Hq, Hkv, D = 1500, 14, 2, 128
    Q, K, V = si.bf16_randn((1, N, Hq, D), 1), si.bf16_randn((1, N, Hkv, D), 2, 3.0), si.bf16_randn((1, N, Hkv, D), 3)
    _full_compare(pa, oracle, Q, K, V, 5, 1, what="peaky bf16")
    _full_compare(pa, oracle, Q, K, V, 5, 1, scale=0.05, o_dtype=torch.float32, what="fp32 out")


def test_strided_inputs(pa, oracle):
    """Q, K, V as head-slices of one fused QKV tensor (non-contiguous sequence stride)."""
    N, Hq, Hkv, D = 700, 8, 2, 128
    qkv = si.bf16_randn((1, N, Hq + 2 * Hkv, D), 5).cuda()
    Q, K, V = qkv[:, :, :Hq], qkv[:, :, Hq:Hq + Hkv], qkv[:, :, Hq + Hkv:]
    rp, ci = pa.pa_build_layout(N, 64, 5, 1)
    o, lse, ws = pa.pa_prefill(Q, K, V, rp, ci)
    pa.pa_prefill_status(ws)
    o_ref, lse_ref, _ = oracle.prefill(Q.cpu().contiguous(), K.cpu().contiguous(), V.cpu().contiguous(), 64, 5, 1)
    compare(o, lse, o_ref, lse_ref, "strided")


def test_other_causal_layouts_through_the_same_kernel(pa, oracle):
    """Dense causal and sliding-window CSRs (built on the host here) run through pa_prefill."""
    N, Hq, Hkv, D = 1100, 8, 2, 128
    Q, K, V = si.bf16_randn((1, N, Hq, D), 7), si.bf16_randn((1, N, Hkv, D), 8), si.bf16_randn((1, N, Hkv, D), 9)
    for use_power, W, S in [(False, 18, 0), (False, 4, 1)]:
        rp, ci = oracle.block_layout(N, 64, W, S, use_power=use_power)
        layout = (torch.as_tensor(rp).cuda(), torch.as_tensor(ci).cuda())
        o, lse = _gpu_prefill(pa, Q, K, V, W, S, layout=layout)
        o_ref, lse_ref, _ = oracle.prefill(Q, K, V, 64, W, S, use_power=use_power)
        compare(o, lse, o_ref, lse_ref, f"use_power={use_power} W={W}")


@pytest.mark.parametrize("N,Hq,Hkv,D,B,W,S", [
    (1500, 7, 1, 128, 256, 5, 1),     # window covers the whole sequence at this size: dense causal
    (3000, 14, 2, 128, 256, 2, 1),    # ragged tail, power-of-two distances 1, 2, 4, 8 in blocks
    (2100, 4, 2, 64, 128, 1, 0),      # 128-token blocks, no sink
    (2048, 8, 2, 128, 256, 0, 0),     # pure power-of-two pattern
])
def test_mask_blocks_larger_than_the_tile(pa, oracle, N, Hq, Hkv, D, B, W, S):
    """The paper's block size (256 tokens, Section 4.1) and other multiples of the kernel's
    64-token tile: the tile CSR of pa_build_tile_layout through pa_prefill against the oracle,
    which applies the token-level predicate with that block size."""
    Q = si.bf16_randn((1, N, Hq, D), 400 + N)
    K = si.bf16_randn((1, N, Hkv, D), 500 + N)
    V = si.bf16_randn((1, N, Hkv, D), 600 + N)
    layout = pa.pa_build_tile_layout(N, B, W, S, 64)
    o, lse = _gpu_prefill(pa, Q, K, V, W, S, layout=layout)
    o_ref, lse_ref, _ = oracle.prefill(Q, K, V, B, W, S)
    compare(o, lse, o_ref, lse_ref, f"B={B} N={N} W={W} S={S}")


def test_paper_block_size_at_32k_on_sampled_rows(pa, oracle):
    """32K tokens in 256-token blocks (the paper's efficiency setting) with the 7B-like heads."""
    w = si.PREFILL_32K
    Q, K, V = si.prefill_inputs(w)
    layout = pa.pa_build_tile_layout(w.seq_len, 256, w.window_blocks, w.sink_blocks, 64)
    o, lse = _gpu_prefill(pa, Q, K, V, w.window_blocks, w.sink_blocks, layout=layout)
    rows = _sampled_rows(w.seq_len, np.random.default_rng(w.seed + 7), n_random=48)
    o_ref, lse_ref, _ = oracle.prefill(Q, K, V, 256, w.window_blocks, w.sink_blocks, rows=rows)
    ridx = torch.as_tensor(rows).cuda()
    compare(o[:, ridx], lse[:, :, ridx], o_ref, lse_ref, "32K, 256-token blocks")


@pytest.mark.parametrize("W", [1, 2, 3])
def test_short_rows_with_several_units_per_cta(pa, oracle, W):
    """Rows of one, two or three blocks on a sequence long enough that every CTA of the
    persistent grid walks several work units: the unit-to-unit hand-overs (Q buffers reloaded
    behind the staged output, first and last step falling together) with nothing in between."""
    N, Hq, Hkv, D = 64 * 200 + 17, 8, 2, 128        # 201 query blocks x 2 KV heads = 402 units
    Q = si.bf16_randn((1, N, Hq, D), 700 + W)
    K = si.bf16_randn((1, N, Hkv, D), 710 + W)
    V = si.bf16_randn((1, N, Hkv, D), 720 + W)
    rp, ci = oracle.block_layout(N, 64, W, 0, use_power=False)
    assert int(np.diff(rp).max()) == W
    layout = (torch.as_tensor(rp).cuda(), torch.as_tensor(ci).cuda())
    o, lse = _gpu_prefill(pa, Q, K, V, W, 0, layout=layout)
    o_ref, lse_ref, _ = oracle.prefill(Q, K, V, 64, W, 0, use_power=False)
    compare(o, lse, o_ref, lse_ref, f"short rows W={W}")


def test_constant_keys_count_the_attended_tokens(pa, oracle):
    """K rows all equal => LSE_q - s_q = ln |A_q|, |A_q| = 64 * #blocks(row) - (63 - q mod 64);
    holds at any size, so it is checked at 32K with the 7B-like heads."""
    N, Hq, Hkv, D, W, S = 32768, 28, 4, 128, 5, 1
    krow = si.bf16_randn((D,), 41)
    K = krow.expand(1, N, Hkv, D).contiguous()
    Q, V = si.bf16_randn((1, N, Hq, D), 42), si.bf16_randn((1, N, Hkv, D), 43)
    o, lse = _gpu_prefill(pa, Q, K, V, W, S)
    rp, _ = oracle.block_layout(N, 64, W, S)
    nblk = np.diff(rp).astype(np.int64)
    qpos = np.arange(N)
    n_att = 64 * nblk[qpos // 64] - (63 - qpos % 64)
    s = (Q[0].double() @ krow.double()).numpy() / np.sqrt(D)          # [N, Hq]
    got = lse[0].double().cpu().numpy().T                              # [N, Hq]
    assert np.abs(got - s - np.log(n_att)[:, None]).max() < 1e-3
    # V constant => every output row equals it (sum of weights is 1)
    vrow = si.bf16_randn((D,), 44)
    Vc = vrow.expand(1, N, Hkv, D).contiguous()
    o, _ = _gpu_prefill(pa, Q, si.bf16_randn((1, N, Hkv, D), 45), Vc, W, S)
    assert (o[0].float().cpu() - vrow.float()).abs().max() < 2e-2


def _sampled_rows(N, rng, n_random=96):
    """Query positions spanning the first and last blocks, power-of-two block boundaries and a
    seeded random sample."""
    rows = {0, 1, 63, 64, 65, N - 1, N - 64, N - 65}
    k = 1
    while 64 * k < N:
        for off in (-1, 0, 1, 37):
            r = 64 * k + off
            if 0 <= r < N:
                rows.add(r)
        k *= 2
    rows.update(int(x) for x in rng.integers(0, N, n_random))
    return sorted(rows)


@pytest.mark.parametrize("w", [si.PREFILL_32K, si.PREFILL_128K], ids=lambda w: w.name)
def test_full_size_workloads_on_sampled_rows(pa, oracle, w):
    """The benchmark's launch configuration; the oracle evaluates sampled query rows, all heads."""
    Q, K, V = si.prefill_inputs(w)
    o, lse = _gpu_prefill(pa, Q, K, V, w.window_blocks, w.sink_blocks)
    rows = _sampled_rows(w.seq_len, np.random.default_rng(w.seed))
    o_ref, lse_ref, _ = oracle.prefill(Q, K, V, 64, w.window_blocks, w.sink_blocks, rows=rows)
    ridx = torch.as_tensor(rows).cuda()
    st = compare(o[:, ridx], lse[:, :, ridx], o_ref, lse_ref, w.name)
    print(w.name, st)
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()


def test_repeated_launches_agree_bit_for_bit(pa):
    """The kernel's arithmetic does not depend on timing (every row is reduced in list order by one
    thread), so launches on the same inputs must agree exactly: a hand-over that sometimes lets a
    tile be read early or overwritten late shows up as a difference.  128K with the default
    layout (rows of 13-14 blocks) and 64K with 256-token blocks (rows of about 40 tiles), where
    the constant-V property (every output row equals that V row) is checked on every row too."""
    w = si.PREFILL_128K
    Q, K, V = (t.cuda() for t in si.prefill_inputs(w))
    rp, ci = pa.pa_build_layout(w.seq_len, 64, w.window_blocks, w.sink_blocks)
    o0, lse0, ws = pa.pa_prefill(Q, K, V, rp, ci)
    pa.pa_prefill_status(ws)
    for _ in range(3):
        o1, lse1, ws1 = pa.pa_prefill(Q, K, V, rp, ci)
        pa.pa_prefill_status(ws1)
        assert torch.equal(o0, o1) and torch.equal(lse0, lse1)
    del o0, o1, lse0, lse1
    N = 65536
    Q, K = Q[:, :N].contiguous(), K[:, :N].contiguous()
    vrow = si.bf16_randn((w.head_dim,), 46)
    Vc = vrow.expand(1, N, w.n_kv_heads, w.head_dim).contiguous().cuda()
    rp, ci = pa.pa_build_tile_layout(N, 256, w.window_blocks, w.sink_blocks, 64)
    o0, lse0, ws = pa.pa_prefill(Q, K, Vc, rp, ci)
    pa.pa_prefill_status(ws)
    assert (o0[0].float() - vrow.float().cuda()).abs().max() < 2e-2
    o1, lse1, ws1 = pa.pa_prefill(Q, K, Vc, rp, ci)
    pa.pa_prefill_status(ws1)
    assert torch.equal(o0, o1) and torch.equal(lse0, lse1)


def test_csr_check_switch_rejects_malformed_layouts(pa, pa_env):
    """PA_VALIDATE=1 makes pa_prefill check the caller's CSR on the device before any attention
    work: each kind of violation comes back as PA_ERR_LAYOUT, and a good layout still runs."""
    pa_env(PA_VALIDATE="1")
    N, Hq, Hkv, D = 1024, 4, 2, 64
    Q = si.bf16_randn((1, N, Hq, D), 51).cuda()
    K = si.bf16_randn((1, N, Hkv, D), 52).cuda()
    V = si.bf16_randn((1, N, Hkv, D), 53).cuda()
    rp, ci = pa.pa_build_layout(N, 64, 2, 1)
    pa.pa_prefill(Q, K, V, rp, ci)  # passes the check
    torch.cuda.synchronize()

    def expect_layout_error(rp_bad, ci_bad):
        with pytest.raises(pa.PaError) as err:
            pa.pa_prefill(Q, K, V, rp_bad, ci_bad)
        assert "PA_ERR_LAYOUT" in str(err.value) or "CSR check" in str(err.value)

    bad = ci.clone(); bad[int(rp[5])] = 9          # a block after the row (non-causal)
    expect_layout_error(rp, bad)
    bad = ci.clone(); bad[int(rp[7]) + 1] = bad[int(rp[7])]  # not ascending
    expect_layout_error(rp, bad)
    bad = rp.clone(); bad[3] = bad[4] + 1           # negative extent
    expect_layout_error(bad, ci)
    bad = rp.clone(); bad[0] = 1                    # does not start at 0
    expect_layout_error(bad, ci)


@pytest.mark.parametrize("o_dtype", [torch.bfloat16, torch.float32])
def test_strided_output_is_written_only_inside_its_view(pa, oracle, o_dtype):
    """O as a view into a larger buffer (extra heads, extra tokens, extra batch stride), with a
    ragged last query block and a 7-head group (one padded head in the kernel's tiles): the view
    holds the result, every element of the buffer outside it keeps its sentinel."""
    N, Hq, Hkv, D = 1000, 7, 1, 128
    Q, K, V = si.bf16_randn((2, N, Hq, D), 61), si.bf16_randn((2, N, Hkv, D), 62), si.bf16_randn((2, N, Hkv, D), 63)
    big = torch.full((2, N + 100, Hq + 3, D), 7.0, dtype=o_dtype, device="cuda")
    o_view = big[:, :N, 1:1 + Hq]
    rp, ci = pa.pa_build_layout(N, 64, 5, 1)
    o, lse, ws = pa.pa_prefill(Q.cuda(), K.cuda(), V.cuda(), rp, ci, o=o_view, o_dtype=o_dtype)
    pa.pa_prefill_status(ws)
    o_ref, lse_ref, _ = oracle.prefill(Q, K, V, 64, 5, 1)
    compare(o_view, lse, o_ref, lse_ref, "strided output")
    outside = torch.ones_like(big, dtype=torch.bool)
    outside[:, :N, 1:1 + Hq] = False
    assert bool((big[outside] == 7.0).all()), "elements outside the output view were overwritten"


@pytest.mark.parametrize("o_dtype", [torch.bfloat16, torch.float32])
def test_variable_length_batch(pa, oracle, o_dtype):
    """Sequences of 1, 63, 64, 65, 0, 5000 and 32768 tokens packed into one call (Algorithm 1 takes no
    batch argument: one layout serves them all).  Oracle side: one sequence at a time.  The output
    buffer has sentinel rows behind the last token and every sequence's neighbours are checked
    by the element-wise comparison itself (a box store over a ragged last block would show there)."""
    Hq, Hkv, D, W, S = 8, 2, 128, 5, 1
    lens = [1, 63, 64, 65, 0, 5000, 32768]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    total = int(cu[-1])
    Q = si.bf16_randn((total, Hq, D), 801)
    K = si.bf16_randn((total, Hkv, D), 802, 2.0)
    V = si.bf16_randn((total, Hkv, D), 803)
    rp, ci = pa.pa_build_layout(max(lens), 64, W, S)
    big = torch.full((total + 70, Hq, D), 7.0, dtype=o_dtype, device="cuda")
    o, lse, ws = pa.pa_prefill_varlen(Q.cuda(), K.cuda(), V.cuda(), torch.as_tensor(cu).cuda(), max(lens), rp, ci,
                                      o=big[:total], o_dtype=o_dtype)
    pa.pa_prefill_status(ws)
    assert bool((big[total:] == 7.0).all()), "rows behind the last sequence were overwritten"
    for b, n in enumerate(lens):
        if n == 0:
            continue
        a, e = int(cu[b]), int(cu[b + 1])
        o_ref, lse_ref, _ = oracle.prefill(Q[None, a:e], K[None, a:e], V[None, a:e], 64, W, S)
        compare(o[None, a:e], lse[None, :, a:e], o_ref, lse_ref, f"sequence {b} of {n} tokens")


def test_variable_length_batch_equals_one_call_per_sequence(pa):
    """Bit for bit: the packed call and separate pa_prefill calls run the same arithmetic per row."""
    Hq, Hkv, D, W, S = 28, 4, 128, 5, 1
    lens = [3000, 130, 4096, 777]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    total = int(cu[-1])
    Q, K, V = (si.bf16_randn((total, h, D), 810 + i).cuda() for i, h in enumerate((Hq, Hkv, Hkv)))
    rp, ci = pa.pa_build_layout(max(lens), 64, W, S)
    o, lse, ws = pa.pa_prefill_varlen(Q, K, V, torch.as_tensor(cu).cuda(), max(lens), rp, ci)
    pa.pa_prefill_status(ws)
    for b, n in enumerate(lens):
        a, e = int(cu[b]), int(cu[b + 1])
        rp1, ci1 = pa.pa_build_layout(n, 64, W, S)
        o1, lse1, ws1 = pa.pa_prefill(Q[None, a:e], K[None, a:e], V[None, a:e], rp1, ci1)
        pa.pa_prefill_status(ws1)
        assert torch.equal(o1[0], o[a:e]) and torch.equal(lse1[0], lse[:, a:e])


def test_rows_the_layout_leaves_empty(pa, oracle):
    """A caller's CSR may list nothing for a query block: its rows get O = 0 and LSE = -inf, the
    other rows are untouched by it (oracle: the dense token mask that the CSR stands for)."""
    N, Hq, Hkv, D = 700, 8, 2, 128
    nqb = (N + 63) // 64
    rp_full, ci_full = oracle.block_layout(N, 64, 5, 1)
    empty = {0, 3, 4, nqb - 1}
    rows = [[] if i in empty else ci_full[rp_full[i]:rp_full[i + 1]].tolist() for i in range(nqb)]
    rp = np.concatenate([[0], np.cumsum([len(r) for r in rows])]).astype(np.int32)
    ci = np.asarray([j for r in rows for j in r], dtype=np.int32)
    dense = np.zeros((N, N), dtype=bool)
    for i, r in enumerate(rows):
        for j in r:
            dense[i * 64:(i + 1) * 64, j * 64:(j + 1) * 64] = True
    dense &= np.tril(np.ones((N, N), dtype=bool))
    Q, K, V = si.bf16_randn((1, N, Hq, D), 821), si.bf16_randn((1, N, Hkv, D), 822), si.bf16_randn((1, N, Hkv, D), 823)
    o, lse, ws = pa.pa_prefill(Q.cuda(), K.cuda(), V.cuda(), torch.as_tensor(rp).cuda(), torch.as_tensor(ci).cuda())
    pa.pa_prefill_status(ws)
    o_ref, lse_ref, cnt = oracle.prefill(Q, K, V, 64, 5, 1, dense=dense)
    dead = np.array([q // 64 in empty for q in range(N)])
    assert (cnt[dead] == 0).all() and (cnt[~dead] > 0).all()
    assert (o[0, dead] == 0).all() and torch.isinf(lse[0, :, dead]).all() and (lse[0, :, dead] < 0).all()
    live = torch.as_tensor(np.nonzero(~dead)[0]).cuda()
    compare(o[:, live], lse[:, :, live], o_ref[:, ~dead], lse_ref[:, :, ~dead], "rows beside empty ones")


def test_batch_of_two_at_32k_on_sampled_rows(pa, oracle):
    """Batch 2 at the 32K workload's shape: the unit grid spans both batch entries."""
    w = si.PREFILL_32K
    Q = si.bf16_randn((2, w.seq_len, w.n_q_heads, w.head_dim), 831)
    K = si.bf16_randn((2, w.seq_len, w.n_kv_heads, w.head_dim), 832, 2.0)
    V = si.bf16_randn((2, w.seq_len, w.n_kv_heads, w.head_dim), 833)
    o, lse = _gpu_prefill(pa, Q, K, V, w.window_blocks, w.sink_blocks)
    rows = _sampled_rows(w.seq_len, np.random.default_rng(834), n_random=40)
    o_ref, lse_ref, _ = oracle.prefill(Q, K, V, 64, w.window_blocks, w.sink_blocks, rows=rows)
    ridx = torch.as_tensor(rows).cuda()
    compare(o[:, ridx], lse[:, :, ridx], o_ref, lse_ref, "batch 2 at 32K")


def test_head_dim_64_at_32k_on_sampled_rows(pa, oracle):
    N, Hq, Hkv, D = 32768, 16, 4, 64
    Q, K, V = si.bf16_randn((1, N, Hq, D), 841), si.bf16_randn((1, N, Hkv, D), 842, 2.0), si.bf16_randn((1, N, Hkv, D), 843)
    o, lse = _gpu_prefill(pa, Q, K, V, 5, 1)
    rows = _sampled_rows(N, np.random.default_rng(844), n_random=64)
    o_ref, lse_ref, _ = oracle.prefill(Q, K, V, 64, 5, 1, rows=rows)
    ridx = torch.as_tensor(rows).cuda()
    compare(o[:, ridx], lse[:, :, ridx], o_ref, lse_ref, "head_dim 64 at 32K")


def _row_matched_window(rp_pa):
    """The sweep's comparison layout: row i lists block 0 and its most recent blocks, as many as
    the PowerAttention row has (so both layouts have the same number of active block pairs)."""
    cols, cnts = [], np.diff(rp_pa)
    for i, cnt in enumerate(cnts):
        recent = list(range(max(1, i - (int(cnt) - 1) + 1), i + 1))
        row = sorted(set([0] + recent))
        lo = max(1, i - (int(cnt) - 1) + 1)
        while len(row) < min(int(cnt), i + 1):      # early rows where the sink falls inside the window
            lo -= 1
            row = sorted(set(row + [lo]))
        cols.append(row)
    rp = np.concatenate([[0], np.cumsum([len(c) for c in cols])]).astype(np.int32)
    return rp, np.asarray([j for c in cols for j in c], dtype=np.int32), cols


def test_sweep_lengths_and_comparison_masks_on_sampled_rows(pa, oracle):
    """The sequence-length sweep's other points, each at its own size on sampled rows: 256K with the
    PowerAttention layout and with the row-matched sliding window, 16K with dense causal, and the
    short ends (4K, 8K, 64K) with the PowerAttention layout."""
    for N in (4096, 8192, 65536):
        w = si.sweep_workload(N)
        Q, K, V = si.prefill_inputs(w)
        o, lse = _gpu_prefill(pa, Q, K, V, w.window_blocks, w.sink_blocks)
        rows = _sampled_rows(N, np.random.default_rng(w.seed), n_random=32)
        o_ref, lse_ref, _ = oracle.prefill(Q, K, V, 64, w.window_blocks, w.sink_blocks, rows=rows)
        ridx = torch.as_tensor(rows).cuda()
        compare(o[:, ridx], lse[:, :, ridx], o_ref, lse_ref, w.name)
    # dense causal at 16K: the window covers every block
    w = si.sweep_workload(16384)
    Q, K, V = si.prefill_inputs(w)
    nqb = w.seq_len // 64
    rp, ci = oracle.block_layout(w.seq_len, 64, nqb, 0, use_power=False)
    assert int(rp[-1]) == nqb * (nqb + 1) // 2
    o, lse = _gpu_prefill(pa, Q, K, V, nqb, 0, layout=(torch.as_tensor(rp).cuda(), torch.as_tensor(ci).cuda()))
    rows = _sampled_rows(w.seq_len, np.random.default_rng(w.seed), n_random=16)
    o_ref, lse_ref, _ = oracle.prefill(Q, K, V, 64, nqb, 0, use_power=False, rows=rows)
    ridx = torch.as_tensor(rows).cuda()
    compare(o[:, ridx], lse[:, :, ridx], o_ref, lse_ref, "dense causal at 16K")
    del Q, K, V, o, lse
    # 256K: the PowerAttention layout, then the row-matched window (per row: sink + a window of cnt - 1 blocks)
    w = si.sweep_workload(262144)
    Q, K, V = si.prefill_inputs(w)
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    rp_pa, ci_pa = pa.pa_build_layout(w.seq_len, 64, w.window_blocks, w.sink_blocks)
    o, lse, ws = pa.pa_prefill(Qd, Kd, Vd, rp_pa, ci_pa)
    pa.pa_prefill_status(ws)
    rows = _sampled_rows(w.seq_len, np.random.default_rng(w.seed), n_random=24)
    o_ref, lse_ref, _ = oracle.prefill(Q, K, V, 64, w.window_blocks, w.sink_blocks, rows=rows, heads=list(range(0, 28, 3)))
    ridx = torch.as_tensor(rows).cuda()
    hidx = torch.arange(0, 28, 3).cuda()
    compare(o[:, ridx][:, :, hidx], lse[:, hidx][:, :, ridx], o_ref, lse_ref, "256K PowerAttention")
    rp_w, ci_w, cols = _row_matched_window(rp_pa.cpu().numpy())
    assert int(rp_w[-1]) == int(rp_pa[-1])
    o, lse, ws = pa.pa_prefill(Qd, Kd, Vd, torch.as_tensor(rp_w).cuda(), torch.as_tensor(ci_w).cuda(), o=o, lse=lse, workspace=ws)
    pa.pa_prefill_status(ws)
    by_w = {}
    for q in rows:
        i = q // 64
        by_w.setdefault(len(cols[i]) - (1 if i >= len(cols[i]) else 0), []).append(q)   # window width in blocks
    for wblocks, qs in by_w.items():
        # rows whose window does not reach block 0 are "sink + window"; early rows are plain causal windows
        o_ref, lse_ref, _ = oracle.prefill(Q, K, V, 64, wblocks, 1, use_power=False, rows=qs, heads=[0, 13, 27])
        qidx, hsel = torch.as_tensor(qs).cuda(), torch.tensor([0, 13, 27]).cuda()
        compare(o[:, qidx][:, :, hsel], lse[:, hsel][:, :, qidx], o_ref, lse_ref, f"256K row-matched window of {wblocks}")


def test_a_wait_that_runs_out_ends_the_kernel_with_a_status(pa, oracle):
    """Every barrier wait inside the prefill kernel is bounded.  With the limit set to one cycle,
    an ordinary wait that is not over at its first try (the epilogue warps wait tens of
    microseconds for a row of 47 blocks to finish) runs out: the call returns, pa_prefill_status
    reports PA_ERR_TIMEOUT with the id of a wait, and the next call, back at the default limit, is
    correct on the same stream."""
    N, Hq, Hkv, D = 3000, 8, 2, 128
    Q, K, V = si.bf16_randn((1, N, Hq, D), 851), si.bf16_randn((1, N, Hkv, D), 852), si.bf16_randn((1, N, Hkv, D), 853)
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    rp, ci = pa.pa_build_window_layout(N, 64, 64, 0)     # the window covers every block: dense causal
    try:
        pa.pa_set_wait_limit_cycles(1)
        o, lse, ws = pa.pa_prefill(Qd, Kd, Vd, rp, ci)
        with pytest.raises(pa.PaError, match="PA_ERR_TIMEOUT") as err:
            pa.pa_prefill_status(ws)
        assert "wait id" in str(err.value)
    finally:
        pa.pa_set_wait_limit_cycles(0)
    o, lse, ws = pa.pa_prefill(Qd, Kd, Vd, rp, ci)
    assert pa.pa_prefill_status(ws) == 0
    o_ref, lse_ref, _ = oracle.prefill(Q, K, V, 64, 64, 0, use_power=False)
    compare(o, lse, o_ref, lse_ref, "after a timed-out call")


def test_kv_head_shards_reproduce_the_whole_call(pa):
    """Head sharding needs no exchange: the ranks' calls on head slices (run here one after the
    other on the one GPU; they do not depend on each other) write disjoint slices of O and LSE that
    agree bit for bit with the unsharded call."""
    from paper_2503_03588_b200.sharding import shard_prefill_tensors

    N, Hq, Hkv, D = 3000, 28, 4, 128
    Q, K, V = (si.bf16_randn((1, N, h, D), 860 + i).cuda() for i, h in enumerate((Hq, Hkv, Hkv)))
    rp, ci = pa.pa_build_layout(N, 64, 5, 1)
    o_full, lse_full, ws = pa.pa_prefill(Q, K, V, rp, ci)
    pa.pa_prefill_status(ws)
    for world in (2, 3, 4):
        o = torch.zeros_like(o_full)
        lse = torch.zeros_like(lse_full)
        for rank in range(world):
            qs_, ks_, vs_, heads = shard_prefill_tensors(Q, K, V, world, rank)
            o_r, lse_r, ws_r = pa.pa_prefill(qs_, ks_, vs_, rp, ci, o=o[:, :, heads])
            pa.pa_prefill_status(ws_r)
            lse[:, heads] = lse_r
        assert torch.equal(o, o_full) and torch.equal(lse, lse_full), world
