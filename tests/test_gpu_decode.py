"""GPU: pa_decode against the fp64 oracle, element by element."""
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


def _run(pa, oracle, q, kc, vc, lens, W, S, scale=0.0, o_dtype=torch.bfloat16):
    dev = "cuda"
    o, lse, _ = pa.pa_decode(q.to(dev), kc.to(dev), vc.to(dev),
                             torch.as_tensor(np.asarray(lens), dtype=torch.int32, device=dev), W, S,
                             softmax_scale=scale, o_dtype=o_dtype)
    torch.cuda.synchronize()
    o_ref, lse_ref, _ = oracle.decode(q, kc, vc, lens, 64, W, S, scale=scale if scale else None)
    return compare(o, lse, o_ref, lse_ref, "decode")


@pytest.mark.parametrize("Hq,Hkv,D", [(28, 4, 128), (8, 8, 64), (16, 2, 128), (6, 2, 64)])
def test_decode_small(pa, oracle, Hq, Hkv, D):
    batch, max_len = 5, 3000
    q = si.bf16_randn((batch, Hq, D), 1)
    kc, vc = si.bf16_randn((batch, max_len, Hkv, D), 2), si.bf16_randn((batch, max_len, Hkv, D), 3)
    lens = np.array([3000, 1, 64, 65, 1987])
    _run(pa, oracle, q, kc, vc, lens, 5, 1)
    _run(pa, oracle, q, kc, vc, lens, 0, 0, scale=0.21, o_dtype=torch.float32)
    _run(pa, oracle, q, kc, vc, lens, 60, 2)      # window covers everything: dense causal row


def test_decode_peaky_logits(pa, oracle):
    batch, max_len, Hq, Hkv, D = 3, 5000, 28, 4, 128
    q = si.bf16_randn((batch, Hq, D), 11)
    kc, vc = si.bf16_randn((batch, max_len, Hkv, D), 12, 3.0), si.bf16_randn((batch, max_len, Hkv, D), 13)
    _run(pa, oracle, q, kc, vc, np.array([5000, 4097, 4096]), 5, 1)


def test_decode_strided_cache_and_bad_length(pa, oracle):
    """Caches that are views into a larger allocation; a length outside [1, max_len] gives zeros."""
    batch, max_len, Hq, Hkv, D = 2, 700, 8, 2, 128
    big_k = si.bf16_randn((batch, max_len, Hkv + 1, D), 21).cuda()
    big_v = si.bf16_randn((batch, max_len, Hkv + 1, D), 22).cuda()
    kc, vc = big_k[:, :, 1:], big_v[:, :, 1:]
    q = si.bf16_randn((batch, Hq, D), 23)
    lens = torch.tensor([700, 333], dtype=torch.int32, device="cuda")
    o, lse, _ = pa.pa_decode(q.cuda(), kc, vc, lens, 5, 1)
    o_ref, lse_ref, _ = oracle.decode(q, kc.cpu().contiguous(), vc.cpu().contiguous(), [700, 333], 64, 5, 1)
    compare(o, lse, o_ref, lse_ref, "strided decode")
    lens_bad = torch.tensor([0, 701], dtype=torch.int32, device="cuda")
    o, lse, _ = pa.pa_decode(q.cuda(), kc, vc, lens_bad, 5, 1)
    torch.cuda.synchronize()
    assert (o == 0).all() and torch.isinf(lse).all() and (lse < 0).all()


def test_decode_equals_prefill_row_closed_forms(pa, oracle):
    """Constant keys: LSE - s = ln |A| with |A| = 64 * (#blocks - 1) + (p mod 64) + 1."""
    batch, max_len, Hq, Hkv, D = 4, 9000, 4, 2, 64
    krow = si.bf16_randn((D,), 31)
    kc = krow.expand(batch, max_len, Hkv, D).contiguous()
    vc = si.bf16_randn((batch, max_len, Hkv, D), 32)
    q = si.bf16_randn((batch, Hq, D), 33)
    lens = np.array([9000, 8193, 100, 4096])
    o, lse, _ = pa.pa_decode(q.cuda(), kc.cuda(), vc.cuda(), torch.as_tensor(lens, dtype=torch.int32).cuda(), 5, 1)
    lse = lse.double().cpu().numpy()
    for b, L in enumerate(lens):
        nblk = len(pa.pa_decode_block_list(int(L), 64, 5, 1))
        n_att = 64 * (nblk - 1) + (L - 1) % 64 + 1
        for h in range(Hq):
            s = float(q[b, h].double() @ krow.double()) / np.sqrt(D)
            assert abs(lse[b, h] - s - np.log(n_att)) < 1e-3


def test_decode_full_size_workload(pa, oracle):
    """Batch 8, 28/4 heads, head_dim 128, cache lengths uniform in [65536, 131072]."""
    w = si.DECODE_B8
    q, kc, vc, lens = si.decode_inputs(w)
    st = _run(pa, oracle, q, kc, vc, lens, w.window_blocks, w.sink_blocks)
    print("decode full-size error stats", st)


@pytest.mark.parametrize("env", [{"PA_DECODE_PATH": "splitk"},
                                 {"PA_DECODE_PATH": "cluster", "PA_DECODE_CLUSTER": "1"},
                                 {"PA_DECODE_PATH": "cluster", "PA_DECODE_CLUSTER": "2"},
                                 {"PA_DECODE_PATH": "cluster", "PA_DECODE_CLUSTER": "7"},
                                 {"PA_DECODE_PATH": "cluster", "PA_DECODE_CLUSTER": "8"},
                                 {"PA_DECODE_PATH": "cluster", "PA_DECODE_CLUSTER": "2", "PA_DECODE_STAGES": "2"},
                                 {"PA_DECODE_PATH": "cluster", "PA_DECODE_CLUSTER": "1", "PA_DECODE_STAGES": "3"},
                                 {"PA_DECODE_PATH": "cluster", "PA_DECODE_CLUSTER": "8", "PA_DECODE_STAGES": "1"},
                                 {"PA_DECODE_PATH": "cluster", "PA_DECODE_CLUSTER": "1", "PA_DECODE_STAGES": "1"},
                                 {"PA_DECODE_PATH": "cluster", "PA_DECODE_CLUSTER": "1", "PA_DECODE_STAGES": "6"},
                                 {"PA_DECODE_PATH": "cluster", "PA_DECODE_CLUSTER": "3", "PA_DECODE_STAGES": "4"},
                                 {"PA_DECODE_PATH": "persist"},
                                 {"PA_DECODE_PATH": "persist", "PA_DECODE_CLUSTER": "1"},
                                 {"PA_DECODE_PATH": "persist", "PA_DECODE_CLUSTER": "1", "PA_DECODE_STAGES": "1"},
                                 {"PA_DECODE_PATH": "persist", "PA_DECODE_CLUSTER": "4", "PA_DECODE_STAGES": "2"},
                                 {"PA_DECODE_PATH": "persist", "PA_DECODE_CLUSTER": "8", "PA_DECODE_STAGES": "6"}])
def test_decode_paths(pa, oracle, pa_env, env):
    """The split-K pair, the single-launch cluster form of the row kernel and its persistent form
    (partials + combine, or direct output with one chunk per row) at several chunk counts and ring
    depths give the same row of Eq. (1)."""
    pa_env(**env)
    batch, max_len, Hq, Hkv, D = 4, 9000, 28, 4, 128
    q = si.bf16_randn((batch, Hq, D), 31)
    kc, vc = si.bf16_randn((batch, max_len, Hkv, D), 32, 2.0), si.bf16_randn((batch, max_len, Hkv, D), 33)
    lens = np.array([9000, 8193, 130, 7])
    _run(pa, oracle, q, kc, vc, lens, 5, 1)
    _run(pa, oracle, q, kc, vc, lens, 3, 2, o_dtype=torch.float32)


def test_decode_short_cache_with_wide_window_and_sinks(pa, oracle):
    """A cache of 32 blocks whose window + sink candidates exceed 32: the bound on listed blocks is
    clamped by the row count, the candidate count is not (the library must pick its path by the
    latter)."""
    batch, max_len, Hq, Hkv, D = 3, 2048, 14, 2, 128
    q = si.bf16_randn((batch, Hq, D), 41)
    kc, vc = si.bf16_randn((batch, max_len, Hkv, D), 42), si.bf16_randn((batch, max_len, Hkv, D), 43)
    lens = np.array([2048, 1999, 700])
    _run(pa, oracle, q, kc, vc, lens, 30, 4)
    _run(pa, oracle, q, kc, vc, lens, 26, 4)   # 26 + 4 + 0 powers = 30 candidates: the cluster path


def test_row_kernel_block_set_is_the_layout_row(pa, oracle):
    """The single-launch kernel enumerates its key blocks one candidate per lane, unsorted: as a
    set (and without duplicates) it must be the layout row of the last position, for lengths on
    and around every power of two up to 2^20 tokens."""
    lens = {1, 2, 63, 64, 65, 127, 128, 129, 1000003, 1 << 20}
    for e in range(7, 21):
        lens.update({(1 << e) - 1, 1 << e, (1 << e) + 1, (1 << e) + 64, 3 * (1 << (e - 1)) + 17})
    for W in (0, 1, 5, 9, 26):
        for S in (0, 1, 3, 4):
            for L in sorted(lens):
                if L > (1 << 20):
                    continue
                rows = (L + 63) // 64
                slots = max(W, 1) + S + sum(1 for k in range(31) if max(W, 1) <= (1 << k) <= rows - 1)
                if slots > 32:       # more candidates than lanes: the library sends such rows down the other path
                    with pytest.raises(pa.PaError, match="PA_ERR_SHAPE"):
                        pa.pa_decode_row_block_set(L, 64, W, S)
                    continue
                got = pa.pa_decode_row_block_set(L, 64, W, S).cpu().numpy()
                ref = oracle.block_row((L - 1) // 64, W, S)
                assert len(set(got.tolist())) == len(got), (L, W, S, got)
                np.testing.assert_array_equal(np.sort(got), ref, err_msg=f"L={L} W={W} S={S}")


@pytest.mark.parametrize("env", [{}, {"PA_DECODE_PATH": "splitk"}, {"PA_DECODE_PATH": "persist"}])
def test_decode_ignores_what_the_cache_holds_beyond_the_length(pa, oracle, pa_env, env):
    """Cache rows past cache_lens (not yet written by the caller) may hold anything, NaN bit
    patterns included: the result must not change."""
    batch, max_len, Hq, Hkv, D = 4, 4096, 14, 2, 128
    q = si.bf16_randn((batch, Hq, D), 51)
    kc, vc = si.bf16_randn((batch, max_len, Hkv, D), 52), si.bf16_randn((batch, max_len, Hkv, D), 53)
    lens = np.array([4000, 1, 65, 2049])
    o_ref, lse_ref, _ = oracle.decode(q, kc, vc, lens, 64, 5, 1)
    kd, vd = kc.cuda(), vc.cuda()
    for b, L in enumerate(lens):
        kd[b, L:] = float("nan")
        vd[b, L:] = float("nan")
    pa_env(**env)
    o, lse, ws = pa.pa_decode(q.cuda(), kd, vd, torch.as_tensor(lens, dtype=torch.int32).cuda(), 5, 1)
    pa.pa_decode_status(ws)
    compare(o, lse, o_ref, lse_ref, "garbage beyond the length")


def _paged_copy(kc, vc, lens, n_pages, rng):
    """Scatters contiguous caches [batch, max_len, Hkv, D] into a pool of 64-token pages in a
    seeded random page order; returns (k_pool, v_pool, block_table)."""
    batch, max_len, Hkv, D = kc.shape
    max_blocks = (max_len + 63) // 64
    table = np.full((batch, max_blocks), -1, dtype=np.int32)
    order = rng.permutation(n_pages)
    k_pool = torch.zeros((n_pages, 64, Hkv, D), dtype=torch.bfloat16)
    v_pool = torch.zeros((n_pages, 64, Hkv, D), dtype=torch.bfloat16)
    nxt = 0
    for b in range(batch):
        for j in range((int(lens[b]) + 63) // 64):
            pg = int(order[nxt]); nxt += 1
            table[b, j] = pg
            n = min(64, max_len - 64 * j)
            k_pool[pg, :n] = kc[b, 64 * j:64 * j + n]
            v_pool[pg, :n] = vc[b, 64 * j:64 * j + n]
    return k_pool, v_pool, table


@pytest.mark.parametrize("env", [{}, {"PA_DECODE_PATH": "splitk"}, {"PA_DECODE_CLUSTER": "2", "PA_DECODE_STAGES": "2"},
                                 {"PA_DECODE_PATH": "persist", "PA_DECODE_CLUSTER": "3"},
                                 {"PA_DECODE_PATH": "persist", "PA_DECODE_CLUSTER": "1"}])
def test_paged_decode_matches_the_oracle(pa, oracle, pa_env, env):
    """The same rows through a pool of 64-token pages in scrambled order (oracle side: the pages
    gathered back into a contiguous cache on the host)."""
    pa_env(**env)
    batch, max_len, Hq, Hkv, D = 5, 9000, 28, 4, 128
    q = si.bf16_randn((batch, Hq, D), 61)
    kc, vc = si.bf16_randn((batch, max_len, Hkv, D), 62), si.bf16_randn((batch, max_len, Hkv, D), 63)
    lens = np.array([9000, 8193, 130, 7, 4096])
    k_pool, v_pool, table = _paged_copy(kc, vc, lens, 800, np.random.default_rng(64))
    o, lse, ws = pa.pa_decode_paged(q.cuda(), k_pool.cuda(), v_pool.cuda(), torch.as_tensor(table).cuda(),
                                    torch.as_tensor(lens, dtype=torch.int32).cuda(), 5, 1)
    pa.pa_decode_status(ws)
    o_ref, lse_ref, _ = oracle.decode(q, kc, vc, lens, 64, 5, 1)
    compare(o, lse, o_ref, lse_ref, "paged decode")


def test_append_and_decode_over_many_steps(pa, oracle):
    """A 16K-token context followed by 1024 decoding steps (Section 4.5's serving shape, shortened
    context): every step appends one token's K and V to the paged cache and decodes against it.
    Every 64th step (and the steps that cross a page boundary) is compared with the oracle on the
    gathered cache; the final cache contents are compared bit for bit."""
    batch, Hq, Hkv, D, W, S = 3, 14, 2, 128, 5, 1
    ctx = np.array([16384, 16000, 777])
    steps = 1024
    max_len = int(ctx.max()) + steps
    max_blocks = (max_len + 63) // 64
    n_pages = batch * max_blocks + 7
    rng = np.random.default_rng(71)
    kc, vc = si.bf16_randn((batch, max_len, Hkv, D), 72), si.bf16_randn((batch, max_len, Hkv, D), 73)
    qs = si.bf16_randn((steps, batch, Hq, D), 74)
    # pages for the whole run are assigned up front (the caller's allocator), the pool holds the context only
    k_pool, v_pool, table = _paged_copy(kc, vc, ctx + steps, n_pages, rng)
    kp, vp = k_pool.cuda(), v_pool.cuda()
    for b in range(batch):   # wipe what lies beyond the context: the appends must put it back
        for pos in range(int(ctx[b]), int(ctx[b]) + steps):
            kp[table[b, pos // 64], pos % 64] = 0
            vp[table[b, pos // 64], pos % 64] = 0
    table_d = torch.as_tensor(table).cuda()
    lens_d = torch.as_tensor(ctx, dtype=torch.int32).cuda()
    kcd, vcd, qd = kc.cuda(), vc.cuda(), qs.cuda()
    idx = torch.arange(batch, device="cuda")
    o = lse = ws = None
    checked = 0
    for t in range(steps):
        cur = lens_d.long()
        pa.pa_kv_append(kcd[idx, cur].contiguous(), vcd[idx, cur].contiguous(), kp, vp, table_d, lens_d)
        o, lse, ws = pa.pa_decode_paged(qd[t], kp, vp, table_d, lens_d, W, S, o=o, lse=lse, workspace=ws)
        if t % 64 == 0 or t in (1, 63, 65, steps - 1):
            lens_now = ctx + t + 1
            assert lens_d.cpu().numpy().tolist() == lens_now.tolist()
            o_ref, lse_ref, _ = oracle.decode(qs[t], kc, vc, lens_now, 64, W, S)
            compare(o, lse, o_ref, lse_ref, f"step {t}")
            checked += 1
    pa.pa_decode_status(ws)
    assert checked >= 16
    kp_h, vp_h = kp.cpu(), vp.cpu()
    for b in range(batch):
        for j in range((int(ctx[b]) + steps + 63) // 64):
            n = min(64, int(ctx[b]) + steps - 64 * j)
            assert torch.equal(kp_h[table[b, j], :n], kc[b, 64 * j:64 * j + n])
            assert torch.equal(vp_h[table[b, j], :n], vc[b, 64 * j:64 * j + n])


def test_append_leaves_sequences_without_a_page_alone(pa):
    batch, Hkv, D = 3, 2, 64
    k_pool = torch.zeros((4, 64, Hkv, D), dtype=torch.bfloat16, device="cuda")
    v_pool = torch.zeros_like(k_pool)
    table = torch.tensor([[0, 1], [2, -1], [3, 9]], dtype=torch.int32, device="cuda")
    lens = torch.tensor([127, 64, 128], dtype=torch.int32, device="cuda")   # last slot; no page; beyond the table
    k_new = si.bf16_randn((batch, Hkv, D), 81).cuda()
    v_new = si.bf16_randn((batch, Hkv, D), 82).cuda()
    pa.pa_kv_append(k_new, v_new, k_pool, v_pool, table, lens)
    torch.cuda.synchronize()
    assert lens.cpu().tolist() == [128, 64, 128]
    assert torch.equal(k_pool[1, 63], k_new[0]) and torch.equal(v_pool[1, 63], v_new[0])
    k_pool[1, 63] = 0
    v_pool[1, 63] = 0
    assert not k_pool.any() and not v_pool.any()


@pytest.mark.parametrize("env", [{}, {"PA_DECODE_CLUSTER": "1"}, {"PA_DECODE_CLUSTER": "5", "PA_DECODE_STAGES": "2"}])
def test_decode_many_rows_through_the_persistent_grid(pa, oracle, pa_env, env):
    """Enough (sequence, KV head) rows that the library picks the persistent form by itself and
    every CTA walks several work items: ring positions, Q prefetch and the hand-over area carry
    over from item to item.  Lengths include invalid ones (outputs zero, LSE -inf)."""
    pa_env(**env)
    batch, max_len, Hq, Hkv, D = 150, 2600, 28, 4, 128
    q = si.bf16_randn((batch, Hq, D), 91)
    kc, vc = si.bf16_randn((batch, max_len, Hkv, D), 92), si.bf16_randn((batch, max_len, Hkv, D), 93)
    lens = np.random.default_rng(94).integers(1, max_len + 1, size=batch)
    lens[:6] = [max_len, 1, 64, 65, 2049, 128]
    _run(pa, oracle, q, kc, vc, lens, 5, 1)
    bad = lens.copy()
    bad[[3, 77]] = [0, max_len + 1]
    o, lse, ws = pa.pa_decode(q.cuda(), kc.cuda(), vc.cuda(), torch.as_tensor(bad, dtype=torch.int32).cuda(), 5, 1)
    pa.pa_decode_status(ws)
    for b in (3, 77):
        assert (o[b] == 0).all() and torch.isinf(lse[b]).all() and (lse[b] < 0).all()
    good = np.setdiff1d(np.arange(batch), [3, 77])
    o_ref, lse_ref, _ = oracle.decode(q[good], kc[good], vc[good], lens[good], 64, 5, 1)
    compare(o[good], lse[good], o_ref, lse_ref, "persistent grid with invalid lengths")

