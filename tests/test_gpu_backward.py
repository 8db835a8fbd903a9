"""GPU: pa_prefill_backward (dQ, dK, dV) against the fp64 oracle's gradients of Eq. (1), element by
element.  The forward pass that feeds it (O, LSE) is the library's own."""
import numpy as np
import pytest
import torch

import synth_inputs as si

pytestmark = pytest.mark.gpu

# bf16 operands (P and dS are rounded to bf16 before their second product), fp32 accumulation and
# fp32 outputs: the same bounds as for the forward output, relative to the largest gradient entry
# when that exceeds one.
G_MAX_ABS = 2e-2
G_MEAN_ABS = 2e-3


@pytest.fixture(scope="module")
def pa():
    import paper_2503_03588_b200 as pa_

    return pa_


def _compare(got, ref, what):
    got = got.double().cpu().numpy()
    assert got.shape == ref.shape and np.isfinite(got).all(), what
    unit = max(1.0, float(np.abs(ref).max()))
    err = np.abs(got - ref)
    assert err.max() <= G_MAX_ABS * unit, (what, float(err.max()), unit)
    assert err.mean() <= G_MEAN_ABS * unit, (what, float(err.mean()), unit)
    return float(err.max()), float(err.mean())


def _run(pa, oracle, N, Hq, Hkv, D, W, S, batch=1, use_power=True, k_scale=1.0, scale=0.0, seed=0):
    Q = si.bf16_randn((batch, N, Hq, D), 1000 + seed)
    K = si.bf16_randn((batch, N, Hkv, D), 1001 + seed, k_scale)
    V = si.bf16_randn((batch, N, Hkv, D), 1002 + seed)
    dO = si.bf16_randn((batch, N, Hq, D), 1003 + seed)
    rp, ci = oracle.block_layout(N, 64, W, S, use_power=use_power)
    rp, ci = torch.as_tensor(rp).cuda(), torch.as_tensor(ci).cuda()
    Qd, Kd, Vd, dOd = Q.cuda(), K.cuda(), V.cuda(), dO.cuda()
    o, lse, ws = pa.pa_prefill(Qd, Kd, Vd, rp, ci, softmax_scale=scale)
    pa.pa_prefill_status(ws)
    dq, dk, dv, wsb = pa.pa_prefill_backward(Qd, Kd, Vd, o, lse, dOd, rp, ci, softmax_scale=scale)
    pa.pa_prefill_status(wsb)   # the backward workspace starts with the same status block; synchronises
    rq, rk, rv = oracle.backward(Q, K, V, dO, 64, W, S, scale=scale if scale else None, use_power=use_power)
    what = f"N={N} Hq={Hq} Hkv={Hkv} D={D} W={W} S={S}"
    return [_compare(g, r, f"{n} {what}") for g, r, n in ((dq, rq, "dQ"), (dk, rk, "dK"), (dv, rv, "dV"))]


@pytest.mark.parametrize("N,Hq,Hkv,D,W,S", [
    (64, 2, 2, 64, 5, 1),        # one block
    (1, 2, 1, 128, 5, 1),        # one token
    (200, 4, 2, 128, 5, 1),      # ragged tail
    (1000, 7, 1, 128, 5, 1),     # a 7-head group
    (1536, 28, 4, 128, 5, 1),    # the 7B-like head shape
    (777, 8, 2, 64, 0, 0),       # pure power-of-two pattern
    (900, 6, 2, 128, 30, 2),     # window covers everything: dense causal
    (130, 5, 1, 128, 2, 1),      # a 5-head group: three head pairs, the last with a padding head
    (4097, 6, 3, 128, 7, 2),     # pairs only, one token in the last block
])
def test_backward_small_shapes(pa, oracle, N, Hq, Hkv, D, W, S):
    _run(pa, oracle, N, Hq, Hkv, D, W, S, batch=2, seed=N)


def test_backward_sink_column_spread_over_many_ctas(pa, oracle):
    """4200 tokens = 66 blocks: the sink block is listed by every row, so its column is cut into
    three chunks whose parts meet through atomics; peaky logits and a custom scale on top."""
    stats = _run(pa, oracle, 4200, 8, 2, 128, 5, 1, k_scale=2.0, scale=0.07, seed=5)
    print("backward error stats (max, mean) for dQ, dK, dV:", stats)


def test_backward_sliding_window_layout(pa, oracle):
    _run(pa, oracle, 1100, 8, 2, 128, 4, 1, use_power=False, seed=6)


@pytest.mark.parametrize("N,Hq,Hkv,W,S", [
    (1000, 7, 1, 5, 1),      # a 7-head group: four head pairs, the last with a padding head
    (2100, 3, 3, 2, 0),      # one query head per KV head: every pair has a padding head
    (4200, 8, 2, 5, 1),      # the sink column in three chunks
])
def test_backward_head_dim_128_on_the_warp_level_kernels(pa, pa_env, oracle, N, Hq, Hkv, W, S):
    """head_dim 128 takes the tcgen05 kernels by default; PA_BACKWARD_PATH=mma sends it through the
    warp-level MMA kernels that head_dim 64 uses.  Both meet the oracle."""
    _run(pa, oracle, N, Hq, Hkv, 128, W, S, seed=N)
    pa_env(PA_BACKWARD_PATH="mma")
    _run(pa, oracle, N, Hq, Hkv, 128, W, S, seed=N)


def test_backward_many_items_per_cta(pa, oracle):
    """12K tokens x 8 heads x batch 2: 1500 (query block, head pair) items for the persistent dQ
    kernel, several per CTA with rows of every length, and dK / dV columns in one to six chunks;
    dK and dV are checked on sampled keys."""
    N, Hq, Hkv, D, W, S = 12000, 8, 2, 128, 3, 1
    Q, K, V = (si.bf16_randn((2, N, h, D), 1200 + i) for i, h in enumerate((Hq, Hkv, Hkv)))
    dO = si.bf16_randn((2, N, Hq, D), 1204)
    rp, ci = pa.pa_build_layout(N, 64, W, S)
    Qd, Kd, Vd, dOd = Q.cuda(), K.cuda(), V.cuda(), dO.cuda()
    o, lse, ws = pa.pa_prefill(Qd, Kd, Vd, rp, ci)
    pa.pa_prefill_status(ws)
    dq, dk, dv, wsb = pa.pa_prefill_backward(Qd, Kd, Vd, o, lse, dOd, rp, ci)
    pa.pa_prefill_status(wsb)
    keys = sorted({0, 63, 64, N - 1, 4095, 4096} | {int(x) for x in np.random.default_rng(1205).integers(0, N, 20)})
    rq, rk, rv = oracle.backward(Q, K, V, dO, 64, W, S, key_rows=keys)
    kidx = torch.as_tensor(keys).cuda()
    _compare(dq, rq, "dQ 12K")
    _compare(dk[:, kidx], rk[:, keys], "dK 12K")
    _compare(dv[:, kidx], rv[:, keys], "dV 12K")


def test_backward_wait_that_runs_out_ends_the_kernels_with_a_status(pa, oracle):
    """The tcgen05 backward kernels bound every barrier wait like the prefill kernel.  With the limit
    at one cycle an ordinary wait that is not over at its first try (the first tiles take microseconds
    to arrive) runs out: the call returns, the status block at the head of the backward workspace
    reports PA_ERR_TIMEOUT, and the next call, back at the default limit, is correct."""
    N, Hq, Hkv, D, W, S = 3000, 8, 2, 128, 5, 1
    Q, K, V = (si.bf16_randn((1, N, h, D), 1300 + i) for i, h in enumerate((Hq, Hkv, Hkv)))
    dO = si.bf16_randn((1, N, Hq, D), 1304)
    rp, ci = pa.pa_build_layout(N, 64, W, S)
    Qd, Kd, Vd, dOd = Q.cuda(), K.cuda(), V.cuda(), dO.cuda()
    o, lse, ws = pa.pa_prefill(Qd, Kd, Vd, rp, ci)
    pa.pa_prefill_status(ws)
    try:
        pa.pa_set_wait_limit_cycles(1)
        dq, dk, dv, wsb = pa.pa_prefill_backward(Qd, Kd, Vd, o, lse, dOd, rp, ci)
        with pytest.raises(pa.PaError, match="PA_ERR_TIMEOUT"):
            pa.pa_prefill_status(wsb)
    finally:
        pa.pa_set_wait_limit_cycles(0)
    dq, dk, dv, wsb = pa.pa_prefill_backward(Qd, Kd, Vd, o, lse, dOd, rp, ci)
    assert pa.pa_prefill_status(wsb) == 0
    rq, rk, rv = oracle.backward(Q, K, V, dO, 64, W, S)
    for g, r, n in ((dq, rq, "dQ"), (dk, rk, "dK"), (dv, rv, "dV")):
        _compare(g, r, n + " after a timed-out call")


def test_backward_at_16k_on_sampled_keys(pa, oracle):
    """A sweep-sized case: 16K tokens with the 7B-like heads.  The oracle evaluates dQ on every row
    (its first pass covers them all anyway) and dK, dV on sampled key positions: the sink block (its
    column is spread over eight CTAs), block boundaries, power-of-two distances and a random draw."""
    N, Hq, Hkv, D, W, S = 16384, 28, 4, 128, 5, 1
    Q, K, V = si.bf16_randn((1, N, Hq, D), 1101), si.bf16_randn((1, N, Hkv, D), 1102), si.bf16_randn((1, N, Hkv, D), 1103)
    dO = si.bf16_randn((1, N, Hq, D), 1104)
    rp, ci = pa.pa_build_layout(N, 64, W, S)
    Qd, Kd, Vd, dOd = Q.cuda(), K.cuda(), V.cuda(), dO.cuda()
    o, lse, ws = pa.pa_prefill(Qd, Kd, Vd, rp, ci)
    pa.pa_prefill_status(ws)
    dq, dk, dv, wsb = pa.pa_prefill_backward(Qd, Kd, Vd, o, lse, dOd, rp, ci)
    pa.pa_prefill_status(wsb)
    keys = sorted({0, 1, 63, 64, 65, N - 1, N - 64, N - 65, 8191, 8192, 12288 + 17}
                  | {int(x) for x in np.random.default_rng(1105).integers(0, N, 24)})
    rq, rk, rv = oracle.backward(Q, K, V, dO, 64, W, S, key_rows=keys)
    kidx = torch.as_tensor(keys).cuda()
    print("16K backward (max, mean):", _compare(dq, rq, "dQ 16K"), _compare(dk[:, kidx], rk[:, keys], "dK 16K"),
          _compare(dv[:, kidx], rv[:, keys], "dV 16K"))


def test_backward_on_views_of_a_packed_qkv_tensor(pa, oracle):
    """Q, K and V as head slices of one [batch, seq, Hq + 2 Hkv, D] tensor: the kernels take the
    strides as given (the tensor maps of the tcgen05 kernels are built from them)."""
    N, Hq, Hkv, D, W, S = 1300, 8, 2, 128, 3, 1
    qkv = si.bf16_randn((2, N, Hq + 2 * Hkv, D), 1400).cuda()
    q, k, v = qkv[:, :, :Hq], qkv[:, :, Hq:Hq + Hkv], qkv[:, :, Hq + Hkv:]
    dO = si.bf16_randn((2, N, Hq, D), 1401)
    rp, ci = pa.pa_build_layout(N, 64, W, S)
    o, lse, ws = pa.pa_prefill(q, k, v, rp, ci)
    pa.pa_prefill_status(ws)
    dq, dk, dv, wsb = pa.pa_prefill_backward(q, k, v, o, lse, dO.cuda(), rp, ci)
    pa.pa_prefill_status(wsb)
    rq, rk, rv = oracle.backward(q.cpu().contiguous(), k.cpu().contiguous(), v.cpu().contiguous(), dO, 64, W, S)
    for g, r, n in ((dq, rq, "dQ"), (dk, rk, "dK"), (dv, rv, "dV")):
        _compare(g, r, n + " packed qkv")


def test_backward_on_kv_head_shards_reproduces_the_whole_call(pa):
    """Head sharding needs no exchange in the backward pass either: dQ belongs to the query heads and
    dK, dV to the KV heads a rank holds.  The ranks' calls on head slices (run here one after the other
    on the one GPU) give dQ bit for bit and dK, dV up to the order of their fp32 additions."""
    from paper_2503_03588_b200.sharding import kv_head_shard, shard_prefill_tensors

    N, Hq, Hkv, D = 3000, 28, 4, 128
    Q, K, V = (si.bf16_randn((1, N, h, D), 1500 + i).cuda() for i, h in enumerate((Hq, Hkv, Hkv)))
    dO = si.bf16_randn((1, N, Hq, D), 1504).cuda()
    rp, ci = pa.pa_build_layout(N, 64, 5, 1)
    o, lse, ws = pa.pa_prefill(Q, K, V, rp, ci)
    pa.pa_prefill_status(ws)
    dq_full, dk_full, dv_full, wsb = pa.pa_prefill_backward(Q, K, V, o, lse, dO, rp, ci)
    pa.pa_prefill_status(wsb)
    for world in (2, 4):
        for rank in range(world):
            qs_, ks_, vs_, heads = shard_prefill_tensors(Q, K, V, world, rank)
            _, kv_heads = kv_head_shard(Hq, Hkv, world, rank)
            dq, dk, dv, wsr = pa.pa_prefill_backward(qs_, ks_, vs_, o[:, :, heads], lse[:, heads].contiguous(), dO[:, :, heads], rp, ci)
            pa.pa_prefill_status(wsr)
            assert torch.equal(dq, dq_full[:, :, heads]), (world, rank)
            assert torch.allclose(dk, dk_full[:, :, kv_heads], rtol=1e-4, atol=1e-5), (world, rank)
            assert torch.allclose(dv, dv_full[:, :, kv_heads], rtol=1e-4, atol=1e-5), (world, rank)
