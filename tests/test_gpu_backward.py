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
    dq, dk, dv, _ = pa.pa_prefill_backward(Qd, Kd, Vd, o, lse, dOd, rp, ci, softmax_scale=scale)
    torch.cuda.synchronize()
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
    dq, dk, dv, _ = pa.pa_prefill_backward(Qd, Kd, Vd, o, lse, dOd, rp, ci)
    torch.cuda.synchronize()
    keys = sorted({0, 1, 63, 64, 65, N - 1, N - 64, N - 65, 8191, 8192, 12288 + 17}
                  | {int(x) for x in np.random.default_rng(1105).integers(0, N, 24)})
    rq, rk, rv = oracle.backward(Q, K, V, dO, 64, W, S, key_rows=keys)
    kidx = torch.as_tensor(keys).cuda()
    print("16K backward (max, mean):", _compare(dq, rq, "dQ 16K"), _compare(dk[:, kidx], rk[:, keys], "dK 16K"),
          _compare(dv[:, kidx], rv[:, keys], "dV 16K"))
