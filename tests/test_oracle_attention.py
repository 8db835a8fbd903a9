"""Pins for the oracle's attention arithmetic (Eq. (1)): library routines on special cases,
closed forms and invariants, so that a dropped term, a wrong index or a transposed operand in
the oracle fails at least one of them."""
import numpy as np
import pytest
import torch
from scipy.special import logsumexp, softmax

import synth_inputs as si


def _f64(t):
    return t.double().numpy()


def _rand(shape, seed, scale=1.0):
    return si.bf16_randn(shape, seed, scale)


def _dense_reference(Q, K, V, allowed, scale):
    """Masked softmax attention from library routines: scipy softmax / logsumexp over -inf-masked
    logits and a matmul, per (batch, head).  allowed: [N, N] bool."""
    q, k, v = _f64(Q), _f64(K), _f64(V)
    batch, N, Hq, D = q.shape
    G = Hq // k.shape[2]
    O = np.zeros((batch, N, Hq, D))
    L = np.zeros((batch, Hq, N))
    for b in range(batch):
        for h in range(Hq):
            s = scale * (q[b, :, h, :] @ k[b, :, h // G, :].T)
            s = np.where(allowed, s, -np.inf)
            O[b, :, h, :] = softmax(s, axis=1) @ v[b, :, h // G, :]
            L[b, h, :] = logsumexp(s, axis=1)
    return O, L


def test_reduces_to_full_causal_attention(oracle):
    """Section 3.1: A_i = {j <= i} is full attention.  With the window covering every block the
    oracle must equal textbook causal softmax attention (scipy), GQA mapping included."""
    batch, N, Hq, Hkv, D, B = 2, 150, 4, 2, 24, 16
    Q, K, V = _rand((batch, N, Hq, D), 1), _rand((batch, N, Hkv, D), 2), _rand((batch, N, Hkv, D), 3)
    scale = 0.37
    O, L, cnt = oracle.prefill(Q, K, V, B, W=10, S=0, scale=scale)
    Or, Lr = _dense_reference(Q, K, V, np.tril(np.ones((N, N), bool)), scale)
    np.testing.assert_allclose(O, Or, rtol=0, atol=1e-12)
    np.testing.assert_allclose(L, Lr, rtol=0, atol=1e-12)
    assert (cnt == np.arange(1, N + 1)).all()
    # default scale is 1/sqrt(d_k) (Eq. (1))
    O2, L2, _ = oracle.prefill(Q, K, V, B, W=10, S=0)
    Or2, Lr2 = _dense_reference(Q, K, V, np.tril(np.ones((N, N), bool)), 1 / np.sqrt(D))
    np.testing.assert_allclose(O2, Or2, atol=1e-12)
    np.testing.assert_allclose(L2, Lr2, atol=1e-12)


def test_sparse_rows_against_library_softmax_on_index_sets(oracle):
    """Eq. (1) row by row: gather the attended keys, scipy softmax, weighted sum."""
    batch, N, Hq, Hkv, D, B, W, S = 1, 203, 6, 2, 16, 8, 2, 1
    Q, K, V = _rand((batch, N, Hq, D), 11), _rand((batch, N, Hkv, D), 12, 2.0), _rand((batch, N, Hkv, D), 13)
    O, L, cnt = oracle.prefill(Q, K, V, B, W, S)
    m = oracle.dense_mask(N, B, W, S)
    q, k, v = _f64(Q), _f64(K), _f64(V)
    scale = 1 / np.sqrt(D)
    for qi in (0, 1, 7, 8, 63, 64, 100, 199, 202):
        idx = np.nonzero(m[qi])[0]
        assert cnt[qi] == len(idx)
        for h in range(Hq):
            s = scale * (k[0, idx, h // 3, :] @ q[0, qi, h, :])
            np.testing.assert_allclose(O[0, qi, h], softmax(s) @ v[0, idx, h // 3, :], atol=1e-12)
            np.testing.assert_allclose(L[0, h, qi], logsumexp(s), atol=1e-12)
    # and the whole thing through the dense reference with the oracle's own (pinned) mask
    Or, Lr = _dense_reference(Q, K, V, m, scale)
    np.testing.assert_allclose(O, Or, atol=1e-12)
    np.testing.assert_allclose(L, Lr, atol=1e-12)


def _n_attended_closed_form(q, B, W, S):
    i = q // B
    ds = {0} | set(range(min(W, i + 1))) | {i - j for j in range(min(S, i + 1))}
    k = 1
    while k <= i:
        ds.add(k)
        k *= 2
    return B * len(ds) - (B - 1 - q % B)


def test_constant_keys_count_the_attended_set(oracle):
    """K rows all equal => every logit of a row equals s, so LSE - s = ln |A_q| and O is the
    plain mean of the attended V rows; |A_q| has a closed form in (q, B, W, S)."""
    N, Hq, Hkv, D, B, W, S = 330, 2, 1, 8, 8, 3, 2
    Q, V = _rand((1, N, Hq, D), 21), _rand((1, N, Hkv, D), 23)
    krow = _rand((D,), 22)
    K = krow.expand(1, N, Hkv, D).contiguous()
    O, L, cnt = oracle.prefill(Q, K, V, B, W, S, scale=0.5)
    q, v = _f64(Q), _f64(V)
    m = oracle.dense_mask(N, B, W, S)
    for qi in range(N):
        n = _n_attended_closed_form(qi, B, W, S)
        assert cnt[qi] == n
        for h in range(Hq):
            s = 0.5 * float(q[0, qi, h] @ _f64(krow))
            assert abs(L[0, h, qi] - s - np.log(n)) < 1e-12
        np.testing.assert_allclose(O[0, qi, 0], v[0, m[qi], 0].mean(axis=0), atol=1e-12)


def test_single_key_row_and_constant_values(oracle):
    N, Hq, Hkv, D, B = 70, 2, 2, 8, 16
    Q, K, V = _rand((1, N, Hq, D), 31), _rand((1, N, Hkv, D), 32), _rand((1, N, Hkv, D), 33)
    O, L, _ = oracle.prefill(Q, K, V, B, 1, 1, scale=0.25, rows=[0])
    q, k, v = _f64(Q), _f64(K), _f64(V)
    for h in range(Hq):
        np.testing.assert_allclose(O[0, 0, h], v[0, 0, h], atol=1e-15)   # o_0 = v_0
        assert abs(L[0, h, 0] - 0.25 * q[0, 0, h] @ k[0, 0, h]) < 1e-13
    vrow = _rand((D,), 34)
    Vc = vrow.expand(1, N, Hkv, D).contiguous()
    O, _, _ = oracle.prefill(Q, K, Vc, B, 1, 1)
    np.testing.assert_allclose(O, np.broadcast_to(_f64(vrow), O.shape), atol=1e-13)  # sum p = 1


def test_vanishing_scale_gives_uniform_weights(oracle):
    N, D, B, W, S = 130, 8, 8, 2, 1
    Q, K, V = _rand((1, N, 1, D), 41), _rand((1, N, 1, D), 42), _rand((1, N, 1, D), 43)
    O, L, cnt = oracle.prefill(Q, K, V, B, W, S, scale=1e-30)
    m = oracle.dense_mask(N, B, W, S)
    v = _f64(V)
    for qi in range(N):
        np.testing.assert_allclose(O[0, qi, 0], v[0, m[qi], 0].mean(axis=0), atol=1e-12)
        assert abs(L[0, 0, qi] - np.log(cnt[qi])) < 1e-12


def test_masked_keys_have_no_influence(oracle):
    """Changing K/V at a position outside A_q leaves row q untouched; inside A_q it does not."""
    N, D, B, W, S = 200, 8, 8, 2, 1
    Q, K, V = _rand((1, N, 1, D), 51), _rand((1, N, 1, D), 52), _rand((1, N, 1, D), 53)
    qi = 199                                               # block 24: attends blocks 0,8,16,20,22,23,24
    base, _, _ = oracle.prefill(Q, K, V, B, W, S, rows=[qi])
    for blk, inside in [(21, False), (19, False), (1, False), (20, True), (16, True), (0, True)]:
        K2, V2 = K.clone(), V.clone()
        K2[0, blk * B + 3] += 1.0
        V2[0, blk * B + 3] += 1.0
        out, _, _ = oracle.prefill(Q, K2, V2, B, W, S, rows=[qi])
        assert (np.abs(out - base).max() > 1e-6) == inside, blk


def test_rows_and_heads_subsets_match_full(oracle):
    N, Hq, Hkv, D, B = 140, 4, 2, 8, 8
    Q, K, V = _rand((2, N, Hq, D), 61), _rand((2, N, Hkv, D), 62), _rand((2, N, Hkv, D), 63)
    O, L, cnt = oracle.prefill(Q, K, V, B, 2, 1)
    rows, heads = [3, 77, 139], [1, 2]
    Os, Ls, cs = oracle.prefill(Q, K, V, B, 2, 1, rows=rows, heads=heads)
    np.testing.assert_array_equal(Os, O[:, rows][:, :, heads])
    np.testing.assert_array_equal(Ls, L[:, heads][:, :, rows])
    np.testing.assert_array_equal(cs, cnt[rows])
    # an explicit dense mask equal to the predicate gives the same numbers
    Od, Ld, _ = oracle.prefill(Q, K, V, B, 2, 1, dense=oracle.dense_mask(N, B, 2, 1))
    np.testing.assert_array_equal(Od, O)
    np.testing.assert_array_equal(Ld, L)


def test_decode_is_the_last_prefill_row(oracle):
    """Section 4.1: the same pattern in prefilling and decoding.  A decode call with cache length
    L equals row L-1 of a prefill over the first L tokens (the token attends to itself)."""
    batch, max_len, Hq, Hkv, D, B, W, S = 3, 260, 4, 2, 16, 8, 3, 1
    Kc, Vc = _rand((batch, max_len, Hkv, D), 71), _rand((batch, max_len, Hkv, D), 72)
    q = _rand((batch, Hq, D), 73)
    lens = np.array([260, 1, 129])
    O, L, cnt = oracle.decode(q, Kc, Vc, lens, B, W, S, scale=0.3)
    for b in range(batch):
        Lb = int(lens[b])
        Qfull = torch.zeros((1, Lb, Hq, D), dtype=torch.bfloat16)
        Qfull[0, Lb - 1] = q[b]
        Op, Lp, cp = oracle.prefill(Qfull, Kc[b:b + 1, :Lb].contiguous(), Vc[b:b + 1, :Lb].contiguous(),
                                    B, W, S, scale=0.3, rows=[Lb - 1])
        np.testing.assert_allclose(O[b], Op[0, 0], atol=1e-14)
        np.testing.assert_allclose(L[b], Lp[0, :, 0], atol=1e-14)
        assert cnt[b] == cp[0] == _n_attended_closed_form(Lb - 1, B, W, S)


def test_bf16_widening_is_exact(oracle):
    """The oracle reads bf16 bit patterns; widening must reproduce torch's bf16 -> fp64 exactly."""
    vals = torch.tensor([0.0, -0.0, 1.0, -2.5, 3.140625, 1e-20, -65280.0, 0.00390625],
                        dtype=torch.float32).to(torch.bfloat16)
    D = vals.numel()
    V = vals.view(1, 1, 1, D).contiguous()
    Q = torch.ones((1, 1, 1, D), dtype=torch.bfloat16)
    O, _, _ = oracle.prefill(Q, Q.clone(), V, 4, 1, 1)
    np.testing.assert_array_equal(O[0, 0, 0], _f64(vals))


# ------------------------------------------------------------------ backward of Eq. (1)

def _autograd_reference(Q, K, V, dO, mask, scale):
    """dQ, dK, dV of softmax-over-the-mask attention by torch's fp64 autograd on the dense form."""
    import torch

    q = Q.double().clone().requires_grad_(True)
    k = K.double().clone().requires_grad_(True)
    v = V.double().clone().requires_grad_(True)
    G = q.shape[2] // k.shape[2]
    kk, vv = k.repeat_interleave(G, dim=2), v.repeat_interleave(G, dim=2)
    s = torch.einsum("bqhd,bkhd->bhqk", q, kk) * scale
    s = s.masked_fill(~torch.as_tensor(mask)[None, None], float("-inf"))
    o = torch.einsum("bhqk,bkhd->bqhd", torch.softmax(s, dim=-1), vv)
    (o * dO.double()).sum().backward()
    return q.grad.numpy(), k.grad.numpy(), v.grad.numpy()


@pytest.mark.parametrize("N,Hq,Hkv,D,B,W,S,use_power", [
    (200, 4, 2, 16, 8, 2, 1, True),        # window + powers + sink, grouped heads, ragged tail
    (130, 3, 1, 8, 16, 0, 0, True),        # pure power-of-two pattern, a group of three
    (96, 2, 2, 32, 4, 3, 2, False),        # sliding window with two sink blocks
    (64, 2, 1, 8, 64, 5, 1, True),         # one block: plain causal attention
])
def test_backward_matches_autograd_on_the_dense_form(oracle, N, Hq, Hkv, D, B, W, S, use_power):
    """The oracle's gradients against torch autograd (fp64) through a dense masked softmax: a
    dropped term, a wrong sign, a missing scale or a wrong head grouping fails here."""
    import synth_inputs as si

    Q, K, V = si.bf16_randn((2, N, Hq, D), 7), si.bf16_randn((2, N, Hkv, D), 8, 2.0), si.bf16_randn((2, N, Hkv, D), 9)
    dO = si.bf16_randn((2, N, Hq, D), 10)
    scale = 0.37
    dq, dk, dv = oracle.backward(Q, K, V, dO, B, W, S, scale=scale, use_power=use_power)
    rq, rk, rv = _autograd_reference(Q, K, V, dO, oracle.dense_mask(N, B, W, S, use_power), scale)
    for got, ref in ((dq, rq), (dk, rk), (dv, rv)):
        assert np.abs(got - ref).max() <= 1e-10 * max(1.0, np.abs(ref).max())
    # an explicit dense mask gives the same
    dq2, dk2, dv2 = oracle.backward(Q, K, V, dO, B, W, S, scale=scale, dense=oracle.dense_mask(N, B, W, S, use_power))
    assert np.abs(dq2 - dq).max() == 0 and np.abs(dk2 - dk).max() == 0 and np.abs(dv2 - dv).max() == 0


def test_backward_closed_forms(oracle):
    """What the calculus fixes without any reference: a constant upstream gradient per row gives
    dS = 0 when V is constant (dP equal for every key), hence dQ = dK = 0 and dV_j = sum of the
    weights that land on key j times dO; and the gradients of a single-key row are those of o = v."""
    import synth_inputs as si

    N, Hq, Hkv, D, B = 96, 2, 1, 8, 8
    Q, K = si.bf16_randn((1, N, Hq, D), 21), si.bf16_randn((1, N, Hkv, D), 22)
    vrow = si.bf16_randn((D,), 23)
    V = vrow.expand(1, N, Hkv, D).contiguous()
    dO = si.bf16_randn((1, N, Hq, D), 24)
    dq, dk, dv = oracle.backward(Q, K, V, dO, B, 2, 1)
    assert np.abs(dq).max() < 1e-12 and np.abs(dk).max() < 1e-12
    # column sums of the weights: sum_j dV_j = sum_i dO_i (each row's weights sum to one)
    assert np.abs(dv[0, :, 0].sum(axis=0) - dO[0].double().numpy().sum(axis=(0, 1))).max() < 1e-9
    # row 0 attends to key 0 only: o_0 = v_0, so dV_0 gets dO_0 of every head in full
    Vr = si.bf16_randn((1, N, Hkv, D), 25)
    dq, dk, dv = oracle.backward(Q, K, Vr, dO, B, 2, 1)
    assert np.abs(dq[0, 0]).max() < 1e-12            # a one-key softmax has no gradient in its logit


def test_backward_key_subset_equals_the_full_pass(oracle):
    import synth_inputs as si

    N, Hq, Hkv, D = 150, 4, 2, 16
    Q, K, V = si.bf16_randn((1, N, Hq, D), 31), si.bf16_randn((1, N, Hkv, D), 32), si.bf16_randn((1, N, Hkv, D), 33)
    dO = si.bf16_randn((1, N, Hq, D), 34)
    dq, dk, dv = oracle.backward(Q, K, V, dO, 8, 2, 1)
    keys = [0, 7, 8, 77, 149]
    dq2, dk2, dv2 = oracle.backward(Q, K, V, dO, 8, 2, 1, key_rows=keys)
    assert np.array_equal(dq, dq2)
    assert np.array_equal(dk[:, keys], dk2[:, keys]) and np.array_equal(dv[:, keys], dv2[:, keys])
    rest = np.setdiff1d(np.arange(N), keys)
    assert not dk2[:, rest].any() and not dv2[:, rest].any()
