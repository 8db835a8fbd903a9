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


@pytest.mark.parametrize("env", [{"PA_DECODE_PATH": "splitk"}, {"PA_DECODE_CLUSTER": "1"}, {"PA_DECODE_CLUSTER": "2"},
                                 {"PA_DECODE_CLUSTER": "7"}, {"PA_DECODE_CLUSTER": "8"},
                                 {"PA_DECODE_CLUSTER": "2", "PA_DECODE_STAGES": "2"},
                                 {"PA_DECODE_CLUSTER": "1", "PA_DECODE_STAGES": "3"},
                                 {"PA_DECODE_CLUSTER": "8", "PA_DECODE_STAGES": "1"}])
def test_decode_paths(pa, oracle, monkeypatch, env):
    """The two-launch split-K path and the single-launch cluster path at several cluster sizes and
    ring depths (the library reads these switches on every call) give the same row of Eq. (1)."""
    for k, v in env.items():
        monkeypatch.setenv(k, v)
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
