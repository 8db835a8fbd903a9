"""GPU: pa_decode_static, the decode entry point for callers that cannot allocate device memory.

Hosts such as allocator callbacks, plug-ins inside a runtime that owns all device memory, or serving
loops that forbid allocation after warm-up cannot give pa_decode a workspace.  pa_decode_static keeps
the split-K scratch in an array built into the library, so here it is called through the C ABI twice
in a row (the second call finds the first call's leftovers in the shared array) and must reproduce
pa_decode's outputs both times.  This file sorts last so that a run that stops at the first failure
has already exercised everything else.
"""
import ctypes

import numpy as np
import pytest
import torch

import synth_inputs as si
from util import LSE_MAX_ABS, O_MAX_ABS

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pa():
    import paper_2503_03588_b200 as pa_

    return pa_


def test_static_decode_matches_workspace_decode_twice(pa):
    batch, max_len, Hq, Hkv, D, W, S = 6, 20000, 28, 4, 128, 5, 1
    kc = si.bf16_randn((batch, max_len, Hkv, D), 902).cuda()
    vc = si.bf16_randn((batch, max_len, Hkv, D), 903).cuda()
    # two different problems back to back: the second must not be disturbed by what the first left
    for call, (seed, lens) in enumerate([(901, [20000, 1, 64, 8193, 12345, 19999]),
                                         (911, [77, 16384, 20000, 4097, 3, 10000])]):
        q = si.bf16_randn((batch, Hq, D), seed).cuda()
        lens_d = torch.tensor(lens, dtype=torch.int32, device="cuda")
        o_ref, lse_ref, _ = pa.pa_decode(q, kc, vc, lens_d, W, S)
        o = torch.full_like(o_ref, float("nan"))
        lse = torch.full_like(lse_ref, float("nan"))
        pa.pa_decode_static(q, kc, vc, lens_d, W, S, o, lse)
        torch.cuda.synchronize()
        assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all(), call
        assert (o.float() - o_ref.float()).abs().max().item() <= O_MAX_ABS, call
        assert (lse - lse_ref).abs().max().item() <= LSE_MAX_ABS, call


def test_static_decode_against_the_oracle(pa, oracle):
    batch, max_len, Hq, Hkv, D, W, S = 3, 3000, 8, 2, 64, 5, 1
    q = si.bf16_randn((batch, Hq, D), 921)
    kc, vc = si.bf16_randn((batch, max_len, Hkv, D), 922), si.bf16_randn((batch, max_len, Hkv, D), 923)
    lens = np.array([3000, 65, 1500])
    o = torch.empty((batch, Hq, D), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((batch, Hq), dtype=torch.float32, device="cuda")
    pa.pa_decode_static(q.cuda(), kc.cuda(), vc.cuda(), torch.as_tensor(lens, dtype=torch.int32).cuda(), W, S, o, lse)
    torch.cuda.synchronize()
    o_ref, lse_ref, _ = oracle.decode(q, kc, vc, lens, 64, W, S)
    assert np.abs(o.double().cpu().numpy() - o_ref).max() <= O_MAX_ABS
    assert np.abs(lse.double().cpu().numpy() - lse_ref).max() <= LSE_MAX_ABS


def test_static_decode_rejects_problems_beyond_its_scratch(pa):
    """A batch whose partials need more than the built-in array is refused before any launch."""
    import paper_2503_03588_b200.binding as b

    s = b.pa_strides(131072 * 4 * 128, 4 * 128, 128)
    params = b.pa_decode_params(64, 28, 4, 128, 64, 5, 1, 131072, 0.0, s, s, b.PA_BF16)
    assert b.pa_decode_workspace_bytes(params) > b.PA_DECODE_STATIC_SCRATCH_BYTES
    dummy = torch.zeros(64, dtype=torch.int32, device="cuda")
    p = ctypes.c_void_p(dummy.data_ptr())
    st = b.lib.pa_decode_static(ctypes.byref(params), p, p, p, p, p, p, ctypes.c_void_p(0))
    assert b.pa_status_string(st) == "PA_ERR_WORKSPACE"
    assert b"built-in array" in b.lib.pa_last_error_message()
