"""GPU: pa_decode_static, the decode entry point for callers that cannot allocate device memory.

Hosts such as allocator callbacks, plug-ins inside a runtime that owns all device memory, or serving
loops that forbid allocation after warm-up cannot give pa_decode a workspace.  pa_decode_static keeps
that workspace in an array built into the library.  The array is only written and read on the
two-kernel (split-K) decode path, so these tests force that path: the entry point is called through
the C ABI twice in a row on different problems (the second call finds the first call's partial
results in the shared array) and must reproduce both pa_decode's outputs and the oracle's both
times.  One case keeps the default single-launch path, which uses only the array's status block.
This file sorts last so that a run that stops at the first failure has already exercised everything
else.
"""
import ctypes

import numpy as np
import pytest
import torch

import synth_inputs as si
from util import LSE_MAX_ABS, O_MAX_ABS, compare

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pa():
    import paper_2503_03588_b200 as pa_

    return pa_


def _two_calls(pa, oracle, batch, max_len, Hq, Hkv, D, W, S, problems):
    kc_h = si.bf16_randn((batch, max_len, Hkv, D), 902)
    vc_h = si.bf16_randn((batch, max_len, Hkv, D), 903)
    kc, vc = kc_h.cuda(), vc_h.cuda()
    for call, (seed, lens) in enumerate(problems):
        q_h = si.bf16_randn((batch, Hq, D), seed)
        q = q_h.cuda()
        lens_d = torch.tensor(lens, dtype=torch.int32, device="cuda")
        o_ws, lse_ws, _ = pa.pa_decode(q, kc, vc, lens_d, W, S)
        o = torch.full_like(o_ws, float("nan"))
        lse = torch.full_like(lse_ws, float("nan"))
        pa.pa_decode_static(q, kc, vc, lens_d, W, S, o, lse)
        torch.cuda.synchronize()
        assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all(), call
        assert (o.float() - o_ws.float()).abs().max().item() <= O_MAX_ABS, call
        assert (lse - lse_ws).abs().max().item() <= LSE_MAX_ABS, call
        o_ref, lse_ref, _ = oracle.decode(q_h, kc_h, vc_h, np.asarray(lens), 64, W, S)
        compare(o, lse, o_ref, lse_ref, f"static decode, call {call}")


def test_static_decode_through_its_scratch_array_twice(pa, oracle, pa_env):
    """Split-K forced: both kernels go through the built-in array; two different problems back to
    back, the second of which must not be disturbed by what the first left there."""
    pa_env(PA_DECODE_PATH="splitk")
    _two_calls(pa, oracle, 6, 20000, 28, 4, 128, 5, 1,
               [(901, [20000, 1, 64, 8193, 12345, 19999]), (911, [77, 16384, 20000, 4097, 3, 10000])])


def test_static_decode_with_a_window_too_wide_for_one_launch(pa, oracle):
    """A 40-block window has more than 32 candidates per row, so the library itself takes the
    two-kernel path (no switch) and the array holds the partial results."""
    _two_calls(pa, oracle, 3, 6000, 8, 2, 64, 40, 2, [(921, [6000, 65, 3000]), (922, [1, 5999, 2560])])


def test_static_decode_on_the_single_launch_path(pa, oracle):
    """The default path for the paper's window: only the status block of the array is used."""
    _two_calls(pa, oracle, 3, 3000, 8, 2, 64, 5, 1, [(931, [3000, 65, 1500]), (932, [64, 2999, 1])])


def test_static_decode_rejects_problems_beyond_its_scratch(pa):
    """A two-kernel-path problem whose partial results need more than the built-in array is
    refused before any launch; the same batch on the single-launch path is not bound by the limit
    (it is refused here only later, for its null pointers)."""
    import paper_2503_03588_b200.binding as b

    s = b.pa_strides(131072 * 4 * 128, 4 * 128, 128)
    params = b.pa_decode_params(64, 28, 4, 128, 64, 40, 1, 131072, 0.0, s, s, b.PA_BF16)
    assert b.pa_decode_workspace_bytes(params) > b.PA_DECODE_STATIC_SCRATCH_BYTES
    dummy = torch.zeros(64, dtype=torch.int32, device="cuda")
    p = ctypes.c_void_p(dummy.data_ptr())
    st = b.lib.pa_decode_static(ctypes.byref(params), p, p, p, p, p, p, ctypes.c_void_p(0))
    assert b.pa_status_string(st) == "PA_ERR_WORKSPACE"
    assert b"built-in array" in b.lib.pa_last_error_message()
    params.window_blocks = 5
    assert b.pa_decode_workspace_bytes(params) > b.PA_DECODE_STATIC_SCRATCH_BYTES
    st = b.lib.pa_decode_static(ctypes.byref(params), ctypes.c_void_p(0), p, p, p, p, p, ctypes.c_void_p(0))
    assert b.pa_status_string(st) == "PA_ERR_INVALID_ARG"
