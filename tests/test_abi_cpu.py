"""CPU-side checks of the C ABI: the library loads without a GPU, exports every declared symbol,
and its host logic (closed-form layout sizes, argument validation) behaves as the header says."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def pa():
    from paper_2503_03588_b200 import build as _build

    _build.build()
    import paper_2503_03588_b200.binding as binding

    return binding


def test_every_declared_symbol_is_exported(pa):
    header = open(os.path.join(ROOT, "include", "powerattn.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(pa_[a-z_0-9]+)\s*\(", header))
    assert declared, "no declarations parsed"
    assert declared == set(pa.EXPORTS)
    for name in declared:
        assert hasattr(pa.lib, name), name


def test_status_strings_and_version(pa):
    assert pa.pa_version() >= 100
    for code, name in enumerate(pa.STATUS_NAMES):
        assert pa.pa_status_string(code) == name


def test_layout_size_matches_oracle(pa, oracle):
    for N in (1, 63, 64, 65, 2048, 4096 + 17, 32768):
        for W in (0, 1, 5, 9):
            for S in (0, 1, 3):
                nqb, nnz = pa.pa_layout_size(N, 64, W, S)
                rp, ci = oracle.block_layout(N, 64, W, S)
                assert nqb == len(rp) - 1 and nnz == int(rp[-1]) == len(ci), (N, W, S)
    # the paper's 256-token blocks and other block sizes
    for B in (4, 256):
        nqb, nnz = pa.pa_layout_size(32768, B, 5, 1)
        rp, _ = oracle.block_layout(32768, B, 5, 1)
        assert (nqb, nnz) == (len(rp) - 1, int(rp[-1]))


def test_tile_layout_size_matches_oracle(pa, oracle):
    """Masks with blocks that are a multiple of the 64-token tile (the paper's 256-token blocks)."""
    for (B, T) in [(256, 64), (128, 64), (64, 64), (8, 2), (256, 256)]:
        for N in (1, T, T + 1, B - 1, B, 5 * B + T + 3, 40 * B):
            for (W, S) in [(5, 1), (0, 0), (1, 2), (9, 3)]:
                nqt, nnz = pa.pa_tile_layout_size(N, B, W, S, T)
                rp, ci = oracle.tile_layout(N, B, W, S, T)
                assert nqt == len(rp) - 1 and nnz == int(rp[-1]) == len(ci), (N, B, T, W, S)
    assert pa.pa_tile_layout_size(32768, 64, 5, 1, 64) == pa.pa_layout_size(32768, 64, 5, 1)
    for bad in [(1000, 256, 5, 1, 96), (1000, 64, 5, 1, 128), (1000, 256, 5, 1, 0)]:
        with pytest.raises(pa.PaError):
            pa.pa_tile_layout_size(*bad)


def test_active_block_counts_of_the_workloads(pa):
    expect = {2048: 215, 4096: 502, 8192: 1141, 16384: 2548, 32768: 5619, 65536: 12274,
              131072: 26609, 262144: 57328}
    for N, nnz in expect.items():
        assert pa.pa_layout_size(N, 64, 5, 1) == (N // 64, nnz)
    assert pa.pa_layout_size(2048, 64, 1, 1) == (32, 187)


def test_argument_validation_happens_before_any_launch(pa, oracle):
    """These calls must fail on the host (no GPU is present in the CPU test run)."""
    with pytest.raises(pa.PaError, match="PA_ERR_INVALID_ARG"):
        pa.pa_layout_size(0, 64, 5, 1)
    with pytest.raises(pa.PaError, match="PA_ERR_INVALID_ARG"):
        pa.pa_layout_size(128, 64, -1, 1)
    null = ctypes.c_void_p(0)
    st = pa.lib.pa_build_layout(4096, 64, 5, 1, null, null, 10**6, null)
    assert pa.pa_status_string(st) == "PA_ERR_INVALID_ARG"
    buf = (ctypes.c_int32 * 64)()
    st = pa.lib.pa_build_layout(4096, 64, 5, 1, ctypes.addressof(buf), ctypes.addressof(buf), 10, null)
    assert pa.pa_status_string(st) == "PA_ERR_LAYOUT"
    assert b"col_capacity" in pa.lib.pa_last_error_message()

    s = pa.pa_strides(0, 512, 128)
    good = pa.pa_prefill_params(1, 4, 2, 128, 4096, 64, 0.0, s, s, s, s, pa.PA_BF16)
    p = ctypes.addressof(buf)

    def prefill_status(params, q=p, nnz=10**6, ws=p, ws_bytes=256):
        return pa.pa_status_string(pa.lib.pa_prefill(ctypes.byref(params), q, p, p, p, p, nnz, p, p, ws,
                                                     ws_bytes, null))

    bad = pa.pa_prefill_params.from_buffer_copy(good); bad.head_dim = 96
    assert prefill_status(bad) == "PA_ERR_SHAPE"
    bad = pa.pa_prefill_params.from_buffer_copy(good); bad.block = 128
    assert prefill_status(bad) == "PA_ERR_SHAPE"
    bad = pa.pa_prefill_params.from_buffer_copy(good); bad.n_q_heads = 3
    assert prefill_status(bad) == "PA_ERR_SHAPE"
    bad = pa.pa_prefill_params.from_buffer_copy(good); bad.q = pa.pa_strides(0, 516, 128)
    assert prefill_status(bad) == "PA_ERR_ALIGNMENT"
    assert prefill_status(good, q=0) == "PA_ERR_INVALID_ARG"
    assert prefill_status(good, q=p + 4) == "PA_ERR_ALIGNMENT"
    assert prefill_status(good, nnz=-1) == "PA_ERR_LAYOUT"
    assert prefill_status(good, ws_bytes=8) == "PA_ERR_WORKSPACE"

    dgood = pa.pa_decode_params(2, 4, 2, 128, 64, 5, 1, 4096, 0.0, s, s, pa.PA_BF16)
    # one (o[128], m, l) slot per query head and chunk; chunks = the longest block list of any row
    rp_ref, _ = oracle.block_layout(4096, 64, 5, 1)
    # a 256-byte status block, then one (o[128], m, l) slot per query head and chunk
    chunks = (pa.pa_decode_workspace_bytes(dgood) - 256) // (2 * 4 * 130 * 4)
    assert pa.pa_decode_workspace_bytes(dgood) == 256 + 2 * 4 * chunks * 130 * 4
    assert chunks == int(np.diff(rp_ref).max()) == 9
    dbad = pa.pa_decode_params.from_buffer_copy(dgood); dbad.n_q_heads = 40
    assert pa.pa_decode_workspace_bytes(dbad) == 0
    st = pa.lib.pa_decode(ctypes.byref(dbad), p, p, p, p, p, p, p, 10**6, null)
    assert pa.pa_status_string(st) == "PA_ERR_SHAPE"
    st = pa.lib.pa_decode(ctypes.byref(dgood), p, p, p, p, p, p, p, 16, null)
    assert pa.pa_status_string(st) == "PA_ERR_WORKSPACE"
    st = pa.lib.pa_decode_block_list(0, 64, 5, 1, p, p, 64, null)
    assert pa.pa_status_string(st) == "PA_ERR_INVALID_ARG"
    st = pa.lib.pa_decode_row_block_set(4096, 64, 40, 1, p, p, 64, null)   # more than 32 candidates
    assert pa.pa_status_string(st) == "PA_ERR_SHAPE"
    st = pa.lib.pa_decode_row_block_set(4096, 64, 5, 1, p, p, 8, null)     # capacity below one warp
    assert pa.pa_status_string(st) == "PA_ERR_INVALID_ARG"

    sp = pa.pa_strides(64 * 2 * 128, 2 * 128, 128)
    pgood = pa.pa_paged_params(2, 4, 2, 128, 64, 5, 1, 100, 64, 0.0, sp, sp, pa.PA_BF16)
    assert pa.pa_decode_paged_workspace_bytes(pgood) == pa.pa_decode_workspace_bytes(dgood)  # 64 blocks = 4096 tokens
    pbad = pa.pa_paged_params.from_buffer_copy(pgood); pbad.n_pages = 0
    assert pa.pa_decode_paged_workspace_bytes(pbad) == 0
    st = pa.lib.pa_decode_paged(ctypes.byref(pgood), p, p, p, 0, p, p, p, p, 10**6, null)
    assert pa.pa_status_string(st) == "PA_ERR_INVALID_ARG"                 # null block table
    st = pa.lib.pa_kv_append(ctypes.byref(pgood), p, p, p, p, p, 0, null)
    assert pa.pa_status_string(st) == "PA_ERR_INVALID_ARG"                 # null cache_lens
    st = pa.lib.pa_decode_status(0, null, None)
    assert pa.pa_status_string(st) == "PA_ERR_INVALID_ARG"


def test_window_layout_size_matches_oracle(pa, oracle):
    """Sliding window (window + sink blocks, no power-of-two term), Section 4.1 "Baseline"."""
    for N in (1, 64, 65, 2048, 4096 + 17, 32768):
        for W in (1, 4, 9):
            for S in (0, 1, 3):
                nqb, nnz = pa.pa_window_layout_size(N, 64, W, S)
                rp, ci = oracle.block_layout(N, 64, W, S, use_power=False)
                assert nqb == len(rp) - 1 and nnz == int(rp[-1]) == len(ci), (N, W, S)
    with pytest.raises(pa.PaError, match="PA_ERR_INVALID_ARG"):
        pa.pa_window_layout_size(4096, 64, 0, 1)      # no window: the diagonal block would be missing


def _read_golden(name):
    out = {}
    with open(os.path.join(ROOT, "tests", "golden", name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                key, *vals = line.split()
                out[key] = [int(v) for v in vals]
    return out


def test_reach_counts_against_the_paper_and_the_oracle(pa, oracle):
    """pa_reach_counts (host BFS over a CSR) on the layouts of the appendix's setting: |B_1| = 10 of
    128 blocks for the 9 + 1 sliding window (Appendix A), the default pattern's 10-block budget and
    full coverage within six steps (Section 4.1, Section 4.3), and the oracle's BFS everywhere."""
    g = _read_golden("sliding_window_B1.txt")
    n, W, S = g["n_blocks"][0], g["window_blocks"][0], g["sink_blocks"][0]
    rp, ci = oracle.block_layout(n * 256, 256, W, S, use_power=False)
    counts = pa.pa_reach_counts(rp, ci, n - 1, 20)
    assert counts[0] == g["alpha1_numerator"][0] == len(g["B1"])
    assert counts == oracle.reach_counts(oracle.block_adjacency(n, W, S, use_power=False), n - 1, 20)
    d = _read_golden("power_attention_default.txt")
    n, W, S = d["n_blocks"][0], d["window_blocks"][0], d["sink_blocks"][0]
    rp, ci = oracle.block_layout(n * 256, 256, W, S)
    counts = pa.pa_reach_counts(rp, ci, n - 1, 8)
    assert counts[0] == d["last_row_blocks"][0]
    assert counts[d["full_coverage_layers_at_most"][0] - 1] == n and counts[d["full_coverage_layers_at_most"][0] - 2] < n
    assert counts == oracle.reach_counts(oracle.block_adjacency(n, W, S), n - 1, 8)
    for start in (0, 1, 77):
        assert pa.pa_reach_counts(rp, ci, start, 5) == oracle.reach_counts(oracle.block_adjacency(n, W, S), start, 5)
    bad = ci.copy(); bad[-1] = n
    with pytest.raises(pa.PaError, match="PA_ERR_LAYOUT"):
        pa.pa_reach_counts(rp, bad, n - 1, 3)
    with pytest.raises(pa.PaError, match="PA_ERR_INVALID_ARG"):
        pa.pa_reach_counts(rp, ci, n, 3)


def test_backward_workspace_size_and_validation(pa):
    """Host side of pa_prefill_backward: the workspace holds a 256-byte status block, delta
    [batch, Hq, N] fp32 (rounded up to 256 bytes) and the transposed layout (two arrays of nqb + 1 and
    one of nnz int32), the sum rounded up to 256 bytes; bad arguments fail before any launch."""
    s = pa.pa_strides(0, 512, 128)
    good = pa.pa_prefill_params(2, 4, 2, 128, 4100, 64, 0.0, s, s, s, s, pa.PA_BF16)
    nnz = 777
    nqb = (4100 + 63) // 64
    delta = 256 + 2 * 4 * 4100 * 4
    delta = (delta + 255) // 256 * 256
    want = (delta + (2 * (nqb + 1) + nnz) * 4 + 255) // 256 * 256
    assert pa.lib.pa_prefill_backward_workspace_bytes(ctypes.byref(good), nnz) == want
    bad = pa.pa_prefill_params.from_buffer_copy(good); bad.o_dtype = pa.PA_F32
    assert pa.lib.pa_prefill_backward_workspace_bytes(ctypes.byref(bad), nnz) == 0
    buf = (ctypes.c_int32 * 64)()
    p, null = ctypes.addressof(buf), ctypes.c_void_p(0)

    def status(params, q=p, ws=p, ws_bytes=10**9, n=nnz):
        return pa.pa_status_string(pa.lib.pa_prefill_backward(ctypes.byref(params), q, p, p, p, p, p, p, p, n, p, p, p,
                                                              ws, ws_bytes, null))

    assert status(bad) == "PA_ERR_SHAPE"
    bad = pa.pa_prefill_params.from_buffer_copy(good); bad.head_dim = 32
    assert status(bad) == "PA_ERR_SHAPE"
    assert status(good, q=0) == "PA_ERR_INVALID_ARG"
    assert status(good, q=p + 2) == "PA_ERR_ALIGNMENT"
    assert status(good, ws_bytes=want - 1) == "PA_ERR_WORKSPACE"
    assert status(good, n=-5) == "PA_ERR_LAYOUT"
