"""GPU: pa_build_layout and the decode block list are bit-exact against the oracle."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pa():
    import paper_2503_03588_b200 as pa_

    return pa_


def _check(pa, oracle, N, B, W, S):
    rp, ci = pa.pa_build_layout(N, B, W, S)
    torch.cuda.synchronize()
    rp_ref, ci_ref = oracle.block_layout(N, B, W, S)
    assert rp.dtype == torch.int32 and ci.dtype == torch.int32
    np.testing.assert_array_equal(rp.cpu().numpy(), rp_ref)
    np.testing.assert_array_equal(ci.cpu().numpy(), ci_ref)


def test_layout_grid_bit_exact(pa, oracle):
    for N in (1, 63, 64, 65, 640, 2048, 4096 + 17, 70000):
        for W in (0, 1, 4, 5, 9):
            for S in (0, 1, 3):
                _check(pa, oracle, N, 64, W, S)
    for B in (4, 8, 256):
        _check(pa, oracle, 5000, B, 5, 1)


def test_layout_matches_token_level_brute_force(pa, oracle):
    for (N, B, W, S) in [(700, 8, 3, 1), (1000, 64, 5, 1), (513, 4, 0, 2)]:
        rp, ci = pa.pa_build_layout(N, B, W, S)
        rp_ref, ci_ref = oracle.block_layout_from_tokens(N, B, W, S)
        np.testing.assert_array_equal(rp.cpu().numpy(), rp_ref)
        np.testing.assert_array_equal(ci.cpu().numpy(), ci_ref)


@pytest.mark.parametrize("N,W,S", [(2048, 1, 1), (32768, 5, 1), (131072, 5, 1), (262144, 5, 1),
                                   (131072, 20, 4)])
def test_layout_workload_configs(pa, oracle, N, W, S):
    _check(pa, oracle, N, 64, W, S)


def test_tile_layout_bit_exact(pa, oracle):
    """The mask with `block`-token blocks listed by `tile`-token tiles: against the tile-level
    enumeration, against token-level brute force on small sizes, and at the paper's block size
    (256) for the 32K and 128K workloads."""
    def check(N, B, W, S, T, ref):
        rp, ci = pa.pa_build_tile_layout(N, B, W, S, T)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(rp.cpu().numpy(), ref[0])
        np.testing.assert_array_equal(ci.cpu().numpy(), ref[1])

    for N in (1, 64, 65, 255, 256, 257, 1000, 5000, 70000):
        for (W, S) in [(5, 1), (0, 0), (1, 2), (9, 3)]:
            check(N, 256, W, S, 64, oracle.tile_layout(N, 256, W, S, 64))
    for (N, B, W, S, T) in [(900, 256, 2, 1, 64), (700, 16, 3, 1, 4), (513, 8, 0, 2, 2), (640, 128, 1, 0, 64)]:
        check(N, B, W, S, T, oracle.tile_layout_from_tokens(N, B, W, S, T))
    check(5000, 64, 5, 1, 64, oracle.block_layout(5000, 64, 5, 1))      # tile == block
    for N in (32768, 131072):
        check(N, 256, 5, 1, 64, oracle.tile_layout(N, 256, 5, 1, 64))
    check(256 * 1500 + 77, 256, 5, 1, 64, oracle.tile_layout(256 * 1500 + 77, 256, 5, 1, 64))  # > 1 scan tile


def test_layout_larger_than_one_scan_tile(pa, oracle):
    _check(pa, oracle, 64 * 5000 + 5, 64, 5, 1)   # 5001 rows: several 1024-row scan tiles + tail


def test_decode_block_list_is_the_layout_row(pa, oracle):
    for (W, S) in [(5, 1), (0, 0), (1, 1), (9, 3)]:
        for L in (1, 64, 65, 4096, 65536, 65537, 100000, 131072):
            got = pa.pa_decode_block_list(L, 64, W, S).cpu().numpy()
            rp, ci = oracle.block_layout(L, 64, W, S)
            np.testing.assert_array_equal(got, ci[rp[-2]:rp[-1]])


def test_window_layout_bit_exact(pa, oracle):
    """pa_build_window_layout (window + sink, no power-of-two term) against the oracle's
    enumeration, against token-level brute force, and at the paper's 9 + 1 setting."""
    for N in (1, 64, 65, 640, 4096 + 17, 70000):
        for W in (1, 4, 9):
            for S in (0, 1, 3):
                rp, ci = pa.pa_build_window_layout(N, 64, W, S)
                rp_ref, ci_ref = oracle.block_layout(N, 64, W, S, use_power=False)
                np.testing.assert_array_equal(rp.cpu().numpy(), rp_ref)
                np.testing.assert_array_equal(ci.cpu().numpy(), ci_ref)
    for (N, B, W, S) in [(700, 8, 3, 1), (513, 4, 2, 2)]:
        rp, ci = pa.pa_build_window_layout(N, B, W, S)
        rp_ref, ci_ref = oracle.block_layout_from_tokens(N, B, W, S, use_power=False)
        np.testing.assert_array_equal(rp.cpu().numpy(), rp_ref)
        np.testing.assert_array_equal(ci.cpu().numpy(), ci_ref)
    rp, ci = pa.pa_build_window_layout(128 * 256, 256, 9, 1)
    assert (ci[int(rp[-2]):].cpu().numpy() + 1).tolist() == [1, 120, 121, 122, 123, 124, 125, 126, 127, 128]
    assert pa.pa_reach_counts(rp.cpu().numpy(), ci.cpu().numpy(), 127, 1) == [10]
