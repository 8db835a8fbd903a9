"""Pins for the oracle's mask predicate, block layouts and receptive-field analysis.

Each test ties the oracle to something the paper or the mathematics fixes -- a printed worked
example, a stated parameter budget, the appendix theorem, a closed form -- not to itself.
"""
import os

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = [int(v) for v in vals]
    return out


# ------------------------------------------------------------------ the paper's worked examples

def test_sliding_window_worked_example(oracle):
    """Appendix A: B_1 of sliding window (9 + 1 sink, 128 blocks) = {1, 120..128}, 1-based.
    Pins the window convention (distances 0..W-1), the sink term and causality."""
    g = _read_golden("sliding_window_B1.txt")
    n, W, S = g["n_blocks"][0], g["window_blocks"][0], g["sink_blocks"][0]
    adj = oracle.block_adjacency(n, W, S, use_power=False)
    assert [j + 1 for j in adj[n - 1]] == g["B1"]
    assert oracle.reach_counts(adj, n - 1, 1)[0] == g["alpha1_numerator"][0]
    # the same through the token-level predicate with the paper's 256-token blocks
    B = 256
    q = n * B - 1
    blocks = sorted({kv // B + 1 for kv in range(0, n * B, 64)
                     if oracle.mask(q, kv, B, W, S, use_power=False)})
    assert blocks == g["B1"]


def test_default_pattern_budget(oracle):
    """Section 4.1: 5 window + 1 sink + 4 power blocks = the sliding window's 10-block budget."""
    g = _read_golden("power_attention_default.txt")
    n, W, S = g["n_blocks"][0], g["window_blocks"][0], g["sink_blocks"][0]
    adj = oracle.block_adjacency(n, W, S)
    last = adj[n - 1]
    assert len(last) == g["last_row_blocks"][0]
    dist = [n - 1 - j for j in last]
    window = [d for d in dist if d < W]
    sink = [j for j in last if j < S]
    extra = [d for d, j in zip(dist, last) if d >= W and j >= S]
    assert len(window) == W and len(sink) == S
    assert len(extra) == g["extra_power_blocks"][0]
    assert all(d & (d - 1) == 0 for d in extra)           # power-of-2 intervals
    assert sorted(extra) == [8, 16, 32, 64]


def test_full_coverage_within_six_layers(oracle):
    """Section 4.3 / Fig. 1(a): at 128 blocks the last block reaches everything in <= 6 steps;
    the sliding window of equal budget does not (O(N) layers, Section 3.2)."""
    g = _read_golden("power_attention_default.txt")
    n = g["n_blocks"][0]
    adj = oracle.block_adjacency(n, g["window_blocks"][0], g["sink_blocks"][0])
    dist = oracle.bfs_distances(adj, n - 1)
    assert dist.min() >= 0 and dist.max() <= g["full_coverage_layers_at_most"][0]
    counts = oracle.reach_counts(adj, n - 1, 6)
    assert counts[0] == 10 and counts[-1] == n and counts == sorted(counts)
    sw = oracle.block_adjacency(n, 9, 1, use_power=False)
    dsw = oracle.bfs_distances(sw, n - 1)
    assert dsw.max() == int(np.ceil((n - 2) / 8))          # 8 new blocks per layer: linear
    assert oracle.reach_counts(sw, n - 1, 6)[-1] < n


# ------------------------------------------------------------------ Appendix B theorem

def test_theorem_distance_is_popcount(oracle):
    """Appendix B: on E = {(i,j): i-j = 2^k} the path built from the binary expansion of i-j has
    popcount(i-j) edges; BFS shows no shorter one exists, and every distance is <= log2 n."""
    n = 2048
    adj = oracle.power_graph(n)
    for start in (n - 1, 1500, 1023, 7):
        dist = oracle.bfs_distances(adj, start)
        for j in range(start + 1):
            assert dist[j] == bin(start - j).count("1")
        assert dist[: start + 1].max() <= np.log2(n)
        assert (dist[start + 1:] == -1).all()              # DAG: nothing later is reachable


def test_theorem_out_degree(oracle):
    """Appendix B (1): one edge per k with 2^k <= i, i.e. bit_length(i) edges for 0-based i."""
    n = 4096
    adj = oracle.power_graph(n)
    for i in range(n):
        assert len(adj[i]) == i.bit_length()
        assert len(adj[i]) <= np.log2(n)


def test_receptive_field_grows_as_two_to_the_d(oracle):
    """Abstract / Section 3.3: after d layers a token sees a complete, continuous span of at
    least 2^d positions.  On the pure power graph the span is exactly min(i+1, 2^(d+1)-1)."""
    n = 2048
    pure = oracle.power_graph(n)
    # the block mask with W <= 1 and no sink is the power graph plus self loops
    blk = oracle.block_adjacency(n, 0, 0)
    for d in range(1, 12):
        c_pure = oracle.contiguous_reach(pure, n - 1, d)
        c_blk = oracle.contiguous_reach(blk, n - 1, d)
        assert c_pure == min(n, 2 ** (d + 1) - 1)
        assert c_blk == c_pure
        assert c_pure >= min(n, 2 ** d)
    full = oracle.block_adjacency(n, 5, 1)
    for d in range(1, 12):
        assert oracle.contiguous_reach(full, n - 1, d) >= min(n, 2 ** d)
    assert oracle.bfs_distances(full, n - 1).max() <= 11


# ------------------------------------------------------------------ predicate, term by term

def test_predicate_terms(oracle):
    B, W = 8, 3
    m = lambda q, kv, S=1, p=True: oracle.mask(q, kv, B, W, S, p)
    assert not m(10, 11)                                   # causal
    assert m(10, 10) and m(10, 8) and not m(8, 10)         # diagonal block, token-level causal
    q = 20 * B + 3
    for d in range(0, 21):
        kv = (20 - d) * B + 7                              # a later offset inside an earlier block
        expect = d < W or d in (1, 2, 4, 8, 16) or (20 - d) < 1
        if d == 0:
            expect = False                                 # kv offset 7 > q offset 3
        assert m(q, kv) == expect, d
    assert m(q, 5) and not m(q, 8, 1)                      # sink is exactly the first S*B tokens
    assert m(q, 15, 2) and not m(q, 16, 2)
    assert not m(q, 5, 0) and not m(q, 5 * B + 1, 1)       # d = 15: not window, power or sink
    assert m(q, 4 * B, 1) and not m(q, 4 * B, 1, False)    # d = 16 only through the power term


def test_dense_mask_is_causal_and_keeps_diagonal(oracle):
    for (N, B, W, S) in [(96, 8, 2, 1), (100, 16, 0, 0), (64, 4, 5, 2)]:
        m = oracle.dense_mask(N, B, W, S)
        assert not np.triu(m, 1).any()
        assert np.diag(m).all()                            # no empty rows: kv = q always passes
        # inside the diagonal block the mask is exactly lower triangular
        for i in range(N // B):
            blk = m[i * B:(i + 1) * B, i * B:(i + 1) * B]
            assert (blk == np.tril(np.ones((B, B), bool))).all()
        # every other listed block pair is fully visible (only the diagonal is partial)
        nb = N // B
        for i in range(nb):
            for j in range(i):
                blk = m[i * B:(i + 1) * B, j * B:(j + 1) * B]
                assert blk.all() or not blk.any()


def test_window_sizes_0_to_3_coincide(oracle):
    """Distances 0, 1, 2 are powers of two (0 passes x & (x-1) == 0), so W in {0,1,2,3} agree."""
    ref = oracle.block_layout(1024, 8, 0, 1)
    for W in (1, 2, 3):
        got = oracle.block_layout(1024, 8, W, 1)
        assert (got[0] == ref[0]).all() and (got[1] == ref[1]).all()
    assert oracle.block_layout(1024, 8, 4, 1)[0][-1] > ref[0][-1]


# ------------------------------------------------------------------ layouts

@pytest.mark.parametrize("B", [4, 8, 64])
def test_block_layout_matches_token_brute_force(oracle, B):
    """Block-level enumeration == brute force over every token pair, ragged tails included."""
    for N in (1, B - 1, B, B + 1, 5 * B, 9 * B + 3, 17 * B - 1, min(1024, 40 * B)):
        for W in (0, 1, 4, 5, 8):
            for S in (0, 1, 3):
                a = oracle.block_layout_from_tokens(N, B, W, S)
                b = oracle.block_layout(N, B, W, S)
                assert (a[0] == b[0]).all() and (a[1] == b[1]).all(), (N, B, W, S)


def test_row_length_closed_form(oracle):
    """|row i| = |{d < min(W, i+1)} U {2^k <= i} U {0} U {i-j : j < min(S, i+1)}| as distances."""
    for (W, S) in [(5, 1), (1, 1), (0, 0), (9, 2), (3, 0)]:
        n = 700
        rp, ci = oracle.block_layout(n * 4, 4, W, S)
        for i in range(n):
            ds = {0} | set(range(min(W, i + 1))) | {i - j for j in range(min(S, i + 1))}
            k = 1
            while k <= i:
                ds.add(k)
                k *= 2
            assert rp[i + 1] - rp[i] == len(ds)
            row = ci[rp[i]:rp[i + 1]]
            assert (np.diff(row) > 0).all() and row[-1] == i
            assert sorted(i - j for j in row) == sorted(ds)


def test_block_row_at_large_indices(oracle):
    """Rows far beyond the sizes the brute force reaches: the vector form of the block predicate
    against the scalar one on every j <= i, and against the closed-form set of distances."""
    for (W, S) in [(5, 1), (0, 0), (9, 3), (26, 4)]:
        for i in (4095, 4096, 4097, 5000, 8191, 8192, 16383, 16384, 70001):
            row = oracle.block_row(i, W, S)
            scalar = [j for j in range(i + 1) if oracle.block_predicate(i, j, W, S)]
            assert row.tolist() == scalar, (i, W, S)
            ds = set(range(min(max(W, 1), i + 1))) | {i - j for j in range(min(S, i + 1))}
            k = 1
            while k <= i:
                ds.add(k)
                k *= 2
            assert sorted(i - j for j in row.tolist()) == sorted(ds), (i, W, S)
        nopow = oracle.block_row(5000, W, S, use_power=False)
        assert nopow.tolist() == [j for j in range(5001) if oracle.block_predicate(5000, j, W, S, False)]


def test_active_block_counts_scale_as_n_log_n(oracle):
    """Section 4.5: O(N log N).  nnz / (nqb * log2 nqb) stays bounded and nnz < dense triangle."""
    prev = None
    for N in (4096, 16384, 65536, 262144):
        rp, _ = oracle.block_layout(N, 64, 5, 1)
        nqb = N // 64
        nnz = int(rp[-1])
        assert nnz < nqb * (5 + 1 + np.log2(nqb))
        assert nnz > nqb * (np.log2(nqb) - 2)
        if prev is not None:
            assert 4 < nnz / prev < 4 * 1.3                 # 4x tokens -> a little over 4x blocks
        prev = nnz
    # the paper's 128K kernel-speedup setting (256-token blocks): dense / sparse block ratio
    rp, _ = oracle.block_layout(131072, 256, 5, 1)
    nqb = 512
    assert 20 < (nqb * (nqb + 1) // 2) / int(rp[-1]) < 27   # paper reports 21.6x in time


# ------------------------------------------------------------------ tile layouts (tile != block)

@pytest.mark.parametrize("B,T", [(8, 2), (16, 4), (256, 64)])
def test_tile_layout_matches_token_brute_force(oracle, B, T):
    """Tile-level enumeration == brute force over every token pair when the mask's block is a
    multiple of the tile (the paper's 256-token blocks on 64-token tiles, Section 4.1)."""
    for N in (1, T + 1, B - 1, B, B + T + 1, 3 * B + 1, 7 * B - T - 1, min(1280, 12 * B)):
        for W in (0, 1, 3, 5):
            for S in (0, 1, 2):
                a = oracle.tile_layout_from_tokens(N, B, W, S, T)
                b = oracle.tile_layout(N, B, W, S, T)
                assert (a[0] == b[0]).all() and (a[1] == b[1]).all(), (N, B, T, W, S)


def test_tile_layout_special_cases(oracle):
    """T == B is the block layout; row length in closed form; the tiles' token count equals the
    token mask's row sums (64 * tiles - (63 - q mod 64) per row, the diagonal tile being partial)."""
    for (N, B, W, S) in [(1000, 8, 5, 1), (515, 4, 0, 0)]:
        a, b = oracle.tile_layout(N, B, W, S, B), oracle.block_layout(N, B, W, S)
        assert (a[0] == b[0]).all() and (a[1] == b[1]).all()
    N, B, T, W, S = 1536, 256, 64, 2, 1
    r = B // T
    rp, ci = oracle.tile_layout(N, B, W, S, T)
    brp, _ = oracle.block_layout(N, B, W, S)
    m = oracle.dense_mask(N, B, W, S)
    for ti in range(N // T):
        i = ti // r
        assert rp[ti + 1] - rp[ti] == r * (brp[i + 1] - brp[i] - 1) + (ti - i * r + 1)
        row = ci[rp[ti]:rp[ti + 1]]
        assert (np.diff(row) > 0).all() and row[-1] == ti
        for q in (ti * T, ti * T + 17, ti * T + T - 1):
            assert m[q].sum() == T * len(row) - (T - 1 - q % T)
