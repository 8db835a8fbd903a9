"""PowerAttention CPU oracle -- TEST INFRASTRUCTURE ONLY.

Python face of ``pa_oracle.c`` (fp64, dense token-level mask, Eq. (1) row by row) plus the
graph-side checks of the paper: brute-force block layout from the token mask, the block-level
predicate for large sizes, and breadth-first reachability over the mask seen as a DAG
(Section 3.1; Appendix A; Appendix B); and the gradients of Eq. (1) for the backward pass.

The product library never imports this module; this module never imports the product.
Every function here is pinned by ``tests/test_oracle_*.py``; none is "parity unpinned".
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pa_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None

_i64 = ctypes.c_int64
_p = ctypes.c_void_p


def build(force: bool = False) -> str:
    """Compile pa_oracle.c with gcc (+OpenMP) into liboracle.so next to it."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        lib.pa_oracle_mask.restype = ctypes.c_int
        lib.pa_oracle_mask.argtypes = [_i64, _i64, _i64, _i64, _i64, ctypes.c_int]
        lib.pa_oracle_mask_row.restype = None
        lib.pa_oracle_mask_row.argtypes = [_i64, _i64, _i64, _i64, _i64, ctypes.c_int, _p]
        lib.pa_oracle_prefill.restype = None
        lib.pa_oracle_prefill.argtypes = [_p, _p, _p, _i64, _i64, _i64, _i64, _i64,
                                          ctypes.c_double, _i64, _i64, _i64, ctypes.c_int, _p,
                                          _p, _i64, _p, _i64, _p, _p, _p, ctypes.c_int]
        lib.pa_oracle_decode.restype = None
        lib.pa_oracle_decode.argtypes = [_p, _p, _p, _p, _i64, _i64, _i64, _i64, _i64,
                                         ctypes.c_double, _i64, _i64, _i64, ctypes.c_int, _p, _p,
                                         _p, ctypes.c_int]
        lib.pa_oracle_backward.restype = None
        lib.pa_oracle_backward.argtypes = [_p, _p, _p, _p, _i64, _i64, _i64, _i64, _i64, ctypes.c_double, _i64, _i64,
                                           _i64, ctypes.c_int, _p, _p, _i64, _p, _p, _p, ctypes.c_int]
        lib.pa_oracle_max_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def max_threads() -> int:
    return int(_load().pa_oracle_max_threads())


def _bf16_bits(x) -> np.ndarray:
    """bf16 torch tensor (CPU) or uint16 numpy array -> contiguous uint16 numpy array."""
    if isinstance(x, np.ndarray):
        assert x.dtype == np.uint16, "numpy inputs must be bf16 bit patterns (uint16)"
        return np.ascontiguousarray(x)
    import torch  # only for the view; no arithmetic

    assert x.dtype == torch.bfloat16 and x.device.type == "cpu"
    return x.contiguous().view(torch.int16).numpy().view(np.uint16)


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(_p)


# --------------------------------------------------------------------------- mask (Algorithm 1)

def mask(q_idx: int, kv_idx: int, B: int, W: int, S: int = 1, use_power: bool = True) -> bool:
    """Algorithm 1 (Section 3.3) for one (q_idx, kv_idx); S sink blocks (paper: 1)."""
    return bool(_load().pa_oracle_mask(q_idx, kv_idx, B, W, S, int(use_power)))


def dense_mask(N: int, B: int, W: int, S: int = 1, use_power: bool = True) -> np.ndarray:
    """The whole token-level mask as a dense [N, N] bool matrix (row = query, column = key)."""
    lib = _load()
    out = np.zeros((N, N), dtype=np.uint8)
    for q in range(N):
        lib.pa_oracle_mask_row(q, N, B, W, S, int(use_power), out[q].ctypes.data_as(_p))
    return out.astype(bool)


# --------------------------------------------------------------------------- block layouts

def _csr_from_block_matrix(blk: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    nqb = blk.shape[0]
    row_ptr = np.zeros(nqb + 1, dtype=np.int32)
    cols = []
    for i in range(nqb):
        js = np.nonzero(blk[i])[0]
        cols.append(js.astype(np.int32))
        row_ptr[i + 1] = row_ptr[i] + len(js)
    col_idx = np.concatenate(cols) if cols else np.zeros(0, dtype=np.int32)
    return row_ptr, col_idx.astype(np.int32)


def block_layout_from_tokens(N: int, B: int, W: int, S: int = 1,
                             use_power: bool = True) -> Tuple[np.ndarray, np.ndarray]:
    """Brute force: key block j is listed for query block i iff some token pair (q, kv) in
    those blocks satisfies the token-level predicate.  O(N^2); for small N only."""
    m = dense_mask(N, B, W, S, use_power)
    nb = -(-N // B)
    pad = np.zeros((nb * B, nb * B), dtype=bool)
    pad[:N, :N] = m
    blk = pad.reshape(nb, B, nb, B).any(axis=(1, 3))
    return _csr_from_block_matrix(blk)


def block_predicate(i: int, j: int, W: int, S: int = 1, use_power: bool = True) -> bool:
    """Algorithm 1 applied to block indices: with equal, aligned query and key blocks the
    window and power terms depend on i - j only, the sink term on j < S, causality on j <= i."""
    if j > i:
        return False
    d = i - j
    return (d < W) or (use_power and (d & (d - 1)) == 0) or (j < S)


def block_row(i: int, W: int, S: int = 1, use_power: bool = True) -> np.ndarray:
    """Every key block j = 0..i that block_predicate lists for query block i, ascending: the
    predicate written out on the whole index range at once (no candidate pruning)."""
    j = np.arange(i + 1, dtype=np.int64)
    d = i - j
    keep = (d < W) | (j < S)
    if use_power:
        keep |= (d & (d - 1)) == 0
    return j[keep].astype(np.int32)


def block_layout(N: int, B: int, W: int, S: int = 1,
                 use_power: bool = True) -> Tuple[np.ndarray, np.ndarray]:
    """Block-level enumeration of every (i, j) pair with j <= i; usable at large N."""
    nb = -(-N // B)
    row_ptr = np.zeros(nb + 1, dtype=np.int32)
    cols = []
    for i in range(nb):
        js = block_row(i, W, S, use_power)
        cols.append(js)
        row_ptr[i + 1] = row_ptr[i] + len(js)
    col_idx = np.concatenate(cols) if cols else np.zeros(0, dtype=np.int32)
    return row_ptr, col_idx.astype(np.int32)


def tile_layout_from_tokens(N: int, B: int, W: int, S: int, T: int,
                            use_power: bool = True) -> Tuple[np.ndarray, np.ndarray]:
    """Brute force at a tile size T that differs from the mask's block size B (the paper's
    efficiency runs use B = 256, Section 4.1): key tile tj is listed for query tile ti iff some
    token pair (q, kv) in those T-token tiles satisfies the token-level predicate of
    Algorithm 1 evaluated with block size B.  O(N^2); for small N only."""
    m = dense_mask(N, B, W, S, use_power)
    nt = -(-N // T)
    pad = np.zeros((nt * T, nt * T), dtype=bool)
    pad[:N, :N] = m
    return _csr_from_block_matrix(pad.reshape(nt, T, nt, T).any(axis=(1, 3)))


def tile_layout(N: int, B: int, W: int, S: int, T: int,
                use_power: bool = True) -> Tuple[np.ndarray, np.ndarray]:
    """The same list without the token matrix, usable at large N, for T dividing B: the window,
    power and sink terms of Algorithm 1 see only the B-token blocks that hold the two tiles, and
    its causal term (kv_idx <= q_idx) leaves tile tj <= ti non-empty and tile tj > ti empty."""
    assert B % T == 0
    r = B // T
    nt = -(-N // T)
    row_ptr = np.zeros(nt + 1, dtype=np.int32)
    cols = []
    for ti in range(nt):
        i = ti // r
        js = [tj for j in block_row(i, W, S, use_power)
              for tj in range(int(j) * r, min((int(j) + 1) * r, ti + 1))]
        cols.append(np.asarray(js, dtype=np.int32))
        row_ptr[ti + 1] = row_ptr[ti] + len(js)
    col_idx = np.concatenate(cols) if cols else np.zeros(0, dtype=np.int32)
    return row_ptr, col_idx.astype(np.int32)


def block_adjacency(n_blocks: int, W: int, S: int = 1, use_power: bool = True) -> list:
    """Out-neighbour lists of the mask seen as a DAG over blocks (Section 3.1)."""
    return [[j for j in range(i + 1) if block_predicate(i, j, W, S, use_power)]
            for i in range(n_blocks)]


def power_graph(n: int) -> list:
    """Appendix B's edge set on vertices 0..n-1: (i, j) with i - j = 2^k, k >= 0."""
    adj = []
    for i in range(n):
        out, k = [], 1
        while k <= i:
            out.append(i - k)
            k *= 2
        adj.append(out)
    return adj


def bfs_distances(adj: list, start: int) -> np.ndarray:
    """Shortest path length (number of layers) from `start` to every vertex; -1 if unreachable.
    Self-edges are ignored (a vertex is at distance 0 from itself)."""
    dist = np.full(len(adj), -1, dtype=np.int64)
    dist[start] = 0
    frontier = [start]
    while frontier:
        nxt = []
        for u in frontier:
            for v in adj[u]:
                if dist[v] < 0:
                    dist[v] = dist[u] + 1
                    nxt.append(v)
        frontier = nxt
    return dist


def reach_counts(adj: list, start: int, max_steps: int) -> list:
    """|B_k| of Appendix A for k = 1..max_steps: how many blocks `start` reaches within k
    steps (itself included, as in the appendix's worked example)."""
    dist = bfs_distances(adj, start)
    return [int(((dist >= 0) & (dist <= k)).sum()) for k in range(1, max_steps + 1)]


def contiguous_reach(adj: list, start: int, k: int) -> int:
    """Length of the unbroken run start, start-1, ... that is reachable within k steps."""
    dist = bfs_distances(adj, start)
    n = 0
    for v in range(start, -1, -1):
        if 0 <= dist[v] <= k:
            n += 1
        else:
            break
    return n


# --------------------------------------------------------------------------- attention, Eq. (1)

def prefill(Q, K, V, B: int, W: int, S: int = 1, scale: Optional[float] = None,
            rows: Optional[Sequence[int]] = None, heads: Optional[Sequence[int]] = None,
            use_power: bool = True, dense: Optional[np.ndarray] = None, threads: int = 0):
    """Eq. (1) under Algorithm 1's mask (or an explicit dense [N, N] mask).

    Q [batch, N, Hq, D], K, V [batch, N, Hkv, D] bf16.  Returns (O, LSE, n_attended):
    O [batch, n_rows, n_heads, D] fp64, LSE [batch, n_heads, n_rows] fp64, n_attended [n_rows].
    """
    lib = _load()
    q, k, v = _bf16_bits(Q), _bf16_bits(K), _bf16_bits(V)
    batch, N, Hq, D = q.shape
    Hkv = k.shape[2]
    assert k.shape == (batch, N, Hkv, D) and v.shape == k.shape and Hq % Hkv == 0
    if scale is None:
        scale = 1.0 / float(np.sqrt(D))
    rows_a = np.arange(N, dtype=np.int64) if rows is None else np.asarray(rows, dtype=np.int64)
    heads_a = np.arange(Hq, dtype=np.int64) if heads is None else np.asarray(heads, dtype=np.int64)
    dm = None
    if dense is not None:
        dm = np.ascontiguousarray(dense.astype(np.uint8))
        assert dm.shape == (N, N)
    O = np.zeros((batch, len(rows_a), len(heads_a), D), dtype=np.float64)
    LSE = np.zeros((batch, len(heads_a), len(rows_a)), dtype=np.float64)
    cnt = np.zeros(len(rows_a), dtype=np.int64)
    lib.pa_oracle_prefill(_ptr(q), _ptr(k), _ptr(v), batch, N, Hq, Hkv, D, float(scale), B, W, S,
                          int(use_power), _ptr(dm), _ptr(rows_a), len(rows_a), _ptr(heads_a),
                          len(heads_a), _ptr(O), _ptr(LSE), _ptr(cnt), int(threads))
    return O, LSE, cnt


def decode(q, Kc, Vc, lens, B: int, W: int, S: int = 1, scale: Optional[float] = None,
           use_power: bool = True, threads: int = 0):
    """One query token per sequence at position lens[b]-1 against its KV cache.

    q [batch, Hq, D], caches [batch, max_len, Hkv, D] bf16, lens [batch] (current token
    included).  Returns (O [batch, Hq, D], LSE [batch, Hq], n_attended [batch]).
    """
    lib = _load()
    qb, kb, vb = _bf16_bits(q), _bf16_bits(Kc), _bf16_bits(Vc)
    batch, Hq, D = qb.shape
    _, max_len, Hkv, _ = kb.shape
    assert kb.shape == (batch, max_len, Hkv, D) and vb.shape == kb.shape
    lens_a = np.ascontiguousarray(np.asarray(lens, dtype=np.int64))
    assert lens_a.shape == (batch,) and lens_a.min() >= 1 and lens_a.max() <= max_len
    if scale is None:
        scale = 1.0 / float(np.sqrt(D))
    O = np.zeros((batch, Hq, D), dtype=np.float64)
    LSE = np.zeros((batch, Hq), dtype=np.float64)
    cnt = np.zeros(batch, dtype=np.int64)
    lib.pa_oracle_decode(_ptr(qb), _ptr(kb), _ptr(vb), _ptr(lens_a), batch, max_len, Hq, Hkv, D,
                         float(scale), B, W, S, int(use_power), _ptr(O), _ptr(LSE), _ptr(cnt),
                         int(threads))
    return O, LSE, cnt


def backward(Q, K, V, dO, B: int, W: int, S: int = 1, scale: Optional[float] = None, use_power: bool = True,
             dense: Optional[np.ndarray] = None, threads: int = 0, key_rows: Optional[Sequence[int]] = None):
    """Gradients of Eq. (1) under Algorithm 1's mask (or an explicit dense [N, N] mask) for an
    upstream gradient dO of the output: returns (dQ [batch, N, Hq, D], dK, dV [batch, N, Hkv, D]) fp64.
    Inputs bf16 as in `prefill`.  dQ is always computed for every row; `key_rows` restricts dK and dV
    to those key positions (the other rows stay zero), which keeps long sequences affordable."""
    lib = _load()
    q, k, v, g = _bf16_bits(Q), _bf16_bits(K), _bf16_bits(V), _bf16_bits(dO)
    batch, N, Hq, D = q.shape
    Hkv = k.shape[2]
    assert k.shape == (batch, N, Hkv, D) and v.shape == k.shape and g.shape == q.shape and Hq % Hkv == 0
    if scale is None:
        scale = 1.0 / float(np.sqrt(D))
    dm = None
    if dense is not None:
        dm = np.ascontiguousarray(dense.astype(np.uint8))
        assert dm.shape == (N, N)
    dQ = np.zeros(q.shape, dtype=np.float64)
    dK = np.zeros(k.shape, dtype=np.float64)
    dV = np.zeros(k.shape, dtype=np.float64)
    kr = None if key_rows is None else np.ascontiguousarray(np.asarray(key_rows, dtype=np.int64))
    lib.pa_oracle_backward(_ptr(q), _ptr(k), _ptr(v), _ptr(g), batch, N, Hq, Hkv, D, float(scale), B, W, S,
                           int(use_power), _ptr(dm), _ptr(kr), 0 if kr is None else len(kr), _ptr(dQ), _ptr(dK),
                           _ptr(dV), int(threads))
    return dQ, dK, dV
