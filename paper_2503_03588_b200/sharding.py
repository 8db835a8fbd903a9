"""KV-head sharding: the one way this operator spreads over GPUs without an exchange step.

Every (batch entry, KV head) is independent in Eq. (1): a KV head's keys and values are read only by
the query heads of its group.  A rank that holds whole KV heads and their query heads therefore runs
the ordinary single-GPU calls on head slices (strided views, no copies) and never talks to its peers;
the outputs are disjoint head slices of O and LSE.  With n_kv_heads KV heads at most n_kv_heads ranks
can take part (4 for the 28/4-head shape).  Argument marshalling only: no arithmetic of the method.
"""
from __future__ import annotations

from typing import Tuple


def kv_head_shard(n_q_heads: int, n_kv_heads: int, world: int, rank: int) -> Tuple[slice, slice]:
    """(query-head slice, KV-head slice) of `rank` among `world` ranks; KV heads are dealt in
    contiguous runs as evenly as possible, and a rank beyond the KV-head count gets empty slices."""
    if n_q_heads % n_kv_heads or world < 1 or not 0 <= rank < world:
        raise ValueError("need n_q_heads % n_kv_heads == 0 and 0 <= rank < world")
    group = n_q_heads // n_kv_heads
    base, extra = divmod(n_kv_heads, world)
    lo = rank * base + min(rank, extra)
    hi = lo + base + (1 if rank < extra else 0)
    return slice(lo * group, hi * group), slice(lo, hi)


def shard_prefill_tensors(q, k, v, world: int, rank: int):
    """Head slices (views) of q [batch, N, Hq, D] and k, v [batch, N, Hkv, D] for `rank`, or None when
    the rank has no KV head."""
    qs, ks = kv_head_shard(q.shape[2], k.shape[2], world, rank)
    if ks.start == ks.stop:
        return None
    return q[:, :, qs], k[:, :, ks], v[:, :, ks], qs
