"""Host-side sharding of a verify-step batch over ranks (one process per GPU).

Sequences are independent in every stage of the verify step (attention, accept /
resample, controller update), so the multi-GPU form is a partition of the batch:
each rank owns a contiguous range of sequences, runs the single-GPU path on it
and never exchanges data with the others inside the step.  The only collectives
are outside the data path: the timing reduction (max over ranks), the token count
(sum over ranks) and, for a caller that wants the whole batch's results in one
place, an all-gather of the per-sequence outputs.

Everything here is plain index arithmetic plus ``torch.distributed`` calls that
work on any backend (``nccl`` on GPUs, ``gloo`` on CPU), so the logic is tested
without a GPU.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


def shard_bounds(n_seq: int, world: int) -> np.ndarray:
    """``world + 1`` boundaries of a balanced contiguous partition of ``n_seq``
    sequences: the first ``n_seq % world`` ranks get one sequence more."""
    if world < 1:
        raise ValueError("world must be >= 1")
    if n_seq < 0:
        raise ValueError("n_seq must be >= 0")
    base, extra = divmod(n_seq, world)
    sizes = np.full(world, base, dtype=np.int64)
    sizes[:extra] += 1
    out = np.zeros(world + 1, dtype=np.int64)
    np.cumsum(sizes, out=out[1:])
    return out


def balanced_bounds(cost: np.ndarray, world: int) -> np.ndarray:
    """Contiguous partition whose boundaries cut the prefix sum of a per-sequence
    cost (e.g. context length: the attention stage's bytes) as evenly as a
    contiguous split allows.  Boundary r is the first sequence whose preceding
    cost reaches r/world of the total."""
    cost = np.asarray(cost, dtype=np.float64)
    if world < 1:
        raise ValueError("world must be >= 1")
    if (cost < 0).any():
        raise ValueError("costs must be non-negative")
    n = cost.shape[0]
    cum = np.concatenate([[0.0], np.cumsum(cost)])
    total = cum[-1]
    out = np.zeros(world + 1, dtype=np.int64)
    out[-1] = n
    for r in range(1, world):
        out[r] = int(np.searchsorted(cum, total * r / world, side="left"))
    return np.maximum.accumulate(np.minimum(out, n))


@dataclass
class LocalBatch:
    """One rank's part of a batch, row offsets rebased to start at zero."""
    first: int                 # index of the rank's first sequence in the whole batch
    count: int
    seq_len: np.ndarray
    gamma: np.ndarray
    cu_q: np.ndarray           # local offsets into the rank's own query / target-logit rows
    cu_d: np.ndarray           # local offsets into the rank's own draft rows
    q_rows: slice              # rows of the whole batch's Q / O / target logits owned by this rank
    d_rows: slice              # rows of the whole batch's draft logits / tokens / uniforms


def local_batch(bounds: np.ndarray, rank: int, seq_len: np.ndarray, gamma: np.ndarray, cu_q: np.ndarray,
                cu_d: np.ndarray) -> LocalBatch:
    """Slice the per-sequence arrays of a whole batch for ``rank``.  ``cu_q`` / ``cu_d``
    are the whole batch's row offsets (packed or padded); the local ones keep the
    same spacing and start at zero, so a padded batch stays padded."""
    lo, hi = int(bounds[rank]), int(bounds[rank + 1])
    cq = np.asarray(cu_q[lo:hi + 1], dtype=np.int64)
    cd = np.asarray(cu_d[lo:hi + 1], dtype=np.int64)
    return LocalBatch(first=lo, count=hi - lo, seq_len=np.ascontiguousarray(seq_len[lo:hi]),
                      gamma=np.ascontiguousarray(gamma[lo:hi]),
                      cu_q=(cq - cq[0]).astype(np.int32), cu_d=(cd - cd[0]).astype(np.int32),
                      q_rows=slice(int(cq[0]), int(cq[-1])), d_rows=slice(int(cd[0]), int(cd[-1])))


def rank_seed(seed: int, rank: int) -> int:
    """Seed of a rank's own synthetic batch under weak scaling (every rank draws a
    full batch of its own)."""
    return int(seed) + 1000 * int(rank)


# ------------------------------------------------------------------------------ collectives
def _dist():
    import torch.distributed as dist
    return dist


def reduce_timing(ms_values, tokens: int, device="cpu", group=None):
    """Max over ranks of each time in ``ms_values`` and the sum over ranks of
    ``tokens``.  Without an initialised process group the inputs come back as they are."""
    import torch
    dist = _dist()
    ms = [float(v) for v in ms_values]
    if not (dist.is_available() and dist.is_initialized()):
        return ms, int(tokens)
    t = torch.tensor(ms, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    c = torch.tensor([int(tokens)], dtype=torch.int64, device=device)
    dist.all_reduce(c, op=dist.ReduceOp.SUM, group=group)
    return [float(v) for v in t.tolist()], int(c[0])


def gather_sequences(local, bounds: np.ndarray, group=None):
    """All-gather a per-sequence tensor (first dimension = the rank's own sequences)
    into the whole batch's order on every rank.  Shards may differ in size; they
    are padded to the largest one for the collective and trimmed afterwards."""
    import torch
    dist = _dist()
    world = len(bounds) - 1
    if not (dist.is_available() and dist.is_initialized()) or world == 1:
        return local
    sizes = np.diff(bounds)
    width = int(sizes.max())
    pad = torch.zeros((width,) + tuple(local.shape[1:]), dtype=local.dtype, device=local.device)
    pad[:local.shape[0]] = local
    parts = [torch.empty_like(pad) for _ in range(world)]
    dist.all_gather(parts, pad, group=group)
    return torch.cat([parts[r][:int(sizes[r])] for r in range(world)], dim=0)
