"""Multi-GPU host logic.

Rows of a batch are independent, so the default split is by rows: every rank holds the whole
vocabulary, its own grammar tables and its own mask cache, and decodes its slice of the batch;
no collective sits on the data path.  The only exchanges are the ones a benchmark or an engine
needs around it: the slowest rank's time, and the chosen tokens if somebody wants them in one
place.

The second split is by vocabulary, for engines whose LM head is tensor-parallel: every rank
holds all rows but only logits[:, v_begin:v_end).  Then the path has one real exchange step:
the per-row (best logit, token id) pairs, packed into one int64 each by
``wg_decode_step_shard``, are MAX-reduced over the ranks (``reduce_best_keys``) before
``wg_advance_keys`` advances the states on every rank.
"""
from __future__ import annotations

from typing import List, Tuple


def shard_rows(n_rows: int, world: int, rank: int) -> Tuple[int, int]:
    """[begin, end) of the rows rank ``rank`` owns: contiguous, sizes differ by at most one."""
    if world < 1 or not 0 <= rank < world or n_rows < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(n_rows, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def max_over_ranks(value: float, device=None) -> float:
    """The largest ``value`` any rank holds (the job is as slow as its slowest rank)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def gather_tokens(tokens, n_rows: int) -> List[int]:
    """All ranks' chosen tokens in row order (``tokens``: this rank's 1-D int tensor)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [int(x) for x in tokens.tolist()]
    world = dist.get_world_size()
    sizes = [shard_rows(n_rows, world, r) for r in range(world)]
    width = max(e - b for b, e in sizes)
    padded = torch.full((width,), -1, dtype=tokens.dtype, device=tokens.device)
    padded[:tokens.numel()] = tokens
    parts = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(parts, padded)
    out: List[int] = []
    for (b, e), part in zip(sizes, parts):
        out.extend(int(x) for x in part[:e - b].tolist())
    return out


def vocab_slices(V: int, world: int, align: int = 8192) -> List[Tuple[int, int]]:
    """[begin, end) of every rank's vocabulary slice: contiguous, every boundary but the last a
    multiple of ``align`` (what ``wg_decode_step_shard`` asks for), sizes as equal as that
    allows.  A rank whose slice would be empty (more ranks than aligned pieces) gets (V, V)."""
    if world < 1 or V < 1 or align < 1:
        raise ValueError("bad slice request")
    pieces = (V + align - 1) // align
    out = []
    for r in range(world):
        b, e = shard_rows(pieces, world, r)
        out.append((min(b * align, V), min(e * align, V)))
    return out


def reduce_best_keys(keys) -> None:
    """In place: the per-row maximum of the packed (value, token) keys over all ranks.  One
    8-byte element per row; NCCL runs it over NVLink / NVSwitch, gloo on CPU."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(keys, op=dist.ReduceOp.MAX)
