"""Vocabulary-parallel verification across ranks (tensor-parallel LM head).

Each rank holds a column range of every logits row.  The path has exactly one exchange step:
every rank reduces its shard to 16-byte per-row records (``mars_top2_shard``), the ranks
all-gather those records into local memory (NCCL through ``torch.distributed``; 16 B x rows
per rank), and every rank then merges and verifies locally (``mars_verify_records``).  The
merge operator is associative and commutative, so all ranks obtain outputs bit-identical to a
single-GPU ``mars_verify_tree`` on the unsharded logits.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_ranges(V: int, world: int) -> list[tuple[int, int]]:
    """Column range [lo, hi) of each rank: contiguous, sizes differ by at most one multiple of
    8 columns so that every shard but the last starts 16-byte aligned in bf16."""
    per = -(-V // world)
    per = -(-per // 8) * 8
    out = []
    for r in range(world):
        lo = min(V, r * per)
        out.append((lo, min(V, lo + per)))
    return out


def verify_tree_vocab_parallel(logits_local: torch.Tensor, id_offset: int, tok, parent, theta: float,
                               group=None, flags: int = 0, debug: bool = False,
                               top2=None, verify=None) -> dict:
    """One vocabulary-parallel verification step on this rank.

    ``logits_local`` is this rank's [B*N, V_local] shard whose first column has global token
    id ``id_offset``.  ``top2`` / ``verify`` default to the CUDA library's entry points; they
    are parameters so that the collective plumbing can be exercised with CPU ranks.
    """
    if top2 is None or verify is None:
        from . import mars
        top2 = top2 or mars.top2_shard
        verify = verify or mars.verify_records
    tok_t = torch.as_tensor(tok)
    B, N = tok_t.shape
    world = dist.get_world_size(group)
    rec = top2(logits_local, B, N, id_offset)
    rec = rec.contiguous()
    flat = torch.empty((world * rec.shape[0],) + tuple(rec.shape[1:]), dtype=rec.dtype, device=rec.device)
    dist.all_gather_into_tensor(flat, rec, group=group)           # rank r's records at rows [r*R, (r+1)*R)
    gathered = flat.view((world,) + tuple(rec.shape))
    return verify(gathered, tok, parent, theta, flags=flags, debug=debug)
