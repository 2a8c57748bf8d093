"""Vocabulary-parallel verification across ranks (tensor-parallel LM head).

Each rank holds a column range of every logits row.  The path has exactly one exchange step:
every rank reduces its shard to 16-byte per-row records (``mars_top2_shard``), the ranks
all-gather those records into local memory (NCCL through ``torch.distributed``; 16 B x rows
per rank), and every rank then merges and verifies locally (``mars_verify_records``).  The
merge operator is associative and commutative, so all ranks obtain outputs bit-identical to a
single-GPU ``mars_verify_tree`` on the unsharded logits.

The stochastic form (``verify_tree_stochastic_vocab_parallel``) has two exchange steps: the
records (with each shard's softmax mass) and the candidates' logits, then the drawn tokens.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_ranges(V: int, world: int) -> list[tuple[int, int]]:
    """Column range [lo, hi) of each rank: contiguous, sizes differ by at most one multiple of
    8 columns so that every shard but the last starts 16-byte aligned in bf16.

    A pure function of (V, world), so every rank reaches the same verdict: if any shard would
    hold fewer than the two columns the library needs, all ranks raise here, before any of them
    enters a collective that the others would then wait in."""
    if world < 1 or V < 2:
        raise ValueError("need world >= 1 and V >= 2")
    per = -(-V // world)
    per = -(-per // 8) * 8
    out = []
    for r in range(world):
        lo = min(V, r * per)
        out.append((lo, min(V, lo + per)))
    short = [r for r, (lo, hi) in enumerate(out) if hi - lo < 2]
    if short:
        raise ValueError(f"V = {V} over {world} ranks in multiples of 8 columns leaves rank(s) {short} with "
                         "fewer than 2 columns; use fewer ranks for this vocabulary")
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


def _all_gather(t: torch.Tensor, world: int, group) -> torch.Tensor:
    t = t.contiguous()
    flat = torch.empty((world * t.shape[0],) + tuple(t.shape[1:]), dtype=t.dtype, device=t.device)
    dist.all_gather_into_tensor(flat, t, group=group)
    return flat.view((world,) + tuple(t.shape))


def verify_tree_stochastic_vocab_parallel(logits_local: torch.Tensor, id_offset: int, tok, parent, uniform,
                                          theta: float, temperature: float, group=None, flags: int = 0,
                                          debug: bool = False, records=None, verify=None, finish=None) -> dict:
    """One vocabulary-parallel stochastic verification step on this rank: per-shard records and
    candidate logits, an all-gather of both (36 B x rows per rank), the walk and the owning
    shard's draw, an all-gather of the drawn tokens (4 B x sequences per rank), and the final
    placement.  ``records`` / ``verify`` / ``finish`` default to the CUDA library's entry points;
    they are parameters so that the collective plumbing can be exercised with CPU ranks."""
    if records is None or verify is None or finish is None:
        from . import mars
        records = records or mars.stochastic_shard_records
        verify = verify or mars.stochastic_shard_verify
        finish = finish or mars.stochastic_shard_finish
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    rec, zl = records(logits_local, tok, parent, id_offset, temperature)
    rec_all = _all_gather(rec, world, group)
    zl_all = _all_gather(zl, world, group)
    out, token_part = verify(logits_local, rec_all, zl_all, rank, id_offset, tok, parent, uniform, theta,
                             temperature, flags=flags, debug=debug)
    token_all = _all_gather(token_part, world, group)
    return finish(token_all, out)
