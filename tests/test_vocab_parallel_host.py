"""Collective plumbing of vocabulary-parallel verification with two CPU ranks (gloo): shard
ranges, the all-gather layout, and that the union of the gathered records holds each row's
global top-2."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2601_15498_b200 import vocab_parallel


def test_shard_ranges_cover_the_vocabulary():
    for V, world in ((151936, 8), (32000, 3), (18, 3), (10, 2), (64, 8), (2, 1)):
        r = vocab_parallel.shard_ranges(V, world)
        assert len(r) == world and r[0][0] == 0 and r[-1][1] == V
        for (a, b), (c, d) in zip(r, r[1:]):
            assert b == c and a <= b
        assert all(lo % 8 == 0 for lo, hi in r)
        assert all(hi - lo >= 2 for lo, hi in r)


def test_shard_ranges_refuse_shards_the_library_cannot_take():
    """A shard of fewer than two columns is rejected by the library on that rank only, which
    would leave the other ranks waiting in the all-gather.  The split is a pure function of
    (V, world), so the refusal happens on every rank, before any collective."""
    import pytest
    for V, world in ((100, 8), (17, 4), (9, 2), (1, 1), (64, 0)):
        with pytest.raises(ValueError):
            vocab_parallel.shard_ranges(V, world)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import mars_oracle as orc
    g = torch.Generator().manual_seed(5)
    B, N, V = 2, 5, 400
    logits = (torch.randn((B * N, V), generator=g) * 3).float()          # same on both ranks
    lo, hi = vocab_parallel.shard_ranges(V, world)[rank]

    def top2(local, B_, N_, off):
        val, idx = orc.top2(np.ascontiguousarray(local.numpy()))
        rec = np.empty((B_ * N_, 4), np.int32)
        rec[:, [0, 2]] = val.view(np.int32)
        rec[:, [1, 3]] = idx + off
        return torch.from_numpy(rec)

    seen = {}

    def verify(gathered, tok, parent, theta, flags=0, debug=False):
        seen["g"] = gathered.clone()
        return {"records": gathered}

    tok = np.zeros((B, N), np.int32)
    par = np.tile(np.arange(-1, N - 1, dtype=np.int32), (B, 1))
    vocab_parallel.verify_tree_vocab_parallel(logits[:, lo:hi], lo, tok, par, 0.9, top2=top2, verify=verify)
    full_val, full_idx = orc.top2(np.ascontiguousarray(logits.numpy()))
    q.put((rank, seen["g"].numpy(), full_idx))
    dist.destroy_process_group()


def test_two_rank_all_gather_layout_and_content():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = {}
    for _ in procs:
        r, g, full_idx = q.get(timeout=120)
        got[r] = (g, full_idx)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    g0, full_idx = got[0]
    g1, _ = got[1]
    assert g0.shape == (2, 10, 4) and np.array_equal(g0, g1)        # every rank holds all shards
    lo1 = vocab_parallel.shard_ranges(400, 2)[1][0]
    assert (g0[0][:, [1, 3]] < lo1).all() and (g0[1][:, [1, 3]] >= lo1).all()   # rank order, global ids
    cand = np.concatenate([g0[0][:, [1, 3]], g0[1][:, [1, 3]]], axis=1)
    for r in range(10):
        assert full_idx[r, 0] in cand[r] and full_idx[r, 1] in cand[r]


def _rank_stochastic(rank, world, port, q):
    """Stand-ins for the three library calls (no arithmetic of the method: they only tag what they
    are given), to check what the orchestration gathers and in which layout."""
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    B, N = 3, 4
    seen = {}

    def records(local, tok, parent, off, T):
        rec = torch.full((B * N, 8), rank, dtype=torch.int32)
        rec[:, 1] = off
        return rec, torch.full((B * N,), float(rank))

    def verify(local, rec_all, zl_all, my_shard, off, tok, parent, uniform, theta, T, flags=0, debug=False):
        seen["rec"], seen["zl"], seen["me"] = rec_all.clone(), zl_all.clone(), my_shard
        part = torch.full((B,), -1, dtype=torch.int32)
        part[rank::world] = 100 + rank          # this "shard" owns every world-th sequence
        return {"accept_len": torch.zeros(B, dtype=torch.int32)}, part

    def finish(token_all, out):
        out["token_all"] = token_all.clone()
        return out

    lo, hi = vocab_parallel.shard_ranges(64, world)[rank]
    out = vocab_parallel.verify_tree_stochastic_vocab_parallel(
        torch.zeros((B * N, hi - lo)), lo, np.zeros((B, N), np.int32), np.zeros((B, N), np.int32),
        np.zeros((B, N), np.float32), 0.9, 1.0, records=records, verify=verify, finish=finish)
    q.put((rank, seen["rec"].numpy(), seen["zl"].numpy(), seen["me"], out["token_all"].numpy()))
    dist.destroy_process_group()


def test_two_rank_stochastic_exchanges():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_stochastic, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = {}
    for _ in procs:
        r, rec, zl, me, tok_all = q.get(timeout=120)
        got[r] = (rec, zl, me, tok_all)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    lo1 = vocab_parallel.shard_ranges(64, 2)[1][0]
    for r in (0, 1):
        rec, zl, me, tok_all = got[r]
        assert me == r and rec.shape == (2, 12, 8) and zl.shape == (2, 12) and tok_all.shape == (2, 3)
        assert (rec[0][:, 0] == 0).all() and (rec[1][:, 0] == 1).all()          # shard g at position g
        assert (rec[0][:, 1] == 0).all() and (rec[1][:, 1] == lo1).all()
        assert (zl[0] == 0).all() and (zl[1] == 1).all()
        assert tok_all.max(axis=0).tolist() == [100, 101, 100]                  # one owner per sequence
    assert np.array_equal(got[0][3], got[1][3])
