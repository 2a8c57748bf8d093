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
    for V, world in ((151936, 8), (32000, 3), (17, 4), (9, 2)):
        r = vocab_parallel.shard_ranges(V, world)
        assert len(r) == world and r[0][0] == 0 and r[-1][1] == V
        for (a, b), (c, d) in zip(r, r[1:]):
            assert b == c and a <= b
        assert all(lo % 8 == 0 for lo, hi in r if hi > lo)


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
