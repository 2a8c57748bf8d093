"""Vocabulary-sharded verification on one GPU: the shards' records are produced one after the
other, stacked as an all-gather would deliver them, merged and verified; outputs must equal
the oracle on the unsharded logits bit for bit, whatever the number and order of shards."""
import numpy as np
import pytest
import torch

from oracle import mars_oracle as orc
from paper_2601_15498_b200 import mars, synth, vocab_parallel

import hookctl as hooks
from tests.test_gpu_parity import KEYS_TREE, assert_same, special_rows

from stochastic_checks import sharded_stochastic

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def sharded(logits, tok, parent, theta, ranges, flags=0, order=None):
    B, N = tok.shape
    recs = []
    for lo, hi in ranges:
        recs.append(mars.top2_shard(logits[:, lo:hi], B, N, lo, V_local=hi - lo))
    if order is not None:
        recs = [recs[i] for i in order]
    return mars.to_host(mars.verify_records(torch.stack(recs), tok, parent, theta, flags, debug=True))


@pytest.mark.parametrize("world", [1, 2, 3, 8])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_sharded_equals_unsharded(world, dtype):
    w = synth.tree_workload("vp", 6, 60, 6, 4, 151936, dtype, DEV, 90 + world, 0.9, 3.0, 15.0, 30.0, 0.3)
    ref = orc.verify_tree(synth.to_numpy_bits(w.logits), w.tok, w.parent, w.theta)
    ranges = vocab_parallel.shard_ranges(w.V, world)
    assert ranges[0][0] == 0 and ranges[-1][1] == w.V
    out = sharded(w.logits, w.tok, w.parent, w.theta, ranges)
    assert_same(out, ref, KEYS_TREE, f"world={world}")
    if world > 1:   # any shard order gives the same bits
        out = sharded(w.logits, w.tok, w.parent, w.theta, ranges, order=list(range(world))[::-1])
        assert_same(out, ref, KEYS_TREE, f"world={world} reversed")


def test_shard_records_against_oracle_top2():
    w = synth.tree_workload("vp", 2, 9, 3, 3, 40000, torch.bfloat16, DEV, 7, 0.9, 3.0, 15.0, 30.0, 0.3)
    lo, hi = 13336, 26672
    rec = mars.top2_shard(w.logits[:, lo:hi], w.B, w.N, lo, V_local=hi - lo).cpu().numpy()
    val, idx = orc.top2(synth.to_numpy_bits(w.logits[:, lo:hi].contiguous()))
    assert np.array_equal(rec[:, [1, 3]], idx + lo)
    assert np.array_equal(rec[:, [0, 2]].view(np.float32), val)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_degenerate_rows_sharded(dtype):
    V = 2048 * 3 + 5
    z = special_rows(V, dtype)
    N = z.shape[0]
    parent = np.arange(-1, N - 1, dtype=np.int32)[None, :]
    ids = orc.top2(synth.to_numpy_bits(z))[1]
    # uneven shards, one of them only two columns wide
    ranges = [(0, 2), (2, 1000), (1000, 1003), (1003, 4100), (4100, V)]
    for which in (0, 1):
        tok = np.full((1, N), -1, np.int32)
        tok[0, 1:] = ids[:-1, which]
        for flags in (0, mars.SIGN_LITERAL):
            out = sharded(z, tok, parent, 0.9, ranges, flags)
            ref = orc.verify_tree(synth.to_numpy_bits(z), tok, parent, 0.9, flags)
            assert_same(out, ref, KEYS_TREE, f"which={which} flags={flags}")


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_lm_head_equals_unsharded_bit_for_bit(world):
    """Each logit is the same fp32 accumulation whichever shard computes it, so the sharded
    output projection followed by the record merge must reproduce mars_lmhead_verify exactly."""
    w = synth.cfg4_operands(DEV, seed=50 + world, B=4, N=30, V=20000 + 8 * world, d=512, depth=4)
    g = torch.Generator(device="cpu"); g.manual_seed(world)
    bias = (torch.randn(w.V, generator=g) * 0.5).to(DEV)
    zz = w.hidden.float() @ w.w_vocab.float().T + bias
    lead = torch.topk(zz, 2, dim=1).indices.cpu().numpy()
    tok = synth.make_tokens(w.parent, lead, w.V, 9)
    ref = mars.to_host(mars.lmhead_verify(w.hidden, w.w_vocab, bias, tok, w.parent, 0.9, debug=True))
    recs = []
    for lo, hi in vocab_parallel.shard_ranges(w.V, world):
        recs.append(mars.lmhead_top2_shard(w.hidden, w.w_vocab[lo:hi].contiguous(), bias[lo:hi].contiguous(),
                                           w.B, w.N, lo))
    out = mars.to_host(mars.verify_records(torch.stack(recs), tok, w.parent, 0.9, debug=True))
    assert_same(out, ref, KEYS_TREE, f"lm head world={world}")
    assert (out["seq_status"] == 0).all() and out["accept_len"].max() >= 1


# ---------------------------------------------------------------- stochastic form (T > 0)

@pytest.mark.parametrize("world", [1, 2, 3, 8])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_stochastic_sharded_against_the_oracle(world, dtype):
    import stochastic_checks as sc
    w = synth.tree_workload("vps", 12, 20, 4, 3, 40009, dtype, DEV, 120 + world, 0.9, 1.0, 9.0, 16.0, 0.4)
    u = synth.make_uniforms(w.B, w.N, 120 + world)
    u[::3, 1:] = np.float32(0.99999)            # a third of the sequences draw at the root
    ref = orc.verify_tree_stochastic(synth.to_numpy_bits(w.logits), w.tok, w.parent, u, w.theta, 1.0)
    ranges = vocab_parallel.shard_ranges(w.V, world)
    for flags in (0, mars.STOCH_PLAIN):
        ref = orc.verify_tree_stochastic(synth.to_numpy_bits(w.logits), w.tok, w.parent, u, w.theta, 1.0, flags)
        outs, token_all = sharded_stochastic(w.logits, w.tok, w.parent, u, w.theta, 1.0, ranges, flags)
        for g, o in enumerate(outs):
            sc.compare(o, ref, w.tok, w.parent, sc.host_f64(w.logits), u, 1.0, f"world={world} rank={g}",
                       max_close_frac=0.1)
        for k in ("accept_len", "out_tokens", "path_nodes", "out_len", "seq_status", "node_how"):
            for o in outs[1:]:
                assert np.array_equal(o[k], outs[0][k]), k      # every rank ends with the same result
        owners = (token_all >= 0).sum(axis=0)
        ok = outs[0]["seq_status"] == 0
        assert (owners[ok] == 1).all()                           # exactly one shard drew each token


def test_stochastic_sharded_degenerate_rows_and_tiny_shards():
    import stochastic_checks as sc
    V = 3000
    w = synth.tree_workload("vps", 8, 10, 3, 3, V, torch.float32, DEV, 131, 0.9, 1.0, 5.0, 8.0, 0.4)
    lg = w.logits.clone()
    lg[0 * 10 + 0, :] = float("-inf")
    lg[1 * 10 + 0, 17] = float("inf")
    lg[2 * 10 + 0, 100:1200] = float("nan")
    lg[3 * 10 + 0, 0:2000] = float("-inf")       # whole shards without mass
    u = synth.make_uniforms(w.B, w.N, 131)
    ranges = [(0, 2), (2, 1000), (1000, 1003), (1003, 2000), (2000, V)]
    ref = orc.verify_tree_stochastic(synth.to_numpy_bits(lg), w.tok, w.parent, u, 0.9, 1.0)
    outs, _ = sharded_stochastic(lg, w.tok, w.parent, u, 0.9, 1.0, ranges)
    assert ref["seq_status"].tolist()[:2] == [4, 4]
    for o in outs:
        sc.compare(o, ref, w.tok, w.parent, sc.host_f64(lg), u, 1.0, "degenerate sharded", max_close_frac=0.3)


@pytest.mark.parametrize("cluster", [1, 4, 8])
def test_stochastic_sharded_cluster_shapes(cluster, monkeypatch):
    import stochastic_checks as sc
    hooks.set("HOOK_STOCH_TAIL_CLUSTER", cluster)
    w = synth.tree_workload("vps", 30, 6, 2, 2, 90011, torch.bfloat16, DEV, 140, 0.9, 1.0, 3.0, 6.0, 0.4)
    u = synth.make_uniforms(w.B, w.N, 140)
    u[::2, 1:] = np.float32(0.99999)
    ref = orc.verify_tree_stochastic(synth.to_numpy_bits(w.logits), w.tok, w.parent, u, 0.9, 1.0, mars.STOCH_PLAIN)
    outs, _ = sharded_stochastic(w.logits, w.tok, w.parent, u, 0.9, 1.0, vocab_parallel.shard_ranges(w.V, 4),
                                 mars.STOCH_PLAIN)
    for g, o in enumerate(outs):
        sc.compare(o, ref, w.tok, w.parent, sc.host_f64(w.logits), u, 1.0, f"cluster {cluster} rank {g}",
                   max_close_frac=0.1)
    drawn = outs[0]["out_tokens"][np.arange(w.B), outs[0]["accept_len"]]
    assert drawn.min() < w.V // 4 and drawn.max() > 3 * w.V // 4       # tokens from the first and the last shard
