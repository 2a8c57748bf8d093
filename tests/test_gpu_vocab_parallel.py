"""Vocabulary-sharded verification on one GPU: the shards' records are produced one after the
other, stacked as an all-gather would deliver them, merged and verified; outputs must equal
the oracle on the unsharded logits bit for bit, whatever the number and order of shards."""
import numpy as np
import pytest
import torch

from oracle import mars_oracle as orc
from paper_2601_15498_b200 import mars, synth, vocab_parallel
from tests.test_gpu_parity import KEYS_TREE, assert_same, special_rows

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
