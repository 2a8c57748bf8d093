"""The synthetic workload generators: shapes, determinism and the stated structure."""
import numpy as np
import torch

from paper_2601_15498_b200 import synth


def test_parents_are_topological_with_stated_depth_and_branching():
    par = synth.make_parents(8, 60, 6, 4, seed=3)
    assert (par[:, 0] == -1).all()
    for b in range(8):
        depth = np.zeros(60, int)
        for i in range(1, 60):
            assert 0 <= par[b, i] < i
            depth[i] = depth[par[b, i]] + 1
        assert depth.max() == 6
        assert np.bincount(par[b, 1:], minlength=60).max() <= 4
    assert (synth.make_parents(8, 60, 6, 4, seed=3) == par).all()
    assert (synth.make_parents(8, 60, 6, 4, seed=4) != par).any()


def test_cfg0_recipe():
    w = synth.cfg0("cpu", seed=0, B=300)
    assert w.logits.shape == (1800, 32000) and w.logits.dtype == torch.float32
    top = torch.topk(w.logits, 2, dim=1)
    assert (top.values[:, 0] == 20.0).all()                     # planted argmax at +20
    ratio = (top.values[:, 1] / top.values[:, 0]).numpy()
    low = ratio >= 0.85
    assert 0.33 < low.mean() < 0.47                             # 40 % planted runner-ups
    assert ratio[~low].max() < 0.6                              # otherwise only N(0, 2^2) noise
    lead = top.indices.numpy().reshape(300, 6, 2)
    hit1 = (w.draft == lead[:, :5, 0]).mean()
    hit2 = (w.draft == lead[:, :5, 1]).mean()
    assert abs(hit1 - 0.6) < 0.05 and abs(hit2 - 0.25) < 0.05   # draft mix
    w2 = synth.cfg0("cpu", seed=0, B=300)
    assert torch.equal(w.logits, w2.logits) and (w.tok == w2.tok).all()


def test_tree_workload_small_vocab_structure():
    w = synth.tree_workload("t", 4, 60, 6, 4, 5000, torch.bfloat16, "cpu", 1, 0.9, 3.0, 15.0, 30.0, 0.3)
    assert w.logits.dtype == torch.bfloat16 and w.logits.shape == (240, 5000)
    assert (w.tok[:, 0] == -1).all() and (w.tok[:, 1:] >= 0).all() and (w.tok < 5000).all()
    for b in range(4):                                          # siblings carry distinct tokens
        for p in range(60):
            kids = w.tok[b, w.parent[b] == p]
            assert len(set(kids.tolist())) == len(kids)
    top = torch.topk(w.logits.float(), 1, dim=1).values
    assert (top >= 14.9).all() and (top <= 30.1).all()
    bits = synth.to_numpy_bits(w.logits)
    assert bits.dtype == np.uint16 and bits.shape == (240, 5000)
