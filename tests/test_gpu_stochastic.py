"""Parity of stochastic (T > 0) verification with the CPU oracle, through the C ABI.  The
comparison policy and its tolerances are in stochastic_checks.py."""
import numpy as np
import pytest
import torch

from oracle import mars_oracle as orc
from paper_2601_15498_b200 import mars, synth

import hookctl as hooks

from stochastic_checks import (DEV, STATS, check_walk_is_valid, compare, compare_sampled, host_f64,
                               sampled_case)

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _no_hooks(monkeypatch):
    hooks.clear("HOOK_FORCE_SPLIT")
    hooks.clear("HOOK_STOCH_TAIL_CLUSTER")


def run_and_compare(logits, tok, parent, u, theta, T, flags=0, Dcap=None, what="", **kw):
    got = mars.to_host(mars.verify_tree_stochastic(logits, tok, parent, u, theta, T, flags, Dcap, debug=True))
    ref = orc.verify_tree_stochastic(synth.to_numpy_bits(logits), tok, parent, u, theta, T, flags, Dcap)
    compare(got, ref, tok, parent, host_f64(logits), u, T, what, **kw)
    return got, ref


def third_candidates(w, seed, delta=1.5, frac=0.3):
    """Input construction for these tests: plants a third logit at z1 - delta in every row and
    aims a fraction of the draft tokens at it, so that candidates which are neither the top-1 nor
    the runner-up carry a visible probability and the Eq. 1 test decides both ways."""
    rng = np.random.default_rng(seed)
    top = torch.topk(w.logits[:, :w.V].float(), 2, dim=1)
    ids3 = torch.as_tensor(rng.integers(0, w.V, w.R), device=w.logits.device)
    clash = (ids3 == top.indices[:, 0]) | (ids3 == top.indices[:, 1])
    ids3 = torch.where(clash, (top.indices.max(dim=1).values + 1) % w.V, ids3)
    clash = (ids3 == top.indices[:, 0]) | (ids3 == top.indices[:, 1])
    ids3 = torch.where(clash, (ids3 + 1) % w.V, ids3)
    rows = torch.arange(w.R, device=w.logits.device)
    w.logits[rows, ids3] = (top.values[:, 0] - delta).to(w.logits.dtype)
    ids3 = ids3.cpu().numpy().reshape(w.B, w.N)
    par = w.parent if w.parent.ndim == 2 else np.tile(w.parent, (w.B, 1))
    for b in range(w.B):
        for i in range(1, w.N):
            if par[b, i] >= 0 and rng.random() < frac:
                w.tok[b, i] = ids3[b, par[b, i]]
    return w


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("flags", [0, mars.STOCH_PLAIN, mars.STOCH_RELAX_ONLY])
@pytest.mark.parametrize("T", [0.7, 1.0, 2.0])
def test_small_trees(dtype, flags, T):
    """Rows of several tiles with a ragged tail; candidates of every kind."""
    w = third_candidates(synth.tree_workload("t", 48, 20, 4, 3, 33333, dtype, DEV, 21, 0.9, 1.0, 9.0, 16.0, 0.4), 21)
    u = synth.make_uniforms(w.B, w.N, 21)
    got, ref = run_and_compare(w.logits, w.tok, w.parent, u, w.theta, T, flags, what=f"{dtype} flags={flags} T={T}")
    how = ref["node_how"]
    assert (how == 4).any()
    if T <= 1.0:
        assert (how == 3).any() and ref["accept_len"].max() >= 1
    if flags == mars.STOCH_PLAIN:
        assert not ((how == 1) | (how == 2)).any()


def test_cfg1_one_tree_rows_split_over_blocks():
    w = synth.cfg1(DEV)
    for seed in range(4):
        u = synth.make_uniforms(w.B, w.N, 100 + seed)
        run_and_compare(w.logits, w.tok, w.parent, u, w.theta, 1.0, what=f"cfg1 seed {seed}")


def test_cfg3_slice_of_the_serving_batch():
    w = synth.cfg3(DEV, B=12)
    u = synth.make_uniforms(w.B, w.N, 3)
    for flags in (0, mars.STOCH_PLAIN):
        run_and_compare(w.logits, w.tok, w.parent, u, w.theta, 1.0, flags, what=f"cfg3 B=12 flags={flags}")


def test_chain_form_equals_the_tree_oracle_on_linear_parents():
    w = synth.cfg2(DEV, B=16)
    u = synth.make_uniforms(w.B, w.N, 2)
    got = mars.to_host(mars.verify_chain_stochastic(w.logits, w.draft, u, w.theta, 1.0, debug=True))
    ref = orc.verify_tree_stochastic(synth.to_numpy_bits(w.logits), w.tok, w.parent, u, w.theta, 1.0)
    got["path_nodes"] = ref["path_nodes"]       # the chain call has no path output
    compare(got, ref, w.tok, w.parent, host_f64(w.logits), u, 1.0, "chain")
    assert (got["out_len"] == got["accept_len"] + 1).all()


def test_cfg0_chain_fp32():
    w = synth.cfg0(DEV, B=64, seed=9)
    u = synth.make_uniforms(w.B, w.N, 9)
    got = mars.to_host(mars.verify_chain_stochastic(w.logits, w.draft, u, w.theta, 1.0, debug=True))
    ref = orc.verify_tree_stochastic(synth.to_numpy_bits(w.logits), w.tok, w.parent, u, w.theta, 1.0)
    got["path_nodes"] = ref["path_nodes"]
    compare(got, ref, w.tok, w.parent, host_f64(w.logits), u, 1.0, "cfg0")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_unaligned_rows_and_odd_sizes(dtype):
    """Row stride and vocabulary that keep no row 16-byte aligned: scalar head / tail in the
    streaming pass, element-wise tiles in the draw."""
    V, ld = 4099, 4103
    w = synth.tree_workload("t", 24, 9, 3, 3, V, dtype, DEV, 33, 0.9, 1.0, 5.0, 8.0, 0.4, ld=ld, pad_value=50.0)
    u = synth.make_uniforms(w.B, w.N, 33)
    base = w.logits.reshape(-1)[1:1 + (w.R - 1) * ld + V]     # shift by one element
    shifted = torch.as_strided(base, (w.R, V), (ld, 1))
    src = w.logits[:, :V].clone()
    shifted.copy_(src)
    got = mars.to_host(mars.verify_tree_stochastic(shifted, w.tok, w.parent, u, 0.9, 1.0, V=V, debug=True))
    ref = orc.verify_tree_stochastic(synth.to_numpy_bits(src), w.tok, w.parent, u, 0.9, 1.0)
    compare(got, ref, w.tok, w.parent, host_f64(src), u, 1.0, "unaligned")


@pytest.mark.parametrize("split", [2, 3, 7])
def test_forced_row_splits(split, monkeypatch):
    hooks.set("HOOK_FORCE_SPLIT", split)
    w = synth.tree_workload("t", 10, 12, 3, 3, 20011, torch.bfloat16, DEV, 44, 0.9, 1.0, 6.0, 9.0, 0.4)
    u = synth.make_uniforms(w.B, w.N, 44)
    run_and_compare(w.logits, w.tok, w.parent, u, 0.9, 1.3, what=f"split {split}")


@pytest.mark.parametrize("cluster", [1, 2, 4, 8])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_draw_with_one_block_and_with_clusters(cluster, dtype, monkeypatch):
    """The draw's pass over the row runs in one block or is shared by a cluster of 2, 4 or 8 blocks
    (distributed shared memory); every shape must resolve the same element.  Many sequences stop at the
    root (uniforms next to one), so every part of the row gets drawn from."""
    hooks.set("HOOK_STOCH_TAIL_CLUSTER", cluster)
    w = synth.tree_workload("t", 96, 6, 2, 2, 70001, dtype, DEV, 66, 0.9, 1.0, 3.0, 6.0, 0.4)
    u = synth.make_uniforms(w.B, w.N, 66)
    u[::2, 1:] = np.float32(0.99999)
    got, ref = run_and_compare(w.logits, w.tok, w.parent, u, 0.9, 1.0, mars.STOCH_PLAIN, what=f"cluster {cluster}")
    drawn = got["out_tokens"][np.arange(w.B), got["accept_len"]]
    assert drawn.min() < w.V // 8 and drawn.max() > 7 * w.V // 8


@pytest.mark.parametrize("dtype,V", [(torch.bfloat16, 270001), (torch.float32, 140003)])
def test_rows_longer_than_the_tile_table(dtype, V):
    """More 32-lane tiles than a block's table of tile sums holds: the table-free search."""
    w = synth.tree_workload("t", 6, 4, 2, 2, V, dtype, DEV, 67, 0.9, 1.0, 3.0, 6.0, 0.4)
    u = synth.make_uniforms(w.B, w.N, 67)
    u[::2, 1:] = np.float32(0.99999)
    run_and_compare(w.logits, w.tok, w.parent, u, 0.9, 1.0, mars.STOCH_PLAIN, what=f"long rows {dtype}",
                    max_close_frac=0.4)


def test_largest_supported_tree():
    """N = 1024 nodes per sequence (the cap): shared-memory footprint of the tail at its maximum,
    children spread over many 32-node ballot rounds."""
    w = third_candidates(synth.tree_workload("t", 3, mars.MAX_NODES, 40, 6, 777, torch.float32, DEV, 71, 0.9, 1.0,
                                             5.0, 8.0, 0.4), 71)
    u = synth.make_uniforms(w.B, w.N, 71)
    for flags in (0, mars.STOCH_PLAIN):
        got, ref = run_and_compare(w.logits, w.tok, w.parent, u, 0.9, 1.0, flags, what="N=1024")
    assert ref["accept_len"].max() >= 1


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_rising_rows_at_low_temperature(dtype):
    """Rows sorted in ascending order at T = 0.05: every thread meets ever larger logits, far beyond
    the slack of its softmax reference (which must then move), and the weights span hundreds of
    binary orders of magnitude."""
    w = third_candidates(synth.tree_workload("t", 8, 6, 2, 2, 60000, dtype, DEV, 91, 0.9, 2.0, 9.0, 12.0, 0.4), 91,
                         delta=0.02)
    srt, order = torch.sort(w.logits.float(), dim=1)
    w.logits.copy_(srt.to(dtype))
    inv = torch.argsort(order, dim=1).cpu().numpy()          # old id -> new id, per row
    par = w.parent
    for b in range(w.B):
        for i in range(1, w.N):
            if par[b, i] >= 0 and w.tok[b, i] >= 0:
                w.tok[b, i] = inv[b * w.N + par[b, i], w.tok[b, i]]
    u = synth.make_uniforms(w.B, w.N, 91)
    for T in (0.05, 1.0):
        run_and_compare(w.logits, w.tok, w.parent, u, 0.9, T, mars.STOCH_PLAIN, what=f"rising rows T={T}",
                        max_close_frac=0.3)


def test_tiny_vocabularies_one_tile():
    for V in (2, 3, 9, 200, 257):
        w = synth.tree_workload("t", 40, 6, 2, 3, V, torch.float32, DEV, 60 + V, 0.9, 1.0, 2.0, 3.0, 0.4)
        u = synth.make_uniforms(w.B, w.N, V)
        run_and_compare(w.logits, w.tok, w.parent, u, 0.9, 1.0, mars.STOCH_PLAIN, what=f"V={V}", max_close_frac=0.05)


def test_special_nodes_duplicates_padding_and_out_of_range_ids():
    w = synth.tree_workload("t", 64, 16, 4, 4, 3000, torch.float32, DEV, 70, 0.9, 1.0, 4.0, 6.0, 0.4)
    tok = w.tok.copy()
    tok[:, 5] = tok[:, 4]            # a repeated token (siblings in many of the trees)
    tok[:, 7] = -1                   # padding node
    tok[:, 9] = w.V + 5              # id outside the vocabulary
    parent = w.parent.copy()
    parent[:, 11] = -1               # absent node
    u = synth.make_uniforms(w.B, w.N, 70)
    for flags in (0, mars.STOCH_PLAIN):
        got, ref = run_and_compare(w.logits, tok, parent, u, 0.9, 1.0, flags, what="special nodes")
        assert (got["node_how"][:, 7] == 0).all() and (got["node_prob"][:, 9] == 0).all()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_degenerate_rows_bad_trees_and_depth_cap(dtype):
    V = 50000
    w = synth.tree_workload("t", 6, 8, 3, 2, V, dtype, DEV, 80, 0.9, 1.0, 5.0, 8.0, 0.4)
    lg = w.logits.clone()
    lg[0 * 8 + 0, :] = float("-inf")                 # sequence 0: root row without a distribution
    lg[1 * 8 + 0, 17] = float("inf")                 # sequence 1: +inf logit
    lg[2 * 8 + 0, 100:200] = float("nan")            # sequence 2: NaNs count as -inf, still fine
    lg[2 * 8 + 0, 30000::997] = float("nan")
    lg[4 * 8 + 1, 7::3] = float("-inf")              # sequence 4: a third of a row at -inf
    parent = w.parent.copy()
    parent[3, 4] = 6                                 # sequence 3: malformed tree
    u = synth.make_uniforms(w.B, w.N, 80)
    got, ref = run_and_compare(lg, w.tok, parent, u, 0.9, 1.0, what="degenerate")
    assert ref["seq_status"].tolist()[:4] == [4, 4, 0, 1]
    assert got["out_tokens"][1, 0] == 17 and got["out_tokens"][0, 0] == 0
    # depth cap: uniforms of zero accept every first child; outputs hold one level only
    u0 = np.zeros_like(u)
    got, ref = run_and_compare(w.logits, w.tok, w.parent, u0, 0.9, 1.0, Dcap=1, what="Dcap")
    assert (ref["seq_status"] == 2).any()


def test_rule_variants_and_sign_flag_pass_through():
    w = synth.tree_workload("t", 32, 12, 3, 3, 9000, torch.bfloat16, DEV, 90, 0.9, 1.0, 6.0, 9.0, 0.5)
    u = synth.make_uniforms(w.B, w.N, 90)
    for flags, theta in ((mars.RULE_MARGIN, 0.75), (mars.RULE_PROB_RATIO, 0.4), (mars.SIGN_LITERAL, 0.9)):
        run_and_compare(w.logits, w.tok, w.parent, u, theta, 1.0, flags, what=f"flags {flags}")


def test_repeated_calls_on_one_workspace():
    """The workspace needs no initialisation and may be reused by later calls."""
    w = synth.cfg3(DEV, B=6)
    u = synth.make_uniforms(w.B, w.N, 8)
    ws = torch.full((int(mars.lib().mars_stochastic_workspace_bytes(w.B, w.N, w.V, mars.BF16)),), 0xAB,
                    dtype=torch.uint8, device=DEV)
    first = mars.to_host(mars.verify_tree_stochastic(w.logits, w.tok, w.parent, u, 0.9, 1.0, debug=True))
    for _ in range(3):
        again = mars.to_host(mars.verify_tree_stochastic(w.logits, w.tok, w.parent, u, 0.9, 1.0, debug=True,
                                                         workspace=ws))
        for k in first:
            assert np.array_equal(first[k], again[k]), k


def test_back_to_back_calls_overlap_without_mixing_their_data():
    """A call's streaming kernel may start while the previous call's tail kernel still reads the
    shared workspace; it must not write its records before that kernel is done.  Two different
    batches alternate through one workspace, twenty calls with nothing in between; every call must
    reproduce what the same batch gives when it runs alone."""
    ws_ = [synth.tree_workload("sb0", 24, 20, 4, 3, 60000, torch.bfloat16, DEV, 911, 0.9, 3.0, 15.0, 30.0, 0.3),
           synth.tree_workload("sb1", 24, 20, 4, 3, 60000, torch.bfloat16, DEV, 912, 0.9, 3.0, 15.0, 30.0, 0.3)]
    us = [synth.make_uniforms(24, 20, 911), synth.make_uniforms(24, 20, 912)]
    alone = [mars.to_host(mars.verify_tree_stochastic(w.logits, w.tok, w.parent, u, 0.9, 1.0, debug=True))
             for w, u in zip(ws_, us)]
    for j in (0, 1):        # and what runs alone agrees with the oracle
        ref = orc.verify_tree_stochastic(synth.to_numpy_bits(ws_[j].logits), ws_[j].tok, ws_[j].parent, us[j], 0.9, 1.0)
        compare(alone[j], ref, ws_[j].tok, ws_[j].parent, host_f64(ws_[j].logits), us[j], 1.0, f"alone {j}")
    work = torch.empty(int(mars.lib().mars_stochastic_workspace_bytes(24, 20, 60000, mars.BF16)), dtype=torch.uint8,
                       device=DEV)
    toks = [torch.as_tensor(w.tok, device=DEV) for w in ws_]
    pars = [torch.as_tensor(w.parent, device=DEV) for w in ws_]
    ud = [torch.as_tensor(u, device=DEV) for u in us]
    outs = [mars.alloc_stochastic_outputs(24, 20, 19, DEV, debug=True) for _ in range(20)]
    for i in range(20):
        j = i & 1
        mars.verify_tree_stochastic(ws_[j].logits, toks[j], pars[j], ud[j], 0.9, 1.0,
                                    flags=(mars.LOGITS_READY if i % 4 < 2 else 0), workspace=work, out=outs[i])
    torch.cuda.synchronize()
    for i in range(20):
        got = mars.to_host(outs[i])
        for k in ("accept_len", "out_tokens", "path_nodes", "out_len", "seq_status", "node_how"):
            assert np.array_equal(got[k], alone[i & 1][k]), (i, k)
        assert np.array_equal(got["node_prob"].view(np.uint32), alone[i & 1]["node_prob"].view(np.uint32)), i


def test_plain_mode_preserves_the_target_distribution_on_the_gpu():
    """A property that needs no oracle: with Eq. 1 alone the first emitted token follows the
    root row's softmax, whatever the candidates are (20 000 sequences over one fixed tree)."""
    rng = np.random.default_rng(5)
    V, N, B, T = 48, 5, 20000, 0.9
    rows = torch.tensor((rng.normal(size=(N, V)) * 1.2).astype(np.float32))
    logits = rows.repeat(B, 1).to(DEV)
    parent = np.array([-1, 0, 0, 0, 1], np.int32)
    lead = torch.topk(rows[0], 3).indices.numpy()
    tok = np.tile(np.array([-1, lead[1], lead[0], lead[2], 7], np.int32), (B, 1))
    u = synth.make_uniforms(B, N, 5)
    got = mars.to_host(mars.verify_tree_stochastic(logits, tok, parent, u, 0.9, T, mars.STOCH_PLAIN))
    P = torch.softmax(rows[0].double() / T, 0).numpy()
    f = np.bincount(got["out_tokens"][:, 0], minlength=V) / B
    sd = np.sqrt(P * (1 - P) / B)
    assert np.all(np.abs(f - P) <= 4.5 * sd + 1e-9)


def test_host_errors():
    w = synth.tree_workload("t", 2, 4, 2, 2, 100, torch.float32, DEV, 1, 0.9, 1.0, 5.0, 6.0, 0.3)
    u = synth.make_uniforms(w.B, w.N, 1)
    for T in (0.0, -1.0, float("nan"), float("inf")):
        with pytest.raises(mars.MarsError, match="invalid argument"):
            mars.verify_tree_stochastic(w.logits, w.tok, w.parent, u, 0.9, T)
    with pytest.raises(mars.MarsError, match="invalid argument"):
        mars.verify_tree_stochastic(w.logits, w.tok, w.parent, u, 0.9, 1.0, mars.STOCH_PLAIN | mars.STOCH_RELAX_ONLY)
    with pytest.raises(mars.MarsError, match="unsupported"):
        mars.verify_tree_stochastic(w.logits, w.tok, w.parent, u, 0.9, 1.0, mars.COUNTERS_ZERO)
    small = torch.empty(256, dtype=torch.uint8, device=DEV)
    with pytest.raises(mars.MarsError, match="workspace"):
        mars.verify_tree_stochastic(w.logits, w.tok, w.parent, u, 0.9, 1.0, workspace=small[:16])


def test_full_size_batch_every_sequence():
    """The serving-scale batch in the launch configuration the benchmark times (256 x 60 rows of
    151 936 bf16 logits): every sequence against the oracle under the tolerance policy, in
    host-memory-sized chunks."""
    w = synth.cfg3(DEV)
    u = synth.make_uniforms(w.B, w.N, 3)
    got = mars.to_host(mars.verify_tree_stochastic(w.logits, w.tok, w.parent, u, w.theta, 1.0, debug=True))
    assert (got["seq_status"] == 0).all()
    step, close, neigh = 16, 0, 0
    for b0 in range(0, w.B, step):
        b1 = b0 + step
        rows = w.logits[b0 * w.N:b1 * w.N]
        ref = orc.verify_tree_stochastic(synth.to_numpy_bits(rows), w.tok[b0:b1], w.parent[b0:b1], u[b0:b1], w.theta, 1.0)
        part = {k: got[k][b0:b1] for k in got}
        c, n = compare(part, ref, w.tok[b0:b1], w.parent[b0:b1], host_f64(rows), u[b0:b1], 1.0,
                       f"sequences {b0}..{b1}", max_close_frac=1.0)
        close += c
        neigh += n
    assert close <= 3 and neigh <= 3, (close, neigh)      # 2e-5 / 1e-5 windows over 256 walks and draws
    for b in range(w.B):
        check_walk_is_valid(got, w.tok, w.parent, b)


# ---------------------------------------------------------------- sampled drafts (general Eq. 1)

@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("flags", [0, mars.STOCH_PLAIN, mars.STOCH_RELAX_ONLY])
def test_sampled_chains(dtype, flags):
    w, qdev, zq, draft, qx, u = sampled_case(31, 64, 6, 30011, dtype, 1.0, 0.9, 1.1, ld_pad=5)
    got = mars.to_host(mars.verify_chain_sampled(w.logits, qdev, draft, qx, u, 0.9, 0.9, 1.1, flags, V=w.V, debug=True))
    ref = orc.verify_chain_sampled(synth.to_numpy_bits(w.logits), synth.to_numpy_bits(zq), draft, qx, u, 0.9, 0.9, 1.1,
                                   flags)
    compare_sampled(got, ref, f"sampled {dtype} {flags}")
    how = ref["node_how"]
    assert (how == 3).any() and (how == 4).any() and ref["accept_len"].max() >= 2


@pytest.mark.parametrize("cluster", [1, 2, 4, 8])
def test_sampled_chains_cluster_shapes(cluster, monkeypatch):
    hooks.set("HOOK_STOCH_TAIL_CLUSTER", cluster)
    w, qdev, zq, draft, qx, u = sampled_case(32, 40, 4, 70001, torch.bfloat16, 1.5)
    u[:, 1] = np.float32(0.99999)          # most sequences reject their first draft: residual draws
    got = mars.to_host(mars.verify_chain_sampled(w.logits, qdev, draft, qx, u, 0.9, 1.0, 1.0, mars.STOCH_PLAIN,
                                                 debug=True))
    ref = orc.verify_chain_sampled(synth.to_numpy_bits(w.logits), synth.to_numpy_bits(zq), draft, qx, u, 0.9, 1.0,
                                   1.0, orc.STOCH_PLAIN)
    compare_sampled(got, ref, f"sampled cluster {cluster}")
    assert (ref["accept_len"] == 0).mean() > 0.5


def test_sampled_chains_special_cases():
    w, qdev, zq, draft, qx, u = sampled_case(33, 12, 5, 5003, torch.float32, 1.0)
    draft[0, 1] = -1                         # the chain of sequence 0 ends after one draft
    qdev[1 * 4 + 0, :] = float("-inf")       # drafter row without a softmax
    zq[1 * 4 + 0, :] = float("-inf")
    u[1, 1] = np.float32(0.999999)           # make sure sequence 1 rejects its first draft
    qdev[2 * 4 + 0, 100:200] = float("nan")
    zq[2 * 4 + 0, 100:200] = float("nan")
    lg = w.logits.clone()
    lg[3 * 5 + 1, :] = float("-inf")         # target row without a softmax on the way
    got = mars.to_host(mars.verify_chain_sampled(lg, qdev, draft, qx, u, 0.9, 1.0, 1.0, debug=True))
    ref = orc.verify_chain_sampled(synth.to_numpy_bits(lg), synth.to_numpy_bits(zq), draft, qx, u, 0.9, 1.0, 1.0)
    compare_sampled(got, ref, "sampled special")
    assert ref["seq_status"][1] == 4 or ref["accept_len"][1] > 0


def test_sampled_plain_mode_preserves_the_target_distribution_on_the_gpu():
    """Speculative sampling on the GPU with drafts really drawn from the drafter: the first emitted
    token follows the target's first row."""
    rng = np.random.default_rng(7)
    V, K, B, T, Tq = 40, 3, 30000, 0.9, 1.3
    rows = torch.tensor((rng.normal(size=(K, V)) * 1.0).astype(np.float32))
    rows_q = rows[:K - 1] + torch.tensor((rng.normal(size=(K - 1, V)) * 0.8).astype(np.float32))
    Q = torch.softmax(rows_q.double() / Tq, dim=1)
    g = torch.Generator().manual_seed(7)
    draft = torch.stack([torch.multinomial(Q[i], B, replacement=True, generator=g) for i in range(K - 1)], dim=1)
    qx = torch.stack([Q[i][draft[:, i]] for i in range(K - 1)], dim=1).float()
    u = synth.make_uniforms(B, K, 7)
    got = mars.to_host(mars.verify_chain_sampled(rows.repeat(B, 1).to(DEV), rows_q.repeat(B, 1).to(DEV),
                                                 draft.int().numpy(), qx.numpy(), u, 0.9, T, Tq, mars.STOCH_PLAIN))
    P = torch.softmax(rows[0].double() / T, 0).numpy()
    f = np.bincount(got["out_tokens"][:, 0], minlength=V) / B
    assert np.all(np.abs(f - P) <= 4.5 * np.sqrt(P * (1 - P) / B) + 1e-9)


def test_sampled_chain_without_drafts_and_many_short_sequences():
    # K = 1: nothing to judge, the token is a draw from the only row
    w = synth.chain_workload("t", 50, 1, 3001, torch.float32, DEV, 35, 0.9, 1.0, 4.0, 6.0, 0.3)
    u = synth.make_uniforms(w.B, 1, 35)
    draft = np.zeros((w.B, 0), np.int32)
    qx = np.zeros((w.B, 0), np.float32)
    got = mars.to_host(mars.verify_chain_sampled(w.logits, None, draft, qx, u, 0.9, 1.0, 1.0, debug=True))
    ref = orc.verify_tree_stochastic(synth.to_numpy_bits(w.logits), w.tok, w.parent, u, 0.9, 1.0)
    assert (got["accept_len"] == 0).all() and np.array_equal(got["out_tokens"], ref["out_tokens"])
    # 3000 sequences of two rows: one block per sequence, many more blocks than the GPU holds at once
    w, qdev, zq, draft, qx, u = sampled_case(36, 3000, 2, 517, torch.bfloat16, 1.0)
    got = mars.to_host(mars.verify_chain_sampled(w.logits, qdev, draft, qx, u, 0.9, 1.0, 1.0, debug=True))
    ref = orc.verify_chain_sampled(synth.to_numpy_bits(w.logits), synth.to_numpy_bits(zq), draft, qx, u, 0.9, 1.0, 1.0)
    compare_sampled(got, ref, "many short sequences")


def test_sampled_host_errors():
    w, qdev, zq, draft, qx, u = sampled_case(34, 2, 3, 200, torch.float32)
    with pytest.raises(mars.MarsError, match="invalid argument"):
        mars.verify_chain_sampled(w.logits, qdev, draft, qx, u, 0.9, 1.0, 0.0)
    with pytest.raises(mars.MarsError, match="dtype"):
        mars.verify_chain_sampled(w.logits, qdev.to(torch.bfloat16), draft, qx, u, 0.9, 1.0, 1.0)


def test_zz_report_tolerated_cases():
    """Not a check of the library: prints how many decisions of this module fell inside the
    tolerances (run with -s to see it) and keeps the share small."""
    print("stochastic parity:", STATS)
    if STATS["sequences"]:
        assert STATS["close"] <= 0.01 * STATS["sequences"] + 2
