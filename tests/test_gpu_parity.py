"""Parity of the CUDA library with the CPU oracle, element by element, through the C ABI.

Bar: bit-exact for token ids, lengths, paths, flags and statuses; the fp32 top-2 values are
compared as bit patterns too (both sides take every decision in fp32).
"""
import os

import numpy as np
import pytest
import torch

from oracle import mars_oracle as orc
from paper_2601_15498_b200 import mars, synth

import hookctl as hooks

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
KEYS_TREE = ("accept_len", "out_tokens", "path_nodes", "out_len", "seq_status", "top2_id",
             "node_flags")


def assert_same(got: dict, want: dict, keys, what=""):
    for k in keys:
        g, w = got[k], want[k]
        assert g.shape == w.shape, (what, k, g.shape, w.shape)
        if not np.array_equal(g, w):
            bad = np.argwhere(g != w)[:5]
            raise AssertionError(f"{what}: {k} differs at {bad.tolist()}: got {g[tuple(bad[0])]}, "
                                 f"want {w[tuple(bad[0])]}")
    g, w = got["top2_val"], want["top2_val"]
    assert np.array_equal(g.view(np.uint32), w.view(np.uint32)), (what, "top2_val")


def run_tree(logits, tok, parent, theta, flags=0, Dcap=None, V=None):
    out = mars.to_host(mars.verify_tree(logits, tok, parent, theta, flags, Dcap, V, debug=True))
    ref = orc.verify_tree(synth.to_numpy_bits(logits), tok, parent, theta, flags, Dcap, V)
    return out, ref


def run_chain(logits, draft, theta, flags=0, V=None):
    out = mars.to_host(mars.verify_chain(logits, draft, theta, flags, V, debug=True))
    ref = orc.verify_chain(synth.to_numpy_bits(logits), draft, theta, flags, V)
    return out, ref


@pytest.fixture(autouse=True)
def _no_forced_split(monkeypatch):
    hooks.clear("HOOK_FORCE_SPLIT")


# ------------------------------------------------------------------ the named workloads

def test_cfg0_chain_b1_fp32():
    w = synth.cfg0(DEV)
    out, ref = run_chain(w.logits, w.draft, w.theta)
    assert_same(out, ref, ("accept_len", "out_tokens", "out_len", "top2_id"), w.name)
    assert (out["seq_status"] == 0).all()


def test_cfg0_many_seeds_statistics():
    """Same recipe, 512 sequences: parity, and the mean accepted length near its closed form."""
    w = synth.cfg0(DEV, seed=100, B=512)
    out, ref = run_chain(w.logits, w.draft, w.theta)
    assert_same(out, ref, ("accept_len", "out_tokens", "out_len", "top2_id"), w.name)
    p = 0.6 + 0.25 * 0.4 * (0.1 / 0.15)
    mean = sum(p ** k for k in range(1, 6))
    assert abs(out["accept_len"].mean() - mean) < 0.25


def test_cfg1_tree_b1_bf16():
    w = synth.cfg1(DEV)
    out, ref = run_tree(w.logits, w.tok, w.parent, w.theta)
    assert_same(out, ref, KEYS_TREE, w.name)


@pytest.mark.parametrize("theta", [0.8, 0.9, 0.95, 1.5])
def test_cfg2_batched_chain_theta_sweep(theta):
    w = synth.cfg2(DEV, theta=theta)
    out, ref = run_chain(w.logits, w.draft, theta)
    assert_same(out, ref, ("accept_len", "out_tokens", "out_len", "top2_id"), f"{w.name} theta={theta}")
    if theta > 1:   # strict greedy: accepted drafts equal the argmax of their rows
        top1 = ref["top2_id"][:, 0].reshape(w.B, w.N)
        for b in range(w.B):
            a = out["accept_len"][b]
            assert (w.draft[b, :a] == top1[b, :a]).all()
            assert a == w.N - 1 or w.draft[b, a] != top1[b, a]


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_cfg3_reduced_batch_full_parity(dtype):
    w = synth.cfg3(DEV, B=24, dtype=dtype)      # 1440 rows: whole rows per block (no split)
    out, ref = run_tree(w.logits, w.tok, w.parent, w.theta)
    assert_same(out, ref, KEYS_TREE, w.name)
    assert out["accept_len"].max() >= 3


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_cfg3_full_size_every_sequence(dtype):
    """The serving-scale workload in the launch configuration the benchmark times: all 256
    sequences (15 360 rows) bit for bit against the oracle, in host-memory-sized chunks."""
    w = synth.cfg3(DEV, dtype=dtype)
    assert w.R == 15360
    # as the benchmark launches it: workspace zeroed once, counters left to the kernel's own reset
    work = torch.zeros(mars.workspace_bytes(w.B, w.N, w.V, mars.BF16 if dtype == torch.bfloat16 else mars.FP32),
                       dtype=torch.uint8, device=DEV)
    mars.verify_tree(w.logits, w.tok, w.parent, w.theta, flags=mars.COUNTERS_ZERO, workspace=work)
    out = mars.to_host(mars.verify_tree(w.logits, w.tok, w.parent, w.theta, flags=mars.COUNTERS_ZERO,
                                        debug=True, workspace=work))
    step = 64
    for b0 in range(0, w.B, step):
        b1 = min(w.B, b0 + step)
        ref = orc.verify_tree(synth.to_numpy_bits(w.logits[b0 * w.N:b1 * w.N]), w.tok[b0:b1], w.parent[b0:b1], w.theta)
        got = {k: (v[b0 * w.N:b1 * w.N] if k in ("top2_val", "top2_id") else v[b0:b1]) for k, v in out.items()}
        assert_same(got, ref, KEYS_TREE, f"{w.name} sequences {b0}..{b1}")
        assert np.array_equal(got["top2_val"].view(np.uint32), ref["top2_val"].view(np.uint32))
    # properties that hold for every sequence
    assert (out["seq_status"] == 0).all()
    assert ((out["accept_len"] >= 0) & (out["accept_len"] <= w.max_depth)).all()
    assert (out["out_len"] == out["accept_len"] + 1).all()
    ids = out["top2_id"].reshape(w.B, w.N, 2)
    for b in range(w.B):
        a = out["accept_len"][b]
        path = out["path_nodes"][b, :a + 1]
        assert path[0] == 0
        for k in range(1, a + 1):
            n, p = path[k], path[k - 1]
            assert w.parent[b, n] == p and w.tok[b, n] in ids[b, p]
            assert out["out_tokens"][b, k - 1] == w.tok[b, n]
        assert out["out_tokens"][b, a] == ids[b, path[a], 0]
    # top-2 values of every row against torch's own top-k on the device (values only)
    for r0 in range(0, w.R, 1024):
        tv = torch.topk(w.logits[r0:r0 + 1024].float(), 2, dim=1).values.cpu().numpy()
        assert np.array_equal(tv, out["top2_val"][r0:r0 + 1024])


# ------------------------------------------------------------------ shapes and layouts

@pytest.mark.parametrize("V", [2, 3, 7, 8, 9, 257, 4099, 32000, 151936])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_odd_vocab_sizes(V, dtype):
    w = synth.tree_workload("odd", 3, 9, 3, 3, V, dtype, DEV, 40 + V % 13, 0.9, 3.0, 15.0, 30.0, 0.5)
    out, ref = run_tree(w.logits, w.tok, w.parent, 0.9)
    assert_same(out, ref, KEYS_TREE, f"V={V} {dtype}")


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("ld_extra,offset", [(1, 0), (3, 1), (5, 3), (8, 0), (13, 7)])
def test_unaligned_rows_with_canaries(dtype, ld_extra, offset):
    """Rows that start off a 16-byte boundary, ld > V, and a huge value in every element the
    library must not read: padding columns and guard rows before and after."""
    B, N, V = 4, 7, 5003
    ld = V + ld_extra
    w = synth.tree_workload("canary", B, N, 3, 3, V, dtype, DEV, 77, 0.9, 3.0, 15.0, 30.0, 0.5)
    big = torch.full((B * N + 2, ld + offset), 3.0e38, dtype=dtype, device=DEV)
    view = big[1:-1, offset:offset + ld]
    view[:, :V] = w.logits
    assert view.stride(0) == ld + offset
    out = mars.to_host(mars.verify_tree(view, w.tok, w.parent, 0.9, V=V, debug=True))
    ref = orc.verify_tree(synth.to_numpy_bits(w.logits), w.tok, w.parent, 0.9)
    assert_same(out, ref, KEYS_TREE, f"ld+{ld_extra} off {offset}")


@pytest.mark.parametrize("S", [1, 2, 3, 7, 16, 61])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_forced_row_split(monkeypatch, S, dtype):
    """The merge is associative and commutative: any number of slices gives the same bits."""
    hooks.set("HOOK_FORCE_SPLIT", S)
    w = synth.tree_workload("split", 5, 12, 4, 3, 40000 + 7, dtype, DEV, 5, 0.9, 3.0, 15.0, 30.0, 0.5)
    out, ref = run_tree(w.logits, w.tok, w.parent, 0.9)
    assert_same(out, ref, KEYS_TREE, f"S={S}")


def test_large_tree_more_than_64_nodes():
    for N, depth in ((65, 10), (200, 12), (1024, 40)):
        w = synth.tree_workload("big", 3, N, depth, 4, 3000, torch.bfloat16, DEV, N, 0.9, 3.0, 15.0,
                                30.0, 0.5)
        # aim most tokens at the leading ids so that deep paths are accepted
        out, ref = run_tree(w.logits, w.tok, w.parent, 0.85)
        assert_same(out, ref, KEYS_TREE, f"N={N}")
    # a long chain through the tree path (N > 64) and through the chain entry point
    w = synth.chain_workload("long", 2, 100, 2000, torch.float32, DEV, 3, 0.9, 2.0, 20.0, 20.0, 0.4)
    lead = torch.topk(w.logits, 2, dim=1).indices.cpu().numpy().reshape(2, 100, 2)
    draft = lead[:, :-1, 0].astype(np.int32).copy()
    draft[1, 70] = 5                                # sequence 1 stops at depth 70
    out, ref = run_chain(w.logits, draft, 0.9)
    assert_same(out, ref, ("accept_len", "out_tokens", "out_len", "top2_id"), "long chain")
    assert out["accept_len"].tolist() == [99, 70]


# ------------------------------------------------------------------ degenerate rows

def special_rows(V, dtype):
    z = torch.randn((12, V), dtype=torch.float32) * 3
    z[0] = 1.5                                   # constant row
    z[1] = torch.round(z[1])                     # heavy ties
    z[2] = float("-inf")                         # all -inf
    z[3] = float("nan")                          # all NaN
    z[4] = float("-inf"); z[4, V - 1] = 0.5      # one finite entry, last position
    z[5] = float("-inf"); z[5, 0] = -2.0
    z[6, 5] = float("inf"); z[6, V // 2] = float("inf")
    z[7] = -torch.abs(z[7]) - 1                  # all negative: z1 < 0
    z[8] = 0.0; z[8, 3] = -0.0                   # zeros of both signs
    z[9, 1::2] = float("nan")
    z[10, :] = -5.0; z[10, V - 2] = 4.0; z[10, V - 1] = 4.0    # tie at the very end
    z[11, :] = 7.0; z[11, 0] = float("nan")
    return z.to(dtype).to(DEV)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("V", [9, 2048, 2048 * 9 + 5])
@pytest.mark.parametrize("flags", [0, mars.SIGN_LITERAL])
def test_degenerate_rows(dtype, V, flags):
    z = special_rows(V, dtype)
    N = z.shape[0]
    parent = np.arange(-1, N - 1, dtype=np.int32)[None, :]
    ids = orc.top2(synth.to_numpy_bits(z))[1]
    for which in (0, 1):                          # drafts = top-1 of every row, then top-2
        tok = np.full((1, N), -1, np.int32)
        tok[0, 1:] = ids[:-1, which]
        for theta in (0.9, 0.0, -1.0):
            out, ref = run_tree(z, tok, parent, theta, flags)
            assert_same(out, ref, KEYS_TREE, f"V={V} which={which} theta={theta} flags={flags}")


def test_one_ulp_around_theta_on_device():
    th = np.float32(0.9)
    rows = []
    for k in (-3, 0, 4):
        z1 = np.float32(2.0 ** k)
        on = np.float32(th * z1)
        for z2 in (np.nextafter(on, np.float32(np.inf), dtype=np.float32), on,
                   np.nextafter(on, np.float32(-np.inf), dtype=np.float32)):
            r = np.full(64, -1.0, np.float32)
            r[10], r[20] = z1, z2
            rows.append(r)
            rows.append(r)                       # second row of the 2-row chain (bonus)
    z = torch.from_numpy(np.stack(rows)).to(DEV)
    draft = np.full((len(rows) // 2, 1), 20, np.int32)
    out, ref = run_chain(z, draft, float(th))
    assert_same(out, ref, ("accept_len", "out_tokens", "out_len", "top2_id"), "ulp")
    assert out["accept_len"].tolist() == [1, 0, 0] * 3


# ------------------------------------------------------------------ trees: flags and statuses

def test_shared_parent_padding_malformed_and_depth_cap():
    w = synth.tree_workload("t", 6, 20, 5, 3, 1000, torch.bfloat16, DEV, 9, 0.9, 3.0, 15.0, 30.0, 0.5)
    par = w.parent.copy()
    tok = w.tok.copy()
    par[1, 7] = -1                     # absent node
    tok[2, 3] = -4                     # padding token
    par[3, 0] = 0                      # malformed: root has a parent
    par[4, 5] = 5                      # malformed: parent[i] >= i
    par[5, 9] = -2                     # malformed: below -1
    tok[0, 4] = 5000                   # id beyond the vocabulary
    out, ref = run_tree(w.logits, tok, par, 0.9)
    assert_same(out, ref, KEYS_TREE, "statuses")
    assert out["seq_status"].tolist() == [0, 0, 0, 1, 1, 1]
    out, ref = run_tree(w.logits, tok, par, 0.9, Dcap=1)
    assert_same(out, ref, KEYS_TREE, "depth cap")
    assert 2 in out["seq_status"]
    # one parent array shared by all sequences
    out, ref = run_tree(w.logits, w.tok, w.parent[0], 0.9)
    assert_same(out, ref, KEYS_TREE, "shared parent")


def test_host_errors_launch_nothing():
    w = synth.tree_workload("t", 2, 5, 3, 3, 100, torch.float32, DEV, 1, 0.9, 3.0, 15.0, 30.0, 0.5)
    out = mars.alloc_outputs(2, 5, 4, DEV)
    with pytest.raises(mars.MarsError, match="invalid argument"):
        mars.verify_tree(w.logits, w.tok, w.parent, float("nan"), out=out)
    with pytest.raises(mars.MarsError, match="unsupported sizes"):      # V < 2: no workspace size
        mars.verify_tree(w.logits, w.tok, w.parent, 0.9, V=1, out=out)
    with pytest.raises(mars.MarsError, match="workspace"):
        mars.verify_tree(w.logits, w.tok, w.parent, 0.9, out=out,
                         workspace=torch.empty(256, dtype=torch.uint8, device=DEV))
    with pytest.raises(mars.MarsError, match="unsupported"):
        mars.verify_tree(w.logits, w.tok, w.parent, 0.9, flags=64, out=out)
    torch.cuda.synchronize()
    assert (out["accept_len"].cpu().numpy() == -777).all()      # nothing was written


def test_workspace_reuse_and_non_default_stream():
    """Back-to-back calls on one workspace (stale contents) and on a side stream."""
    w = synth.cfg2(DEV, seed=12, B=8)
    need = mars.workspace_bytes(w.B, w.N, w.V, mars.BF16)
    ws = torch.randint(0, 255, (need,), dtype=torch.uint8, device=DEV)      # garbage
    ref = orc.verify_chain(synth.to_numpy_bits(w.logits), w.draft, 0.9)
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(st):
        outs = [mars.verify_chain(w.logits, w.draft, 0.9, debug=True, workspace=ws) for _ in range(3)]
    st.synchronize()
    for o in outs:
        assert_same(mars.to_host(o), ref, ("accept_len", "out_tokens", "out_len", "top2_id"), "reuse")


def test_counters_zero_flag_skips_the_memset_safely():
    """With MARS_COUNTERS_ZERO the library does not clear the arrival counters itself; they
    are zero after a memset of the workspace and after every completed call."""
    big = synth.cfg2(DEV, seed=31, B=12)
    small = synth.tree_workload("z", 5, 9, 3, 3, 40000, torch.float32, DEV, 32, 0.9, 3.0, 15.0, 30.0, 0.5)
    need = max(mars.workspace_bytes(big.B, big.N, big.V, mars.BF16),
               mars.workspace_bytes(small.B, small.N, small.V, mars.FP32))
    ws = torch.zeros(need, dtype=torch.uint8, device=DEV)
    ref_big = orc.verify_chain(synth.to_numpy_bits(big.logits), big.draft, 0.9)
    ref_small = orc.verify_tree(synth.to_numpy_bits(small.logits), small.tok, small.parent, 0.9)
    for _ in range(3):      # alternate shapes (split and unsplit rows) on the same workspace
        out = mars.to_host(mars.verify_chain(big.logits, big.draft, 0.9, flags=mars.COUNTERS_ZERO,
                                             debug=True, workspace=ws))
        assert_same(out, ref_big, ("accept_len", "out_tokens", "out_len", "top2_id"), "flag chain")
        out = mars.to_host(mars.verify_tree(small.logits, small.tok, small.parent, 0.9,
                                            flags=mars.COUNTERS_ZERO, debug=True, workspace=ws))
        assert_same(out, ref_small, KEYS_TREE, "flag tree")
    assert int(ws[:256].to(torch.int32).sum()) == 0              # counters are back at zero


def test_minimal_shapes_and_extreme_thetas():
    """K = 1 chains (no drafts: only the bonus token), single-node trees, Dcap = 0, many short
    sequences, and thresholds at the ends of the float range."""
    g = torch.Generator(device="cpu"); g.manual_seed(3)
    z = (torch.randn((40, 300), generator=g) * 3 + 5).to(DEV)
    out, ref = run_chain(z, np.empty((40, 0), np.int32), 0.9)                 # K = 1
    assert_same(out, ref, ("accept_len", "out_tokens", "out_len", "top2_id"), "K=1")
    assert (out["accept_len"] == 0).all() and (out["out_len"] == 1).all()
    tok = np.full((40, 1), -1, np.int32)
    par = np.full((40, 1), -1, np.int32)
    out, ref = run_tree(z, tok, par, 0.9)                                     # N = 1
    assert_same(out, ref, KEYS_TREE, "N=1")
    w = synth.tree_workload("m", 2000, 4, 2, 2, 64, torch.bfloat16, DEV, 8, 0.9, 3.0, 15.0, 30.0, 0.5)
    for theta in (0.9, float("inf"), float("-inf"), 3.0e38, -3.0e38, 0.0):
        out, ref = run_tree(w.logits, w.tok, w.parent, theta)
        assert_same(out, ref, KEYS_TREE, f"B=2000 theta={theta}")
    out, ref = run_tree(w.logits, w.tok, w.parent, 0.5, Dcap=0)               # every accept overflows
    assert_same(out, ref, KEYS_TREE, "Dcap=0")
    assert set(out["seq_status"].tolist()) <= {0, 2} and 2 in out["seq_status"]


def test_cuda_graph_replay_with_changing_inputs():
    """The calls only enqueue work (one optional memset, one kernel) and allocate nothing, so a
    captured step can be replayed on new data written into the same buffers."""
    ws_list = [synth.tree_workload("g", 4, 30, 5, 3, 50000, torch.bfloat16, DEV, 60 + i, 0.9, 3.0, 15.0,
                                   30.0, 0.4) for i in range(3)]
    w0 = ws_list[0]
    logits = torch.empty_like(w0.logits)
    tok = torch.zeros((w0.B, w0.N), dtype=torch.int32, device=DEV)
    parent = torch.zeros((w0.B, w0.N), dtype=torch.int32, device=DEV)
    work = torch.zeros(mars.workspace_bytes(w0.B, w0.N, w0.V, mars.BF16), dtype=torch.uint8, device=DEV)
    out = mars.alloc_outputs(w0.B, w0.N, w0.N - 1, DEV, debug=True)
    logits.copy_(w0.logits); tok.copy_(torch.as_tensor(w0.tok)); parent.copy_(torch.as_tensor(w0.parent))
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        mars.verify_tree(logits, tok, parent, 0.9, workspace=work, out=out)     # warm-up outside capture
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        mars.verify_tree(logits, tok, parent, 0.9, workspace=work, out=out)
    for w in ws_list[::-1]:
        logits.copy_(w.logits); tok.copy_(torch.as_tensor(w.tok)); parent.copy_(torch.as_tensor(w.parent))
        graph.replay()
        got = mars.to_host(out)
        ref = orc.verify_tree(synth.to_numpy_bits(w.logits), w.tok, w.parent, 0.9)
        assert_same(got, ref, KEYS_TREE, "graph replay")


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_rule_variants_margin_and_probability_ratio(dtype):
    w = synth.tree_workload("rv", 12, 40, 5, 3, 30000, dtype, DEV, 70, 0.9, 3.0, 15.0, 30.0, 0.5)
    bits = synth.to_numpy_bits(w.logits)
    seen = set()
    for flags, thetas in ((mars.RULE_MARGIN, (0.0, 0.5, 1.0, 2.5, 100.0)),
                          (mars.RULE_PROB_RATIO, (-1.0, 0.0, 0.05, 0.3, 0.6, 1.0))):
        for theta in thetas:
            out = mars.to_host(mars.verify_tree(w.logits, w.tok, w.parent, theta, flags, debug=True))
            ref = orc.verify_tree(bits, w.tok, w.parent, theta, flags)
            assert_same(out, ref, KEYS_TREE, f"flags={flags} theta={theta}")
            seen.add(tuple(out["accept_len"].tolist()))
    assert len(seen) >= 3                       # the thresholds really change decisions
    with pytest.raises(mars.MarsError, match="invalid argument"):
        mars.verify_tree(w.logits, w.tok, w.parent, 0.5, mars.RULE_MARGIN | mars.RULE_PROB_RATIO)
    # chain entry point and the records path take the same flags
    c = synth.cfg2(DEV, seed=71, B=6)
    out = mars.to_host(mars.verify_chain(c.logits, c.draft, 1.0, mars.RULE_MARGIN, debug=True))
    ref = orc.verify_chain(synth.to_numpy_bits(c.logits), c.draft, 1.0, orc.RULE_MARGIN)
    assert_same(out, ref, ("accept_len", "out_tokens", "out_len", "top2_id"), "chain margin")
    rec = mars.top2_shard(w.logits, w.B, w.N, 0)
    out = mars.to_host(mars.verify_records(rec[None].contiguous(), w.tok, w.parent, 0.3,
                                           mars.RULE_PROB_RATIO, debug=True))
    ref = orc.verify_tree(bits, w.tok, w.parent, 0.3, orc.RULE_PROB_RATIO)
    assert_same(out, ref, KEYS_TREE, "records prob ratio")


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_sorted_rows_worst_case_for_the_filter(dtype):
    """Ascending rows make every batch beat the running bound (the exact path runs all the
    time); descending rows decide everything in the first batch.  Both must stay exact,
    including the many ties that bf16 rounding creates in a ramp."""
    V = 151936
    ramp = torch.linspace(-20.0, 20.0, V)
    rows = torch.stack([ramp, ramp.flip(0), ramp * 0.5 + 3, (ramp * 0.25).flip(0), ramp.abs(), -ramp.abs()])
    z = rows.repeat(4, 1).to(dtype).to(DEV)                     # 24 rows -> rows are split
    N = 6
    parent = np.tile(np.arange(-1, N - 1, dtype=np.int32), (4, 1))
    ids = orc.top2(synth.to_numpy_bits(z))[1].reshape(4, N, 2)
    tok = np.full((4, N), -1, np.int32)
    tok[:, 1:] = ids[:, :-1, 1]                                 # always draft the runner-up
    for theta in (0.9, 0.9999):
        out, ref = run_tree(z, tok, parent, theta)
        assert_same(out, ref, KEYS_TREE, f"sorted rows theta={theta}")
    big = rows[:2].repeat(1300, 1).to(dtype).to(DEV)            # 2600 rows: one block per row
    val, idx = orc.top2(synth.to_numpy_bits(big[:2]))
    out = mars.to_host(mars.verify_chain(big, np.zeros((1300, 1), np.int32), 0.9, debug=True))
    assert np.array_equal(out["top2_id"][:2], idx) and np.array_equal(out["top2_id"][-2:], idx)
    assert np.array_equal(out["top2_val"][:2].view(np.uint32), val.view(np.uint32))


def test_device_matches_what_the_launch_shapes_are_tuned_for():
    """Grid sizes assume 148 SMs; the check reports the device's count so that a part with
    fewer enabled SMs is noticed (results stay correct, waves fill unevenly)."""
    info = mars.device_check()
    assert info["sm_tuned"] == 148
    assert info["sm_count"] == torch.cuda.get_device_properties(0).multi_processor_count
    assert (info["status"] == 0) == (info["sm_count"] == 148)


@pytest.mark.parametrize("early", [False, True])
@pytest.mark.parametrize("use_graph", [False, True])
def test_back_to_back_calls_overlap_without_mixing_their_data(use_graph, early):
    """With MARS_LOGITS_READY consecutive calls on one stream overlap on the GPU (the later one
    streams its logits while the earlier one drains), without it only their launches do; they
    share one workspace here.  Two different batches alternate,
    forty calls in a row with nothing in between, directly and from a CUDA graph; every call's
    outputs must be the oracle's for its own batch."""
    ws = [synth.tree_workload("bb0", 48, 12, 4, 3, 50000, torch.bfloat16, DEV, 901, 0.9, 3.0, 15.0, 30.0, 0.3),
          synth.tree_workload("bb1", 48, 12, 4, 3, 50000, torch.bfloat16, DEV, 902, 0.9, 3.0, 15.0, 30.0, 0.3)]
    refs = [orc.verify_tree(synth.to_numpy_bits(w.logits), w.tok, w.parent, w.theta) for w in ws]
    toks = [torch.as_tensor(w.tok, device=DEV) for w in ws]
    pars = [torch.as_tensor(w.parent, device=DEV) for w in ws]
    n_calls = 40
    outs = [mars.alloc_outputs(48, 12, 11, DEV, debug=True) for _ in range(n_calls)]
    work = torch.zeros(mars.workspace_bytes(48, 12, 50000, mars.BF16), dtype=torch.uint8, device=DEV)

    def run_all():
        for i in range(n_calls):
            j = i & 1
            mars.verify_tree(ws[j].logits, toks[j], pars[j], 0.9,
                             flags=mars.COUNTERS_ZERO | (mars.LOGITS_READY if early else 0), workspace=work, out=outs[i])

    mars.verify_tree(ws[0].logits, toks[0], pars[0], 0.9, workspace=work)      # counters start at zero
    torch.cuda.synchronize()
    if use_graph:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            run_all()
        g.replay()
        g.replay()
    else:
        run_all()
    torch.cuda.synchronize()
    for i in range(n_calls):
        got = mars.to_host(outs[i])
        assert_same(got, refs[i & 1], KEYS_TREE, f"call {i}")
        assert np.array_equal(got["top2_val"].view(np.uint32), refs[i & 1]["top2_val"].view(np.uint32))


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_host_buffer_entry_point(dtype):
    """mars_verify_tree_host: inputs and outputs in (pinned) host memory, one call does the copies
    in, the verification and the copies out; results are the oracle's, twice in a row on one
    staging buffer, with and without the optional outputs, and for a padded row stride."""
    w = synth.tree_workload("hb", 9, 21, 4, 3, 30011, dtype, "cpu", 931, 0.9, 3.0, 15.0, 30.0, 0.3, ld=30016)
    ref = orc.verify_tree(synth.to_numpy_bits(w.logits), w.tok, w.parent, w.theta, V=w.V)
    lg = w.logits.pin_memory()
    tok, par = torch.as_tensor(w.tok).pin_memory(), torch.as_tensor(w.parent).pin_memory()
    code = mars.BF16 if dtype == torch.bfloat16 else mars.FP32
    need = int(mars.lib().mars_verify_tree_host_staging_bytes(w.B, w.N, w.V, code, 30016, w.N - 1))
    assert need > w.logits.numel() * w.logits.element_size()
    staging = torch.full((need,), 0xCD, dtype=torch.uint8, device=DEV)
    for rep in range(2):
        out = mars.alloc_host_outputs(w.B, w.N - 1)
        if rep == 1:
            del out["path_nodes"], out["seq_status"]
        mars.verify_tree_host(lg, tok, par, w.theta, staging, out, V=w.V)
        torch.cuda.synchronize()
        for k, v in out.items():
            assert np.array_equal(v.numpy(), ref[k]), (rep, k)
    small = torch.empty(need - 256, dtype=torch.uint8, device=DEV)
    with pytest.raises(mars.MarsError, match="workspace"):
        mars.verify_tree_host(lg, tok, par, w.theta, small, mars.alloc_host_outputs(w.B, w.N - 1), V=w.V)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_very_long_rows(dtype):
    """Rows of two million logits (fourteen times the largest vocabulary of the paper's models):
    many batches per block when rows are whole, and every slice far beyond one batch when the few
    rows are split; the winners sit in the last elements of the row, and ids need 21 bits."""
    V = (1 << 21) + 37
    g = torch.Generator(device=DEV); g.manual_seed(21)
    z = (torch.randn((5, V), generator=g, device=DEV) * 3).to(dtype)
    z[0, V - 1] = 40.0
    z[0, V - 2] = 39.0
    z[1, V - 3] = 25.0
    z[2, 0] = 33.0
    z[2, V - 1] = 33.0                                  # a tie across the whole row: the lower id leads
    tok = np.array([[-1, V - 1, V - 3, 0, V - 1]], np.int32)
    parent = np.array([[-1, 0, 1, 2, 2]], np.int32)
    ref = orc.verify_tree(synth.to_numpy_bits(z), tok, parent, 0.9)
    got = mars.to_host(mars.verify_tree(z, tok, parent, 0.9, debug=True))
    assert_same(got, ref, KEYS_TREE, "long rows")
    assert np.array_equal(got["top2_val"].view(np.uint32), ref["top2_val"].view(np.uint32))
    assert ref["top2_id"][0].tolist() == [V - 1, V - 2] and ref["top2_id"][2].tolist() == [0, V - 1]
    assert ref["accept_len"][0] >= 2
    val, idx = mars.topk_rows(z, 10)
    torch.cuda.synchronize()
    rv, ri = orc.topk(synth.to_numpy_bits(z), 10)
    assert np.array_equal(idx.cpu().numpy(), ri) and np.array_equal(val.cpu().numpy().view(np.uint32), rv.view(np.uint32))


@pytest.mark.parametrize("B,N,V", [(75, 8, 32000), (100, 7, 151936), (40, 40, 50000)])
def test_batches_just_above_one_wave_and_short_rows(B, N, V):
    """Row counts between 593 and about 900, and short rows in larger batches, run the bf16 variant
    with 8 resident blocks per SM: same bits as the oracle."""
    w = synth.tree_workload("w8", B, N, 3, 3, V, torch.bfloat16, DEV, 940 + N, 0.9, 3.0, 15.0, 30.0, 0.3)
    assert w.R > 592
    ref = orc.verify_tree(synth.to_numpy_bits(w.logits), w.tok, w.parent, w.theta)
    got = mars.to_host(mars.verify_tree(w.logits, w.tok, w.parent, w.theta, debug=True))
    assert_same(got, ref, KEYS_TREE, w.name)
    assert np.array_equal(got["top2_val"].view(np.uint32), ref["top2_val"].view(np.uint32))


def test_default_calls_are_ordered_behind_a_producer_that_rewrites_the_logits():
    """Without MARS_LOGITS_READY a call may be scheduled early but reads nothing before its
    predecessor on the stream is done.  One logits buffer is rewritten in place by a copy kernel
    between calls of three different entry points (deterministic tree, top-k, stochastic tree),
    thirty rounds with nothing in between; every call must see exactly the contents that stream
    order gives it."""
    B, N, V = 24, 10, 40000
    ws = [synth.tree_workload(f"mix{j}", B, N, 4, 3, V, torch.bfloat16, DEV, 940 + j, 0.9, 3.0, 15.0, 30.0, 0.3)
          for j in range(2)]
    hosts = [synth.to_numpy_bits(w.logits) for w in ws]
    tok = torch.as_tensor(ws[0].tok, device=DEV)
    par = torch.as_tensor(ws[0].parent, device=DEV)
    u = synth.make_uniforms(B, N, 7)
    u_dev = torch.as_tensor(u, device=DEV)
    ref_tree = [orc.verify_tree(h, ws[0].tok, ws[0].parent, 0.9) for h in hosts]
    ref_topk = [orc.topk(h, 10) for h in hosts]
    ref_st = [orc.verify_tree_stochastic(h, ws[0].tok, ws[0].parent, u, 0.9, 1.0) for h in hosts]
    live = torch.empty_like(ws[0].logits)
    rounds = 30
    o_tree = [mars.alloc_outputs(B, N, N - 1, DEV, debug=True) for _ in range(rounds)]
    o_topk = [(torch.empty((B * N, 10), dtype=torch.float32, device=DEV),
               torch.empty((B * N, 10), dtype=torch.int32, device=DEV)) for _ in range(rounds)]
    o_st = [mars.alloc_stochastic_outputs(B, N, N - 1, DEV, debug=True) for _ in range(rounds)]
    work = torch.zeros(mars.workspace_bytes(B, N, V, mars.BF16), dtype=torch.uint8, device=DEV)
    work_k = torch.empty(int(mars.lib().mars_topk_workspace_bytes(B * N, V, mars.BF16, 10)), dtype=torch.uint8, device=DEV)
    work_s = torch.empty(int(mars.lib().mars_stochastic_workspace_bytes(B, N, V, mars.BF16)), dtype=torch.uint8, device=DEV)
    torch.cuda.synchronize()
    for i in range(rounds):
        live.copy_(ws[i & 1].logits)                       # the producer: rewrites the rows in place
        mars.verify_tree(live, tok, par, 0.9, workspace=work, out=o_tree[i])
        mars.topk_rows(live, 10, workspace=work_k, out=o_topk[i])
        mars.verify_tree_stochastic(live, tok, par, u_dev, 0.9, 1.0, workspace=work_s, out=o_st[i])
    torch.cuda.synchronize()
    import stochastic_checks as ts
    for i in range(rounds):
        j = i & 1
        assert_same(mars.to_host(o_tree[i]), ref_tree[j], KEYS_TREE, f"round {i} tree")
        assert np.array_equal(o_topk[i][1].cpu().numpy(), ref_topk[j][1]), f"round {i} top-k ids"
        assert np.array_equal(o_topk[i][0].cpu().numpy().view(np.uint32), ref_topk[j][0].view(np.uint32)), i
        ts.compare(mars.to_host(o_st[i]), ref_st[j], ws[0].tok, ws[0].parent,
                   ws[j].logits.float().cpu().numpy().astype(np.float64), u, 1.0, f"round {i} stochastic")
