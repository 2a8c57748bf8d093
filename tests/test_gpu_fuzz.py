"""Seeded differential fuzzing of the CUDA library against the CPU oracle: random batch shapes,
vocabularies, row strides and alignments, thresholds, flags, padding nodes and special values
(NaN, +-inf, equal logits), for the deterministic calls (bit-exact) and the stochastic calls
(the tolerance policy of test_gpu_stochastic.py)."""
import numpy as np
import pytest
import torch

from oracle import mars_oracle as orc
from paper_2601_15498_b200 import mars, synth

import hookctl as hooks

import stochastic_checks as ts

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def random_case(rng, stochastic: bool):
    B = int(rng.integers(1, 24))
    N = int(rng.choice([1, 2, 3, 5, 8, 17, 33, 64, 65, 70]))
    V = int(rng.choice([2, 3, 7, 64, 255, 256, 257, 1000, 4096, 5001, 20000]))
    dtype = torch.bfloat16 if rng.random() < 0.5 else torch.float32
    pad = int(rng.choice([0, 0, 1, 3, 8]))
    shift = int(rng.choice([0, 0, 1, 2, 5]))
    ld = V + pad
    R = B * N
    sigma = float(rng.choice([0.5, 1.0, 3.0]))
    z = torch.tensor(rng.normal(size=(R, V)) * sigma, dtype=torch.float32)
    top = rng.uniform(2.0, 12.0, R)
    ids = rng.integers(0, V, (R, 2))
    z[torch.arange(R), torch.as_tensor(ids[:, 0])] = torch.tensor(top, dtype=torch.float32)
    low = rng.random(R) < 0.4
    rho = rng.uniform(0.8, 1.0, R)
    for r in np.flatnonzero(low):
        if ids[r, 1] != ids[r, 0]:
            z[r, ids[r, 1]] = float(rho[r] * top[r])
    if rng.random() < 0.5:      # coarse values: plenty of exact ties
        z = torch.round(z * 2) / 2
    if rng.random() < 0.4:      # special values
        k = max(1, R * V // 50)
        rr, cc = rng.integers(0, R, k), rng.integers(0, V, k)
        vals = rng.choice([np.nan, -np.inf, 0.0, -0.0], k)
        z[torch.as_tensor(rr), torch.as_tensor(cc)] = torch.tensor(vals, dtype=torch.float32)
        if not stochastic and rng.random() < 0.3:
            z[int(rng.integers(0, R)), int(rng.integers(0, V))] = float("inf")
    z = z.to(dtype)
    # device layout: [R, ld] with an element shift of the base pointer
    flat = torch.full((R * ld + shift + 8,), 77.0, dtype=dtype, device=DEV)
    view = torch.as_strided(flat[shift:], (R, V), (ld, 1))
    view.copy_(z.to(DEV))
    # tree
    depth = int(rng.integers(1, 8))
    parent = synth.make_parents(B, N, min(depth, max(N - 1, 0)), int(rng.integers(1, 5)), int(rng.integers(1 << 30)))
    lead = torch.topk(z.float().nan_to_num(nan=-np.inf), min(2, V), dim=1).indices.numpy()
    tok = synth.make_tokens(parent, lead, V, int(rng.integers(1 << 30)), p_top1=0.5, p_top2=0.3)
    if N > 3 and rng.random() < 0.5:
        tok[:, int(rng.integers(1, N))] = -1
        parent[:, N - 1] = -1
    if N > 2 and rng.random() < 0.15:
        parent[int(rng.integers(0, B)), N - 1] = N - 1     # malformed
    shared = rng.random() < 0.2
    if shared:
        parent = np.ascontiguousarray(parent[0])
    theta = float(rng.choice([0.5, 0.8, 0.9, 0.95, 1.0, 1.5, -0.5]))
    flags = 0
    r = rng.random()
    if r < 0.15:
        flags |= mars.SIGN_LITERAL
    elif r < 0.3:
        flags |= mars.RULE_MARGIN
        theta = float(rng.choice([0.25, 1.0, 3.0]))
    elif r < 0.45:
        flags |= mars.RULE_PROB_RATIO
        theta = float(rng.choice([0.1, 0.5, 0.9]))
    Dcap = N - 1 if rng.random() < 0.8 else int(rng.integers(0, max(N - 1, 1)))
    host = synth.to_numpy_bits(z)
    return dict(B=B, N=N, V=V, view=view, host=host, z=z, tok=tok, parent=parent, theta=theta, flags=flags,
                Dcap=Dcap, keep=flat)


@pytest.mark.parametrize("seed", range(40))
def test_deterministic_tree_and_chain(seed, monkeypatch):
    rng = np.random.default_rng(1000 + seed)
    if rng.random() < 0.3:
        hooks.set("HOOK_FORCE_SPLIT", int(rng.integers(2, 6)))
    else:
        hooks.clear("HOOK_FORCE_SPLIT")
    for _ in range(4):
        c = random_case(rng, stochastic=False)
        got = mars.to_host(mars.verify_tree(c["view"], c["tok"], c["parent"], c["theta"], c["flags"], c["Dcap"],
                                            debug=True))
        ref = orc.verify_tree(c["host"], c["tok"], c["parent"], c["theta"], c["flags"], c["Dcap"])
        for k in ("accept_len", "out_tokens", "path_nodes", "out_len", "seq_status", "top2_id", "node_flags"):
            assert np.array_equal(got[k], ref[k]), (seed, k, c["B"], c["N"], c["V"])
        assert np.array_equal(got["top2_val"].view(np.uint32), ref["top2_val"].view(np.uint32)), seed
        if c["parent"].ndim == 2 and c["N"] > 1:
            draft = np.ascontiguousarray(c["tok"][:, 1:])
            gc = mars.to_host(mars.verify_chain(c["view"], draft, c["theta"], c["flags"], debug=True))
            rc = orc.verify_chain(c["host"], draft, c["theta"], c["flags"])
            for k in ("accept_len", "out_tokens", "out_len", "top2_id"):
                assert np.array_equal(gc[k], rc[k]), (seed, "chain", k)


@pytest.mark.parametrize("seed", range(40))
def test_stochastic_tree(seed, monkeypatch):
    rng = np.random.default_rng(5000 + seed)
    hooks.clear("HOOK_FORCE_SPLIT")
    if rng.random() < 0.3:
        hooks.set("HOOK_FORCE_SPLIT", int(rng.integers(2, 6)))
    if rng.random() < 0.5:
        hooks.set("HOOK_STOCH_TAIL_CLUSTER", int(rng.choice([1, 2, 4, 8])))
    else:
        hooks.clear("HOOK_STOCH_TAIL_CLUSTER")
    for _ in range(3):
        c = random_case(rng, stochastic=True)
        T = float(rng.choice([0.02, 0.3, 0.7, 1.0, 1.7, 50.0]))
        flags = c["flags"] | int(rng.choice([0, mars.STOCH_PLAIN, mars.STOCH_RELAX_ONLY]))
        u = synth.make_uniforms(c["B"], c["N"], int(rng.integers(1 << 30)))
        if rng.random() < 0.3:
            u[:, 1:] = np.float32(0.9999)
        got = mars.to_host(mars.verify_tree_stochastic(c["view"], c["tok"], c["parent"], u, c["theta"], T, flags,
                                                       c["Dcap"], debug=True))
        ref = orc.verify_tree_stochastic(c["host"], c["tok"], c["parent"], u, c["theta"], T, flags, c["Dcap"])
        ts.compare(got, ref, c["tok"], c["parent"], c["z"].double().numpy(), u, T, f"fuzz {seed}",
                   max_close_frac=0.25)


@pytest.mark.parametrize("seed", range(20))
def test_sampled_chains(seed, monkeypatch):
    rng = np.random.default_rng(9000 + seed)
    hooks.clear("HOOK_FORCE_SPLIT")
    if rng.random() < 0.5:
        hooks.set("HOOK_STOCH_TAIL_CLUSTER", int(rng.choice([1, 2, 4, 8])))
    else:
        hooks.clear("HOOK_STOCH_TAIL_CLUSTER")
    for _ in range(3):
        B, K = int(rng.integers(1, 40)), int(rng.choice([2, 3, 5, 9]))
        V = int(rng.choice([9, 257, 1000, 5001, 40000]))
        dtype = torch.bfloat16 if rng.random() < 0.5 else torch.float32
        T, Tq = float(rng.choice([0.5, 1.0, 2.0])), float(rng.choice([0.7, 1.0, 1.5]))
        flags = int(rng.choice([0, mars.STOCH_PLAIN, mars.STOCH_RELAX_ONLY]))
        w, qdev, zq, draft, qx, u = ts.sampled_case(int(rng.integers(1 << 20)), B, K, V, dtype,
                                                    float(rng.choice([0.3, 1.0, 2.0])), T, Tq,
                                                    ld_pad=int(rng.choice([0, 3])))
        if rng.random() < 0.3:
            u[:, 1:] = np.float32(0.9999)
        got = mars.to_host(mars.verify_chain_sampled(w.logits, qdev, draft, qx, u, 0.9, T, Tq, flags, V=V, debug=True))
        ref = orc.verify_chain_sampled(synth.to_numpy_bits(w.logits), synth.to_numpy_bits(zq), draft, qx, u, 0.9, T, Tq,
                                       flags)
        ts.compare_sampled(got, ref, f"fuzz sampled {seed}")


@pytest.mark.parametrize("seed", range(20))
def test_sharded_stochastic_tree(seed, monkeypatch):
    rng = np.random.default_rng(7000 + seed)
    hooks.clear("HOOK_FORCE_SPLIT")
    hooks.clear("HOOK_STOCH_TAIL_CLUSTER")
    for _ in range(2):
        c = random_case(rng, stochastic=True)
        if c["V"] < 8:
            continue
        V = c["V"]
        cuts = sorted(set(int(x) for x in rng.integers(2, V - 2, int(rng.integers(0, 4)))))
        edges = [0] + [x for x in cuts if 2 <= x <= V - 2] + [V]
        ranges = [(a, b) for a, b in zip(edges, edges[1:]) if b - a >= 2]
        if not ranges or ranges[0][0] != 0 or ranges[-1][1] != V or any(a2 != b1 for (_, b1), (a2, _) in zip(ranges, ranges[1:])):
            ranges = [(0, V)]
        T = float(rng.choice([0.5, 1.0, 2.0]))
        flags = c["flags"] | int(rng.choice([0, mars.STOCH_PLAIN]))
        u = synth.make_uniforms(c["B"], c["N"], int(rng.integers(1 << 30)))
        logits = c["view"].contiguous()
        ref = orc.verify_tree_stochastic(c["host"], c["tok"], c["parent"], u, c["theta"], T, flags)
        outs, _ = ts.sharded_stochastic(logits, c["tok"], c["parent"], u, c["theta"], T, ranges, flags)
        for o in outs:
            ts.compare(o, ref, c["tok"], c["parent"], c["z"].double().numpy(), u, T, f"fuzz sharded {seed}",
                       max_close_frac=0.25)


@pytest.mark.parametrize("seed", range(30))
def test_topk_rows(seed):
    """Exact top-k against the oracle over random shapes, k, dtypes, value patterns that stress
    the floor and the queue (ties, sorted rows, constant rows, NaN / +-inf / +-0, a heavy second
    half), unaligned padded views and forced row splits; a second call must repeat the first."""
    rng = np.random.default_rng(7000 + seed)
    for _ in range(4):
        V = int(rng.choice([int(rng.integers(1, 300)), int(rng.integers(300, 20000)), int(rng.integers(20000, 160000))]))
        k = int(min(V, rng.choice([1, 2, 3, 7, 10, 16, 31, 32])))
        rows = int(max(1, min(rng.choice([1, 3, 17, 200, 700]), 12_000_000 // V)))
        dtype = torch.bfloat16 if rng.random() < 0.6 else torch.float32
        kind = str(rng.choice(["normal", "ties", "asc", "desc", "const", "special", "blocks"]))
        g = torch.Generator(device=DEV)
        g.manual_seed(int(rng.integers(1 << 30)))
        z = torch.randn((rows, V), generator=g, device=DEV) * 3
        if kind == "ties":
            z = torch.round(z)
        elif kind == "asc":
            z = torch.sort(z, dim=1).values
        elif kind == "desc":
            z = torch.sort(z, dim=1, descending=True).values
        elif kind == "const":
            z[:] = 1.5
        elif kind == "special":
            m = torch.rand((rows, V), generator=g, device=DEV)
            z[m < 0.01] = float("nan")
            z[(m > 0.01) & (m < 0.02)] = float("-inf")
            z[(m > 0.02) & (m < 0.021)] = float("inf")
            z[m > 0.9] = 0.0
            z[(m > 0.8) & (m < 0.9)] = -0.0
        elif kind == "blocks":
            z[:, V // 2:] += 10
        if rng.random() < 0.3 and V > 16:
            big = torch.full((rows, V + 13), 3e38, dtype=dtype, device=DEV)
            zz = big[:, 5:5 + V]
            zz.copy_(z.to(dtype))
        else:
            zz = z.to(dtype)
        hooks.set("HOOK_FORCE_SPLIT", int(rng.choice([0, 0, 0, 2, 5])))
        val, idx = mars.topk_rows(zz, k)
        val2, idx2 = mars.topk_rows(zz, k)
        torch.cuda.synchronize()
        hooks.clear("HOOK_FORCE_SPLIT")
        rv, ri = orc.topk(synth.to_numpy_bits(zz.contiguous()), k)
        what = (V, k, rows, str(dtype), kind)
        assert np.array_equal(idx.cpu().numpy(), ri), what
        assert np.array_equal(val.cpu().numpy().view(np.uint32), rv.view(np.uint32)), what
        assert torch.equal(idx, idx2) and torch.equal(val.view(torch.int32), val2.view(torch.int32)), what
