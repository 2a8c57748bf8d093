"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each expected value comes from an
independent route: a library sort, brute force, a closed form, a value the paper prints,
or a hand-built row whose answer is known by construction.
"""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import mars_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
F32 = np.float32


def bf16_bits(a):
    t = torch.from_numpy(np.asarray(a, np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def widen(a):
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << 16).view(np.float32)
    return a


def sort_top2(row):
    """Top-2 by a library sort on (-value, id); NaN counts as -inf."""
    x = widen(row).astype(np.float64)
    x = np.where(np.isnan(x), -np.inf, x)
    order = np.lexsort((np.arange(len(x)), -x))
    return order[0], order[1], x[order[0]], x[order[1]]


# --------------------------------------------------------------------------- top-2

@pytest.mark.parametrize("V", [2, 3, 7, 8, 9, 64, 257, 5000])
@pytest.mark.parametrize("kind", ["f32", "bf16", "f64"])
def test_top2_matches_library_sort(V, kind):
    rng = np.random.default_rng(V * 7 + len(kind))
    z = rng.normal(0, 3, size=(16, V)).astype(np.float32)
    z[3] = np.round(z[3])               # heavy ties
    z[4] = 1.5                          # constant row
    if V > 4:
        z[5, 1] = np.nan
        z[5, V - 1] = np.inf
        z[6, :] = -np.inf
        z[6, V // 2] = 0.25
        z[7, :] = np.nan
    a = bf16_bits(z) if kind == "bf16" else z.astype(np.float64) if kind == "f64" else z
    val, idx = orc.top2(a)
    for r in range(len(a)):
        i1, i2, v1, v2 = sort_top2(a[r])
        assert (idx[r, 0], idx[r, 1]) == (i1, i2), (r, V, kind)
        assert val[r, 0] == v1 and val[r, 1] == v2


def test_top2_brute_force_rank():
    """O(V^2) definition: the top-1 is beaten by nobody, the top-2 by exactly one."""
    rng = np.random.default_rng(11)
    for V in (2, 5, 33, 64):
        z = rng.integers(-3, 4, size=(32, V)).astype(np.float32)  # many ties
        _, idx = orc.top2(z)
        for r in range(32):
            for want, got in ((0, idx[r, 0]), (1, idx[r, 1])):
                x = z[r, got]
                beaten_by = sum(1 for j in range(V)
                                if z[r, j] > x or (z[r, j] == x and j < got))
                assert beaten_by == want


def test_top2_hand_rows():
    # equal logits: lowest id first; -0 == +0 and is reported as +0
    val, idx = orc.top2(np.array([[1, 5, 5, 5, 2]], F32))
    assert idx.tolist() == [[1, 2]] and val.tolist() == [[5, 5]]
    val, idx = orc.top2(np.array([[-1, -0.0, 0.0, -2]], F32))
    assert idx.tolist() == [[1, 2]]
    assert not np.signbit(val).any()
    # NaN = -inf: a row with one finite entry takes the lowest other id as runner-up
    val, idx = orc.top2(np.array([[np.nan, -np.inf, 3.0, np.nan]], F32))
    assert idx.tolist() == [[2, 0]] and val[0, 0] == 3 and val[0, 1] == -np.inf
    val, idx = orc.top2(np.array([[7.0, np.nan, np.nan]], F32))
    assert idx.tolist() == [[0, 1]]
    val, idx = orc.top2(np.full((1, 5), -np.inf, F32))
    assert idx.tolist() == [[0, 1]]
    # ld > V: the padding is never read
    z = np.array([[1, 2, 3, 99, 99]], F32)
    val, idx = orc.top2(z, V=3)
    assert idx.tolist() == [[2, 1]]


# --------------------------------------------------------------------------- ratio rule

def read_fig2():
    rows = []
    with open(os.path.join(GOLDEN, "fig2_workflow.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                th, r, which, dec = line.split()
                rows.append((float(th), float(r), which, dec))
    return rows


def test_fig2_worked_example():
    """The paper's Fig. 2: theta = 0.9, r = 0.911 accepts the top-2 draft, r = 0.728 rejects
    it and emits the target's top-1."""
    rows = read_fig2()
    assert len(rows) == 2
    for theta, r, which, decision in rows:
        assert which == "top2"
        z = np.zeros((2, 16), F32)
        z[:, 4] = 10.0
        z[:, 9] = 10.0 * r
        draft = np.array([[9]], np.int32)
        out = orc.verify_chain(z, draft, theta)
        assert abs(out["top2_val"][0, 1] / out["top2_val"][0, 0] - r) < 1e-6
        if decision == "accept":
            assert out["accept_len"][0] == 1 and out["out_tokens"][0].tolist() == [9, 4]
        else:
            assert out["accept_len"][0] == 0 and out["out_tokens"][0].tolist() == [4, -1]


PRECISIONS = [pytest.param(False, id="fp32"), pytest.param(True, id="fp64")]


def _ty(fp64):
    """Decision type of the stored-logits path (fp32) or of the projected-logits path (fp64)."""
    return np.float64 if fp64 else F32


@pytest.mark.parametrize("fp64", PRECISIONS)
@pytest.mark.parametrize("theta", [0.9, 0.84, 0.95, 0.5])
@pytest.mark.parametrize("k", [-3, 0, 4])
def test_ratio_one_ulp_around_theta(theta, k, fp64):
    """z1 a power of two makes z2/z1 exact, so r > theta iff z2 > theta*z1 (strict); the planted
    values sit one ulp of the decision type around theta*z1."""
    T = _ty(fp64)
    th = T(F32(theta))                   # theta is handed to the library as an fp32 value
    z1 = T(2.0 ** k)
    on = T(th * z1)                      # exact: scaling by a power of two
    up = np.nextafter(on, T(np.inf), dtype=T)
    dn = np.nextafter(on, T(-np.inf), dtype=T)
    assert up > on > dn
    assert orc.relax(z1, up, th, fp64=fp64)
    assert not orc.relax(z1, on, th, fp64=fp64)     # r == theta rejects
    assert not orc.relax(z1, dn, th, fp64=fp64)
    # operands the other way round would accept all three (z1/z2 > 1 > theta)
    # through the whole path as well
    for z2, want in ((up, 1), (on, 0), (dn, 0)):
        z = np.full((2, 8), -1.0, T)
        z[:, 2] = z1
        z[:, 5] = z2
        out = orc.verify_chain(z, np.array([[5]], np.int32), float(th))
        assert out["accept_len"][0] == want
        tok = np.array([[-1, 5]], np.int32)
        par = np.array([[-1, 0]], np.int32)
        assert orc.verify_tree(z, tok, par, float(th))["accept_len"][0] == want


@pytest.mark.parametrize("fp64", PRECISIONS)
def test_ratio_equals_adaptive_margin_form(fp64):
    """Eq. 6: r > theta  <=>  Delta < (1 - theta) z1, checked in fp64 away from equality."""
    rng = np.random.default_rng(5)
    n = 0
    for _ in range(20000):
        z1 = F32(rng.uniform(-5, 30))
        z2 = F32(z1 - abs(rng.normal(0, 2)))
        theta = F32(rng.choice([0.8, 0.84, 0.9, 0.95, 0.98]))
        lhs = float(z1) - float(z2)
        rhs = (1.0 - float(theta)) * float(z1)
        if abs(lhs - rhs) < 1e-4 * max(1.0, abs(float(z1))):
            continue
        n += 1
        assert orc.relax(z1, z2, theta, fp64=fp64) == (lhs < rhs), (z1, z2, theta)
    assert n > 15000


@pytest.mark.parametrize("fp64", PRECISIONS)
def test_ratio_bounded_on_positive_rows_and_sign_guard(fp64):
    rng = np.random.default_rng(6)
    z = (np.abs(rng.normal(0, 3, size=(64, 100))) + 0.01).astype(_ty(fp64))
    val, _ = orc.top2(z)
    assert val.dtype == _ty(fp64)
    r = val[:, 1] / val[:, 0]
    assert ((r > 0) & (r <= 1)).all()           # Sec. 3.3: r in (0, 1] on positive logits

    def rx(z1, z2, theta, flags=0):
        return orc.relax(z1, z2, theta, flags, fp64=fp64)
    # non-positive top-1: the guarded rule never relaxes; the literal ratio would
    assert not rx(-2.0, -3.0, 0.9)
    assert rx(-2.0, -3.0, 0.9, orc.SIGN_LITERAL)       # (-3)/(-2) = 1.5 > 0.9
    assert not rx(0.0, -1.0, 0.9) and not rx(0.0, -1.0, 0.9, orc.SIGN_LITERAL)
    assert not rx(0.0, 0.0, 0.9, orc.SIGN_LITERAL)     # 0/0 = NaN compares false
    assert not rx(np.inf, np.inf, 0.9)                 # inf/inf = NaN
    assert not rx(5.0, -1.0, 0.0)                      # r < 0
    assert rx(4.0, 4.0, 0.999)                         # exact tie: r = 1
    assert not rx(4.0, 4.0, 1.0)                       # theta >= 1 is strict greedy
    assert not rx(4.0, 3.999, 1.0) and not rx(4.0, 4.0, 1.5)


def test_scale_invariance_power_of_two():
    rng = np.random.default_rng(7)
    z = (rng.normal(0, 3, size=(48, 300)) + 6).astype(np.float32)
    draft = rng.integers(0, 300, size=(8, 5)).astype(np.int32)
    _, idx = orc.top2(z)
    draft[:, 0] = idx[::6, 0][:8]
    draft[:, 1] = idx[1::6, 1][:8]
    a = orc.verify_chain(z, draft, 0.9)
    for s in (0.25, 8.0, 1024.0):
        b = orc.verify_chain((z * F32(s)).astype(np.float32), draft, 0.9)
        for key in ("accept_len", "out_tokens", "out_len", "top2_id"):
            assert (a[key] == b[key]).all()


# --------------------------------------------------------------------------- chain

def greedy_chain(z, draft):
    """Strict greedy verification (T = 0): accept while draft == argmax, then emit argmax."""
    B, Km1 = draft.shape
    K = Km1 + 1
    acc, toks = [], []
    for b in range(B):
        out, a = [], 0
        for i in range(Km1):
            top = int(np.argmax(z[b * K + i]))         # first maximum = lowest id
            if draft[b, i] == top:
                out.append(top); a += 1
            else:
                out.append(top); break
        else:
            out.append(int(np.argmax(z[b * K + K - 1])))
        acc.append(a); toks.append(out + [-1] * (K - len(out)))
    return np.array(acc), np.array(toks)


def planted_chain(rng, B, K, V, p_top1=0.6, p_top2=0.25, p_low=0.4):
    z = rng.normal(0, 2, size=(B * K, V)).astype(np.float32)
    draft = np.empty((B, K - 1), np.int32)
    for r in range(B * K):
        a, b = rng.choice(V, 2, replace=False)
        z[r, a] = 20.0
        second = int(np.argmax(np.where(np.arange(V) == a, -np.inf, z[r])))
        if rng.random() < p_low:
            z[r, b] = 20.0 * rng.uniform(0.85, 1.0)
            second = b
        if r % K < K - 1:
            u = rng.random()
            draft[r // K, r % K] = a if u < p_top1 else second if u < p_top1 + p_top2 else rng.integers(V)
    return z, draft


@pytest.mark.parametrize("theta", [1.0, 1.5, 100.0])
def test_theta_ge_one_is_strict_greedy(theta):
    rng = np.random.default_rng(8)
    z, draft = planted_chain(rng, 200, 6, 64)
    z[::7, 3] = 20.0     # exact ties with the planted top: r = 1 must still not relax
    out = orc.verify_chain(z, draft, theta)
    acc, toks = greedy_chain(z, draft)
    assert (out["accept_len"] == acc).all() and (out["out_tokens"] == toks).all()
    assert (out["out_len"] == acc + 1).all()


def test_chain_monotone_in_theta_and_bounds():
    rng = np.random.default_rng(9)
    z, draft = planted_chain(rng, 300, 8, 50)
    prev = None
    for theta in (0.5, 0.8, 0.9, 0.95, 1.0):
        out = orc.verify_chain(z, draft, theta)
        assert ((out["out_len"] >= 1) & (out["out_len"] <= 8)).all()      # tau <= K + 1
        assert (out["out_len"] == out["accept_len"] + 1).all()
        if prev is not None:
            assert (out["accept_len"] <= prev).all()                      # MARS only adds accepts
        prev = out["accept_len"]
    # some relaxed accepts exist, so the sweep is not vacuous
    assert (orc.verify_chain(z, draft, 0.5)["accept_len"] > prev).any()


def test_chain_closed_form_acceptance_length():
    """Per-position acceptance is i.i.d. with p known from the input recipe, so the accepted
    length is a truncated geometric: E[a] = sum_{k=1..K-1} p^k."""
    B, K, V, theta = 8000, 6, 256, 0.9
    rng = np.random.default_rng(10)
    z, draft = planted_chain(rng, B, K, V)
    out = orc.verify_chain(z, draft, theta)
    q = 0.4 * (1.0 - 0.9) / 0.15 * 0 + 0.4 * (0.1 / 0.15)      # runner-up planted and rho > 0.9
    p = 0.6 + 0.25 * q + 0.15 * (1.0 + q) / V
    pk = np.array([p ** k for k in range(1, K)])
    mean = pk.sum()
    # E[a^2] = sum (2k-1) p^k for a truncated geometric
    second = sum((2 * k - 1) * p ** k for k in range(1, K))
    sd = np.sqrt(second - mean ** 2) / np.sqrt(B)
    got = out["accept_len"].mean()
    assert abs(got - mean) < 4 * sd, (got, mean, sd)
    # the fraction accepted at the first position pins p itself
    p_hat = (out["accept_len"] >= 1).mean()
    assert abs(p_hat - p) < 4 * np.sqrt(p * (1 - p) / B)


# --------------------------------------------------------------------------- tree

def all_parent_arrays(N):
    for tail in itertools.product(*[range(i) for i in range(1, N)]):
        yield (-1,) + tail


def path_to(parent, i):
    path = []
    while i != 0:
        path.append(i)
        i = parent[i]
    return path[::-1]


def test_tree_brute_force_all_small_trees():
    """Every tree shape with N <= 5 (and a sample of N = 6), every per-node match kind
    {none, top-1, top-2} and every per-row relaxation bit, against an explicit enumeration
    of root-to-node paths, each judged token by token with the three-way rule."""
    V = 6
    rng = np.random.default_rng(12)
    cases = []
    for N in (1, 2, 3, 4, 5):
        for par in all_parent_arrays(N):
            for kinds in itertools.product((0, 1, 2), repeat=N - 1):
                for rbits in itertools.product((0, 1), repeat=N):
                    cases.append((N, par, (0,) + kinds, rbits))
    shapes6 = list(all_parent_arrays(6))
    for _ in range(4000):
        par = shapes6[rng.integers(len(shapes6))]
        cases.append((6, par, (0,) + tuple(rng.integers(0, 3, 5)), tuple(rng.integers(0, 2, 6))))
    by_n = {}
    for c in cases:
        by_n.setdefault(c[0], []).append(c)
    for N, cs in by_n.items():
        B = len(cs)
        z = np.zeros((B * N, V), F32)
        tok = np.full((B, N), -1, np.int32)
        parent = np.empty((B, N), np.int32)
        top1 = np.empty((B, N), np.int64)
        for b, (_, par, kinds, rbits) in enumerate(cs):
            parent[b] = par
            for i in range(N):
                i1, i2, other = rng.choice(V, 3, replace=False)
                z[b * N + i, i1] = 10.0
                z[b * N + i, i2] = 9.5 if rbits[i] else 5.0
                top1[b, i] = i1
                # children of i read this row: remember its ids for them
                z[b * N + i, other] = 1.0     # marks the "no match" token
            for i in range(1, N):
                p = par[i]
                row = z[b * N + p]
                i1 = int(np.argmax(row))
                i2 = int(np.argmax(np.where(np.arange(V) == i1, -1, row)))
                other = int(np.flatnonzero(row == 1.0)[0])
                tok[b, i] = (other, i1, i2)[kinds[i]]
        out = orc.verify_tree(z, tok, parent, 0.9)
        assert (out["seq_status"] == 0).all()
        for b, (_, par, kinds, rbits) in enumerate(cs):
            best, best_d = 0, 0
            accepted = {0}
            for i in range(1, N):
                ok = True
                for n in path_to(par, i):
                    k, p = kinds[n], par[n]
                    ok = ok and (k == 1 or (k == 2 and rbits[p] == 1))
                if ok:
                    accepted.add(i)
                    d = len(path_to(par, i))
                    if d > best_d:
                        best, best_d = i, d
            assert out["accept_len"][b] == best_d, (N, par, kinds, rbits)
            want_path = [0] + path_to(par, best)
            assert out["path_nodes"][b, :best_d + 1].tolist() == want_path
            assert (out["path_nodes"][b, best_d + 1:] == -1).all()
            want_tok = [tok[b, n] for n in want_path[1:]] + [top1[b, best]]
            assert out["out_tokens"][b, :best_d + 1].tolist() == want_tok
            assert (out["out_tokens"][b, best_d + 1:] == -1).all()
            assert out["out_len"][b] == best_d + 1
            flags = out["node_flags"][b]
            assert {i for i in range(N) if flags[i] & 4} == accepted
            assert {i for i in range(N) if flags[i] & 8} == set(want_path)


def test_chain_equals_tree_with_linear_parents():
    rng = np.random.default_rng(13)
    B, K, V = 150, 7, 40
    z, draft = planted_chain(rng, B, K, V)
    zb = bf16_bits(z)
    for logits in (z, zb):
        for theta in (0.8, 0.9, 1.0):
            c = orc.verify_chain(logits, draft, theta)
            tok = np.concatenate([np.full((B, 1), -1, np.int32), draft], axis=1)
            par = np.tile(np.arange(-1, K - 1, dtype=np.int32), (B, 1))
            t = orc.verify_tree(logits, tok, par, theta)
            assert (c["accept_len"] == t["accept_len"]).all()
            assert (c["out_tokens"] == t["out_tokens"]).all()
            assert (c["out_len"] == t["out_len"]).all()
            t2 = orc.verify_tree(logits, tok, par[0], theta)           # shared parent array
            assert (t2["out_tokens"] == t["out_tokens"]).all()


def test_tree_invariants_random():
    from paper_2601_15498_b200 import synth
    w = synth.tree_workload("t", 40, 60, 6, 4, 2000, torch.bfloat16, "cpu", 21, 0.9, 3.0, 15.0,
                            30.0, 0.3)
    out = orc.verify_tree(synth.to_numpy_bits(w.logits), w.tok, w.parent, w.theta)
    depth = np.zeros((w.B, w.N), int)
    for b in range(w.B):
        for i in range(1, w.N):
            depth[b, i] = depth[b, w.parent[b, i]] + 1
        f = out["node_flags"][b]
        acc = (f & 4) != 0
        assert acc[0]
        for i in range(1, w.N):
            if acc[i]:
                assert acc[w.parent[b, i]] and (f[i] & 3) != 0       # ancestor-closed
        a = out["accept_len"][b]
        assert a == depth[b][acc].max() <= w.max_depth                # accepted length <= depth
        path = out["path_nodes"][b, :a + 1]
        assert path[0] == 0 and all(w.parent[b, path[k]] == path[k - 1] for k in range(1, a + 1))
        assert acc[path].all()
        # lowest index among the deepest accepted nodes
        assert path[-1] == np.flatnonzero(acc & (depth[b] == a))[0]
    assert out["accept_len"].max() >= 3 and out["accept_len"].min() == 0   # not vacuous


def test_tree_padding_and_malformed():
    z = np.zeros((4, 8), F32)
    z[:, 1] = 5.0
    z[:, 2] = 4.9
    tok = np.array([[-1, 1, 2, 1]], np.int32)
    # node 2 is padding (parent -1): never accepted, and neither is its child
    out = orc.verify_tree(z, tok, np.array([[-1, 0, -1, 2]], np.int32), 0.9)
    assert out["seq_status"][0] == 0 and out["accept_len"][0] == 1
    assert out["path_nodes"][0].tolist() == [0, 1, -1, -1]
    # negative token = padding
    out = orc.verify_tree(z, np.array([[-1, -5, 2, 1]], np.int32),
                          np.array([[-1, 0, 0, 2]], np.int32), 0.9)
    assert out["accept_len"][0] == 2 and out["out_tokens"][0].tolist() == [2, 1, 1, -1]
    # token id beyond the vocabulary never matches
    out = orc.verify_tree(z, np.array([[-1, 99, 99, 99]], np.int32),
                          np.array([[-1, 0, 0, 0]], np.int32), 0.9)
    assert out["accept_len"][0] == 0 and out["out_tokens"][0, 0] == 1
    for bad in ([0, 0, 1, 2], [-1, 1, 0, 0], [-1, 0, 5, 0], [-1, 0, -2, 0]):
        out = orc.verify_tree(z, tok, np.array([bad], np.int32), 0.9)
        assert out["seq_status"][0] == 1
        assert out["accept_len"][0] == 0 and out["out_len"][0] == 1
        assert out["out_tokens"][0].tolist() == [1, -1, -1, -1]
        assert out["node_flags"][0].tolist() == [12, 0, 0, 0]
    # depth cap exceeded -> status 2 and the safe output
    out = orc.verify_tree(z, np.array([[-1, 1, 1, 1]], np.int32),
                          np.array([[-1, 0, 1, 2]], np.int32), 0.9, Dcap=2)
    assert out["seq_status"][0] == 2 and out["accept_len"][0] == 0
    out = orc.verify_tree(z, np.array([[-1, 1, 1, 7]], np.int32),
                          np.array([[-1, 0, 1, 2]], np.int32), 0.9, Dcap=2)
    assert out["seq_status"][0] == 0 and out["accept_len"][0] == 2


# --------------------------------------------------------------------------- LM head

def test_lmhead_one_hot_weights_reduce_to_gather():
    """With W_o rows that are scaled unit vectors, z[r, j] = c_j * h[r, k_j]: the top-2 is
    known without any contraction."""
    rng = np.random.default_rng(14)
    M, V, d = 6, 40, 16
    h = rng.integers(1, 9, size=(M, d)).astype(np.float32)     # exactly representable in bf16
    w = np.zeros((V, d), np.float32)
    col = rng.integers(0, d, V)
    w[np.arange(V), col] = 1.0
    z = orc.lmhead_logits(bf16_bits(h), bf16_bits(w))
    assert (z == h[:, col]).all()
    bias = rng.normal(size=V)
    zb = orc.lmhead_logits(bf16_bits(h), bf16_bits(w), bias)
    assert np.allclose(zb, h[:, col] + bias[None, :], rtol=0, atol=0)


def test_lmhead_small_against_hand_fp64():
    rng = np.random.default_rng(15)
    M, V, d = 8, 64, 32
    hb = bf16_bits(rng.normal(size=(M, d)))
    wb = bf16_bits(rng.normal(size=(V, d)) * 0.2)
    hf, wf = widen(hb).astype(np.float64), widen(wb).astype(np.float64)
    z = np.array([[sum(hf[r, k] * wf[j, k] for k in range(d)) for j in range(V)] for r in range(M)])
    got = orc.lmhead_logits(hb, wb)
    assert np.allclose(got, z, rtol=1e-13, atol=1e-13)
    tok = np.full((1, M), -1, np.int32)
    par = np.arange(-1, M - 1, dtype=np.int32)[None, :]
    order = np.argsort(-z, axis=1, kind="stable")
    tok[0, 1:] = order[:-1, 0]
    tok[0, 3] = order[2, 1]                                   # a runner-up draft at node 3
    out = orc.lmhead_verify_tree(hb, wb, None, tok, par, 0.0)
    r2 = z[2, order[2, 1]] / z[2, order[2, 0]]
    want = M - 1 if (z[2, order[2, 0]] > 0 and r2 > 0.0) else 2
    assert out["accept_len"][0] == want
    assert (out["top2_id"] == order[:, :2]).all()


@pytest.mark.parametrize("sign_literal", [False, True])
def test_lmhead_planted_ratio_decides_in_fp64(sign_literal):
    """One-hot W_o turns the projection into a gather, so every logit is known exactly and the
    ratio of the planted pair can be put just above / exactly at / just below theta = 3/4 with
    z1 a power of two (the division is exact).  The hidden values are bf16-representable, and one
    bf16 step at 12 is far more than one fp64 ulp, so this pins direction and strictness of the
    fp64 rule through the projection; the guard is pinned by the negative-logit rows."""
    d, V = 8, 12
    theta = 0.75
    w = np.zeros((V, d), np.float32)
    w[np.arange(V), np.arange(V) % d] = 1.0          # z[r, j] = h[r, j % d]
    w[d:, :] = 0.0                                   # columns 8..11 stay at logit 0
    cases = [                                        # (h0 = z1 at id 0, h1 = z2 at id 1, relaxes?)
        (16.0, 12.0625, True),                       # r = 0.75390625 > theta
        (16.0, 12.0, False),                         # r == theta rejects
        (16.0, 11.9375, False),
    ]
    for h0, h1, want in cases:
        h = np.full((2, d), -4.0, np.float32)
        h[:, 0], h[:, 1] = h0, h1
        hb, wb = bf16_bits(h), bf16_bits(w)
        z = orc.lmhead_logits(hb, wb)
        assert z[0, 0] == h0 and z[0, 1] == h1 and (z[0, 2:8] == -4.0).all() and (z[0, 8:] == 0).all()
        tok = np.array([[-1, 1]], np.int32)
        par = np.array([[-1, 0]], np.int32)
        flags = orc.SIGN_LITERAL if sign_literal else 0
        out = orc.lmhead_verify_tree(hb, wb, None, tok, par, theta, flags)
        assert out["top2_id"][0].tolist() == [0, 1]
        assert out["accept_len"][0] == int(want), (h0, h1)
        assert out["out_tokens"][0].tolist() == ([1, 0] if want else [0, -1])
    # all logits negative: top-1 = -8 at id 0, runner-up -12 at id 1, ratio 1.5 > theta.  The
    # guarded rule must not relax, the literal one does.
    w2 = np.eye(d, dtype=np.float32)                 # V = d: z[r, j] = h[r, j], no zero logits
    h = np.full((2, d), -30.0, np.float32)
    h[:, 0], h[:, 1] = -8.0, -12.0
    hb, wb = bf16_bits(h), bf16_bits(w2)
    out = orc.lmhead_verify_tree(hb, wb, None, np.array([[-1, 1]], np.int32), np.array([[-1, 0]], np.int32),
                                 theta, orc.SIGN_LITERAL if sign_literal else 0)
    assert out["top2_id"][0].tolist() == [0, 1]
    assert out["accept_len"][0] == int(sign_literal)


# --------------------------------------------------------------------------- rule variants

@pytest.mark.parametrize("fp64", PRECISIONS)
def test_margin_variant_one_ulp_and_through_chain(fp64):
    """Fixed-margin indicator: relax iff Delta = z1 - z2 < c (strict), one subtraction in the
    decision type."""
    T = _ty(fp64)
    c = T(0.5)
    z1 = T(8.0)
    on = T(7.5)                                             # Delta == c exactly
    closer = np.nextafter(on, T(np.inf), dtype=T)           # Delta just below c
    farther = np.nextafter(on, T(-np.inf), dtype=T)

    def rx(a, b, th, flags):
        return orc.relax(a, b, th, flags, fp64=fp64)
    assert rx(z1, closer, c, orc.RULE_MARGIN)
    assert not rx(z1, on, c, orc.RULE_MARGIN)
    assert not rx(z1, farther, c, orc.RULE_MARGIN)
    assert rx(-3.0, -3.25, c, orc.RULE_MARGIN)              # no sign guard for this indicator
    assert not rx(5.0, -np.inf, c, orc.RULE_MARGIN)
    for z2, want in ((closer, 1), (on, 0)):
        z = np.full((2, 8), -1.0, T)
        z[:, 2] = z1
        z[:, 5] = z2
        out = orc.verify_chain(z, np.array([[5]], np.int32), float(c), orc.RULE_MARGIN)
        assert out["accept_len"][0] == want
        out = orc.verify_chain(z, np.array([[2]], np.int32), float(c), orc.RULE_MARGIN)
        assert out["accept_len"][0] == 1                     # exact match is unaffected


@pytest.mark.parametrize("fp64", PRECISIONS)
def test_prob_ratio_variant_against_softmax_definition(fp64):
    """p2/p1 > theta with p = softmax(z) (Eq. 3) evaluated in fp64 on whole rows, away from
    the boundary; and the limits theta <= 0 (always) / theta >= 1 (never for distinct logits)."""
    rng = np.random.default_rng(21)

    def rx(a, b, th, flags):
        return orc.relax(a, b, th, flags, fp64=fp64)
    n = 0
    for _ in range(3000):
        z = rng.normal(0, 3, 50).astype(np.float32)
        theta = F32(rng.uniform(0.05, 0.95))
        zs = np.sort(z.astype(np.float64))[::-1]
        p = np.exp(zs - zs[0]); p /= p.sum()
        ratio = p[1] / p[0]
        if abs(ratio - float(theta)) < 1e-4:
            continue
        n += 1
        assert rx(zs[0], zs[1], theta, orc.RULE_PROB_RATIO) == (ratio > float(theta))
    assert n > 2500
    assert rx(3.0, -40.0, 0.0, orc.RULE_PROB_RATIO) and rx(3.0, -40.0, -1.0, orc.RULE_PROB_RATIO)
    assert not rx(3.0, 2.999, 1.0, orc.RULE_PROB_RATIO)
    assert not rx(3.0, 3.0, 1.0, orc.RULE_PROB_RATIO)      # p2/p1 == 1 is not > 1
    # equal to the margin variant at c = -ln(theta)
    for theta in (0.3, 0.6, 0.9):
        c = F32(-np.log(np.float64(F32(theta))))
        for z2 in np.linspace(1.0, 3.0, 41):
            assert rx(3.0, z2, theta, orc.RULE_PROB_RATIO) == rx(3.0, z2, c, orc.RULE_MARGIN)


def test_variants_only_change_relaxed_accepts():
    rng = np.random.default_rng(22)
    z, draft = planted_chain(rng, 300, 6, 64)
    strict = orc.verify_chain(z, draft, 1.5)["accept_len"]
    for flags, th in ((orc.RULE_MARGIN, 0.0), (orc.RULE_PROB_RATIO, 1.0)):      # nothing relaxes
        assert (orc.verify_chain(z, draft, th, flags)["accept_len"] == strict).all()
    loose = orc.verify_chain(z, draft, 100.0, orc.RULE_MARGIN)["accept_len"]    # every runner-up relaxes
    assert (loose >= strict).all() and (loose > strict).any()
    mid = orc.verify_chain(z, draft, 2.0, orc.RULE_MARGIN)["accept_len"]        # planted gaps 0..3
    assert (mid >= strict).all() and (mid <= loose).all() and (mid != loose).any() and (mid != strict).any()


# --------------------------------------------------------------------------- telemetry

def test_histograms_against_numpy_histogram():
    """z1, z2/z1 and p2/p1 = exp(z2 - z1) binned by numpy in fp64, on values kept away from
    the bin edges; plus hand rows for the edge conventions."""
    rng = np.random.default_rng(31)
    nb, lo, hi = 20, 0.0, 40.0
    z1 = rng.uniform(0.5, 39.5, 20000)
    r = rng.uniform(0.0, 1.0, 20000)
    z2 = z1 * r
    v = np.stack([z1, z2], 1).astype(np.float32)
    z1f, z2f = v[:, 0].astype(np.float64), v[:, 1].astype(np.float64)
    q = [(z1f - lo) / (hi - lo) * nb, z2f / z1f * nb, np.exp(z2f - z1f) * nb]
    keep = np.ones(len(v), bool)
    for x in q:
        keep &= np.abs(x - np.round(x)) > 1e-3
    v = v[keep]
    hist, outl = orc.histograms(v, lo, hi, nb)
    z1f, z2f = v[:, 0].astype(np.float64), v[:, 1].astype(np.float64)
    assert (hist[0] == np.histogram(z1f, nb, (lo, hi))[0]).all()
    assert (hist[1] == np.histogram(z2f / z1f, nb, (0.0, 1.0))[0]).all()
    assert (hist[2] == np.histogram(np.exp(z2f - z1f), nb, (0.0, 1.0))[0]).all()
    assert outl.tolist() == [0, 0, 0] and hist.sum(1).tolist() == [len(v)] * 3
    hand = np.array([[10, 9], [20, 5], [5, 5], [-1, -2], [3, -np.inf], [np.nan, np.nan], [40, 1]], np.float32)
    hist, outl = orc.histograms(hand, 0, 30, 6)
    assert hist[0].tolist() == [1, 1, 1, 0, 1, 0] and hist[1].tolist() == [1, 1, 0, 0, 0, 2]
    assert hist[2].tolist() == [3, 0, 2, 0, 0, 1] and outl.tolist() == [3, 3, 1]


# --------------------------------------------------------------------------- top-k

@pytest.mark.parametrize("k", [1, 2, 10, 32])
def test_topk_matches_library_sort_and_top2(k):
    rng = np.random.default_rng(40 + k)
    V = 500
    z = rng.normal(0, 3, size=(12, V)).astype(np.float32)
    z[2] = np.round(z[2])                   # ties
    z[3] = 2.0                              # constant
    z[4, ::3] = np.nan
    z[5] = -np.inf
    z[5, [7, 400]] = [1.0, 1.0]             # only two entries above -inf
    for a in (z, bf16_bits(z), z.astype(np.float64)):
        val, idx = orc.topk(a, k)
        x = widen(a).astype(np.float64)
        x = np.where(np.isnan(x), -np.inf, x)
        for r in range(len(a)):
            order = np.lexsort((np.arange(V), -x[r]))[:k]
            assert idx[r].tolist() == order.tolist(), (r, k)
            assert (val[r] == x[r][order]).all()
        if k == 2:
            v2, i2 = orc.top2(a)
            assert (i2 == idx).all() and (v2 == val).all()
