"""Pins of the stochastic (T > 0) part of the CPU oracle against what the paper and the
mathematics fix (CPU only):

* the target probabilities are the softmax of the logits (Eq. 3) -> a library softmax;
* the final draw inverts the residual's CDF -> numpy cumsum + searchsorted;
* accepting with Eq. 1 and drawing the correction from the residual preserves the target
  distribution exactly (the theorem behind Eq. 1, Sec. 2.2) -> empirical frequencies of the
  first and of the second emitted token against the softmax of the rows that judge them;
* T -> 0 is greedy decoding (Sec. 2.2): the walk equals strict tree verification;
* with uniforms next to 1 the Eq. 1 test never fires, so the default (rule-first) mode on a
  chain equals Algorithm 1;
* scaling logits and T by a power of two changes nothing.

How the relaxation composes with Eq. 1 is this repository's reading (the paper does not say):
those tests check the stated reading for self-consistency, not against the paper.
"""
import numpy as np
import pytest
import torch
from scipy.special import softmax

from oracle import mars_oracle as orc
from paper_2601_15498_b200 import synth


def _rand_case(seed, B, N, V, sigma=2.0, depth=3, branch=3, dtype=np.float32):
    rng = np.random.default_rng(seed)
    logits = (rng.normal(size=(B * N, V)) * sigma).astype(dtype)
    parent = synth.make_parents(B, N, min(depth, N - 1), branch, seed)
    tok = rng.integers(0, V, (B, N)).astype(np.int32)
    tok[:, 0] = -1
    u = rng.random((B, N)).astype(np.float32)
    return logits, tok, parent, u


@pytest.mark.parametrize("T", [0.5, 1.0, 2.5])
def test_node_prob_is_a_library_softmax(T):
    logits, tok, parent, u = _rand_case(1, 6, 9, 50)
    out = orc.verify_tree_stochastic(logits, tok, parent, u, 0.9, T, orc.STOCH_PLAIN)
    P = softmax(logits.astype(np.float64) / T, axis=1)
    B, N = tok.shape
    for b in range(B):
        assert out["node_prob"][b, 0] == 0.0
        for i in range(1, N):
            want = P[b * N + parent[b, i], tok[b, i]]
            assert out["node_prob"][b, i] == pytest.approx(want, rel=1e-12)


def test_bf16_rows_widen_exactly():
    logits, tok, parent, u = _rand_case(2, 3, 7, 40)
    lb = torch.tensor(logits).to(torch.bfloat16)
    bits = synth.to_numpy_bits(lb)
    a = orc.verify_tree_stochastic(bits, tok, parent, u, 0.9, 1.0)
    b = orc.verify_tree_stochastic(lb.float().numpy(), tok, parent, u, 0.9, 1.0)
    for k in a:
        assert np.array_equal(a[k], b[k]), k


def test_final_draw_inverts_the_cdf_of_the_residual():
    """No children at all: the emitted token is a draw from the root row's softmax by CDF
    inversion; with children that are all rejected, from the row without their tokens."""
    rng = np.random.default_rng(3)
    B, V = 400, 23
    logits = (rng.normal(size=(B * 3, V)) * 2).astype(np.float32)
    u = rng.random((B, 3)).astype(np.float32)
    # (a) leaf root: N = 1 is not allowed by the shapes used elsewhere, so mark both children absent
    tok = np.full((B, 3), -1, np.int32)
    parent = np.tile(np.array([-1, 0, 0], np.int32), (B, 1))
    out = orc.verify_tree_stochastic(logits, tok, parent, u, 0.9, 1.3, orc.STOCH_PLAIN)
    for b in range(B):
        w = np.exp((logits[3 * b].astype(np.float64) - logits[3 * b].max()) / 1.3)
        c = np.cumsum(w)
        want = int(np.searchsorted(c, float(u[b, 0]) * c[-1], side="right"))
        assert out["accept_len"][b] == 0 and out["out_tokens"][b, 0] == want
    # (b) two distinct children judged with uniforms of 0.999999 (never accepted): both removed
    tok[:, 1] = rng.integers(0, V, B)
    tok[:, 2] = (tok[:, 1] + 1 + rng.integers(0, V - 1, B)) % V
    u[:, 1:] = np.float32(0.999999)
    out = orc.verify_tree_stochastic(logits, tok, parent, u, 0.9, 1.3, orc.STOCH_PLAIN)
    n_checked = 0
    for b in range(B):
        if out["accept_len"][b] != 0:
            continue   # a child with probability above 0.999999
        w = np.exp((logits[3 * b].astype(np.float64) - logits[3 * b].max()) / 1.3)
        w[tok[b, 1]] = 0.0
        w[tok[b, 2]] = 0.0
        c = np.cumsum(w)
        want = int(np.searchsorted(c, float(u[b, 0]) * c[-1], side="right"))
        assert out["out_tokens"][b, 0] == want
        assert want not in (tok[b, 1], tok[b, 2])
        n_checked += 1
    assert n_checked > B // 2


def _freq_close(tokens, p, n_sigma=4.5):
    n = len(tokens)
    f = np.bincount(tokens, minlength=len(p)) / n
    sd = np.sqrt(np.maximum(p * (1 - p), 1e-12) / n)
    assert np.all(np.abs(f - p) <= n_sigma * sd + 1e-9), (f, p)


def test_plain_mode_preserves_the_target_distribution():
    """Eq. 1 + residual (point-mass drafts, siblings tried in turn): the first emitted token is
    distributed as the root row's softmax and, given that node c was accepted, the second as row
    c's softmax.  One fixed tree, many independent uniforms."""
    rng = np.random.default_rng(4)
    V, N, B, T = 6, 7, 150_000, 0.8
    rows = (rng.normal(size=(N, V)) * 0.6).astype(np.float32)   # every token keeps a visible probability
    parent1 = np.array([-1, 0, 0, 0, 1, 1, 2], np.int32)
    tok1 = np.array([-1, 2, 5, 0, 1, 3, 4], np.int32)
    logits = np.ascontiguousarray(np.tile(rows, (B, 1)))
    tok = np.tile(tok1, (B, 1))
    u = rng.random((B, N)).astype(np.float32)
    out = orc.verify_tree_stochastic(logits, tok, parent1, u, 0.9, T, orc.STOCH_PLAIN)
    assert (out["seq_status"] == 0).all()
    P = softmax(rows.astype(np.float64) / T, axis=1)
    _freq_close(out["out_tokens"][:, 0], P[0])
    # every accepted first-level child occurs with its own probability, in any sibling position
    for c in (1, 2, 3):
        sel = out["path_nodes"][:, 1] == c
        assert abs(sel.mean() - P[0, tok1[c]]) < 4.5 * np.sqrt(P[0, tok1[c]] / B) + 1e-9
        if sel.sum() > 2000:
            _freq_close(out["out_tokens"][sel, 1], P[c])


def test_default_mode_accepts_more_than_plain_on_chains():
    """On a chain the rule-first composition can only lengthen the accepted prefix for the same
    uniforms, and the relax-only mode lies in between."""
    w = synth.chain_workload("t", 300, 6, 200, torch.float32, "cpu", 5, 0.9,
                             2.0, 6.0, 9.0, 0.5)
    logits = synth.to_numpy_bits(w.logits)
    u = np.random.default_rng(5).random((w.B, w.N)).astype(np.float32)
    a = orc.verify_tree_stochastic(logits, w.tok, w.parent, u, 0.9, 1.0, orc.STOCH_PLAIN)["accept_len"]
    r = orc.verify_tree_stochastic(logits, w.tok, w.parent, u, 0.9, 1.0, orc.STOCH_RELAX_ONLY)["accept_len"]
    d = orc.verify_tree_stochastic(logits, w.tok, w.parent, u, 0.9, 1.0, 0)["accept_len"]
    assert (a <= r).all() and (r <= d).all()
    assert a.sum() < r.sum() < d.sum()


def test_uniforms_next_to_one_reduce_the_default_mode_to_algorithm_1():
    w = synth.chain_workload("t", 200, 7, 300, torch.float32, "cpu", 6, 0.9,
                             2.0, 6.0, 9.0, 0.5)
    logits = synth.to_numpy_bits(w.logits)
    u = np.full((w.B, w.N), np.float32(1.0) - np.float32(2.0 ** -24), np.float32)
    s = orc.verify_tree_stochastic(logits, w.tok, w.parent, u, 0.9, 1.0, 0)
    g = orc.verify_chain(logits, w.draft, 0.9)
    assert np.array_equal(s["accept_len"], g["accept_len"])
    for b in range(w.B):
        a = g["accept_len"][b]
        assert np.array_equal(s["out_tokens"][b, :a], g["out_tokens"][b, :a])
    how = s["node_how"]
    assert not (how == 3).any() and (how == 1).any() and (how == 2).any() and (how == 4).any()


def test_temperature_to_zero_is_strict_greedy_tree_verification():
    """T -> 0: P collapses onto the argmax, Eq. 1 accepts exactly the top-1 child and the draw
    returns the argmax: the result of strict verification (theta >= 1)."""
    w = synth.tree_workload("t", 40, 20, 4, 3, 500, torch.float32, "cpu", 7, 0.9,
                            1.0, 8.0, 12.0, 0.3)
    logits = synth.to_numpy_bits(w.logits)
    u = np.random.default_rng(7).random((w.B, w.N)).astype(np.float32)
    u = np.clip(u, 1e-3, 1 - 1e-3).astype(np.float32)
    s = orc.verify_tree_stochastic(logits, w.tok, w.parent, u, 0.9, 1e-3, orc.STOCH_PLAIN)
    g = orc.verify_tree(logits, w.tok, w.parent, 1.5)
    for k in ("accept_len", "out_tokens", "path_nodes", "out_len"):
        assert np.array_equal(s[k], g[k]), k
    assert g["accept_len"].max() >= 2


def test_power_of_two_scaling_of_logits_and_temperature_changes_nothing():
    logits, tok, parent, u = _rand_case(8, 50, 12, 64)
    a = orc.verify_tree_stochastic(logits, tok, parent, u, 0.9, 0.7)
    b = orc.verify_tree_stochastic(logits * np.float32(4), tok, parent, u, 0.9, 2.8)
    for k in ("accept_len", "out_tokens", "path_nodes", "node_how"):
        assert np.array_equal(a[k], b[k]), k
    assert np.allclose(a["node_prob"], b["node_prob"], rtol=1e-12)


def test_structure_of_the_walk():
    """Whatever the mode: the path is a root-to-node chain of accepted nodes, every visited
    sibling before the accepted one is rejected, nothing after it is visited, a rejected
    token is never emitted as the correction, and a repeated sibling token is never accepted
    by Eq. 1."""
    logits, tok, parent, u = _rand_case(9, 300, 14, 12, depth=4, branch=4)
    tok[:, 5] = tok[:, 4]   # plant duplicates (siblings only where the tree makes them so)
    for flags in (0, orc.STOCH_PLAIN, orc.STOCH_RELAX_ONLY):
        out = orc.verify_tree_stochastic(logits, tok, parent, u, 0.9, 1.0, flags)
        B, N = tok.shape
        for b in range(B):
            a = out["accept_len"][b]
            path = out["path_nodes"][b, :a + 1]
            assert path[0] == 0 and out["out_len"][b] == a + 1
            for d in range(1, a + 1):
                c = path[d]
                assert parent[b, c] == path[d - 1] and out["node_how"][b, c] in (1, 2, 3)
                assert out["out_tokens"][b, d - 1] == tok[b, c]
            for d in range(a + 1):
                kids = [i for i in range(1, N) if parent[b, i] == path[d]]
                nxt = path[d + 1] if d < a else N
                rejected = []
                for i in kids:
                    h = out["node_how"][b, i]
                    if i < nxt:
                        assert h == 4
                        rejected.append(tok[b, i])
                    elif i > nxt:
                        assert h == 0
                if d == a:
                    assert out["out_tokens"][b, a] not in rejected
            off_path = set(range(N)) - set(path.tolist())
            for i in off_path:
                if parent[b, i] not in path.tolist():
                    assert out["node_how"][b, i] == 0
        assert out["accept_len"].max() >= 2


def test_duplicate_sibling_is_not_accepted_twice_by_eq1():
    V = 9
    rows = np.zeros((3, V), np.float32)
    rows[0, 4] = 3.0
    parent = np.array([-1, 0, 0], np.int32)
    tok = np.array([[-1, 4, 4]], np.int32)
    # first copy rejected (u above P), second copy has u = 0 and would pass any positive mass
    P4 = softmax(rows[0].astype(np.float64))[4]
    u = np.array([[0.5, np.float32(P4 + 0.01), 0.0]], np.float32)
    out = orc.verify_tree_stochastic(rows, tok, parent, u, 0.9, 1.0, orc.STOCH_PLAIN)
    assert out["node_how"][0].tolist() == [0, 4, 4] and out["accept_len"][0] == 0
    assert out["out_tokens"][0, 0] != 4


def test_removed_tokens_are_forgotten_at_the_next_level():
    """The residual belongs to one row: a token rejected among the root's children is an
    ordinary candidate again under the accepted child's row."""
    V = 5
    parent = np.array([-1, 0, 0, 2], np.int32)
    tok = np.array([[-1, 1, 2, 1]], np.int32)          # token 1: rejected at the root, offered again below node 2
    rows = np.zeros((4, V), np.float32)
    u = np.array([[0.99, 0.9, 0.0, 0.1]], np.float32)  # node 1 rejected (0.9 > 0.2), node 2 accepted, node 3: 0.1 < 0.2
    out = orc.verify_tree_stochastic(rows, tok, parent, u, 0.9, 1.0, orc.STOCH_PLAIN)
    assert out["node_how"][0].tolist() == [0, 4, 3, 3]
    assert out["accept_len"][0] == 2 and out["out_tokens"][0, :2].tolist() == [2, 1]
    # and with node 3 rejected the draw at node 2 excludes token 1 only, not the root's rejected token too
    tok[0, 3] = 4
    u[0, 3] = 0.9
    out = orc.verify_tree_stochastic(rows, tok, parent, u, 0.9, 1.0, orc.STOCH_PLAIN)
    assert out["accept_len"][0] == 1
    # residual at node 2: tokens {0,1,2,3} with weight 1/4 each; u = 0.99 falls on token 3
    assert out["out_tokens"][0, 1] == 3
    u[0, 0] = 0.3                                      # 0.3 * 4 = 1.2 -> second surviving token, which is token 1
    out = orc.verify_tree_stochastic(rows, tok, parent, u, 0.9, 1.0, orc.STOCH_PLAIN)
    assert out["out_tokens"][0, 1] == 1


def test_degenerate_rows_and_bad_trees():
    V = 8
    rows = np.zeros((2, V), np.float32)
    rows[0, :] = -np.inf
    parent = np.array([-1, 0], np.int32)
    tok = np.array([[-1, 3]], np.int32)
    u = np.array([[0.3, 0.3]], np.float32)
    out = orc.verify_tree_stochastic(rows, tok, parent, u, 0.9, 1.0)
    assert out["seq_status"][0] == 4 and out["accept_len"][0] == 0 and out["out_tokens"][0, 0] == 0
    rows[0, :] = 0.0
    rows[0, 2] = np.inf
    out = orc.verify_tree_stochastic(rows, tok, parent, u, 0.9, 1.0)
    assert out["seq_status"][0] == 4 and out["out_tokens"][0, 0] == 2
    rows[0, 2] = np.nan       # NaN counts as -inf: an ordinary row again
    out = orc.verify_tree_stochastic(rows, tok, parent, u, 0.9, 1.0)
    assert out["seq_status"][0] == 0
    bad = np.array([-1, 1], np.int32)
    out = orc.verify_tree_stochastic(rows, tok, bad, u, 0.9, 1.0)
    assert out["seq_status"][0] == 1 and out["accept_len"][0] == 0 and out["out_len"][0] == 1
    # path deeper than the outputs
    rows3 = np.zeros((3, V), np.float32)
    rows3[:, 1] = 30.0
    out = orc.verify_tree_stochastic(rows3, np.array([[-1, 1, 1]], np.int32), np.array([-1, 0, 1], np.int32),
                                     np.full((1, 3), 0.5, np.float32), 0.9, 1.0, Dcap=1)
    assert out["seq_status"][0] == 2 and out["accept_len"][0] == 0 and out["out_tokens"][0].tolist() == [1, -1]


def test_margins_report_how_close_each_decision_was():
    rows = np.zeros((2, 4), np.float32)          # uniform row: P = 1/4 each
    parent = np.array([-1, 0], np.int32)
    tok = np.array([[-1, 1]], np.int32)
    u = np.array([[0.6, 0.2]], np.float32)       # 0.2 < 0.25: accepted with margin 0.05
    out = orc.verify_tree_stochastic(rows, tok, parent, u, 0.9, 1.0, orc.STOCH_PLAIN)
    assert out["accept_len"][0] == 1
    assert out["margin"][0, 0] == pytest.approx(0.25 - float(np.float32(0.2)), abs=1e-12)
    # the draw at node 1 (a leaf, nothing removed): u = 0.6 falls in token 2's interval [0.5, 0.75)
    assert out["out_tokens"][0, 1] == 2
    assert out["margin"][0, 1] == pytest.approx(min(float(np.float32(0.6)) - 0.5, 0.75 - float(np.float32(0.6))), abs=1e-12)


# ---------------------------------------------------------------- sampled drafts (general Eq. 1)

def _sampled_case(seed, B, K, V, sigma_p=1.0, sigma_q=1.0, T=1.0, Tq=1.0, same_rows=True):
    """Target and drafter rows, drafts actually sampled from the drafter's softmax (numpy), and the
    probability with which each was drawn."""
    rng = np.random.default_rng(seed)
    if same_rows:
        rows_p = (rng.normal(size=(K, V)) * sigma_p).astype(np.float32)
        rows_q = (rows_p[:K - 1] + rng.normal(size=(K - 1, V)) * sigma_q).astype(np.float32)
        logits = np.ascontiguousarray(np.tile(rows_p, (B, 1)))
        qlogits = np.ascontiguousarray(np.tile(rows_q, (B, 1)))
    else:
        logits = (rng.normal(size=(B * K, V)) * sigma_p).astype(np.float32)
        qlogits = (logits.reshape(B, K, V)[:, :K - 1].reshape(-1, V)
                   + rng.normal(size=(B * (K - 1), V)) * sigma_q).astype(np.float32)
    Q = softmax(qlogits.astype(np.float64) / Tq, axis=1)
    cdf = np.cumsum(Q, axis=1)
    r = rng.random(B * (K - 1))
    draft = np.minimum((cdf < r[:, None]).sum(axis=1), V - 1).astype(np.int32)
    qx = Q[np.arange(B * (K - 1)), draft].astype(np.float32)
    u = rng.random((B, K)).astype(np.float32)
    return logits, qlogits, draft.reshape(B, K - 1), qx.reshape(B, K - 1), u


def test_sampled_drafts_plain_mode_preserves_the_target_distribution():
    """Speculative sampling (Eq. 1 + residual) with drafts really drawn from the drafter: the
    first emitted token follows the target's row 0 and, where draft 0 was accepted, the second
    follows row 1 -- whatever the drafter's distribution is."""
    V, K, B, T, Tq = 7, 3, 200_000, 0.9, 1.2
    logits, qlogits, draft, qx, u = _sampled_case(11, B, K, V, 0.8, 0.9, T, Tq)
    out = orc.verify_chain_sampled(logits, qlogits, draft, qx, u, 0.9, T, Tq, orc.STOCH_PLAIN)
    assert (out["seq_status"] == 0).all()
    P = softmax(logits[:K].astype(np.float64) / T, axis=1)
    _freq_close(out["out_tokens"][:, 0], P[0])
    acc0 = out["accept_len"] >= 1
    assert 0.2 < acc0.mean() < 0.95
    _freq_close(out["out_tokens"][acc0, 1], P[1])
    # acceptance rate of the first draft = sum_v min(P, Q)
    Q0 = softmax(qlogits[0].astype(np.float64) / Tq)
    want = np.minimum(P[0], Q0).sum()
    assert abs(acc0.mean() - want) < 4.5 * np.sqrt(want * (1 - want) / B)


def test_sampled_drafts_with_a_point_mass_drafter_equal_the_tree_form():
    """A drafter that puts all its mass on the draft (Q = one-hot, qx = 1) turns the general rule
    into the point-mass form: same decisions, same drawn tokens as the tree oracle on a chain."""
    rng = np.random.default_rng(12)
    B, K, V = 300, 5, 40
    logits = (rng.normal(size=(B * K, V)) * 1.5).astype(np.float32)
    draft = rng.integers(0, V, (B, K - 1)).astype(np.int32)
    best = logits.reshape(B, K, V)[:, :K - 1].argmax(axis=2).astype(np.int32)
    draft = np.where(rng.random((B, K - 1)) < 0.6, best, draft)     # most drafts aim at the target's top token
    qlogits = np.full((B * (K - 1), V), -1e4, np.float32)
    qlogits[np.arange(B * (K - 1)), draft.reshape(-1)] = 0.0
    qx = np.ones((B, K - 1), np.float32)
    u = rng.random((B, K)).astype(np.float32)
    tok = np.concatenate([np.full((B, 1), -1, np.int32), draft], axis=1)
    parent = synth.chain_parents(B, K)
    for flags in (0, orc.STOCH_PLAIN, orc.STOCH_RELAX_ONLY):
        a = orc.verify_chain_sampled(logits, qlogits, draft, qx, u, 0.9, 1.0, 1.0, flags)
        t = orc.verify_tree_stochastic(logits, tok, parent, u, 0.9, 1.0, flags)
        for k in ("accept_len", "out_tokens", "out_len", "node_how"):
            assert np.array_equal(a[k], t[k]), (flags, k)
        assert np.allclose(a["node_prob"], t["node_prob"], rtol=1e-12)
    assert a["accept_len"].min() == 0 and a["accept_len"].max() >= 2


def test_a_perfect_drafter_is_always_accepted():
    logits, qlogits, draft, qx, u = _sampled_case(13, 400, 4, 30, 1.5, 0.0, same_rows=False)
    out = orc.verify_chain_sampled(logits, qlogits, draft, qx, u, 0.9, 1.0, 1.0, orc.STOCH_PLAIN)
    assert (out["accept_len"] == 3).all() and (out["node_how"][:, 1:] == 3).all()


def test_residual_draw_of_the_general_form_against_numpy():
    V, K, B = 19, 2, 600
    logits, qlogits, draft, qx, u = _sampled_case(14, B, K, V, 1.2, 1.0, 1.1, 0.8, same_rows=False)
    u[:, 1] = np.float32(0.999999)          # reject (almost) every draft
    out = orc.verify_chain_sampled(logits, qlogits, draft, qx, u, 0.9, 1.1, 0.8, orc.STOCH_PLAIN)
    P = softmax(logits.astype(np.float64) / 1.1, axis=1)
    Q = softmax(qlogits.astype(np.float64) / 0.8, axis=1)
    n = 0
    for b in range(B):
        if out["accept_len"][b] != 0:
            continue
        w = np.maximum(P[b * K] - Q[b], 0.0)
        c = np.cumsum(w)
        want = int(np.searchsorted(c, float(u[b, 0]) * c[-1], side="right"))
        assert out["out_tokens"][b, 0] == want
        n += 1
    assert n > B // 2


def test_sampled_modes_are_nested():
    logits, qlogits, draft, qx, u = _sampled_case(15, 500, 6, 50, 2.0, 1.0, same_rows=False)
    a = orc.verify_chain_sampled(logits, qlogits, draft, qx, u, 0.9, 1.0, 1.0, orc.STOCH_PLAIN)["accept_len"]
    r = orc.verify_chain_sampled(logits, qlogits, draft, qx, u, 0.9, 1.0, 1.0, orc.STOCH_RELAX_ONLY)["accept_len"]
    d = orc.verify_chain_sampled(logits, qlogits, draft, qx, u, 0.9, 1.0, 1.0, 0)["accept_len"]
    assert (a <= r).all() and (r <= d).all() and a.sum() < d.sum()


def test_a_negative_draft_ends_the_chain_and_the_token_comes_from_the_target_row():
    """Reading: a negative draft id is padding -- there is no draft at that position, so nothing
    was rejected and no residual applies.  The accepted prefix ends there and the emitted token
    is a plain draw from the target's distribution of that row (numpy CDF inversion of
    softmax(row / T)), exactly as for the bonus token of a fully accepted chain.  The drafter's
    row at that position must not enter: the residual max(0, P - Q) would pick another token."""
    V, K, B, T, Tq = 23, 5, 400, 1.1, 0.7
    logits, qlogits, draft, qx, u = _sampled_case(16, B, K, V, 1.2, 1.5, T, Tq, same_rows=False)
    u[:, 1:] = np.float32(1e-7)             # every real draft passes Eq. 1 (P(x) > 1e-7 Q(x))
    rng = np.random.default_rng(160)
    cut = rng.integers(0, K - 1, B)         # position of the first padding draft
    for b in range(B):
        draft[b, cut[b]] = -1
    full = orc.verify_chain_sampled(logits, qlogits, draft, qx, u, 0.9, T, Tq, orc.STOCH_PLAIN)
    assert (full["seq_status"] == 0).all()
    assert np.array_equal(full["accept_len"], cut.astype(np.int32))
    assert np.array_equal(full["out_len"], cut.astype(np.int32) + 1)
    P = softmax(logits.astype(np.float64) / T, axis=1)
    Q = softmax(qlogits.astype(np.float64) / Tq, axis=1)
    differs = 0
    for b in range(B):
        i = int(cut[b])
        assert np.array_equal(full["out_tokens"][b, :i], draft[b, :i])
        assert (full["out_tokens"][b, i + 1:] == -1).all()
        assert full["node_how"][b, i + 1] == 0          # never judged
        c = np.cumsum(P[b * K + i])
        want = int(np.searchsorted(c, float(u[b, 0]) * c[-1], side="right"))
        assert full["out_tokens"][b, i] == want
        w = np.maximum(P[b * K + i] - Q[b * (K - 1) + i], 0.0)
        cr = np.cumsum(w)
        differs += int(np.searchsorted(cr, float(u[b, 0]) * cr[-1], side="right")) != want
    assert differs > B // 4                 # the residual would have given another answer
    # drafts behind the padding are never looked at
    other = draft.copy()
    for b in range(B):
        other[b, cut[b] + 1:] = (other[b, cut[b] + 1:] + 1) % V
    again = orc.verify_chain_sampled(logits, qlogits, other, qx, u, 0.9, T, Tq, orc.STOCH_PLAIN)
    for k in ("accept_len", "out_tokens", "out_len"):
        assert np.array_equal(full[k], again[k]), k
