"""Comparison policy and case builders shared by the GPU tests of stochastic verification (not a
test module).

The oracle evaluates the softmax in fp64, the library in fp32 with the hardware 2^x; the
uniforms are inputs shared by both.  Bar:
  * top-2 based decisions (exact match, relaxed runner-up) are bit-exact as everywhere else;
  * node probabilities agree within PROB_RTOL;
  * a sequence whose every Eq. 1 test was decided by more than DECISION_TOL (of the row's total
    mass; the oracle reports the smallest such margin) must have the same walk: accepted length,
    path, per-node decisions, accepted tokens; closer ones may differ, are counted, bounded,
    and must still be valid walks;
  * where the walk is the same the drawn token must be the oracle's, or else u*W must lie within
    DRAW_TOL * W of the fp64 CDF interval of the token the library drew (a neighbouring step).
Where the tolerances come from: an fp32 weight 2^(z*c - ref) carries the rounding of its
exponent (|z*c - ref| up to about 2^6 where it matters, so about 2^-18 * ln 2 absolute, 3e-6
relative) and 2 ulp of the approximation; the denominator is an fp32 sum of up to 151 936 such
terms in a tree of partial sums (about 1e-6 relative); the draw accumulates in fp64, so its
position error is that of the weights.  DECISION_TOL = 2e-5 and DRAW_TOL = 1e-5 leave a margin
of several times over these and flag only a few decisions in 10^5.
"""
import os

import numpy as np
import torch

from paper_2601_15498_b200 import mars, synth

DEV = os.environ.get("MARS_TEST_DEVICE", "cuda:0")
PROB_RTOL = 2e-5
DECISION_TOL = 2e-5
DRAW_TOL = 1e-5
WALK_KEYS = ("accept_len", "path_nodes", "out_len", "seq_status", "node_how")
STATS = {"close": 0, "draw_neighbour": 0, "sequences": 0, "max_draw_dist": 0.0}


def check_walk_is_valid(got, tok, parent, b):
    a = int(got["accept_len"][b])
    path = got["path_nodes"][b, :a + 1]
    assert path[0] == 0 and got["out_len"][b] == a + 1
    par = parent if parent.ndim == 1 else parent[b]
    for d in range(1, a + 1):
        c = int(path[d])
        assert par[c] == path[d - 1] and got["node_how"][b, c] in (1, 2, 3)
        assert got["out_tokens"][b, d - 1] == tok[b, c]
    assert got["out_tokens"][b, a] >= 0


def draw_distance(row_f64, T, removed, u0, token):
    """Distance (in units of the residual mass W) of u0*W from the CDF interval of `token`."""
    w = np.exp((row_f64 - np.max(row_f64[np.isfinite(row_f64)])) / T)
    w[np.isnan(w)] = 0.0
    w[list(removed)] = 0.0
    c = np.cumsum(w)
    W = c[-1]
    lo, hi = (c[token - 1] if token > 0 else 0.0), c[token]
    t = float(u0) * W
    if w[token] <= 0.0:
        return np.inf
    return max(lo - t, t - hi, 0.0) / W


def compare(got, ref, tok, parent, logits_host, u, T, what="", max_close_frac=0.02):
    """logits_host: float64 [R, V] view of the rows (exact widening)."""
    B, N = tok.shape
    n_close = n_neigh = 0
    for b in range(B):
        par = parent if parent.ndim == 1 else parent[b]
        a = int(ref["accept_len"][b])
        same_walk = all(np.array_equal(got[k][b], ref[k][b]) for k in WALK_KEYS) and \
            np.array_equal(got["out_tokens"][b, :a], ref["out_tokens"][b, :a])
        if not same_walk:
            if ref["margin"][b, 0] < DECISION_TOL:
                n_close += 1
                if got["seq_status"][b] == 0:
                    check_walk_is_valid(got, tok, parent, b)
                continue
            diff = {k: (got[k][b].tolist(), ref[k][b].tolist()) for k in WALK_KEYS + ("out_tokens",)
                    if not np.array_equal(got[k][b], ref[k][b])}
            raise AssertionError(f"{what}: sequence {b} differs (margins {ref['margin'][b]}): {diff}")
        g, r = int(got["out_tokens"][b, a]), int(ref["out_tokens"][b, a])
        assert (got["out_tokens"][b, a + 1:] == -1).all()
        if g != r:
            assert ref["seq_status"][b] == 0, (what, b)
            cur = int(ref["path_nodes"][b, a])
            removed = {int(tok[b, i]) for i in range(1, N) if par[i] == cur and ref["node_how"][b, i] == 4
                       and 0 <= tok[b, i] < logits_host.shape[1]}
            d = draw_distance(logits_host[b * N + cur], T, removed, u[b, 0], g)
            STATS["max_draw_dist"] = max(STATS["max_draw_dist"], float(d))
            assert d <= DRAW_TOL, (what, b, g, r, d)
            n_neigh += 1
    ok = ref["seq_status"] != 1
    np.testing.assert_allclose(got["node_prob"][ok], ref["node_prob"][ok], rtol=PROB_RTOL, atol=1e-30,
                               err_msg=what)
    STATS["close"] += n_close
    STATS["draw_neighbour"] += n_neigh
    STATS["sequences"] += B
    assert n_close <= max(2, int(max_close_frac * B)), (what, n_close, B)
    assert n_neigh <= max(2, int(0.1 * B)), (what, n_neigh, B)
    return n_close, n_neigh


def host_f64(logits, V=None):
    x = logits.detach().float().cpu().numpy().astype(np.float64)
    return x if V is None else x[:, :V]




# ---- sampled chains and the vocabulary-sharded form: shared case builders and checks ----

def sampled_case(seed, B, K, V, dtype, sigma_q=1.0, T=1.0, Tq=1.0, ld_pad=0):
    """Target rows from the chain recipe, drafter rows = target rows + noise, drafts really drawn
    from the drafter's softmax (torch, on the host) with their probabilities."""
    w = synth.chain_workload("t", B, K, V, dtype, DEV, seed, 0.9, 1.5, 6.0, 10.0, 0.4)
    g = torch.Generator().manual_seed(seed)
    z = w.logits.float().cpu().reshape(B, K, V)[:, :K - 1].reshape(-1, V)
    zq = (z + torch.randn(z.shape, generator=g) * sigma_q).to(dtype)
    Q = torch.softmax(zq.double() / Tq, dim=1)
    draft = torch.multinomial(Q, 1, generator=g).reshape(-1)
    qx = Q[torch.arange(Q.shape[0]), draft].float()
    qdev = torch.full((B * (K - 1), V + ld_pad), 55.0, dtype=dtype, device=DEV)
    qdev[:, :V] = zq.to(DEV)
    u = synth.make_uniforms(B, K, seed)
    return w, qdev, zq, draft.reshape(B, K - 1).numpy().astype(np.int32), qx.reshape(B, K - 1).numpy(), u


def compare_sampled(got, ref, what):
    B = ref["accept_len"].shape[0]
    n_close = 0
    for b in range(B):
        a = int(ref["accept_len"][b])
        same_walk = all(np.array_equal(got[k][b], ref[k][b]) for k in ("accept_len", "out_len", "seq_status", "node_how")) \
            and np.array_equal(got["out_tokens"][b, :a], ref["out_tokens"][b, :a])
        if not same_walk:
            assert ref["margin"][b, 0] < DECISION_TOL, (what, b, ref["margin"][b])
            n_close += 1
            continue
        if got["out_tokens"][b, a] != ref["out_tokens"][b, a]:
            # the draw margin of this oracle is in units of total probability
            assert ref["margin"][b, 1] < 2e-6, (what, b, got["out_tokens"][b], ref["out_tokens"][b], ref["margin"][b])
            n_close += 1
    np.testing.assert_allclose(got["node_prob"], ref["node_prob"], rtol=PROB_RTOL, atol=1e-30, err_msg=what)
    assert n_close <= max(2, B // 50), (what, n_close)


def sharded_stochastic(logits, tok, parent, u, theta, T, ranges, flags=0):
    """The ranks' calls made one after the other on one GPU, stacked as the all-gathers would
    deliver them; returns every rank's final outputs."""
    G = len(ranges)
    recs, zls = [], []
    for lo, hi in ranges:
        r, z = mars.stochastic_shard_records(logits[:, lo:hi], tok, parent, lo, T, V_local=hi - lo)
        recs.append(r)
        zls.append(z)
    rec_all, zl_all = torch.stack(recs), torch.stack(zls)
    outs, parts = [], []
    for g, (lo, hi) in enumerate(ranges):
        o, part = mars.stochastic_shard_verify(logits[:, lo:hi], rec_all, zl_all, g, lo, tok, parent, u, theta, T,
                                               flags, V_local=hi - lo, debug=True)
        outs.append(o)
        parts.append(part)
    token_all = torch.stack(parts)
    return [mars.to_host(mars.stochastic_shard_finish(token_all, o)) for o in outs], token_all.cpu().numpy()
