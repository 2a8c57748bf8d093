"""Seeded synthetic verification workloads.

Input construction only: this module holds none of the verification arithmetic and is
the one module that the CPU oracle's tests and the CUDA library's tests both use.  It
produces logits rows, draft tokens and token trees with the shapes and value
distributions of speculative-decoding verification on Vicuna-class (|V| = 32 000) and
Qwen3-class (|V| = 151 936) targets: positive top-1 logits, a visible fraction of
low-margin rows whose top-2 logit ratio lies in [0.85, 1), chains of K rows and
EAGLE-style trees of 60 nodes and depth 6.

Logits are drawn with a torch generator on the requested device (so the large
workloads can be built directly in device memory) and the small integer inputs with
numpy's Philox generator.  Everything is a pure function of (seed, device type).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

V_VICUNA = 32000
V_QWEN3 = 151936


@dataclass
class Workload:
    name: str
    kind: str                 # "chain" | "tree"
    B: int
    N: int                    # rows per sequence (chain: K rows = K-1 drafts + bonus row)
    V: int
    theta: float
    logits: torch.Tensor      # [B*N, ld], bf16 or fp32
    tok: np.ndarray           # int32 [B, N]; tok[:, 0] is unused
    parent: np.ndarray        # int32 [B, N]; parent[:, 0] = -1
    max_depth: int
    meta: dict = field(default_factory=dict)

    @property
    def R(self) -> int:
        return self.B * self.N

    @property
    def draft(self) -> np.ndarray:
        """Chain view of the draft tokens: [B, N-1]."""
        return np.ascontiguousarray(self.tok[:, 1:])

    @property
    def logits_bytes(self) -> int:
        return self.R * self.V * self.logits.element_size()


def make_parents(B: int, N: int, max_depth: int, max_children: int, seed: int) -> np.ndarray:
    """Random token trees in topological order (parent[i] < i, parent[0] = -1).

    The first ``max_depth`` nodes after the root form a spine so that every tree reaches
    the stated depth; the remaining nodes attach to a uniformly chosen earlier node that
    still has room (depth < max_depth, fewer than ``max_children`` children).
    """
    rng = np.random.Generator(np.random.Philox(key=[seed, 0x7EE5]))
    parent = np.full((B, N), -1, np.int32)
    for b in range(B):
        depth = np.zeros(N, np.int32)
        kids = np.zeros(N, np.int32)
        for i in range(1, N):
            if i <= max_depth:
                p = i - 1
            else:
                ok = np.flatnonzero((depth[:i] < max_depth) & (kids[:i] < max_children))
                p = int(ok[rng.integers(len(ok))]) if len(ok) else i - 1
            parent[b, i] = p
            depth[i] = depth[p] + 1
            kids[p] += 1
    return parent


def chain_parents(B: int, K: int) -> np.ndarray:
    par = np.tile(np.arange(-1, K - 1, dtype=np.int32), (B, 1))
    return np.ascontiguousarray(par)


def make_logits(R: int, V: int, dtype: torch.dtype, device, seed: int, sigma: float,
                z1_lo: float, z1_hi: float, p_low_margin: float, rho_lo: float = 0.85,
                rho_hi: float = 1.0, ld: int | None = None, pad_value: float | None = None,
                chunk_rows: int = 512):
    """Rows of N(0, sigma^2) noise with a planted top logit and, in a fraction of the rows,
    a planted runner-up at ratio rho.  Returns (logits [R, ld], lead [R, 2] int64 on CPU):
    ``lead`` holds the ids of the two largest entries of each finished row as found by
    ``torch.topk`` -- used only to aim draft tokens at them.
    """
    ld = V if ld is None else ld
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(0x5EED0000 + seed)
    out = torch.empty((R, ld), dtype=dtype, device=dev)
    if ld > V:
        out[:, V:] = 0.0 if pad_value is None else pad_value
    lead = torch.empty((R, 2), dtype=torch.int64)
    for r0 in range(0, R, chunk_rows):
        n = min(chunk_rows, R - r0)
        z = torch.randn((n, V), generator=g, device=dev, dtype=torch.float32) * sigma
        u = torch.rand((n, 4), generator=g, device=dev, dtype=torch.float32)
        ids = torch.randint(0, V, (n, 2), generator=g, device=dev)
        ids[:, 1] = torch.where(ids[:, 1] == ids[:, 0], (ids[:, 1] + 1) % V, ids[:, 1])
        z1 = z1_lo + (z1_hi - z1_lo) * u[:, 0]
        rho = rho_lo + (rho_hi - rho_lo) * u[:, 1]
        rows = torch.arange(n, device=dev)
        z[rows, ids[:, 0]] = z1
        low = u[:, 2] < p_low_margin
        z[rows[low], ids[low, 1]] = (rho * z1)[low]
        zc = z.to(dtype)
        out[r0:r0 + n, :V] = zc
        lead[r0:r0 + n] = torch.topk(zc.float(), 2, dim=1).indices.cpu()
    return out, lead


def _draft_mix(rng, lead_row, V: int, p_top1: float, p_top2: float) -> int:
    u = rng.random()
    if u < p_top1:
        return int(lead_row[0])
    if u < p_top1 + p_top2:
        return int(lead_row[1])
    return int(rng.integers(V))


def make_tokens(parent: np.ndarray, lead: np.ndarray, V: int, seed: int, p_top1: float = 0.6,
                p_top2: float = 0.25, dedupe_siblings: bool = True) -> np.ndarray:
    """Draft token per node, aimed at the parent row's leading ids: top-1 with
    probability p_top1, runner-up with p_top2, otherwise a uniform id.  Repeated tokens
    among siblings are redrawn uniformly, as in a top-k expansion."""
    rng = np.random.Generator(np.random.Philox(key=[seed, 0xD4AF7]))
    B, N = parent.shape
    tok = np.full((B, N), -1, np.int32)
    lead = np.asarray(lead).reshape(B, N, 2)
    for b in range(B):
        seen: dict[int, set] = {}
        for i in range(1, N):
            p = int(parent[b, i])
            t = _draft_mix(rng, lead[b, p], V, p_top1, p_top2)
            if dedupe_siblings:
                s = seen.setdefault(p, set())
                tries = 0
                while t in s and len(s) < V and tries < 64:   # tiny vocabularies may not allow it
                    t = int(rng.integers(V))
                    tries += 1
                s.add(t)
            tok[b, i] = t
    return tok


def chain_workload(name: str, B: int, K: int, V: int, dtype, device, seed: int, theta: float,
                   sigma: float, z1_lo: float, z1_hi: float, p_low: float, **kw) -> Workload:
    parent = chain_parents(B, K)
    logits, lead = make_logits(B * K, V, dtype, device, seed, sigma, z1_lo, z1_hi, p_low, **kw)
    tok = make_tokens(parent, lead.numpy(), V, seed, dedupe_siblings=False)
    return Workload(name, "chain", B, K, V, theta, logits, tok, parent, K - 1,
                    {"seed": seed, "sigma": sigma, "z1": [z1_lo, z1_hi], "p_low_margin": p_low})


def tree_workload(name: str, B: int, N: int, depth: int, branch: int, V: int, dtype, device,
                  seed: int, theta: float, sigma: float, z1_lo: float, z1_hi: float,
                  p_low: float, **kw) -> Workload:
    parent = make_parents(B, N, depth, branch, seed)
    logits, lead = make_logits(B * N, V, dtype, device, seed, sigma, z1_lo, z1_hi, p_low, **kw)
    tok = make_tokens(parent, lead.numpy(), V, seed)
    return Workload(name, "tree", B, N, V, theta, logits, tok, parent, depth,
                    {"seed": seed, "sigma": sigma, "z1": [z1_lo, z1_hi], "p_low_margin": p_low,
                     "branch": branch})


# ---- the named workloads -------------------------------------------------------------

def cfg0(device="cpu", seed: int = 0, B: int = 1) -> Workload:
    """Chain, 6 rows (5 drafts + bonus row), |V| = 32 000, fp32 N(0, 2^2), top logit +20,
    40 % of rows with a planted runner-up at ratio U[0.85, 1)."""
    return chain_workload("cfg0_chain_b1_k6_v32000_fp32", B, 6, V_VICUNA, torch.float32, device,
                          seed, 0.9, 2.0, 20.0, 20.0, 0.4)


def cfg1(device="cpu", seed: int = 1, B: int = 1, dtype=torch.bfloat16) -> Workload:
    """One 60-node depth-6 tree (branching <= 4), |V| = 151 936, bf16 N(0, 3^2), top logit
    U[15, 30], 30 % low-margin rows."""
    return tree_workload("cfg1_tree_b1_n60_v151936_bf16", B, 60, 6, 4, V_QWEN3, dtype, device,
                         seed, 0.9, 3.0, 15.0, 30.0, 0.3)


def cfg2(device="cpu", seed: int = 2, B: int = 64, theta: float = 0.9) -> Workload:
    """Batched chains: B = 64, 8 rows (7 drafts + bonus row), cfg1's distribution."""
    return chain_workload("cfg2_chain_b64_k8_v151936_bf16", B, 8, V_QWEN3, torch.bfloat16, device,
                          seed, theta, 3.0, 15.0, 30.0, 0.3)


def cfg3(device="cpu", seed: int = 3, B: int = 256, dtype=torch.bfloat16) -> Workload:
    """Serving scale: B = 256 sequences x 60-node depth-6 trees (15 360 rows), |V| = 151 936;
    the fp32 variant holds the same draws without bf16 rounding."""
    tag = "bf16" if dtype == torch.bfloat16 else "fp32"
    return tree_workload(f"cfg3_tree_b{B}_n60_v151936_{tag}", B, 60, 6, 4, V_QWEN3, dtype, device,
                         seed, 0.9, 3.0, 15.0, 30.0, 0.3)


@dataclass
class LmHeadWorkload:
    name: str
    B: int
    N: int
    V: int
    d: int
    theta: float
    hidden: torch.Tensor      # bf16 [B*N, d]
    w_vocab: torch.Tensor     # bf16 [V, d]
    parent: np.ndarray
    max_depth: int


def cfg4_operands(device="cpu", seed: int = 4, B: int = 64, N: int = 60, V: int = V_QWEN3,
                  d: int = 4096, depth: int = 6, branch: int = 4) -> LmHeadWorkload:
    """LM-head operands: hidden N(0,1) bf16 [B*N, d], W_vocab N(0, 0.02^2) bf16 [V, d].
    Draft tokens depend on the projected logits' leading ids, which the caller supplies
    to ``make_tokens`` (they are inputs to verification, not part of it)."""
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(0x5EED0000 + seed)
    hidden = torch.randn((B * N, d), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    w = torch.empty((V, d), dtype=torch.bfloat16, device=dev)
    step = 8192
    for v0 in range(0, V, step):
        n = min(step, V - v0)
        w[v0:v0 + n] = (torch.randn((n, d), generator=g, device=dev, dtype=torch.float32) * 0.02
                        ).to(torch.bfloat16)
    parent = make_parents(B, N, min(depth, N - 1), branch, seed)
    return LmHeadWorkload(f"cfg4_lmhead_b{B}_n{N}_v{V}_d{d}", B, N, V, d, 0.9, hidden, w, parent,
                          min(depth, N - 1))


def to_numpy_bits(t: torch.Tensor) -> np.ndarray:
    """Host copy of a tensor as the oracle wants it: bf16 -> uint16 bit patterns."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def make_uniforms(B: int, N: int, seed: int) -> np.ndarray:
    """float32 uniforms in [0, 1) for stochastic verification: [b, i > 0] judges node i,
    [b, 0] draws the next token.  They are inputs of the method, drawn here so that the oracle
    and the library consume the same numbers."""
    rng = np.random.Generator(np.random.Philox(key=[seed, 0x0A11CE]))
    u = rng.random((B, N), dtype=np.float32)
    return np.minimum(u, np.float32(1.0) - np.float32(2.0 ** -24))
