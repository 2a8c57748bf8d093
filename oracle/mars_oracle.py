"""ctypes front end of the CPU oracle (TEST INFRASTRUCTURE, not a product path).

Builds ``mars_oracle.c`` with gcc on first use and exposes numpy-level calls for the
tests, the smoke check and the benchmark's CPU-baseline leg.  Nothing here imports, or
is imported by, the CUDA library or its Python binding.

Arrays: logits are numpy arrays of shape [R, ld] holding bf16 bit patterns
(``uint16``), ``float32`` or ``float64``; token / parent arrays are ``int32``.

The one piece of arithmetic done here rather than in C is the output projection
z = W_o h + b_o (Eq. 2 of the paper), evaluated as an fp64 numpy matmul.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mars_oracle.c")
_LIB = os.path.join(_HERE, "libmars_oracle.so")
_lock = threading.Lock()
_lib = None

SIGN_LITERAL = 1
SHARED_PARENT = 2
RULE_MARGIN = 8
RULE_PROB_RATIO = 16

_DT = {np.dtype(np.uint16): 0, np.dtype(np.float32): 1, np.dtype(np.float64): 2}


def build(force: bool = False) -> str:
    """Compile the oracle (no fast-math, no FMA contraction, OpenMP over rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["gcc", "-std=c11", "-O2", "-fno-fast-math", "-ffp-contract=off", "-fopenmp",
               "-shared", "-fPIC", "-Wall", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    with _lock:
        if _lib is None:
            build()
            L = ctypes.CDLL(_LIB)
            vp, i32, i64, u32, f64 = (ctypes.c_void_p, ctypes.c_int, ctypes.c_int64,
                                      ctypes.c_uint32, ctypes.c_double)
            L.mars_oracle_threads.restype = ctypes.c_int
            L.mars_oracle_set_threads.argtypes = [ctypes.c_int]
            L.mars_oracle_set_threads.restype = None
            L.mars_oracle_set_threads(usable_cores())
            L.mars_oracle_top2.argtypes = [vp, i32, i64, i64, i64, vp, vp]
            L.mars_oracle_top2.restype = None
            L.mars_oracle_relax_f32.argtypes = [ctypes.c_float, ctypes.c_float, ctypes.c_float, u32]
            L.mars_oracle_relax_f32.restype = ctypes.c_int
            L.mars_oracle_relax_f64.argtypes = [f64, f64, f64, u32]
            L.mars_oracle_relax_f64.restype = ctypes.c_int
            L.mars_oracle_verify_tree.argtypes = [vp, i32, i64, vp, vp, i32, i32, i64, f64, u32,
                                                  i32] + [vp] * 13
            L.mars_oracle_verify_tree.restype = None
            L.mars_oracle_verify_chain.argtypes = [vp, i32, i64, vp, i32, i32, i64, f64, u32] + [vp] * 7
            L.mars_oracle_verify_chain.restype = None
            L.mars_oracle_histograms.argtypes = [vp, i64, ctypes.c_float, ctypes.c_float, i32, vp, vp]
            L.mars_oracle_histograms.restype = None
            L.mars_oracle_topk.argtypes = [vp, i32, i64, i64, i64, i32, vp, vp]
            L.mars_oracle_topk.restype = None
            L.mars_oracle_verify_tree_stochastic.argtypes = [vp, i32, i64, vp, vp, vp, i32, i32, i64, f64,
                                                             f64, u32, i32] + [vp] * 8
            L.mars_oracle_verify_tree_stochastic.restype = None
            L.mars_oracle_verify_chain_sampled.argtypes = [vp, i32, i64, vp, i32, i64, vp, vp, vp, i32, i32, i64,
                                                           f64, f64, f64, u32] + [vp] * 7
            L.mars_oracle_verify_chain_sampled.restype = None
            _lib = L
    return _lib


def usable_cores() -> int:
    """Cores this process may really use: scheduler affinity, capped by the cgroup CPU quota.
    OpenMP's default (every core of the machine) oversubscribes a quota-limited container."""
    n = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    for path in ("/sys/fs/cgroup/cpu.max", "/sys/fs/cgroup/cpu/cpu.cfs_quota_us"):
        try:
            with open(path) as f:
                parts = f.read().split()
            if path.endswith("cpu.max"):
                if parts[0] != "max":
                    n = min(n, max(1, int(int(parts[0]) / int(parts[1]))))
            else:
                quota = int(parts[0])
                if quota > 0:
                    with open("/sys/fs/cgroup/cpu/cpu.cfs_period_us") as g:
                        n = min(n, max(1, int(quota / int(g.read()))))
            break
        except Exception:
            continue
    env = os.environ.get("OMP_NUM_THREADS")
    if env and env.isdigit() and int(env) >= 1:
        n = min(n, int(env))
    return max(1, min(n, 32))


def threads() -> int:
    """Host threads the row loop will use (OpenMP default)."""
    return int(lib().mars_oracle_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check_logits(logits, V):
    if logits.ndim != 2 or not logits.flags.c_contiguous or logits.dtype not in _DT:
        raise ValueError("logits must be a C-contiguous [R, ld] array of uint16/float32/float64")
    V = logits.shape[1] if V is None else int(V)
    if V < 2 or V > logits.shape[1]:
        raise ValueError("need 2 <= V <= ld")
    return _DT[logits.dtype], V


def top2(logits: np.ndarray, V: int | None = None):
    """Per-row top-2 (values [R,2], ids [R,2]) under (value desc, id asc), NaN = -inf."""
    dt, V = _check_logits(logits, V)
    R, ld = logits.shape
    val = np.empty((R, 2), np.float64 if dt == 2 else np.float32)
    idx = np.empty((R, 2), np.int32)
    lib().mars_oracle_top2(_p(logits), dt, ld, R, V, _p(val), _p(idx))
    return val, idx


def relax(z1, z2, theta, flags: int = 0, fp64: bool = False) -> bool:
    """Adaptive-relaxation bit for one row: sign guard and r = z2/z1 > theta."""
    if fp64:
        return bool(lib().mars_oracle_relax_f64(float(z1), float(z2), float(theta), flags))
    return bool(lib().mars_oracle_relax_f32(float(z1), float(z2), float(theta), flags))


def verify_tree(logits, tok, parent, theta, flags: int = 0, Dcap: int | None = None,
                V: int | None = None) -> dict:
    """Tree verification of B sequences of N nodes; see mars_oracle.c for the rule."""
    dt, V = _check_logits(logits, V)
    tok = np.ascontiguousarray(tok, np.int32)
    parent = np.ascontiguousarray(parent, np.int32)
    B, N = tok.shape
    if parent.ndim == 1:
        flags |= SHARED_PARENT
    elif flags & SHARED_PARENT:
        raise ValueError("SHARED_PARENT needs a 1-D parent array")
    if logits.shape[0] != B * N or parent.shape[-1] != N:
        raise ValueError("shape mismatch")
    if Dcap is None:
        Dcap = N - 1
    out = {
        "accept_len": np.empty(B, np.int32),
        "out_tokens": np.empty((B, Dcap + 1), np.int32),
        "path_nodes": np.empty((B, Dcap + 1), np.int32),
        "out_len": np.empty(B, np.int32),
        "seq_status": np.empty(B, np.int32),
        "top2_val": np.empty((B * N, 2), np.float64 if dt == 2 else np.float32),
        "top2_id": np.empty((B * N, 2), np.int32),
        "node_flags": np.empty((B, N), np.uint8),
    }
    val = np.empty((B * N, 2), np.float64)
    idb = np.empty((B * N, 2), np.int32)
    rl = np.empty(B * N, np.uint8)
    dp = np.empty(N, np.int32)
    ac = np.empty(N, np.uint8)
    lib().mars_oracle_verify_tree(_p(logits), dt, logits.shape[1], _p(tok), _p(parent), B, N, V,
                                  float(theta), flags, Dcap, _p(out["accept_len"]),
                                  _p(out["out_tokens"]), _p(out["path_nodes"]), _p(out["out_len"]),
                                  _p(out["seq_status"]), _p(out["top2_val"]), _p(out["top2_id"]),
                                  _p(out["node_flags"]), _p(val), _p(idb), _p(rl), _p(dp), _p(ac))
    return out


def verify_chain(logits, draft, theta, flags: int = 0, V: int | None = None) -> dict:
    """Chain verification (Algorithm 1 plus the bonus token): K rows, K-1 drafts."""
    dt, V = _check_logits(logits, V)
    draft = np.ascontiguousarray(draft, np.int32)
    B, Km1 = draft.shape
    K = Km1 + 1
    if logits.shape[0] != B * K:
        raise ValueError("shape mismatch")
    out = {
        "accept_len": np.empty(B, np.int32),
        "out_tokens": np.empty((B, K), np.int32),
        "out_len": np.empty(B, np.int32),
        "top2_val": np.empty((B * K, 2), np.float64 if dt == 2 else np.float32),
        "top2_id": np.empty((B * K, 2), np.int32),
    }
    val = np.empty((B * K, 2), np.float64)
    idb = np.empty((B * K, 2), np.int32)
    lib().mars_oracle_verify_chain(_p(logits), dt, logits.shape[1], _p(draft), B, K, V,
                                   float(theta), flags, _p(out["accept_len"]),
                                   _p(out["out_tokens"]), _p(out["out_len"]), _p(out["top2_val"]),
                                   _p(out["top2_id"]), _p(val), _p(idb))
    return out


def bf16_bits_to_f64(a: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float64."""
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def lmhead_logits(hidden_bits: np.ndarray, w_bits: np.ndarray, bias=None) -> np.ndarray:
    """z = W_o h + b_o (Eq. 2) in fp64 from bf16 operands: hidden [M,d], w [V,d] -> [M,V]."""
    z = bf16_bits_to_f64(hidden_bits) @ bf16_bits_to_f64(w_bits).T
    if bias is not None:
        z = z + np.asarray(bias, np.float64)[None, :]
    return np.ascontiguousarray(z)


def lmhead_verify_tree(hidden_bits, w_bits, bias, tok, parent, theta, flags: int = 0,
                       Dcap: int | None = None) -> dict:
    """Output projection in fp64 followed by the tree rule taken in fp64."""
    z = lmhead_logits(hidden_bits, w_bits, bias)
    out = verify_tree(z, tok, parent, float(np.float32(theta)), flags, Dcap)
    out["logits"] = z
    return out


def histograms(top2_val: np.ndarray, lo: float, hi: float, nbins: int):
    """Histograms of z1, z2/z1 and p2/p1 from [rows, 2] fp32 top-2 values; see mars_oracle.c."""
    v = np.ascontiguousarray(top2_val, np.float32)
    hist = np.zeros((3, nbins), np.uint32)
    outl = np.zeros(3, np.uint32)
    lib().mars_oracle_histograms(_p(v), v.shape[0], float(lo), float(hi), int(nbins), _p(hist), _p(outl))
    return hist, outl


def topk(logits: np.ndarray, k: int, V: int | None = None):
    """Exact top-k per row (values [R,k], ids [R,k], best first) under the library's total order."""
    if logits.ndim != 2 or not logits.flags.c_contiguous or logits.dtype not in _DT:
        raise ValueError("logits must be a C-contiguous [R, ld] array of uint16/float32/float64")
    dt = _DT[logits.dtype]
    V = logits.shape[1] if V is None else int(V)
    if not (1 <= k <= 64 and k <= V <= logits.shape[1]):
        raise ValueError("need 1 <= k <= min(64, V) and V <= ld")
    R, ld = logits.shape
    val = np.empty((R, k), np.float64 if dt == 2 else np.float32)
    idx = np.empty((R, k), np.int32)
    lib().mars_oracle_topk(_p(logits), dt, ld, R, V, int(k), _p(val), _p(idx))
    return val, idx


STOCH_PLAIN = 32
STOCH_RELAX_ONLY = 64


def verify_tree_stochastic(logits, tok, parent, uniform, theta, temperature, flags: int = 0,
                           Dcap: int | None = None, V: int | None = None) -> dict:
    """Stochastic (T > 0) tree verification; see the block comment in mars_oracle.c.
    ``uniform`` is float32 [B, N]: [b, i>0] judges node i, [b, 0] draws the final token."""
    dt, V = _check_logits(logits, V)
    tok = np.ascontiguousarray(tok, np.int32)
    parent = np.ascontiguousarray(parent, np.int32)
    uniform = np.ascontiguousarray(uniform, np.float32)
    B, N = tok.shape
    if parent.ndim == 1:
        flags |= SHARED_PARENT
    if logits.shape[0] != B * N or parent.shape[-1] != N or uniform.shape != (B, N):
        raise ValueError("shape mismatch")
    if not (temperature > 0 and np.isfinite(temperature)):
        raise ValueError("temperature must be positive and finite")
    if N > 1024:
        raise ValueError("N <= 1024")
    if Dcap is None:
        Dcap = N - 1
    out = {
        "accept_len": np.empty(B, np.int32),
        "out_tokens": np.empty((B, Dcap + 1), np.int32),
        "path_nodes": np.empty((B, Dcap + 1), np.int32),
        "out_len": np.empty(B, np.int32),
        "seq_status": np.empty(B, np.int32),
        "node_prob": np.empty((B, N), np.float64),
        "node_how": np.empty((B, N), np.uint8),
        "margin": np.empty((B, 2), np.float64),
    }
    L = lib()
    L.mars_oracle_verify_tree_stochastic(
        _p(logits), dt, logits.shape[1], _p(tok), _p(parent), _p(uniform), B, N, V, float(theta),
        float(temperature), flags, Dcap, _p(out["accept_len"]), _p(out["out_tokens"]),
        _p(out["path_nodes"]), _p(out["out_len"]), _p(out["seq_status"]), _p(out["node_prob"]),
        _p(out["node_how"]), _p(out["margin"]))
    return out


def verify_chain_sampled(logits, qlogits, draft, qx, uniform, theta, temperature, draft_temperature,
                         flags: int = 0, V: int | None = None) -> dict:
    """Stochastic verification of chains with sampled drafts (general Eq. 1); see mars_oracle.c.
    logits [B*K, ld], qlogits [B*(K-1), ldq], draft / qx [B, K-1], uniform [B, K]."""
    dt, V = _check_logits(logits, V)
    draft = np.ascontiguousarray(draft, np.int32)
    qx = np.ascontiguousarray(qx, np.float32)
    uniform = np.ascontiguousarray(uniform, np.float32)
    B, Km1 = draft.shape
    K = Km1 + 1
    if qlogits.ndim != 2 or not qlogits.flags.c_contiguous or qlogits.dtype not in _DT or qlogits.shape[1] < V:
        raise ValueError("qlogits must be a C-contiguous [B*(K-1), >=V] array")
    if logits.shape[0] != B * K or qlogits.shape[0] != B * Km1 or qx.shape != (B, Km1) or uniform.shape != (B, K):
        raise ValueError("shape mismatch")
    if not (temperature > 0 and draft_temperature > 0):
        raise ValueError("temperatures must be positive")
    out = {
        "accept_len": np.empty(B, np.int32),
        "out_tokens": np.empty((B, K), np.int32),
        "out_len": np.empty(B, np.int32),
        "seq_status": np.empty(B, np.int32),
        "node_prob": np.empty((B, K), np.float64),
        "node_how": np.empty((B, K), np.uint8),
        "margin": np.empty((B, 2), np.float64),
    }
    lib().mars_oracle_verify_chain_sampled(
        _p(logits), dt, logits.shape[1], _p(qlogits), _DT[qlogits.dtype], qlogits.shape[1], _p(draft), _p(qx),
        _p(uniform), B, K, V, float(theta), float(temperature), float(draft_temperature), flags,
        _p(out["accept_len"]), _p(out["out_tokens"]), _p(out["out_len"]), _p(out["seq_status"]),
        _p(out["node_prob"]), _p(out["node_how"]), _p(out["margin"]))
    return out
