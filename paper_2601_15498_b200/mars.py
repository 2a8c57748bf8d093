"""ctypes binding of libmars (argument marshalling only).

Every step of verification runs inside the CUDA library; this module turns torch CUDA
tensors into device pointers, provides the workspace and the current stream, and checks
the returned status.  There is no CPU path: a missing library or a failed call raises.
"""
from __future__ import annotations

import ctypes
import os
import threading

import torch

from . import build as _build

BF16, FP32 = 0, 1
SIGN_LITERAL, SHARED_PARENT, COUNTERS_ZERO, RULE_MARGIN, RULE_PROB_RATIO = 1, 2, 4, 8, 16
STOCH_PLAIN, STOCH_RELAX_ONLY = 32, 64
LOGITS_READY = 128
MAX_NODES = 1024

_lock = threading.Lock()
_lib = None


class MarsError(RuntimeError):
    pass


class _DebugOut(ctypes.Structure):
    _fields_ = [("top2_val", ctypes.c_void_p), ("top2_id", ctypes.c_void_p),
                ("node_flags", ctypes.c_void_p)]


def lib() -> ctypes.CDLL:
    """Open libmars.so (built in-tree by ``build.build()``); raises if it is missing."""
    global _lib
    with _lock:
        if _lib is None:
            path = _build.LIB
            if not os.path.exists(path):
                raise MarsError(f"{path} not found: run paper_2601_15498_b200.build.build() "
                                "(nvcc, sm_100a); there is no fallback path")
            L = ctypes.CDLL(path)
            vp, i32, i64, u32, f32, sz = (ctypes.c_void_p, ctypes.c_int, ctypes.c_int64,
                                          ctypes.c_uint32, ctypes.c_float, ctypes.c_size_t)
            L.mars_workspace_bytes.argtypes = [i32, i32, i32, i32]
            L.mars_workspace_bytes.restype = sz
            L.mars_verify_chain.argtypes = [vp, i64, i32, vp, i32, i32, i32, f32, u32, vp, vp, vp,
                                            vp, ctypes.POINTER(_DebugOut), vp, sz, vp]
            L.mars_verify_chain.restype = i32
            L.mars_verify_tree.argtypes = [vp, i64, i32, vp, vp, i32, i32, i32, f32, u32, vp, vp,
                                           vp, vp, i32, vp, ctypes.POINTER(_DebugOut), vp, sz, vp]
            L.mars_verify_tree.restype = i32
            L.mars_lmhead_workspace_bytes.argtypes = [i32, i32, i32, i32]
            L.mars_lmhead_workspace_bytes.restype = sz
            L.mars_lmhead_verify.argtypes = [vp, vp, vp, i32, vp, vp, i32, i32, i32, f32, u32, vp, vp,
                                             vp, vp, i32, vp, ctypes.POINTER(_DebugOut), vp, sz, vp]
            L.mars_lmhead_verify.restype = i32
            L.mars_verify_tree_static.argtypes = [vp, i64, i32, vp, vp, i32, i32, i32, f32, u32, vp,
                                                  vp, vp, vp, i32, vp, ctypes.POINTER(_DebugOut), vp]
            L.mars_verify_tree_static.restype = i32
            L.mars_static_scratch_bytes.argtypes = []
            L.mars_static_scratch_bytes.restype = sz
            L.mars_top2_shard.argtypes = [vp, i64, i32, i32, i32, i32, i32, vp, u32, vp, sz, vp]
            L.mars_top2_shard.restype = i32
            L.mars_verify_records.argtypes = [vp, i32, vp, vp, i32, i32, f32, u32, vp, vp, vp, vp, i32,
                                              vp, ctypes.POINTER(_DebugOut), vp]
            L.mars_verify_records.restype = i32
            L.mars_selftest_bounded_wait.argtypes = [i64, vp, vp]
            L.mars_selftest_bounded_wait.restype = i32
            L.mars_top2_histograms.argtypes = [vp, i64, f32, f32, i32, vp, vp, vp]
            L.mars_top2_histograms.restype = i32
            L.mars_topk_workspace_bytes.argtypes = [i64, i32, i32, i32]
            L.mars_topk_workspace_bytes.restype = sz
            L.mars_topk_rows.argtypes = [vp, i64, i32, i64, i32, i32, vp, vp, vp, sz, vp]
            L.mars_topk_rows.restype = i32
            L.mars_lmhead_top2_shard.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp, vp, sz, vp]
            L.mars_lmhead_top2_shard.restype = i32
            L.mars_stochastic_workspace_bytes.argtypes = [i32, i32, i32, i32]
            L.mars_stochastic_workspace_bytes.restype = sz
            L.mars_verify_tree_stochastic.argtypes = [vp, i64, i32, vp, vp, vp, i32, i32, i32, f32, f32, u32,
                                                      vp, vp, vp, vp, i32, vp, vp, vp, vp, sz, vp]
            L.mars_verify_tree_stochastic.restype = i32
            L.mars_verify_chain_stochastic.argtypes = [vp, i64, i32, vp, vp, i32, i32, i32, f32, f32, u32,
                                                       vp, vp, vp, vp, vp, vp, vp, sz, vp]
            L.mars_verify_chain_stochastic.restype = i32
            L.mars_verify_chain_sampled.argtypes = [vp, i64, i32, vp, i64, vp, vp, vp, i32, i32, i32, f32, f32, f32,
                                                    u32, vp, vp, vp, vp, vp, vp, vp, sz, vp]
            L.mars_verify_chain_sampled.restype = i32
            L.mars_stochastic_shard_records.argtypes = [vp, i64, i32, vp, vp, i32, i32, i32, i32, f32, u32, vp, vp,
                                                        vp, sz, vp]
            L.mars_stochastic_shard_records.restype = i32
            L.mars_stochastic_shard_verify.argtypes = [vp, i64, i32, vp, vp, i32, i32, vp, vp, vp, i32, i32, i32,
                                                       i32, f32, f32, u32, vp, vp, vp, vp, i32, vp, vp, vp, vp, vp]
            L.mars_stochastic_shard_verify.restype = i32
            L.mars_stochastic_shard_finish.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp]
            L.mars_stochastic_shard_finish.restype = i32
            L.mars_selftest_stream_read.argtypes = [vp, sz, sz, vp, vp]
            L.mars_selftest_stream_read.restype = i32
            L.mars_status_string.argtypes = [i32]
            L.mars_status_string.restype = ctypes.c_char_p
            L.mars_verify_tree_host_staging_bytes.argtypes = [i32, i32, i32, i32, i64, i32]
            L.mars_verify_tree_host_staging_bytes.restype = sz
            L.mars_verify_tree_host.argtypes = [vp, i64, i32, vp, vp, i32, i32, i32, f32, u32, vp, vp, vp, vp, i32,
                                                vp, vp, sz, vp]
            L.mars_verify_tree_host.restype = i32
            L.mars_test_hook.argtypes = [i32, i32]
            L.mars_test_hook.restype = i32
            L.mars_device_check.argtypes = [ctypes.POINTER(i32), ctypes.POINTER(i32)]
            L.mars_device_check.restype = i32
            _lib = L
    return _lib


HOOK_FORCE_SPLIT, HOOK_LMHEAD_SINGLE_BLOCK, HOOK_STOCH_TAIL_CLUSTER, HOOK_NO_OVERLAP, HOOK_TOPK_VARIANT = 0, 1, 2, 3, 4


def test_hook(which: int, value: int) -> int:
    """Set a test hook of the library (0 clears it); returns the previous value."""
    prev = lib().mars_test_hook(int(which), int(value))
    if prev < 0:
        raise MarsError(f"unknown test hook {which} or negative value {value}")
    return prev


def device_check() -> dict:
    """SM count of the current device against the count the launch shapes are tuned for."""
    sm, tuned = ctypes.c_int(0), ctypes.c_int(0)
    code = lib().mars_device_check(ctypes.byref(sm), ctypes.byref(tuned))
    return {"status": int(code), "sm_count": sm.value, "sm_tuned": tuned.value}


def _check(code: int, what: str) -> None:
    if code != 0:
        raise MarsError(f"{what}: {lib().mars_status_string(code).decode()} (status {code})")


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return FP32
    raise MarsError(f"logits must be bfloat16 or float32, got {t.dtype}")


def _dev_i32(x, device) -> torch.Tensor:
    t = torch.as_tensor(x)
    if t.dtype != torch.int32 or t.device != device or not t.is_contiguous():
        t = t.to(device=device, dtype=torch.int32).contiguous()
    return t


def workspace_bytes(B: int, N: int, V: int, dtype_code: int) -> int:
    return int(lib().mars_workspace_bytes(B, N, V, dtype_code))


def _workspace(B, N, V, dt, device, workspace):
    need = workspace_bytes(B, N, V, dt)
    if need == 0:
        raise MarsError("unsupported sizes")
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=device)
    return workspace, workspace.numel() * workspace.element_size()


def _logits_args(logits: torch.Tensor, rows: int, V):
    if not logits.is_cuda:
        raise MarsError("logits must live in device memory")
    if logits.dim() != 2 or logits.stride(1) != 1 or logits.shape[0] != rows:
        raise MarsError("logits must be [rows, >=V] with unit inner stride")
    V = logits.shape[1] if V is None else int(V)
    return _dtype_code(logits), int(logits.stride(0)), V


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def verify_tree(logits: torch.Tensor, tok, parent, theta: float, flags: int = 0,
                Dcap: int | None = None, V: int | None = None, debug: bool = False,
                workspace: torch.Tensor | None = None, out: dict | None = None) -> dict:
    """mars_verify_tree on the current stream.  Returns device tensors; asynchronous."""
    dev = logits.device
    tok = _dev_i32(tok, dev)
    parent = _dev_i32(parent, dev)
    B, N = tok.shape
    if parent.dim() == 1:
        flags |= SHARED_PARENT
    dt, ld, V = _logits_args(logits, B * N, V)
    Dcap = N - 1 if Dcap is None else int(Dcap)
    workspace, wbytes = _workspace(B, N, V, dt, dev, workspace)
    if out is None:
        out = alloc_outputs(B, N, Dcap, dev, debug)
    dbg = None
    if "top2_val" in out:
        dbg = _DebugOut(out["top2_val"].data_ptr(), out["top2_id"].data_ptr(),
                        out["node_flags"].data_ptr())
    with torch.cuda.device(dev):
        code = lib().mars_verify_tree(
            logits.data_ptr(), ld, dt, tok.data_ptr(), parent.data_ptr(), B, N, V, float(theta),
            flags, out["accept_len"].data_ptr(), out["out_tokens"].data_ptr(),
            out["path_nodes"].data_ptr(), out["out_len"].data_ptr(), Dcap,
            out["seq_status"].data_ptr(), ctypes.byref(dbg) if dbg is not None else None,
            workspace.data_ptr(), wbytes, _stream())
    _check(code, "mars_verify_tree")
    out["_keepalive"] = (tok, parent, workspace)
    return out


def verify_tree_static(logits: torch.Tensor, tok: torch.Tensor, parent: torch.Tensor, theta: float,
                       out: dict, flags: int = 0, Dcap: int | None = None,
                       V: int | None = None) -> dict:
    """mars_verify_tree_static on the current stream.

    For callers that may not allocate device memory: the library's built-in scratch array
    replaces the workspace, and this wrapper allocates nothing either -- `tok`, `parent`
    (int32 device tensors) and every buffer in `out` (see ``alloc_outputs``) must already
    exist.  Calls that may overlap on the GPU must not share a device (they share the array).
    """
    dev = logits.device
    for t in (tok, parent):
        if not (t.is_cuda and t.dtype == torch.int32 and t.is_contiguous()):
            raise MarsError("tok and parent must be contiguous int32 device tensors")
    B, N = tok.shape
    if parent.dim() == 1:
        flags |= SHARED_PARENT
    dt, ld, V = _logits_args(logits, B * N, V)
    Dcap = N - 1 if Dcap is None else int(Dcap)
    dbg = None
    if "top2_val" in out:
        dbg = _DebugOut(out["top2_val"].data_ptr(), out["top2_id"].data_ptr(),
                        out["node_flags"].data_ptr())
    with torch.cuda.device(dev):
        code = lib().mars_verify_tree_static(
            logits.data_ptr(), ld, dt, tok.data_ptr(), parent.data_ptr(), B, N, V, float(theta),
            flags, out["accept_len"].data_ptr(), out["out_tokens"].data_ptr(),
            out["path_nodes"].data_ptr(), out["out_len"].data_ptr(), Dcap,
            out["seq_status"].data_ptr(), ctypes.byref(dbg) if dbg is not None else None, _stream())
    _check(code, "mars_verify_tree_static")
    return out


def alloc_host_outputs(B: int, Dcap: int) -> dict:
    """Pinned host buffers for the results of ``verify_tree_host``."""
    def full(shape):
        return torch.full(shape, -777, dtype=torch.int32).pin_memory()
    return {"accept_len": full((B,)), "out_tokens": full((B, Dcap + 1)), "path_nodes": full((B, Dcap + 1)),
            "out_len": full((B,)), "seq_status": full((B,))}


def verify_tree_host(logits_host: torch.Tensor, tok_host: torch.Tensor, parent_host: torch.Tensor, theta: float,
                     staging: torch.Tensor, out_host: dict, flags: int = 0, Dcap: int | None = None,
                     V: int | None = None) -> dict:
    """mars_verify_tree_host on the current stream of `staging`'s device: every input and output is a
    HOST tensor (pinned for asynchronous copies), `staging` a uint8 device tensor of at least
    ``mars_verify_tree_host_staging_bytes`` bytes.  Results are valid once the stream has passed."""
    for t in (logits_host, tok_host, parent_host, *out_host.values()):
        if t.is_cuda or not t.is_contiguous():
            raise MarsError("inputs and outputs of verify_tree_host are contiguous host tensors")
    if tok_host.dtype != torch.int32 or parent_host.dtype != torch.int32:
        raise MarsError("tok and parent must be int32")
    B, N = tok_host.shape
    if parent_host.dim() == 1:
        flags |= SHARED_PARENT
    dt = _dtype_code(logits_host)
    if logits_host.dim() != 2 or logits_host.shape[0] != B * N:
        raise MarsError("logits must be [B*N, ld]")
    ld = logits_host.shape[1]
    V = ld if V is None else int(V)
    Dcap = N - 1 if Dcap is None else int(Dcap)
    with torch.cuda.device(staging.device):
        code = lib().mars_verify_tree_host(
            logits_host.data_ptr(), ld, dt, tok_host.data_ptr(), parent_host.data_ptr(), B, N, V, float(theta), flags,
            out_host["accept_len"].data_ptr(), out_host["out_tokens"].data_ptr(),
            out_host["path_nodes"].data_ptr() if "path_nodes" in out_host else None,
            out_host["out_len"].data_ptr(),
            Dcap, out_host["seq_status"].data_ptr() if "seq_status" in out_host else None,
            staging.data_ptr(), staging.numel(), _stream())
    _check(code, "mars_verify_tree_host")
    return out_host


def verify_chain(logits: torch.Tensor, draft, theta: float, flags: int = 0, V: int | None = None,
                 debug: bool = False, workspace: torch.Tensor | None = None,
                 out: dict | None = None) -> dict:
    """mars_verify_chain on the current stream: K rows and K-1 drafts per sequence."""
    dev = logits.device
    draft = _dev_i32(draft, dev)
    B, Km1 = draft.shape
    K = Km1 + 1
    dt, ld, V = _logits_args(logits, B * K, V)
    workspace, wbytes = _workspace(B, K, V, dt, dev, workspace)
    if out is None:
        out = alloc_outputs(B, K, K - 1, dev, debug)
    dbg = None
    if "top2_val" in out:
        dbg = _DebugOut(out["top2_val"].data_ptr(), out["top2_id"].data_ptr(),
                        out["node_flags"].data_ptr())
    with torch.cuda.device(dev):
        code = lib().mars_verify_chain(
            logits.data_ptr(), ld, dt, draft.data_ptr() if Km1 > 0 else None, B, K, V,
            float(theta), flags, out["accept_len"].data_ptr(), out["out_tokens"].data_ptr(),
            out["out_len"].data_ptr(), out["seq_status"].data_ptr(),
            ctypes.byref(dbg) if dbg is not None else None, workspace.data_ptr(), wbytes, _stream())
    _check(code, "mars_verify_chain")
    out["_keepalive"] = (draft, workspace)
    return out


def lmhead_verify(hidden: torch.Tensor, w_vocab: torch.Tensor, bias, tok, parent, theta: float,
                  flags: int = 0, Dcap: int | None = None, debug: bool = False,
                  workspace: torch.Tensor | None = None, out: dict | None = None) -> dict:
    """mars_lmhead_verify on the current stream: hidden bf16 [B*N, d], w_vocab bf16 [V, d]."""
    dev = hidden.device
    if not (hidden.is_cuda and w_vocab.is_cuda and hidden.dtype == torch.bfloat16
            and w_vocab.dtype == torch.bfloat16 and hidden.is_contiguous() and w_vocab.is_contiguous()):
        raise MarsError("hidden and w_vocab must be contiguous bfloat16 device tensors")
    tok = _dev_i32(tok, dev)
    parent = _dev_i32(parent, dev)
    B, N = tok.shape
    if parent.dim() == 1:
        flags |= SHARED_PARENT
    M, d = hidden.shape
    V = w_vocab.shape[0]
    if M != B * N or w_vocab.shape[1] != d:
        raise MarsError("shape mismatch")
    if bias is not None:
        bias = bias.to(device=dev, dtype=torch.float32).contiguous()
    Dcap = N - 1 if Dcap is None else int(Dcap)
    need = int(lib().mars_lmhead_workspace_bytes(B, N, V, d))
    if need == 0:
        raise MarsError("unsupported sizes")
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=dev)
    if out is None:
        out = alloc_outputs(B, N, Dcap, dev, debug)
    dbg = None
    if "top2_val" in out:
        dbg = _DebugOut(out["top2_val"].data_ptr(), out["top2_id"].data_ptr(),
                        out["node_flags"].data_ptr())
    with torch.cuda.device(dev):
        code = lib().mars_lmhead_verify(
            hidden.data_ptr(), w_vocab.data_ptr(), bias.data_ptr() if bias is not None else None, d,
            tok.data_ptr(), parent.data_ptr(), B, N, V, float(theta), flags,
            out["accept_len"].data_ptr(), out["out_tokens"].data_ptr(), out["path_nodes"].data_ptr(),
            out["out_len"].data_ptr(), Dcap, out["seq_status"].data_ptr(),
            ctypes.byref(dbg) if dbg is not None else None, workspace.data_ptr(),
            workspace.numel(), _stream())
    _check(code, "mars_lmhead_verify")
    out["_keepalive"] = (tok, parent, workspace, bias)
    return out


def _dev_f32(x, device) -> torch.Tensor:
    t = torch.as_tensor(x)
    if t.dtype != torch.float32 or t.device != device or not t.is_contiguous():
        t = t.to(device=device, dtype=torch.float32).contiguous()
    return t


def alloc_stochastic_outputs(B: int, N: int, Dcap: int, device, debug: bool = False) -> dict:
    out = alloc_outputs(B, N, Dcap, device)
    if debug:
        out["node_prob"] = torch.full((B, N), float("nan"), dtype=torch.float32, device=device)
        out["node_how"] = torch.full((B, N), 255, dtype=torch.uint8, device=device)
    return out


def _stoch_workspace(B, N, V, dt, device, workspace):
    need = int(lib().mars_stochastic_workspace_bytes(B, N, V, dt))
    if need == 0:
        raise MarsError("unsupported sizes")
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=device)
    return workspace, workspace.numel() * workspace.element_size()


def verify_tree_stochastic(logits: torch.Tensor, tok, parent, uniform, theta: float, temperature: float,
                           flags: int = 0, Dcap: int | None = None, V: int | None = None,
                           debug: bool = False, workspace: torch.Tensor | None = None,
                           out: dict | None = None) -> dict:
    """mars_verify_tree_stochastic on the current stream; `uniform` is float32 [B, N]."""
    dev = logits.device
    tok = _dev_i32(tok, dev)
    parent = _dev_i32(parent, dev)
    uniform = _dev_f32(uniform, dev)
    B, N = tok.shape
    if parent.dim() == 1:
        flags |= SHARED_PARENT
    if tuple(uniform.shape) != (B, N):
        raise MarsError("uniform must be [B, N]")
    dt, ld, V = _logits_args(logits, B * N, V)
    Dcap = N - 1 if Dcap is None else int(Dcap)
    workspace, wbytes = _stoch_workspace(B, N, V, dt, dev, workspace)
    if out is None:
        out = alloc_stochastic_outputs(B, N, Dcap, dev, debug)
    with torch.cuda.device(dev):
        code = lib().mars_verify_tree_stochastic(
            logits.data_ptr(), ld, dt, tok.data_ptr(), parent.data_ptr(), uniform.data_ptr(), B, N, V,
            float(theta), float(temperature), flags, out["accept_len"].data_ptr(),
            out["out_tokens"].data_ptr(), out["path_nodes"].data_ptr(), out["out_len"].data_ptr(), Dcap,
            out["seq_status"].data_ptr(),
            out["node_prob"].data_ptr() if "node_prob" in out else None,
            out["node_how"].data_ptr() if "node_how" in out else None,
            workspace.data_ptr(), wbytes, _stream())
    _check(code, "mars_verify_tree_stochastic")
    out["_keepalive"] = (tok, parent, uniform, workspace)
    return out


def verify_chain_stochastic(logits: torch.Tensor, draft, uniform, theta: float, temperature: float,
                            flags: int = 0, V: int | None = None, debug: bool = False,
                            workspace: torch.Tensor | None = None, out: dict | None = None) -> dict:
    """mars_verify_chain_stochastic on the current stream: K rows, K-1 drafts, uniform [B, K]."""
    dev = logits.device
    draft = _dev_i32(draft, dev)
    uniform = _dev_f32(uniform, dev)
    B, Km1 = draft.shape
    K = Km1 + 1
    if tuple(uniform.shape) != (B, K):
        raise MarsError("uniform must be [B, K]")
    dt, ld, V = _logits_args(logits, B * K, V)
    workspace, wbytes = _stoch_workspace(B, K, V, dt, dev, workspace)
    if out is None:
        out = alloc_stochastic_outputs(B, K, K - 1, dev, debug)
    with torch.cuda.device(dev):
        code = lib().mars_verify_chain_stochastic(
            logits.data_ptr(), ld, dt, draft.data_ptr() if Km1 > 0 else None, uniform.data_ptr(), B, K, V,
            float(theta), float(temperature), flags, out["accept_len"].data_ptr(),
            out["out_tokens"].data_ptr(), out["out_len"].data_ptr(), out["seq_status"].data_ptr(),
            out["node_prob"].data_ptr() if "node_prob" in out else None,
            out["node_how"].data_ptr() if "node_how" in out else None,
            workspace.data_ptr(), wbytes, _stream())
    _check(code, "mars_verify_chain_stochastic")
    out["_keepalive"] = (draft, uniform, workspace)
    return out


def verify_chain_sampled(logits: torch.Tensor, draft_logits: torch.Tensor, draft, draft_prob, uniform,
                         theta: float, temperature: float, draft_temperature: float, flags: int = 0,
                         V: int | None = None, debug: bool = False, workspace: torch.Tensor | None = None,
                         out: dict | None = None) -> dict:
    """mars_verify_chain_sampled on the current stream: K target rows and K-1 drafter rows per
    sequence, drafts [B, K-1] with their drafter probabilities, uniform [B, K]."""
    dev = logits.device
    draft = _dev_i32(draft, dev)
    draft_prob = _dev_f32(draft_prob, dev)
    uniform = _dev_f32(uniform, dev)
    B, Km1 = draft.shape
    K = Km1 + 1
    if tuple(uniform.shape) != (B, K) or tuple(draft_prob.shape) != (B, Km1):
        raise MarsError("uniform must be [B, K] and draft_prob [B, K-1]")
    dt, ld, V = _logits_args(logits, B * K, V)
    if Km1 > 0:
        dtq, ldq, _ = _logits_args(draft_logits, B * Km1, V)
        if dtq != dt or draft_logits.shape[1] < V:
            raise MarsError("draft_logits must have the dtype of logits and at least V columns")
    else:
        ldq = V
    workspace, wbytes = _stoch_workspace(B, K, V, dt, dev, workspace)
    if out is None:
        out = alloc_stochastic_outputs(B, K, K - 1, dev, debug)
    with torch.cuda.device(dev):
        code = lib().mars_verify_chain_sampled(
            logits.data_ptr(), ld, dt, draft_logits.data_ptr() if Km1 > 0 else None, ldq,
            draft.data_ptr() if Km1 > 0 else None, draft_prob.data_ptr() if Km1 > 0 else None,
            uniform.data_ptr(), B, K, V, float(theta), float(temperature), float(draft_temperature), flags,
            out["accept_len"].data_ptr(), out["out_tokens"].data_ptr(), out["out_len"].data_ptr(),
            out["seq_status"].data_ptr(),
            out["node_prob"].data_ptr() if "node_prob" in out else None,
            out["node_how"].data_ptr() if "node_how" in out else None,
            workspace.data_ptr(), wbytes, _stream())
    _check(code, "mars_verify_chain_sampled")
    out["_keepalive"] = (draft, draft_prob, uniform, draft_logits, workspace)
    return out


def stochastic_shard_records(logits_local: torch.Tensor, tok, parent, id_offset: int, temperature: float,
                             V_local: int | None = None, flags: int = 0,
                             workspace: torch.Tensor | None = None):
    """mars_stochastic_shard_records on the current stream: (records int32 [B*N, 8], node_logit
    float32 [B*N]) of one vocabulary shard."""
    dev = logits_local.device
    tok = _dev_i32(tok, dev)
    parent = _dev_i32(parent, dev)
    B, N = tok.shape
    if parent.dim() == 1:
        flags |= SHARED_PARENT
    dt, ld, V_local = _logits_args(logits_local, B * N, V_local)
    workspace, wbytes = _stoch_workspace(B, N, V_local, dt, dev, workspace)
    records = torch.empty((B * N, 8), dtype=torch.int32, device=dev)
    node_logit = torch.empty((B * N,), dtype=torch.float32, device=dev)
    with torch.cuda.device(dev):
        code = lib().mars_stochastic_shard_records(
            logits_local.data_ptr(), ld, dt, tok.data_ptr(), parent.data_ptr(), B, N, V_local, int(id_offset),
            float(temperature), flags, records.data_ptr(), node_logit.data_ptr(), workspace.data_ptr(), wbytes,
            _stream())
    _check(code, "mars_stochastic_shard_records")
    return records, node_logit


def stochastic_shard_verify(logits_local: torch.Tensor, records_all: torch.Tensor, node_logit_all: torch.Tensor,
                            my_shard: int, id_offset: int, tok, parent, uniform, theta: float,
                            temperature: float, flags: int = 0, Dcap: int | None = None,
                            V_local: int | None = None, debug: bool = False, out: dict | None = None):
    """mars_stochastic_shard_verify on the current stream: records_all int32 [G, B*N, 8],
    node_logit_all float32 [G, B*N].  Returns (outputs, token_part int32 [B])."""
    dev = logits_local.device
    tok = _dev_i32(tok, dev)
    parent = _dev_i32(parent, dev)
    uniform = _dev_f32(uniform, dev)
    B, N = tok.shape
    if parent.dim() == 1:
        flags |= SHARED_PARENT
    dt, ld, V_local = _logits_args(logits_local, B * N, V_local)
    G = records_all.shape[0]
    if not (records_all.is_cuda and records_all.dtype == torch.int32 and records_all.is_contiguous()
            and tuple(records_all.shape) == (G, B * N, 8) and node_logit_all.is_contiguous()
            and node_logit_all.dtype == torch.float32 and tuple(node_logit_all.shape) == (G, B * N)):
        raise MarsError("records_all must be int32 [G, B*N, 8] and node_logit_all float32 [G, B*N], contiguous")
    Dcap = N - 1 if Dcap is None else int(Dcap)
    if out is None:
        out = alloc_stochastic_outputs(B, N, Dcap, dev, debug)
    token_part = torch.full((B,), -777, dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        code = lib().mars_stochastic_shard_verify(
            logits_local.data_ptr(), ld, dt, records_all.data_ptr(), node_logit_all.data_ptr(), G, int(my_shard),
            tok.data_ptr(), parent.data_ptr(), uniform.data_ptr(), B, N, V_local, int(id_offset), float(theta),
            float(temperature), flags, out["accept_len"].data_ptr(), out["out_tokens"].data_ptr(),
            out["path_nodes"].data_ptr(), out["out_len"].data_ptr(), Dcap, out["seq_status"].data_ptr(),
            out["node_prob"].data_ptr() if "node_prob" in out else None,
            out["node_how"].data_ptr() if "node_how" in out else None, token_part.data_ptr(), _stream())
    _check(code, "mars_stochastic_shard_verify")
    out["_keepalive"] = (tok, parent, uniform, records_all, node_logit_all)
    return out, token_part


def stochastic_shard_finish(token_all: torch.Tensor, out: dict) -> dict:
    """mars_stochastic_shard_finish on the current stream: token_all int32 [G, B]."""
    if not (token_all.is_cuda and token_all.dtype == torch.int32 and token_all.is_contiguous() and token_all.dim() == 2):
        raise MarsError("token_all must be a contiguous int32 [G, B] device tensor")
    G, B = token_all.shape
    Dcap = out["out_tokens"].shape[1] - 1
    with torch.cuda.device(token_all.device):
        code = lib().mars_stochastic_shard_finish(token_all.data_ptr(), G, B, Dcap, out["accept_len"].data_ptr(),
                                                  out["out_tokens"].data_ptr(), out["seq_status"].data_ptr(), _stream())
    _check(code, "mars_stochastic_shard_finish")
    return out


def stream_read_probe(buffer: torch.Tensor, chunk_bytes: int, out: torch.Tensor | None = None) -> torch.Tensor:
    """mars_selftest_stream_read on the current stream over the whole (contiguous) tensor; returns
    the one-word result tensor (the call is asynchronous).  `out` (int32 [1], zeroed by the
    caller) avoids the allocation and the fill kernel of a fresh result word."""
    if not (buffer.is_cuda and buffer.is_contiguous()):
        raise MarsError("buffer must be a contiguous device tensor")
    if out is None:
        out = torch.zeros((1,), dtype=torch.int32, device=buffer.device)
    with torch.cuda.device(buffer.device):
        code = lib().mars_selftest_stream_read(buffer.data_ptr(), buffer.numel() * buffer.element_size(),
                                               int(chunk_bytes), out.data_ptr(), _stream())
    _check(code, "mars_selftest_stream_read")
    return out


def top2_shard(logits_local: torch.Tensor, B: int, N: int, id_offset: int, V_local: int | None = None,
               flags: int = 0, workspace: torch.Tensor | None = None,
               records: torch.Tensor | None = None) -> torch.Tensor:
    """mars_top2_shard on the current stream: per-row records of one vocabulary shard as an
    int32 [B*N, 4] tensor (z1 bits, global id1, z2 bits, global id2)."""
    dev = logits_local.device
    dt, ld, V_local = _logits_args(logits_local, B * N, V_local)
    workspace, wbytes = _workspace(B, N, V_local, dt, dev, workspace)
    if records is None:
        records = torch.empty((B * N, 4), dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        code = lib().mars_top2_shard(logits_local.data_ptr(), ld, dt, B, N, V_local, int(id_offset),
                                     records.data_ptr(), flags, workspace.data_ptr(), wbytes, _stream())
    _check(code, "mars_top2_shard")
    return records


def lmhead_top2_shard(hidden: torch.Tensor, w_shard: torch.Tensor, bias_shard, B: int, N: int,
                      id_offset: int, workspace: torch.Tensor | None = None) -> torch.Tensor:
    """mars_lmhead_top2_shard on the current stream: records int32 [B*N, 4] of one vocabulary
    shard of the output projection (hidden bf16 [B*N, d], w_shard bf16 [V_local, d])."""
    dev = hidden.device
    if not (hidden.is_cuda and w_shard.is_cuda and hidden.dtype == torch.bfloat16
            and w_shard.dtype == torch.bfloat16 and hidden.is_contiguous() and w_shard.is_contiguous()):
        raise MarsError("hidden and w_shard must be contiguous bfloat16 device tensors")
    M, d = hidden.shape
    V_local = w_shard.shape[0]
    if M != B * N or w_shard.shape[1] != d:
        raise MarsError("shape mismatch")
    if bias_shard is not None:
        bias_shard = bias_shard.to(device=dev, dtype=torch.float32).contiguous()
    need = int(lib().mars_lmhead_workspace_bytes(B, N, V_local, d))
    if need == 0:
        raise MarsError("unsupported sizes")
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=dev)
    records = torch.empty((M, 4), dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        code = lib().mars_lmhead_top2_shard(
            hidden.data_ptr(), w_shard.data_ptr(), bias_shard.data_ptr() if bias_shard is not None else None,
            d, B, N, V_local, int(id_offset), records.data_ptr(), workspace.data_ptr(), workspace.numel(),
            _stream())
    _check(code, "mars_lmhead_top2_shard")
    return records


def verify_records(records: torch.Tensor, tok, parent, theta: float, flags: int = 0,
                   Dcap: int | None = None, debug: bool = False, out: dict | None = None) -> dict:
    """mars_verify_records on the current stream: records int32 [G, B*N, 4]."""
    dev = records.device
    tok = _dev_i32(tok, dev)
    parent = _dev_i32(parent, dev)
    B, N = tok.shape
    if parent.dim() == 1:
        flags |= SHARED_PARENT
    if not (records.is_cuda and records.dtype == torch.int32 and records.is_contiguous()
            and records.dim() == 3 and records.shape[1:] == (B * N, 4)):
        raise MarsError("records must be a contiguous int32 [G, B*N, 4] device tensor")
    G = records.shape[0]
    Dcap = N - 1 if Dcap is None else int(Dcap)
    if out is None:
        out = alloc_outputs(B, N, Dcap, dev, debug)
    dbg = None
    if "top2_val" in out:
        dbg = _DebugOut(out["top2_val"].data_ptr(), out["top2_id"].data_ptr(),
                        out["node_flags"].data_ptr())
    with torch.cuda.device(dev):
        code = lib().mars_verify_records(
            records.data_ptr(), G, tok.data_ptr(), parent.data_ptr(), B, N, float(theta), flags,
            out["accept_len"].data_ptr(), out["out_tokens"].data_ptr(), out["path_nodes"].data_ptr(),
            out["out_len"].data_ptr(), Dcap, out["seq_status"].data_ptr(),
            ctypes.byref(dbg) if dbg is not None else None, _stream())
    _check(code, "mars_verify_records")
    out["_keepalive"] = (tok, parent, records)
    return out


def top2_histograms(top2_val: torch.Tensor, z1_lo: float, z1_hi: float, nbins: int, out=None):
    """mars_top2_histograms on the current stream: returns (hist uint32-as-int32 [3, nbins],
    outliers [3]) device tensors; `out` = such a pair to write into."""
    if not (top2_val.is_cuda and top2_val.dtype == torch.float32 and top2_val.is_contiguous()
            and top2_val.dim() == 2 and top2_val.shape[1] == 2):
        raise MarsError("top2_val must be a contiguous float32 [rows, 2] device tensor")
    dev = top2_val.device
    if out is None:
        hist = torch.empty((3, nbins), dtype=torch.int32, device=dev)
        outl = torch.empty((3,), dtype=torch.int32, device=dev)
    else:
        hist, outl = out
    with torch.cuda.device(dev):
        code = lib().mars_top2_histograms(top2_val.data_ptr(), top2_val.shape[0], float(z1_lo),
                                          float(z1_hi), int(nbins), hist.data_ptr(), outl.data_ptr(),
                                          _stream())
    _check(code, "mars_top2_histograms")
    return hist, outl


def topk_rows(logits: torch.Tensor, k: int, V: int | None = None,
              workspace: torch.Tensor | None = None, out=None):
    """mars_topk_rows on the current stream: (values float32 [rows, k], ids int32 [rows, k]);
    `out` = such a pair to write into."""
    dev = logits.device
    dt, ld, V = _logits_args(logits, logits.shape[0], V)
    rows = logits.shape[0]
    need = int(lib().mars_topk_workspace_bytes(rows, V, dt, int(k)))
    if need == 0:
        raise MarsError("unsupported sizes")
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=dev)
    if out is None:
        val = torch.empty((rows, k), dtype=torch.float32, device=dev)
        idx = torch.empty((rows, k), dtype=torch.int32, device=dev)
    else:
        val, idx = out
    with torch.cuda.device(dev):
        code = lib().mars_topk_rows(logits.data_ptr(), ld, dt, rows, V, int(k), val.data_ptr(),
                                    idx.data_ptr(), workspace.data_ptr(), workspace.numel(), _stream())
    _check(code, "mars_topk_rows")
    return val, idx


def alloc_outputs(B: int, N: int, Dcap: int, device, debug: bool = False) -> dict:
    """Output buffers in device memory (filled with a poison value so that unwritten
    slots are noticed)."""
    def full(shape, dtype, v):
        return torch.full(shape, v, dtype=dtype, device=device)
    out = {
        "accept_len": full((B,), torch.int32, -777),
        "out_tokens": full((B, Dcap + 1), torch.int32, -777),
        "path_nodes": full((B, Dcap + 1), torch.int32, -777),
        "out_len": full((B,), torch.int32, -777),
        "seq_status": full((B,), torch.int32, -777),
    }
    if debug:
        out["top2_val"] = full((B * N, 2), torch.float32, float("nan"))
        out["top2_id"] = full((B * N, 2), torch.int32, -777)
        out["node_flags"] = full((B, N), torch.uint8, 255)
    return out


def to_host(out: dict) -> dict:
    """Synchronise and copy every output tensor to numpy."""
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items() if isinstance(v, torch.Tensor)}
