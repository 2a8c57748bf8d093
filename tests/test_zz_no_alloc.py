"""mars_verify_tree_static: verification for callers that cannot allocate device memory.

Some users of this library run inside another system's memory regime (a server that gave all
free HBM to its cache pool, a plug-in op, a loop that cannot afford cudaMalloc's implicit
synchronisation) and therefore cannot hand over a workspace.  The static entry point uses a
fixed scratch array inside the library instead.  This test calls it through the C ABI twice in
a row -- the second call with different inputs, so stale scratch contents would show -- and
requires the same bits as the regular entry point and as the CPU oracle (the library's
tolerance for this path is bit-exactness).  It also checks the capacity error, and that a
caller's MARS_COUNTERS_ZERO promise -- which nobody can keep for an array they do not own --
is ignored rather than trusted.  The file name sorts last on purpose: a
run that stops at the first failure has then already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import mars_oracle as orc
from paper_2601_15498_b200 import mars, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
KEYS = ("accept_len", "out_tokens", "path_nodes", "out_len", "seq_status", "top2_id", "node_flags")


def _run_both(w, flags=0):
    tok = torch.as_tensor(w.tok, device=DEV)
    parent = torch.as_tensor(w.parent, device=DEV)
    ref = mars.to_host(mars.verify_tree(w.logits, tok, parent, w.theta, debug=True))
    out = mars.alloc_outputs(w.B, w.N, w.N - 1, DEV, debug=True)
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    mars.verify_tree_static(w.logits, tok, parent, w.theta, out, flags=flags)
    assert torch.cuda.memory_allocated() == before        # the wrapper allocated nothing either
    got = mars.to_host(out)
    want = orc.verify_tree(synth.to_numpy_bits(w.logits), w.tok, w.parent, w.theta)
    for k in KEYS:
        assert np.array_equal(got[k], ref[k]), k
        assert np.array_equal(got[k], want[k]), ("oracle", k)
    assert np.array_equal(got["top2_val"].view(np.uint32), ref["top2_val"].view(np.uint32))
    assert np.array_equal(got["top2_val"].view(np.uint32), want["top2_val"].view(np.uint32))
    return got


def test_static_scratch_matches_workspace_entry_point_twice():
    assert mars.lib().mars_static_scratch_bytes() == 1 << 20
    # call 1: few rows, so rows are split over many blocks (many partial records + counters)
    a = _run_both(synth.tree_workload("na1", 3, 60, 6, 4, 40000, torch.bfloat16, DEV, 501, 0.9,
                                      3.0, 15.0, 30.0, 0.3))
    # call 2 right after, other shape / dtype / data: leftovers of call 1 must not matter
    b = _run_both(synth.tree_workload("na2", 7, 33, 5, 3, 32000, torch.float32, DEV, 502, 0.9,
                                      2.0, 20.0, 20.0, 0.4))
    # call 3: the first shape again
    c = _run_both(synth.tree_workload("na1", 3, 60, 6, 4, 40000, torch.bfloat16, DEV, 501, 0.9,
                                      3.0, 15.0, 30.0, 0.3))
    assert np.array_equal(a["out_tokens"], c["out_tokens"])
    assert a["accept_len"].shape != b["accept_len"].shape


def test_counters_zero_flag_is_not_trusted_for_the_shared_array():
    """A small batch leaves top-2 records right behind its (short) counter region.  A larger
    batch whose counter region covers those bytes, called with MARS_COUNTERS_ZERO, would start
    from dirty counters if the flag were honoured: no sequence would ever see its last arrival
    and the outputs would stay unwritten."""
    _run_both(synth.tree_workload("na3", 3, 12, 4, 3, 9000, torch.float32, DEV, 503, 0.9,
                                  2.0, 20.0, 20.0, 0.4))
    big = synth.tree_workload("na4", 100, 12, 4, 3, 9000, torch.float32, DEV, 504, 0.9,
                              2.0, 20.0, 20.0, 0.4)
    _run_both(big, flags=mars.COUNTERS_ZERO)
    _run_both(big, flags=mars.COUNTERS_ZERO)


def test_static_scratch_rejects_batches_beyond_capacity():
    lib = mars.lib()
    B, N, V = 1200, 60, 1000                       # 72 000 rows x 16 B > 1 MiB
    assert lib.mars_workspace_bytes(B, N, V, mars.BF16) > lib.mars_static_scratch_bytes()
    logits = torch.zeros((B * N, V), dtype=torch.bfloat16, device=DEV)
    tok = torch.zeros((B, N), dtype=torch.int32, device=DEV)
    parent = torch.as_tensor(synth.chain_parents(B, N), device=DEV)
    out = mars.alloc_outputs(B, N, N - 1, DEV)
    with pytest.raises(mars.MarsError, match="built-in static"):
        mars.verify_tree_static(logits, tok, parent, 0.9, out)
    torch.cuda.synchronize()
    assert (out["accept_len"].cpu().numpy() == -777).all()          # nothing ran
    assert lib.mars_status_string(5) == b"batch needs more scratch than the built-in static array holds"
