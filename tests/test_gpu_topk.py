"""Exact top-k of logits rows on the device against the oracle: ids and value bits."""
import numpy as np
import pytest
import torch

from oracle import mars_oracle as orc
from paper_2601_15498_b200 import mars, synth

import hookctl as hooks
from tests.test_gpu_parity import special_rows

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def check(logits, k, V=None):
    val, idx = mars.topk_rows(logits, k, V=V)
    torch.cuda.synchronize()
    src = logits if V is None else logits[:, :V].contiguous()
    rv, ri = orc.topk(synth.to_numpy_bits(src), k)
    assert np.array_equal(idx.cpu().numpy(), ri), f"ids k={k}"
    assert np.array_equal(val.cpu().numpy().view(np.uint32), rv.view(np.uint32)), f"values k={k}"


@pytest.fixture(autouse=True)
def _no_forced_split(monkeypatch):
    hooks.clear("HOOK_FORCE_SPLIT")
    hooks.clear("HOOK_TOPK_VARIANT")


@pytest.mark.parametrize("k", [1, 2, 10, 32])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_topk_qwen_and_vicuna_sized_rows(k, dtype):
    g = torch.Generator(device=DEV); g.manual_seed(k)
    for R, V in ((60, 151936), (700, 32000), (10, 32000)):       # split rows, whole rows, few rows
        z = (torch.randn((R, V), generator=g, device=DEV) * 3).to(dtype)
        check(z, k)


@pytest.mark.parametrize("V", [1, 2, 9, 33, 257, 4099, 18437])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_topk_odd_sizes_and_degenerate_rows(V, dtype):
    g = torch.Generator(device="cpu"); g.manual_seed(V)
    z = (torch.randn((5, V), generator=g) * 3).to(dtype).to(DEV)
    for k in sorted({1, min(2, V), min(10, V), min(32, V)}):
        check(z, k)
    if V >= 9:
        s = special_rows(V, dtype)
        for k in (2, min(9, V)):
            check(s, k)


@pytest.mark.parametrize("S", [2, 5, 64])
def test_topk_forced_split_and_unaligned(monkeypatch, S):
    hooks.set("HOOK_FORCE_SPLIT", S)
    g = torch.Generator(device=DEV); g.manual_seed(S)
    big = torch.full((9, 40007 + 11), 3.0e38, dtype=torch.bfloat16, device=DEV)     # canaries around
    view = big[1:-1, 3:3 + 40007]
    view.copy_((torch.randn((7, 40007), generator=g, device=DEV) * 3).to(torch.bfloat16))
    view[2] = torch.round(view[2].float()).to(torch.bfloat16)                      # heavy ties
    val, idx = mars.topk_rows(view, 10)
    torch.cuda.synchronize()
    rv, ri = orc.topk(synth.to_numpy_bits(view.contiguous()), 10)
    assert np.array_equal(idx.cpu().numpy(), ri) and np.array_equal(val.cpu().numpy(), rv)
    asc = torch.linspace(-5, 5, 40007, device=DEV).repeat(3, 1).to(torch.bfloat16)   # worst case for the filter
    check(asc, 10)


def test_topk_host_errors():
    z = torch.zeros((4, 100), device=DEV)
    for k in (0, 33, 101):
        with pytest.raises(mars.MarsError):
            mars.topk_rows(z, k)


@pytest.mark.parametrize("variant", [1, 2])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_topk_both_batch_shapes_of_the_kernel(dtype, variant):
    """The kernel has two launch shapes (8 vectors per batch at 4 blocks per SM, 4 at 6) and picks
    by size; both are forced here on whole rows, split rows, ragged and degenerate rows."""
    hooks.set("HOOK_TOPK_VARIANT", variant)
    g = torch.Generator(device=DEV); g.manual_seed(variant)
    for R, V in ((700, 40007), (9, 151936), (650, 2049)):
        z = (torch.randn((R, V), generator=g, device=DEV) * 3).to(dtype)
        z[0] = torch.linspace(-8, 8, V, device=DEV).to(dtype)         # overflows the queue
        z[1] = 0.5
        z[2] = float("-inf"); z[2, V // 2] = 3.0
        for k in (1, 10, 32):
            check(z, k)
    check(special_rows(4099, dtype), 9)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_topk_whole_rows_that_defeat_the_floor(dtype):
    """Whole rows (one block per row): ascending values overflow the candidate buffer and take the
    exact fallback; constant rows tie everywhere (lowest ids win); a row whose large values all sit
    in the last batch; and a row with fewer than k entries above -inf."""
    V, k = 151936, 10
    z = torch.empty((600, V), dtype=dtype, device=DEV)
    g = torch.Generator(device=DEV); g.manual_seed(77)
    z.copy_((torch.randn((600, V), generator=g, device=DEV) * 3).to(dtype))
    z[0] = torch.linspace(-8, 8, V, device=DEV).to(dtype)
    z[1] = 1.25
    z[2, -500:] += 40.0
    z[3] = float("-inf"); z[3, 77] = 1.0; z[3, 140000] = float("nan"); z[3, 9] = -2.0
    z[4] = torch.linspace(8, -8, V, device=DEV).to(dtype)
    check(z, k)
    check(z[:8], 32)


def test_topk_back_to_back_calls_share_a_workspace():
    """Consecutive top-k calls overlap on the GPU; alternating inputs through one workspace must
    still give each call its own rows' answer."""
    g = torch.Generator(device=DEV); g.manual_seed(5)
    zs = [(torch.randn((300, 40000), generator=g, device=DEV) * 3).to(torch.bfloat16) for _ in range(2)]
    want = [orc.topk(synth.to_numpy_bits(z), 10) for z in zs]
    need = int(mars.lib().mars_topk_workspace_bytes(300, 40000, mars.BF16, 10))
    work = torch.empty(need, dtype=torch.uint8, device=DEV)
    outs = [(torch.empty((300, 10), dtype=torch.float32, device=DEV), torch.empty((300, 10), dtype=torch.int32, device=DEV))
            for _ in range(30)]
    for i in range(30):
        mars.topk_rows(zs[i & 1], 10, workspace=work, out=outs[i])
    torch.cuda.synchronize()
    for i in range(30):
        rv, ri = want[i & 1]
        assert np.array_equal(outs[i][1].cpu().numpy(), ri), i
        assert np.array_equal(outs[i][0].cpu().numpy().view(np.uint32), rv.view(np.uint32)), i


@pytest.mark.parametrize("k,dtype", [(10, torch.bfloat16), (32, torch.bfloat16), (10, torch.float32)])
def test_topk_full_bench_batch_every_row(k, dtype):
    """The batch the bench times (7 680 rows of 151 936 logits, one launch, one block per row):
    every row against the oracle, values and ids."""
    w = synth.cfg3(DEV, seed=5, B=128, dtype=dtype)
    assert w.R == 7680
    val, idx = mars.topk_rows(w.logits, k)
    torch.cuda.synchronize()
    val, idx = val.cpu().numpy(), idx.cpu().numpy()
    for lo in range(0, w.R, 1920):                        # the oracle takes the rows in four parts
        rv, ri = orc.topk(synth.to_numpy_bits(w.logits[lo:lo + 1920]), k)
        assert np.array_equal(idx[lo:lo + 1920], ri), (k, lo)
        assert np.array_equal(val[lo:lo + 1920].view(np.uint32), rv.view(np.uint32)), (k, lo)
