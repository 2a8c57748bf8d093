"""Telemetry histograms on the device against the oracle: exact counts."""
import numpy as np
import pytest
import torch

from oracle import mars_oracle as orc
from paper_2601_15498_b200 import mars, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("nbins", [1, 7, 50, 256])
def test_histograms_match_oracle(nbins):
    w = synth.cfg3(DEV, B=40)                                   # 2400 rows
    out = mars.verify_tree(w.logits, w.tok, w.parent, w.theta, debug=True)
    val = out["top2_val"]
    extra = torch.tensor([[5.0, 5.0], [-1.0, -2.0], [3.0, float("-inf")], [float("nan"), 1.0],
                          [float("inf"), 2.0], [0.0, 0.0], [30.0, 29.999], [15.0, -3.0]], device=DEV)
    val = torch.cat([val, extra]).contiguous()
    hist, outl = mars.top2_histograms(val, 10.0, 30.0, nbins)
    torch.cuda.synchronize()
    h_ref, o_ref = orc.histograms(val.cpu().numpy(), 10.0, 30.0, nbins)
    assert np.array_equal(hist.cpu().numpy().view(np.uint32), h_ref)
    assert np.array_equal(outl.cpu().numpy().view(np.uint32), o_ref)
    assert int(h_ref[1].sum()) > 2000 and h_ref[1][-max(1, nbins // 10):].sum() > 0     # low-margin rows exist


def test_histogram_argument_checks():
    v = torch.zeros((4, 2), device=DEV)
    with pytest.raises(mars.MarsError, match="unsupported"):
        mars.top2_histograms(v, 0.0, 1.0, 257)
    with pytest.raises(mars.MarsError, match="invalid argument"):
        mars.top2_histograms(v, 1.0, 1.0, 8)
    hist, outl = mars.top2_histograms(v[:0].contiguous(), 0.0, 1.0, 8)                  # no rows
    torch.cuda.synchronize()
    assert int(hist.sum()) == 0 and int(outl.sum()) == 0


def test_stream_read_probe_reads_every_word():
    """The read-only probe returns the maximum of the 32-bit words of the buffer, whatever the
    chunking -- which it can only do if every word was read."""
    g = torch.Generator().manual_seed(3)
    buf = torch.randint(0, 2 ** 30, (1 << 20,), generator=g, dtype=torch.int32)
    buf[777_777] = 2 ** 31 - 5
    d = buf.to("cuda:0")
    for chunk in (16, 4096, 303872, 1 << 22):
        out = mars.stream_read_probe(d, chunk)
        torch.cuda.synchronize()
        assert int(out.item()) == 2 ** 31 - 5, chunk
    assert int(mars.stream_read_probe(d[:777_000], 303872).item()) == int(buf[:777_000].max())
