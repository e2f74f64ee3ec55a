"""Parity at the workloads' full sizes, in the launch configuration bench.py times (all streams of
the batch, all segments and the end of input in one push_last with the default row block).  Streams are independent, so the oracle
is run only on a sample of streams and compared with exactly those streams of the device result;
the rest is covered by properties that hold at any size (shape, finiteness, batch-mate independence)."""
import numpy as np
import pytest
import torch

from paper_1804_10727_b200 import idf, workloads
from helpers import assert_close, assert_equal

pytestmark = pytest.mark.gpu

# (workload, sampled streams)
CASES = [("toy1d", [0]), ("mnist2d", [0, 1, 2, 3, 1000, 2047, 4095]), ("audio1d", [0, 511, 1023]),
         ("vgg2d", [0, 63]), ("events2d", [0, 2047])]


@pytest.mark.parametrize("name,sample", CASES, ids=[c[0] for c in CASES])
def test_full_size_sampled_streams_match_oracle(orc, name, sample):
    w = workloads.get(name)
    ws, bs = workloads.make_params(w)
    net = idf.net_from_workload(w, ws, bs)
    # the device runs the whole batch; the inputs of the sampled streams are regenerated for the oracle
    x = workloads.make_input(w)
    seg = idf.segments_from_maps(x, w.dtype).cuda()
    out = net.alloc_out(w.H)
    net.open()
    rows = net.push_last(seg, out)
    tc = net.status()
    assert rows == net.out_shape(w.H)[0]
    got_all = out[:, :rows]
    if w.dtype != "i8":
        assert bool(torch.isfinite(got_all).all())
    if w.dtype in ("bf16", "i8"):
        assert any(t > 0 for t in tc), "no layer took the tensor-core path"
    for s in sample:
        xs = workloads.make_input(w, first=s, count=1)
        assert np.array_equal(xs[0], x[s])                      # same seeded data on both sides
        want = orc.forward(w.dtype, w.layers, xs, ws, bs)[0]
        got = got_all[s].cpu().numpy()
        if w.dtype == "i8":
            assert_equal(got, want, f"{name} stream {s}")
        elif w.dtype == "f32":
            assert_close(got, want, f"{name} stream {s}")
        else:
            # bf16 nets end to end: statistical criterion (every hidden activation is a rounding decision
            # on an fp32 sum in tensor-core order); the strict per-layer comparison is in test_parity_gpu.py
            err = got - want
            rel_rms = np.sqrt((err ** 2).mean() / (want ** 2).mean())
            assert rel_rms < 2.0 ** -7, (name, s, rel_rms)
            assert np.abs(err).max() < 2.0 ** -3 * np.abs(want).max()


def test_full_size_state_bytes_are_the_ring_formula():
    want = {"toy1d": 240, "mnist2d": 18432, "audio1d": 17024, "vgg2d": 1247232 + 14336, "events2d": 261248}
    for name, b in want.items():
        w = workloads.get(name)
        net = idf.net_from_workload(w, *workloads.make_params(w))
        assert net.state_bytes == b
