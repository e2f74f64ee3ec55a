"""Output sinks: the global-average unit of the paper's Fig. 1 and a fully connected output layer (the ten
output units of its experiment) fed incrementally, row by row, against the CPU oracle; and the running
output read between pushes against the oracle's result on the rows that have arrived."""
import numpy as np
import pytest
import torch

from paper_1804_10727_b200 import idf
from paper_1804_10727_b200.workloads import Layer, conv, POOL
from helpers import assert_close, assert_equal, rand_net, with_shifts

pytestmark = pytest.mark.gpu

AVG = Layer("avg")


def _fc(cin, n_out, h, w, relu=0, shift=0):
    return Layer("conv", cin, n_out, h, w, h, 0, relu, shift, 0)


AVG_NETS = {
    "conv_avg": ((conv(2, 6, 3), conv(6, 5, 3, pad=1), AVG), 17, 12),
    "pool_avg": ((conv(3, 8, 3, pad=1), POOL, conv(8, 4, 3), AVG), 21, 14),
    "oned_avg": ((conv(1, 4, 9, stride=2, one_d=True), conv(4, 7, 5, one_d=True), AVG), 90, 1),
    "wide_avg": ((conv(16, 32, 3, pad=1), conv(32, 32, 3, pad=1), POOL, AVG), 16, 16),     # tensor-core layers in bf16/i8
}


@pytest.mark.parametrize("name", list(AVG_NETS))
@pytest.mark.parametrize("mode", ["f32", "bf16", "i8"])
def test_global_average_sink_matches_oracle(orc, name, mode):
    layers, H, W = AVG_NETS[name]
    if mode == "i8":
        layers = with_shifts(layers, 8)
    C0 = layers[0].cin
    x, ws, bs = rand_net(mode, layers, H, W, C0, S=6, seed=3)
    want = orc.forward(mode, layers, x, ws, bs)
    assert want.shape == (6, 1, 1, layers[-2].cout if layers[-2].kind == "conv" else layers[-3].cout)
    for chunks, rb, last in ((None, 0, False), ([1] * H, 0, True), ([5, 1, 3], 2, False), ([H - 1], 0, True)):
        net = idf.Net(mode, layers, W, C0, 6, ws, bs, row_block=rb)
        got = idf.infer(net, x, chunks=chunks, last=last)
        assert got.dtype == np.float32 and got.shape == want.shape
        if mode == "i8":
            # the sum is exact in int32 and divided once in double precision: the nearest fp32 of the exact mean
            assert np.array_equal(got, want.astype(np.float32)), (name, chunks)
        elif mode == "f32":
            assert_close(got, want, f"{name}/{mode}")
        else:
            assert np.abs(got - want).max() <= 2.0 ** -7 * np.abs(want).max(), (name, np.abs(got - want).max())
        net.close()


@pytest.mark.parametrize("mode", ["f32", "i8"])
def test_running_average_between_pushes(orc, mode):
    """After every push the output is the mean over the rows of the last map that are complete by then."""
    layers = (conv(2, 5, 3), conv(5, 4, 3, stride=2), AVG)
    if mode == "i8":
        layers = with_shifts(layers, 8)
    H, W, S = 23, 11, 4
    x, ws, bs = rand_net(mode, layers, H, W, 2, S=S, seed=9)
    full = orc.forward(mode, layers, x, ws, bs, return_all=True)[-2]          # the map the sink averages
    net = idf.Net(mode, layers, W, 2, S, ws, bs)
    seg = idf.segments_from_maps(x, net.dtype).cuda()
    out = net.alloc_out(H)
    net.open()
    for r in range(H):
        em = net.push(seg[r:r + 1].contiguous(), out)
        q = r + 1 - 3                                   # rows of the first layer complete after r + 1 segments ...
        k1 = 0 if q < 0 else q + 1
        q = k1 - 3
        k2 = 0 if q < 0 else q // 2 + 1                 # ... and of the second
        if k2 == 0:
            assert em == 0
            continue
        got = out[:, 0].cpu().numpy().reshape(S, -1)
        want = full[:, :k2].astype(np.float64).mean(axis=(1, 2))
        if mode == "i8":
            assert np.array_equal(got, want.astype(np.float32)), r
        else:
            assert_close(got, want, f"after {r + 1} segments")
    assert net.finish(out) == 1
    net.close()


@pytest.mark.parametrize("mode", ["f32", "bf16", "i8"])
def test_fully_connected_output_layer(orc, mode):
    """A classifier-shaped net: conv, conv, pool, ten fully connected output units over the whole pooled map."""
    H = W = 14
    layers = (conv(1, 8, 3), conv(8, 16, 3), POOL, _fc(16, 10, 5, 5, shift=0))
    if mode == "i8":
        layers = with_shifts(layers[:3], 8) + (_fc(16, 10, 5, 5, shift=10),)
    x, ws, bs = rand_net(mode, layers, H, W, 1, S=7, seed=5)
    want = orc.forward(mode, layers, x, ws, bs)
    assert want.shape == (7, 1, 1, 10)
    for chunks, rb in ((None, 0), ([1] * H, 1), ([4, 3], 0)):
        net = idf.Net(mode, layers, W, 1, 7, ws, bs, row_block=rb)
        assert net.state_bytes == (3 * 12 * 8 + 3 * 10 * 16) * 4 + 5 * 16 * {"f32": 4, "bf16": 2, "i8": 1}[mode] + 10 * 4
        got = idf.infer(net, x, chunks=chunks)
        if mode == "i8":
            assert_equal(got, want, "fc/i8")
        elif mode == "f32":
            assert_close(got, want, "fc/f32")
        else:
            assert np.abs(got - want).max() <= 2.0 ** -6 * np.abs(want).max()
        net.close()


def test_sink_state_survives_a_snapshot(orc):
    layers = with_shifts((conv(2, 6, 3), conv(6, 5, 3, pad=1), AVG), 8)
    H, W, S = 17, 12, 3
    x, ws, bs = rand_net("i8", layers, H, W, 2, S=S, seed=4)
    want = orc.forward("i8", layers, x, ws, bs)
    a = idf.Net("i8", layers, W, 2, S, ws, bs)
    b = idf.Net("i8", layers, W, 2, S, ws, bs)
    seg = idf.segments_from_maps(x, a.dtype).cuda()
    out_a, out_b = a.alloc_out(H), b.alloc_out(H)
    a.open(); b.open()
    a.push(seg[:9].contiguous(), out_a)
    snap = a.save_state()
    b.restore_state(snap)
    assert b.push_last(seg[9:].contiguous(), out_b) == 1
    assert np.array_equal(out_b.cpu().numpy(), want.astype(np.float32))
    a.close(); b.close()


def test_mnist_shaped_classifier_many_streams(orc):
    """The paper's experiment in shape: 28x28 images fed row by row through the mnist2d conv stack and ten fully
    connected output units (random weights: accuracy is not the point), 512 streams, int8, bit-exact."""
    from paper_1804_10727_b200 import workloads
    w = workloads.get("mnist2d", n_streams=512)
    x = workloads.make_input(w)
    ws, bs = workloads.make_params(w)
    layers = tuple(w.layers) + (_fc(32, 10, 10, 10, shift=11),)
    r = np.random.default_rng(12)
    ws = list(ws) + [r.integers(-127, 128, size=(10, 10, 10, 32)).astype(np.int8)]
    bs = list(bs) + [r.integers(-2000, 2000, size=(10,)).astype(np.int32)]
    want = orc.forward("i8", layers, x, ws, bs)
    assert want.shape == (512, 1, 1, 10) and len(np.unique(want)) > 20          # the logits are not saturated
    net = idf.Net("i8", layers, w.W, w.C, 512, ws, bs)
    got = idf.infer(net, x, chunks=[1] * w.H, last=True)                        # one image row per push
    assert_equal(got, want, "classifier")
    assert net.state_bytes == 18432 + 10 * 4
    net.close()
