"""The range-checked build of the library (libidf_bounds.so, the same sources compiled with -DIDF_BOUNDS).

compute-sanitizer is not available where these tests run, so the library carries its own net: in this build every
index into a ring, a row buffer, shared memory or tensor memory is compared with the extent of what it addresses;
an index out of range is recorded in the handle's status word (idf_stream_status -> IDF_ERR_BOUNDS) and the access
skipped.  The small nets of the other tests - every kernel, every layer kind, awkward groupings of rows - run through
it here: results must still equal the oracle's (a skipped access would show) and the status must stay clean."""
import numpy as np
import pytest
import torch

from paper_1804_10727_b200 import idf
from paper_1804_10727_b200.workloads import Layer, conv, POOL
from helpers import SMALL_NETS, assert_close, assert_equal, rand_net, small_dims, with_path, with_shifts

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def bounds_library():
    regular = idf.LIB_PATH
    idf.use_library(idf.BOUNDS_LIB_PATH)
    yield
    idf.use_library(regular)


def _check(mode, got, want, what):
    if mode == "i8":
        assert_equal(got, want, what)
    elif mode == "f32":
        assert_close(got, want, what)
    else:
        err = np.abs(got - want)
        assert (err <= 1e-4 + 1e-3 * np.abs(want)).mean() > 0.97 and err.max() < 0.06, what


@pytest.mark.parametrize("name", list(SMALL_NETS))
@pytest.mark.parametrize("mode", ["f32", "bf16", "i8"])
def test_small_nets_through_the_range_checked_build(orc, name, mode):
    layers = SMALL_NETS[name]
    if mode == "i8":
        layers = with_shifts(layers, 8)
    H, W = small_dims(name)
    C0 = next(l.cin for l in layers if l.kind == "conv")
    x, ws, bs = rand_net(mode, layers, H, W, C0, S=5, seed=len(name))
    want = orc.forward(mode, layers, x, ws, bs)
    for chunks, rb, last in ((None, 0, False), ([1] * H, 0, True), ([5, 1, 3], 2, False), ([H - 1], 3, True)):
        net = idf.Net(mode, layers, W, C0, 5, ws, bs, row_block=rb)
        got = idf.infer(net, x, chunks=chunks, last=last)            # infer() ends with net.status(): raises on IDF_ERR_BOUNDS
        _check(mode, got, want, f"{name}/{mode}/chunks={chunks}/rb={rb}")
        net.close()


TC_NETS = [
    ("i8_conv_pool_conv", "i8", (conv(32, 64, 3, pad=1), POOL, conv(64, 32, 3, pad=1), POOL), 22, 40, 5),
    ("i8_valid_stride2", "i8", (conv(32, 32, 5, stride=2, pad=2), conv(32, 32, 3)), 31, 18, 3),
    ("bf16_pool_then_conv", "bf16", (conv(64, 64, 3, pad=1), POOL, conv(64, 16, 3, pad=1)), 16, 24, 5),
    ("i8_unfold_pool", "i8", (conv(16, 32, 3, pad=1), POOL), 15, 26, 7),
    ("i8_1d_chunks", "i8", (conv(32, 64, 9, stride=2, one_d=True), conv(64, 64, 9, one_d=True)), 700, 1, 40),
    ("i8_sparse_first", "i8", with_path((conv(2, 16, 3), POOL, conv(16, 8, 3, pad=1)), idf.PATH_SPARSE), 25, 18, 3),
    ("i8_wide_two_x_tiles", "i8", (conv(32, 16, 3, pad=1), POOL), 9, 224, 2),
]


@pytest.mark.parametrize("name,mode,layers,H,W,S", TC_NETS, ids=[c[0] for c in TC_NETS])
def test_tensor_core_and_sparse_kernels_through_the_range_checked_build(orc, name, mode, layers, H, W, S):
    if mode == "i8":
        layers = with_shifts(layers, 9)
    C0 = layers[0].cin
    x, ws, bs = rand_net(mode, layers, H, W, C0, S=S, seed=3 + len(name))
    want = orc.forward(mode, layers, x, ws, bs)
    for chunks, rb, last in ((None, 0, True), ([1] * min(H, 40), 0, False), ([3, 2, 5, 1], 3, True), ([H // 2 + 1], 64, False)):
        net = idf.Net(mode, layers, W, C0, S, ws, bs, row_block=rb)
        got = idf.infer(net, x, chunks=chunks, last=last)
        _check(mode, got, want, f"{name}/chunks={chunks}/rb={rb}")
        net.close()


def test_sinks_and_eager_mode_through_the_range_checked_build(orc):
    avg = Layer("avg")
    layers = with_shifts((conv(2, 6, 3), conv(6, 5, 3, pad=1), avg), 8)
    x, ws, bs = rand_net("i8", layers, 17, 12, 2, S=4, seed=4)
    want = orc.forward("i8", layers, x, ws, bs)
    net = idf.Net("i8", layers, 12, 2, 4, ws, bs, row_block=2)
    assert np.array_equal(idf.infer(net, x, chunks=[5, 1, 3]), want.astype(np.float32))
    net.close()
    layers = with_shifts(SMALL_NETS["same_pool"], 7)
    x, ws, bs = rand_net("i8", layers, 19, 14, 3, S=3, seed=6)
    net = idf.Net("i8", layers, 14, 3, 3, ws, bs, eager=True)
    assert_equal(idf.infer(net, x, chunks=[4, 1]), orc.forward("i8", layers, x, ws, bs), "eager")
    net.close()


def test_the_range_checked_build_exports_the_same_calls():
    import ctypes
    lib = ctypes.CDLL(str(idf.BOUNDS_LIB_PATH))
    for name in idf.EXPORTS:
        assert hasattr(lib, name), name
