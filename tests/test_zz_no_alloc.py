"""The allocation-free conv entry point (collected last on purpose).

Some users of the library cannot allocate device memory where they call it: they were handed an
input and an output buffer and nothing else (a plugin inside a host application, code living in a
fixed memory pool, a real-time loop).  idf_conv_rows_noalloc serves them from a fixed scratch array
inside the library.  Its results must equal those of the regular entry points, call after call,
even though every call reuses the same scratch and finds the previous call's leftovers in it.
"""
import gc

import numpy as np
import pytest
import torch

from paper_1804_10727_b200 import idf
from paper_1804_10727_b200.workloads import conv
from helpers import assert_close, rand_net

pytestmark = pytest.mark.gpu


def _regular(layer, x, w, b):
    net = idf.Net("f32", (layer,), x.shape[2], x.shape[3], x.shape[0], [w], [b])
    return idf.infer(net, x)


def _noalloc(layer, x, w, b):
    seg = idf.segments_from_maps(x, "f32").cuda()
    dw = torch.from_numpy(w).cuda()
    db = torch.from_numpy(b).cuda() if b is not None else None
    H = x.shape[1]
    rows = (H + 2 * layer.pad - layer.kh) // layer.stride + 1
    wo = 1 if x.shape[2] == 1 else (x.shape[2] + 2 * layer.pad - layer.kw) // layer.stride + 1
    out = torch.full((x.shape[0], rows, wo, layer.cout), float("nan"), device="cuda")
    gc.collect()                                            # (tensors of earlier tests must not be freed in between)
    before = torch.cuda.memory_allocated()
    got_rows = idf.conv_rows_noalloc(seg, dw, db, layer.stride, layer.pad, bool(layer.relu), out)
    assert torch.cuda.memory_allocated() == before          # torch's allocator was not touched either
    torch.cuda.synchronize()
    assert got_rows == rows
    return out.cpu().numpy()


def test_two_calls_in_a_row_match_the_regular_entry_point(orc):
    # first call: 3x3, stride 1, same padding; it leaves partial rows and its weights in the scratch
    l1 = conv(3, 8, 3, pad=1)
    x1, w1, b1 = rand_net("f32", (l1,), 21, 17, 3, S=4, seed=31)
    # second call: different shape, stride 2, no padding: must not see anything of the first
    l2 = conv(2, 5, 5, stride=2)
    x2, w2, b2 = rand_net("f32", (l2,), 30, 23, 2, S=3, seed=32)
    for layer, x, w, b in ((l1, x1, w1[0], b1[0]), (l2, x2, w2[0], b2[0]), (l1, x1, w1[0], None)):
        got = _noalloc(layer, x, w, b)
        want = _regular(layer, x, w, b)
        assert not np.isnan(got).any()
        assert_close(got, want, "noalloc vs regular entry point")
        # ... and both equal the CPU oracle's conventional result
        assert_close(got, orc.forward("f32", (layer,), x, [w], [b]), "noalloc vs oracle")


def test_sizes_beyond_the_built_in_scratch_are_refused():
    S, W, C = 64, 256, 64                                   # ring 3*64*256*64*4 B = 12 MiB > 8 MiB
    seg = torch.zeros((3, S, W, 2), device="cuda")
    w = torch.zeros((C, 3, 3, 2), device="cuda")
    out = torch.zeros((S, 1, W - 2, C), device="cuda")
    with pytest.raises(idf.IdfError) as e:
        idf.conv_rows_noalloc(seg, w, None, 1, 0, True, out)
    assert e.value.code == idf.ERR_CAPACITY and "scratch" in str(e.value)


def test_an_output_buffer_narrower_than_the_rows_is_refused_before_any_launch():
    # the C call sees only a pointer: the binding must not let a too-narrow buffer through (it would be overrun)
    seg = torch.zeros((6, 2, 20, 3), device="cuda")
    w = torch.zeros((4, 3, 3, 3), device="cuda")
    narrow = torch.zeros((2, 4, 17, 4), device="cuda")       # the layer emits rows of width 18
    with pytest.raises(AssertionError):
        idf.conv_rows_noalloc(seg, w, None, 1, 0, True, narrow)
    with pytest.raises(AssertionError):
        idf.conv_rows_noalloc(seg, w, torch.zeros(3, device="cuda"), 1, 0, True, torch.zeros((2, 4, 18, 4), device="cuda"))
