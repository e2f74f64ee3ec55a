"""Host-side behaviour of the C-ABI library that needs no GPU: exported symbols, spec validation,
shape inference, the state-size formula and its invariants, the call-order state machine."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_1804_10727_b200 import idf, workloads
from paper_1804_10727_b200.workloads import Layer, conv, POOL

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _mk(layers, dtype="f32", in_w=8, in_c=None, S=2, row_block=0):
    in_c = in_c or next(l.cin for l in layers if l.kind == "conv")
    ws = [None if l.kind != "conv" else np.zeros((l.cout, l.kh, l.kw, l.cin), dtype=np.float32) for l in layers]
    return idf.Net(dtype, layers, in_w, in_c, S, ws, None, row_block=row_block)


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "idf.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(idf_[a-z_]+)\s*\(", hdr))
    assert declared == set(idf.EXPORTS), declared ^ set(idf.EXPORTS)
    L = ctypes.CDLL(str(idf.LIB_PATH))
    for name in declared:
        assert hasattr(L, name), name


def test_state_bytes_of_the_five_workloads():
    # sum over conv layers of ceil(Kh/stride) rows * Wout * Cout * 4 B, plus one row per pool
    want = {"toy1d": 240, "mnist2d": 18432, "audio1d": 17024, "events2d": 261248,
            # the last pool of vgg2d holds unrounded fp32 values: 28*256*4 instead of *2 bytes
            "vgg2d": 1247232 + 28 * 256 * 2}
    for name, b in want.items():
        w = workloads.get(name, n_streams=3)
        ws, bs = workloads.make_params(w)
        net = idf.net_from_workload(w, ws, bs)
        assert net.state_bytes == b, name
        assert net.workspace_bytes >= 3 * b
        net.close()


def test_state_is_constant_in_length_and_linear_in_width():
    w1 = workloads.get("audio1d", n_streams=1)
    ws, bs = workloads.make_params(w1)
    net = idf.net_from_workload(w1, ws, bs)
    # the handle does not even know the input length: nothing to vary; out rows grow, state does not
    assert net.out_shape(16000)[0] == 1969 and net.out_shape(4_000_000)[0] > 400_000
    assert net.state_bytes == 17024
    sizes = []
    for W in (56, 112, 224):
        w = workloads.get("vgg2d", n_streams=1, W=W)
        net = idf.net_from_workload(w, *workloads.make_params(w))
        sizes.append(net.state_bytes)
    assert sizes[1] == 2 * sizes[0] and sizes[2] == 4 * sizes[0]      # memory ~ sqrt(N) for a square image


def test_fig1_ring_count_is_seven():
    # two k=3 conv layers with one channel keep 3 + 3 state words; the averaging output unit of
    # Fig. 1 adds one more (it is not part of this library), 7 in total
    seven = int([l for l in open(os.path.join(ROOT, "tests", "golden", "fig1_state_count.txt")) if l[0] != "#"][0])
    net = _mk((conv(1, 1, 3, one_d=True), conv(1, 1, 3, one_d=True)), in_w=1)
    assert net.state_bytes // 4 + 1 == seven
    # ... and with the averaging unit as the library's global-average sink the count is the library's own
    net = _mk((conv(1, 1, 3, one_d=True), conv(1, 1, 3, one_d=True), Layer("avg")), in_w=1)
    assert net.state_bytes == 4 * seven


def test_sink_layers_shapes_and_state():
    # global average: one output row of width 1, one state word per channel, only as the last layer
    net = _mk((conv(2, 6, 3), POOL, Layer("avg")), in_w=12, in_c=2)
    assert net.out_shape(0) == (0, 1, 6) and net.out_shape(5) == (1, 1, 6) and net.out_shape(500) == (1, 1, 6)
    assert net.state_bytes == 3 * 10 * 6 * 4 + 5 * 6 * 4 + 6 * 4
    with pytest.raises(idf.IdfError) as e:
        _mk((conv(2, 6, 3), Layer("avg"), conv(6, 2, 3)), in_w=12, in_c=2)
    assert e.value.code == idf.ERR_SPEC
    # a fully connected layer over a 7 x 9 x 6 map is a conv layer with kh = 7, kw = 9, stride = 7: one ring row
    fc = Layer("conv", 6, 10, 7, 9, 7, 0, 0, 0, 0)
    net = _mk((conv(2, 6, 3), fc), in_w=11, in_c=2)
    assert net.out_shape(9) == (1, 1, 10) and net.out_shape(8) == (0, 1, 10)
    assert net.state_bytes == 3 * 9 * 6 * 4 + 10 * 4


def test_out_shape_follows_the_floor_formula():
    net = _mk((conv(2, 4, 3, stride=2, pad=1), POOL, conv(4, 4, 3)), in_w=20)
    for H in (0, 1, 5, 17, 64):
        h = (H + 2 - 3) // 2 + 1 if H > 0 else 0
        h = h // 2
        h = h - 2 if h >= 3 else 0
        assert net.out_shape(H) == (h, (((20 + 2 - 3) // 2 + 1) // 2) - 2, 4), H


@pytest.mark.parametrize("bad,code", [
    ((conv(3, 4, 3), conv(5, 4, 3)), idf.ERR_SPEC),                       # channel mismatch
    ((Layer("conv", 2, 4, 0, 3, 1, 0, 1, 0, 0),), idf.ERR_SPEC),           # kh = 0
    ((conv(2, 4, 3, stride=4),), idf.ERR_SPEC),                            # stride > kh
    ((conv(2, 4, 3, pad=3),), idf.ERR_SPEC),                               # pad >= kh
    ((POOL,), idf.ERR_SPEC),                                               # no conv layer
    ((conv(2, 4, 3, shift=31),), idf.ERR_SPEC),
    ((Layer("conv", 2, 4, 3, 3, 1, 0, 1, 0, 7),), idf.ERR_SPEC),           # unknown path
])
def test_bad_specs_are_rejected(bad, code):
    with pytest.raises(idf.IdfError) as e:
        _mk(bad, in_c=2)
    assert e.value.code == code and str(e.value)


def test_bad_arguments_and_call_order():
    L = idf.lib()
    assert L.idf_net_create(None, None, None, None) == idf.ERR_ARG
    assert L.idf_net_state_bytes(None) == 0 and L.idf_net_workspace_bytes(None) == 0
    with pytest.raises(idf.IdfError) as e:
        idf.Net("f32", (conv(2, 2, 3),), 0, 2, 1, [np.zeros((2, 3, 3, 2), np.float32)])
    assert e.value.code == idf.ERR_SPEC
    with pytest.raises(idf.IdfError) as e:
        idf.Net("f32", (conv(2, 2, 3),), 8, 2, 1, [None])                  # weights missing
    assert e.value.code == idf.ERR_ARG
    net = _mk((conv(2, 2, 3),))
    em = ctypes.c_int()
    # push / finish before open: refused on the host, nothing is enqueued
    assert L.idf_stream_push(net._h, 256, 1, 256, 4, ctypes.byref(em)) == idf.ERR_STATE
    assert L.idf_stream_finish(net._h, 256, 4, None) == idf.ERR_STATE
    assert L.idf_stream_push_last(net._h, 256, 1, 256, 4, None) == idf.ERR_STATE
    assert L.idf_stream_reset(net._h) == idf.ERR_STATE
    assert b"before stream_open" in L.idf_last_error()
    assert L.idf_stream_set_out_base(net._h, 0) == idf.ERR_STATE and L.idf_stream_set_out_base(None, 0) == idf.ERR_ARG
    assert L.idf_stream_open(net._h, None, 0, None) == idf.ERR_ARG
    assert L.idf_stream_open(net._h, 256, 16, None) == idf.ERR_CAPACITY
    assert L.idf_stream_open(net._h, 257, 1 << 30, None) == idf.ERR_ARG    # misaligned workspace


def test_snapshot_size_and_call_order():
    L = idf.lib()
    assert L.idf_state_snapshot_bytes(None) == 0
    w = workloads.get("mnist2d", n_streams=3)
    net = idf.net_from_workload(w, *workloads.make_params(w))
    n = L.idf_state_snapshot_bytes(net._h)
    # header + three words per layer + every layer's state of all streams, each rounded up to 256 bytes
    assert 3 * net.state_bytes <= n <= 3 * net.state_bytes + 256 * len(w.layers) + 64 + 24 * len(w.layers)
    buf = (ctypes.c_ubyte * n)()
    assert L.idf_state_save(None, buf, n) == idf.ERR_ARG
    assert L.idf_state_save(net._h, None, n) == idf.ERR_ARG
    assert L.idf_state_save(net._h, buf, n) == idf.ERR_STATE            # no open streams
    assert L.idf_state_restore(net._h, buf, n) == idf.ERR_STATE          # no workspace bound
    assert L.idf_state_restore(net._h, None, n) == idf.ERR_ARG


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(idf, "_lib", None)
    monkeypatch.setattr(idf, "LIB_PATH", tmp_path / "libidf.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        idf.lib()
