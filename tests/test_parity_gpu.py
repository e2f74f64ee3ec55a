"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Integer nets must match bit for bit; float nets within |g - o| <= 1e-4 + 1e-3 |o|."""
import numpy as np
import pytest
import torch

from paper_1804_10727_b200 import idf, workloads
from paper_1804_10727_b200.workloads import Layer, conv, POOL
from helpers import (SMALL_NETS, assert_bf16_end_to_end, assert_close, assert_equal, rand_net, small_dims, with_path, with_shifts)

pytestmark = pytest.mark.gpu


def _run(mode, layers, x, ws, bs, chunks=None, row_block=0, last=False):
    S, H, W, C = x.shape
    net = idf.Net(mode, layers, W, C, S, ws, bs, row_block=row_block)
    try:
        return idf.infer(net, x, chunks=chunks, last=last), net
    finally:
        pass


def _compare(mode, got, want, what=""):
    if mode == "i8":
        assert_equal(got, want, what)
    else:
        assert_close(got, want, what)


def _random_chunks(H, seed):
    r = np.random.default_rng(seed)
    out, left = [], H
    while left > 0:
        n = int(r.integers(1, 8))
        out.append(min(n, left))
        left -= out[-1]
    return out


# ---- small nets: every layer kind, stride, padding, 1D and 2D, every type ----------------------
@pytest.mark.parametrize("name", list(SMALL_NETS))
@pytest.mark.parametrize("mode", ["f32", "bf16", "i8"])
def test_small_nets_match_oracle(orc, name, mode):
    layers = SMALL_NETS[name]
    if mode == "i8":
        layers = with_shifts(layers, 8)
    H, W = small_dims(name)
    C0 = next(l.cin for l in layers if l.kind == "conv")
    x, ws, bs = rand_net(mode, layers, H, W, C0, S=5, seed=len(name))
    want = orc.forward(mode, layers, x, ws, bs)
    if mode == "bf16":
        # two conv layers at most between the input and an unrounded output: a rounding flip of a
        # single hidden activation is possible, so allow a few elements at one bf16 ulp of slack
        got, _ = _run(mode, layers, x, ws, bs)
        err = np.abs(got - want)
        ok = err <= 1e-4 + 1e-3 * np.abs(want)
        assert ok.mean() > 0.97 and err.max() < 0.05, (ok.mean(), err.max())
        return
    for chunks, rb in ((None, 0), ([1] * H, 0), (_random_chunks(H, 1), 3), (None, 1), ([H], 64)):
        got, _ = _run(mode, layers, x, ws, bs, chunks=chunks, row_block=rb)
        _compare(mode, got, want, f"{name}/{mode}/chunks={chunks and len(chunks)}/rb={rb}")


# ---- the end of input given with the last segments (push_last) equals push + finish -------------
@pytest.mark.parametrize("name", list(SMALL_NETS))
@pytest.mark.parametrize("mode", ["f32", "i8"])
def test_push_last_equals_push_then_finish(orc, name, mode):
    layers = SMALL_NETS[name]
    if mode == "i8":
        layers = with_shifts(layers, 8)
    H, W = small_dims(name)
    C0 = next(l.cin for l in layers if l.kind == "conv")
    x, ws, bs = rand_net(mode, layers, H, W, C0, S=4, seed=7 + len(name))
    want = orc.forward(mode, layers, x, ws, bs)
    for chunks, rb in ((None, 0), ([H - 1], 0), (_random_chunks(H, 2), 3), ([1] * H, 1), (None, 2)):
        got, _ = _run(mode, layers, x, ws, bs, chunks=chunks, row_block=rb, last=True)
        _compare(mode, got, want, f"push_last {name}/{mode}/chunks={chunks and len(chunks)}/rb={rb}")


def test_push_last_on_tensor_core_layers_matches_oracle(orc):
    # same-padded dense int8 layers wide enough for the tensor-core kernel: the rows that end on bottom
    # padding are completed by the launch that applies the last input rows
    layers = with_shifts((conv(16, 32, 3, pad=1), conv(32, 32, 3, pad=1), POOL, conv(32, 16, 3, pad=1)), 8)
    x, ws, bs = rand_net("i8", layers, 21, 40, 16, S=5, seed=11)
    want = orc.forward("i8", layers, x, ws, bs)
    for chunks, rb in ((None, 0), ([20], 0), ([7, 7], 4), (None, 5)):
        got, net = _run("i8", layers, x, ws, bs, chunks=chunks, row_block=rb, last=True)
        assert_equal(got, want, f"push_last tc chunks={chunks} rb={rb}")
        assert any(t > 0 for t in net.status()), "no layer took the tensor-core path"
    net = idf.Net("i8", layers, 40, 16, 5, ws, bs)
    seg = idf.segments_from_maps(x, "i8").cuda()
    out = net.alloc_out(21)
    net.open()
    assert net.push_last(seg, out) == want.shape[1]
    with pytest.raises(idf.IdfError) as e:                      # the stream has ended
        net.push(seg, out)
    assert e.value.code == idf.ERR_STATE
    net.open()
    net.push(seg, out)
    assert net.push_last(seg[:0], out) == want.shape[1]         # no segments: the same as finish
    assert_equal(out.cpu().numpy(), want, "push + empty push_last")
    out.zero_()
    net.reset()                                                 # new streams, parameters kept
    assert net.push_last(seg, out) == want.shape[1]
    assert_equal(out.cpu().numpy(), want, "reset + push_last")
    net.reset()
    net.push(seg[:9], out)                                      # abandoned half way ...
    net.reset()                                                 # ... and started again
    out.zero_()
    net.push(seg[:13], out)
    net.push_last(seg[13:], out)
    assert_equal(out.cpu().numpy(), want, "reset in the middle of streams")


@pytest.mark.parametrize("mode", ["f32", "i8"])
def test_chunking_invariance_is_bit_exact_for_ints(orc, mode):
    layers = SMALL_NETS["same_pool"]
    if mode == "i8":
        layers = with_shifts(layers, 8)
    x, ws, bs = rand_net(mode, layers, 33, 21, 3, S=3, seed=3)
    a, _ = _run(mode, layers, x, ws, bs, chunks=None)
    b, _ = _run(mode, layers, x, ws, bs, chunks=[1] * 33)
    c, _ = _run(mode, layers, x, ws, bs, chunks=_random_chunks(33, 9), row_block=5)
    if mode == "i8":
        assert np.array_equal(a, b) and np.array_equal(a, c)
    else:
        assert_close(b, a); assert_close(c, a)


def test_streams_are_independent(orc):
    layers = with_shifts(SMALL_NETS["stride2"], 8)
    x, ws, bs = rand_net("i8", layers, 20, 16, 2, S=6, seed=11)
    base, _ = _run("i8", layers, x, ws, bs)
    perm = np.array([3, 0, 5, 1, 4, 2])
    got, _ = _run("i8", layers, x[perm], ws, bs)
    assert np.array_equal(got, base[perm])
    x2 = x.copy(); x2[1:] = 0                      # batch mates changed: stream 0 must not notice
    got2, _ = _run("i8", layers, x2, ws, bs)
    assert np.array_equal(got2[0], base[0])
    lf = SMALL_NETS["same_pool"]
    xf, wf, bf = rand_net("f32", lf, 16, 12, 3, S=4, seed=12)
    basef, _ = _run("f32", lf, xf, wf, bf)
    xf2 = xf.copy(); xf2[1:] = 0
    gotf, _ = _run("f32", lf, xf2, wf, bf)
    assert np.array_equal(gotf[0], basef[0])      # bit-exact: the reduction order does not depend on batch mates


def test_output_rows_appear_progressively_and_causally(orc):
    layers = SMALL_NETS["same_pool"]
    x, ws, bs = rand_net("f32", layers, 24, 12, 3, S=2, seed=4)
    want = orc.forward("f32", layers, x, ws, bs)
    net = idf.Net("f32", layers, 12, 3, 2, ws, bs)
    seg = idf.segments_from_maps(x, "f32").cuda()
    out = net.alloc_out(24)
    net.open()
    seen = 0
    for r in range(24):
        seen += net.push(seg[r:r + 1], out)
        # output row o needs input rows up to 4 o + 6 (two same-padded 3x3 convs, two pools)
        assert seen == max(0, (r - 6) // 4 + 1)
        torch.cuda.synchronize()
        if seen:
            assert_close(out[:, :seen].cpu().numpy(), want[:, :seen])
    total = net.finish(out)
    assert total == want.shape[1]
    assert_close(out.cpu().numpy(), want)


def test_zero_input_gives_zero_events_and_zero_output(orc):
    layers = with_path(with_shifts((conv(2, 8, 3), conv(8, 8, 3)), 4), idf.PATH_SPARSE)
    x, ws, _ = rand_net("i8", layers, 12, 12, 2, S=3, bias=False, seed=2)
    got, net = _run("i8", layers, np.zeros_like(x), ws, None)
    assert not got.any()
    assert net.event_counts() == [0, 0]


def test_sparse_path_counts_exactly_the_nonzero_events_and_equals_dense(orc):
    base = with_shifts((conv(2, 16, 3, pad=1), conv(16, 8, 3, stride=2), POOL), 6)
    x, ws, bs = rand_net("i8", base, 30, 40, 2, S=4, seed=8, zero_frac=0.9)
    want = orc.forward("i8", base, x, ws, bs)
    dense, _ = _run("i8", with_path(base, idf.PATH_DENSE), x, ws, bs)
    sparse, net = _run("i8", with_path(base, idf.PATH_SPARSE), x, ws, bs, chunks=_random_chunks(30, 2), row_block=4)
    assert_equal(dense, want); assert_equal(sparse, want)
    ev = net.event_counts()
    assert ev[0] == int((x != 0).sum())
    hidden = orc.forward("i8", base[:1], x, ws[:1], bs[:1])
    assert ev[1] == int((hidden != 0).sum())
    # float nets may take the sparse path too (atomics: order differs, tolerance applies)
    lf = with_path((conv(1, 8, 3), conv(8, 4, 3)), idf.PATH_SPARSE)
    xf, wf, bf = rand_net("f32", lf, 20, 20, 1, S=2, seed=5)
    xf[np.random.default_rng(0).random(xf.shape) < 0.8] = 0
    gotf, _ = _run("f32", lf, xf, wf, bf)
    assert_close(gotf, orc.forward("f32", lf, xf, wf, bf))


def test_wide_rows_take_the_global_ring_and_long_event_lists(orc):
    # ring of 3 * 1200 * 48 * 4 B exceeds shared memory; 1200 * 2 components exceed one list pass
    layers = with_path(with_shifts((conv(2, 48, 3),), 5), idf.PATH_SPARSE)
    x, ws, bs = rand_net("i8", layers, 7, 1202, 2, S=2, seed=6, zero_frac=0.05)
    got, net = _run("i8", layers, x, ws, bs)
    assert_equal(got, orc.forward("i8", layers, x, ws, bs))
    assert net.event_counts()[0] == int((x != 0).sum())


def test_capacity_and_state_errors():
    layers = (conv(2, 2, 3),)
    x, ws, bs = rand_net("f32", layers, 10, 8, 2, S=1, seed=1)
    net = idf.Net("f32", layers, 8, 2, 1, ws, bs)
    seg = idf.segments_from_maps(x, "f32").cuda()
    small = torch.zeros((1, 3, 6, 2), device="cuda")
    net.open()
    net.push(seg[:5], small)                                   # rows 0..2 fit
    with pytest.raises(idf.IdfError) as e:
        net.push(seg[5:], small)                               # row 3 would not
    assert e.value.code == idf.ERR_CAPACITY
    out = net.alloc_out(10)
    net.open()
    net.push(seg, out)
    net.finish(out)
    with pytest.raises(idf.IdfError) as e:
        net.push(seg, out)
    assert e.value.code == idf.ERR_STATE
    net.open()                                                 # a finished handle can be reopened
    assert net.push(seg, out) == 8


# ---- the five workloads (reduced stream counts; full shapes) -----------------------------------
CASES = [("toy1d", 1, None), ("mnist2d", 96, None), ("audio1d", 3, 3000), ("vgg2d", 2, None), ("events2d", 3, None)]


@pytest.mark.parametrize("name,S,H", CASES)
def test_workloads_match_oracle(orc, name, S, H):
    w = workloads.get(name, n_streams=S, H=H)
    x = workloads.make_input(w)
    ws, bs = workloads.make_params(w)
    want = orc.forward(w.dtype, w.layers, x, ws, bs)
    net = idf.net_from_workload(w, ws, bs)
    got = idf.infer(net, x)
    assert got.shape == want.shape
    if w.dtype == "i8":
        assert_equal(got, want, name)
    elif w.dtype == "f32":
        assert_close(got, want, name)
    else:
        # bf16 nets: every hidden activation is a rounding decision taken on an fp32 sum whose
        # order differs from the oracle's float64 sum; a decision that falls on the other side
        # moves that activation by one bf16 ulp (2^-8 relative).  The end-to-end comparison is
        # therefore statistical; the strict tolerance is checked layer by layer below.
        assert_bf16_end_to_end(name, got, want, name)


@pytest.mark.parametrize("name,S,H", [("audio1d", 3, 3000), ("vgg2d", 2, None)])
def test_bf16_workloads_layer_by_layer_strict(orc, name, S, H):
    """Each conv layer of the bf16 workloads, fed the oracle's own (bf16-valued) input map of that
    layer, must reproduce the oracle's unrounded output within the strict tolerance."""
    w = workloads.get(name, n_streams=S, H=H)
    x = workloads.make_input(w)
    ws, bs = workloads.make_params(w)
    maps = orc.forward(w.dtype, w.layers, x, ws, bs, return_all=True)
    for i, l in enumerate(w.layers):
        if l.kind != "conv":
            continue
        a = maps[i].astype(np.float32)
        want = orc.conv_layer("bf16", l, a, ws[i], bs[i])            # unrounded f(c)
        net = idf.Net("bf16", (l,), a.shape[2], a.shape[3], S, [ws[i]], [bs[i]])
        got = idf.infer(net, a)
        assert_close(got, want, f"{name} layer {i}")
        net.close()


# ---- idf_run_host: host buffers in and out, copies pipelined with the compute ---------------------
@pytest.mark.parametrize("name,mode,rb", [("same_pool", "f32", 4), ("stride2", "i8", 3), ("oned_k9", "f32", 16), ("valid3", "bf16", 0)])
def test_run_host_equals_device_path(orc, name, mode, rb):
    layers = SMALL_NETS[name]
    if mode == "i8":
        layers = with_shifts(layers, 8)
    H, W = small_dims(name)
    C0 = next(l.cin for l in layers if l.kind == "conv")
    x, ws, bs = rand_net(mode, layers, H, W, C0, S=5, seed=21)
    # (run_host feeds the net half a row block at a time, the first and the last step half of that again when there
    # are at least three steps' worth of rows; fp32 sums depend on how the rows are grouped into pushes)
    chunks = None
    if rb:
        pipe = max(rb // 2, 1)
        edge = pipe // 2 if (H >= 3 * pipe and pipe >= 2) else 0
        chunks, pos = ([edge] if edge else []), edge
        while pos < H - edge:
            n = min(pipe, H - edge - pos)
            chunks.append(n); pos += n
        if edge:
            chunks.append(edge)
    ref, _ = _run(mode, layers, x, ws, bs, row_block=rb, chunks=chunks, last=True)
    net = idf.Net(mode, layers, W, C0, 5, ws, bs, row_block=rb)
    h_seg = idf.segments_from_maps(x, net.dtype).pin_memory()
    d_seg = torch.empty_like(h_seg, device="cuda")
    d_out = net.alloc_out(H)
    h_out = torch.full(d_out.shape, 77, dtype=d_out.dtype).pin_memory()
    net.open()
    for _ in range(2):                                  # twice: the second call reuses streams, events and buffers
        net.reset()
        h_out.fill_(77)
        rows = net.run_host(h_seg, d_seg, h_out, d_out)
        net.status()
        assert rows == ref.shape[1]
        assert np.array_equal(h_out[:, :rows].numpy().view(np.uint8), ref.view(np.uint8)), (name, mode)
    net.close()
