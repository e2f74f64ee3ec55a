"""Checkpointing running streams (idf_state_save / idf_state_restore): streams taken off the device
between two pushes and continued on another handle give the same output, bit for bit, as streams that
were never interrupted, and that output matches the CPU oracle."""
import ctypes

import numpy as np
import pytest
import torch

from paper_1804_10727_b200 import idf, workloads
from helpers import SMALL_NETS, assert_close, assert_equal, rand_net, small_dims, with_shifts

pytestmark = pytest.mark.gpu


def _segments(net, x):
    return idf.segments_from_maps(x, net.dtype).cuda()


def _rows_complete_after(layers, n_seg):
    """Output rows of the net whose last tap lies within the first n_seg segments (no end of input yet)."""
    r = n_seg
    for l in layers:
        if l.kind == "conv":
            q = r + l.pad - l.kh
            r = 0 if q < 0 else q // l.stride + 1
        else:
            r //= 2
    return r


def _interrupted(mode, layers, x, ws, bs, cut, row_block=0, pieces=(3, 1, 4)):
    """Rows [0, cut) on one handle, snapshot, rows [cut, H) on a second handle; plus the same pushes on one handle."""
    S, H, W, C = x.shape
    nets = [idf.Net(mode, layers, W, C, S, ws, bs, row_block=row_block) for _ in range(3)]
    a, b, ref = nets
    seg = _segments(a, x)
    outs = [n.alloc_out(H) for n in nets]
    for n in nets:
        n.open()

    def push_rows(n, out, lo, hi, last):
        r = lo
        k = 0
        while r < hi:
            m = min(pieces[k % len(pieces)], hi - r)
            k += 1
            if last and r + m == hi:
                n.push_last(seg[r:r + m].contiguous(), out)
            else:
                n.push(seg[r:r + m].contiguous(), out)
            r += m
        if last and lo == hi:
            n.push_last(seg[0:0].contiguous(), out)

    push_rows(a, outs[0], 0, cut, False)
    snap = a.save_state()
    a.reset()                                               # the first handle forgets the streams
    b.push(seg[0:min(2, H)].contiguous(), outs[1])          # the second one was busy with other streams
    b.restore_state(snap)
    push_rows(b, outs[1], cut, H, True)
    push_rows(ref, outs[2], 0, cut, False)
    push_rows(ref, outs[2], cut, H, True)
    for n in nets:
        n.status()
    got_a, got_b, got_ref = (o.cpu().numpy() for o in outs)
    for n in nets:
        n.close()
    return got_a, got_b, got_ref


@pytest.mark.parametrize("name", ["same_pool", "stride2", "oned_k9", "oned_pad", "k5"])
@pytest.mark.parametrize("mode", ["f32", "i8"])
def test_restored_streams_continue_bit_identically(orc, name, mode):
    layers = SMALL_NETS[name]
    if mode == "i8":
        layers = with_shifts(layers, 8)
    H, W = small_dims(name)
    C0 = next(l.cin for l in layers if l.kind == "conv")
    x, ws, bs = rand_net(mode, layers, H, W, C0, S=3, seed=11 + len(name))
    want = orc.forward(mode, layers, x, ws, bs)
    for cut in (0, 1, H // 2, H - 1, H):
        got_a, got_b, got_ref = _interrupted(mode, layers, x, ws, bs, cut, row_block=3)
        # rows completed before the snapshot sit in the first handle's output, the rest in the second's
        n_before = _rows_complete_after(layers, cut)
        merged = got_b.copy()
        merged[:, :n_before] = got_a[:, :n_before]
        assert np.array_equal(merged.view(np.uint8), got_ref.view(np.uint8)), (name, mode, cut)
        if mode == "i8":
            assert_equal(merged, want, f"{name}/{mode}/cut={cut}")
        else:
            assert_close(merged, want, f"{name}/{mode}/cut={cut}")


@pytest.mark.parametrize("wname,S,H", [("vgg2d", 3, 40), ("events2d", 4, 37), ("audio1d", 5, 700)])
def test_restore_on_workload_nets(orc, wname, S, H):
    """Tensor-core, x-unfold, fused-pool and sparse-event layers: their rings and pool rows survive a snapshot."""
    w = workloads.get(wname, n_streams=S, H=H)
    x = workloads.make_input(w)
    ws, bs = workloads.make_params(w)
    want = orc.forward(w.dtype, w.layers, x, ws, bs)
    got_a, got_b, got_ref = _interrupted(w.dtype, w.layers, x, ws, bs, cut=H // 2 + 1, pieces=(7, 2, 16))
    n_before = _rows_complete_after(w.layers, H // 2 + 1)
    merged = got_b.copy()
    merged[:, :n_before] = got_a[:, :n_before]
    assert np.array_equal(merged.view(np.uint8), got_ref.view(np.uint8)), wname
    if w.dtype == "i8":
        assert_equal(merged, want, wname)
    else:
        rel = np.sqrt(((merged - want) ** 2).mean() / (want ** 2).mean())
        assert rel < 2.0 ** -7, (wname, rel)


def test_snapshot_of_another_net_is_refused():
    layers = SMALL_NETS["valid3"]
    x, ws, bs = rand_net("f32", layers, 12, 10, 2, S=2)
    a = idf.Net("f32", layers, 10, 2, 2, ws, bs)
    b = idf.Net("f32", layers, 10, 2, 3, ws, bs)            # one more stream
    c = idf.Net("f32", layers, 12, 2, 2, ws, bs)            # wider rows
    for n in (a, b, c):
        n.open()
    snap = a.save_state()
    for other in (b, c):
        with pytest.raises(idf.IdfError) as e:
            other.restore_state(snap)
        assert e.value.code == idf.ERR_SPEC
    bad = snap.clone(); bad[0] ^= 0xFF
    with pytest.raises(idf.IdfError) as e:
        a.restore_state(bad)
    assert e.value.code == idf.ERR_ARG
    with pytest.raises(idf.IdfError) as e:
        a.restore_state(snap[: snap.numel() // 2].contiguous())
    assert e.value.code == idf.ERR_ARG
    out = a.alloc_out(12)
    a.finish(out)
    L = idf.lib()
    buf = (ctypes.c_ubyte * snap.numel())()
    assert L.idf_state_save(a._h, buf, snap.numel()) == idf.ERR_STATE      # streams have ended
    a.restore_state(snap)                                                   # ... and can be brought back
    a.finish(out)
    for n in (a, b, c):
        n.close()


@pytest.mark.parametrize("name,mode", [("oned_k9", "f32"), ("oned_pad", "i8"), ("same_pool", "i8"), ("stride2", "f32")])
def test_bounded_output_window_on_long_streams(orc, name, mode):
    """A small output buffer reused from its start (idf_stream_set_out_base) collects the same rows as a full one."""
    layers = SMALL_NETS[name]
    if mode == "i8":
        layers = with_shifts(layers, 8)
    H, W = small_dims(name)
    H *= 3
    C0 = next(l.cin for l in layers if l.kind == "conv")
    x, ws, bs = rand_net(mode, layers, H, W, C0, S=3, seed=31)
    want = orc.forward(mode, layers, x, ws, bs)
    net = idf.Net(mode, layers, W, C0, 3, ws, bs, row_block=4)
    seg = _segments(net, x)
    cap = 9                                                  # rows of output buffer; a push of 7 segments never emits more
    out = torch.zeros((3, cap) + tuple(want.shape[2:]), dtype=net.out_torch_dtype, device="cuda")
    net.open()
    got, total, r, k = [], 0, 0, 0
    while r < H:
        m = min((7, 1, 5, 2)[k % 4], H - r)
        k += 1
        net.set_out_base(total)
        if r + m == H:
            new_total = net.push_last(seg[r:r + m].contiguous(), out)
            em = new_total - total
        else:
            em = net.push(seg[r:r + m].contiguous(), out)
        got.append(out[:, :em].cpu().numpy().copy())
        total += em
        r += m
    net.status()
    merged = np.concatenate(got, axis=1)
    assert merged.shape == want.shape
    if mode == "i8":
        assert_equal(merged, want, name)
    else:
        assert_close(merged, want, name)
    # rows still to come must not land below index 0, and a full window refuses further rows
    net.reset()
    with pytest.raises(idf.IdfError) as e:
        net.set_out_base(1)
    assert e.value.code == idf.ERR_ARG
    with pytest.raises(idf.IdfError) as e:
        net.push(seg[:H].contiguous(), out)
    assert e.value.code == idf.ERR_CAPACITY
    net.close()
