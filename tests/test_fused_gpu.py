"""All layers in one launch, the streams' rolling state in shared memory (depth_first_kernel).

The launch must give what the per-layer kernels give - the oracle's result - for every net whose per-stream state fits
a CTA, leave the state in global memory in the per-layer kernels' format (the two may advance a stream in turn), and be
what the library picks by itself for small pushes."""
import numpy as np
import pytest
import torch

from paper_1804_10727_b200 import idf, workloads
from paper_1804_10727_b200.workloads import conv, POOL
from helpers import SMALL_NETS, assert_close, assert_equal, rand_net, small_dims, with_path, with_shifts

pytestmark = [pytest.mark.gpu, pytest.mark.own_routing]


@pytest.fixture(autouse=True)
def _defaults_afterwards():
    yield
    idf.set_debug_flags(0)


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
def test_all_layers_in_one_launch_matches_oracle(orc, name, mode):
    idf.set_debug_flags(idf.DEBUG_FORCE_FUSED)
    layers = SMALL_NETS[name]
    if mode == "i8":
        layers = with_shifts(layers, 8)
    H, W = small_dims(name)
    C0 = next(l.cin for l in layers if l.kind == "conv")
    x, ws, bs = rand_net(mode, layers, H, W, C0, S=37, seed=len(name))          # several CTAs, a ragged last group
    want = orc.forward(mode, layers, x, ws, bs)
    for chunks, last in ((None, False), (None, True), ([1] * H, True), ([5, 1, 3], False), ([H - 1], True)):
        net = idf.Net(mode, layers, W, C0, 37, ws, bs)
        got = idf.infer(net, x, chunks=chunks, last=last)
        assert net.launches == len(chunks or [1]) + (0 if last else 1) + (1 if chunks and sum(chunks) < H else 0), (name, chunks, net.launches)
        _check(mode, got, want, f"{name}/{mode}/chunks={chunks}/last={last}")
        net.close()


@pytest.mark.parametrize("mode", ["f32", "i8"])
def test_per_layer_kernels_and_the_single_launch_take_turns_on_one_stream(orc, mode):
    """The state they leave behind has one format: pushes may alternate between the two."""
    for name in ("same_pool", "stride2", "oned_pad", "k5"):
        layers = SMALL_NETS[name]
        if mode == "i8":
            layers = with_shifts(layers, 8)
        H, W = small_dims(name)
        C0 = next(l.cin for l in layers if l.kind == "conv")
        x, ws, bs = rand_net(mode, layers, H, W, C0, S=6, seed=3)
        want = orc.forward(mode, layers, x, ws, bs)
        net = idf.Net(mode, layers, W, C0, 6, ws, bs, row_block=3)
        seg = idf.segments_from_maps(x, mode).cuda()
        out = net.alloc_out(H)
        net.open()
        pos, k = 0, 0
        for n in (4, 1, 3, 2, 5, 1, 1, 100):
            n = min(n, H - pos)
            if n <= 0:
                break
            idf.set_debug_flags(idf.DEBUG_FORCE_FUSED if k % 2 == 0 else idf.DEBUG_NO_FUSED)
            net.push(seg[pos:pos + n], out)
            pos += n; k += 1
        idf.set_debug_flags(idf.DEBUG_FORCE_FUSED if k % 2 == 0 else idf.DEBUG_NO_FUSED)
        rows = net.finish(out)
        net.status()
        _check(mode, out[:, :rows].cpu().numpy(), want, f"{name}/{mode} alternating")
        net.close()


def test_small_pushes_take_the_single_launch_by_default(orc):
    """One image row per push on the mnist2d net with a single stream: one launch per push (the per-layer kernels
    need three to five); with hundreds of streams a push is real work and stays with the per-layer kernels."""
    w = workloads.get("mnist2d", n_streams=1)
    x = workloads.make_input(w)
    ws, bs = workloads.make_params(w)
    want = orc.forward(w.dtype, w.layers, x, ws, bs)
    net = idf.net_from_workload(w, ws, bs)
    got = idf.infer(net, x, chunks=[1] * w.H, last=True)
    assert net.launches == w.H
    assert_equal(got, want, "mnist2d, one row per push")
    assert net.event_counts()[0] == int((x != 0).sum())          # the sparse first layer still reports its events
    assert net.state_bytes == 18432
    net.close()
    w = workloads.get("mnist2d", n_streams=300)
    x = workloads.make_input(w)
    want = orc.forward(w.dtype, w.layers, x, ws, bs)
    net = idf.net_from_workload(w, ws, bs)
    got = idf.infer(net, x, chunks=[1] * w.H, last=True)
    assert net.launches > w.H and any(t > 0 for t in net.status())
    assert_equal(got, want, "mnist2d, 300 streams, one row per push")
    net.close()
    # toy1d, a few samples per push
    t = workloads.get("toy1d", H=301)
    xt = workloads.make_input(t)
    wt, bt = workloads.make_params(t)
    net = idf.net_from_workload(t, wt, bt)
    got = idf.infer(net, xt, chunks=[2] * 150, last=True)
    assert net.launches == 151
    assert_close(got, orc.forward(t.dtype, t.layers, xt, wt, bt), "toy1d")
    net.close()


def test_snapshot_between_single_launch_pushes(orc):
    layers = with_shifts(SMALL_NETS["same_pool"], 8)
    H, W = small_dims("same_pool")
    x, ws, bs = rand_net("i8", layers, H, W, 3, S=5, seed=9)
    want = orc.forward("i8", layers, x, ws, bs)
    a = idf.Net("i8", layers, W, 3, 5, ws, bs)
    b = idf.Net("i8", layers, W, 3, 5, ws, bs)
    seg = idf.segments_from_maps(x, "i8").cuda()
    oa, ob = a.alloc_out(H), b.alloc_out(H)
    a.open(); b.open()
    done_a = 0
    for r in range(7):
        done_a += a.push(seg[r:r + 1], oa)            # one row per push: the single launch
    snap = a.save_state()
    b.restore_state(snap)
    for r in range(7, H - 1):
        b.push(seg[r:r + 1], ob)
    rows = b.push_last(seg[H - 1:], ob)
    # rows finished before the snapshot are in a's buffer, the later ones in b's
    got = torch.cat([oa[:, :done_a], ob[:, done_a:rows]], dim=1).cpu().numpy()
    assert_equal(got, want, "snapshot between single-launch pushes")
    a.close(); b.close()
