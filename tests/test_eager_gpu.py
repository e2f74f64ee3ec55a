"""Eager (anytime) emission on the device: the paper's literal rule (Eq. 3-5), one segment at a time.

After every pushed segment the output buffer holds what every unit of the last layer has announced so far:
finished rows and, above them, the partial rows of the input cone.  It is compared, push by push, with the CPU
event checker's per-segment eager policy (a stream that does not know where its input ends is the checker run on
a taller map of which only the first rows are presented), the event counts with the checker's, and the result
after idf_stream_finish with the layer-by-layer oracle (Eq. 1)."""
import numpy as np
import pytest
import torch

from paper_1804_10727_b200 import idf
from paper_1804_10727_b200.workloads import Layer, conv, POOL
from helpers import SMALL_NETS, assert_close, assert_equal, rand_net, small_dims, with_shifts

pytestmark = pytest.mark.gpu

EAGER_NETS = ["valid3", "same_pool", "stride2", "stride2_pad", "oned_k9", "oned_k3", "oned_pad", "k5", "norelu", "k3s3"]


def _fc(cin, n_out, h, w, relu=0, shift=0):
    return Layer("conv", cin, n_out, h, w, h, 0, relu, shift, 0)


@pytest.mark.parametrize("name", EAGER_NETS)
@pytest.mark.parametrize("mode", ["f32", "bf16", "i8"])
def test_eager_output_after_every_push_matches_the_event_checker(orc, name, mode):
    layers = SMALL_NETS[name]
    if mode == "i8":
        layers = with_shifts(layers, 7)
    H, W = small_dims(name)
    H = min(H, 24) if W > 1 else H
    EXT = 12                                                  # rows the stream does not know it will never get
    C0 = next(l.cin for l in layers if l.kind == "conv")
    S = 3
    x, ws, _ = rand_net(mode, layers, H + EXT, W, C0, S=S, bias=False, seed=5 + len(name))
    want = orc.forward(mode, layers, x[:, :H], ws, None)
    net = idf.Net(mode, layers, W, C0, S, ws, None, eager=True)
    seg = idf.segments_from_maps(x[:, :H], mode).cuda()
    out = net.alloc_out(H)
    net.open()
    chk = [orc.event_run(mode, layers, x[s], ws, None, eager=2, n_feed=H, steps=True) for s in range(S)]
    emitted = 0
    for r in range(H):
        emitted += net.push(seg[r:r + 1], out)
        got = out.cpu().numpy()
        for s in range(S):
            snap = chk[s]["steps"][r]
            rows = min(snap.shape[0], got.shape[1])
            # rows nothing has reached yet are zero on both sides; compare everything the buffer holds
            if mode == "i8":
                assert_equal(got[s, :rows], snap[:rows], f"{name} stream {s} after segment {r}")
            elif mode == "f32":
                assert_close(got[s, :rows], snap[:rows], f"{name} stream {s} after segment {r}")
            else:
                # bf16 nets: a hidden activation near a rounding boundary may round the other way (fp32 vs float64 sums)
                err = np.abs(got[s, :rows] - snap[:rows])
                assert (err <= 1e-4 + 1e-3 * np.abs(snap[:rows])).mean() > 0.97 and err.max(initial=0) < 0.06
    if mode != "bf16":
        ev = net.event_counts()
        total = np.sum([c["events"] for c in chk], axis=0)
        assert ev[0] == int((x[:, :H] != 0).sum()) == total[0]
        if mode == "i8":
            assert list(ev[1:]) == list(total[1:len(layers)]), (ev, total)          # events layer i has received
    rows = net.finish(out)
    assert rows == want.shape[1] and emitted <= rows
    got = out[:, :rows].cpu().numpy()
    if mode == "i8":
        assert_equal(got, want, f"{name} after finish")
    elif mode == "f32":
        assert_close(got, want, f"{name} after finish")
    else:
        err = np.abs(got - want)
        assert (err <= 1e-4 + 1e-3 * np.abs(want)).mean() > 0.97 and err.max() < 0.06
    net.close()


@pytest.mark.parametrize("mode", ["f32", "i8"])
def test_eager_with_biases_and_any_grouping_ends_at_the_conventional_result(orc, mode):
    """Units with a bias announce f(b) when their row is first touched; grouping segments into pushes changes nothing."""
    for name in ("same_pool", "stride2", "oned_pad"):
        layers = SMALL_NETS[name]
        if mode == "i8":
            layers = with_shifts(layers, 7)
        H, W = small_dims(name)
        C0 = next(l.cin for l in layers if l.kind == "conv")
        x, ws, bs = rand_net(mode, layers, H, W, C0, S=4, bias=True, seed=11)
        want = orc.forward(mode, layers, x, ws, bs)
        first = None
        for chunks, last in ((None, False), ([1] * H, True), ([5, 1, 3], False), ([H - 1], True)):
            net = idf.Net(mode, layers, W, C0, 4, ws, bs, eager=True)
            got = idf.infer(net, x, chunks=chunks, last=last)
            (assert_equal if mode == "i8" else assert_close)(got, want, f"{name} chunks={chunks}")
            if mode == "i8":
                first = got if first is None else first
                assert np.array_equal(got, first)
            net.close()


def test_classifier_output_converges_over_the_presentations(orc):
    """The paper's experiment in shape: rows of a 28-wide image presented one at a time, ten fully connected output
    units whose value can be read after every presentation and ends at the conventional result."""
    H = W = 28
    layers = with_shifts((conv(1, 8, 3), conv(8, 16, 3), POOL), 8) + (_fc(16, 10, 12, 12, shift=10),)
    S = 16
    x, ws, _ = rand_net("i8", layers, H, W, 1, S=S, bias=False, seed=3, zero_frac=0.8)
    want = orc.forward("i8", layers, x, ws, None)
    net = idf.Net("i8", layers, W, 1, S, ws, None, eager=True)
    seg = idf.segments_from_maps(x, "i8").cuda()
    out = net.alloc_out(H)
    net.open()
    chk = orc.event_run("i8", layers, x[0], ws, None, eager=2, steps=True)
    seen_partial = False
    for r in range(H):
        em = net.push(seg[r:r + 1], out)
        got = out[0, 0].cpu().numpy()
        assert_equal(got, chk["steps"][r][0], f"logits after {r + 1} presentations")
        seen_partial |= bool(r < H - 2 and got.any())
        assert em == (1 if r == H - 1 else 0)           # the output row is final only with the last presentation
    assert seen_partial                                  # the logits move long before the image is complete
    assert net.finish(out) == 1
    assert_equal(out[:, :1].cpu().numpy(), want, "classifier")      # (row 1 held partial sums of rows past the image; taken back)
    assert not out[:, 1:].any()
    net.close()


def test_eager_state_is_the_input_cone_and_unsupported_calls_say_so():
    layers = (conv(1, 1, 3, one_d=True), conv(1, 1, 3, one_d=True))
    w = [np.ones((1, 3, 1, 1), np.float32)] * 2
    d = idf.Net("f32", layers, 1, 1, 1, w, None)
    e = idf.Net("f32", layers, 1, 1, 1, w, None, eager=True)
    assert d.state_bytes == (3 + 3) * 4                  # K rows per layer
    assert e.state_bytes == (3 + 5) * 8                  # the cone: 3 and 5 rows, state and announced activation
    e.open()
    with pytest.raises(idf.IdfError) as err:
        e.save_state()
    assert err.value.code == idf.ERR_UNSUPPORTED
    with pytest.raises(idf.IdfError) as err:
        idf.Net("f32", layers + (Layer("avg"),), 1, 1, 1, w + [None], None, eager=True)
    assert err.value.code == idf.ERR_UNSUPPORTED
    out = torch.zeros((1, 2, 1, 1), device="cuda")
    with pytest.raises(idf.IdfError) as err:             # the cone rows must fit the buffer too
        e.push(torch.ones((6, 1, 1, 1), device="cuda"), out)
    assert err.value.code == idf.ERR_CAPACITY
    d.close(); e.close()
