"""Parity at the workloads' full sizes, in the launch configuration bench.py times (all streams of
the batch, all segments and the end of input in one push_last with the default row block).  Streams are independent, so the oracle
is run only on a sample of streams and compared with exactly those streams of the device result;
the rest is covered by properties that hold at any size (shape, finiteness, batch-mate independence)."""
import numpy as np
import pytest
import torch

from paper_1804_10727_b200 import idf, workloads
from helpers import assert_bf16_end_to_end, assert_close, assert_equal

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
            # bf16 nets end to end: statistical criterion (the strict per-layer comparison is further down)
            assert_bf16_end_to_end(name, got, want, f"{name} stream {s}")


@pytest.mark.parametrize("name,sample", [("vgg2d", [0, 63]), ("events2d", [5, 2047]), ("mnist2d", [0, 4095])])
def test_full_size_one_segment_per_push_matches_oracle(orc, name, sample):
    """The launch configuration of bench.py's `streaming` figure: all streams of the batch, one segment per push, the
    last push carrying the end of input.  Every launch then brings one row: all rows exchange state with the ring
    and spread over the epilogue groups by ring slot."""
    w = workloads.get(name)
    ws, bs = workloads.make_params(w)
    net = idf.net_from_workload(w, ws, bs)
    x = workloads.make_input(w)
    seg = idf.segments_from_maps(x, w.dtype).cuda()
    out = net.alloc_out(w.H)
    net.open()
    for r in range(w.H - 1):
        net.push(seg[r:r + 1], out)
    rows = net.push_last(seg[w.H - 1:], out)
    net.status()
    assert rows == net.out_shape(w.H)[0]
    for s in sample:
        want = orc.forward(w.dtype, w.layers, x[s:s + 1], ws, bs)[0]
        got = out[s, :rows].cpu().numpy()
        if w.dtype == "i8":
            assert_equal(got, want, f"{name} stream {s}, one segment per push")
        else:
            assert_bf16_end_to_end(name, got, want, f"{name} stream {s}, one segment per push")
    if w.dtype == "i8":
        # integer nets: the grouping of segments into pushes changes nothing at all
        whole = net.alloc_out(w.H)
        net.reset()
        assert net.push_last(seg, whole) == rows
        assert torch.equal(whole[:, :rows], out[:, :rows])
    net.close()


def test_full_size_state_bytes_are_the_ring_formula():
    want = {"toy1d": 240, "mnist2d": 18432, "audio1d": 17024, "vgg2d": 1247232 + 14336, "events2d": 261248}
    for name, b in want.items():
        w = workloads.get(name)
        net = idf.net_from_workload(w, *workloads.make_params(w))
        assert net.state_bytes == b


# ---- strict bf16 parity, layer by layer, in the tile plans the full-size batch uses -----------------------
def _layer_inputs(w):
    """(index, layer, H, W, C of its input, pool follows?, is it the net's last conv?) for every conv layer."""
    H, W, C = w.H, w.W, w.C
    convs = [i for i, l in enumerate(w.layers) if l.kind == "conv"]
    out = []
    for i, l in enumerate(w.layers):
        if l.kind == "conv":
            pool_next = i + 1 < len(w.layers) and w.layers[i + 1].kind == "pool"
            out.append((i, l, H, W, C, pool_next, i == convs[-1]))
            H = (H + 2 * l.pad - l.kh) // l.stride + 1
            W = 1 if W == 1 else (W + 2 * l.pad - l.kw) // l.stride + 1
            C = l.cout
        else:
            H, W = H // 2, (1 if W == 1 else W // 2)
    return out


def _bf16_down_up(v):
    """The bfloat16 values just below-or-equal and just above-or-equal every entry of v (float64 in, float64 out)."""
    f = np.asarray(v, dtype=np.float64)
    r = torch.from_numpy(f).float().bfloat16().float().numpy()          # nearest bf16 (as float32)
    bits = r.view(np.uint32).astype(np.int64)
    mag, neg = bits & 0x7FFFFFFF, (bits >> 31) != 0
    tiny = np.float32(2.0 ** -133)

    def from_parts(m, n):
        return ((m.astype(np.uint32)) | (n.astype(np.uint32) << 31)).view(np.float32)
    # one bf16 step toward +inf / toward -inf
    up_mag = np.where(neg, mag - 0x10000, mag + 0x10000)
    up = np.where(mag == 0, tiny, from_parts(np.maximum(up_mag, 0), neg & (up_mag > 0)))
    dn_mag = np.where(neg, mag + 0x10000, mag - 0x10000)
    dn = np.where(mag == 0, -tiny, from_parts(np.maximum(dn_mag, 0), neg | (dn_mag < 0)))
    dn = np.where((~neg) & (dn_mag == 0), np.float32(0.0), dn)
    r64 = r.astype(np.float64)
    lo = np.where(r64 <= f, r64, dn.astype(np.float64))
    hi = np.where(r64 >= f, r64, up.astype(np.float64))
    return lo, hi


@pytest.mark.parametrize("name,sample", [("vgg2d", [0, 37, 63]), ("audio1d", [0, 700, 1023])])
def test_bf16_layers_strict_in_the_full_size_plans(orc, name, sample):
    """Every conv layer of the bf16 workloads at the FULL stream count (so that the kernel picks the tiles, stream
    packing, row chunks and pool folding it uses in the benchmarked batch), fed a seeded bf16 map of the layer's real
    input shape; the oracle recomputes sampled streams.  The net's last conv layer emits unrounded fp32 and is held
    to |g - o| <= 1e-4 + 1e-3 |o| directly.  A hidden layer must round to bf16 (so that its tile plan is the one of
    the full net); a 1x1 identity conv behind it passes the rounded values through exactly, and each must be the
    bf16 rounding of SOME value within that tolerance of the oracle's unrounded result."""
    w = workloads.get(name)
    ws, bs = workloads.make_params(w)
    S = w.n_streams
    for i, l, H, W, C, pool_next, is_last in _layer_inputs(w):
        g = torch.Generator().manual_seed(1000 + 17 * i)
        # post-ReLU-like activations (the first layer sees the signed input): bf16 values, segment layout [H][S][W][C]
        seg = torch.empty((H, S, W, C), dtype=torch.bfloat16)
        for h0 in range(0, H, 64):
            blk = torch.randn((min(64, H - h0), S, W, C), generator=g)
            seg[h0:h0 + 64] = (blk if i == 0 else blk.abs()).bfloat16()
        layers = [l] + ([workloads.POOL] if pool_next else [])
        wts, bias = [ws[i]] + ([None] if pool_next else []), [bs[i]] + ([None] if pool_next else [])
        if not is_last:
            layers.append(workloads.conv(l.cout, l.cout, 1, one_d=(W == 1), relu=0))
            wts.append(np.eye(l.cout, dtype=np.float32).reshape(l.cout, 1, 1, l.cout)); bias.append(None)
        net = idf.Net("bf16", tuple(layers), W, C, S, wts, bias)
        out = net.alloc_out(H)
        net.open()
        rows = net.push_last(seg.cuda(), out)
        tc = net.status()
        assert tc[0] > 0 or C * 2 < 32, f"{name} layer {i}: not on the tensor-core path"
        for s in sample:
            a = seg[:, s].float().numpy()[None]                              # [1][H][W][C]
            want = orc.conv_layer("bf16", l, a, ws[i], bs[i])                # unrounded f(c), float64
            if pool_next:
                want = orc.pool_layer("bf16", want)
            got = out[s, :rows].cpu().numpy().astype(np.float64)
            assert got.shape == want[0].shape, (got.shape, want.shape)
            tol = 1e-4 + 1e-3 * np.abs(want[0])
            if is_last:
                bad = np.abs(got - want[0]) > tol
            else:
                lo, _ = _bf16_down_up(want[0] - tol)
                _, hi = _bf16_down_up(want[0] + tol)
                bad = (got < lo) | (got > hi)
            assert not bad.any(), f"{name} layer {i} stream {s}: {bad.sum()} of {bad.size} outside the strict tolerance"
        net.close()
        del seg, out
        torch.cuda.empty_cache()
