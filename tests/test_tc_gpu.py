"""GPU parity of the tensor-core (tcgen05) dense path: single layers and short nets whose shapes
qualify for it, against the CPU oracle.  A single bf16 conv layer emits unrounded fp32, so the strict
float tolerance applies; int8 layers must match bit for bit.  Every case also checks that the
launches really took the tensor-core path and that no bounded device wait ran out."""
import numpy as np
import pytest

from paper_1804_10727_b200 import idf
from paper_1804_10727_b200.workloads import conv, POOL
from helpers import assert_close, assert_equal, rand_net, with_shifts

pytestmark = pytest.mark.gpu


def _run(mode, layers, x, ws, bs, chunks=None, row_block=0):
    S, H, W, C = x.shape
    net = idf.Net(mode, layers, W, C, S, ws, bs, row_block=row_block)
    seg = idf.segments_from_maps(x, mode).cuda()
    out = net.alloc_out(H)
    net.open()
    pos = 0
    for n in (chunks or [H]):
        n = min(n, H - pos)
        if n > 0:
            net.push(seg[pos:pos + n], out)
        pos += n
    if pos < H:
        net.push(seg[pos:], out)
    rows = net.finish(out)
    tc = net.status()
    return out[:, :rows].cpu().numpy(), tc


# (name, mode, layers, H, W, S)
CASES = [
    ("bf16_64_w16", "bf16", (conv(64, 64, 3, pad=1),), 10, 16, 8),
    ("bf16_64_w16_ragged_streams", "bf16", (conv(64, 64, 3, pad=1),), 11, 16, 5),
    ("bf16_64_valid", "bf16", (conv(64, 32, 3),), 12, 20, 7),
    ("bf16_128_w40", "bf16", (conv(128, 64, 3, pad=1),), 9, 40, 4),
    ("bf16_64_wide", "bf16", (conv(64, 64, 3, pad=1),), 7, 224, 2),
    ("bf16_64_w130", "bf16", (conv(64, 16, 3, pad=1),), 6, 130, 3),
    ("bf16_256_n32", "bf16", (conv(256, 256, 3, pad=1),), 8, 28, 9),
    ("bf16_stride2y_1d", "bf16", (conv(64, 128, 9, stride=2, one_d=True),), 80, 1, 200),
    ("bf16_1d_k9", "bf16", (conv(128, 128, 9, one_d=True),), 40, 1, 130),
    ("bf16_32ch", "bf16", (conv(32, 64, 9, stride=2, one_d=True),), 60, 1, 77),
    ("bf16_16ch", "bf16", (conv(16, 32, 3, pad=1),), 12, 24, 6),
    ("bf16_two_layers", "bf16", (conv(64, 64, 3, pad=1), POOL, conv(64, 128, 3, pad=1)), 16, 24, 5),
    ("bf16_k5", "bf16", (conv(64, 32, 5, pad=2),), 14, 33, 4),
    # thin or x-strided layers reach the tensor cores through the x-unfold pre-pass
    ("bf16_3ch_unfold", "bf16", (conv(3, 64, 3, pad=1),), 13, 40, 5),
    ("bf16_1ch_1d_unfold", "bf16", (conv(1, 32, 9, stride=2, one_d=True),), 70, 1, 150),
    ("bf16_stride2_unfold", "bf16", (conv(64, 64, 3, stride=2, pad=1),), 15, 31, 4),
    ("bf16_5ch_k5_unfold", "bf16", (conv(5, 16, 5, stride=2, pad=2),), 17, 29, 3),
    ("i8_16ch_unfold", "i8", (conv(16, 32, 3),), 12, 26, 7),
    # x-strided layers with 32- or 64-byte rows: the tensor map walks the input row in steps of the stride
    ("i8_stride2_x", "i8", (conv(32, 64, 3, stride=2),), 21, 33, 5),
    ("i8_stride2_x_pad", "i8", (conv(64, 32, 3, stride=2, pad=1),), 22, 37, 4),
    ("i8_stride2_x_wide", "i8", (conv(32, 32, 3, stride=2, pad=1),), 9, 300, 2),
    ("i8_stride3_x_k5", "i8", (conv(32, 16, 5, stride=3, pad=2),), 23, 41, 3),
    ("bf16_stride2_x_16ch", "bf16", (conv(16, 32, 3, stride=2),), 19, 30, 6),
    ("bf16_stride2_x_32ch_pad", "bf16", (conv(32, 64, 3, stride=2, pad=1),), 18, 53, 3),
    ("i8_stride2_x_pool", "i8", (conv(32, 32, 3, stride=2), POOL), 27, 45, 5),
    ("i8_2ch_unfold", "i8", (conv(2, 32, 3, path=1),), 12, 30, 6),     # forced dense: AUTO would scatter events
    ("i8_64", "i8", (conv(64, 64, 3),), 12, 30, 6),
    ("i8_32", "i8", (conv(32, 64, 3),), 12, 30, 6),
    ("i8_128", "i8", (conv(128, 32, 3, pad=1),), 9, 20, 7),
    ("i8_256", "i8", (conv(256, 64, 3, pad=1),), 9, 20, 7),
    ("i8_net", "i8", (conv(32, 32, 3), POOL, conv(32, 64, 3, pad=1)), 20, 26, 9),
]


@pytest.mark.parametrize("name,mode,layers,H,W,S", CASES, ids=[c[0] for c in CASES])
def test_tensor_core_layers_match_oracle(orc, name, mode, layers, H, W, S):
    if mode == "i8":
        layers = with_shifts(layers, 9)
    C0 = layers[0].cin
    x, ws, bs = rand_net(mode, layers, H, W, C0, S=S, seed=len(name))
    want = orc.forward(mode, layers, x, ws, bs)
    n_conv = sum(l.kind == "conv" for l in layers)
    for chunks, rb in ((None, 0), ([1] * H, 0), ([3, 2, 5], 3), (None, 64)):
        got, tc = _run(mode, layers, x, ws, bs, chunks=chunks, row_block=rb)
        assert sum(t > 0 for t in tc) == n_conv, f"{name}: tensor-core path not taken: {tc}"
        what = f"{name}/chunks={chunks and len(chunks)}/rb={rb}"
        if mode == "i8":
            assert_equal(got, want, what)
        elif n_conv == 1:
            assert_close(got, want, what)
        else:
            err = np.abs(got - want)
            ok = err <= 1e-4 + 1e-3 * np.abs(want)
            assert ok.mean() > 0.97 and err.max() < 0.05, (what, ok.mean(), err.max())


def test_tensor_core_and_cuda_core_paths_agree_bitwise_on_int8(orc, debug_flags):
    layers = with_shifts((conv(64, 64, 3, pad=1), conv(64, 32, 3, stride=1)), 9)
    x, ws, bs = rand_net("i8", layers, 18, 37, 64, S=5, seed=77)
    got_tc, tc = _run("i8", layers, x, ws, bs)
    assert all(t > 0 for t in tc)
    debug_flags(idf.DEBUG_NO_TENSOR_CORES)
    got_cc, tc2 = _run("i8", layers, x, ws, bs)
    assert not any(tc2)
    assert np.array_equal(got_tc, got_cc)


# ---- 2x2 max-pooling folded into the emission of the conv layer in front of it ----------------------
POOL_CASES = [
    # (name, mode, layers, H, W, S)
    ("i8_conv_pool", "i8", (conv(32, 32, 3, pad=1), POOL), 18, 24, 7),
    ("i8_conv_pool_conv", "i8", (conv(32, 64, 3, pad=1), POOL, conv(64, 32, 3, pad=1), POOL), 22, 40, 5),
    ("i8_pool_odd_rows_valid", "i8", (conv(64, 32, 3), POOL, conv(32, 32, 3)), 21, 30, 6),
    ("i8_pool_wide_two_x_tiles", "i8", (conv(32, 16, 3, pad=1), POOL), 9, 224, 2),
    ("i8_pool_odd_width", "i8", (conv(32, 32, 3), POOL), 12, 29, 4),            # Wout = 27: the last column is dropped
    ("bf16_last_conv_pool_fp32", "bf16", (conv(64, 32, 3, pad=1), POOL), 14, 56, 5),   # fp32 rows pooled
    ("bf16_pool_then_conv", "bf16", (conv(64, 64, 3, pad=1), POOL, conv(64, 16, 3, pad=1)), 16, 24, 5),
    ("i8_unfold_pool", "i8", (conv(16, 32, 3, pad=1), POOL), 15, 26, 7),
]


@pytest.mark.parametrize("name,mode,layers,H,W,S", POOL_CASES, ids=[c[0] for c in POOL_CASES])
def test_pool_folded_into_the_conv_launch_matches_oracle(orc, debug_flags, name, mode, layers, H, W, S):
    if mode == "i8":
        layers = with_shifts(layers, 9)
    x, ws, bs = rand_net(mode, layers, H, W, layers[0].cin, S=S, seed=3 + len(name))
    want = orc.forward(mode, layers, x, ws, bs)
    n_conv = sum(l.kind == "conv" for l in layers)

    def run(chunks, rb, last):
        net = idf.Net(mode, layers, W, layers[0].cin, S, ws, bs, row_block=rb)
        got = idf.infer(net, x, chunks=chunks, last=last)
        return got, net.launches

    def check(got, what):
        if mode == "i8":
            assert_equal(got, want, what)
        elif n_conv == 1:
            assert_close(got, want, what)
        else:
            err = np.abs(got - want)
            ok = err <= 1e-4 + 1e-3 * np.abs(want)
            assert ok.mean() > 0.97 and err.max() < 0.05, (what, ok.mean(), err.max())

    # pairs of rows split across launches in every way: one row at a time, odd groups, everything at once
    fused_launches = None
    for chunks, rb, last in ((None, 0, True), (None, 0, False), ([1] * H, 0, False), ([3, 2, 5, 1], 3, True),
                             ([H - 1], 0, True), (None, 5, True)):
        got, n = run(chunks, rb, last)
        check(got, f"{name}/chunks={chunks}/rb={rb}/last={last}")
        if chunks is None and rb == 0 and last:
            fused_launches = n
    # the same net with the folding switched off runs the pool layers as launches of their own
    debug_flags(idf.DEBUG_NO_POOL_FUSION)
    got, n = run(None, 0, True)
    check(got, f"{name}/unfused")
    if name == "i8_pool_odd_width":          # an odd tile width cannot pair lanes: this net never folds
        assert n == fused_launches
    else:
        assert n > fused_launches, (n, fused_launches)


# ---- few streams, many rows: the block's output rows are spread over CTAs in chunks ------------------
CHUNK_CASES = [
    ("i8_same_pad", "i8", (conv(32, 32, 3, pad=1),), 150, 20, 3),
    ("i8_valid_pool", "i8", (conv(32, 32, 3), POOL, conv(32, 16, 3, pad=1)), 131, 24, 2),
    ("i8_stride2_1d", "i8", (conv(32, 64, 9, stride=2, one_d=True), conv(64, 64, 9, one_d=True)), 700, 1, 40),
    ("i8_k5_pool_pool", "i8", (conv(64, 32, 5, pad=2), POOL, conv(32, 32, 3, pad=1), POOL), 97, 16, 4),
    ("bf16_1d_single", "bf16", (conv(64, 64, 9, stride=2, one_d=True),), 900, 1, 100),
]


@pytest.mark.parametrize("name,mode,layers,H,W,S", CHUNK_CASES, ids=[c[0] for c in CHUNK_CASES])
def test_row_chunks_match_oracle(orc, debug_flags, name, mode, layers, H, W, S):
    if mode == "i8":
        layers = with_shifts(layers, 9)
    x, ws, bs = rand_net(mode, layers, H, W, layers[0].cin, S=S, seed=11 + len(name))
    want = orc.forward(mode, layers, x, ws, bs)
    # blocks that begin, continue and end streams, with rows carried over launch boundaries in both directions
    for chunks, rb, last in ((None, 0, True), (None, 0, False), ([H // 2 + 1], 0, True), ([H // 2, H // 4], 0, False),
                             ([37, 50], 64, False), (None, 1024, True)):
        net = idf.Net(mode, layers, W, layers[0].cin, S, ws, bs, row_block=rb)
        got = idf.infer(net, x, chunks=chunks, last=last)
        what = f"{name}/chunks={chunks}/rb={rb}/last={last}"
        if mode == "i8":
            assert_equal(got, want, what)
        else:
            assert_close(got, want, what)
    if mode == "i8":
        # the same with the rows of a block kept in one CTA per tile: bit-identical
        debug_flags(idf.DEBUG_NO_ROW_CHUNKS)
        net = idf.Net(mode, layers, W, layers[0].cin, S, ws, bs)
        assert_equal(idf.infer(net, x, last=True), want, name + "/unchunked")


# ---- thin layers: the whole receptive field in one shared-memory row, a kernel of its own ------------------------
THIN_CASES = [
    # (name, mode, layers, H, W, S)
    ("bf16_rgb_3x3_same", "bf16", (conv(3, 64, 3, pad=1), conv(64, 16, 3, pad=1)), 30, 40, 5),
    ("i8_rgb_3x3_valid", "i8", (conv(3, 32, 3, path=1), conv(32, 32, 3, pad=1)), 26, 37, 4),
    ("bf16_1d_k9_stride2", "bf16", (conv(1, 32, 9, stride=2, one_d=True), conv(32, 32, 9, one_d=True)), 300, 1, 200),
    ("i8_1d_k9", "i8", (conv(2, 16, 9, one_d=True, path=1),), 120, 1, 70),                   # 16 channels: 16-column chunks
    ("bf16_wide_three_x_tiles", "bf16", (conv(2, 32, 3, pad=1),), 12, 300, 2),
    ("i8_many_channels", "i8", (conv(4, 256, 3, pad=1, path=1), conv(256, 16, 1)), 14, 20, 3),   # one row per work item
    ("i8_5x5_stride2", "i8", (conv(4, 32, 5, stride=2, pad=2, path=1), conv(32, 16, 3)), 41, 30, 3),   # 100-byte rows
    ("bf16_last_layer_fp32", "bf16", (conv(3, 32, 3, pad=1),), 20, 24, 6),
]


@pytest.mark.parametrize("name,mode,layers,H,W,S", THIN_CASES, ids=[c[0] for c in THIN_CASES])
def test_thin_layers_match_oracle(orc, debug_flags, name, mode, layers, H, W, S):
    debug_flags(idf.DEBUG_PREFER_THIN)          # (2D layers take x-unfold + row ring by default; here every case runs the thin kernel)
    if mode == "i8":
        layers = with_shifts(layers, 8)
    x, ws, bs = rand_net(mode, layers, H, W, layers[0].cin, S=S, seed=7 + len(name))
    want = orc.forward(mode, layers, x, ws, bs)
    n_conv = sum(l.kind == "conv" for l in layers)
    # whole streams at once, blocks that begin / continue / end streams (rows carried through the ring at both ends of
    # a block), row by row (no row is determined by one block alone: the ring kernel takes everything)
    for chunks, rb, last in ((None, 0, True), (None, 0, False), ([H // 2 + 1], 0, True), ([7, 9, 5], 8, False), ([1] * min(H, 30), 0, True)):
        got, tc = _run(mode, layers, x, ws, bs, chunks=chunks, row_block=rb) if not last else (None, None)
        if last:
            net = idf.Net(mode, layers, W, layers[0].cin, S, ws, bs, row_block=rb)
            got = idf.infer(net, x, chunks=chunks, last=True)
            tc = net.status()
        what = f"{name}/chunks={chunks}/rb={rb}/last={last}"
        if chunks is None:
            assert tc[0] > 0, f"{what}: the first layer did not take a tensor-core kernel: {tc}"
        if mode == "i8":
            assert_equal(got, want, what)
        elif n_conv == 1:
            assert_close(got, want, what)
        else:
            err = np.abs(got - want)
            ok = err <= 1e-4 + 1e-3 * np.abs(want)
            assert ok.mean() > 0.97 and err.max() < 0.05, (what, ok.mean(), err.max())
