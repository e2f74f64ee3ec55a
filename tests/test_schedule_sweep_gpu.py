"""Every way a block of rows can meet a kernel that keeps state between launches.

The result must not depend on how segments are grouped into pushes (the paper's output is defined by
the whole input, Eq. 1).  Each kernel that exchanges rows with state in global memory - the CUDA-core
conv (ring), the sparse conv (ring), the stand-alone max-pool (one state row), the tensor-core conv
with and without row chunks (ring), its folded max-pool (pool state row) and the averaging sink (sums) -
is driven through every combination of
    first row of the launch even/odd  x  last row even/odd  x  1, 2 or many rows per launch
    x  rows begun by an earlier launch or not  x  rows left open for a later launch or not,
compared with the CPU oracle, and repeated: an integer result must come out bit-identical every time
(a schedule whose result depends on the order in which CTAs happen to run shows up as a difference
between two runs, or between a run and the oracle).
"""
import itertools

import numpy as np
import pytest
import torch

from paper_1804_10727_b200 import idf
from paper_1804_10727_b200.workloads import Layer, conv, POOL
from helpers import assert_close, assert_equal, rand_net, with_path, with_shifts

pytestmark = pytest.mark.gpu

AVG = Layer("avg")


def _pushes(net, seg, out, groups, last):
    """Push the row groups one call each; returns the number of output rows."""
    net.reset()
    rows = None
    for k, (a, b) in enumerate(groups):
        if last and k == len(groups) - 1:
            rows = net.push_last(seg[a:b], out)
        else:
            net.push(seg[a:b], out)
    if rows is None:
        rows = net.finish(out)
    return rows


def _groups(H, sizes):
    g, pos = [], 0
    for n in itertools.cycle(sizes):
        if pos >= H:
            break
        g.append((pos, min(H, pos + n)))
        pos += n
    return g


# Push sizes that make a launch's first and last row even or odd in every combination, with one, two and
# many rows per launch, for a layer at any fixed row offset behind the input (cycled until the input ends).
SIZE_PATTERNS = [(1,), (2,), (3,), (1, 2), (2, 1, 1), (5, 4), (4, 5, 2), (7, 2, 2, 1), (6,), (9, 1), (1, 1, 8), (2, 9, 3)]

# (name, mode, layers, H, W, S, C0): small nets, one per stateful kernel (and the pairs that hand rows to one another)
SWEEP_NETS = [
    ("cuda_core_conv_pool_f32", "f32", (conv(4, 8, 3, pad=1), POOL, conv(8, 4, 3)), 23, 12, 3, 4),
    ("cuda_core_stride2_i8", "i8", (conv(2, 4, 3, stride=2, pad=1), conv(4, 4, 3), POOL), 27, 14, 3, 2),
    ("sparse_conv_pool_i8", "i8", with_path((conv(2, 16, 3), POOL, conv(16, 8, 3, pad=1)), idf.PATH_SPARSE), 25, 18, 3, 2),
    ("pool_vec_first_i8", "i8", (POOL, conv(16, 16, 1), POOL), 26, 12, 4, 16),        # stand-alone vector pool fed the pushes themselves
    ("pool_vec_first_f32", "f32", (POOL, conv(4, 4, 1, relu=0)), 21, 10, 4, 4),
    ("tc_conv_fused_pool_i8", "i8", (conv(32, 32, 3, pad=1), POOL, conv(32, 32, 3, pad=1), POOL), 26, 24, 3, 32),
    ("tc_conv_valid_pool_i8", "i8", (conv(32, 32, 3), POOL, conv(32, 16, 3)), 25, 20, 3, 32),
    ("tc_1x1_pool_i8", "i8", (conv(32, 32, 1), POOL, conv(32, 16, 3, pad=1)), 22, 16, 3, 32),    # no ring rows carried: the pool state alone crosses launches
    ("tc_stride2_k5_i8", "i8", (conv(32, 32, 5, stride=2, pad=2), conv(32, 32, 3)), 31, 18, 3, 32),
    ("avg_sink_i8", "i8", (conv(2, 8, 3), AVG), 20, 9, 3, 2),
]


@pytest.mark.parametrize("name,mode,layers,H,W,S,C0", SWEEP_NETS, ids=[c[0] for c in SWEEP_NETS])
def test_every_grouping_of_rows_gives_the_oracle_result(orc, name, mode, layers, H, W, S, C0):
    if mode == "i8":
        layers = with_shifts(layers, 7)
    x, ws, bs = rand_net(mode, layers, H, W, C0, S=S, seed=41 + len(name))
    want = orc.forward(mode, layers, x, ws, bs)
    seg = idf.segments_from_maps(x, mode).cuda()
    for rb in (0, 2, 3):
        net = idf.Net(mode, layers, W, C0, S, ws, bs, row_block=rb)
        out = net.alloc_out(H)
        net.open()
        for sizes in SIZE_PATTERNS:
            for last in (False, True):
                out.zero_()
                rows = _pushes(net, seg, out, _groups(H, sizes), last)
                net.status()
                got = out[:, :rows].cpu().numpy()
                what = f"{name}/rb={rb}/sizes={sizes}/last={last}"
                if mode == "i8" and layers[-1].kind != "avg":
                    assert_equal(got, want, what)
                elif mode == "i8":
                    assert np.array_equal(got, want.astype(np.float32)), what
                else:
                    assert_close(got, want, what)
        net.close()


@pytest.mark.parametrize("name,mode,layers,H,W,S,C0", [c for c in SWEEP_NETS if c[1] == "i8"],
                         ids=[c[0] for c in SWEEP_NETS if c[1] == "i8"])
def test_integer_results_are_bit_identical_run_after_run(name, mode, layers, H, W, S, C0):
    layers = with_shifts(layers, 7)
    x, ws, bs = rand_net(mode, layers, H, W, C0, S=S, seed=41 + len(name))
    seg = idf.segments_from_maps(x, mode).cuda()
    net = idf.Net(mode, layers, W, C0, S, ws, bs, row_block=3)
    out = net.alloc_out(H)
    net.open()
    for sizes in ((5, 4), (2, 9, 3), (1,)):
        first = None
        for rep in range(10):
            out.zero_()
            rows = _pushes(net, seg, out, _groups(H, sizes), rep % 2 == 1)
            net.status()
            got = out[:, :rows].clone()
            if first is None:
                first = got
            assert torch.equal(got, first), f"{name}/sizes={sizes}: run {rep} differs from run 0"
    net.close()


# ---- the stand-alone vector pool with its state row read AND written in one launch ------------------------
@pytest.mark.parametrize("mode,C,S,W,H,reps", [("i8", 32, 96, 128, 23, 20), ("f32", 32, 32, 128, 23, 20), ("bf16", 64, 48, 96, 23, 20),
                                               ("f32", 32, 6, 16, 205, 10), ("i8", 16, 24, 64, 205, 10)])
def test_pool_launch_that_takes_and_parks_a_row(orc, mode, C, S, W, H, reps):
    """A pool layer fed rows [odd, odd): the first visited row takes its first half from the state row, the
    last one parks its first half there.  The two accesses belong to different output rows, which in a
    row-parallel kernel means different threads, possibly different CTAs on different SMs (hundreds of CTAs
    in the wide cases, three in the narrow ones, where reader and writer start at the same moment); the result
    must equal the oracle's every time."""
    layers = (POOL, conv(C, 16, 1, relu=0, shift=0))          # the pool is fed the pushes themselves; a 1x1 conv behind it
    x, ws, bs = rand_net(mode, layers, H, W, C, S=S, seed=5, zero_frac=0.0, bias=False)
    if mode == "i8":
        # small weights, so that the 1x1 conv behind the pool does not saturate and every pooled value shows
        ws[1] = np.sign(ws[1]).astype(np.int8)
        layers = with_shifts(layers, 4)
    want = orc.forward(mode, layers, x, ws, bs)
    seg = idf.segments_from_maps(x, mode).cuda()
    net = idf.Net(mode, layers, W, C, S, ws, bs, row_block=64)
    out = net.alloc_out(H)
    net.open()
    # launches of the pool: [0,5) [5,7) [7,9) [9,13) [13,19) [19,21) ...: rows begin and end on odd indices,
    # two rows (reader and writer next to each other) and more
    groups = [(0, 5), (5, 7), (7, 9), (9, 13), (13, 19)]
    while groups[-1][1] < H:
        groups.append((groups[-1][1], min(H, groups[-1][1] + 2)))
    for rep in range(reps):
        out.zero_()
        rows = _pushes(net, seg, out, groups, rep % 2 == 0)
        net.status()
        got = out[:, :rows].cpu().numpy()
        if mode == "i8":
            assert_equal(got, want, f"pool state, run {rep}")
        else:
            # (the conv behind the pool is the net's last conv layer: its output is unrounded fp32 in bf16 nets too)
            assert_close(got, want, f"pool state, run {rep}")
    net.close()
