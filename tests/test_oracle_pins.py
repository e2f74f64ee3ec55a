"""Pins for the CPU oracle: everything here checks oracle/ against something that
is not the oracle's own arithmetic (a library routine, a closed form, a brute-force
sum written out separately, the paper's printed value, the event-by-event checker)."""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from paper_1804_10727_b200.workloads import Layer, conv, POOL

rng = np.random.default_rng(1234)


def _rand_net(mode, layers, H, W, C0, S=2, bias=True, seed=0):
    r = np.random.default_rng(seed)
    if mode == "i8":
        x = r.integers(-127, 128, size=(S, H, W, C0)).astype(np.int32)
        x[r.random(x.shape) < 0.5] = 0
    else:
        x = r.standard_normal((S, H, W, C0))
        if mode == "bf16":
            x = torch.tensor(x, dtype=torch.float32).bfloat16().double().numpy()
    ws, bs = [], []
    for l in layers:
        if l.kind != "conv":
            ws.append(None); bs.append(None); continue
        if mode == "i8":
            ws.append(r.integers(-127, 128, size=(l.cout, l.kh, l.kw, l.cin)).astype(np.int32))
            bs.append(r.integers(-500, 500, size=(l.cout,)).astype(np.int32) if bias else None)
        else:
            w = r.standard_normal((l.cout, l.kh, l.kw, l.cin)) * (2.0 / (l.cin * l.kh * l.kw)) ** 0.5
            if mode == "bf16":
                w = torch.tensor(w, dtype=torch.float32).bfloat16().double().numpy()
            ws.append(w)
            bs.append(r.standard_normal((l.cout,)) * 0.1 if bias else None)
    return x, ws, bs


def _torch_forward(mode, layers, x, ws, bs):
    """Conventional inference with torch.nn.functional in float64 (exact for the integer nets)."""
    a = torch.tensor(np.asarray(x, dtype=np.float64)).permute(0, 3, 1, 2)   # NCHW
    convs = [i for i, l in enumerate(layers) if l.kind == "conv"]
    for i, l in enumerate(layers):
        if l.kind == "conv":
            w = torch.tensor(np.asarray(ws[i], dtype=np.float64)).permute(0, 3, 1, 2)  # [Cout][Cin][Kh][Kw]
            b = None if bs[i] is None else torch.tensor(np.asarray(bs[i], dtype=np.float64))
            one_d = a.shape[3] == 1 and l.kw == 1
            a = F.conv2d(a, w, b, stride=(l.stride, 1 if one_d else l.stride), padding=(l.pad, 0 if one_d else l.pad))
            if l.relu:
                a = F.relu(a)
            if mode == "bf16" and i != convs[-1]:
                a = a.float().bfloat16().double()       # float64 -> float32 is exact enough here? see test below
            if mode == "i8":
                ai = a.to(torch.int64)
                if l.shift > 0:
                    ai = torch.div(ai + (1 << (l.shift - 1)), 1 << l.shift, rounding_mode="floor")
                a = ai.clamp(0 if l.relu else -127, 127).double()
        else:
            if a.shape[3] == 1:
                a = F.max_pool2d(a, kernel_size=(2, 1), stride=(2, 1))
            else:
                a = F.max_pool2d(a, kernel_size=2, stride=2)
    return a.permute(0, 2, 3, 1).numpy()


NETS = {
    "valid3": (conv(2, 4, 3), conv(4, 3, 3)),
    "same_pool": (conv(3, 4, 3, pad=1), POOL, conv(4, 5, 3, pad=1), POOL),
    "stride2": (conv(2, 4, 3, stride=2), conv(4, 4, 3, stride=1), POOL),
    "stride2_pad": (conv(2, 3, 3, stride=2, pad=1), conv(3, 4, 3, stride=2, pad=1)),
    "oned_k9": (conv(1, 4, 9, stride=2, one_d=True), conv(4, 5, 9, one_d=True)),
    "oned_k3": (conv(1, 8, 3, one_d=True), conv(8, 8, 3, one_d=True), conv(8, 4, 3, one_d=True)),
    "oned_pad": (conv(2, 3, 5, stride=2, pad=2, one_d=True), POOL, conv(3, 4, 3, pad=1, one_d=True)),
    "k5": (conv(2, 3, 5, stride=2, pad=2), conv(3, 2, 3)),
    "norelu": (conv(2, 3, 3, relu=0), conv(3, 2, 3, relu=0)),
}


def _with_shifts(layers, s=7):
    return tuple(Layer(**{**l.__dict__, "shift": s}) if l.kind == "conv" else l for l in layers)


def _dims(name):
    if name.startswith("oned"):
        return 60, 1
    return 17, 14


# ---- P1: the library routine -------------------------------------------------------------------
@pytest.mark.parametrize("name", list(NETS))
@pytest.mark.parametrize("mode", ["f32", "bf16", "i8"])
def test_matches_torch_functional(orc, name, mode):
    layers = NETS[name]
    if mode == "i8":
        layers = _with_shifts(layers, 8)
    H, W = _dims(name)
    x, ws, bs = _rand_net(mode, layers, H, W, layers[0].cin, S=2, seed=hash(name) % 1000)
    got = orc.forward(mode, layers, x, ws, bs)
    want = _torch_forward(mode, layers, x, ws, bs)
    assert got.shape == want.shape
    if mode == "i8":
        assert np.array_equal(got, want.astype(np.int32))
    elif mode == "f32":
        np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)
    else:
        # float32 conv results passed through bf16 on the torch side may hit a double-rounding
        # tie that the oracle's direct rounding does not: allow a handful of 1-ulp deviations
        close = np.isclose(got, want, rtol=1e-10, atol=1e-12)
        assert close.mean() > 0.999
        np.testing.assert_allclose(got, want, rtol=2.0 ** -6, atol=1e-6)


# ---- P2: single-unit brute force ---------------------------------------------------------------
def test_single_unit_brute_force(orc):
    l = conv(3, 5, 3, stride=2, pad=1, relu=0)
    x, ws, bs = _rand_net("f32", (l,), 11, 9, 3, S=1, seed=5)
    got = orc.forward("f32", (l,), x, ws, bs)[0]
    r = np.random.default_rng(0)
    for _ in range(50):
        oy, ox, co = r.integers(got.shape[0]), r.integers(got.shape[1]), r.integers(5)
        acc = Fraction(float(bs[0][co]))
        for ky in range(3):
            for kx in range(3):
                iy, ix = oy * 2 - 1 + ky, ox * 2 - 1 + kx
                if 0 <= iy < 11 and 0 <= ix < 9:
                    for ci in range(3):
                        acc += Fraction(float(ws[0][co, ky, kx, ci])) * Fraction(float(x[0, iy, ix, ci]))
        assert abs(float(acc) - got[oy, ox, co]) < 1e-12


# ---- P4: closed forms --------------------------------------------------------------------------
@pytest.mark.parametrize("stride,pad", [(1, 0), (1, 1), (2, 0), (2, 1)])
def test_impulse_response_is_the_kernel(orc, stride, pad):
    l = conv(2, 3, 3, stride=stride, pad=pad, relu=0)
    H, W = 9, 8
    _, ws, _ = _rand_net("f32", (l,), H, W, 2, S=1, bias=False, seed=3)
    y0, x0, ci = 4, 3, 1
    x = np.zeros((1, H, W, 2)); x[0, y0, x0, ci] = 1.0
    got = orc.forward("f32", (l,), x, ws, None)[0]
    for oy in range(got.shape[0]):
        for ox in range(got.shape[1]):
            ky, kx = y0 + pad - oy * stride, x0 + pad - ox * stride
            for co in range(3):
                want = ws[0][co, ky, kx, ci] if (0 <= ky < 3 and 0 <= kx < 3) else 0.0
                assert got[oy, ox, co] == want


def test_all_ones_counts_fan_in(orc):
    layers = (conv(2, 3, 3, relu=0), conv(3, 2, 3, relu=0))
    ws = [np.ones((3, 3, 3, 2)), np.ones((2, 3, 3, 3))]
    x = np.ones((1, 8, 8, 2))
    got = orc.forward("f32", layers, x, ws, None)
    assert np.all(got == 18 * 27)
    # with same padding, a corner unit sees only 2x2 taps
    l = conv(2, 1, 3, pad=1, relu=0)
    got = orc.forward("f32", (l,), x, [np.ones((1, 3, 3, 2))], None)[0]
    assert got[0, 0, 0] == 8 and got[0, 3, 0] == 12 and got[3, 3, 0] == 18


def test_linearity_and_positive_homogeneity(orc):
    lin = NETS["norelu"]
    x, ws, _ = _rand_net("f32", lin, 9, 9, 2, S=2, bias=False, seed=9)
    y = np.random.default_rng(1).standard_normal(x.shape)
    f = lambda v: orc.forward("f32", lin, v, ws, None)
    np.testing.assert_allclose(f(2.5 * x - 0.5 * y), 2.5 * f(x) - 0.5 * f(y), rtol=1e-11, atol=1e-12)
    rel = NETS["same_pool"]
    x, ws, _ = _rand_net("f32", rel, 12, 12, 3, S=1, bias=False, seed=10)
    g = lambda v: orc.forward("f32", rel, v, ws, None)
    assert np.array_equal(g(4.0 * x), 4.0 * g(x))      # power of two: exact


# ---- bf16 rounding and requantisation ----------------------------------------------------------
def test_bf16_rounding_matches_torch_and_ties(orc):
    v = torch.randn(20000, dtype=torch.float32) * torch.logspace(-20, 20, 20000, base=2.0)
    want = v.bfloat16().double().numpy()
    got = orc.round_bf16(v.double().numpy())
    assert np.array_equal(got, want)
    # ties go to the even neighbour; just above a tie goes up (a case float32 double rounding gets wrong)
    assert orc.round_bf16(np.array([1 + 2.0 ** -8]))[0] == 1.0
    assert orc.round_bf16(np.array([1 + 3 * 2.0 ** -8]))[0] == 1 + 2.0 ** -6
    assert orc.round_bf16(np.array([1 + 2.0 ** -8 + 2.0 ** -40]))[0] == 1 + 2.0 ** -7
    assert orc.round_bf16(np.array([-(1 + 2.0 ** -8 + 2.0 ** -40)]))[0] == -(1 + 2.0 ** -7)
    assert orc.round_bf16(np.array([0.0]))[0] == 0.0


def test_bf16_rounding_of_subnormals_matches_torch_and_closed_forms(orc):
    """The subnormal range of bfloat16 (below 2^-126, spacing 2^-133): fewer significant bits are kept there.
    torch's fp32 -> bf16 conversion rounds these to nearest even too, so it pins the branch; the hand-made
    values pin the ties and the underflow to zero."""
    r = np.random.default_rng(3)
    # fp32 bit patterns with biased exponents 0..12: fp32 subnormals and the smallest normals, both signs
    bits = (r.integers(0, 13, size=40000).astype(np.uint32) << 23) | r.integers(0, 1 << 23, size=40000).astype(np.uint32)
    bits |= (r.integers(0, 2, size=40000).astype(np.uint32) << 31)
    v = torch.from_numpy(bits.view(np.float32).copy())
    want = v.bfloat16().double().numpy()
    got = orc.round_bf16(v.double().numpy())
    assert np.array_equal(got, want) and np.array_equal(np.signbit(got), np.signbit(want))
    assert (want != 0).any() and (want == 0).any() and (np.abs(want[want != 0]) < 2.0 ** -126).any()
    tiny = 2.0 ** -133                                       # the smallest positive bfloat16
    one = lambda x: orc.round_bf16(np.array([x], dtype=np.float64))[0]
    assert one(tiny) == tiny and one(-tiny) == -tiny
    assert one(tiny / 2) == 0.0                              # tie between 0 and tiny: to even (zero)
    assert one(tiny / 2 * (1 + 2.0 ** -30)) == tiny          # just above the tie
    assert one(tiny / 4) == 0.0
    assert one(1.5 * tiny) == 2 * tiny                       # tie between tiny and 2 tiny: to even
    assert one(2.5 * tiny) == 2 * tiny                       # tie between 2 tiny and 3 tiny: to even
    assert one(2.0 ** -126 - tiny / 4) == 2.0 ** -126        # rounds up into the normal range
    assert one(-(2.0 ** -126 - 0.75 * tiny)) == -(2.0 ** -126 - tiny)


def test_requant_matches_exact_rationals(orc):
    r = np.random.default_rng(2)
    c = r.integers(-200000, 200000, size=4000).astype(np.int32)
    for shift in (0, 1, 4, 9):
        for relu in (0, 1):
            got = orc.requant(c, shift, relu)
            for ci, gi in zip(c[:500], got[:500]):
                q = Fraction(int(ci), 1 << shift)
                v = int((q + Fraction(1, 2)).__floor__()) if shift > 0 else int(ci)  # round half up
                v = max(0 if relu else -127, min(127, v))
                assert v == gi


# ---- P3/P5/P6: the event-by-event implementation and the paper's invariants --------------------
@pytest.mark.parametrize("name", list(NETS))
@pytest.mark.parametrize("mode", ["f32", "bf16", "i8"])
@pytest.mark.parametrize("eager", [True, False])
def test_event_by_event_equals_layer_by_layer(orc, name, mode, eager):
    layers = NETS[name]
    if mode == "i8":
        layers = _with_shifts(layers, 8)
    H, W = (40, 1) if name.startswith("oned") else (11, 10)
    x, ws, bs = _rand_net(mode, layers, H, W, layers[0].cin, S=1, seed=7)
    want = orc.forward(mode, layers, x, ws, bs)[0]
    ev = orc.event_run(mode, layers, x[0], ws, bs, eager=eager)
    if mode == "i8":
        assert np.array_equal(ev["out"], want.astype(np.float64))
        assert ev["telescoping_err"] == 0.0
    elif mode == "f32":
        np.testing.assert_allclose(ev["out"], want, rtol=1e-9, atol=1e-9)
        assert ev["telescoping_err"] < 1e-9
    else:
        # event order changes the low bits of c, which can flip a bf16 rounding: rare, one ulp
        close = np.isclose(ev["out"], want, rtol=1e-9, atol=1e-9)
        assert close.mean() > 0.98
        np.testing.assert_allclose(ev["out"], want, rtol=0.05, atol=0.02)
    np.testing.assert_allclose(ev["sum_dh"], ev["out"], atol=1e-9)     # events telescope to the activation


@pytest.mark.parametrize("eager", [True, False])
def test_zero_input_emits_no_events(orc, eager):
    layers = NETS["same_pool"]
    _, ws, _ = _rand_net("f32", layers, 10, 10, 3, S=1, bias=False, seed=1)
    ev = orc.event_run("f32", layers, np.zeros((10, 10, 3)), ws, None, eager=eager)
    assert ev["events"].sum() == 0 and ev["updates"].sum() == 0
    assert np.all(ev["out"] == 0)
    assert np.all(orc.forward("f32", layers, np.zeros((1, 10, 10, 3)), ws, None) == 0)


def test_sparse_input_costs_proportionally_fewer_updates(orc):
    l = (conv(1, 4, 3),)
    _, ws, _ = _rand_net("f32", l, 12, 12, 1, S=1, bias=False, seed=1)
    x = np.zeros((12, 12, 1)); x[5, 5, 0] = 1.0; x[2, 9, 0] = -2.0
    ev = orc.event_run("f32", l, x, ws, None, eager=True)
    assert ev["events"][0] == 2 and ev["updates"][1] == 2 * 9 * 4


def _golden_int(name):
    path = os.path.join(os.path.dirname(__file__), "golden", name)
    vals = [ln.strip() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    return int(vals[0])


@pytest.mark.parametrize("length", [16, 64, 200])
def test_fig1_toy_net_stores_seven_activations(orc, length):
    """Fig. 1: two hidden layers with 3x1 kernels and one averaging output neuron need 7 stored
    activations whatever the input length."""
    seven = _golden_int("fig1_state_count.txt")
    layers = (conv(1, 1, 3, one_d=True, relu=0), conv(1, 1, 3, one_d=True, relu=0), Layer("avg"))
    r = np.random.default_rng(length)
    ws = [r.standard_normal((1, 3, 1, 1)) + 2.0, r.standard_normal((1, 3, 1, 1)) + 2.0, None]
    x = r.standard_normal((length, 1, 1)) + 3.0
    ev = orc.event_run("f32", layers, x, ws, None, eager=True)
    assert int(ev["live_between"][1:].sum()) == seven            # 2 + 4 + 1 between input steps
    ev = orc.event_run("f32", layers, x, ws, None, eager=False)
    assert int(ev["live_peak"][1:].sum()) == seven               # 3 + 3 + 1 with K-row rings
    want = orc.forward("f32", layers, x[None], ws, None)[0]
    np.testing.assert_allclose(ev["out"], want, rtol=1e-10)


def test_deferred_state_is_ring_of_k_rows_independent_of_height(orc):
    layers = (conv(2, 3, 3, pad=1), conv(3, 4, 3, stride=2), POOL)
    peaks = []
    for H in (12, 24):
        x, ws, bs = _rand_net("f32", layers, H, 10, 2, S=1, seed=H)
        x = np.abs(x) + 0.1
        ws = [None if w is None else np.abs(w) for w in ws]
        ev = orc.event_run("f32", layers, x[0], ws, None, eager=False)
        peaks.append(ev["live_peak"][1:].tolist())
    assert peaks[0] == peaks[1]
    # ceil(Kh/stride) rows of Wout*Cout for convs, one row for the pool
    assert peaks[0] == [3 * 10 * 3, 2 * 4 * 4, 1 * 2 * 4]
    # doubling the width doubles the state (2D memory is proportional to the row width)
    x, ws2, _ = _rand_net("f32", layers, 12, 20, 2, S=1, seed=1)
    ev = orc.event_run("f32", layers, np.abs(x[0]) + 0.1, [None if w is None else np.abs(w) for w in ws2], None, eager=False)
    assert ev["live_peak"][1] == 2 * peaks[0][0]


def test_causality_rows_do_not_depend_on_later_input(orc):
    layers = NETS["same_pool"]
    x, ws, bs = _rand_net("f32", layers, 16, 12, 3, S=1, seed=4)
    full = orc.forward("f32", layers, x, ws, bs)[0]
    x2 = x.copy(); x2[0, 10:] = 7.0
    alt = orc.forward("f32", layers, x2, ws, bs)[0]
    # receptive field of output row o ends at input row 4*o + 6: rows 0..0 are safe for r = 9
    safe = [o for o in range(full.shape[0]) if 4 * o + 6 <= 9]
    assert safe and np.array_equal(full[safe], alt[safe])
    assert not np.array_equal(full, alt)


@pytest.mark.parametrize("mode", ["f32", "i8"])
def test_output_sinks_reduce_to_matrix_product_and_mean(orc, mode):
    """A fully connected output layer is the conv layer whose kernel covers the whole map (one output position):
    it must equal a matrix-vector product over the flattened map; the global-average sink must equal the exact
    rational mean; and the event-by-event checker must reach both."""
    H, W, C, n_out = 5, 4, 3, 6
    fc = Layer("conv", C, n_out, H, W, H, 0, 0, 9 if mode == "i8" else 0, 0)
    x, ws, bs = _rand_net(mode, (fc,), H, W, C, S=3, seed=8)
    got = orc.forward(mode, (fc,), x, ws, bs)
    assert got.shape == (3, 1, 1, n_out)
    flat = torch.tensor(np.asarray(x, dtype=np.float64).reshape(3, -1))
    wmat = torch.tensor(np.asarray(ws[0], dtype=np.float64).reshape(n_out, -1))
    lin = torch.nn.functional.linear(flat, wmat, torch.tensor(np.asarray(bs[0], dtype=np.float64))).numpy()
    if mode == "i8":
        lin = np.clip(np.floor((lin + 2 ** 8) / 2 ** 9), -127, 127)
        assert np.array_equal(got.reshape(3, n_out), lin.astype(np.int64))
    else:
        np.testing.assert_allclose(got.reshape(3, n_out), lin, rtol=1e-12, atol=1e-12)
    ev = orc.event_run(mode, (fc,), x[0], ws, bs, eager=True)
    np.testing.assert_allclose(ev["out"].reshape(-1), got[0].reshape(-1), rtol=1e-10, atol=1e-10)
    # global average behind a conv layer: exact fractions
    from fractions import Fraction
    layers = (conv(C, 2, 3, shift=7 if mode == "i8" else 0), Layer("avg"))
    x, ws, bs = _rand_net(mode, layers, 6, 5, C, S=2, seed=9)
    maps = orc.forward(mode, layers, x, ws, bs, return_all=True)
    pre, avg = maps[-2], maps[-1]
    assert avg.shape == (2, 1, 1, 2)
    for s in range(2):
        for c in range(2):
            vals = pre[s, :, :, c].reshape(-1)
            exact = sum(Fraction(float(v)) for v in vals) / len(vals)
            assert abs(Fraction(float(avg[s, 0, 0, c])) - exact) <= abs(exact) * Fraction(1, 10 ** 12)


# ---- the per-segment form of the paper's eager rule (what the device's eager mode computes) --------------------
@pytest.mark.parametrize("mode", ["f32", "i8"])
@pytest.mark.parametrize("name", ["valid3", "same_pool", "stride2", "stride2_pad", "k5", "oned_k9", "oned_pad", "k3s3"])
def test_per_segment_eager_equals_component_eager_after_every_segment(orc, name, mode):
    """Delivering a whole segment before the layers re-evaluate changes when events are sent, not what the units
    hold once the segment has been absorbed (Eq. 3-5 telescope): after every segment the last layer's map equals
    that of the one-component-at-a-time rule, the final map equals Eq. 1, no more events are sent than one at a time,
    the input events are the same, and a stream that has seen only its first rows shows, in the rows nothing can reach
    any more, exactly the rows of the conventional result."""
    from helpers import SMALL_NETS, small_dims, with_shifts
    layers = SMALL_NETS[name]
    if mode == "i8":
        layers = with_shifts(layers, 6)
    H, W = small_dims(name)
    H = min(H, 25)
    C0 = next(l.cin for l in layers if l.kind == "conv")
    x, ws, _ = _rand_net(mode, layers, H, W, C0, S=1, bias=False, seed=31)
    want = orc.forward(mode, layers, x, ws, None)[0]
    one = orc.event_run(mode, layers, x[0], ws, None, eager=1, steps=True)
    seg = orc.event_run(mode, layers, x[0], ws, None, eager=2, steps=True)
    tol = 0 if mode == "i8" else 1e-9
    assert np.abs(seg["out"] - want).max() <= tol and np.abs(one["out"] - want).max() <= tol
    assert np.abs(seg["steps"] - one["steps"]).max() <= tol
    assert seg["telescoping_err"] <= tol
    assert seg["events"][0] == one["events"][0] == int((x != 0).sum())
    assert all(a <= b for a, b in zip(seg["events"], one["events"]))
    # presenting only the first rows gives the same snapshots as the full run (causality) ...
    part = orc.event_run(mode, layers, x[0], ws, None, eager=2, n_feed=H // 2, steps=True)
    assert np.array_equal(part["steps"], seg["steps"][:H // 2])
    # ... and rows that are final after r segments already hold the conventional values
    for r in range(H):
        rows = r + 1
        for l in layers:
            if l.kind == "conv":
                q = rows + l.pad - l.kh
                rows = 0 if q < 0 else q // l.stride + 1
            else:
                rows //= 2
        rows = min(rows, want.shape[0])
        assert np.abs(seg["steps"][r][:rows] - want[:rows]).max(initial=0) <= tol


def test_per_segment_eager_zero_input_sends_nothing(orc):
    layers = (conv(2, 3, 3, pad=1), POOL, conv(3, 2, 3))
    x, ws, _ = _rand_net("f32", layers, 12, 10, 2, S=1, bias=False, seed=2)
    res = orc.event_run("f32", layers, np.zeros_like(x[0]), ws, None, eager=2, steps=True)
    assert not res["events"].any() and not res["steps"].any()
