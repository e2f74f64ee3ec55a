"""Shared helpers of the tests (no arithmetic of the method lives here)."""
import numpy as np
import torch

from paper_1804_10727_b200.workloads import Layer, conv, POOL

# the tolerance for floating-point nets: |gpu - oracle| <= ATOL + RTOL * |oracle|
RTOL, ATOL = 1e-3, 1e-4


def assert_close(got, want, what=""):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (got.shape, want.shape)
    err = np.abs(got - want)
    lim = ATOL + RTOL * np.abs(want)
    bad = err > lim
    if bad.any():
        i = np.unravel_index(np.argmax(err - lim), err.shape)
        raise AssertionError(f"{what}: {bad.sum()} of {bad.size} outside tolerance; worst at {i}: got {got[i]!r} want {want[i]!r}")


def assert_equal(got, want, what=""):
    got = np.asarray(got).astype(np.int64)
    want = np.asarray(want).astype(np.int64)
    assert got.shape == want.shape, (got.shape, want.shape)
    if not np.array_equal(got, want):
        bad = got != want
        i = np.unravel_index(np.argmax(bad), bad.shape)
        raise AssertionError(f"{what}: {bad.sum()} of {bad.size} differ; first at {i}: got {got[i]} want {want[i]}")


def bf16_values(a):
    return torch.tensor(np.asarray(a), dtype=torch.float32).bfloat16().float().numpy()


def rand_net(mode, layers, H, W, C0, S=2, bias=True, seed=0, zero_frac=0.5):
    """Random input and parameters for a small net (test data only)."""
    r = np.random.default_rng(seed)
    if mode == "i8":
        x = r.integers(-127, 128, size=(S, H, W, C0)).astype(np.int8)
        x[r.random(x.shape) < zero_frac] = 0
    else:
        x = r.standard_normal((S, H, W, C0)).astype(np.float32)
        if mode == "bf16":
            x = bf16_values(x)
    ws, bs = [], []
    for l in layers:
        if l.kind != "conv":
            ws.append(None); bs.append(None); continue
        if mode == "i8":
            ws.append(r.integers(-127, 128, size=(l.cout, l.kh, l.kw, l.cin)).astype(np.int8))
            bs.append(r.integers(-500, 500, size=(l.cout,)).astype(np.int32) if bias else None)
        else:
            w = (r.standard_normal((l.cout, l.kh, l.kw, l.cin)) * (2.0 / (l.cin * l.kh * l.kw)) ** 0.5).astype(np.float32)
            if mode == "bf16":
                w = bf16_values(w)
            ws.append(w)
            bs.append((r.standard_normal((l.cout,)) * 0.1).astype(np.float32) if bias else None)
    return x, ws, bs


def with_shifts(layers, s=8):
    return tuple(Layer(**{**l.__dict__, "shift": s}) if l.kind == "conv" else l for l in layers)


def with_path(layers, path):
    return tuple(Layer(**{**l.__dict__, "path": path}) if l.kind == "conv" else l for l in layers)


SMALL_NETS = {
    "valid3": (conv(2, 4, 3), conv(4, 3, 3)),
    "same_pool": (conv(3, 4, 3, pad=1), POOL, conv(4, 5, 3, pad=1), POOL),
    "stride2": (conv(2, 4, 3, stride=2), conv(4, 4, 3, stride=1), POOL),
    "stride2_pad": (conv(2, 3, 3, stride=2, pad=1), conv(3, 4, 3, stride=2, pad=1)),
    "oned_k9": (conv(1, 4, 9, stride=2, one_d=True), conv(4, 5, 9, one_d=True)),
    "oned_k3": (conv(1, 8, 3, one_d=True), conv(8, 8, 3, one_d=True), conv(8, 4, 3, one_d=True)),
    "oned_pad": (conv(2, 3, 5, stride=2, pad=2, one_d=True), POOL, conv(3, 4, 3, pad=1, one_d=True)),
    "k5": (conv(2, 3, 5, stride=2, pad=2), conv(3, 2, 3)),
    "norelu": (conv(2, 3, 3, relu=0), conv(3, 2, 3, relu=0)),
    "pool_first": (POOL, conv(2, 3, 3, pad=1)),
    "k3s3": (conv(2, 3, 3, stride=3, pad=1), conv(3, 3, 2, stride=2)),
}


def small_dims(name):
    return (61, 1) if name.startswith("oned") else (19, 14)


# End-to-end criterion for the bf16 workloads (every hidden activation is a rounding decision on an fp32 sum in
# tensor-core order; the strict tolerance holds layer by layer, see test_full_size_gpu.py): about twice what is measured
# (vgg2d: relative rms 2^-9.3, largest error 2^-8.1 of max|o|, 66 % of the outputs inside 1e-4 + 1e-3|o|;
#  audio1d: 2^-11.1 ... 2^-11.5, 2^-8.8, 96-98 %).
BF16_E2E = {"vgg2d": (2.0 ** -8.3, 2.0 ** -7.1, 0.55), "audio1d": (2.0 ** -10.1, 2.0 ** -7.8, 0.93)}


def assert_bf16_end_to_end(name, got, want, what=""):
    rms_lim, max_lim, frac_lim = BF16_E2E[name]
    err = np.asarray(got, dtype=np.float64) - np.asarray(want, dtype=np.float64)
    rel_rms = np.sqrt((err ** 2).mean() / (want ** 2).mean())
    rel_max = np.abs(err).max() / np.abs(want).max()
    frac = (np.abs(err) <= ATOL + RTOL * np.abs(want)).mean()
    print(f"{what}: relative rms 2^{np.log2(rel_rms):.2f}, largest error 2^{np.log2(rel_max):.2f} of max|o|, {100 * frac:.1f} % inside the strict tolerance")
    assert rel_rms < rms_lim and rel_max < max_lim and frac > frac_lim, (what, rel_rms, rel_max, frac)
