"""Seeded synthetic workloads: net descriptions, inputs and parameters.

This module only *describes* nets and draws random data; it contains none of
the method's arithmetic and is the one piece shared by the CUDA path, the CPU
oracle, the tests and the benchmark.  Everything is generated on the CPU with a
seeded ``torch.Generator`` in blocks of ``BLOCK`` streams, so the first k
streams of a workload are the same whatever total stream count is requested.

The five workloads stand in for the uses the paper names (row-by-row MNIST
classification in its experiment section; audio and embedded vision in its
introduction); no item of any dataset is used.

  toy1d    1D, fp32:   4096 samples N(0,1); conv k3 1->8->8->4, ReLU, bias 0.01, 1 stream, seed 0
  mnist2d  2D, int8:   28x28x1, U[0,1] with 80 % of pixels zeroed, q = round(127 u);
                       conv3x3 1->16, 16->32, maxpool2, conv3x3 32->32, ReLU; 4096 streams, seed 1
  audio1d  1D, bf16:   16000 samples of Gaussian noise low-passed (brick wall) at 4 kHz of 16 kHz,
                       unit variance; conv k9 1->32->64->64->128->128->128, stride 2,2,2,1,1,1; 1024 streams, seed 2
  vgg2d    2D, bf16:   224x224x3 N(0,1); conv3x3 same-padding 64,64,pool,128,128,pool,256,256,256,pool; 64 streams, seed 3
  events2d 2D, int8:   256x256x2, 3 % of entries non-zero with value +1/-1; conv3x3 2->32 (s1), 32->64 (s2),
                       64->64 (s1), ReLU, maxpool2; 2048 streams, seed 4

Weights ~ N(0, var) with var = 1/(Cin*k) for toy1d and 2/(Cin*Kh*Kw) for the
others; bf16 nets round them to bfloat16; int8 nets quantise them symmetrically
per layer to [-127, 127].  The requantisation shifts of the int8 nets were
calibrated once on the CPU oracle (oracle/calibrate_shifts.py) and are frozen
in ``_SHIFTS`` below.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Optional

import numpy as np
import torch

BLOCK = 32  # streams per generator block


@dataclass(frozen=True)
class Layer:
    kind: str = "conv"          # 'conv' | 'pool' | 'avg' (global-average output sink, last layer only)
    cin: int = 0
    cout: int = 0
    kh: int = 1
    kw: int = 1
    stride: int = 1
    pad: int = 0
    relu: int = 1
    shift: int = 0              # int8 nets: requantisation shift
    path: int = 0               # 0 auto, 1 dense, 2 sparse


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: str                  # 'f32' | 'bf16' | 'i8'
    H: int                      # number of segments (rows / samples) per stream
    W: int                      # row width (1 for 1D)
    C: int                      # input channels
    n_streams: int
    layers: tuple
    seed: int
    bias: float = 0.0
    weight_var_gain: float = 2.0

    @property
    def pixels_per_stream(self) -> int:
        return self.H * self.W


def conv(cin, cout, k, stride=1, pad=0, one_d=False, shift=0, relu=1, path=0) -> Layer:
    return Layer("conv", cin, cout, k, 1 if one_d else k, stride, pad, relu, shift, path)


POOL = Layer("pool")

# Requantisation shifts calibrated on the oracle (smallest shift that keeps the 99.9th
# percentile of the pre-clamp activation at or below 127); written by oracle/calibrate_shifts.py.
_SHIFTS = {
    "mnist2d": (8, 8, 9),
    "events2d": (0, 9, 9),
}


def _mk(name: str) -> Workload:
    if name == "toy1d":
        ls = (conv(1, 8, 3, one_d=True), conv(8, 8, 3, one_d=True), conv(8, 4, 3, one_d=True))
        return Workload(name, "f32", 4096, 1, 1, 1, ls, 0, bias=0.01, weight_var_gain=1.0)
    if name == "mnist2d":
        s = _SHIFTS[name]
        ls = (conv(1, 16, 3, shift=s[0]), conv(16, 32, 3, shift=s[1]), POOL, conv(32, 32, 3, shift=s[2]))
        return Workload(name, "i8", 28, 28, 1, 4096, ls, 1)
    if name == "audio1d":
        ch = (1, 32, 64, 64, 128, 128, 128)
        st = (2, 2, 2, 1, 1, 1)
        ls = tuple(conv(ch[i], ch[i + 1], 9, st[i], one_d=True) for i in range(6))
        return Workload(name, "bf16", 16000, 1, 1, 1024, ls, 2)
    if name == "vgg2d":
        ls = (conv(3, 64, 3, pad=1), conv(64, 64, 3, pad=1), POOL,
              conv(64, 128, 3, pad=1), conv(128, 128, 3, pad=1), POOL,
              conv(128, 256, 3, pad=1), conv(256, 256, 3, pad=1), conv(256, 256, 3, pad=1), POOL)
        return Workload(name, "bf16", 224, 224, 3, 64, ls, 3)
    if name == "events2d":
        s = _SHIFTS[name]
        ls = (conv(2, 32, 3, 1, shift=s[0]), conv(32, 64, 3, 2, shift=s[1]), conv(64, 64, 3, 1, shift=s[2]), POOL)
        return Workload(name, "i8", 256, 256, 2, 2048, ls, 4)
    raise KeyError(name)


NAMES = ("toy1d", "mnist2d", "audio1d", "vgg2d", "events2d")


def get(name: str, n_streams: Optional[int] = None, H: Optional[int] = None, W: Optional[int] = None) -> Workload:
    """The named workload, optionally with fewer streams or a smaller extent (same recipe)."""
    w = _mk(name)
    kw = {}
    if n_streams is not None:
        kw["n_streams"] = int(n_streams)
    if H is not None:
        kw["H"] = int(H)
    if W is not None:
        kw["W"] = int(W)
    return replace(w, **kw) if kw else w


def _gen(seed: int, block: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed((seed + 1) * 1_000_003 + block)
    return g


def _to_bf16_values(t: torch.Tensor) -> torch.Tensor:
    return t.to(torch.bfloat16).to(torch.float32)


def _input_block(w: Workload, block: int) -> np.ndarray:
    g = _gen(w.seed, block)
    shape = (BLOCK, w.H, w.W, w.C)
    if w.name == "toy1d":
        return torch.randn(shape, generator=g, dtype=torch.float32).numpy()
    if w.name == "mnist2d":
        u = torch.rand(shape, generator=g, dtype=torch.float32)
        keep = torch.rand(shape, generator=g, dtype=torch.float32) >= 0.8
        return torch.round(127.0 * u * keep).to(torch.int8).numpy()
    if w.name == "audio1d":
        x = torch.randn((BLOCK, w.H), generator=g, dtype=torch.float64)
        spec = torch.fft.rfft(x, dim=1)
        freqs = torch.fft.rfftfreq(w.H, d=1.0 / 16000.0)
        spec[:, freqs > 4000.0] = 0
        y = torch.fft.irfft(spec, n=w.H, dim=1)
        y = y / y.std(dim=1, keepdim=True)
        return _to_bf16_values(y.to(torch.float32)).reshape(shape).numpy()
    if w.name == "vgg2d":
        return _to_bf16_values(torch.randn(shape, generator=g, dtype=torch.float32)).numpy()
    if w.name == "events2d":
        nz = torch.rand(shape, generator=g, dtype=torch.float32) < 0.03
        sign = torch.rand(shape, generator=g, dtype=torch.float32) < 0.5
        v = torch.where(sign, torch.ones(()), -torch.ones(()))
        return (v * nz).to(torch.int8).numpy()
    raise KeyError(w.name)


def make_input(w: Workload, first: int = 0, count: Optional[int] = None) -> np.ndarray:
    """Input of streams [first, first+count): ``[count][H][W][C]``, float32 (f32/bf16 nets;
    bf16 nets hold bfloat16-representable values) or int8."""
    count = w.n_streams - first if count is None else count
    out = []
    b0, b1 = first // BLOCK, (first + count + BLOCK - 1) // BLOCK
    for b in range(b0, b1):
        out.append(_input_block(w, b))
    a = np.concatenate(out, axis=0) if out else np.zeros((0, w.H, w.W, w.C), dtype=np.float32)
    lo = first - b0 * BLOCK
    return np.ascontiguousarray(a[lo:lo + count])


def make_params(w: Workload):
    """(weights, biases): one entry per layer, None for non-conv layers.

    weights[i]: ``[Cout][Kh][Kw][Cin]`` float32 (f32, bf16-valued for bf16 nets) or int8;
    biases[i]: ``[Cout]`` float32 / int32, or None when the workload's bias is zero.
    """
    g = _gen(w.seed, 1 << 20)
    ws: List[Optional[np.ndarray]] = []
    bs: List[Optional[np.ndarray]] = []
    for l in w.layers:
        if l.kind != "conv":
            ws.append(None)
            bs.append(None)
            continue
        fan = l.cin * l.kh * l.kw
        std = (w.weight_var_gain / fan) ** 0.5
        t = torch.randn((l.cout, l.kh, l.kw, l.cin), generator=g, dtype=torch.float32) * std
        if w.dtype == "bf16":
            t = _to_bf16_values(t)
        if w.dtype == "i8":
            scale = 127.0 / float(t.abs().max())
            ws.append(torch.round(t * scale).clamp(-127, 127).to(torch.int8).numpy())
        else:
            ws.append(t.numpy())
        if w.bias != 0.0:
            if w.dtype == "i8":
                bs.append(np.full((l.cout,), int(round(w.bias)), dtype=np.int32))
            else:
                bs.append(np.full((l.cout,), w.bias, dtype=np.float32))
        else:
            bs.append(None)
    return ws, bs
