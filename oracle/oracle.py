"""Python face of the CPU oracle (test infrastructure only).

Loads the two plain-C files of this directory (the layer-by-layer forward pass
of Eq. 1 and the event-by-event checker of Eq. 2-5) through ctypes and drives
them one layer at a time.  Nothing here is used by the product path: only the
tests, the smoke check and the CPU-baseline leg of the benchmark import it.

A net is described by plain dicts/objects with the attributes
``kind ('conv'|'pool'|'avg'), cin, cout, kh, kw, stride, pad, relu, shift``;
maps are numpy arrays ``[n_streams][H][W][C]`` (channels innermost), weights
``[Cout][Kh][Kw][Cin]``.

Numeric modes (the paper fixes no number format; these are this build's):
  'f32'   everything in float64 (the exact result the fp32 device path approximates)
  'bf16'  float64 accumulation; the activation of a conv layer that feeds a later
          conv layer is rounded to the nearest bfloat16 (ties to even); the last
          conv layer (and anything after it) stays unrounded
  'i8'    int32 accumulation, then shift-requantisation to the int8 range per conv layer
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_LIB_PATH = _HERE / "liboracle.so"
_SOURCES = [_HERE / "idf_oracle.c", _HERE / "idf_event_checker.c"]
_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle's C sources into ``liboracle.so`` next to them."""
    newest = max(p.stat().st_mtime for p in _SOURCES)
    if not force and _LIB_PATH.exists() and _LIB_PATH.stat().st_mtime >= newest:
        return _LIB_PATH
    tmp = _LIB_PATH.with_suffix(f".tmp{os.getpid()}.so")
    cmd = ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-Wall", "-o", str(tmp)] + [str(p) for p in _SOURCES] + ["-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(str(_LIB_PATH))
        _lib.orc_num_threads.restype = ctypes.c_int
        _lib.evc_run.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct)) if a is not None else None


def _kind(layer) -> str:
    k = layer.kind if hasattr(layer, "kind") else layer["kind"]
    return {0: "conv", 1: "pool", 2: "avg"}.get(k, k)


def _g(layer, name):
    return getattr(layer, name) if hasattr(layer, name) else layer[name]


def conv_out(n: int, k: int, stride: int, pad: int) -> int:
    return (n + 2 * pad - k) // stride + 1


def out_shape(layers, H: int, W: int, C: int):
    """Shape of every map, input first: list of (H, W, C)."""
    shapes = [(H, W, C)]
    for l in layers:
        kind = _kind(l)
        if kind == "conv":
            one_d = (W == 1 and _g(l, "kw") == 1)
            H = conv_out(H, _g(l, "kh"), _g(l, "stride"), _g(l, "pad"))
            W = 1 if one_d else conv_out(W, _g(l, "kw"), _g(l, "stride"), _g(l, "pad"))
            C = _g(l, "cout")
        elif kind == "pool":
            H, W = H // 2, (1 if W == 1 else W // 2)
        else:
            H, W = 1, 1
        shapes.append((H, W, C))
    return shapes


def round_bf16(a: np.ndarray) -> np.ndarray:
    out = np.ascontiguousarray(a, dtype=np.float64).copy()
    lib().orc_round_bf16(_p(out, ctypes.c_double), ctypes.c_longlong(out.size))
    return out


def requant(c: np.ndarray, shift: int, relu: int) -> np.ndarray:
    out = np.ascontiguousarray(c, dtype=np.int32).copy()
    lib().orc_requant_i32(_p(out, ctypes.c_int32), ctypes.c_longlong(out.size), int(shift), int(relu))
    return out


def conv_layer(mode: str, layer, x: np.ndarray, w: np.ndarray, b) -> np.ndarray:
    """One conv layer of Eq. 1 on whole maps; returns f(c) before any rounding/requantisation."""
    S, H, W, Cin = x.shape
    Cout, Kh, Kw = _g(layer, "cout"), _g(layer, "kh"), _g(layer, "kw")
    st, pd, relu = _g(layer, "stride"), _g(layer, "pad"), _g(layer, "relu")
    assert Cin == _g(layer, "cin") and w.shape == (Cout, Kh, Kw, Cin), (x.shape, w.shape)
    Ho = conv_out(H, Kh, st, pd)
    Wo = 1 if (W == 1 and Kw == 1) else conv_out(W, Kw, st, pd)     # 1D: degenerate x axis
    assert Ho >= 1 and Wo >= 1
    L = lib()
    if mode == "i8":
        xi = np.ascontiguousarray(x, dtype=np.int32)
        wi = np.ascontiguousarray(w, dtype=np.int32)
        bi = None if b is None else np.ascontiguousarray(b, dtype=np.int32)
        out = np.zeros((S, Ho, Wo, Cout), dtype=np.int32)
        L.orc_conv_i32(_p(xi, ctypes.c_int32), ctypes.c_longlong(S), H, W, Cin, _p(wi, ctypes.c_int32),
                       _p(bi, ctypes.c_int32), Cout, Kh, Kw, st, pd, int(relu), _p(out, ctypes.c_int32))
        return out
    xd = np.ascontiguousarray(x, dtype=np.float64)
    wd = np.ascontiguousarray(w, dtype=np.float64)
    bd = None if b is None else np.ascontiguousarray(b, dtype=np.float64)
    out = np.zeros((S, Ho, Wo, Cout), dtype=np.float64)
    L.orc_conv_f64(_p(xd, ctypes.c_double), ctypes.c_longlong(S), H, W, Cin, _p(wd, ctypes.c_double),
                   _p(bd, ctypes.c_double), Cout, Kh, Kw, st, pd, int(relu), _p(out, ctypes.c_double))
    return out


def pool_layer(mode: str, x: np.ndarray) -> np.ndarray:
    S, H, W, C = x.shape
    Ho, Wo = H // 2, (1 if W == 1 else W // 2)
    L = lib()
    if mode == "i8":
        xi = np.ascontiguousarray(x, dtype=np.int32)
        out = np.zeros((S, Ho, Wo, C), dtype=np.int32)
        L.orc_maxpool2_i32(_p(xi, ctypes.c_int32), ctypes.c_longlong(S), H, W, C, _p(out, ctypes.c_int32))
        return out
    xd = np.ascontiguousarray(x, dtype=np.float64)
    out = np.zeros((S, Ho, Wo, C), dtype=np.float64)
    L.orc_maxpool2_f64(_p(xd, ctypes.c_double), ctypes.c_longlong(S), H, W, C, _p(out, ctypes.c_double))
    return out


def forward(mode: str, layers, x: np.ndarray, weights, biases=None, return_all: bool = False):
    """Layer-by-layer forward pass (Eq. 1) of a whole net on whole maps.

    ``weights``/``biases``: one entry per layer (None for non-conv layers).
    Returns the final map (float64 for float modes, int32 holding int8-range
    values for 'i8'); with ``return_all`` the list of all maps, input first,
    each as the next layer receives it.
    """
    assert mode in ("f32", "bf16", "i8")
    a = np.ascontiguousarray(x, dtype=np.int32 if mode == "i8" else np.float64)
    maps = [a]
    conv_idx = [i for i, l in enumerate(layers) if _kind(l) == "conv"]
    last_conv = conv_idx[-1] if conv_idx else -1
    for i, l in enumerate(layers):
        kind = _kind(l)
        if kind == "conv":
            b = None if biases is None else biases[i]
            a = conv_layer(mode, l, a, weights[i], b)
            if mode == "bf16" and i != last_conv:
                a = round_bf16(a)
            elif mode == "i8":
                a = requant(a, _g(l, "shift"), _g(l, "relu"))
        elif kind == "pool":
            a = pool_layer(mode, a)
        elif kind == "avg":
            a = a.astype(np.float64).mean(axis=(1, 2), keepdims=True)
        else:
            raise ValueError(kind)
        maps.append(a)
    return maps if return_all else a


# ----------------------------------------------------------------------------------------------
# event-by-event checker
# ----------------------------------------------------------------------------------------------
class _EvcLayer(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("kind", "cin", "cout", "kh", "kw", "stride", "pad", "relu", "shift")]


def event_run(mode: str, layers, x: np.ndarray, weights, biases=None, eager=True, n_feed=None, steps: bool = False):
    """Run ONE stream (x: [H][W][C]) through the event-by-event checker (Eq. 2-5).

    ``eager``: False/0 = a unit emits once when nothing can reach it any more; True/1 = the paper's rule, one input
    component at a time; 2 = the paper's rule with a whole segment delivered before the layers re-evaluate.
    ``n_feed``: present only the first n_feed rows (the maps stay sized for all H rows: a stream that does not know
    where its input ends).  ``steps``: also return the last layer's map after every presented row.

    Returns a dict: out (final map of the last layer), sum_dh (sum of the last
    layer's emitted events per unit), events / updates (per layer, index 0 =
    input), live_between, live_peak (units holding reachable state, per layer),
    telescoping_err, and steps ([n_feed][Hout][Wout][C]) if asked for.
    """
    H, W, C0 = x.shape
    n_feed = H if n_feed is None else int(n_feed)
    n = len(layers)
    arr = (_EvcLayer * n)()
    kinds = {"conv": 0, "pool": 1, "avg": 2}
    for i, l in enumerate(layers):
        k = _kind(l)
        arr[i].kind = kinds[k]
        for f in ("cin", "cout", "kh", "kw", "stride", "pad", "relu", "shift"):
            setattr(arr[i], f, int(_g(l, f)) if k == "conv" else 0)
    wk, bk = [], []
    wptr = (ctypes.POINTER(ctypes.c_double) * n)()
    bptr = (ctypes.POINTER(ctypes.c_double) * n)()
    for i in range(n):
        if weights[i] is not None:
            wk.append(np.ascontiguousarray(weights[i], dtype=np.float64))
            wptr[i] = _p(wk[-1], ctypes.c_double)
        if biases is not None and biases[i] is not None:
            bk.append(np.ascontiguousarray(biases[i], dtype=np.float64))
            bptr[i] = _p(bk[-1], ctypes.c_double)
    shapes = out_shape(layers, H, W, C0)
    oh, ow, oc = shapes[-1]
    out = np.zeros((oh, ow, oc), dtype=np.float64)
    sdh = np.zeros_like(out)
    st = np.zeros(n + 1, dtype=np.int64)
    st2 = np.zeros(n + 1, dtype=np.int64)
    lb = np.zeros(n + 1, dtype=np.int64)
    lp = np.zeros(n + 1, dtype=np.int64)
    terr = ctypes.c_double(0)
    xd = np.ascontiguousarray(x, dtype=np.float64)
    snap = np.zeros((n_feed, oh, ow, oc), dtype=np.float64) if steps else None
    modes = {"f32": 0, "bf16": 1, "i8": 2}
    rc = lib().evc_run_steps(modes[mode], int(eager), n, arr, wptr, bptr, H, W, C0, _p(xd, ctypes.c_double),
                             ctypes.c_int(n_feed), _p(snap, ctypes.c_double) if steps else None,
                             _p(out, ctypes.c_double), _p(sdh, ctypes.c_double), _p(st, ctypes.c_longlong),
                             _p(st2, ctypes.c_longlong), _p(lb, ctypes.c_longlong), _p(lp, ctypes.c_longlong),
                             ctypes.byref(terr))
    if rc != 0:
        raise ValueError("event checker rejected the net")
    res = dict(out=out, sum_dh=sdh, events=st, updates=st2, live_between=lb, live_peak=lp,
               telescoping_err=float(terr.value))
    if steps:
        res["steps"] = snap
    return res
