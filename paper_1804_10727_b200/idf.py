"""Thin ctypes binding over the C ABI in ``include/idf.h`` (argument marshalling only).

PyTorch provides device memory and CUDA streams; every step of the path runs in
the library's kernels.  There is no fallback: if ``libidf.so`` has not been
built, loading raises.
"""
from __future__ import annotations

import ctypes
from pathlib import Path
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = Path(__file__).resolve().parent
LIB_PATH = _HERE / "libidf.so"
BOUNDS_LIB_PATH = _HERE / "libidf_bounds.so"      # the range-checked build of the same sources (-DIDF_BOUNDS)
_lib = None


def use_library(path) -> None:
    """Load the library from ``path`` from now on (e.g. ``BOUNDS_LIB_PATH``); handles made before stay with theirs."""
    global _lib, LIB_PATH
    LIB_PATH = Path(path)
    _lib = None

F32, BF16_F32, I8_I32 = 0, 1, 2
CONV, MAXPOOL2, GLOBAL_AVG = 0, 1, 2
PATH_AUTO, PATH_DENSE, PATH_SPARSE = 0, 1, 2
DTYPES = {"f32": F32, "bf16": BF16_F32, "i8": I8_I32}

OK, ERR_ARG, ERR_SPEC, ERR_STATE, ERR_CAPACITY, ERR_UNSUPPORTED, ERR_CUDA, ERR_TIMEOUT, ERR_BOUNDS = 0, -1, -2, -3, -4, -5, -6, -7, -8

EXPORTS = (
    "idf_net_create", "idf_net_destroy", "idf_net_state_bytes", "idf_net_workspace_bytes", "idf_out_shape",
    "idf_stream_open", "idf_stream_reset", "idf_stream_push", "idf_stream_push_last", "idf_stream_finish", "idf_run_host", "idf_event_counts",
    "idf_launch_count", "idf_stream_status", "idf_set_timing", "idf_layer_times", "idf_conv_rows_noalloc", "idf_last_error",
    "idf_state_snapshot_bytes", "idf_state_save", "idf_state_restore", "idf_stream_set_out_base", "idf_set_debug_flags", "idf_out_rows_needed",
)
DEBUG_NO_TENSOR_CORES, DEBUG_NO_POOL_FUSION, DEBUG_NO_ROW_CHUNKS, DEBUG_NO_PDL, DEBUG_PREFER_THIN = 1, 2, 4, 8, 16
DEBUG_NO_FUSED, DEBUG_FORCE_FUSED = 32, 64


class IdfLayer(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("kind", "cin", "cout", "kh", "kw", "stride", "pad", "relu", "shift", "path")]


class IdfSpec(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int), ("layers", ctypes.POINTER(IdfLayer)), ("dtype", ctypes.c_int),
                ("in_w", ctypes.c_int), ("in_c", ctypes.c_int), ("n_streams", ctypes.c_int),
                ("row_block", ctypes.c_int), ("emission", ctypes.c_int)]


class IdfError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"idf error {code}: {msg}")
        self.code = code


def lib():
    """Load ``libidf.so`` (built by ``python -m paper_1804_10727_b200.build``)."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_1804_10727_b200.build` "
                               "(there is no CPU fallback)")
        L = ctypes.CDLL(str(LIB_PATH))
        vp, ll, sz = ctypes.c_void_p, ctypes.c_longlong, ctypes.c_size_t
        L.idf_net_create.argtypes = [ctypes.POINTER(IdfSpec), ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(vp)]
        L.idf_net_destroy.argtypes = [vp]
        L.idf_net_state_bytes.argtypes = [vp]; L.idf_net_state_bytes.restype = sz
        L.idf_net_workspace_bytes.argtypes = [vp]; L.idf_net_workspace_bytes.restype = sz
        L.idf_out_shape.argtypes = [vp, ll, ctypes.POINTER(ll), ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_int)]
        L.idf_stream_open.argtypes = [vp, vp, sz, vp]
        L.idf_stream_reset.argtypes = [vp]
        L.idf_stream_push.argtypes = [vp, vp, ctypes.c_int, vp, ll, ctypes.POINTER(ctypes.c_int)]
        L.idf_stream_finish.argtypes = [vp, vp, ll, ctypes.POINTER(ll)]
        L.idf_stream_push_last.argtypes = [vp, vp, ctypes.c_int, vp, ll, ctypes.POINTER(ll)]
        L.idf_run_host.argtypes = [vp, vp, ctypes.c_int, vp, vp, vp, ll, ctypes.POINTER(ll)]
        L.idf_event_counts.argtypes = [vp, ctypes.POINTER(ll)]
        L.idf_launch_count.argtypes = [vp]; L.idf_launch_count.restype = ll
        L.idf_stream_status.argtypes = [vp, ctypes.POINTER(ll)]
        L.idf_set_timing.argtypes = [vp, ctypes.c_int]
        L.idf_layer_times.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ll)]
        L.idf_conv_rows_noalloc.argtypes = [vp, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, vp, vp,
                                            ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                            ctypes.c_int, vp, ll, ctypes.POINTER(ll), vp]
        L.idf_stream_set_out_base.argtypes = [vp, ll]
        L.idf_state_snapshot_bytes.argtypes = [vp]; L.idf_state_snapshot_bytes.restype = sz
        L.idf_state_save.argtypes = [vp, vp, sz]
        L.idf_state_restore.argtypes = [vp, vp, sz]
        L.idf_set_debug_flags.argtypes = [ctypes.c_uint]
        L.idf_out_rows_needed.argtypes = [vp, ll]; L.idf_out_rows_needed.restype = ll
        L.idf_last_error.restype = ctypes.c_char_p
        _lib = L
    return _lib


def _check(rc: int):
    if rc != 0:
        raise IdfError(rc, lib().idf_last_error().decode())


def set_debug_flags(flags: int):
    """Debug only: route work away from the default kernels (see idf_set_debug_flags); 0 restores the defaults."""
    _check(lib().idf_set_debug_flags(int(flags)))


def _layer_struct(l) -> IdfLayer:
    kind = l.kind if isinstance(l.kind, int) else {"conv": CONV, "pool": MAXPOOL2, "avg": GLOBAL_AVG}[l.kind]
    return IdfLayer(kind, l.cin, l.cout, l.kh, l.kw, l.stride, l.pad, l.relu, l.shift, l.path)


def _act_torch_dtype(dtype: int):
    return {F32: torch.float32, BF16_F32: torch.bfloat16, I8_I32: torch.int8}[dtype]


def to_act_bits(a: np.ndarray, dtype: int) -> np.ndarray:
    """Host array in the activation type's memory format (bf16 -> uint16 bit patterns)."""
    if dtype == F32:
        return np.ascontiguousarray(a, dtype=np.float32)
    if dtype == I8_I32:
        return np.ascontiguousarray(a, dtype=np.int8)
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


class Net:
    """A net handle: ``net_create`` on construction, ``net_destroy`` on close()."""

    def __init__(self, dtype, layers: Sequence, in_w: int, in_c: int, n_streams: int,
                 weights: Sequence[Optional[np.ndarray]], biases: Optional[Sequence[Optional[np.ndarray]]] = None,
                 row_block: int = 0, eager: bool = False):
        self.dtype = DTYPES[dtype] if isinstance(dtype, str) else int(dtype)
        self.n_streams, self.in_w, self.in_c = int(n_streams), int(in_w), int(in_c)
        n = len(layers)
        self._layers = (IdfLayer * n)(*[_layer_struct(l) for l in layers])
        spec = IdfSpec(n, self._layers, self.dtype, in_w, in_c, n_streams, row_block, 1 if eager else 0)
        keep = []
        wptr = (ctypes.c_void_p * n)()
        bptr = (ctypes.c_void_p * n)()
        for i in range(n):
            if weights[i] is not None:
                w = to_act_bits(weights[i], self.dtype)
                keep.append(w)
                wptr[i] = w.ctypes.data
            if biases is not None and biases[i] is not None:
                b = np.ascontiguousarray(biases[i], dtype=np.int32 if self.dtype == I8_I32 else np.float32)
                keep.append(b)
                bptr[i] = b.ctypes.data
        h = ctypes.c_void_p()
        _check(lib().idf_net_create(ctypes.byref(spec), wptr, bptr, ctypes.byref(h)))
        self._h = h
        self._ws = None
        self.n_layers = n
        self._avg_sink = int(self._layers[n - 1].kind) == GLOBAL_AVG

    # -- queries ---------------------------------------------------------------------------------
    @property
    def state_bytes(self) -> int:
        return int(lib().idf_net_state_bytes(self._h))

    @property
    def workspace_bytes(self) -> int:
        return int(lib().idf_net_workspace_bytes(self._h))

    def out_shape(self, in_rows: int):
        r, w, c = ctypes.c_longlong(), ctypes.c_int(), ctypes.c_int()
        _check(lib().idf_out_shape(self._h, in_rows, ctypes.byref(r), ctypes.byref(w), ctypes.byref(c)))
        return int(r.value), int(w.value), int(c.value)

    @property
    def out_torch_dtype(self):
        return torch.int8 if self.dtype == I8_I32 and not self._avg_sink else torch.float32

    @property
    def act_torch_dtype(self):
        return _act_torch_dtype(self.dtype)

    @property
    def launches(self) -> int:
        return int(lib().idf_launch_count(self._h))

    def event_counts(self):
        ev = (ctypes.c_longlong * self.n_layers)()
        _check(lib().idf_event_counts(self._h, ev))
        return list(ev)

    def status(self):
        """Synchronise; raise if a kernel gave up on a bounded wait; return tensor-core launches per layer."""
        n = (ctypes.c_longlong * self.n_layers)()
        _check(lib().idf_stream_status(self._h, n))
        return list(n)

    def set_timing(self, on: bool):
        _check(lib().idf_set_timing(self._h, int(on)))

    def layer_times(self):
        """(ms, launches) per layer since the last query; synchronises the stream."""
        ms = (ctypes.c_double * self.n_layers)()
        n = (ctypes.c_longlong * self.n_layers)()
        _check(lib().idf_layer_times(self._h, ms, n))
        return list(ms), list(n)

    # -- streaming -------------------------------------------------------------------------------
    def open(self, device="cuda:0", stream: Optional[torch.cuda.Stream] = None, workspace: Optional[torch.Tensor] = None):
        if workspace is None:
            if self._ws is None or self._ws.device != torch.device(device):
                self._ws = torch.empty(self.workspace_bytes + 256, dtype=torch.uint8, device=device)
            workspace = self._ws
        self._ws = workspace
        base = workspace.data_ptr()
        aligned = (base + 255) // 256 * 256
        nbytes = workspace.numel() - (aligned - base)
        st = stream.cuda_stream if stream is not None else torch.cuda.current_stream(workspace.device).cuda_stream
        _check(lib().idf_stream_open(self._h, aligned, nbytes, st))

    def reset(self):
        """New streams on the workspace of the last open(): state and counters to zero, parameters stay."""
        _check(lib().idf_stream_reset(self._h))

    def alloc_out(self, in_rows: int, device="cuda:0") -> torch.Tensor:
        _, w, c = self.out_shape(in_rows)
        r = int(lib().idf_out_rows_needed(self._h, in_rows))
        return torch.zeros((self.n_streams, max(r, 1), w, c), dtype=self.out_torch_dtype, device=device)

    def push(self, segments: torch.Tensor, out: torch.Tensor) -> int:
        """segments: device tensor [n_seg][n_streams][in_w][in_c] in the activation type."""
        assert segments.is_cuda and segments.is_contiguous() and out.is_cuda and out.is_contiguous()
        assert segments.dtype == self.act_torch_dtype and out.dtype == self.out_torch_dtype
        assert tuple(segments.shape[1:]) == (self.n_streams, self.in_w, self.in_c), segments.shape
        em = ctypes.c_int()
        _check(lib().idf_stream_push(self._h, segments.data_ptr(), segments.shape[0], out.data_ptr(), out.shape[1],
                                     ctypes.byref(em)))
        return int(em.value)

    def push_last(self, segments: torch.Tensor, out: torch.Tensor) -> int:
        """The last segments and the end of input in one call; returns the total number of output rows."""
        assert segments.is_cuda and segments.is_contiguous() and out.is_cuda and out.is_contiguous()
        assert segments.dtype == self.act_torch_dtype and out.dtype == self.out_torch_dtype
        assert tuple(segments.shape[1:]) == (self.n_streams, self.in_w, self.in_c), segments.shape
        tot = ctypes.c_longlong()
        _check(lib().idf_stream_push_last(self._h, segments.data_ptr(), segments.shape[0], out.data_ptr(), out.shape[1],
                                          ctypes.byref(tot)))
        return int(tot.value)

    def set_out_base(self, first_row: int):
        """Later output rows are written at index (row - first_row) of the output buffer; see idf_stream_set_out_base."""
        _check(lib().idf_stream_set_out_base(self._h, int(first_row)))

    def finish(self, out: torch.Tensor) -> int:
        tot = ctypes.c_longlong()
        _check(lib().idf_stream_finish(self._h, out.data_ptr(), out.shape[1], ctypes.byref(tot)))
        return int(tot.value)

    def run_host(self, h_segments: torch.Tensor, d_segments: torch.Tensor, h_out: torch.Tensor, d_out: torch.Tensor) -> int:
        """Whole streams from (pinned) host memory and back; see idf_run_host."""
        assert not h_segments.is_cuda and not h_out.is_cuda and d_segments.is_cuda and d_out.is_cuda
        assert h_segments.is_contiguous() and h_out.is_contiguous()
        assert h_segments.dtype == self.act_torch_dtype and h_out.dtype == self.out_torch_dtype
        assert h_out.shape == d_out.shape and h_segments.shape == d_segments.shape
        tot = ctypes.c_longlong()
        _check(lib().idf_run_host(self._h, h_segments.data_ptr(), h_segments.shape[0], d_segments.data_ptr(),
                                  h_out.data_ptr(), d_out.data_ptr(), d_out.shape[1], ctypes.byref(tot)))
        return int(tot.value)

    def save_state(self) -> torch.Tensor:
        """Snapshot of the open streams (host uint8 tensor); see idf_state_save."""
        buf = torch.empty(int(lib().idf_state_snapshot_bytes(self._h)), dtype=torch.uint8)
        _check(lib().idf_state_save(self._h, buf.data_ptr(), buf.numel()))
        return buf

    def restore_state(self, snapshot: torch.Tensor):
        """Replace this handle's streams by the saved ones; see idf_state_restore."""
        assert not snapshot.is_cuda and snapshot.dtype == torch.uint8 and snapshot.is_contiguous()
        _check(lib().idf_state_restore(self._h, snapshot.data_ptr(), snapshot.numel()))

    def close(self):
        if self._h:
            lib().idf_net_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def segments_from_maps(x: np.ndarray, dtype) -> torch.Tensor:
    """Host maps [n_streams][H][W][C] -> host tensor [H][n_streams][W][C] in the activation type."""
    d = DTYPES[dtype] if isinstance(dtype, str) else dtype
    t = torch.from_numpy(np.ascontiguousarray(x))
    t = t.permute(1, 0, 2, 3).contiguous()
    return t.to(_act_torch_dtype(d))


def net_from_workload(w, weights, biases, n_streams: Optional[int] = None, row_block: int = 0) -> Net:
    return Net(w.dtype, w.layers, w.W, w.C, n_streams or w.n_streams, weights, biases, row_block=row_block)


def infer(net: Net, x: np.ndarray, chunks: Optional[Sequence[int]] = None, device="cuda:0", last: bool = False) -> np.ndarray:
    """Run whole maps x [n_streams][H][W][C] through the net; ``chunks`` gives the number of
    segments per push (default: one push).  With ``last`` the final group of segments and the end
    of input go through ``push_last`` instead of ``push`` + ``finish``.  Returns the output map as
    a numpy array."""
    seg = segments_from_maps(x, net.dtype).to(device)
    H = seg.shape[0]
    out = net.alloc_out(H, device)
    net.open(device)
    groups, pos = [], 0
    for n in (chunks or [H]):
        n = min(n, H - pos)
        if n > 0:
            groups.append((pos, pos + n))
        pos += n
    if pos < H:
        groups.append((pos, H))
    rows = None
    for k, (a, b) in enumerate(groups):
        if last and k == len(groups) - 1:
            rows = net.push_last(seg[a:b], out)
        else:
            net.push(seg[a:b], out)
    if rows is None:
        rows = net.finish(out)
    net.status()
    torch.cuda.synchronize()
    assert rows == net.out_shape(H)[0], (rows, net.out_shape(H))
    return out[:, :rows].cpu().numpy()


NOALLOC_SCRATCH_BYTES = 8 << 20


def conv_rows_noalloc(segments: torch.Tensor, weights: torch.Tensor, bias: Optional[torch.Tensor], stride: int, pad: int,
                      relu: bool, out: torch.Tensor) -> int:
    """One fp32 conv layer over whole streams without any device allocation (idf_conv_rows_noalloc).

    For callers that own only their input and output buffers and may not allocate: the ring state
    and the repacked weights live in a fixed array inside the library (8 MiB per GPU, shared by
    all calls, so calls must not overlap on the GPU).  ``segments`` [n_rows][n_streams][in_w][cin],
    ``weights`` [cout][kh][kw][cin], ``out`` [n_streams][capacity][out_w][cout], all fp32 device
    tensors owned by the caller.  Enqueues on the current stream; returns the number of output rows.
    """
    assert segments.is_cuda and weights.is_cuda and out.is_cuda
    assert segments.dtype == weights.dtype == out.dtype == torch.float32
    assert segments.is_contiguous() and weights.is_contiguous() and out.is_contiguous()
    n_rows, S, in_w, cin = segments.shape
    cout, kh, kw, cin2 = weights.shape
    assert cin == cin2 and out.dim() == 4 and out.shape[0] == S and out.shape[3] == cout
    # the C call cannot see the width of `out`: a buffer narrower than the layer's rows would be overrun
    out_w = 1 if in_w == 1 else (in_w + 2 * pad - kw) // stride + 1
    assert out.shape[2] == out_w, f"out has width {out.shape[2]}, the layer emits rows of width {out_w}"
    if bias is not None:
        assert bias.is_cuda and bias.dtype == torch.float32 and bias.is_contiguous() and tuple(bias.shape) == (cout,)
    rows = ctypes.c_longlong()
    st = torch.cuda.current_stream(segments.device).cuda_stream
    _check(lib().idf_conv_rows_noalloc(segments.data_ptr(), n_rows, S, in_w, cin, weights.data_ptr(),
                                       bias.data_ptr() if bias is not None else None, cout, kh, kw, stride, pad,
                                       int(relu), out.data_ptr(), out.shape[1], ctypes.byref(rows), st))
    return int(rows.value)
