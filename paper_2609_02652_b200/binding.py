"""Thin ctypes binding of libllvq.so (declared in include/llvq.h): argument marshalling only.

Every function has the name of the C entry point without its prefix and takes torch CUDA tensors
where the C call takes device pointers.  Nothing is computed here; if the shared library is
missing or a call fails, an exception is raised - there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from typing import Sequence

import torch

PLANES = 0
ONEHOT = 1
PLANES13 = 2      # the 14-byte layout's codes with a one-byte header: 13 bytes a block
PLANES10X = 3     # three-bit window codes, 10 bytes a block, plus a table of the blocks no window holds
MAX_GROUP = 8
_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libllvq.so")
_lib = None

SYMBOLS = (
    "llvq_create", "llvq_destroy", "llvq_strerror", "llvq_status", "llvq_selftest_wait_limit", "llvq_set_pdl", "llvq_num_classes", "llvq_class_base", "llvq_layout_bytes",
    "llvq_expand", "llvq_gemv", "llvq_gemv_batch", "llvq_gemv_plan", "llvq_gemv_grouped", "llvq_gemv_static", "llvq_gemv_fp16", "llvq_gemv_noweights", "llvq_dequant_fp16",
    "llvq_decode_i8", "llvq_rotate", "llvq_rotate_block", "llvq_gemv_rotated", "llvq_static_status", "llvq_static_selftest_wait_limit",
    "llvq_overlay_count", "llvq_overlay_bytes",
)


class LlvqError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        msg = load().llvq_strerror(code).decode() if _lib is not None else str(code)
        super().__init__(f"{what} failed: {msg} ({code})")


class Problem(ctypes.Structure):
    _fields_ = [("layout", ctypes.c_void_p), ("row_scale", ctypes.c_void_p), ("y", ctypes.c_void_p),
                ("rows", ctypes.c_int64), ("gain", ctypes.c_float * 2)]


class Rotation(ctypes.Structure):
    _fields_ = [("negate_bits", ctypes.c_void_p), ("n", ctypes.c_int64), ("block", ctypes.c_int64)]


def load() -> ctypes.CDLL:
    """Loads libllvq.so from the package directory; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_02652_b200.build` "
                               "(nvcc, sm_100a); there is no CPU fallback")
        L = ctypes.CDLL(LIB_PATH)
        vp, i64, ci, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_size_t
        L.llvq_create.argtypes = [ctypes.POINTER(vp), ci, sz]
        L.llvq_destroy.argtypes = [vp]
        L.llvq_destroy.restype = None
        L.llvq_strerror.argtypes = [ci]
        L.llvq_strerror.restype = ctypes.c_char_p
        L.llvq_num_classes.argtypes = [vp]
        L.llvq_status.argtypes = [vp, vp]
        L.llvq_set_pdl.argtypes = [vp, ci]
        L.llvq_selftest_wait_limit.argtypes = [vp, vp]
        L.llvq_class_base.argtypes = [vp, ci]
        L.llvq_class_base.restype = ctypes.c_uint64
        L.llvq_layout_bytes.argtypes = [ci, i64, i64, ctypes.POINTER(sz)]
        L.llvq_expand.argtypes = [vp, ci, vp, i64, i64, vp, sz, vp, vp]
        L.llvq_gemv.argtypes = [vp, ci, vp, vp, ctypes.POINTER(ctypes.c_float), vp, vp, i64, i64, vp]
        L.llvq_gemv_plan.argtypes = [ci, ctypes.POINTER(ctypes.c_int64), ci, i64, ci, ctypes.POINTER(ctypes.c_int32), ci]
        L.llvq_gemv_batch.argtypes = [vp, vp, vp, ctypes.POINTER(ctypes.c_float), vp, vp, i64, i64, ci, vp]
        L.llvq_gemv_grouped.argtypes = [vp, ci, ctypes.POINTER(Problem), ci, vp, i64, vp]
        L.llvq_gemv_static.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_float), vp, vp, i64, i64, vp]
        L.llvq_gemv_fp16.argtypes = [vp, vp, vp, i64, i64, vp]
        L.llvq_gemv_noweights.argtypes = [vp, vp, vp, vp, i64, i64, vp]
        L.llvq_dequant_fp16.argtypes = [vp, ci, vp, vp, ctypes.POINTER(ctypes.c_float), vp, i64, i64, vp]
        L.llvq_decode_i8.argtypes = [vp, ci, vp, vp, vp, i64, i64, vp]
        L.llvq_rotate.argtypes = [vp, vp, vp, vp, i64, i64, vp]
        L.llvq_gemv_rotated.argtypes = [vp, ctypes.POINTER(Problem), ci, vp, i64, ctypes.POINTER(Rotation), vp]
        L.llvq_static_status.argtypes = [vp]
        L.llvq_static_selftest_wait_limit.argtypes = [vp]
        L.llvq_overlay_count.argtypes = [vp, vp, i64, i64, ctypes.POINTER(ctypes.c_uint64), vp]
        L.llvq_overlay_bytes.argtypes = [i64, i64, ctypes.c_uint64, ctypes.POINTER(sz)]
        L.llvq_rotate_block.argtypes = [i64, i64]
        L.llvq_rotate_block.restype = i64
        for name in SYMBOLS:
            if name not in ("llvq_destroy", "llvq_strerror", "llvq_class_base", "llvq_rotate_block"):
                getattr(L, name).restype = ci
        _lib = L
    return _lib


def _check(code: int, what: str) -> None:
    if code != 0:
        raise LlvqError(code, what)


def _dev(t: torch.Tensor, dtype, what: str) -> int:
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise TypeError(f"{what}: expected a contiguous CUDA tensor of dtype {dtype}")
    return t.data_ptr()


def _stream(stream) -> int:
    return (stream if stream is not None else torch.cuda.current_stream()).cuda_stream


def _gain(gain: Sequence[float]):
    return (ctypes.c_float * 2)(float(gain[0]), float(gain[1]))


class Context:
    """Owns a llvq_ctx: the device tables and the reduction scratch of one stream's launches."""

    def __init__(self, device: int = 0, scratch_bytes: int = 0):
        self._p = ctypes.c_void_p()
        _check(load().llvq_create(ctypes.byref(self._p), int(device), int(scratch_bytes)), "llvq_create")
        self.device = int(device)

    @property
    def ptr(self) -> ctypes.c_void_p:
        if not self._p:
            raise RuntimeError("context already destroyed")
        return self._p

    def close(self) -> None:
        if self._p:
            load().llvq_destroy(self._p)
            self._p = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def create(device: int = 0, scratch_bytes: int = 0) -> Context:
    return Context(device, scratch_bytes)


def destroy(ctx: Context) -> None:
    ctx.close()


def status(ctx: Context, stream=None) -> None:
    """Synchronises the stream; raises LlvqError(-5) if a kernel on this context gave up on a bounded wait, else
    LlvqError(-3) if a PLANES10X expansion had more exceptions than its buffer had room for, else LlvqError(-6) if an
    expansion since the last call met a code word that names no point."""
    _check(load().llvq_status(ctx.ptr, _stream(stream)), "llvq_status")


def selftest_wait_limit(ctx: Context, stream=None) -> None:
    """Enqueues the bounded-wait self-test; the next status() raises LlvqError(-5)."""
    _check(load().llvq_selftest_wait_limit(ctx.ptr, _stream(stream)), "llvq_selftest_wait_limit")


def set_pdl(ctx: Context, enabled: bool) -> None:
    _check(load().llvq_set_pdl(ctx.ptr, int(bool(enabled))), "llvq_set_pdl")


def num_classes(ctx: Context) -> int:
    return load().llvq_num_classes(ctx.ptr)


def class_base(ctx: Context, c: int) -> int:
    return int(load().llvq_class_base(ctx.ptr, int(c)))


def layout_bytes(layout: int, rows: int, k_padded: int) -> int:
    n = ctypes.c_size_t()
    _check(load().llvq_layout_bytes(int(layout), int(rows), int(k_padded), ctypes.byref(n)), "llvq_layout_bytes")
    return int(n.value)


def overlay_bytes(rows: int, k_padded: int, exceptions: int) -> int:
    """Bytes of a PLANES10X buffer with room for `exceptions` entries in its exception table."""
    n = ctypes.c_size_t()
    _check(load().llvq_overlay_bytes(int(rows), int(k_padded), int(exceptions), ctypes.byref(n)), "llvq_overlay_bytes")
    return int(n.value)


def overlay_count(ctx: Context, codes: torch.Tensor, rows: int, nb: int, stream=None) -> int:
    """Blocks of the matrix that PLANES10X keeps in its exception table (synchronises the stream)."""
    n = ctypes.c_uint64()
    _check(load().llvq_overlay_count(ctx.ptr, _dev(codes, torch.int64, "codes"), int(rows), int(nb), ctypes.byref(n), _stream(stream)),
           "llvq_overlay_count")
    return int(n.value)


def expand(ctx: Context, layout: int, codes: torch.Tensor, rows: int, nb: int, out: torch.Tensor | None = None,
           bad_count: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """codes: int64 CUDA tensor of rows*nb code words -> uint8 layout buffer (PLANES10X: sized by llvq_layout_bytes,
    i.e. with room for one exception in 32 blocks, unless `out` is given)."""
    if out is None:
        out = torch.empty(layout_bytes(layout, rows, nb * 24), dtype=torch.uint8, device=codes.device)
    bc = _dev(bad_count, torch.int32, "bad_count") if bad_count is not None else None
    _check(load().llvq_expand(ctx.ptr, int(layout), _dev(codes, torch.int64, "codes"), int(rows), int(nb),
                              _dev(out, torch.uint8, "out"), out.numel(), bc, _stream(stream)), "llvq_expand")
    return out


def gemv(ctx: Context, layout: int, layout_buf: torch.Tensor, row_scale: torch.Tensor, gain, x: torch.Tensor,
         rows: int, k_padded: int, y: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    if y is None:
        y = torch.empty(rows, dtype=torch.float32, device=x.device)
    _check(load().llvq_gemv(ctx.ptr, int(layout), _dev(layout_buf, torch.uint8, "layout_buf"),
                            _dev(row_scale, torch.float16, "row_scale"), _gain(gain), _dev(x, torch.float16, "x"),
                            _dev(y, torch.float32, "y"), int(rows), int(k_padded), _stream(stream)), "llvq_gemv")
    return y


def gemv_batch(ctx: Context, layout_buf: torch.Tensor, row_scale: torch.Tensor, gain, x: torch.Tensor, rows: int,
               k_padded: int, y: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """llvq_gemv_batch: x is fp16 [batch, k_padded] (contiguous), the result f32 [batch, rows]."""
    batch = int(x.shape[0])
    if x.dim() != 2 or int(x.shape[1]) != int(k_padded) or not x.is_contiguous():
        raise ValueError("x must be a contiguous [batch, k_padded] tensor")
    if y is None:
        y = torch.empty((batch, rows), dtype=torch.float32, device=x.device)
    _check(load().llvq_gemv_batch(ctx.ptr, _dev(layout_buf, torch.uint8, "layout_buf"), _dev(row_scale, torch.float16, "row_scale"),
                                  _gain(gain), _dev(x, torch.float16, "x"), _dev(y, torch.float32, "y"), int(rows), int(k_padded),
                                  batch, _stream(stream)), "llvq_gemv_batch")
    return y


def gemv_plan(sm_count: int, rows, k_padded: int, batch: int = 1) -> dict:
    """llvq_gemv_plan: the launch plan for matrices of `rows` rows each (a host query, no GPU needed)."""
    rows = list(rows)
    arr = (ctypes.c_int64 * len(rows))(*rows)
    out = (ctypes.c_int32 * (8 + 256 + 1))()
    _check(load().llvq_gemv_plan(int(sm_count), arr, len(rows), int(k_padded), int(batch), out, len(out)), "llvq_gemv_plan")
    grid = out[0]
    return dict(grid=grid, smem=out[1], units=out[2], total_units=out[3], panel=out[4], npanels=out[5], xblocks=out[6],
                groups=out[7], cta_first=[out[8 + c] for c in range(grid + 1)])


def gemv_static(layout_buf: torch.Tensor, row_scale: torch.Tensor, gain, x: torch.Tensor, rows: int, k_padded: int,
                y: torch.Tensor, stream=None) -> torch.Tensor:
    """llvq_gemv_static: no context and no allocation inside the library; the caller supplies y.  Runs on the
    current CUDA device; at most 65536 rows; calls must not overlap on the GPU (they share built-in scratch)."""
    _check(load().llvq_gemv_static(_dev(layout_buf, torch.uint8, "layout_buf"), _dev(row_scale, torch.float16, "row_scale"),
                                   _gain(gain), _dev(x, torch.float16, "x"), _dev(y, torch.float32, "y"), int(rows),
                                   int(k_padded), _stream(stream)), "llvq_gemv_static")
    return y


def static_status(stream=None) -> None:
    """llvq_static_status: synchronises the stream; raises LlvqError(-5) if a llvq_gemv_static launch on the current
    device gave up on a bounded wait (the built-in flag and scratch are then cleared)."""
    _check(load().llvq_static_status(_stream(stream)), "llvq_static_status")


def static_selftest_wait_limit(stream=None) -> None:
    """Enqueues the bounded-wait self-test against the static entry point's flag; the next static_status() raises."""
    _check(load().llvq_static_selftest_wait_limit(_stream(stream)), "llvq_static_selftest_wait_limit")


def make_problems(problems) -> ctypes.Array:
    """problems: sequence of (layout_buf, row_scale, gain, y, rows) -> host array of llvq_problem."""
    arr = (Problem * len(problems))()
    for i, (buf, rs, gain, y, rows) in enumerate(problems):
        arr[i].layout = _dev(buf, torch.uint8, "layout_buf")
        arr[i].row_scale = _dev(rs, torch.float16, "row_scale")
        arr[i].y = _dev(y, torch.float32, "y")
        arr[i].rows = int(rows)
        arr[i].gain[0], arr[i].gain[1] = float(gain[0]), float(gain[1])
    return arr


def gemv_grouped(ctx: Context, layout: int, problems, x: torch.Tensor, k_padded: int, stream=None) -> None:
    """problems: a host array from make_problems, or the sequence make_problems takes."""
    arr = problems if isinstance(problems, ctypes.Array) else make_problems(problems)
    _check(load().llvq_gemv_grouped(ctx.ptr, int(layout), arr, len(arr), _dev(x, torch.float16, "x"), int(k_padded),
                                    _stream(stream)), "llvq_gemv_grouped")


def gemv_rotated(ctx: Context, problems, x: torch.Tensor, k_padded: int, n: int, block: int = 0,
                 negate_bits: torch.Tensor | None = None, stream=None) -> None:
    """llvq_gemv_rotated: the grouped 14-byte-layout GEMV on rotate(x[:n]) (the rest of x passes through), one launch."""
    arr = problems if isinstance(problems, ctypes.Array) else make_problems(problems)
    rot = Rotation(None if negate_bits is None else _dev(negate_bits, torch.int32, "negate_bits"), int(n), int(block))
    _check(load().llvq_gemv_rotated(ctx.ptr, arr, len(arr), _dev(x, torch.float16, "x"), int(k_padded), ctypes.byref(rot),
                                    _stream(stream)), "llvq_gemv_rotated")


def gemv_fp16(W: torch.Tensor, x: torch.Tensor, rows: int, k: int, y: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    if y is None:
        y = torch.empty(rows, dtype=torch.float32, device=x.device)
    _check(load().llvq_gemv_fp16(_dev(W, torch.float16, "W"), _dev(x, torch.float16, "x"), _dev(y, torch.float32, "y"),
                                 int(rows), int(k), _stream(stream)), "llvq_gemv_fp16")
    return y


def rotate_block(n: int, block: int = 0) -> int:
    """Block length `rotate` uses for a vector of n entries (0 if it would refuse them).  Host query."""
    return int(load().llvq_rotate_block(int(n), int(block)))


def rotate(ctx: Context, x: torch.Tensor, block: int = 0, negate_bits: torch.Tensor | None = None,
           y: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """llvq_rotate: block-diagonal Walsh-Hadamard rotation of the fp16 vector x; `negate_bits` int32 words, bit i = flip x_i."""
    if y is None:
        y = torch.empty_like(x)
    _check(load().llvq_rotate(ctx.ptr, _dev(x, torch.float16, "x"), _dev(y, torch.float16, "y"),
                              None if negate_bits is None else _dev(negate_bits, torch.int32, "negate_bits"),
                              int(x.numel()), int(block), _stream(stream)), "llvq_rotate")
    return y


def gemv_noweights(ctx: Context, row_scale: torch.Tensor, x: torch.Tensor, rows: int, k_padded: int,
                   y: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    if y is None:
        y = torch.empty(rows, dtype=torch.float32, device=x.device)
    _check(load().llvq_gemv_noweights(ctx.ptr, _dev(row_scale, torch.float16, "row_scale"), _dev(x, torch.float16, "x"),
                                      _dev(y, torch.float32, "y"), int(rows), int(k_padded), _stream(stream)),
           "llvq_gemv_noweights")
    return y


def dequant_fp16(ctx: Context, layout: int, layout_buf: torch.Tensor, row_scale: torch.Tensor, gain, rows: int,
                 k_padded: int, W: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    if W is None:
        W = torch.empty((rows, k_padded), dtype=torch.float16, device=layout_buf.device)
    _check(load().llvq_dequant_fp16(ctx.ptr, int(layout), _dev(layout_buf, torch.uint8, "layout_buf"),
                                    _dev(row_scale, torch.float16, "row_scale"), _gain(gain), _dev(W, torch.float16, "W"),
                                    int(rows), int(k_padded), _stream(stream)), "llvq_dequant_fp16")
    return W


def decode_i8(ctx: Context, layout: int, layout_buf: torch.Tensor, rows: int, nb: int, stream=None):
    coords = torch.empty((rows, nb, 24), dtype=torch.int8, device=layout_buf.device)
    cls = torch.empty((rows, nb), dtype=torch.int16, device=layout_buf.device)
    _check(load().llvq_decode_i8(ctx.ptr, int(layout), _dev(layout_buf, torch.uint8, "layout_buf"),
                                 _dev(coords, torch.int8, "coords"), _dev(cls, torch.int16, "class_ids"), int(rows), int(nb),
                                 _stream(stream)), "llvq_decode_i8")
    return coords, cls
