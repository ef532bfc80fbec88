"""ctypes front end of the CPU oracle (oracle/llvq_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the benchmark's
CPU-baseline leg; never by the product package.  It compiles the C file with gcc on first use
(the shared object is a build artefact, not a source of truth) and exposes numpy-level calls.
Every function below names the paper passage its C counterpart follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "llvq_oracle.c")
_LIB = os.path.join(_HERE, "libllvq_oracle.so")
_lock = threading.Lock()
_lib = None

N_POINTS = 111_043_117_458_000  # Sec. 2.1: points of the ball, printed by the paper
SENTINEL_CLASS = 511


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or older than its source."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-shared", "-fPIC", "-pthread", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    with _lock:
        if _lib is None:
            L = ctypes.CDLL(build())
            u64, i64, vp, ci = ctypes.c_uint64, ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
            L.llvqo_init.restype = ci
            L.llvqo_init_shells.argtypes = [ci]
            L.llvqo_init_shells.restype = ci
            L.llvqo_num_classes.restype = ci
            L.llvqo_total_points.restype = u64
            L.llvqo_shell_count.argtypes = [ci]
            L.llvqo_shell_count.restype = u64
            L.llvqo_class_info.argtypes = [ci, vp, vp, vp, vp]
            L.llvqo_class_info.restype = ci
            L.llvqo_golay_word.argtypes = [ci]
            L.llvqo_golay_word.restype = ctypes.c_uint32
            L.llvqo_golay_sorted.argtypes = [ci]
            L.llvqo_golay_sorted.restype = ctypes.c_uint32
            L.llvqo_decode.argtypes = [u64, vp]
            L.llvqo_decode.restype = ci
            L.llvqo_encode.argtypes = [vp]
            L.llvqo_encode.restype = i64
            L.llvqo_record.argtypes = [u64, vp, vp]
            L.llvqo_record.restype = ci
            L.llvqo_planes_bytes.argtypes = [i64, i64]
            L.llvqo_planes_bytes.restype = ctypes.c_size_t
            L.llvqo_onehot_bytes.argtypes = [i64, i64]
            L.llvqo_onehot_bytes.restype = ctypes.c_size_t
            L.llvqo_pack_planes.argtypes = [vp, i64, i64, vp]
            L.llvqo_pack_planes.restype = None
            L.llvqo_pack_onehot.argtypes = [vp, i64, i64, vp]
            L.llvqo_pack_planes13.argtypes = [vp, i64, i64, vp]
            L.llvqo_pack_planes13.restype = None
            L.llvqo_planes13_bytes.argtypes = [i64, i64]
            L.llvqo_planes13_bytes.restype = ctypes.c_size_t
            L.llvqo_pack_onehot.restype = None
            L.llvqo_planes10x_bytes.argtypes = [i64, i64, u64]
            L.llvqo_planes10x_bytes.restype = ctypes.c_size_t
            L.llvqo_pack_planes10x.argtypes = [vp, i64, i64, vp, u64]
            L.llvqo_pack_planes10x.restype = i64
            L.llvqo_dequant.argtypes = [vp, i64, i64, vp, vp, vp]
            L.llvqo_dequant.restype = None
            L.llvqo_matvec.argtypes = [vp, i64, i64, vp, vp, vp, vp, vp, vp, ci]
            L.llvqo_matvec.restype = None
            L.llvqo_decode_batch.argtypes = [vp, i64, vp, vp]
            L.llvqo_rotate.argtypes = [vp, i64, i64, vp, vp]
            L.llvqo_rotate.restype = i64
            L.llvqo_rotate_block.argtypes = [i64, i64]
            L.llvqo_rotate_block.restype = i64
            L.llvqo_double_to_half.argtypes = [ctypes.c_double]
            L.llvqo_double_to_half.restype = ctypes.c_uint16
            L.llvqo_decode_batch.restype = None
            L.llvqo_init()
            _lib = L
    return _lib


def _ptr(a: np.ndarray) -> int:
    return a.ctypes.data


def init_shells(max_shell: int) -> int:
    """Rebuild the class list for shells 2..max_shell (Sec. 2.1; 12 is the served ball)."""
    return lib().llvqo_init_shells(int(max_shell))


def num_classes() -> int:
    return lib().llvqo_num_classes()


def total_points() -> int:
    return int(lib().llvqo_total_points())


def shell_count(m: int) -> int:
    return int(lib().llvqo_shell_count(int(m)))


def class_info(c: int) -> dict:
    """Shell, type, Golay weight, sorted magnitudes, size and first index of class c (Sec. 2.1)."""
    out = np.zeros(6, np.int32)
    mags = np.zeros(24, np.int32)
    size = np.zeros(1, np.uint64)
    base = np.zeros(1, np.uint64)
    if lib().llvqo_class_info(int(c), _ptr(out), _ptr(mags), _ptr(size), _ptr(base)) != 0:
        raise IndexError(c)
    return dict(shell=int(out[0]), odd=int(out[1]), w=int(out[2]), ndist=int(out[3]), nzB=int(out[4]),
                mags=mags.tolist(), size=int(size[0]), base=int(base[0]))


def golay_words() -> np.ndarray:
    """The 4096 codewords in message order (word k = XOR of the generator rows named by k's bits)."""
    L = lib()
    return np.array([L.llvqo_golay_word(k) for k in range(4096)], dtype=np.uint32)


def decode(idx: int) -> tuple[int, np.ndarray]:
    """Index -> (class id, 24 integer coordinates); class id -1 if idx names no point (Sec. 2.1)."""
    x = np.zeros(24, np.int8)
    c = lib().llvqo_decode(int(idx), _ptr(x))
    return c, x


def encode(x) -> int:
    """Point -> index, -1 when x is not a lattice point of the ball (inverse of decode)."""
    a = np.ascontiguousarray(x, dtype=np.int8)
    return int(lib().llvqo_encode(_ptr(a)))


def decode_batch(codes: np.ndarray) -> tuple[np.ndarray, np.ndarray]:
    """48-bit codes (index | gain << 47) -> coordinates [n, 24] int8 and class ids [n] (-1 = invalid)."""
    codes = np.ascontiguousarray(codes, dtype=np.uint64).ravel()
    x = np.zeros((codes.size, 24), np.int8)
    cls = np.zeros(codes.size, np.int32)
    lib().llvqo_decode_batch(_ptr(codes), codes.size, _ptr(x), _ptr(cls))
    return x, cls


def record(code: int) -> dict:
    """The decoded-field record of one block (Sec. 2.2): class, gain, sign mask, planes, one-hot masks."""
    f = np.zeros(10, np.uint32)
    x = np.zeros(24, np.int8)
    lib().llvqo_record(int(code), _ptr(f), _ptr(x))
    return dict(cls=int(f[0]), gain=int(f[1]), smask=int(f[2]), planes=[int(v) for v in f[3:6]],
                onehot=[int(v) for v in f[6:10]], x=x)


def planes_bytes(rows: int, nb: int) -> int:
    return int(lib().llvqo_planes_bytes(rows, nb))


def onehot_bytes(rows: int, nb: int) -> int:
    return int(lib().llvqo_onehot_bytes(rows, nb))


def pack_planes(codes: np.ndarray, rows: int, nb: int) -> np.ndarray:
    """Expected bytes of the 14-byte layout (LLVQ_PLANES) for a rows x nb matrix of codes."""
    codes = np.ascontiguousarray(codes, dtype=np.uint64).ravel()
    assert codes.size == rows * nb
    out = np.zeros(planes_bytes(rows, nb), np.uint8)
    lib().llvqo_pack_planes(_ptr(codes), rows, nb, _ptr(out))
    return out


def planes13_bytes(rows: int, nb: int) -> int:
    return int(lib().llvqo_planes13_bytes(rows, nb))


def pack_planes13(codes: np.ndarray, rows: int, nb: int) -> np.ndarray:
    """Expected bytes of the 13-byte layout: the 14-byte layout's codes with a one-byte header (shell, parity, gain)."""
    codes = np.ascontiguousarray(codes, dtype=np.uint64).ravel()
    assert codes.size == rows * nb
    out = np.zeros(planes13_bytes(rows, nb), np.uint8)
    lib().llvqo_pack_planes13(_ptr(codes), rows, nb, _ptr(out))
    return out


def planes10x_bytes(rows: int, nb: int, exceptions: int) -> int:
    return int(lib().llvqo_planes10x_bytes(rows, nb, exceptions))


def pack_planes10x(codes: np.ndarray, rows: int, nb: int, capacity: int | None = None) -> tuple[np.ndarray, int]:
    """The 10-byte layout with its exception table (Sec. 3.3, the sparse overlay): the buffer with room for
    `capacity` table entries (default: exactly as many as the matrix has) and the number of exceptions met."""
    codes = np.ascontiguousarray(codes, dtype=np.uint64)
    assert codes.size == rows * nb
    if capacity is None:
        scratch = np.zeros(planes10x_bytes(rows, nb, 0), np.uint8)
        capacity = int(lib().llvqo_pack_planes10x(_ptr(codes), rows, nb, _ptr(scratch), 0))
    out = np.zeros(planes10x_bytes(rows, nb, capacity), np.uint8)
    n = int(lib().llvqo_pack_planes10x(_ptr(codes), rows, nb, _ptr(out), capacity))
    return out, n


def pack_onehot(codes: np.ndarray, rows: int, nb: int) -> np.ndarray:
    """Expected bytes of the one-hot layout (20 B a block)."""
    codes = np.ascontiguousarray(codes, dtype=np.uint64).ravel()
    assert codes.size == rows * nb
    out = np.zeros(onehot_bytes(rows, nb), np.uint8)
    lib().llvqo_pack_onehot(_ptr(codes), rows, nb, _ptr(out))
    return out


def dequant(codes, rows, nb, row_scale_f16, gain) -> np.ndarray:
    """Dequantised weights W[rows, 24 nb] in f64: r_row * gain[g] * x_i / (4 sqrt(m)) (Sec. 2.3)."""
    codes = np.ascontiguousarray(codes, dtype=np.uint64).ravel()
    rs = np.ascontiguousarray(row_scale_f16, dtype=np.float16).view(np.uint16)
    g = np.ascontiguousarray(gain, dtype=np.float64)
    W = np.zeros((rows, nb * 24), np.float64)
    lib().llvqo_dequant(_ptr(codes), rows, nb, _ptr(rs), _ptr(g), _ptr(W))
    return W


def matvec(codes, rows, nb, row_scale_f16, gain, x_f16, nthreads: int = 1):
    """y = W x in f64 (Sec. 2.3), plus per-row ||W_row||_2 and sum |w x| for the two error metrics."""
    codes = np.ascontiguousarray(codes, dtype=np.uint64).ravel()
    assert codes.size == rows * nb
    rs = np.ascontiguousarray(row_scale_f16, dtype=np.float16).view(np.uint16)
    xv = np.ascontiguousarray(x_f16, dtype=np.float16).view(np.uint16)
    assert rs.size == rows and xv.size == nb * 24
    g = np.ascontiguousarray(gain, dtype=np.float64)
    y = np.zeros(rows, np.float64)
    wn = np.zeros(rows, np.float64)
    ab = np.zeros(rows, np.float64)
    lib().llvqo_matvec(_ptr(codes), rows, nb, _ptr(rs), _ptr(g), _ptr(xv), _ptr(y), _ptr(wn), _ptr(ab), int(nthreads))
    return y, wn, ab


def rotate_block(n: int, block: int = 0) -> int:
    """Block length of the rotation of an n-vector: `block`, or the largest power of two (<= 16384) dividing n."""
    return int(lib().llvqo_rotate_block(int(n), int(block)))


def double_to_half_bits(v: float) -> int:
    """FP16 bit pattern of a double rounded to nearest even (the rounding step of `rotate`)."""
    return int(lib().llvqo_double_to_half(float(v)))


def rotate(x_f16, block: int = 0, negate=None) -> np.ndarray:
    """Block-diagonal normalised Walsh-Hadamard rotation of an FP16 vector, by the definition (Sec. 2.3, Sec. 5).

    y[B c + k] = sum_i (-1)^popcount(i & k) s_i x[B c + i] / sqrt(B), summed exactly and rounded once to FP16.
    """
    xv = np.ascontiguousarray(x_f16, dtype=np.float16).ravel().view(np.uint16)
    out = np.zeros(xv.size, np.uint16)
    ng = None if negate is None else np.ascontiguousarray(np.asarray(negate) != 0, dtype=np.uint8)
    assert ng is None or ng.size == xv.size
    B = lib().llvqo_rotate(_ptr(xv), xv.size, int(block), None if ng is None else _ptr(ng), _ptr(out))
    if B == 0:
        raise ValueError("block must be a power of two (<= 16384) that divides the length")
    return out.view(np.float16)
