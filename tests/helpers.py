"""Shared helpers of the GPU parity tests: build one synthetic matrix on the host and the device."""
from __future__ import annotations

import dataclasses

import numpy as np
import torch

from paper_2609_02652_b200 import datagen

GAIN = datagen.GAIN
TOL_NORMALISED = 1e-4      # max |y - y_ref| / (||W_row||_2 ||x||_2), the stated bar
TOL_PAPER = 1e-5           # |y - y_ref| <= 1e-5 * sum |w x|  (Sec. 2.4)


@dataclasses.dataclass
class Case:
    rows: int
    nb: int
    codes: np.ndarray          # uint64 [rows*nb]
    row_scale: np.ndarray      # float16 [rows]
    x: np.ndarray              # float16 [24 nb]
    d_codes: torch.Tensor | None = None
    d_scale: torch.Tensor | None = None
    d_x: torch.Tensor | None = None


def make_case(rows: int, k: int, seed: int, tensor_id: int = 0, device: str | None = "cuda") -> Case:
    nb = (k + 23) // 24
    codes_t = datagen.make_codes(rows, nb, seed, tensor_id)
    rs = datagen.make_row_scale(rows, seed, tensor_id)
    x = datagen.make_x(k, nb * 24, seed, tensor_id)
    c = Case(rows, nb, codes_t.numpy().astype(np.uint64), rs.numpy(), x.numpy())
    if device is not None:
        c.d_codes, c.d_scale, c.d_x = codes_t.to(device), rs.to(device), x.to(device)
    return c


def check_gemv(oracle, case: Case, y: torch.Tensor, gain=GAIN, nthreads: int = 8):
    """Every row against the f64 oracle, with the normalised metric and the paper's own bound."""
    y_ref, wnorm, abssum = oracle.matvec(case.codes, case.rows, case.nb, case.row_scale, gain, case.x, nthreads=nthreads)
    yv = y.detach().cpu().numpy().astype(np.float64)
    assert np.isfinite(yv).all()
    xnorm = float(np.linalg.norm(case.x.astype(np.float64)))
    denom = wnorm * xnorm
    err = np.abs(yv - y_ref)
    zero = denom == 0
    assert (yv[zero] == 0).all()
    ratio = np.where(zero, 0.0, err / np.where(zero, 1.0, denom))
    assert ratio.max() <= TOL_NORMALISED, f"normalised error {ratio.max():.3e}"
    assert (err <= TOL_PAPER * abssum + 1e-30).all(), f"paper bound: {np.max(err / np.maximum(abssum, 1e-30)):.3e}"
    return float(ratio.max()), float(np.max(err / np.maximum(abssum, 1e-30)))


def window_base(x: np.ndarray) -> np.ndarray:
    """Window base of the 10-byte layout for coordinates x [n, 24] (written out from the layout's rule, in numpy):
    u = 8 + floor(x / 2); the smallest o in 3..6 with o <= min u and max u <= o + 7, or 0 if there is none."""
    u = 8 + np.floor_divide(x.astype(np.int64), 2)
    lo, hi = u.min(1), u.max(1)
    o = np.maximum(3, hi - 7)
    return np.where((o <= np.minimum(6, lo)), o, 0)


def exception_codes(oracle, want: int = 64, seed: int = 77) -> np.ndarray:
    """Code words whose blocks the 10-byte layout cannot hold in its short record: those that occur in the synthetic
    stream (about one block in 8000), plus twice a shortest vector in a few arrangements, (8, -8, 0^22) and the like."""
    stream = datagen.make_codes(4096, 128, seed).numpy().astype(np.uint64).ravel()
    xs, cls = oracle.decode_batch(stream)
    found = stream[(window_base(xs) == 0) & (cls >= 0)][:want]
    made = []
    for i, j in ((0, 1), (5, 17), (22, 23), (3, 12)):
        x = np.zeros(24, np.int8)
        x[i], x[j] = 8, -8
        idx = oracle.encode(x)
        assert idx >= 0
        made += [idx, idx | (1 << 47)]
    return np.concatenate([found, np.array(made, np.uint64)])


def make_overlay_case(oracle, rows: int, k: int, seed: int, rate: float, tensor_id: int = 0, device: str | None = "cuda") -> Case:
    """make_case with a fraction `rate` of the blocks replaced by exception blocks (seeded)."""
    c = make_case(rows, k, seed, tensor_id, device=None)
    pool = exception_codes(oracle)
    rng = np.random.default_rng(seed * 1000 + tensor_id)
    hit = rng.random(c.codes.size) < rate
    c.codes = c.codes.copy()
    c.codes[hit] = pool[rng.integers(0, pool.size, int(hit.sum()))]
    if device is not None:
        c.d_codes = torch.from_numpy(c.codes.view(np.int64)).to(device)
        c.d_scale, c.d_x = torch.from_numpy(c.row_scale).to(device), torch.from_numpy(c.x).to(device)
    return c
