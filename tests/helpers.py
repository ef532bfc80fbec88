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
