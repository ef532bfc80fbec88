"""Parity of llvq_rotate (the activation rotation ahead of a projection) against the CPU oracle: bit for bit."""
import dataclasses

import numpy as np
import pytest
import torch

from helpers import GAIN, check_gemv, make_case

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2609_02652_b200 import binding

    binding.load()
    return binding


@pytest.fixture(scope="module")
def ctx(B):
    c = B.create(0)
    yield c
    c.close()


def _x(n, seed, kind="normal"):
    rng = np.random.default_rng(seed)
    if kind == "normal":
        v = rng.normal(size=n)
    elif kind == "wide":                      # magnitudes over the whole fp16 range, subnormals included
        v = rng.normal(size=n) * np.exp2(rng.integers(-26, 12, size=n))
    elif kind == "large":                     # sums that overflow fp16 in places
        v = rng.normal(size=n) * 2.0e4
    elif kind == "sparse":
        v = rng.normal(size=n) * (rng.random(n) < 0.03)
    else:
        raise ValueError(kind)
    return np.clip(v, -65504, 65504).astype(np.float16)


def _bits(neg):
    packed = np.packbits(neg.astype(np.uint8), bitorder="little")
    packed = np.concatenate([packed, np.zeros((-packed.size) % 4, np.uint8)])
    return torch.from_numpy(packed.view(np.int32).copy()).cuda()


def _same(got: torch.Tensor, want: np.ndarray):
    g = got.cpu().numpy().view(np.uint16)
    w = want.view(np.uint16)
    # +0 and -0 are the same value: the oracle and the kernel both produce +0 for an exact zero sum, but do not insist
    both_zero = ((g & 0x7fff) == 0) & ((w & 0x7fff) == 0)
    assert np.array_equal(np.where(both_zero, 0, g), np.where(both_zero, 0, w)), \
        f"{np.count_nonzero(np.where(both_zero, 0, g) != np.where(both_zero, 0, w))} of {g.size} differ"


# the activation lengths of the paper's models (hidden and intermediate sizes), a power of two, short and odd cases
LENGTHS = [8, 24, 40, 2560, 4096, 5120, 9728, 12288, 17408, 25600, 24 * 107, 24 * 171, 4104, 8200]


@pytest.mark.parametrize("n", LENGTHS)
def test_rotate_bit_exact_default_block(B, ctx, oracle, n):
    x = _x(n, n)
    y = B.rotate(ctx, torch.from_numpy(x).cuda())
    assert B.rotate_block(n) == oracle.rotate_block(n)
    _same(y, oracle.rotate(x))


@pytest.mark.parametrize("kind", ["wide", "large", "sparse"])
@pytest.mark.parametrize("n,block", [(4096, 0), (9728, 0), (2560, 64), (4096, 1), (4096, 2), (4096, 4), (4096, 8), (4096, 16),
                                     (12288, 1024), (8192, 8192)])
def test_rotate_bit_exact_value_ranges_blocks_and_signs(B, ctx, oracle, kind, n, block):
    x = _x(n, 3 * n + block, kind)
    neg = np.random.default_rng(n + block).integers(0, 2, size=n)
    y = B.rotate(ctx, torch.from_numpy(x).cuda(), block=block, negate_bits=_bits(neg))
    _same(y, oracle.rotate(x, block, neg))


def test_rotate_largest_block_in_place_and_several_ctas(B, ctx, oracle):
    n = 16384 * 2 + 0
    x = _x(n, 77)
    d = torch.from_numpy(x).cuda()
    assert B.rotate_block(n) == 16384
    out = B.rotate(ctx, d, y=d)                                  # in place
    assert out.data_ptr() == d.data_ptr()
    _same(d, oracle.rotate(x))
    # a vector longer than one CTA's piece whose last piece is short: 4096 + 4096 + 1536 coordinates of 512-blocks
    x = _x(9728, 78)
    _same(B.rotate(ctx, torch.from_numpy(x).cuda()), oracle.rotate(x))


def test_rotate_twice_returns_x_up_to_rounding(B, ctx):
    x = torch.from_numpy(_x(12288, 5)).cuda()
    back = B.rotate(ctx, B.rotate(ctx, x))
    assert (back.double() - x.double()).abs().max().item() <= 2.0 ** -8


def test_rotate_then_gemv_matches_oracle_chain(B, ctx, oracle):
    """The served order: rotate x, then the lattice GEMV on the rotated vector, back to back on one stream."""
    for rows, k in ((256, 2560), (96, 4096), (64, 24 * 107)):
        case = make_case(rows, k, seed=rows + k)
        buf = B.expand(ctx, 0, case.d_codes, case.rows, case.nb)
        neg = np.random.default_rng(k).integers(0, 2, size=case.nb * 24)
        xr = B.rotate(ctx, case.d_x, negate_bits=_bits(neg))
        y = B.gemv(ctx, 0, buf, case.d_scale, GAIN, xr, case.rows, case.nb * 24)
        torch.cuda.synchronize()
        want_x = oracle.rotate(case.x, 0, neg)
        _same(xr, want_x)
        check_gemv(oracle, dataclasses.replace(case, x=want_x), y)


def test_rotate_without_programmatic_dependent_launch(B, oracle):
    c = B.create(0)
    try:
        B.set_pdl(c, False)
        x = _x(9728, 9)
        _same(B.rotate(c, torch.from_numpy(x).cuda()), oracle.rotate(x))
    finally:
        c.close()


def test_rotate_error_codes(B, ctx):
    x = torch.zeros(4096, dtype=torch.float16, device="cuda")
    for kwargs, code in (({"block": 3}, -1), ({"block": 32768}, -1), ({"block": 8192}, -1)):
        with pytest.raises(B.LlvqError) as e:
            B.rotate(ctx, x[:4096] if kwargs["block"] != 8192 else x[:4096 - 8], **kwargs)
        assert e.value.code == code
    with pytest.raises(B.LlvqError) as e:
        B.rotate(ctx, x[:12])                                    # not a multiple of 8
    assert e.value.code == -1
    with pytest.raises(B.LlvqError) as e:
        B.rotate(ctx, x[4:4 + 64])                               # 8-byte aligned only
    assert e.value.code == -2
    assert B.rotate_block(4096, 3) == 0 and B.rotate_block(0) == 0
    y = B.rotate(ctx, x)
    assert not y.any()
