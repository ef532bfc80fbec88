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


# ---------------------------------------------------------------- the rotation inside the GEMV's launch
def _rotated_reference(oracle, case, k, block, neg):
    xr = np.concatenate([oracle.rotate(case.x[:k], block, neg), case.x[k:]])
    return dataclasses.replace(case, x=xr)


@pytest.mark.parametrize("rows,k,block,signs", [
    (256, 2560, 0, False), (96, 4096, 0, True), (64, 9728, 0, True), (40, 17408, 0, False), (72, 5120, 0, True),
    (33, 2560, 8, True), (64, 2560, 64, False), (48, 12288, 1024, True), (32, 16384, 0, False), (8, 32768, 8192, True),
    (1, 24, 0, False), (300, 96, 32, True), (4096, 2560, 0, True)])
def test_gemv_rotated_matches_oracle_chain_and_the_two_launch_form(B, ctx, oracle, rows, k, block, signs):
    case = make_case(rows, k, seed=3 * rows + k)
    kp = case.nb * 24
    if k == 24:
        k = 24                                                   # 24 = 8 * 3: blocks of eight
    neg = np.random.default_rng(k + rows).integers(0, 2, size=k) if signs else None
    bits = None if neg is None else _bits(neg)
    buf = B.expand(ctx, 0, case.d_codes, case.rows, case.nb)
    y = torch.full((rows,), float("nan"), dtype=torch.float32, device="cuda")
    B.gemv_rotated(ctx, [(buf, case.d_scale, GAIN, y, rows)], case.d_x, kp, n=k, block=block, negate_bits=bits)
    torch.cuda.synchronize()
    ref = _rotated_reference(oracle, case, k, block, neg)
    err, _ = check_gemv(oracle, ref, y)
    assert err <= 1e-6
    # the same through llvq_rotate and llvq_gemv: the two differ only by the fixed-point quantum of the GEMV
    xr = case.d_x.clone()
    B.rotate(ctx, case.d_x[:k], block=block, negate_bits=bits, y=xr[:k])
    _same(xr, ref.x)
    y2 = B.gemv(ctx, 0, buf, case.d_scale, GAIN, xr, rows, kp)
    torch.cuda.synchronize()
    _, wnorm, _ = oracle.matvec(case.codes, rows, case.nb, case.row_scale, GAIN, ref.x, nthreads=8)
    bound = 1e-6 * wnorm * float(np.linalg.norm(ref.x.astype(np.float64))) + 1e-30
    assert (np.abs(y.cpu().numpy().astype(np.float64) - y2.cpu().numpy().astype(np.float64)) <= bound).all()
    assert torch.equal(case.d_x.cpu(), torch.from_numpy(case.x))      # x itself is left alone


def test_gemv_rotated_grouped_launch_and_outlier_activation(B, ctx, oracle):
    """q/k/v-like group sharing one x; x with one huge entry (what the rotation is for): the bound on the
    rotated magnitudes is then loosest, and the result must still meet the bar with room."""
    k = 2560
    cases = [make_case(r, k, seed=50 + i, tensor_id=i) for i, r in enumerate((128, 32, 40))]
    x = cases[0].x.copy()
    x[777] = np.float16(30000.0)
    d_x = torch.from_numpy(x).cuda()
    kp = cases[0].nb * 24
    bufs = [B.expand(ctx, 0, c.d_codes, c.rows, c.nb) for c in cases]
    ys = [torch.empty(c.rows, dtype=torch.float32, device="cuda") for c in cases]
    B.gemv_rotated(ctx, [(b, c.d_scale, GAIN, y, c.rows) for b, c, y in zip(bufs, cases, ys)], d_x, kp, n=k)
    torch.cuda.synchronize()
    xr = np.concatenate([oracle.rotate(x[:k]), x[k:]])
    for c, y in zip(cases, ys):
        err, _ = check_gemv(oracle, dataclasses.replace(c, x=xr), y)
        assert err <= 1e-5


def test_gemv_rotated_error_codes(B, ctx):
    case = make_case(64, 96, seed=1)
    buf = B.expand(ctx, 0, case.d_codes, case.rows, case.nb)
    y = torch.empty(64, dtype=torch.float32, device="cuda")
    prob = [(buf, case.d_scale, GAIN, y, 64)]
    for kwargs in ({"n": 96, "block": 4}, {"n": 104}, {"n": 0}, {"n": 92}, {"n": 96, "block": 64}, {"n": 96, "block": 3}):
        with pytest.raises(B.LlvqError) as e:
            B.gemv_rotated(ctx, prob, case.d_x, 96, **kwargs)
        assert e.value.code == -1
    B.gemv_rotated(ctx, prob, case.d_x, 96, n=96)
    torch.cuda.synchronize()
    assert torch.isfinite(y).all()


def test_gemv_rotated_partial_length_passes_the_rest_through(B, ctx, oracle):
    """Only the first n entries are rotated; the entries after them - here real values, not padding - enter the
    matvec as they are."""
    rows, k = 96, 2560
    case = make_case(rows, k, seed=77)
    kp = case.nb * 24
    buf = B.expand(ctx, 0, case.d_codes, case.rows, case.nb)
    for n, block in ((2048, 0), (1024, 256), (2560 - 512, 512), (8, 8)):
        y = torch.empty(rows, dtype=torch.float32, device="cuda")
        B.gemv_rotated(ctx, [(buf, case.d_scale, GAIN, y, rows)], case.d_x, kp, n=n, block=block)
        torch.cuda.synchronize()
        ref = _rotated_reference(oracle, case, n, block, None)
        assert np.array_equal(ref.x[n:], case.x[n:]) and np.abs(case.x[n:k].astype(np.float64)).max() > 0
        err, _ = check_gemv(oracle, ref, y)
        assert err <= 1e-6


def test_gemv_rotated_refuses_a_block_that_does_not_fit_shared_memory(B, ctx):
    """A CTA rotates whole blocks: with three matrices' block-constant tables beside a 16384-coordinate block the
    shared memory of a multiprocessor is exceeded, and the call says so instead of launching."""
    k = 16384
    cases = [make_case(32, k, seed=5, tensor_id=i) for i in range(8)]
    kp = cases[0].nb * 24
    bufs = [B.expand(ctx, 0, c.d_codes, c.rows, c.nb) for c in cases]
    ys = [torch.empty(c.rows, dtype=torch.float32, device="cuda") for c in cases]
    probs = [(b, c.d_scale, GAIN, y, c.rows) for b, c, y in zip(bufs, cases, ys)]
    with pytest.raises(B.LlvqError) as e:
        B.gemv_rotated(ctx, probs, cases[0].d_x, kp, n=k)
    assert e.value.code == -3
    B.gemv_rotated(ctx, probs, cases[0].d_x, kp, n=k, block=1024)       # a shorter block fits
    torch.cuda.synchronize()
    assert all(torch.isfinite(y).all() for y in ys)


def test_gemv_rotated_random_shapes(B, ctx, oracle):
    """Seeded random shapes, rotated lengths, block lengths, sign vectors and groupings, each against the oracle chain."""
    rng = np.random.default_rng(2026)
    for it in range(30):
        k = int(rng.integers(1, 260)) * 24 if it % 3 else int(rng.choice([2560, 4096, 5120, 1536, 9728, 3072]))
        kp = (k + 23) // 24 * 24
        nmat = int(rng.integers(1, 4))
        rows = [int(rng.integers(1, 200)) for _ in range(nmat)]
        cases = [make_case(r, k, seed=1000 + it, tensor_id=i) for i, r in enumerate(rows)]
        x = cases[0].x
        # the rotated length: a multiple of 8, anywhere up to k_padded; the block: any power of two >= 8 dividing it
        n = int(rng.integers(1, kp // 8 + 1)) * 8
        divisors = [b for b in (8, 16, 32, 64, 128, 256, 512, 1024, 2048, 4096) if n % b == 0]
        block = int(rng.choice(divisors + [0]))
        neg = rng.integers(0, 2, size=n) if rng.random() < 0.5 else None
        bufs = [B.expand(ctx, 0, c.d_codes, c.rows, c.nb) for c in cases]
        ys = [torch.full((c.rows,), float("nan"), dtype=torch.float32, device="cuda") for c in cases]
        B.gemv_rotated(ctx, [(b_, c.d_scale, GAIN, y, c.rows) for b_, c, y in zip(bufs, cases, ys)], cases[0].d_x, kp, n=n, block=block,
                       negate_bits=None if neg is None else _bits(neg))
        torch.cuda.synchronize()
        B.status(ctx)
        xr = np.concatenate([oracle.rotate(x[:n], block, neg), x[n:]])
        for c, y in zip(cases, ys):
            err, _ = check_gemv(oracle, dataclasses.replace(c, x=xr), y)
            assert err <= 1e-5, (it, k, n, block, rows)
