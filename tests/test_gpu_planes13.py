"""Parity of the 13-byte layout (the 14-byte layout's codes, one header byte a block) against the CPU oracle."""
import numpy as np
import pytest
import torch

from helpers import GAIN, check_gemv, make_case

pytestmark = pytest.mark.gpu
N_POINTS = 111_043_117_458_000
L13 = 2


@pytest.fixture(scope="module")
def B():
    from paper_2609_02652_b200 import binding

    binding.load()
    assert binding.PLANES13 == L13
    return binding


@pytest.fixture(scope="module")
def ctx(B):
    c = B.create(0)
    yield c
    c.close()


SHAPES = [(1, 24), (3, 48), (33, 24 * 33), (40, 24 * 7), (64, 24 * 9 - 5), (32, 96), (31, 24 * 13), (257, 24 * 21), (70, 24 * 30),
          (96, 24 * 406), (1024, 2560), (3072, 3072)]


@pytest.mark.parametrize("rows,k", SHAPES)
def test_expand_bit_exact_and_size(B, ctx, oracle, rows, k):
    case = make_case(rows, k, seed=40 + rows)
    out = B.expand(ctx, L13, case.d_codes, rows, case.nb)
    torch.cuda.synchronize()
    assert out.numel() == B.layout_bytes(L13, rows, case.nb * 24) == oracle.planes13_bytes(rows, case.nb)
    assert out.numel() * 14 == B.layout_bytes(0, rows, case.nb * 24) * 13
    assert np.array_equal(out.cpu().numpy(), oracle.pack_planes13(case.codes, rows, case.nb))


def test_expand_invalid_codes_and_full_first_shell(B, ctx, oracle):
    codes = np.arange(196_560, dtype=np.uint64)                  # every point of the first shell, as 1365 x 144
    d = torch.from_numpy(codes.view(np.int64)).cuda()
    out = B.expand(ctx, L13, d, 1365, 144)
    assert np.array_equal(out.cpu().numpy(), oracle.pack_planes13(codes, 1365, 144))
    bad = np.array([N_POINTS, N_POINTS + 5, (1 << 47) - 1, 7, (1 << 47) | 9, 1 << 50], np.uint64)
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = B.expand(ctx, L13, torch.from_numpy(bad.view(np.int64)).cuda(), 2, 3, bad_count=cnt)
    assert np.array_equal(out.cpu().numpy(), oracle.pack_planes13(bad, 2, 3))
    assert cnt.item() == 4
    with pytest.raises(B.LlvqError) as e:                     # the context counted them too
        B.status(ctx)
    assert e.value.code == -6


@pytest.mark.parametrize("rows,k", [(40, 24 * 7), (257, 24 * 21), (3072, 3072), (33, 24 * 2), (5, 24)])
def test_decode_bit_exact(B, ctx, oracle, rows, k):
    """Coordinates bit for bit; the layout keeps no class id - the header byte is shell | parity << 4 | gain << 5."""
    case = make_case(rows, k, seed=3)
    buf = B.expand(ctx, L13, case.d_codes, rows, case.nb)
    coords, hdr = B.decode_i8(ctx, L13, buf, rows, case.nb)
    xs, _ = oracle.decode_batch(case.codes)
    assert np.array_equal(coords.cpu().numpy().reshape(-1, 24), xs)
    shell = (xs.astype(np.int64) ** 2).sum(1) // 16
    want = shell | ((xs[:, 0].astype(np.int64) & 1) << 4) | ((case.codes >> np.uint64(47)).astype(np.int64) << 5)
    assert np.array_equal(hdr.cpu().numpy().ravel().astype(np.int64), want)
    # and the 14-byte layout decodes to the same coordinates
    c14, _ = B.decode_i8(ctx, 0, B.expand(ctx, 0, case.d_codes, rows, case.nb), rows, case.nb)
    assert torch.equal(c14, coords)


@pytest.mark.parametrize("rows,k", SHAPES)
def test_gemv_every_row_and_same_as_14_byte_layout(B, ctx, oracle, rows, k):
    case = make_case(rows, k, seed=rows + k)
    buf = B.expand(ctx, L13, case.d_codes, rows, case.nb)
    y = B.gemv(ctx, L13, buf, case.d_scale, GAIN, case.d_x, rows, case.nb * 24)
    B.status(ctx)
    check_gemv(oracle, case, y)
    # the same arithmetic on the same codes: bit for bit the 14-byte layout's result
    y14 = B.gemv(ctx, 0, B.expand(ctx, 0, case.d_codes, rows, case.nb), case.d_scale, GAIN, case.d_x, rows, case.nb * 24)
    assert torch.equal(y, y14)
    y2 = B.gemv(ctx, L13, buf, case.d_scale, GAIN, case.d_x, rows, case.nb * 24)
    assert torch.equal(y, y2)


def test_gemv_special_cases_and_grouped(B, ctx, oracle):
    case = make_case(70, 24 * 30, seed=9)
    case.row_scale[5] = 0.0
    case.codes[17] = N_POINTS
    case.d_scale = torch.from_numpy(case.row_scale).cuda()
    case.d_codes = torch.from_numpy(case.codes.view(np.int64)).cuda()
    buf = B.expand(ctx, L13, case.d_codes, case.rows, case.nb)
    with pytest.raises(B.LlvqError) as e:                     # the one code that names no point is reported
        B.status(ctx)
    assert e.value.code == -6
    y = B.gemv(ctx, L13, buf, case.d_scale, GAIN, case.d_x, case.rows, case.nb * 24)
    check_gemv(oracle, case, y)
    assert y[5].item() == 0.0
    y1 = B.gemv(ctx, L13, buf, case.d_scale, (1.0, 1.0), case.d_x, case.rows, case.nb * 24)
    check_gemv(oracle, case, y1, gain=(1.0, 1.0))
    # q/k/v-like group sharing x: one launch, every matrix against the oracle and against its own launch
    k = 2560
    cases = [make_case(r, k, seed=11, tensor_id=i) for i, r in enumerate((4096, 1024, 1000))]
    x = cases[0].d_x
    bufs = [B.expand(ctx, L13, c.d_codes, c.rows, c.nb) for c in cases]
    ys = [torch.empty(c.rows, dtype=torch.float32, device="cuda") for c in cases]
    B.gemv_grouped(ctx, L13, [(b, c.d_scale, GAIN, y_, c.rows) for b, c, y_ in zip(bufs, cases, ys)], x, cases[0].nb * 24)
    torch.cuda.synchronize()
    for c, b, y_ in zip(cases, bufs, ys):
        c.x = cases[0].x
        check_gemv(oracle, c, y_)
        assert torch.equal(y_, B.gemv(ctx, L13, b, c.d_scale, GAIN, x, c.rows, c.nb * 24))


def test_what_the_layout_does_not_take(B, ctx):
    case = make_case(64, 96, seed=1)
    buf = B.expand(ctx, L13, case.d_codes, case.rows, case.nb)
    y = torch.empty(64, dtype=torch.float32, device="cuda")
    with pytest.raises(B.LlvqError) as e:
        B.dequant_fp16(ctx, L13, buf, case.d_scale, GAIN, 64, 96)
    assert e.value.code == -1
    with pytest.raises(B.LlvqError) as e:
        B.gemv(ctx, 4, buf, case.d_scale, GAIN, case.d_x, 64, 96)
    assert e.value.code == -1
    with pytest.raises(B.LlvqError) as e:
        B.gemv(ctx, L13, buf[16:], case.d_scale, GAIN, case.d_x, 64, 96)
    assert e.value.code == -2
    with pytest.raises(B.LlvqError) as e:
        B.expand(ctx, L13, case.d_codes, case.rows, case.nb, out=torch.empty(100, dtype=torch.uint8, device="cuda"))
    assert e.value.code == -3
    B.gemv(ctx, L13, buf, case.d_scale, GAIN, case.d_x, 64, 96, y=y)
    assert torch.isfinite(y).all()


def test_gemv_random_shapes_grouped(B, ctx, oracle):
    """Seeded random shapes and groupings in the 13-byte layout: the oracle's bar on every row, and bit for bit the
    14-byte layout's result."""
    rng = np.random.default_rng(13)
    for it in range(25):
        k = int(rng.integers(1, 300)) * 24 - int(rng.integers(0, 24))
        k = max(k, 1)
        nmat = int(rng.integers(1, 5))
        rows = [int(rng.integers(1, 300)) for _ in range(nmat)]
        cases = [make_case(r, k, seed=500 + it, tensor_id=i) for i, r in enumerate(rows)]
        kp = cases[0].nb * 24
        x = cases[0].d_x
        ys = {}
        for layout in (L13, 0):
            bufs = [B.expand(ctx, layout, c.d_codes, c.rows, c.nb) for c in cases]
            ys[layout] = [torch.full((c.rows,), float("nan"), dtype=torch.float32, device="cuda") for c in cases]
            B.gemv_grouped(ctx, layout, [(b_, c.d_scale, GAIN, y, c.rows) for b_, c, y in zip(bufs, cases, ys[layout])], x, kp)
        torch.cuda.synchronize()
        B.status(ctx)
        for i, c in enumerate(cases):
            c.x = cases[0].x
            check_gemv(oracle, c, ys[L13][i])
            assert torch.equal(ys[L13][i], ys[0][i]), (it, k, rows)
