"""Parity of the 10-byte layout (three-bit window codes plus the table of exact records, the sparse overlay of the
paper's Sec. 3.3) against the CPU oracle: bytes of the expander, decoded coordinates, the matvec on every row."""
import numpy as np
import pytest
import torch

from helpers import GAIN, check_gemv, make_case, make_overlay_case

pytestmark = pytest.mark.gpu
N_POINTS = 111_043_117_458_000
L10 = 3


@pytest.fixture(scope="module")
def B():
    from paper_2609_02652_b200 import binding

    binding.load()
    assert binding.PLANES10X == L10
    return binding


@pytest.fixture(scope="module")
def ctx(B):
    c = B.create(0)
    yield c
    c.close()


def expand_exact(B, ctx, case):
    """Count, size the buffer for exactly that many entries, expand."""
    n = B.overlay_count(ctx, case.d_codes, case.rows, case.nb)
    out = torch.full((B.overlay_bytes(case.rows, case.nb * 24, n),), 0xA5, dtype=torch.uint8, device="cuda")
    B.expand(ctx, L10, case.d_codes, case.rows, case.nb, out=out)
    return out, n


# (rows, k, share of the blocks replaced by exception blocks)
SHAPES = [(1, 24, 0.0), (3, 96, 0.5), (33, 24 * 33, 0.1), (40, 24 * 7, 0.3), (64, 24 * 9 - 5, 0.0), (32, 96, 1.0), (31, 24 * 13, 0.05),
          (257, 24 * 21, 0.02), (70, 24 * 30, 0.2), (96, 24 * 406, 0.01), (1024, 2560, 0.0), (3072, 3072, 0.03), (2100, 24 * 130, 0.5),
          (64, 98304, 0.01), (1, 98304, 0.2), (5000, 24 * 5, 0.3), (70000, 48, 0.1)]      # the longest rows the GEMV takes; tall and thin; no tile at all


@pytest.mark.parametrize("rows,k,rate", SHAPES)
def test_expand_bit_exact_and_size(B, ctx, oracle, rows, k, rate):
    case = make_overlay_case(oracle, rows, k, seed=40 + rows, rate=rate)
    out, n = expand_exact(B, ctx, case)
    B.status(ctx)
    want, n_ref = oracle.pack_planes10x(case.codes, rows, case.nb)
    assert n == n_ref and out.numel() == want.size == oracle.planes10x_bytes(rows, case.nb, n)
    assert np.array_equal(out.cpu().numpy(), want)
    if rate == 0.0 and rows * case.nb < 10000:
        assert n <= 2                                     # the synthetic stream: about one block in eight thousand
    if rate >= 0.3:
        assert n > 0


def test_room_for_the_table(B, ctx, oracle):
    """The default size has room for one exception in 32 blocks; a table that is too small keeps its first entries,
    the index stops at the capacity, the status call reports it once, and the matvec still reads nothing past the table."""
    case = make_overlay_case(oracle, 200, 24 * 40, seed=4, rate=0.02)
    want, n = oracle.pack_planes10x(case.codes, case.rows, case.nb)
    assert 0 < n <= (case.rows * case.nb + 31) // 32
    out = B.expand(ctx, L10, case.d_codes, case.rows, case.nb)
    B.status(ctx)
    assert out.numel() == B.layout_bytes(L10, case.rows, case.nb * 24)
    assert np.array_equal(out[: want.size].cpu().numpy(), want)
    y = B.gemv(ctx, L10, out, case.d_scale, GAIN, case.d_x, case.rows, case.nb * 24)
    check_gemv(oracle, case, y)
    # half the room
    small = torch.zeros(B.overlay_bytes(case.rows, case.nb * 24, n // 2), dtype=torch.uint8, device="cuda")
    B.expand(ctx, L10, case.d_codes, case.rows, case.nb, out=small)
    with pytest.raises(B.LlvqError) as e:
        B.status(ctx)
    assert e.value.code == -3
    B.status(ctx)                                             # reported once
    want_small, n2 = oracle.pack_planes10x(case.codes, case.rows, case.nb, capacity=n // 2)
    assert n2 == n and np.array_equal(small.cpu().numpy(), want_small)
    y = B.gemv(ctx, L10, small, case.d_scale, GAIN, case.d_x, case.rows, case.nb * 24)      # incomplete, but in bounds
    assert torch.isfinite(y).all()
    B.status(ctx)
    # no room at all is still a valid buffer
    none = torch.zeros(B.overlay_bytes(case.rows, case.nb * 24, 0), dtype=torch.uint8, device="cuda")
    B.expand(ctx, L10, case.d_codes, case.rows, case.nb, out=none)
    with pytest.raises(B.LlvqError) as e:
        B.status(ctx)
    assert e.value.code == -3
    with pytest.raises(B.LlvqError) as e:                     # less than the fixed part is refused
        B.expand(ctx, L10, case.d_codes, case.rows, case.nb, out=none[:-16])
    assert e.value.code == -3


def test_expand_invalid_codes_and_full_first_shell(B, ctx, oracle):
    codes = np.arange(196_560, dtype=np.uint64)                  # every point of the first shell, as 1365 x 144
    d = torch.from_numpy(codes.view(np.int64)).cuda()
    assert B.overlay_count(ctx, d, 1365, 144) == 0               # coordinates within -4..4 and one +-8 with zeros: all fit
    out = B.expand(ctx, L10, d, 1365, 144, out=torch.empty(B.overlay_bytes(1365, 144 * 24, 0), dtype=torch.uint8, device="cuda"))
    want, n = oracle.pack_planes10x(codes, 1365, 144)
    assert n == 0 and np.array_equal(out.cpu().numpy(), want)
    bad = np.array([N_POINTS, N_POINTS + 5, (1 << 47) - 1, 7, (1 << 47) | 9, 1 << 50, 3, 4], np.uint64)
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = B.expand(ctx, L10, torch.from_numpy(bad.view(np.int64)).cuda(), 2, 4, bad_count=cnt,
                   out=torch.empty(B.overlay_bytes(2, 96, 0), dtype=torch.uint8, device="cuda"))
    want, n = oracle.pack_planes10x(bad, 2, 4)
    assert n == 0 and np.array_equal(out.cpu().numpy(), want)
    assert cnt.item() == 4
    with pytest.raises(B.LlvqError) as e:                     # the context counted them too
        B.status(ctx)
    assert e.value.code == -6


@pytest.mark.parametrize("rows,k,rate", [(40, 24 * 7, 0.3), (257, 24 * 21, 0.05), (3072, 3072, 0.0), (33, 24 * 2, 0.5), (5, 24, 1.0), (70, 24 * 12, 1.0)])
def test_decode_bit_exact(B, ctx, oracle, rows, k, rate):
    """Short records and table together give back every coordinate; the header byte is shell | parity << 4 | gain << 5."""
    case = make_overlay_case(oracle, rows, k, seed=3, rate=rate)
    buf, _ = expand_exact(B, ctx, case)
    coords, hdr = B.decode_i8(ctx, L10, buf, rows, case.nb)
    xs, _ = oracle.decode_batch(case.codes)
    assert np.array_equal(coords.cpu().numpy().reshape(-1, 24), xs)
    shell = (xs.astype(np.int64) ** 2).sum(1) // 16
    want = shell | ((xs[:, 0].astype(np.int64) & 1) << 4) | ((case.codes >> np.uint64(47)).astype(np.int64) << 5)
    assert np.array_equal(hdr.cpu().numpy().ravel().astype(np.int64), want)


@pytest.mark.parametrize("rows,k,rate", SHAPES)
def test_gemv_every_row(B, ctx, oracle, rows, k, rate):
    case = make_overlay_case(oracle, rows, k, seed=rows + k, rate=rate)
    buf, n = expand_exact(B, ctx, case)
    y = B.gemv(ctx, L10, buf, case.d_scale, GAIN, case.d_x, rows, case.nb * 24)
    B.status(ctx)
    check_gemv(oracle, case, y)
    y2 = B.gemv(ctx, L10, buf, case.d_scale, GAIN, case.d_x, rows, case.nb * 24)
    assert torch.equal(y, y2)
    y14 = B.gemv(ctx, 0, B.expand(ctx, 0, case.d_codes, rows, case.nb), case.d_scale, GAIN, case.d_x, rows, case.nb * 24)
    # Not bit for bit the 14-byte layout's result: a block's integer sum is the same, but it is formed in two halves
    # (low and high limb pair) whose split depends on the stored code, each half is rounded to f32, and an exception's
    # product is rounded to the accumulator's quantum by itself.  The two agree to far below f32's step.
    assert float((y - y14).abs().max()) <= 1e-6 * float(y14.abs().max())
    assert n > 0 or rate == 0.0 or case.nb < 4          # blocks past the tiles are never exceptions


def test_gemv_special_cases_and_grouped(B, ctx, oracle):
    case = make_overlay_case(oracle, 70, 24 * 30, seed=9, rate=0.1)
    case.row_scale[5] = 0.0
    case.codes[17] = N_POINTS
    case.d_scale = torch.from_numpy(case.row_scale).cuda()
    case.d_codes = torch.from_numpy(case.codes.view(np.int64)).cuda()
    buf, _ = expand_exact(B, ctx, case)
    with pytest.raises(B.LlvqError) as e:                     # the one code that names no point is reported
        B.status(ctx)
    assert e.value.code == -6
    y = B.gemv(ctx, L10, buf, case.d_scale, GAIN, case.d_x, case.rows, case.nb * 24)
    check_gemv(oracle, case, y)
    assert y[5].item() == 0.0
    y1 = B.gemv(ctx, L10, buf, case.d_scale, (1.0, 1.0), case.d_x, case.rows, case.nb * 24)
    check_gemv(oracle, case, y1, gain=(1.0, 1.0))
    # q/k/v-like group sharing x: one launch, every matrix against the oracle and against its own launch
    k = 2560
    cases = [make_overlay_case(oracle, r, k, seed=11, rate=rate, tensor_id=i) for i, (r, rate) in enumerate(((4096, 0.01), (1024, 0.0), (1000, 0.2)))]
    x = cases[0].d_x
    bufs = [expand_exact(B, ctx, c)[0] for c in cases]
    ys = [torch.empty(c.rows, dtype=torch.float32, device="cuda") for c in cases]
    B.gemv_grouped(ctx, L10, [(b, c.d_scale, GAIN, y_, c.rows) for b, c, y_ in zip(bufs, cases, ys)], x, cases[0].nb * 24)
    torch.cuda.synchronize()
    for c, b, y_ in zip(cases, bufs, ys):
        c.x = cases[0].x
        check_gemv(oracle, c, y_)
        assert torch.equal(y_, B.gemv(ctx, L10, b, c.d_scale, GAIN, x, c.rows, c.nb * 24))


def test_what_the_layout_does_not_take(B, ctx):
    case = make_case(64, 96, seed=1)
    buf = B.expand(ctx, L10, case.d_codes, case.rows, case.nb)
    y = torch.empty(64, dtype=torch.float32, device="cuda")
    with pytest.raises(B.LlvqError) as e:
        B.dequant_fp16(ctx, L10, buf, case.d_scale, GAIN, 64, 96)
    assert e.value.code == -1
    with pytest.raises(B.LlvqError) as e:
        B.gemv(ctx, 4, buf, case.d_scale, GAIN, case.d_x, 64, 96)
    assert e.value.code == -1
    with pytest.raises(B.LlvqError) as e:
        B.gemv(ctx, L10, buf[16:], case.d_scale, GAIN, case.d_x, 64, 96)
    assert e.value.code == -2
    with pytest.raises(B.LlvqError) as e:
        B.expand(ctx, L10, case.d_codes, case.rows, case.nb, out=torch.empty(100, dtype=torch.uint8, device="cuda"))
    assert e.value.code == -3
    B.gemv(ctx, L10, buf, case.d_scale, GAIN, case.d_x, 64, 96, y=y)
    assert torch.isfinite(y).all()
    B.status(ctx)


def test_gemv_random_shapes_grouped(B, ctx, oracle):
    """Seeded random shapes, groupings and exception rates: the oracle's bar on every row."""
    rng = np.random.default_rng(17)
    for it in range(25):
        k = max(int(rng.integers(1, 300)) * 24 - int(rng.integers(0, 24)), 1)
        nmat = int(rng.integers(1, 5))
        rows = [int(rng.integers(1, 300)) for _ in range(nmat)]
        rate = float(rng.choice([0.0, 0.01, 0.1, 0.6]))
        cases = [make_overlay_case(oracle, r, k, seed=500 + it, rate=rate, tensor_id=i) for i, r in enumerate(rows)]
        kp = cases[0].nb * 24
        x = cases[0].d_x
        bufs = [expand_exact(B, ctx, c)[0] for c in cases]
        ys = [torch.full((c.rows,), float("nan"), dtype=torch.float32, device="cuda") for c in cases]
        B.gemv_grouped(ctx, L10, [(b_, c.d_scale, GAIN, y, c.rows) for b_, c, y in zip(bufs, cases, ys)], x, kp)
        torch.cuda.synchronize()
        B.status(ctx)
        for i, c in enumerate(cases):
            c.x = cases[0].x
            check_gemv(oracle, c, ys[i])
