"""Parity of the CUDA path against the CPU oracle, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

from helpers import GAIN, check_gemv, make_case

pytestmark = pytest.mark.gpu

N_POINTS = 111_043_117_458_000


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


def _expected(oracle, layout, case):
    return oracle.pack_planes(case.codes, case.rows, case.nb) if layout == 0 else oracle.pack_onehot(case.codes, case.rows, case.nb)


SMALL = [(1, 24), (3, 48), (33, 24 * 33), (40, 24 * 7), (64, 24 * 9 - 5), (32, 96), (31, 24 * 13), (257, 24 * 21)]


def test_tables_agree_with_oracle(B, ctx, oracle):
    assert B.num_classes(ctx) == oracle.num_classes() == 301
    for c in range(301):
        assert B.class_base(ctx, c) == oracle.class_info(c)["base"]
    assert B.class_base(ctx, 301) == N_POINTS


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("rows,k", SMALL)
def test_expand_bit_exact_small(B, ctx, oracle, layout, rows, k):
    case = make_case(rows, k, seed=20 + rows)
    out = B.expand(ctx, layout, case.d_codes, rows, case.nb)
    torch.cuda.synchronize()
    assert out.numel() == B.layout_bytes(layout, rows, case.nb * 24)
    assert np.array_equal(out.cpu().numpy(), _expected(oracle, layout, case))


@pytest.mark.parametrize("layout", [0, 1])
def test_expand_bit_exact_config0_and_extra_indices(B, ctx, oracle, layout):
    from paper_2609_02652_b200 import datagen

    case = make_case(3072, 3072, seed=0)
    out = B.expand(ctx, layout, case.d_codes, case.rows, case.nb)
    assert np.array_equal(out.cpu().numpy(), _expected(oracle, layout, case))
    # 10 000 more indices, no gain bit, as a 100 x 100 matrix
    extra = datagen.make_indices(10_000, seed=0)
    case.rows, case.nb, case.codes = 100, 100, extra.numpy().astype(np.uint64)
    out = B.expand(ctx, layout, extra.cuda(), 100, 100)
    assert np.array_equal(out.cpu().numpy(), _expected(oracle, layout, case))


@pytest.mark.parametrize("layout", [0, 1])
def test_expand_whole_first_shell_class_edges_and_bad_codes(B, ctx, oracle, layout):
    # all 196 560 indices of shell 2 as a 4095 x 48 matrix
    codes = np.arange(196_560, dtype=np.uint64)
    case = make_case(1, 24, 0, device=None)
    case.rows, case.nb, case.codes = 4095, 48, codes
    out = B.expand(ctx, layout, torch.from_numpy(codes.astype(np.int64)).cuda(), 4095, 48)
    assert np.array_equal(out.cpu().numpy(), _expected(oracle, layout, case))
    # first and last index of every class, with and without the gain bit; then codes naming no point
    edges = []
    for c in range(301):
        i = oracle.class_info(c)
        edges += [i["base"], i["base"] + i["size"] - 1, (i["base"] + i["size"] // 2) | (1 << 47)]
    bad = [N_POINTS, N_POINTS + 12345, (1 << 47) - 1, N_POINTS | (1 << 47), 1 << 48, (1 << 63) | 5]
    codes = np.array(edges + bad + [0] * (7 * 131 - len(edges) - len(bad)), dtype=np.uint64)
    case.rows, case.nb, case.codes = 131, 7, codes
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = B.expand(ctx, layout, torch.from_numpy(codes.view(np.int64)).cuda(), 131, 7, bad_count=cnt)
    assert np.array_equal(out.cpu().numpy(), _expected(oracle, layout, case))
    assert int(cnt.item()) == len(bad)
    with pytest.raises(B.LlvqError) as e:                     # the context counted them too
        B.status(ctx)
    assert e.value.code == -6


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("rows,k", [(40, 24 * 7), (257, 24 * 21), (3072, 3072)])
def test_decode_bit_exact(B, ctx, oracle, layout, rows, k):
    case = make_case(rows, k, seed=3)
    buf = B.expand(ctx, layout, case.d_codes, rows, case.nb)
    coords, cls = B.decode_i8(ctx, layout, buf, rows, case.nb)
    xs, ref_cls = oracle.decode_batch(case.codes)
    assert np.array_equal(coords.cpu().numpy().reshape(-1, 24), xs)
    assert np.array_equal(cls.cpu().numpy().ravel().astype(np.int32), ref_cls)


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("rows,k", SMALL + [(3072, 3072), (1024, 2560), (96, 24 * 406)])
def test_gemv_every_row(B, ctx, oracle, layout, rows, k):
    case = make_case(rows, k, seed=rows + k)
    buf = B.expand(ctx, layout, case.d_codes, rows, case.nb)
    y = B.gemv(ctx, layout, buf, case.d_scale, GAIN, case.d_x, rows, case.nb * 24)
    B.status(ctx)                      # no bounded wait ran out
    check_gemv(oracle, case, y)
    # a second launch on the same context finds the scratch clean
    y2 = B.gemv(ctx, layout, buf, case.d_scale, GAIN, case.d_x, rows, case.nb * 24)
    assert torch.equal(y, y2)


def test_gemv_special_cases(B, ctx, oracle):
    case = make_case(70, 24 * 30, seed=9)
    case.row_scale[5] = 0.0            # a scale that rounds to zero: y must be exactly zero
    case.codes[17] = N_POINTS          # a code naming no point contributes nothing
    case.d_scale = torch.from_numpy(case.row_scale).cuda()
    case.d_codes = torch.from_numpy(case.codes.view(np.int64)).cuda()
    buf = B.expand(ctx, 0, case.d_codes, case.rows, case.nb)
    with pytest.raises(B.LlvqError) as e:                     # the one code that names no point is reported
        B.status(ctx)
    assert e.value.code == -6
    y = B.gemv(ctx, 0, buf, case.d_scale, GAIN, case.d_x, case.rows, case.nb * 24)
    check_gemv(oracle, case, y)
    assert y[5].item() == 0.0
    # gain (1, 1) is the gain-free result
    y1 = B.gemv(ctx, 0, buf, case.d_scale, (1.0, 1.0), case.d_x, case.rows, case.nb * 24)
    check_gemv(oracle, case, y1, gain=(1.0, 1.0))
    # x = e_j returns column j of the dequantised matrix
    W = oracle.dequant(case.codes, case.rows, case.nb, case.row_scale, GAIN)
    for j in (0, 23, 24 * 30 - 1, 333):
        e = torch.zeros(case.nb * 24, dtype=torch.float16, device="cuda")
        e[j] = 1
        yj = B.gemv(ctx, 0, buf, case.d_scale, GAIN, e, case.rows, case.nb * 24).cpu().numpy()
        assert np.allclose(yj, W[:, j], rtol=2e-7, atol=0)


def test_planes_and_onehot_agree(B, ctx):
    case = make_case(520, 24 * 45, seed=4)
    bp = B.expand(ctx, 0, case.d_codes, case.rows, case.nb)
    bo = B.expand(ctx, 1, case.d_codes, case.rows, case.nb)
    cp, kp = B.decode_i8(ctx, 0, bp, case.rows, case.nb)
    co, ko = B.decode_i8(ctx, 1, bo, case.rows, case.nb)
    assert torch.equal(cp, co) and torch.equal(kp, ko)


@pytest.mark.parametrize("layout", [0, 1])
def test_grouped_launch_is_bit_identical(B, ctx, oracle, layout):
    k = 2560
    shapes = [(4096, 0), (1024, 1), (1000, 2)]
    cases = [make_case(r, k, seed=1, tensor_id=t) for r, t in shapes]
    for c in cases[1:]:
        c.x, c.d_x = cases[0].x, cases[0].d_x          # a fused group shares x
    bufs = [B.expand(ctx, layout, c.d_codes, c.rows, c.nb) for c in cases]
    gains = [(0.75, 1.5), (1.0, 0.5), (1.25, 2.0)]
    single = [B.gemv(ctx, layout, b, c.d_scale, g, c.d_x, c.rows, c.nb * 24) for b, c, g in zip(bufs, cases, gains)]
    ys = [torch.full((c.rows,), float("nan"), dtype=torch.float32, device="cuda") for c in cases]
    B.gemv_grouped(ctx, layout, [(b, c.d_scale, g, y, c.rows) for b, c, g, y in zip(bufs, cases, gains, ys)], cases[0].d_x, cases[0].nb * 24)
    for s, y, c, g in zip(single, ys, cases, gains):
        assert torch.equal(s, y)
        check_gemv(oracle, c, y, gain=g)


def test_fp16_arm_and_dequant(B, ctx, oracle):
    case = make_case(300, 24 * 50, seed=12)
    for layout in (0, 1):
        buf = B.expand(ctx, layout, case.d_codes, case.rows, case.nb)
        W = B.dequant_fp16(ctx, layout, buf, case.d_scale, GAIN, case.rows, case.nb * 24)
        ref = oracle.dequant(case.codes, case.rows, case.nb, case.row_scale, GAIN)
        got = W.cpu().numpy().astype(np.float64)
        # one rounding to fp16 of an f32 product: within one fp16 ulp of the exactly rounded value
        ulp = np.maximum(np.abs(ref) * 2.0**-10, 2.0**-24)
        assert (np.abs(got - ref) <= ulp).all()
    y = B.gemv_fp16(W, case.d_x, case.rows, case.nb * 24)
    ref_y = W.cpu().numpy().astype(np.float64) @ case.x.astype(np.float64)
    scale = np.linalg.norm(W.cpu().numpy().astype(np.float64), axis=1) * np.linalg.norm(case.x.astype(np.float64))
    assert (np.abs(y.cpu().numpy() - ref_y) <= 1e-5 * np.maximum(scale, 1e-30)).all()


def test_noweights_control_returns_zero(B, ctx):
    case = make_case(4096, 4096, seed=2)
    y = torch.full((case.rows,), float("nan"), dtype=torch.float32, device="cuda")
    B.gemv_noweights(ctx, case.d_scale, case.d_x, case.rows, case.nb * 24, y=y)
    assert (y == 0).all()


def test_error_codes(B, ctx):
    case = make_case(64, 96, seed=1)
    buf = B.expand(ctx, 0, case.d_codes, case.rows, case.nb)
    with pytest.raises(B.LlvqError) as e:
        B.gemv(ctx, 7, buf, case.d_scale, GAIN, case.d_x, case.rows, 96)
    assert e.value.code == -1
    with pytest.raises(B.LlvqError) as e:
        B.gemv(ctx, 0, buf, case.d_scale, GAIN, case.d_x, case.rows, 95)
    assert e.value.code == -1
    with pytest.raises(B.LlvqError) as e:
        B.gemv(ctx, 0, buf[16:], case.d_scale, GAIN, case.d_x, case.rows, 96)      # misaligned layout
    assert e.value.code == -2
    with pytest.raises(B.LlvqError) as e:
        B.expand(ctx, 0, case.d_codes, case.rows, case.nb, out=torch.empty(100, dtype=torch.uint8, device="cuda"))
    assert e.value.code == -3
    # the context is still usable
    y = B.gemv(ctx, 0, buf, case.d_scale, GAIN, case.d_x, case.rows, 96)
    assert torch.isfinite(y).all()


def test_wide_matrix_many_groups_and_size_limits(B, ctx, oracle):
    # a long row (1024 blocks) and a launch over eight matrices
    case = make_case(70, 24 * 1024, seed=41)
    buf = B.expand(ctx, 0, case.d_codes, case.rows, case.nb)
    y = B.gemv(ctx, 0, buf, case.d_scale, GAIN, case.d_x, case.rows, case.nb * 24)
    B.status(ctx)
    check_gemv(oracle, case, y)
    cases = [make_case(32 + 17 * i, 24 * 40, seed=50, tensor_id=i) for i in range(8)]
    for c in cases[1:]:
        c.x, c.d_x = cases[0].x, cases[0].d_x
    bufs = [B.expand(ctx, 0, c.d_codes, c.rows, c.nb) for c in cases]
    gains = [(0.5 + 0.25 * i, 1.0 + 0.125 * i) for i in range(8)]
    ys = [torch.full((c.rows,), float("nan"), dtype=torch.float32, device="cuda") for c in cases]
    B.gemv_grouped(ctx, 0, [(b, c.d_scale, g, y, c.rows) for b, c, g, y in zip(bufs, cases, gains, ys)], cases[0].d_x, 24 * 40)
    B.status(ctx)
    for c, g, y in zip(cases, gains, ys):
        check_gemv(oracle, c, y, gain=g)
    # nine matrices, and an in-dimension above the documented maximum: refused, nothing launched
    with pytest.raises(B.LlvqError) as e:
        B.gemv_grouped(ctx, 0, [(bufs[0], cases[0].d_scale, GAIN, ys[0], cases[0].rows)] * 9, cases[0].d_x, 24 * 40)
    assert e.value.code == -1
    big_k = 98304 + 24
    xx = torch.zeros(big_k, dtype=torch.float16, device="cuda")
    with pytest.raises(B.LlvqError) as e:
        B.gemv(ctx, 0, bufs[0], cases[0].d_scale, GAIN, xx, 32, big_k)
    assert e.value.code == -3
    # the maximum itself works: 4096 blocks a row, one more than the tiles of 1023 columns would hold
    case = make_case(40, 98304, seed=43)
    buf = B.expand(ctx, 0, case.d_codes, case.rows, case.nb)
    y = B.gemv(ctx, 0, buf, case.d_scale, GAIN, case.d_x, case.rows, case.nb * 24)
    B.status(ctx)
    check_gemv(oracle, case, y)
    # negative and zero gains are legal
    y = B.gemv(ctx, 0, bufs[0], cases[0].d_scale, (-1.25, 0.0), cases[0].d_x, cases[0].rows, 24 * 40)
    check_gemv(oracle, cases[0], y, gain=(-1.25, 0.0))


@pytest.mark.parametrize("scale", [0.0, 6e-8, 1e-4, 3.0e3])
def test_gemv_extreme_activation_ranges(B, ctx, oracle, scale):
    """All-zero x, fp16-subnormal x, small x and x near the top of the fp16 range: the fixed-point quantum
    follows max |x|, so the normalised error bound holds at every scale."""
    case = make_case(96, 24 * 57, seed=77)
    xs = (case.x.astype(np.float64) * scale).astype(np.float16)
    if scale == 6e-8:
        assert (np.abs(xs[xs != 0]) < 6.2e-5).all()          # every non-zero entry is an fp16 subnormal
    case.x, case.d_x = xs, torch.from_numpy(xs).cuda()
    buf = B.expand(ctx, 0, case.d_codes, case.rows, case.nb)
    y = B.gemv(ctx, 0, buf, case.d_scale, GAIN, case.d_x, case.rows, case.nb * 24)
    B.status(ctx)
    if not xs.any():
        assert (y == 0).all()
    else:
        check_gemv(oracle, case, y)


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable(B, oracle):
    """No fault is injected: a one-warp kernel waits about a millisecond on a barrier nothing completes."""
    ctx = B.create(0)
    try:
        B.status(ctx)
        B.selftest_wait_limit(ctx)
        with pytest.raises(B.LlvqError) as e:
            B.status(ctx)
        assert e.value.code == -5
        B.status(ctx)                          # the flag was reset
        case = make_case(100, 24 * 20, seed=3)
        buf = B.expand(ctx, 0, case.d_codes, case.rows, case.nb)
        y = B.gemv(ctx, 0, buf, case.d_scale, GAIN, case.d_x, case.rows, case.nb * 24)
        B.status(ctx)
        check_gemv(oracle, case, y)
    finally:
        ctx.close()


def test_gemv_fixed_point_activations_inside_one_vector(B, ctx, oracle):
    """The 14-byte GEMV takes x as fixed point on a scale set by the largest |x| (include/llvq.h): entries within
    2^-18 of the largest are exact, smaller ones are rounded to within 2^-29 of the largest.  One huge entry among
    small ones: the result stays within that bound of the f64 oracle, row by row, and the normalised bar holds."""
    case = make_case(128, 24 * 41, seed=91)
    xs = (case.x.astype(np.float64) * 2.0**-12).astype(np.float16)          # |x| around 2^-12
    xs[500] = np.float16(40000.0)                                           # and one entry 2^27 times larger
    case.x, case.d_x = xs, torch.from_numpy(xs).cuda()
    buf = B.expand(ctx, 0, case.d_codes, case.rows, case.nb)
    y = B.gemv(ctx, 0, buf, case.d_scale, GAIN, case.d_x, case.rows, case.nb * 24)
    B.status(ctx)
    y_ref, wnorm, abssum = oracle.matvec(case.codes, case.rows, case.nb, case.row_scale, GAIN, case.x)
    err = np.abs(y.cpu().numpy().astype(np.float64) - y_ref)
    xnorm = float(np.linalg.norm(xs.astype(np.float64)))
    assert (err <= 1e-4 * wnorm * xnorm).all()
    # every coordinate's activation is off by at most 2^-29 * 65536 (the largest is below 2^16); the weights of a
    # row are at most |w_i| each, so the row is off by at most that times sum |w_i|, plus f32 rounding of the sums
    W = oracle.dequant(case.codes, case.rows, case.nb, case.row_scale, GAIN)
    bound = 2.0**-29 * 65536.0 * np.abs(W).sum(axis=1) + 2.0**-22 * abssum
    assert (err <= bound).all(), float(np.max(err / bound))


@pytest.mark.parametrize("rows,k,batch", [(70, 24 * 30, 2), (257, 24 * 21, 3), (96, 24 * 406, 4), (33, 24 * 33, 4), (1024, 2560, 2), (3072, 3072, 4), (130, 24 * 50, 7), (64, 24 * 9, 8)])
def test_gemv_batch_matches_single_vector_calls_and_oracle(B, ctx, oracle, rows, k, batch):
    """Small-batch decode: one pass over the records for several activation vectors.  Every vector's result is
    bit-identical to llvq_gemv on that vector alone, and within the bar of the f64 oracle."""
    case = make_case(rows, k, seed=rows + k + batch)
    buf = B.expand(ctx, 0, case.d_codes, rows, case.nb)
    kp = case.nb * 24
    xs = []
    for j in range(batch):
        xj = (case.x.astype(np.float64) * (0.25 * 3.0**j)).astype(np.float16) if j else case.x.copy()
        xj = np.roll(xj[:k], 7 * j)                      # distinct vectors of very different magnitude
        xs.append(np.concatenate([xj, np.zeros(kp - k, dtype=np.float16)]))
    X = torch.from_numpy(np.stack(xs)).cuda()
    Y = B.gemv_batch(ctx, buf, case.d_scale, GAIN, X, rows, kp)
    B.status(ctx)
    assert Y.shape == (batch, rows)
    for j in range(batch):
        yj = B.gemv(ctx, 0, buf, case.d_scale, GAIN, X[j].contiguous(), rows, kp)
        assert torch.equal(Y[j], yj)
        cj = make_case(rows, k, seed=rows + k + batch, device=None)
        cj.x = xs[j]
        check_gemv(oracle, cj, Y[j])
    # a second batched launch finds the scratch clean
    Y2 = B.gemv_batch(ctx, buf, case.d_scale, GAIN, X, rows, kp)
    assert torch.equal(Y, Y2)


def test_gemv_batch_limits(B, ctx):
    case = make_case(64, 96, seed=1)
    buf = B.expand(ctx, 0, case.d_codes, case.rows, case.nb)
    X = torch.zeros((9, 96), dtype=torch.float16, device="cuda")
    with pytest.raises(B.LlvqError) as e:
        B.gemv_batch(ctx, buf, case.d_scale, GAIN, X, case.rows, 96)                # more vectors than LLVQ_MAX_BATCH
    assert e.value.code == -1
    small = B.create(0, scratch_bytes=64 * 8)                                      # scratch for one vector of 64 rows only
    try:
        with pytest.raises(B.LlvqError) as e:
            B.gemv_batch(small, buf, case.d_scale, GAIN, X[:2].contiguous(), case.rows, 96)
        assert e.value.code == -3
        y = B.gemv_batch(small, buf, case.d_scale, GAIN, X[:1].contiguous(), case.rows, 96)
        assert (y == 0).all()
    finally:
        small.close()


def test_gemv_random_shapes_grouped_and_batched(B, ctx, oracle):
    """Thirty seeded random shapes (rows 1..700, 1..260 blocks a row: every leftover count, row groups that end
    mid-group, launches smaller and larger than the grid), each through a plain, a grouped and a batched launch."""
    rng = np.random.default_rng(20260925)
    for it in range(30):
        rows = int(rng.integers(1, 700))
        nb = int(rng.integers(1, 260))
        case = make_case(rows, 24 * nb, seed=1000 + it)
        buf = B.expand(ctx, 0, case.d_codes, rows, nb)
        gain = (float(rng.uniform(0.25, 2.0)), float(rng.uniform(0.25, 2.0)))
        y = B.gemv(ctx, 0, buf, case.d_scale, gain, case.d_x, rows, 24 * nb)
        check_gemv(oracle, case, y, gain=gain)
        # the same matrix as the second member of a group, behind a matrix of another height
        other = make_case(int(rng.integers(1, 300)), 24 * nb, seed=2000 + it, tensor_id=1)
        other.d_x = case.d_x
        bo = B.expand(ctx, 0, other.d_codes, other.rows, nb)
        yo = torch.empty(other.rows, dtype=torch.float32, device="cuda")
        yg = torch.full((rows,), float("nan"), dtype=torch.float32, device="cuda")
        B.gemv_grouped(ctx, 0, [(bo, other.d_scale, GAIN, yo, other.rows), (buf, case.d_scale, gain, yg, rows)], case.d_x, 24 * nb)
        assert torch.equal(y, yg)
        # and as vector 1 of a batch of three
        X = torch.stack([other.d_x.flip(0), case.d_x, (case.d_x.float() * 0.5).half()]).contiguous()
        Y = B.gemv_batch(ctx, buf, case.d_scale, gain, X, rows, 24 * nb)
        assert torch.equal(Y[1], y)
    B.status(ctx)


def test_gemv_without_programmatic_dependent_launch(B, oracle):
    """llvq_set_pdl(0): the same kernel as an ordinary launch; same bits."""
    ctx = B.create(0)
    try:
        case = make_case(300, 24 * 77, seed=21)
        buf = B.expand(ctx, 0, case.d_codes, case.rows, case.nb)
        y1 = B.gemv(ctx, 0, buf, case.d_scale, GAIN, case.d_x, case.rows, case.nb * 24)
        B.set_pdl(ctx, False)
        y2 = B.gemv(ctx, 0, buf, case.d_scale, GAIN, case.d_x, case.rows, case.nb * 24)
        y3 = B.gemv(ctx, 0, buf, case.d_scale, GAIN, case.d_x, case.rows, case.nb * 24)
        B.status(ctx)
        assert torch.equal(y1, y2) and torch.equal(y2, y3)
        check_gemv(oracle, case, y2)
    finally:
        ctx.close()


def test_invalid_codes_surface_through_status(B, ctx):
    """A caller that passes no bad_count still learns that codes named no point: llvq_status returns LLVQ_EINDEX
    once, then LLVQ_OK; a clean expansion in between does not raise."""
    case = make_case(64, 96, seed=7)
    B.expand(ctx, B.PLANES, case.d_codes, case.rows, case.nb)
    B.status(ctx)
    bad = case.d_codes.clone()
    bad[5] = (1 << 47) - 1                                  # index 2^47 - 1 >= number of points
    bad[70] = 1 << 60                                       # bits above bit 47
    for layout in (B.PLANES, B.ONEHOT, B.PLANES13):
        B.expand(ctx, layout, bad, case.rows, case.nb)      # bad_count = None
        with pytest.raises(B.LlvqError) as e:
            B.status(ctx)
        assert e.value.code == -6 and "no point" in str(e.value)
        B.status(ctx)


def test_expand_then_gemv_back_to_back_on_fresh_buffers(B, ctx, oracle):
    """llvq_expand followed at once by llvq_gemv on the same stream, programmatic dependent launch on: the GEMV
    reads records ahead of its dependency wait, so the library launches this one as an ordinary kernel.  Fresh
    buffers every round (filled with the pattern a stale read would show)."""
    case = make_case(2048, 3072, seed=9)
    y_ref = None
    for it in range(20):
        buf = torch.full((B.layout_bytes(B.PLANES, case.rows, case.nb * 24),), 0x88, dtype=torch.uint8, device="cuda")
        B.expand(ctx, B.PLANES, case.d_codes, case.rows, case.nb, out=buf)
        y = B.gemv(ctx, B.PLANES, buf, case.d_scale, GAIN, case.d_x, case.rows, case.nb * 24)
        if y_ref is None:
            check_gemv(oracle, case, y)
            y_ref = y.clone()
        assert torch.equal(y, y_ref), it
    B.status(ctx)


def test_gain_range(B, ctx):
    case = make_case(64, 96, seed=11)
    buf = B.expand(ctx, B.PLANES, case.d_codes, case.rows, case.nb)
    for gain in ((1e-30, 1e-31), (3e18, 1.0), (float("inf"), 1.0)):
        with pytest.raises(B.LlvqError) as e:
            B.gemv(ctx, B.PLANES, buf, case.d_scale, gain, case.d_x, case.rows, 96)
        assert e.value.code == -1
    y = B.gemv(ctx, B.PLANES, buf, case.d_scale, (0.0, 0.0), case.d_x, case.rows, 96)
    assert (y == 0).all()
    y = B.gemv(ctx, B.PLANES, buf, case.d_scale, (2.0 ** -59, 2.0 ** -59), case.d_x, case.rows, 96)
    assert torch.isfinite(y).all()
    y1 = B.gemv(ctx, B.PLANES, buf, case.d_scale, (1.0, 1.0), case.d_x, case.rows, 96)
    assert torch.allclose(y.double() * 2.0 ** 59, y1.double(), rtol=1e-6, atol=0)
