"""Full-size parity (needs a B200): the 8192 x 8192 sweep matrix in full, and the 8B- and 14B-like
stacks in the launch configuration the bench times, checked on sampled rows and row groups."""
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


def test_config4_in_full(B, ctx, oracle):
    case = make_case(8192, 8192, seed=4)
    for layout in (B.PLANES, B.ONEHOT):
        buf = B.expand(ctx, layout, case.d_codes, case.rows, case.nb)
        expect = oracle.pack_planes(case.codes, case.rows, case.nb) if layout == B.PLANES else oracle.pack_onehot(case.codes, case.rows, case.nb)
        assert np.array_equal(buf.cpu().numpy(), expect)
        y = B.gemv(ctx, layout, buf, case.d_scale, GAIN, case.d_x, case.rows, case.nb * 24)
        B.status(ctx)
        check_gemv(oracle, case, y, nthreads=16)
        del buf


def test_config1_in_full(B, ctx, oracle):
    """The 4B-like layer in full: every record of its seven matrices byte for byte against the oracle, and every
    row of the row-concatenated launches the bench times against the f64 matvec."""
    from paper_2609_02652_b200 import datagen

    wl = datagen.workload(1)
    groups = {}
    for m in wl.matrices:
        groups.setdefault(m.group, []).append(m)
    for members in groups.values():
        probs, keep = [], []
        for m in members:
            case = make_case(m.rows, m.k, seed=wl.seed, tensor_id=m.tensor_id)
            buf = B.expand(ctx, B.PLANES, case.d_codes, m.rows, m.nb)
            assert np.array_equal(buf.cpu().numpy(), oracle.pack_planes(case.codes, m.rows, m.nb)), m.name
            y = torch.full((m.rows,), float("nan"), dtype=torch.float32, device="cuda")
            probs.append((buf, case.d_scale, GAIN, y, m.rows))
            keep.append((m, case, y))
        # members of a group share x (the first member's)
        x = keep[0][1]
        B.gemv_grouped(ctx, B.PLANES, probs, x.d_x, members[0].k_padded)
        B.status(ctx)
        for m, case, y in keep:
            case.x = x.x
            check_gemv(oracle, case, y, nthreads=16)


def test_config1_in_full_in_the_10_byte_layout(B, ctx, oracle):
    """The same layer in the 10-byte layout with its exception table, as the bench's arm runs it: buffers sized from the
    count call, every byte (short records, index, table) against the oracle, every row of the grouped launches."""
    from paper_2609_02652_b200 import datagen

    wl = datagen.workload(1)
    groups = {}
    for m in wl.matrices:
        groups.setdefault(m.group, []).append(m)
    exceptions = 0
    for members in groups.values():
        probs, keep = [], []
        for m in members:
            case = make_case(m.rows, m.k, seed=wl.seed, tensor_id=m.tensor_id)
            n = B.overlay_count(ctx, case.d_codes, m.rows, m.nb)
            buf = B.expand(ctx, B.PLANES10X, case.d_codes, m.rows, m.nb,
                           out=torch.empty(B.overlay_bytes(m.rows, m.k_padded, n), dtype=torch.uint8, device="cuda"))
            want, n_ref = oracle.pack_planes10x(case.codes, m.rows, m.nb)
            assert n == n_ref and np.array_equal(buf.cpu().numpy(), want), m.name
            exceptions += n
            y = torch.full((m.rows,), float("nan"), dtype=torch.float32, device="cuda")
            probs.append((buf, case.d_scale, GAIN, y, m.rows))
            keep.append((m, case, y))
        x = keep[0][1]
        B.gemv_grouped(ctx, B.PLANES10X, probs, x.d_x, members[0].k_padded)
        B.status(ctx)
        for m, case, y in keep:
            case.x = x.x
            check_gemv(oracle, case, y, nthreads=16)
    assert 100 < exceptions < 2000          # about one block in eight thousand of the 4.2 million


@pytest.mark.parametrize("config,layers", [(2, (0, 17, 35)), (3, (0, 39))])
def test_stacks_sampled(B, ctx, oracle, config, layers):
    """Every matrix of the sampled layers runs as the bench runs it (row-concatenated groups); 96 rows
    and two row groups of every matrix are checked against the oracle, the rest must be finite."""
    from paper_2609_02652_b200 import datagen

    wl = datagen.workload(config)
    rng = np.random.default_rng(config)
    per_layer = 7
    for layer in layers:
        mats = wl.matrices[layer * per_layer:(layer + 1) * per_layer]
        groups = {}
        for m in mats:
            groups.setdefault(m.group, []).append(m)
        for members in groups.values():
            x = datagen.make_x(members[0].k, members[0].k_padded, wl.seed, members[0].tensor_id)
            dx = x.cuda()
            probs, keep = [], []
            for m in members:
                codes = datagen.make_codes(m.rows, m.nb, wl.seed, m.tensor_id, device="cuda")
                scale = datagen.make_row_scale(m.rows, wl.seed, m.tensor_id)
                buf = B.expand(ctx, B.PLANES, codes, m.rows, m.nb)
                y = torch.full((m.rows,), float("nan"), dtype=torch.float32, device="cuda")
                probs.append((buf, scale.cuda(), GAIN, y, m.rows))
                keep.append((m, codes, scale, buf, y))
            B.gemv_grouped(ctx, B.PLANES, probs, dx, members[0].k_padded)
            B.status(ctx)
            for m, codes, scale, buf, y in keep:
                yv = y.cpu().numpy().astype(np.float64)
                assert np.isfinite(yv).all()
                rows = np.sort(rng.choice(m.rows, size=96, replace=False))
                sub = codes.view(m.rows, m.nb)[torch.from_numpy(rows).cuda()].cpu().numpy().astype(np.uint64)
                y_ref, wn, ab = oracle.matvec(sub, len(rows), m.nb, scale.numpy()[rows], GAIN, x.numpy(), nthreads=8)
                den = wn * float(np.linalg.norm(x.numpy().astype(np.float64)))
                err = np.abs(yv[rows] - y_ref)
                assert (err <= 1e-4 * den).all() and (err <= 1e-5 * ab + 1e-30).all(), m.name
                # two whole row groups of the layout, byte for byte
                for rg in (0, int(rng.integers(m.rows // 32))):
                    sub = codes.view(m.rows, m.nb)[rg * 32:(rg + 1) * 32].cpu().numpy().astype(np.uint64)
                    expect = oracle.pack_planes(sub, 32, m.nb)
                    got = buf[rg * m.nb * 448:(rg + 1) * m.nb * 448].cpu().numpy()
                    assert np.array_equal(got, expect), (m.name, rg)
            del keep, probs
            torch.cuda.empty_cache()
