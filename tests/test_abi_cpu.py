"""The C ABI without a GPU: the library loads, exports what include/llvq.h declares, and the
host-only entry points validate their arguments."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_02652_b200 import binding, build

    build.build()
    return binding.load()


def _declared():
    text = open(os.path.join(ROOT, "include", "llvq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(llvq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2609_02652_b200 import binding

    names = _declared()
    assert len(names) >= 13
    for n in names:
        assert hasattr(lib, n), n
    assert set(binding.SYMBOLS) <= set(names)


def test_layout_bytes_and_argument_checks(lib):
    from paper_2609_02652_b200 import binding

    assert binding.layout_bytes(binding.PLANES, 3072, 3072) == 3072 * 128 * 14
    assert binding.layout_bytes(binding.PLANES, 33, 48) == 2 * 2 * 448
    assert binding.layout_bytes(binding.ONEHOT, 8192, 8208) == 8192 * 342 * 20
    n = ctypes.c_size_t()
    assert lib.llvq_layout_bytes(5, 32, 24, ctypes.byref(n)) == -1
    assert lib.llvq_layout_bytes(0, 32, 25, ctypes.byref(n)) == -1
    assert lib.llvq_layout_bytes(0, 0, 24, ctypes.byref(n)) == -1
    assert lib.llvq_gemv_fp16(None, None, None, 8, 8, None) == -1
    assert lib.llvq_gemv(None, 0, None, None, None, None, None, 1, 24, None) == -1
    assert b"aligned" in lib.llvq_strerror(-2)
    # the code for an expanded code word that names no point is declared and named
    assert "#define LLVQ_EINDEX (-6)" in open(os.path.join(ROOT, "include", "llvq.h")).read()
    assert b"no point" in lib.llvq_strerror(-6)
    # the 13-byte layout: 13/14 of the 14-byte layout's size, for any shape
    assert binding.layout_bytes(binding.PLANES13, 3072, 3072) == 3072 * 128 * 13
    assert binding.layout_bytes(binding.PLANES13, 33, 48) == 2 * 2 * 416
    assert lib.llvq_layout_bytes(4, 32, 24, ctypes.byref(n)) == -1
    # the 10-byte layout: tiles of 1280 bytes, leftover blocks of 416, then (128-byte aligned) the index and the table
    from oracle import oracle as O
    for rows, nb, exc in ((32, 4, 0), (33, 7, 5), (3072, 128, 100), (70, 1, 0), (64, 9, 3)):
        assert binding.overlay_bytes(rows, 24 * nb, exc) == O.planes10x_bytes(rows, nb, exc)
        assert binding.layout_bytes(binding.PLANES10X, rows, 24 * nb) == O.planes10x_bytes(rows, nb, (rows * nb + 31) // 32)
    assert binding.overlay_bytes(32, 96, 0) == 1280 + 128
    assert lib.llvq_overlay_bytes(32, 24 << 19, 0, ctypes.byref(n)) == -1          # block columns must stay below 2^19
    assert lib.llvq_overlay_count(None, None, 1, 1, None, None) == -1


def test_rotation_block_rule_and_argument_checks(lib):
    """The host query of the rotation, against the oracle's rule (largest power of two dividing n, at most 16384)."""
    from oracle import oracle as O
    from paper_2609_02652_b200 import binding

    for n in (8, 24, 2560, 4096, 5120, 9728, 12288, 17408, 25600, 98304, 7, 1, 3 * 16384, 5 * 32768):
        assert binding.rotate_block(n) == O.rotate_block(n), n
        for b in (1, 2, 8, 64, 512, 4096, 16384, 32768, 3, 0):
            assert binding.rotate_block(n, b) == O.rotate_block(n, b), (n, b)
    assert binding.rotate_block(0) == 0 and binding.rotate_block(-8) == 0
    assert lib.llvq_rotate(None, None, None, None, 8, 0, None) == -1
    assert lib.llvq_gemv_rotated(None, None, 1, None, 24, None, None) == -1


def test_missing_library_fails_loudly(monkeypatch):
    from paper_2609_02652_b200 import binding

    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libllvq.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.load()


def _plan_invariants(plan, sm_count, rows, k_padded, batch, must_fit=True):
    nb = k_padded // 24
    tiles, left = divmod(nb, 4)
    units = tiles + (1 if left else 0)
    groups = sum((r + 31) // 32 for r in rows)
    total = groups * units
    assert plan["units"] == units and plan["groups"] == groups and plan["total_units"] == total
    grid = plan["grid"]
    assert 1 <= grid <= min(sm_count, 256) and grid <= max(total, 1)
    cf = plan["cta_first"]
    assert cf[0] == 0 and cf[-1] == total and all(a <= b for a, b in zip(cf, cf[1:]))
    # the first CTAs lead: shares never grow with the CTA index by more than the rounding, and stay within
    # ten units (or 60 % of the mean) of the mean
    shares = [b - a for a, b in zip(cf, cf[1:])]
    mean = total / grid
    lead = min(10.0, 0.6 * mean)
    assert all(abs(s - mean) <= lead + 1.5 for s in shares[:-1])
    assert all(shares[i + 1] <= shares[i] + 1 for i in range(len(shares) - 2))
    # panels tile the unit columns; the x blocks a CTA prepares are those of the panels its units lie in
    P, npan = plan["panel"], plan["npanels"]
    assert P >= 1 and (npan - 1) * P < units <= npan * P
    def panel_of(f):
        return min(f // (groups * P), npan - 1)
    need = 0
    for a, b in zip(cf, cf[1:]):
        lo = panel_of(a) * P * 4
        hi = min(nb, (panel_of(max(b - 1, a)) + 1) * P * 4)
        need = max(need, hi - lo)
        # every unit of the CTA lies in those panels
        for f in (a, max(b - 1, a)):
            j = panel_of(f)
            assert lo <= j * P * 4 and min(nb, (j + 1) * P * 4) <= hi
    assert plan["xblocks"] == need <= nb
    vectors = 1 if batch == 1 else (2 if batch == 2 else 4)
    assert plan["smem"] >= 16 * 2 * 1792 + len(rows) * 8192 + vectors * need * 112
    # the query has no device to ask: a plan beyond a multiprocessor's shared memory is what makes the launch
    # itself return LLVQ_ESIZE (few multiprocessors and a very long row: one CTA then needs most of x)
    fits = plan["smem"] + 1024 <= 227 * 1024
    assert fits or not must_fit
    return fits


def test_launch_plan_invariants():
    """The host-side planner of the GEMV (no GPU): CTA shares, panels, shared-memory need."""
    from paper_2609_02652_b200 import binding

    cases = [(148, [8192], 8208, 1), (148, [4096, 1024, 1024], 2568, 1), (148, [9728, 9728], 2568, 1), (148, [2560], 9744, 1),
             (148, [1], 24, 1), (148, [33], 48, 1), (148, [70], 24 * 1024, 1), (148, [40], 98304, 1), (148, [24576], 4104, 4),
             (132, [5120], 17424, 2), (300, [100000], 4104, 1), (8, [3072], 3072, 1), (148, [32 + 17 * i for i in range(8)], 960, 1)]
    for sm, rows, k, batch in cases:
        _plan_invariants(binding.gemv_plan(sm, rows, k, batch), sm, rows, k, batch)
    # argument checks
    with pytest.raises(binding.LlvqError):
        binding.gemv_plan(148, [8192], 8209)
    with pytest.raises(binding.LlvqError):
        binding.gemv_plan(148, [8192], 98304 + 24)
    with pytest.raises(binding.LlvqError):
        binding.gemv_plan(148, [8192] * 9, 8208)
    with pytest.raises(binding.LlvqError):
        binding.gemv_plan(148, [8192], 8208, batch=5)


def test_launch_plan_invariants_random_shapes():
    """The same invariants over a few hundred seeded random launches: grids of 1..320 multiprocessors, one to eight
    matrices of 1..60 000 rows, 1..4096 blocks a row, 1 / 2 / 4 vectors."""
    import numpy as np

    from paper_2609_02652_b200 import binding

    rng = np.random.default_rng(31)
    checked = 0
    for it in range(300):
        sm = int(rng.choice([1, 8, 72, 108, 132, 148, 160, 256, 320]))
        nmat = int(rng.integers(1, 9))
        rows = [int(rng.integers(1, 60_000 if it % 4 == 0 else 3_000)) for _ in range(nmat)]
        nb = int(rng.integers(1, 4097 if it % 7 == 0 else 600))
        batch = int(rng.choice([1, 1, 2, 4])) if nmat == 1 else 1
        try:
            plan = binding.gemv_plan(sm, rows, 24 * nb, batch)
        except binding.LlvqError as e:
            assert e.code == -3                                   # the accepted sizes are bounded; nothing else may fail
            continue
        fits = _plan_invariants(plan, sm, rows, 24 * nb, batch, must_fit=False)
        # on a full-size part every accepted row length fits when the launch has work for the whole grid
        groups = sum((r + 31) // 32 for r in rows)
        if sm >= 132 and groups * ((nb + 3) // 4) >= 4 * sm and len(rows) <= 3:
            assert fits, (sm, rows, nb, batch, plan["smem"])
        checked += 1
    assert checked >= 250
