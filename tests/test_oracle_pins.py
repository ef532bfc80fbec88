"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

Nothing here re-calls the oracle's own formulas: the Golay code, the lattice membership test,
the theta series and the layout unpackers below are written separately in Python.
"""
import itertools
import math

import numpy as np
import pytest

N_PAPER = 111_043_117_458_000           # Sec. 2.1
N13_PAPER = 280_974_212_784_720         # Sec. 2.4, "Invariant locks upstream"
KISSING = 196_560                       # Sec. 2.4


def _golden(name):
    import os

    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", name)


def paper_constants():
    out = {}
    for line in open(_golden("paper_constants.txt")):
        if line.strip() and not line.startswith("#"):
            name, value, _cite = line.rstrip("\n").split("\t")
            out[name] = int(value)
    return out


# ---------------------------------------------------------------- independent ingredients
def golay_set():
    """All multiples of g(x) = x^11+x^10+x^6+x^5+x^4+x^2+1 of degree < 23, plus a parity bit."""
    g = (1 << 11) | (1 << 10) | (1 << 6) | (1 << 5) | (1 << 4) | (1 << 2) | 1
    words = set()
    for m in range(4096):
        w = 0
        for i in range(12):
            if (m >> i) & 1:
                w ^= g << i          # carry-less product m(x) g(x)
        if bin(w).count("1") & 1:
            w |= 1 << 23
        words.add(w)
    return words


GOLAY = golay_set()


def is_leech_point(x) -> bool:
    """Sec. 2.1's three conditions in sqrt(8) Lambda24: parity, Golay word on a residue class mod 4, sum mod 8."""
    x = [int(v) for v in x]
    par = x[0] % 2
    if any(v % 2 != par for v in x):
        return False
    word = 0
    for i, v in enumerate(x):
        if ((v - par) // 2) % 2:
            word |= 1 << i
    return word in GOLAY and sum(x) % 8 == (4 * par) % 8


def tau(nmax):
    poly = [1] + [0] * nmax
    for n in range(1, nmax + 1):
        for _ in range(24):
            for k in range(nmax, n - 1, -1):
                poly[k] -= poly[k - n]
    return [0] + poly[:nmax]


def theta(m, t):
    s11 = sum(d**11 for d in range(1, m + 1) if m % d == 0)
    v, r = divmod(65520 * (s11 - t[m]), 691)
    assert r == 0
    return v


# ---------------------------------------------------------------- Golay code
def test_golay_weight_enumerator_and_duality(oracle):
    words = oracle.golay_words()
    assert len(set(words.tolist())) == 4096
    assert set(words.tolist()) == GOLAY
    hist = np.bincount([bin(int(w)).count("1") for w in words], minlength=25)
    assert {int(k): int(v) for k, v in enumerate(hist) if v} == {0: 1, 8: 759, 12: 2576, 16: 759, 24: 1}
    rows = [int(words[1 << i]) for i in range(12)]
    for a, b in itertools.product(rows, rows):
        assert bin(a & b).count("1") % 2 == 0          # self-dual
    # cyclic on the first 23 coordinates: g(x) divides x^23 - 1
    for w in rows:
        lo = w & ((1 << 23) - 1)
        rot = ((lo << 1) | (lo >> 22)) & ((1 << 23) - 1)
        assert (rot | (w & (1 << 23))) in GOLAY


# ---------------------------------------------------------------- classes
def test_class_count_and_totals(oracle):
    assert oracle.num_classes() == 301                 # Sec. 2.1
    assert oracle.total_points() == N_PAPER
    assert math.ceil(math.log2(N_PAPER)) == 47
    t = tau(13)
    assert t[1:8] == [1, -24, 252, -1472, 4830, -6048, -16744]   # textbook values of Ramanujan's tau
    assert theta(2, t) == KISSING
    for m in range(2, 13):
        assert oracle.shell_count(m) == theta(m, t), m
    infos = [oracle.class_info(c) for c in range(301)]
    assert sum(i["size"] for i in infos) == N_PAPER
    assert all(1 <= i["ndist"] <= 5 for i in infos)    # Sec. 2.3: at most five values a class
    assert sum(1 for i in infos if i["odd"]) == 121
    base = 0
    for i in infos:                                    # contiguous, in order
        assert i["base"] == base
        base += i["size"]
    keys = [(i["shell"], i["odd"], i["w"], tuple(i["mags"])) for i in infos]
    assert keys == sorted(keys) and len(set(keys)) == 301


def test_against_the_values_the_paper_prints(oracle):
    c = paper_constants()
    assert oracle.total_points() == c["ball_points"] == N_PAPER
    assert math.ceil(math.log2(c["ball_points"])) == c["index_bits"]
    assert oracle.num_classes() == c["classes"]
    infos = [oracle.class_info(k) for k in range(oracle.num_classes())]
    assert len({i["shell"] for i in infos}) == c["shells"]
    assert oracle.shell_count(2) == c["kissing_number"] == KISSING
    assert max(i["ndist"] for i in infos) == c["max_levels_per_class"]
    assert 9 + 1 + 24 + 3 * 24 == c["planes_payload_bits"] and c["planes_payload_bits"] <= 8 * c["planes_record_bytes"]
    assert oracle.planes_bytes(32, 1) == 32 * c["planes_record_bytes"]
    assert oracle.num_classes() <= c["class_table_slots"] and oracle.SENTINEL_CLASS < c["class_table_slots"]
    try:
        oracle.init_shells(13)
        assert oracle.total_points() == c["points_through_shell_13"] == N13_PAPER
    finally:
        oracle.init_shells(12)


def test_stored_index_examples_still_decode_the_same(oracle):
    """Regression pin of the index order (the reading of Sec. 2.1): examples written by the oracle itself,
    each also a lattice point of its class's shell and a fixed point of encode."""
    n = 0
    for line in open(_golden("index_examples.txt")):
        if line.startswith("#"):
            continue
        idx, cls, coords = line.rstrip("\n").split("\t")
        x = np.array([int(v) for v in coords.split()], dtype=np.int8)
        c, got = oracle.decode(int(idx))
        assert c == int(cls) and got.tolist() == x.tolist()
        assert is_leech_point(x) and oracle.encode(x) == int(idx)
        assert int((x.astype(int) ** 2).sum()) == 16 * oracle.class_info(c)["shell"]
        n += 1
    assert n >= 16


def test_count_through_shell_13(oracle):
    try:
        assert oracle.init_shells(13) == 383
        assert oracle.total_points() == N13_PAPER      # Sec. 2.4
        assert oracle.shell_count(13) == theta(13, tau(13))
    finally:
        oracle.init_shells(12)
    assert oracle.num_classes() == 301


def test_shell2_classes_by_hand(oracle):
    # the 196 560 minimal vectors: (+-4^2, 0^22), (+-2^8, 0^16), (-+3, +-1^23)
    sizes = [oracle.class_info(c)["size"] for c in range(3)]
    assert sizes == [1104, 97152, 98304]


# ---------------------------------------------------------------- decoder
def _sample_indices(oracle, per_shell=300, seed=7):
    rng = np.random.default_rng(seed)
    out = []
    for c in range(301):
        i = oracle.class_info(c)
        out += [i["base"], i["base"] + i["size"] - 1]
        out += (i["base"] + rng.integers(0, i["size"], size=6)).tolist()
    out += rng.integers(0, N_PAPER, size=per_shell * 11).tolist()
    return np.array(out, dtype=np.uint64)


def test_decoded_points_are_lattice_points_of_the_right_shell(oracle):
    idx = _sample_indices(oracle)
    xs, cls = oracle.decode_batch(idx)
    assert (cls >= 0).all()
    for i, x, c in zip(idx.tolist(), xs, cls.tolist()):
        info = oracle.class_info(c)
        assert info["base"] <= i < info["base"] + info["size"]
        assert is_leech_point(x), (i, x)
        assert int((x.astype(int) ** 2).sum()) == 16 * info["shell"]
        mags = np.abs(x.astype(int))
        if info["odd"]:
            assert sorted(mags.tolist()) == info["mags"]
        else:
            assert sorted(mags.tolist()) == sorted(info["mags"])
    # lattice closure and integrality of the scaled inner product
    X = xs.astype(np.int64)
    rng = np.random.default_rng(3)
    for _ in range(2000):
        a, b = X[rng.integers(len(X))], X[rng.integers(len(X))]
        assert int(a @ b) % 8 == 0 and int(a @ a) % 16 == 0
        assert is_leech_point(a + b) and is_leech_point(a - b)


def test_round_trip_encode_decode(oracle):
    idx = _sample_indices(oracle, per_shell=1000, seed=11)
    xs, _ = oracle.decode_batch(idx)
    for i, x in zip(idx.tolist(), xs):
        assert oracle.encode(x) == i
    assert oracle.decode(N_PAPER)[0] == -1
    assert oracle.decode((1 << 47) - 1)[0] == -1
    assert oracle.encode(np.zeros(24, np.int8)) == -1
    bad = np.array([4, 4] + [0] * 22, np.int8)
    bad[0] = 2
    assert oracle.encode(bad) == -1


def test_shell2_is_enumerated_exactly_once(oracle):
    xs, cls = oracle.decode_batch(np.arange(KISSING, dtype=np.uint64))
    assert set(cls.tolist()) == {0, 1, 2}
    packed = np.ascontiguousarray(xs).view([("a", "u8"), ("b", "u8"), ("c", "u8")]).ravel()
    assert np.unique(packed).size == KISSING           # injective, and 196 560 is the whole shell
    assert ((xs.astype(int) ** 2).sum(1) == 32).all()
    assert all(is_leech_point(x) for x in xs[::97])


def test_shell3_is_enumerated_exactly_once(oracle):
    """All 16 773 120 indices of the second non-empty shell decode to distinct points of norm 48: the decode is
    injective there, and since the count is the theta coefficient it is onto as well."""
    lo, hi = KISSING, 16_969_680
    parts = []
    for a in range(lo, hi, 1 << 21):
        b = min(a + (1 << 21), hi)
        xs, _ = oracle.decode_batch(np.arange(a, b, dtype=np.uint64))
        assert ((xs.astype(np.int32) ** 2).sum(1) == 48).all()
        parts.append(np.ascontiguousarray(xs).view([("a", "u8"), ("b", "u8"), ("c", "u8")]).ravel().copy())
    packed = np.concatenate(parts)
    del parts
    assert packed.size == hi - lo == 16_773_120
    assert np.unique(packed).size == hi - lo


def test_worked_values_of_the_index_order(oracle):
    """Index -> (class, point) for indices spread over the ball, worked out independently of this oracle (a separate
    program written from the same readings before the oracle existed: class order = shell, even before odd, codeword
    weight, magnitude tuples; order inside a class = codeword rank, arrangement ranks, sign bits, the last support
    sign repairing the sum; odd classes = arrangement rank * 4096 + message bits).  A change to any of those readings
    moves these points."""
    expect = {
        196_559: (2, [3, -1, 1, 1, -1, 1, -1, -1, -1, -1, 1, -1, 1, 1, -1, -1, 1, -1, 1, 1, 1, 1, -1, 1]),
        196_560: (3, [2, 2, 2, 2, 2, 0, 0, 2, 0, 0, 2, 0, -2] + [0] * 10 + [4]),
        16_969_680: (7, [0] * 23 + [8]),
        40_556_880_458_640: (222, [0] * 21 + [8, 8, 8]),
        12_345_678_901_234: (163, [5, -1, 1, -5, 5, 1, 1, -3, -1, 3, -1, 1, 3, -1, -1, 3, 1, -3, 1, -3, 3, -3, -1, -1]),
        N_PAPER - 1: (300, [3, 3, -3, -3, 3, -3, 3, 3, 3, 3, -3, 3, -3, -3, 3, 3, -3, 3, -3, -3, -3, 1, -1, 1]),
    }
    for idx, (cls, x) in expect.items():
        c, got = oracle.decode(idx)
        assert c == cls and got.tolist() == x, idx
        assert oracle.encode(np.array(x, dtype=np.int8)) == idx


def test_worked_examples_derived_by_hand(oracle):
    """First and last points of the first classes, worked out from the stated order by hand."""
    # class 0: off-support multiset {0^22, 4, 4}; rank 0 puts the zeros first; sign bit 0 is the
    # first non-zero coordinate
    assert oracle.decode(0)[1].tolist() == [0] * 22 + [4, 4]
    assert oracle.decode(1)[1].tolist() == [0] * 22 + [-4, 4]
    assert oracle.decode(1103)[1].tolist() == [-4, -4] + [0] * 22       # 276 * 4 - 1
    # class 1 starts with the smallest weight-8 word; its support all +2 sums to 16 = 0 mod 8
    c, x = oracle.decode(1104)
    assert c == 1 and sorted(np.flatnonzero(x).tolist()) == [i for i in range(24) if (min(w for w in GOLAY if bin(w).count("1") == 8) >> i) & 1]
    assert (x[np.flatnonzero(x)] == 2).all()
    # next index flips the first support coordinate; the last one repairs the sum
    x2 = oracle.decode(1105)[1]
    sup = np.flatnonzero(x).tolist()
    assert x2[sup[0]] == -2 and x2[sup[-1]] == -2 and (x2[sup[1:-1]] == 2).all()
    # class 2, zero codeword: every coordinate is 1 mod 4, so the 3 comes out negative
    assert oracle.decode(1104 + 97152)[1].tolist() == [1] * 23 + [-3]
    # first point of shell 4 and of shell 12
    assert oracle.decode(16_969_680)[1].tolist() == [0] * 23 + [8]
    assert oracle.decode(40_556_880_458_640)[1].tolist() == [0] * 21 + [8, 8, 8]


# ---------------------------------------------------------------- records and layouts
def _unpack_planes_cell(buf, nb, row, b):
    """Reader of the 14-byte layout written from its description, in the direction opposite to the packer's:
    from (row, block, coordinate) to the byte and nibble that hold its code."""
    rg, r = divmod(row, 32)
    m, e, g = r // 16, (r // 8) % 2, r % 8
    grp = rg * nb * 448
    ntiles, left = divmod(nb, 4)

    def word(off):
        return int.from_bytes(buf[off: off + 4].tobytes(), "little")

    j = b - 4 * ntiles
    if j < 0:                                   # inside a tile
        base = grp + (b // 4) * 1792
        slot, h = b % 2, 2 * ((b % 4) // 2) + m
        addr = lambda q, lane: base + 512 * ((3 * h + q) >> 2) + 16 * lane + 4 * ((3 * h + q) & 3)
        hdr_word = word(base + 1536 + 16 * (2 * g + slot) + 4 * h)
    elif left >= 2 and j < 2:                   # the pair after the tiles
        base = grp + ntiles * 1792
        slot = j
        addr = lambda q, lane: base + 128 * (3 * m + q) + 4 * lane
        hdr_word = word(base + 768 + 8 * (2 * g + slot) + 4 * m)
    else:                                       # the single at the very end: the slot is the row half
        base = grp + ntiles * 1792 + (896 if left == 3 else 0)
        slot = m
        addr = lambda q, lane: base + 128 * q + 4 * lane
        hdr_word = word(base + 384 + 4 * (2 * g + slot))
    hdr = (hdr_word >> (16 * e)) & 0xFFFF
    cls, gain = hdr & 511, (hdr >> 9) & 1
    assert hdr >> 10 == 0
    codes = []
    for i in range(24):
        kappa = 24 * slot + i
        if kappa < 32:
            c, t, ii = kappa // 16, (kappa % 16) // 4, kappa % 4
            w = word(addr(e, 4 * g + t))        # Wa for e = 0, Wb for e = 1
        else:
            c, t, ii = e, (kappa - 32) // 4, (kappa - 32) % 4
            w = word(addr(2, 4 * g + t))        # Wc: the nibble column picks the row
        codes.append((w >> (4 * (2 * ii + c))) & 15)
    return cls, gain, codes


def _codes(oracle, rows, nb, seed):
    from paper_2609_02652_b200 import datagen

    return datagen.make_codes(rows, nb, seed).numpy().astype(np.uint64)


@pytest.mark.parametrize("rows,nb", [(32, 4), (40, 7), (3, 1), (64, 9), (33, 2), (20, 6), (50, 3)])
def test_planes_layout_round_trip(oracle, rows, nb):
    codes = _codes(oracle, rows, nb, seed=5)
    codes[0] = N_PAPER                       # a code that names no point
    buf = oracle.pack_planes(codes, rows, nb)
    assert buf.size == ((rows + 31) // 32) * nb * 448
    xs, cls = oracle.decode_batch(codes)
    for row in range(((rows + 31) // 32) * 32):
        for b in range(nb):
            c, g, u = _unpack_planes_cell(buf, nb, row, b)
            if row >= rows or cls[row * nb + b] < 0:
                assert c == 511 and g == 0 and u == [8] * 24
                continue
            code = int(codes[row * nb + b])
            assert c == cls[row * nb + b] and g == code >> 47
            par = oracle.class_info(c)["odd"]
            assert [2 * (v - 8) + par for v in u] == xs[row * nb + b].tolist()
            # the same 106 bits as the record's sign mask and level planes
            rec = oracle.record(code)
            for i, v in enumerate(u):
                level = sum(((rec["planes"][t] >> i) & 1) << t for t in range(3))
                assert v == (8 - level - par if (rec["smask"] >> i) & 1 else 8 + level)


def _unpack_planes13_cell(buf, nb, row, b):
    """Reader of the 13-byte layout from its description: (row, block) -> header byte fields and the 24 codes."""
    rg, r = divmod(row, 32)
    m, e, g = r // 16, (r // 8) % 2, r % 8
    grp = rg * nb * 416
    ntiles, left = divmod(nb, 4)

    def word(off):
        return int.from_bytes(buf[off: off + 4].tobytes(), "little")

    j = b - 4 * ntiles
    if j < 0:
        base = grp + (b // 4) * 1664
        slot, h = b % 2, 2 * ((b % 4) // 2) + m
        addr = lambda q, lane: base + 512 * ((3 * h + q) >> 2) + 16 * lane + 4 * ((3 * h + q) & 3)
        hb = int(buf[base + 1536 + 8 * (2 * g + slot) + 2 * h + e])
    elif left >= 2 and j < 2:
        base = grp + ntiles * 1664
        slot = j
        addr = lambda q, lane: base + 128 * (3 * m + q) + 4 * lane
        hb = int(buf[base + 768 + 4 * (2 * g + slot) + 2 * m + e])
    else:
        base = grp + ntiles * 1664 + (832 if left == 3 else 0)
        slot = m
        addr = lambda q, lane: base + 128 * q + 4 * lane
        hb = int(buf[base + 384 + 2 * (2 * g + slot) + e])
    assert hb >> 6 == 0
    codes = []
    for i in range(24):
        kappa = 24 * slot + i
        if kappa < 32:
            c, t, ii = kappa // 16, (kappa % 16) // 4, kappa % 4
            w = word(addr(e, 4 * g + t))
        else:
            c, t, ii = e, (kappa - 32) // 4, (kappa - 32) % 4
            w = word(addr(2, 4 * g + t))
        codes.append((w >> (4 * (2 * ii + c))) & 15)
    return hb & 15, (hb >> 4) & 1, (hb >> 5) & 1, codes


@pytest.mark.parametrize("rows,nb", [(32, 4), (37, 7), (64, 1), (5, 2), (33, 3), (20, 6), (50, 9)])
def test_planes13_layout_round_trip(oracle, rows, nb):
    """The 13-byte layout holds, for every block, the shell, the parity and the gain bit in its header byte and the
    same 24 codes as the 14-byte layout: enough to rebuild the block's weights exactly."""
    codes = _codes(oracle, rows, nb, seed=8)
    buf = oracle.pack_planes13(codes, rows, nb)
    assert buf.size == ((rows + 31) // 32) * nb * 416 == oracle.planes13_bytes(rows, nb)
    xs, cls = oracle.decode_batch(codes)
    seen = np.zeros(buf.size, bool)
    for row in range(((rows + 31) // 32) * 32):
        for b in range(nb):
            shell, par, gain, u = _unpack_planes13_cell(buf, nb, row, b)
            if row >= rows or cls[row * nb + b] < 0:
                assert (shell, par, gain) == (0, 0, 0) and u == [8] * 24
                continue
            x = xs[row * nb + b]
            assert shell == int((x.astype(np.int64) ** 2).sum()) // 16 and par == int(x[0]) & 1
            assert gain == int(codes[row * nb + b]) >> 47
            assert [2 * (v - 8) + par for v in u] == x.tolist()
            assert _unpack_planes_cell(oracle.pack_planes(codes, rows, nb), nb, row, b)[2] == u
    # 13 bytes a block: 12 of codes, one header byte (4.33 bits a weight)
    assert buf.size * 8 / (((rows + 31) // 32) * 32 * nb * 24) == pytest.approx(13 * 8 / 24)


def test_planes13_layout_worked_example_by_hand(oracle):
    """One row, one block, index 0 = (0^22, 4, 4) in shell 2, even: codes 8 except the last two (10); the single's
    header bytes sit at 384 + 2 P + e, and row 0 is (g, e, half) = (0, 0, 0): byte 384 = shell 2, no parity, no gain."""
    buf = oracle.pack_planes13(np.array([0], np.uint64), 1, 1)
    assert buf.size == 416
    words = buf[:384].view(np.uint32)
    assert int(words[1]) == 0xA8A88888                        # as in the 14-byte layout: the same code words
    assert [int(w) for i, w in enumerate(words) if i != 1] == [0x88888888] * 95
    assert int(buf[384]) == 2 and not buf[385:].any()
    buf = oracle.pack_planes13(np.array([1 << 47], np.uint64), 1, 1)
    assert int(buf[384]) == 2 | (1 << 5)


def _p10_offsets(rows, nb):
    groups = (rows + 31) // 32
    gbytes = (nb // 4) * 1280 + (nb % 4) * 416
    idx = -(-groups * gbytes // 128) * 128
    return groups, gbytes, idx, idx + -(-(groups * (nb // 4) + 1) * 4 // 128) * 128


def _unpack_planes10x_cell(buf, rows, nb, row, b):
    """Reader of the 10-byte layout's short record from its description: (row, block) -> header byte, window base
    (None for a block past the tiles, whose codes are four-bit) and the 24 stored codes."""
    rg, r = divmod(row, 32)
    m, e, g = r // 16, (r // 8) % 2, r % 8
    _, gbytes, _, _ = _p10_offsets(rows, nb)
    grp = rg * gbytes
    ntiles, left = divmod(nb, 4)

    def word(off):
        return int.from_bytes(buf[off: off + 4].tobytes(), "little")

    j = b - 4 * ntiles
    if j >= 0:                                   # pair or single, as in the 13-byte layout
        if left >= 2 and j < 2:
            base, slot = grp + ntiles * 1280, j
            addr = lambda q, lane: base + 128 * (3 * m + q) + 4 * lane
            hb = int(buf[base + 768 + 4 * (2 * g + slot) + 2 * m + e])
        else:
            base, slot = grp + ntiles * 1280 + (832 if left == 3 else 0), m
            addr = lambda q, lane: base + 128 * q + 4 * lane
            hb = int(buf[base + 384 + 2 * (2 * g + slot) + e])
        codes = []
        for i in range(24):
            kappa = 24 * slot + i
            if kappa < 32:
                c, t, ii = kappa // 16, (kappa % 16) // 4, kappa % 4
                w = word(addr(e, 4 * g + t))
            else:
                c, t, ii = e, (kappa - 32) // 4, (kappa - 32) % 4
                w = word(addr(2, 4 * g + t))
            codes.append((w >> (4 * (2 * ii + c))) & 15)
        assert hb >> 6 == 0
        return hb, None, codes
    base = grp + (b // 4) * 1280
    slot, h = b % 2, 2 * ((b % 4) // 2) + m

    def V(k, lane):
        return word(base + (16 * lane + 4 * k if k < 4 else (512 + 16 * lane + 4 * (k - 4) if k < 8 else 1024 + 4 * lane)))

    left_over = [(0, 1), (1, 1), (2, 0), (2, 1), (3, 0), (3, 1)]       # the groups X0..X5 as (h, e)
    codes = []
    for i in range(24):
        kappa = 24 * slot + i
        if kappa < 32:
            c, t, ii = kappa // 16, (kappa % 16) // 4, kappa % 4
            codes.append((V(2 * h + e, 4 * g + t) >> (8 * ii + 3 * c)) & 7)
            continue
        t, ii = (kappa - 32) // 4, (kappa - 32) % 4
        lane = 4 * g + t
        if (h, e) == (0, 0):
            codes.append((V(8, lane) >> (8 * ii)) & 7)
        elif (h, e) == (1, 0):
            codes.append((V(8, lane) >> (8 * ii + 3)) & 7)
        else:
            k = left_over.index((h, e))
            low = (V(k, lane) >> (8 * ii + 6)) & 3
            high = (V(6 + (k >> 1), lane) >> (8 * ii + 6 + (k & 1))) & 1
            codes.append(low | high << 2)
    hb = int(buf[base + 1152 + 8 * (2 * g + slot) + 2 * h + e])
    return hb, 3 + ((hb ^ (hb >> 4)) & 3), codes


@pytest.mark.parametrize("rows,nb,rate", [(32, 4, 0.0), (37, 7, 0.3), (64, 1, 0.5), (5, 2, 0.5), (33, 3, 0.2), (20, 6, 0.1), (50, 9, 0.25),
                                          (70, 12, 1.0), (96, 8, 0.02)])
def test_planes10x_layout_round_trip(oracle, rows, nb, rate):
    """Short records plus exception table rebuild every block exactly; the window base is the smallest that fits; the
    table is ordered row group, tile, block, row; the index counts it; everything else in the buffer is zero."""
    from helpers import make_overlay_case, window_base

    codes = make_overlay_case(oracle, rows, 24 * nb, seed=8, rate=rate, device=None).codes
    codes[min(3, codes.size - 1)] = N_PAPER                      # a code that names no point
    buf, n = oracle.pack_planes10x(codes, rows, nb)
    groups, gbytes, idx_off, tab_off = _p10_offsets(rows, nb)
    assert buf.size == tab_off + 16 * n == oracle.planes10x_bytes(rows, nb, n)
    xs, cls = oracle.decode_batch(codes)
    want_o = window_base(xs)
    ntiles = nb // 4
    index = buf[idx_off: idx_off + 4 * (groups * ntiles + 1)].view(np.uint32)
    table = buf[tab_off:].view(np.uint32).reshape(-1, 4)
    assert index[0] == 0 and index[-1] == n and (np.diff(index.astype(np.int64)) >= 0).all()
    assert not buf[groups * gbytes: idx_off].any() and not buf[idx_off + 4 * (groups * ntiles + 1): tab_off].any()
    expected_entries = []
    for rg in range(groups):
        per_group = []
        for row in range(32 * rg, 32 * rg + 32):
            for b in range(nb):
                hb, o, v = _unpack_planes10x_cell(buf, rows, nb, row, b)
                at = row * nb + b
                if row >= rows or cls[at] < 0:
                    assert hb == 0 and (v == [0] * 24 if o is not None else v == [8] * 24)
                    continue
                x = xs[at]
                shell, par, gain = int((x.astype(np.int64) ** 2).sum()) // 16, int(x[0]) & 1, int(codes[at]) >> 47
                u = [8 + (int(c) - par) // 2 for c in x]
                if o is None:                        # past the tiles: four-bit codes, always exact
                    assert hb == shell | par << 4 | gain << 5 and v == u
                elif want_o[at] == 0:                # an exception: nothing in the short record, everything in the table
                    assert hb == 0 and v == [0] * 24
                    per_group.append((b // 4, b % 4, row % 32, shell | par << 4 | gain << 5, u))
                else:
                    assert o == want_o[at] and hb == (((o - 3) | par << 2 | gain << 3) ^ shell) | shell << 4
                    assert [c + o for c in v] == u and [2 * (c + o - 8) + par for c in v] == x.tolist()
        per_group.sort(key=lambda t: t[:3])
        for T in range(ntiles):                      # one index entry a tile: the entries of the tiles before it
            assert index[rg * ntiles + T] == len(expected_entries) + sum(1 for t in per_group if t[0] < T)
        expected_entries += per_group
    assert len(expected_entries) == n
    for ent, (tile, q, r, hb, u) in zip(table, expected_entries):
        assert int(ent[0]) == hb | r << 8 | (4 * tile + q) << 13
        assert [(int(ent[1 + i // 8]) >> (4 * (i % 8))) & 15 for i in range(24)] == u
    # a table with less room keeps the first entries, and the index stops at the capacity
    if n > 1:
        small, n2 = oracle.pack_planes10x(codes, rows, nb, capacity=n // 2)
        assert n2 == n and small.size == tab_off + 16 * (n // 2)
        assert np.array_equal(small[:idx_off], buf[:idx_off]) and np.array_equal(small[tab_off:], buf[tab_off: tab_off + 16 * (n // 2)])
        assert np.array_equal(small[idx_off: idx_off + 4 * (groups * ntiles + 1)].view(np.uint32), np.minimum(index, n // 2))


def test_planes10x_layout_worked_example_by_hand(oracle):
    """One row, four blocks: index 0 = (0^22, 4, 4) (shell 2: codes 8 and 10, window base 3, stored 5 and 7), a code
    that names no point, index 0 with the gain bit, and (8, -8, 0^22) (shell 8: codes 12, 4, 8 - no window)."""
    x = np.zeros(24, np.int8)
    x[0], x[1] = 8, -8
    wide = oracle.encode(x)
    buf, n = oracle.pack_planes10x(np.array([0, N_PAPER, 1 << 47, wide], np.uint64), 1, 4)
    assert n == 1 and buf.size == 1280 + 128 + 16
    words = buf[:1152].view(np.uint32)
    # row 0 is (m, e, g) = (0, 0, 0): lanes 0..3.  Block 0 is slot 0 of half-step 0: V0 of lane t holds its coordinates
    # 4t.. in bits 0..2 and, for t < 2, 16 + 4t.. in bits 3..5 (for t >= 2 those are block 1's: zero)
    assert [int(words[4 * t]) for t in range(4)] == [0x2D2D2D2D, 0x3D3D2D2D, 0x05050505, 0x05050505]
    # positions 32.. belong to slot 1 (block 1, empty), so V8 is zero; block 2 is slot 0 of half-step 2: V4 of the
    # same lanes, at byte 512 + 16 t
    assert [int(words[128 + 4 * t]) for t in range(4)] == [0x2D2D2D2D, 0x3D3D2D2D, 0x05050505, 0x05050505]
    assert not words[256:].any()                             # V8 of every lane
    rest = np.ones(1152 // 4, bool)
    rest[[0, 4, 8, 12, 128, 132, 136, 140]] = False
    assert not words[rest].any()
    hdr = buf[1152:1280]
    assert int(hdr[0]) == (2 << 4 | 2) and int(hdr[4]) == (2 << 4 | (8 ^ 2)) and int(hdr.astype(np.int64).sum()) == 34 + 42
    assert buf[1280:1288].view(np.uint32).tolist() == [0, 1]           # one tile: nothing before it, one entry in all
    assert buf[1408:1424].view(np.uint32).tolist() == [8 | 0 << 8 | 3 << 13, 0x8888884C, 0x88888888, 0x88888888]


def test_planes10x_rate_on_the_synthetic_stream(oracle):
    """About one block in eight thousand of the synthetic stream is an exception; the paper's rule (five levels)
    would send about one in 160 to the table."""
    from helpers import window_base
    from paper_2609_02652_b200 import datagen

    codes = datagen.make_codes(1024, 128, 21).numpy().astype(np.uint64).ravel()
    xs, _ = oracle.decode_batch(codes)
    rate = float((window_base(xs) == 0).mean())
    assert 0.00005 < rate < 0.0004
    levels = np.array([len(set(np.abs(r).tolist())) for r in xs[:20000]])
    assert 0.004 < float((levels >= 5).mean()) < 0.009
    _, n = oracle.pack_planes10x(codes, 1024, 128)
    assert n == int((window_base(xs) == 0).sum())


@pytest.mark.parametrize("rows,nb", [(32, 3), (37, 5)])
def test_onehot_layout_round_trip_and_field_widths(oracle, rows, nb):
    codes = _codes(oracle, rows, nb, seed=6)
    buf = oracle.pack_onehot(codes, rows, nb).view(np.uint32)
    assert buf.size * 4 == ((rows + 31) // 32) * nb * 640
    xs, cls = oracle.decode_batch(codes)
    for row in range(rows):
        rg, l = divmod(row, 32)
        for b in range(nb):
            v = [int(buf[(rg * nb + b) * 160 + 32 * t + l]) for t in range(5)]
            c = (v[0] >> 24) | (((v[1] >> 24) & 1) << 8)
            g = (v[1] >> 25) & 1
            smask = v[0] & 0xFFFFFF
            masks = [v[1] & 0xFFFFFF, v[2], v[3], v[4]]
            info = oracle.class_info(c)
            dist = sorted(set(info["mags"]))
            assert c == cls[row * nb + b] and g == int(codes[row * nb + b]) >> 47
            assert all(m >> 24 == 0 for m in masks[1:])
            assert all(masks[t] == 0 for t in range(len(dist) - 1, 4))        # 9 + 1 + 24 L bits used
            x = []
            for i in range(24):
                lv = sum((t + 1) * ((masks[t] >> i) & 1) for t in range(4))
                assert sum((masks[t] >> i) & 1 for t in range(4)) <= 1
                x.append((-1 if (smask >> i) & 1 else 1) * dist[lv])
            assert x == xs[row * nb + b].tolist()
            # the same block through the logical record: planes and one-hot agree
            rec = oracle.record(int(codes[row * nb + b]))
            lv_planes = [sum(((rec["planes"][t] >> i) & 1) << t for t in range(3)) for i in range(24)]
            assert [2 * p + info["odd"] for p in lv_planes] == [abs(a) for a in x]
            assert rec["smask"] == smask and rec["cls"] == c


def test_record_payload_is_106_bits():
    assert 9 + 1 + 24 + 3 * 24 == 106 <= 14 * 8        # Sec. 2.3: 106 payload bits in a 112-bit record


# ---------------------------------------------------------------- f64 matvec
def test_matvec_against_numpy_and_special_cases(oracle):
    from paper_2609_02652_b200 import datagen

    rows, nb = 21, 13
    codes = _codes(oracle, rows, nb, seed=8)
    rs = datagen.make_row_scale(rows, 8).numpy()
    x = datagen.make_x(nb * 24 - 5, nb * 24, 8).numpy()
    gain = (0.75, 1.5)
    xs, cls = oracle.decode_batch(codes)
    # weights written out independently: r * gamma_g * x_i / (4 sqrt m)
    W = np.zeros((rows, nb * 24))
    for r in range(rows):
        for b in range(nb):
            m = oracle.class_info(int(cls[r * nb + b]))["shell"]
            g = gain[int(codes[r * nb + b]) >> 47]
            W[r, 24 * b:24 * b + 24] = float(rs[r]) * g * xs[r * nb + b].astype(float) / (4 * math.sqrt(m))
    y, wn, ab = oracle.matvec(codes, rows, nb, rs, gain, x, nthreads=3)
    ref = W @ x.astype(np.float64)
    assert np.allclose(y, ref, rtol=0, atol=1e-13)
    assert np.allclose(wn, np.linalg.norm(W, axis=1), rtol=1e-13)
    assert np.allclose(ab, np.abs(W * x.astype(np.float64)).sum(1), rtol=1e-13)
    assert np.allclose(oracle.dequant(codes, rows, nb, rs, gain), W, rtol=0, atol=1e-15)
    y1, _, _ = oracle.matvec(codes, rows, nb, rs, gain, x, nthreads=1)
    assert (y1 == y).all()                                   # thread split does not change a row
    # unit directions: with r = 1 and gamma = 1 every block has norm 1
    one = np.ones(rows, np.float16)
    Wu = oracle.dequant(codes, rows, nb, one, (1.0, 1.0)).reshape(rows, nb, 24)
    assert np.allclose((Wu**2).sum(-1), 1.0, atol=1e-14)
    # x = e_j picks column j
    for j in (0, 17, nb * 24 - 1):
        e = np.zeros(nb * 24, np.float16)
        e[j] = 1
        yj, _, _ = oracle.matvec(codes, rows, nb, one, (1.0, 1.0), e)
        assert np.allclose(yj, Wu.reshape(rows, -1)[:, j], atol=1e-15)
    # a code that names no point contributes nothing
    codes2 = codes.copy()
    codes2[:] = N_PAPER
    assert (oracle.matvec(codes2, rows, nb, rs, gain, x)[0] == 0).all()


def test_generator_draws_valid_shell_uniform_indices(oracle):
    from paper_2609_02652_b200 import datagen

    sizes, bases = datagen.shell_sizes(), datagen.shell_bases()
    assert [sizes[m] for m in range(2, 13)] == [oracle.shell_count(m) for m in range(2, 13)]
    assert bases[13] == N_PAPER
    codes = datagen.make_codes(64, 128, 0).numpy().astype(np.uint64)
    idx = codes & np.uint64((1 << 47) - 1)
    assert (idx < N_PAPER).all()
    shell = np.searchsorted([bases[m] for m in range(2, 14)], idx, side="right") + 1
    hist = np.bincount(shell, minlength=13)[2:13]
    assert hist.min() > 0.7 * hist.mean() and hist.max() < 1.3 * hist.mean()
    g = (codes >> np.uint64(47)).astype(int)
    assert 0.45 < g.mean() < 0.55 and g.max() == 1
    assert (datagen.make_codes(64, 128, 0, start=100, count=50).numpy() == datagen.make_codes(64, 128, 0).numpy()[100:150]).all()


def test_planes_layout_worked_example_by_hand(oracle):
    """One row, one block, index 0 (x = 0,...,0,4,4; class 0), written out by hand from the layout's description.
    Codes: u = 8 everywhere except coordinates 22 and 23, where u = 8 + 4/2 = 10.  With one block the piece is a single:
    row 0 is (m,e,g) = (0,0,0), its slot is its row half 0, so coordinate i sits at position i.  Positions 22 and 23
    are 16*1 + 4*1 + 2 and 16*1 + 4*1 + 3: column c = 1, t = 1, i = 2 and 3, i.e. nibbles 2*2+1 = 5 and 2*3+1 = 7
    of word Wa of lane 4*0 + 1, which is stored at byte 128*0 + 4*1.  Every other nibble of the 448 bytes of payload
    is 8 (row 0's other codes and the empty records of rows 1..31).  Headers: pair 2*0 + 0 holds row 0 (class 0,
    gain 0) in its low half and row 8 (empty: 511) in its high half, at byte 384; all other halves are 511."""
    buf = oracle.pack_planes(np.array([0], dtype=np.uint64), 1, 1)
    assert buf.size == 448
    words = buf.view(np.uint32)
    expect = np.full(112, 0x88888888, dtype=np.uint32)
    expect[1] = 0xA8A88888
    expect[96:] = 0x01FF01FF
    expect[96] = 0x01FF0000
    assert (words == expect).all()
    # with the gain bit set only the header changes: class | 1 << 9
    buf2 = oracle.pack_planes(np.array([1 << 47], dtype=np.uint64), 1, 1).view(np.uint32)
    expect[96] = 0x01FF0200
    assert (buf2 == expect).all()


# ---------------------------------------------------------------- activation rotation (Sec. 2.3, Sec. 5)
def _oracle():
    from oracle import oracle as O

    return O


def test_rotation_rounding_step_matches_numpy_float16():
    """The oracle's f64 -> FP16 rounding against numpy's conversion: ties, subnormals, overflow, random values."""
    O = _oracle()
    rng = np.random.default_rng(5)
    vals = [0.0, -0.0, 1.0, -1.0, 65504.0, 65519.9, 65520.0, 1e6, -1e6, 2.0 ** -24, 2.0 ** -25, 2.0 ** -25 * 1.0000001,
            3 * 2.0 ** -25, 2.0 ** -14, 2.0 ** -14 - 2.0 ** -25, 1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 1.0 + 2.0 ** -11 + 2.0 ** -30,
            2047.5, 2048.5, 2049.5, 0.1, -0.3]
    vals += list(rng.normal(size=4000) * np.exp(rng.uniform(-18, 11, size=4000)))
    # exact ties in every binade: (2 m + 1) / 2 quanta
    for e in range(-14, 16):
        for m in (1024, 1025, 1536, 2046, 2047):
            vals.append((2 * m + 1) * 2.0 ** (e - 11))
    with np.errstate(over="ignore"):
        want = np.array(vals, np.float64).astype(np.float16).view(np.uint16)
    got = np.array([O.double_to_half_bits(v) for v in vals], np.uint16)
    np.testing.assert_array_equal(got, want)


def test_rotation_worked_examples_by_hand():
    """H_4 (1,2,3,4) / 2 = (5,-1,-2,0); a unit vector returns a column of H_B / sqrt(B); a constant lands on k = 0."""
    O = _oracle()
    y = O.rotate(np.array([1, 2, 3, 4], np.float16))
    np.testing.assert_array_equal(y.astype(np.float64), [5.0, -1.0, -2.0, 0.0])
    for B, j in ((8, 5), (64, 37), (256, 255)):
        x = np.zeros(B, np.float16)
        x[j] = 3.0
        y = O.rotate(x).astype(np.float64)
        sign = np.array([(-1) ** bin(j & k).count("1") for k in range(B)], np.float64)
        want = (3.0 * sign / math.sqrt(B)).astype(np.float16).astype(np.float64)
        np.testing.assert_array_equal(y, want)
    y = O.rotate(np.full(1024, 0.5, np.float16)).astype(np.float64)
    assert y[0] == 16.0 and not y[1:].any()
    # block length 1 is the identity, and so is any length whose largest power-of-two divisor is 1
    x = np.arange(7, dtype=np.float16) - 3
    np.testing.assert_array_equal(O.rotate(x), x)
    np.testing.assert_array_equal(O.rotate(np.arange(8, dtype=np.float16), block=1), np.arange(8, dtype=np.float16))


def test_rotation_block_rule():
    O = _oracle()
    # the lengths of the paper's activations: hidden and intermediate sizes of the 4B / 8B / 14B / 32B models
    assert [O.rotate_block(n) for n in (2560, 9728, 4096, 12288, 5120, 17408, 25600, 24, 98304, 7)] == \
        [512, 512, 4096, 4096, 1024, 1024, 1024, 8, 16384, 1]
    assert O.rotate_block(2560, 128) == 128
    for n, b in ((2560, 1024), (4096, 3), (4096, 32768), (100, 8), (0, 0)):
        assert O.rotate_block(n, b) == 0
    with pytest.raises(ValueError):
        O.rotate(np.zeros(24, np.float16), block=16)


@pytest.mark.parametrize("n,block", [(24, 0), (96, 0), (2560, 0), (2560, 64), (4096, 0), (9728, 0), (1536, 512)])
def test_rotation_against_scipy_hadamard_and_invariants(n, block):
    """The definition against scipy's Hadamard matrix (a library routine the oracle does not call), plus
    orthogonality: the norm is kept and applying the rotation twice returns x, both up to FP16 rounding."""
    import scipy.linalg

    O = _oracle()
    rng = np.random.default_rng(n + block)
    x = rng.normal(size=n).astype(np.float16)
    neg = rng.integers(0, 2, size=n).astype(np.uint8) if block else None
    B = O.rotate_block(n, block)
    y = O.rotate(x, block, neg)
    H = scipy.linalg.hadamard(B).astype(np.float64) if B > 1 else np.ones((1, 1))
    xs = x.astype(np.float64) * (1.0 if neg is None else 1.0 - 2.0 * neg)
    want = (xs.reshape(n // B, B) @ H.T / math.sqrt(B)).ravel()
    # f64 matmul of these sizes carries ~1e-13 of error: compare before rounding, then the rounding itself
    assert np.abs(y.astype(np.float64) - want).max() <= np.abs(want).max() * 2.0 ** -11 + 1e-12
    same = want.astype(np.float16) == y
    assert same.mean() > 0.999                       # the few others sit on a rounding boundary of the matmul's error
    np.testing.assert_array_less(np.abs(y[~same].astype(np.float64) - want[~same]), np.abs(want[~same]) * 2.0 ** -10 + 2.0 ** -24)
    nx, ny = np.linalg.norm(xs), np.linalg.norm(y.astype(np.float64))
    assert abs(nx - ny) <= 2.0 ** -10 * nx
    if neg is None:
        back = O.rotate(y, block).astype(np.float64)
        assert np.abs(back - x.astype(np.float64)).max() <= 2.0 ** -9 * max(1.0, np.abs(want).max())


def test_rotation_is_exact_where_floats_would_round():
    """A large and a tiny value in one block: the exact sum keeps both (an f32 butterfly would lose the small one)."""
    O = _oracle()
    x = np.zeros(4, np.float16)
    x[0], x[1] = 2048.0, 2.0 ** -14
    y = O.rotate(x).astype(np.float64)
    # (2048 +- 2^-14) / 2 rounds to 1024 in FP16; with x0 = 0 the small value alone survives
    np.testing.assert_array_equal(y, [1024.0, 1024.0, 1024.0, 1024.0])
    x[0] = 0
    np.testing.assert_array_equal(O.rotate(x).astype(np.float64), np.array([1, -1, 1, -1]) * 2.0 ** -15)
    # cancellation: two large values cancel exactly and leave the small one (k = 0 and k = 2); where they add,
    # (2000 +- 2^-10) / 2 rounds to 1000
    x = np.array([1000.0, -1000.0, 2.0 ** -10, 0.0], np.float16)
    np.testing.assert_array_equal(O.rotate(x).astype(np.float64), [2.0 ** -11, 1000.0, -(2.0 ** -11), 1000.0])
