"""Pins for the CPU oracle: things the definitions and plain mathematics fix, none of which call
the oracle to produce their own expected value.  Hand-derived fixtures live in tests/golden/.
Brute-force comparisons are written in Python big integers and bytes slicing, a different
language and a different decomposition from the C++ loops."""
import os

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
M64 = 1 << 64


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield [c.strip() for c in line.split("|")]


def _ints(s):
    return [int(x) for x in s.split(",")] if s else []


def py_checksum(data: bytes, B: int):
    """Big-integer statement of the checksum definition."""
    out = []
    for start in range(0, len(data), B):
        chunk = data[start:start + B]
        chunk = chunk + b"\0" * (-len(chunk) % 8)
        words = [int.from_bytes(chunk[8 * i:8 * i + 8], "little") for i in range(len(chunk) // 8)]
        out.append(sum(w * (2 * i + 1) for i, w in enumerate(words)) % M64)
    return out


def py_pack(tensors, B):
    """bytes.join statement of the packed stream."""
    s = b""
    offs = []
    for t in tensors:
        s += b"\0" * (-len(s) % 256)
        offs.append(len(s))
        s += t
    s += b"\0" * (-len(s) % 256)
    return s, offs


def rand_tensors(rng, n, sizes=(2, 6, 254, 256, 258, 510, 514, 1016, 2000, 4098)):
    return [rng.integers(0, 256, int(rng.choice(sizes)), dtype=np.uint8) for _ in range(n)]


# ------------------------------------------------------------------ checksum


def test_checksum_golden(oracle_mod):
    for name, data, B, expect in _rows("checksum_cases.txt"):
        if data.startswith("w:"):
            arr = np.array(_ints(data[2:]), dtype=np.uint64)
        else:
            arr = np.frombuffer(bytes.fromhex(data), dtype=np.uint8)
        got = [int(x) for x in oracle_mod.checksum(arr, int(B))]
        assert got == _ints(expect), name


@pytest.mark.parametrize("c,n", [(1, 1), (3, 7), (M64 - 1, 3), (0x3F8000003F800000, 1024),
                                 (0xDEADBEEFCAFEF00D, 4096), (12345678901234567, 131072)])
def test_checksum_constant_word_closed_form(oracle_mod, c, n):
    # sum_{i<n} (2i+1) = n^2
    words = np.full(n, c, dtype=np.uint64)
    B = ((8 * n + 255) // 256) * 256
    assert int(oracle_mod.checksum(words, B)[0]) == (c * n * n) % M64


@pytest.mark.parametrize("i,w", [(0, 5), (1, 5), (31, M64 - 1), (1000, 0x0123456789ABCDEF)])
def test_checksum_one_hot(oracle_mod, i, w):
    words = np.zeros(1024, dtype=np.uint64)
    words[i] = w
    assert int(oracle_mod.checksum(words, 8192)[0]) == (w * (2 * i + 1)) % M64


def test_checksum_linearity_shift_and_zero_extension(oracle_mod):
    rng = np.random.default_rng(11)
    a = rng.integers(0, M64, 512, dtype=np.uint64)
    b = rng.integers(0, M64, 512, dtype=np.uint64)
    B = 4096
    C = lambda x: int(oracle_mod.checksum(x, B)[0])
    assert C(a + b) == (C(a) + C(b)) % M64                      # word-wise add mod 2^64
    s = 77
    shifted = np.concatenate([np.zeros(s, dtype=np.uint64), a[:512 - s]])
    base = a[:512 - s]
    sum_w = sum(int(x) for x in base) % M64
    assert C(shifted) == (C(base) + 2 * s * sum_w) % M64        # prepend s zero words
    assert C(np.concatenate([base, np.zeros(s, dtype=np.uint64)])) == C(base)  # append zero words


@pytest.mark.parametrize("nbytes,B", [(1, 256), (7, 256), (8, 256), (255, 256), (256, 256), (257, 256),
                                      (1000, 512), (4096, 1024), (4099, 1024), (70001, 4096)])
def test_checksum_brute_force(oracle_mod, nbytes, B):
    rng = np.random.default_rng(nbytes * 31 + B)
    data = rng.integers(0, 256, nbytes, dtype=np.uint8)
    assert [int(x) for x in oracle_mod.checksum(data, B)] == py_checksum(data.tobytes(), B)


def test_checksum_empty_and_errors(oracle_mod):
    assert oracle_mod.checksum(np.zeros(0, dtype=np.uint8), 256).size == 0
    with pytest.raises(oracle_mod.OracleError) as e:
        oracle_mod.checksum(np.zeros(8, dtype=np.uint8), 100)
    assert e.value.code == -2


# ------------------------------------------------------------------ layout / pack / unpack


def test_layout_golden(oracle_mod):
    for sizes, B, offs, T, nb in _rows("layout_cases.txt"):
        off, total, n_buckets = oracle_mod.layout(_ints(sizes), int(B))
        assert [int(x) for x in off] == _ints(offs)
        assert (total, n_buckets) == (int(T), int(nb))


def test_layout_invariants(oracle_mod):
    rng = np.random.default_rng(5)
    for trial in range(20):
        sizes = [2 * int(rng.integers(1, 3000)) for _ in range(int(rng.integers(1, 40)))]
        B = 256 * int(rng.integers(1, 9))
        off, T, nb = oracle_mod.layout(sizes, B)
        off = [int(x) for x in off]
        assert off[0] == 0 and all(o % 256 == 0 for o in off) and T % 256 == 0
        for k in range(1, len(off)):
            assert off[k] >= off[k - 1] + sizes[k - 1]          # no overlap
            assert off[k] - (off[k - 1] + sizes[k - 1]) < 256   # minimal padding
        assert 0 <= T - (off[-1] + sizes[-1]) < 256
        assert nb == -(-T // B)


def test_layout_errors(oracle_mod):
    for sizes, B, code in (([4], 100, -2), ([4], 0, -1), ([0], 256, -1), ([3], 256, -1), ([], 256, -1)):
        with pytest.raises(oracle_mod.OracleError) as e:
            oracle_mod.layout(sizes, B)
        assert e.value.code == code


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("B", [256, 512, 768, 1024])
def test_pack_brute_force(oracle_mod, seed, B):
    rng = np.random.default_rng(seed)
    tensors = rand_tensors(rng, int(rng.integers(1, 9)))
    stream, cks = oracle_mod.pack(tensors, B)
    expect, offs = py_pack([t.tobytes() for t in tensors], B)
    assert stream.tobytes() == expect
    assert [int(x) for x in cks] == py_checksum(expect, B)
    assert [int(x) for x in oracle_mod.layout([t.size for t in tensors], B)[0]] == offs


def test_pack_padding_is_zero_and_round_trip(oracle_mod):
    rng = np.random.default_rng(99)
    tensors = [rng.integers(1, 256, n, dtype=np.uint8) for n in (2, 254, 258, 1000, 256, 6)]  # no zero bytes
    sizes = [t.size for t in tensors]
    stream, _ = oracle_mod.pack(tensors, 512)
    off, T, _ = oracle_mod.layout(sizes, 512)
    covered = np.zeros(T, dtype=bool)
    for o, n in zip(off, sizes):
        covered[int(o):int(o) + n] = True
    assert stream.size == T
    assert np.all(stream[~covered] == 0) and np.all(stream[covered] != 0)
    back = oracle_mod.unpack(stream, sizes)
    for t, b in zip(tensors, back):
        assert np.array_equal(t, b)


def test_unpack_ignores_padding(oracle_mod):
    rng = np.random.default_rng(3)
    tensors = rand_tensors(rng, 5)
    sizes = [t.size for t in tensors]
    stream, _ = oracle_mod.pack(tensors, 256)
    off, T, _ = oracle_mod.layout(sizes, 256)
    dirty = stream.copy()
    covered = np.zeros(T, dtype=bool)
    for o, n in zip(off, sizes):
        covered[int(o):int(o) + n] = True
    dirty[~covered] = 0xEE
    for t, b in zip(tensors, oracle_mod.unpack(dirty, sizes)):
        assert np.array_equal(t, b)


def test_pack_range_is_a_slice_of_pack(oracle_mod):
    rng = np.random.default_rng(8)
    tensors = rand_tensors(rng, 7)
    sizes = [t.size for t in tensors]
    stream, _ = oracle_mod.pack(tensors, 512)
    expect, offs = py_pack([t.tobytes() for t in tensors], 512)
    for lo, hi in ((0, stream.size), (256, 768), (512, 512), (stream.size - 256, stream.size)):
        assert oracle_mod.pack_range(tensors, sizes, lo, hi).tobytes() == expect[lo:hi]
    # tensors outside the range may be omitted
    lo, hi = offs[3], offs[3] + 256
    sparse = [t if (o < hi and o + t.size > lo) else None for t, o in zip(tensors, offs)]
    assert oracle_mod.pack_range(sparse, sizes, lo, hi).tobytes() == expect[lo:hi]


def test_norm_vector_of_ones_closed_form(oracle_mod):
    # A 2048-element fp32 vector of 1.0 is 1024 words c = 0x3F8000003F800000; placed at word s of a
    # bucket it contributes c*((s+1024)^2 - s^2).  Isolated through linearity.
    rng = np.random.default_rng(21)
    before = rng.integers(0, 256, 2 * 4096 + 512, dtype=np.uint8)       # ends off a 256 boundary
    norm = np.ones(2048, dtype=np.float32)
    after = rng.integers(0, 256, 3000, dtype=np.uint8)
    B = 64 * 1024
    with_norm, c1 = oracle_mod.pack([before, norm, after], B)
    without, c0 = oracle_mod.pack([before, np.zeros(2048, dtype=np.float32), after], B)
    s = ((before.size + 255) // 256 * 256) // 8
    c = 0x3F8000003F800000
    assert (int(c1[0]) - int(c0[0])) % M64 == (c * ((s + 1024) ** 2 - s ** 2)) % M64


# ------------------------------------------------------------------ shard


def test_shard_bounds_golden(oracle_mod):
    for N, D, r, lo, hi in _rows("shard_cases.txt"):
        assert oracle_mod.shard_bounds(int(N), int(r), int(D)) == (int(lo), int(hi))


def test_shard_bounds_tile_exactly_and_need_128_bits(oracle_mod):
    for N, D in ((0, 5), (1, 64), (63, 64), (64, 64), (1000003, 64), (1 << 63, (1 << 32) - 1),
                 ((1 << 64) - 1, (1 << 32) - 1)):
        rs = range(D) if D <= 64 else [0, 1, 2, D // 2, D - 2, D - 1]
        prev_hi = None
        for r in rs:
            lo, hi = oracle_mod.shard_bounds(N, r, D)
            assert (lo, hi) == ((r * N) // D, ((r + 1) * N) // D)   # Python integers do not overflow
            assert hi - lo in (N // D, N // D + 1)
            if prev_hi is not None and D <= 64:
                assert lo == prev_hi
            prev_hi = hi
        assert oracle_mod.shard_bounds(N, 0, D)[0] == 0
        assert oracle_mod.shard_bounds(N, D - 1, D)[1] == N


@pytest.mark.parametrize("e", [2, 4, 8])
@pytest.mark.parametrize("D", [1, 2, 3, 7, 64])
def test_shard_union_and_brute_force(oracle_mod, e, D):
    rng = np.random.default_rng(e * 100 + D)
    counts = [int(rng.choice([1, 3, 5, 127, 129, 257])) for _ in range(int(rng.integers(1, 7)))]
    tensors = [rng.integers(0, 256, c * e, dtype=np.uint8) for c in counts]
    sizes = [t.size for t in tensors]
    flat = b"".join(t.tobytes() for t in tensors)
    N = len(flat) // e
    parts = []
    for r in range(D):
        got = oracle_mod.shard(tensors, sizes, e, r, D).tobytes()
        lo, hi = (r * N) // D, ((r + 1) * N) // D
        assert got == flat[lo * e:hi * e]
        parts.append(got)
    assert b"".join(parts) == flat


def test_shard_errors(oracle_mod):
    t = [np.zeros(8, dtype=np.uint8)]
    for e, r, D, code in ((4, 2, 2, -5), (4, 0, 0, -5), (3, 0, 1, -6), (8, 0, 1, 0)):
        if code == 0:
            assert oracle_mod.shard(t, [8], e, r, D).size == 8
            continue
        with pytest.raises(oracle_mod.OracleError) as ex:
            oracle_mod.shard(t, [8], e, r, D)
        assert ex.value.code == code
    with pytest.raises(oracle_mod.OracleError) as ex:   # nbytes not a multiple of elem_size
        oracle_mod.shard([np.zeros(6, dtype=np.uint8)], [6], 4, 0, 1)
    assert ex.value.code == -1


# ------------------------------------------------------------------ shard insert


@pytest.mark.parametrize("e", [2, 4, 8])
@pytest.mark.parametrize("D", [1, 3, 64])
def test_shard_insert_brute_force_and_inverse(oracle_mod, e, D):
    rng = np.random.default_rng(e * 1000 + D)
    counts = [int(rng.choice([1, 3, 5, 127, 129, 257])) for _ in range(int(rng.integers(1, 7)))]
    tensors = [rng.integers(0, 256, c * e, dtype=np.uint8) for c in counts]
    sizes = [t.size for t in tensors]
    flat = bytearray(b"".join(t.tobytes() for t in tensors))
    N = len(flat) // e
    for r in sorted({0, D // 2, D - 1}):
        lo, hi = (r * N) // D, ((r + 1) * N) // D
        data = rng.integers(0, 256, (hi - lo) * e, dtype=np.uint8)
        work = [t.copy() for t in tensors]
        assert oracle_mod.shard_insert(work, sizes, e, r, D, data) == hi - lo
        expect = bytearray(flat)
        expect[lo * e:hi * e] = data.tobytes()                         # Python slice assignment
        assert b"".join(t.tobytes() for t in work) == bytes(expect)
        assert oracle_mod.shard(work, sizes, e, r, D).tobytes() == data.tobytes()   # extract(insert(x)) == x
    # inserting every shard of another plane rebuilds that plane
    other = [rng.integers(0, 256, t.size, dtype=np.uint8) for t in tensors]
    work = [t.copy() for t in tensors]
    for r in range(D):
        oracle_mod.shard_insert(work, sizes, e, r, D, oracle_mod.shard(other, sizes, e, r, D))
    assert all(np.array_equal(a, b) for a, b in zip(work, other))


def test_shard_insert_errors(oracle_mod):
    t = [np.zeros(8, dtype=np.uint8)]
    for e, r, D, n, code in ((4, 2, 2, 8, -5), (3, 0, 1, 8, -6), (4, 0, 1, 4, -3)):
        with pytest.raises(oracle_mod.OracleError) as ex:
            oracle_mod.shard_insert(t, [8], e, r, D, np.zeros(n, dtype=np.uint8))
        assert ex.value.code == code
