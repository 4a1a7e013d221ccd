"""Host-side checks of the C-ABI library that need no GPU: it loads, exports everything the header
declares, plans layouts that agree with the oracle's independent arithmetic, and rejects bad
arguments before anything could be launched."""
import ctypes
import os
import re

import numpy as np
import pytest
import torch

from paper_2412_12636_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FAKE = 0x7F00_0000_0000  # plausible device address; never dereferenced on the host


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def test_library_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "tm_state.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(tm_[a-z_0-9]+)\s*\(", header))
    assert declared == set(binding.SIGNATURES), declared ^ set(binding.SIGNATURES)
    for name in declared:
        assert hasattr(lib, name), name
    assert lib.tm_strerror(0) == b"ok" and lib.tm_strerror(-8) == b"bounded device wait expired"


def _descs(sizes, elem=2, base=FAKE, stride=1 << 24):
    return [(base + k * stride, n, elem, 0) for k, n in enumerate(sizes)]


@pytest.mark.parametrize("seed", range(5))
def test_plan_layout_matches_oracle(lib, oracle_mod, seed):
    rng = np.random.default_rng(seed)
    sizes = [2 * int(rng.integers(1, 200_000)) for _ in range(int(rng.integers(1, 50)))]
    B = 256 * int(rng.integers(1, 600))
    plan = binding.Plan(_descs(sizes), B)
    off, T, nb = oracle_mod.layout(sizes, B)
    assert plan.offsets() == [int(x) for x in off]
    assert (plan.total_bytes, plan.n_buckets) == (T, nb)
    assert plan.workspace_bytes % 256 == 0 and plan.workspace_bytes >= 512


def test_plan_full_size_configs_match_oracle(lib, oracle_mod):
    from paper_2412_12636_b200 import layouts
    for idx in range(4):
        cfg = layouts.role_config(idx)
        sizes = [s.nbytes for s in cfg.specs()]
        descs = []
        addr = FAKE
        for s in cfg.specs():
            descs.append((addr, s.nbytes, s.elem_size, s.plane))
            addr += (s.nbytes + 511) // 512 * 512
        plan = binding.Plan(descs, cfg.bucket_bytes)
        off, T, nb = oracle_mod.layout(sizes, cfg.bucket_bytes)
        assert plan.offsets() == [int(x) for x in off] and (plan.total_bytes, plan.n_buckets) == (T, nb)


def test_plan_rejects_bad_arguments(lib):
    cases = [
        ([(FAKE, 4, 2, 0)], 100, binding.TM_ERR_ALIGN),       # bucket not a multiple of 256
        ([(FAKE, 4, 2, 0)], 0, binding.TM_ERR_ARG),
        ([(FAKE, 4, 2, 0)], (1 << 35) + 256, binding.TM_ERR_ARG),
        ([(FAKE + 1, 4, 2, 0)], 256, binding.TM_ERR_ALIGN),   # odd address
        ([(FAKE, 0, 2, 0)], 256, binding.TM_ERR_ARG),
        ([(FAKE, 6, 4, 0)], 256, binding.TM_ERR_ARG),         # not a whole number of elements
        ([(FAKE, 6, 3, 0)], 256, binding.TM_ERR_DTYPE),
        ([(0, 4, 2, 0)], 256, binding.TM_ERR_ARG),
        ([], 256, binding.TM_ERR_ARG),
        ([(FAKE, (1 << 46) + 2, 2, 0)], 256, binding.TM_ERR_ARG),   # absurd size: refused, no overflow
    ]
    for descs, B, code in cases:
        with pytest.raises(binding.TmError) as e:
            binding.Plan(descs, B)
        assert e.value.status == code, (descs, B)


def test_ops_refuse_a_plan_without_work_list(lib):
    plan = binding.Plan(_descs([512, 1024]), 256)
    for call in (lambda: binding.tm_state_pack(plan, FAKE + (1 << 30), 1 << 20, None, 0),
                 lambda: binding.tm_state_unpack(plan, FAKE + (1 << 30), 1 << 20, 0)):
        with pytest.raises(binding.TmError) as e:
            call()
        assert e.value.status == binding.TM_ERR_STATE


def test_shard_bounds_and_validation(lib):
    for N, D in ((10, 3), (1069711360, 24), (1, 64), ((1 << 64) - 1, (1 << 32) - 1)):
        for r in sorted({0, 1 % D, D // 2, D - 1}):
            assert binding.tm_shard_bounds(N, r, D) == ((r * N) // D, ((r + 1) * N) // D)
    for r, D in ((2, 2), (0, 0)):
        with pytest.raises(binding.TmError) as e:
            binding.tm_shard_bounds(10, r, D)
        assert e.value.status == binding.TM_ERR_RANK
    mixed = [(FAKE, 8, 4, 1), (FAKE + 4096, 8, 2, 0)]
    with pytest.raises(binding.TmError) as e:
        binding.tm_shard_workspace(mixed, 0, 2)
    assert e.value.status == binding.TM_ERR_DTYPE
    with pytest.raises(binding.TmError) as e:
        binding.tm_shard_workspace(_descs([8, 8], elem=4), 3, 2)
    assert e.value.status == binding.TM_ERR_RANK
    assert binding.tm_shard_workspace(_descs([1 << 20, 1 << 20], elem=4), 1, 2) >= 512
    # argument errors are reported before any device work
    with pytest.raises(binding.TmError) as e:
        binding.tm_shard_extract(_descs([1 << 20], elem=4), 0, 1, FAKE + 4096, 1 << 20, FAKE + (1 << 30), 1 << 20, 0)
    assert e.value.status == binding.TM_ERR_OVERLAP
    with pytest.raises(binding.TmError) as e:
        binding.tm_shard_extract(_descs([1 << 20], elem=4), 0, 1, FAKE + (1 << 28), 100, FAKE + (1 << 30), 1 << 20, 0)
    assert e.value.status == binding.TM_ERR_CAPACITY


def test_checksum_argument_validation(lib):
    for args, code in (((FAKE, 1024, 100, FAKE + 4096, 0), binding.TM_ERR_ALIGN),
                       ((FAKE, 1024, 0, FAKE + 4096, 0), binding.TM_ERR_ARG),
                       ((FAKE + 8, 1024, 256, FAKE + 4096, 0), binding.TM_ERR_ALIGN),
                       ((FAKE, 1024, 256, None, 0), binding.TM_ERR_ARG)):
        with pytest.raises(binding.TmError) as e:
            binding.tm_checksum(*args)
        assert e.value.status == code
    binding.tm_checksum(FAKE, 0, 256, None, 0)   # empty input: nothing to do


@pytest.mark.skipif(torch.cuda.is_available(), reason="only meaningful on a machine without a GPU")
def test_no_cpu_fallback_without_a_gpu(lib):
    host = np.zeros(1024, dtype=np.uint8)
    out = np.zeros(4, dtype=np.uint64)
    before = binding.tm_launch_count()
    with pytest.raises(binding.TmError) as e:
        binding.tm_checksum(host.ctypes.data & ~15, 512, 256, out.ctypes.data, 0)
    assert e.value.status == binding.TM_ERR_CUDA
    assert binding.tm_launch_count() == before and not out.any()


def test_header_is_plain_c_and_library_links_from_c(lib, tmp_path):
    import subprocess
    exe = tmp_path / "c_abi_check"
    libdir = os.path.dirname(binding.LIB_PATH)
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
                    os.path.join(ROOT, "tests", "c_abi_check.c"), "-o", str(exe), "-L", libdir, "-ltm_state",
                    f"-Wl,-rpath,{libdir}"], check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0, (out.returncode, out.stdout, out.stderr)
    assert "c abi ok, 0 launches" in out.stdout


@pytest.mark.parametrize("seed", range(12))
def test_work_list_tiles_the_stream_exactly(lib, oracle_mod, seed):
    """Planner invariants, checked on the host against the oracle's layout: the pieces cover
    [0, T) without gap or overlap, stay inside one bucket, carry the right word index and tensor
    address, and the items partition the pieces within one bucket."""
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(1, 60))
    log_sizes = rng.uniform(0, 21, n)
    sizes = [2 * max(1, int(2 ** x) // 2) for x in log_sizes]
    B = 256 * int(rng.choice([1, 3, 16, 4096, 32768, 1 << 20]))
    addr, descs = FAKE, []
    for k, nb in enumerate(sizes):
        addr += 2 * int(rng.integers(0, 64))
        descs.append((addr, nb, 2, 0))
        addr += nb
    plan = binding.Plan(descs, B)
    off, T, nbuckets = oracle_mod.layout(sizes, B)
    pieces, items = plan.pieces()
    assert items[0] == 0 and items[-1] == pieces.size and np.all(np.diff(items.astype(np.int64)) > 0)
    pos, k, within = 0, 0, 0          # stream position, current tensor, bytes of it already seen
    for p in pieces:
        assert int(p["off"]) == pos and p["nbytes"] > 0 and p["nbytes"] % 2 == 0
        assert int(p["off"]) == int(off[k]) + within
        assert int(p["tensor"]) == descs[k][0] + within
        b = int(p["off"]) // B
        assert int(p["bucket"]) == b and int(p["word0"]) == (int(p["off"]) - b * B) // 8
        end = int(p["off"]) + int(p["nbytes"]) + int(p["pad"])
        assert end <= (b + 1) * B                                   # never crosses a bucket boundary
        within += int(p["nbytes"])
        if within == sizes[k]:
            assert end % 256 == 0 and int(p["pad"]) < 256
            k, within = k + 1, 0
        else:
            assert p["pad"] == 0
        pos = end
    assert pos == T and k == n
    for a, b_ in zip(items[:-1], items[1:]):                        # an item never mixes buckets
        assert len(set(pieces["bucket"][a:b_].tolist())) == 1


def _random_role(rng, n_max=40, log_max=20):
    n = int(rng.integers(1, n_max))
    sizes = [8 * max(1, int(2 ** x) // 8) for x in rng.uniform(3, log_max, n)]
    addr, descs = FAKE, []
    for nb in sizes:
        addr += 2 * int(rng.integers(0, 64))
        descs.append((addr, nb, 4, 1))
        addr += nb
    return sizes, descs


@pytest.mark.parametrize("seed", range(10))
def test_range_plans_concatenate_to_the_whole_plan(lib, oracle_mod, seed):
    """A role cut into runs of whole buckets: every range plan tiles its own slot exactly, and shifted
    by its stream offset the ranges reproduce the oracle's layout of the complete stream."""
    rng = np.random.default_rng(500 + seed)
    sizes, descs = _random_role(rng)
    B = 256 * int(rng.choice([1, 3, 16, 4096, 32768]))
    off, T, nbuckets = oracle_mod.layout(sizes, B)
    per = int(rng.integers(1, max(2, nbuckets // 2 + 1)))
    covered = np.zeros(T, dtype=np.int8)                       # 1 data, 2 padding
    src = np.full(T, -1, dtype=np.int64)                       # tensor address of every data byte
    first, n_ranges = 0, 0
    while first < nbuckets:
        plan = binding.Plan(descs, B, first, per)
        lo, hi = first * B, min((first + per) * B, T)
        assert (plan.first_bucket, plan.stream_begin, plan.whole_bytes, plan.whole_buckets) == (first, lo, T, nbuckets)
        assert (plan.total_bytes, plan.n_buckets) == (hi - lo, min(per, nbuckets - first))
        assert plan.offsets() == [int(x) for x in off]
        pieces, items = plan.pieces()
        pos = 0
        for p in pieces:
            o, n, pad = int(p["off"]), int(p["nbytes"]), int(p["pad"])
            assert o == pos                                     # data and padding tile the slot without a gap
            b = o // B
            assert int(p["bucket"]) == b and int(p["word0"]) == (o - b * B) // 8 and o + n + pad <= (b + 1) * B
            assert not covered[lo + o:lo + o + n + pad].any()
            covered[lo + o:lo + o + n] = 1
            covered[lo + o + n:lo + o + n + pad] = 2
            src[lo + o:lo + o + n] = int(p["tensor"]) + np.arange(n)
            pos = o + n + pad
        assert pos == hi - lo
        for a, b_ in zip(items[:-1], items[1:]):
            assert len(set(pieces["bucket"][a:b_].tolist())) == 1
        first += per
        n_ranges += 1
    assert n_ranges == -(-nbuckets // per)
    for k, n in enumerate(sizes):                             # data bytes sit where the oracle's layout puts them
        o = int(off[k])
        assert (covered[o:o + n] == 1).all() and np.array_equal(src[o:o + n], descs[k][0] + np.arange(n))
        assert (covered[o + n:(o + n + 255) // 256 * 256] == 2).all()
    assert int((covered == 1).sum()) == sum(sizes) and (covered != 0).all()
    with pytest.raises(binding.TmError) as e:
        binding.Plan(descs, B, nbuckets, 1)
    assert e.value.status == binding.TM_ERR_ARG


@pytest.mark.parametrize("seed", range(8))
def test_emit_records_tile_the_shards_exactly(lib, oracle_mod, seed):
    """The second destinations attached to the pack pieces: over all pieces (of one plan, or of the
    range plans of a role) they write every byte of every shard output exactly once, from the tensor
    byte the oracle's bounds name."""
    rng = np.random.default_rng(900 + seed)
    sizes, descs = _random_role(rng, n_max=30, log_max=19)
    n = len(sizes)
    cut = sorted(set(int(x) for x in rng.integers(0, n + 1, 3)) | {0, n})
    planes = [(a, b - a) for a, b in zip(cut[:-1], cut[1:]) if b > a][:3]
    D = int(rng.integers(1, 9))
    r = int(rng.integers(0, D))
    B = 256 * int(rng.choice([2, 64, 4096]))
    _, T, nbuckets = oracle_mod.layout(sizes, B)
    per = nbuckets if seed % 2 == 0 else max(1, nbuckets // 3)
    outs_base = [FAKE + (1 << 40) + (p << 36) + 2 * p for p in range(len(planes))]
    bounds = [oracle_mod.shard_bounds(sum(sizes[f:f + c]) // 4, r, D) for f, c in planes]
    written = [np.zeros((hi - lo) * 4, dtype=np.int64) - 1 for lo, hi in bounds]
    first = 0
    while first < nbuckets:
        plan = binding.Plan(descs, B, first, per)
        elems, need = binding.tm_plan_attach_shards(plan, planes, r, D, outs_base, [1 << 36] * len(planes), None, 0, 0)
        assert elems == [hi - lo for lo, hi in bounds] and need >= plan.workspace_bytes
        pieces, _ = plan.pieces()
        emits = plan.emits()
        assert emits.size == pieces.size
        for p, em in zip(pieces, emits):
            if em["len"] == 0:
                continue
            assert int(em["begin"]) + int(em["len"]) <= int(p["nbytes"]) and em["len"] % 4 == 0
            q = max(i for i, ob in enumerate(outs_base) if ob <= int(em["out"]))
            o = int(em["out"]) - outs_base[q]
            assert (written[q][o:o + int(em["len"])] == -1).all()
            written[q][o:o + int(em["len"])] = int(p["tensor"]) + int(em["begin"]) + np.arange(int(em["len"]))
        with pytest.raises(binding.TmError) as e:             # records computed, nothing uploaded
            binding.tm_state_pack_emit(plan, FAKE + (1 << 50), 1 << 40, None, 0)
        assert e.value.status == binding.TM_ERR_STATE
        first += per
    for (f, c), (lo, hi), w in zip(planes, bounds, written):
        flat = np.concatenate([descs[k][0] + np.arange(sizes[k]) for k in range(f, f + c)])
        assert np.array_equal(w, flat[lo * 4:hi * 4])


@pytest.mark.parametrize("seed", range(8))
def test_shard_plan_pieces_tile_the_outputs_exactly(lib, oracle_mod, seed):
    """Work list of a bound shard plan: the pieces write [0, (hi-lo)*e) of every flat buffer exactly
    once, from the tensor bytes the oracle's bounds name, never exceed the chunk size, and stay
    inside their tensor."""
    rng = np.random.default_rng(1300 + seed)
    planes, D = [], int(rng.integers(1, 70))
    r = int(rng.integers(0, D))
    for e in (4, 2, 8)[:int(rng.integers(1, 4))]:
        sizes, descs = _random_role(rng, n_max=25, log_max=19)
        planes.append([(a + (e << 44), nb, e, 0) for a, nb, _, _ in descs])
    sp = binding.ShardPlan(planes, r, D)
    flats = [FAKE + (1 << 50) + (p << 40) + 2 * int(rng.integers(0, 8)) for p in range(len(planes))]
    bounds = [oracle_mod.shard_bounds(sum(d[1] for d in pl) // pl[0][2], r, D) for pl in planes]
    assert sp.elems == [hi - lo for lo, hi in bounds]
    sp.bind(flats, [1 << 40] * len(planes), None, 0, 0)
    pieces, items, base = sp.pieces()
    chunk = binding.tm_options_get()["shard_chunk_bytes"]
    assert base == min(f for f, (lo, hi) in zip(flats, bounds) if hi > lo) if any(hi > lo for lo, hi in bounds) else True
    written = [np.zeros((hi - lo) * pl[0][2], dtype=np.int64) - 1 for (lo, hi), pl in zip(bounds, planes)]
    for p in pieces:
        addr, n = base + int(p["off"]), int(p["nbytes"])
        assert 0 < n <= chunk and p["pad"] == 0
        q = max(i for i, f in enumerate(flats) if f <= addr)
        o = addr - flats[q]
        assert (written[q][o:o + n] == -1).all()
        written[q][o:o + n] = int(p["tensor"]) + np.arange(n)
        assert any(d[0] <= int(p["tensor"]) and int(p["tensor"]) + n <= d[0] + d[1] for d in planes[q])
    for pl, (lo, hi), w in zip(planes, bounds, written):
        e = pl[0][2]
        flat = np.concatenate([d[0] + np.arange(d[1]) for d in pl])
        assert np.array_equal(w, flat[lo * e:hi * e])
    assert items[0] == 0 and items[-1] == pieces.size
    if pieces.size:
        with pytest.raises(binding.TmError) as ex:              # list built on the host only: nothing to launch with
            sp.extract(0)
        assert ex.value.status == binding.TM_ERR_STATE
    else:
        sp.extract(0)                                           # every shard empty: nothing to do


def test_options_round_trip_and_validation(lib):
    d = binding.tm_options_get()
    assert d["chunk_bytes"] == 256 * 1024 and d["shard_chunk_bytes"] == 64 * 1024 and d["wait_limit_ns"] == 2_000_000_000
    try:
        binding.tm_options_set(chunk_bytes=8192, small_bytes=1024)
        assert binding.tm_options_get()["chunk_bytes"] == 8192
        plan = binding.Plan(_descs([40000]), 1 << 20)
        pieces, _ = plan.pieces()
        assert pieces["nbytes"].tolist() == [8192, 8192, 8192, 8192, 40000 - 4 * 8192]
        for bad, code in ((dict(chunk_bytes=1000), binding.TM_ERR_ARG), (dict(chunk_bytes=4096 + 2), binding.TM_ERR_ALIGN),
                          (dict(wait_limit_ns=0), binding.TM_ERR_ARG), (dict(ring_ctas_per_sm=3), binding.TM_ERR_ARG),
                          (dict(group_max=0), binding.TM_ERR_ARG)):
            with pytest.raises(binding.TmError) as e:
                binding.tm_options_set(**bad)
            assert e.value.status == code
        assert binding.tm_options_get()["chunk_bytes"] == 8192     # a refused set changes nothing
    finally:
        binding.tm_options_set()
    assert binding.tm_options_get() == d


def test_plan_refuses_sizes_whose_sum_could_wrap(lib):
    big = [(FAKE, 1 << 46, 2, 0)] * 1025                          # 2^56 + 2^46 bytes of stream
    with pytest.raises(binding.TmError) as e:
        binding.Plan(big, 1 << 30)
    assert e.value.status == binding.TM_ERR_ARG
    with pytest.raises(binding.TmError) as e:
        binding.tm_shard_workspace(big, 0, 2)
    assert e.value.status == binding.TM_ERR_ARG


def test_lists_too_long_to_build_are_refused_before_any_allocation(lib):
    """Sizes that pass the per-tensor limits but would need hundreds of millions of pieces (a 64 TiB
    tensor in 256-byte buckets) are refused at once with TM_ERR_CAPACITY instead of exhausting host
    memory while the list grows."""
    import time
    huge = [(FAKE, 1 << 46, 4, 1)]
    t0 = time.perf_counter()
    for B in (256, 1 << 20, 1 << 35):
        with pytest.raises(binding.TmError) as e:
            binding.Plan(huge, B)
        assert e.value.status == binding.TM_ERR_CAPACITY
        with pytest.raises(binding.TmError) as e:
            binding.Plan(huge, B, 0, 1 << 30)
        assert e.value.status == binding.TM_ERR_CAPACITY
    small_range = binding.Plan(huge, 1 << 30, 5, 2)               # two buckets of it are a reasonable plan
    assert small_range.total_bytes == 2 << 30 and small_range.stream_begin == 5 << 30
    sp = binding.ShardPlan([huge], 0, 2)
    assert sp.out_bytes == [1 << 45]
    with pytest.raises(binding.TmError) as e:
        sp.bind([FAKE + (1 << 60)], [1 << 62], None, 0, 0)
    assert e.value.status == binding.TM_ERR_CAPACITY
    h = ctypes.c_void_p()
    arr = binding.make_descs(huge)
    assert lib.tm_xfer_create(arr, 1, 1 << 20, 1, 2, ctypes.byref(h)) == binding.TM_ERR_ARG          # over 2^20 waves
    assert lib.tm_xfer_create(arr, 1, 1 << 30, 1024, 2, ctypes.byref(h)) == binding.TM_ERR_CAPACITY  # 64 waves, too many pieces
    assert not h.value
    assert time.perf_counter() - t0 < 5.0


def test_transfer_endpoint_geometry_and_validation(lib, oracle_mod):
    """tm_xfer_create / tm_xfer_query are host-only: waves, slot and ring sizes follow from the
    oracle's layout; bad geometry is refused."""
    rng = np.random.default_rng(77)
    sizes, descs = _random_role(rng)
    B = 4096
    _, T, nb = oracle_mod.layout(sizes, B)
    arr = binding.make_descs(descs)
    for per_wave, n_slots in ((1, 1), (3, 2), (nb + 5, 4)):
        h = ctypes.c_void_p()
        assert lib.tm_xfer_create(arr, len(arr), B, per_wave, n_slots, ctypes.byref(h)) == binding.TM_OK
        nw, sb, rb, wb, nbk = ctypes.c_uint32(), ctypes.c_uint64(), ctypes.c_uint64(), ctypes.c_uint64(), ctypes.c_uint64()
        assert lib.tm_xfer_query(h, ctypes.byref(nw), ctypes.byref(sb), ctypes.byref(rb), ctypes.byref(wb), ctypes.byref(nbk)) == 0
        assert (nw.value, sb.value, rb.value, nbk.value) == (-(-nb // per_wave), per_wave * B, n_slots * per_wave * B, nb)
        assert wb.value % 256 == 0 and wb.value >= 512 * nw.value
        # not bound yet: running a side is refused, nothing is launched
        t = binding.TmTransport()
        assert lib.tm_xfer_send(h, ctypes.byref(t), None, None, 3, None) == binding.TM_ERR_STATE
        lib.tm_xfer_destroy(h)
    h = ctypes.c_void_p()
    for per_wave, n_slots, code in ((0, 2, binding.TM_ERR_ARG), (2, 0, binding.TM_ERR_ARG), (2, 65, binding.TM_ERR_ARG),
                                    (1 << 40, 2, binding.TM_ERR_ARG)):
        assert lib.tm_xfer_create(arr, len(arr), B, per_wave, n_slots, ctypes.byref(h)) == code and not h.value
    assert lib.tm_xfer_create(arr, len(arr), 100, 2, 2, ctypes.byref(h)) == binding.TM_ERR_ALIGN
    assert lib.tm_xfer_create(None, 0, B, 2, 2, ctypes.byref(h)) == binding.TM_ERR_ARG


def test_shard_plan_and_attach_validation_without_a_device(lib):
    """Argument checks of the reusable shard plan and of the shard attachment run before any device
    work, so they can be exercised with no workspace at all."""
    plane = _descs([4096, 8192, 4096], elem=4)                       # three fp32 tensors, 16 MiB apart
    sp = binding.ShardPlan([plane], 0, 2)
    assert sp.elems == [2048] and sp.out_bytes == [8192]
    far = FAKE + (1 << 40)
    cases = [
        ([far + 1], [8192], binding.TM_ERR_ALIGN),                   # odd output address
        ([far], [8191], binding.TM_ERR_CAPACITY),                    # output too small
        ([plane[0][0] + 64], [1 << 20], binding.TM_ERR_OVERLAP),     # output inside a source tensor
        ([0], [8192], binding.TM_ERR_ARG),                           # missing output
    ]
    for flats, caps, code in cases:
        with pytest.raises(binding.TmError) as e:
            sp.bind(flats, caps, None, 0, 0)
        assert e.value.status == code, (flats, caps)
    two = binding.ShardPlan([plane, _descs([4096], elem=2, base=FAKE + (1 << 36))], 1, 2)
    with pytest.raises(binding.TmError) as e:                        # the two outputs overlap each other
        two.bind([far, far + 100], [1 << 20, 1 << 20], None, 0, 0)
    assert e.value.status == binding.TM_ERR_OVERLAP
    with pytest.raises(binding.TmError) as e:                        # never bound: nothing to run
        binding.ShardPlan([plane], 0, 2).extract(0)
    assert e.value.status == binding.TM_ERR_STATE
    for bad in ((0, 0), (2, 2)):
        with pytest.raises(binding.TmError) as e:
            binding.ShardPlan([plane], *bad)
        assert e.value.status == binding.TM_ERR_RANK
    with pytest.raises(binding.TmError) as e:                        # mixed element sizes inside one plane
        binding.ShardPlan([plane + _descs([64], elem=2, base=FAKE + (1 << 37))], 0, 2)
    assert e.value.status == binding.TM_ERR_DTYPE

    plan = binding.Plan(plane, 4096)
    ok_out, cap = [far], [1 << 20]
    for planes, outs, caps, code in (
            ([(0, 3)], [plane[1][0]], cap, binding.TM_ERR_OVERLAP),  # shard output on top of a tensor
            ([(0, 3)], [far + 1], cap, binding.TM_ERR_ALIGN),
            ([(0, 3)], ok_out, [100], binding.TM_ERR_CAPACITY),
            ([(0, 4)], ok_out, cap, binding.TM_ERR_ARG),             # plane runs past the descriptors
            ([(0, 2), (1, 2)], [far, far + (1 << 30)], [1 << 20] * 2, binding.TM_ERR_ARG),   # planes overlap
            ([(0, 0)], ok_out, cap, binding.TM_ERR_ARG)):            # empty plane
        with pytest.raises(binding.TmError) as e:
            binding.tm_plan_attach_shards(plan, planes, 0, 2, outs, caps, None, 0, 0)
        assert e.value.status == code, (planes, outs)
    elems, need = binding.tm_plan_attach_shards(plan, [(0, 3)], 1, 2, ok_out, cap, None, 0, 0)
    assert elems == [2048] and need > plan.workspace_bytes
    emits = plan.emits()
    assert int(emits["len"].sum()) == 8192                           # the shard's bytes, each named once


def test_random_arguments_never_crash_the_host_entry_points(lib, oracle_mod):
    """Random, mostly unreasonable arguments to every host-only entry point: the call either succeeds
    with a layout that agrees with the oracle, or returns a negative status — it never crashes, and
    never reports sizes that wrapped around."""
    rng = np.random.default_rng(2024)
    sizes_pool = [0, 1, 2, 6, 254, 256, 258, 4096, (1 << 20) + 2, 1 << 33, (1 << 46), (1 << 46) + 8, (1 << 63)]
    for trial in range(300):
        n = int(rng.integers(0, 6))
        descs = []
        for k in range(n):
            e = int(rng.choice([2, 4, 8, 8, 4, 2, 3, 0, 16]))
            nb = int(rng.choice(sizes_pool))
            ptr = int(rng.choice([FAKE + (k << 47), FAKE + (k << 47) + 1, 0, FAKE]))   # FAKE twice: overlapping tensors
            descs.append((ptr, nb, e, 0))
        B = int(rng.choice([0, 100, 256, 768, 1 << 20, 1 << 35, (1 << 35) + 256]))
        first, count = int(rng.integers(0, 5)), int(rng.integers(0, 4))
        ok_sizes = all(d[1] > 0 and d[2] in (2, 4, 8) and d[1] % d[2] == 0 and d[1] <= (1 << 46) and d[0] and d[0] % 2 == 0
                       for d in descs)
        try:
            plan = binding.Plan(descs, B, first, count) if trial % 2 else binding.Plan(descs, B)
        except binding.TmError as e:
            assert e.status < 0
            plan = None
        if plan is not None:
            assert n > 0 and ok_sizes and B % 256 == 0 and 0 < B <= (1 << 35)
            off, T, nbk = oracle_mod.layout([d[1] for d in descs], B)
            assert plan.offsets() == [int(x) for x in off] and (plan.whole_bytes, plan.whole_buckets) == (T, nbk)
            assert plan.total_bytes <= T and plan.n_buckets <= nbk
            pieces, items = plan.pieces()
            assert int(pieces["nbytes"].astype(np.uint64).sum() + pieces["pad"].astype(np.uint64).sum()) == plan.total_bytes
        r, D = int(rng.integers(0, 4)), int(rng.integers(0, 4))
        try:
            sp = binding.ShardPlan([descs], r, D) if n else None
            if sp is not None:
                e0 = descs[0][2]
                assert ok_sizes and all(d[2] == e0 for d in descs) and D > 0 and r < D
                N = sum(d[1] for d in descs) // e0
                assert sp.elems == [oracle_mod.shard_bounds(N, r, D)[1] - oracle_mod.shard_bounds(N, r, D)[0]]
                try:
                    sp.bind([FAKE + (1 << 60)], [1 << 62], None, 0, 0)        # host-only: the list is only built
                    p2, _, _ = sp.pieces()
                    assert int(p2["nbytes"].astype(np.uint64).sum()) == sp.out_bytes[0]
                except (binding.TmError, MemoryError) as e:
                    assert not isinstance(e, binding.TmError) or e.status < 0
        except binding.TmError as e:
            assert e.status < 0
