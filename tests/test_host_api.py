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
