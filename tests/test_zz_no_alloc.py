"""tm_shard_extract_static: the shard extract for callers that cannot allocate device memory (a
recovery hook running while the framework's allocator owns the GPU, code that must not call
cudaMalloc, a plugin without an allocator).  It keeps its work list in a fixed 1 MiB array inside
the library instead of a caller workspace, so its output must equal tm_shard_extract's byte for
byte — also on a second call, when the array still holds the first call's list.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test; it also passes when run alone in a fresh process."""
import numpy as np
import pytest
import torch

from paper_2412_12636_b200 import binding, layouts
from paper_2412_12636_b200.mover import ShardExtractor

pytestmark = pytest.mark.gpu

GUARD = 512


def _oracle_shard(oracle, state, indices, r, D):
    host = [state.host_bytes(i) for i in indices]
    return oracle.shard(host, [h.size for h in host], state.specs[indices[0]].elem_size, r, D)


def _both_ways(descs, r, D, misalign=0):
    """(bytes from tm_shard_extract, bytes from tm_shard_extract_static, guard bands intact)."""
    stream = torch.cuda.current_stream().cuda_stream
    ex = ShardExtractor(descs, r, D)
    ref = ex.alloc_out()
    n_ref = ex.extract(ref)
    whole = torch.full((ex.out_bytes + 2 * GUARD + 16,), 0x5A, dtype=torch.uint8, device="cuda")
    out = whole[GUARD + misalign:GUARD + misalign + ex.out_bytes]
    n = binding.tm_shard_extract_static(descs, r, D, out.data_ptr(), ex.out_bytes, stream)
    torch.cuda.synchronize()
    assert n == n_ref == ex.hi - ex.lo
    intact = bool((whole[:GUARD + misalign] == 0x5A).all()) and bool((whole[GUARD + misalign + ex.out_bytes:] == 0x5A).all())
    return ref.cpu().numpy(), out.cpu().numpy(), intact


def test_static_scratch_shard_matches_workspace_shard_twice_in_a_row(oracle_mod):
    assert torch.cuda.is_available()
    binding.load_library()
    torch.cuda.set_device(0)
    launches = binding.tm_launch_count()
    # first call: a long list (config 0's fp32 master plane, mid-tensor shard boundaries)
    cfg = layouts.role_config(0)
    state = layouts.materialize(cfg, "cuda")
    master = state.plane_indices(layouts.PLANE_MASTER)
    plane = [state.descs()[i] for i in master]
    ref, got, intact = _both_ways(plane, 1, 3)
    assert ref.size == 4 * (2 * 1_842_176 // 3 - 1_842_176 // 3) and intact
    assert np.array_equal(ref, got)
    # and against the CPU oracle directly: the two entry points share the host planner, so agreeing
    # with each other would not show a mistake made there
    assert np.array_equal(got, _oracle_shard(oracle_mod, state, master, 1, 3))
    # second call, straight after: a shorter list of awkward pieces at 2-byte-granular addresses, so
    # most of the first call's list is still sitting in the array behind it
    odd = layouts.materialize_adversarial(layouts.odd_specs(7, n_tensors=12), "cuda", seed=7)
    for e in (4, 2, 8):
        idx = odd.elem_size_indices(e)
        if idx:
            ref, got, intact = _both_ways([odd.descs()[i] for i in idx], 2, 5, misalign=6)
            assert intact and np.array_equal(ref, got)
            assert np.array_equal(got, _oracle_shard(oracle_mod, odd, idx, 2, 5))
    # and the first request again
    ref, got, intact = _both_ways(plane, 1, 3)
    assert intact and np.array_equal(ref, got)
    assert np.array_equal(got, _oracle_shard(oracle_mod, state, master, 1, 3))
    assert binding.tm_launch_count() > launches


def test_static_scratch_calls_from_two_threads_on_one_stream(oracle_mod):
    """The entry point documents that host threads sharing ONE stream may call it concurrently: the
    clear / copy / copy / launch sequence of a call runs under one lock, so every kernel reads the
    list its own call wrote.  Two threads issue different requests on the same stream many times."""
    import threading
    binding.load_library()
    torch.cuda.set_device(0)
    state = layouts.materialize(layouts.role_config(0), "cuda")
    stream = torch.cuda.current_stream().cuda_stream
    jobs = []
    for plane, r, D in ((layouts.PLANE_MASTER, 1, 3), (layouts.PLANE_V, 4, 5)):
        idx = state.plane_indices(plane)
        expect = _oracle_shard(oracle_mod, state, idx, r, D)
        descs = binding.make_descs([state.descs()[i] for i in idx])
        outs = [torch.zeros(expect.size, dtype=torch.uint8, device="cuda") for _ in range(20)]
        jobs.append((descs, r, D, outs, expect))
    errors = []

    def work(job):
        descs, r, D, outs, expect = job
        try:
            torch.cuda.set_device(0)
            for out in outs:
                binding.tm_shard_extract_static(descs, r, D, out.data_ptr(), out.numel(), stream)
        except Exception as e:
            errors.append(e)

    threads = [threading.Thread(target=work, args=(j,)) for j in jobs]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    assert not errors, errors
    for descs, r, D, outs, expect in jobs:
        for out in outs:
            assert np.array_equal(out.cpu().numpy(), expect)


def test_static_scratch_refuses_what_does_not_fit():
    binding.load_library()
    stream = torch.cuda.current_stream().cuda_stream
    launches = binding.tm_launch_count()
    fake = 0x7F00_0000_0000                     # never dereferenced: the request is refused on the host
    huge = [(fake, 64 << 30, 4, 1)]             # a 64 GiB shard needs ~1M pieces of 64 KiB
    with pytest.raises(binding.TmError) as e:
        binding.tm_shard_extract_static(huge, 0, 1, fake + (128 << 30), 64 << 30, stream)
    assert e.value.status == binding.TM_ERR_CAPACITY
    with pytest.raises(binding.TmError) as e:   # the usual argument checks still apply
        binding.tm_shard_extract_static([(fake, 1024, 4, 1)], 3, 2, fake + (1 << 30), 1024, stream)
    assert e.value.status == binding.TM_ERR_RANK
    assert binding.tm_launch_count() == launches
