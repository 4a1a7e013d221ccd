"""GPU parity of the fused and reusable forms: pack that emits the shards from the same staged copy
(whole plans and range plans), reusable shard plans, buckets that live in pinned host memory, and
the kernels' bounded waits made to expire.  Everything is compared with the CPU oracle bit for bit."""
import numpy as np
import pytest
import torch

from paper_2412_12636_b200 import binding, layouts
from paper_2412_12636_b200.mover import RoleMover, ShardPlanMover, WaveMover

import gpu_util as G

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _cuda():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    binding.load_library()
    torch.cuda.set_device(0)
    yield


def _adversarial_by_elem_size(n, max_log2, seed):
    specs = sorted(layouts.adversarial_specs(n, max_log2=max_log2), key=lambda s: s.elem_size)
    state = layouts.materialize_adversarial(specs, "cuda", seed=seed)
    runs, k = [], 0
    for e in (2, 4, 8):
        c = sum(1 for s in specs if s.elem_size == e)
        runs.append((k, c))
        k += c
    return state, runs


def _expected_shards(oracle, host, state, planes, r, D):
    out = []
    for first, count in planes:
        sub = host[first:first + count]
        out.append(oracle.shard(sub, [h.size for h in sub], state.specs[first].elem_size, r, D))
    return out


@pytest.mark.parametrize("case", ["cfg0-r1of2", "cfg0-r2of3-small-buckets", "adv-r5of7", "adv-r63of64", "adv-D>N"])
def test_range_plans_pack_emit_through_a_slot_ring(oracle_mod, case):
    """The role travels as runs of whole buckets through two recycled slots; every run's launch also
    writes its part of the three shards.  Stream, checksums and shards must equal the oracle's."""
    if case.startswith("cfg0"):
        cfg = layouts.role_config(0)
        state = layouts.materialize(cfg, "cuda")
        P = len(cfg.model)
        planes = [(P, P), (2 * P, P), (3 * P, P)]
        r, D, B, per = (1, 2, cfg.bucket_bytes, 3) if case == "cfg0-r1of2" else (2, 3, 256 * 1024, 7)
    else:
        state, planes = _adversarial_by_elem_size(700, 18, seed=13)
        r, D = {"adv-r5of7": (5, 7), "adv-r63of64": (63, 64), "adv-D>N": (10 ** 9 - 1, 10 ** 9)}[case]
        B, per = 1 << 20, 5
    host = G.host_tensors(state)
    exp_stream, exp_cks = oracle_mod.pack(host, B)
    exp_shards = _expected_shards(oracle_mod, host, state, planes, r, D)
    descs = state.descs()
    outs = [G.guarded(e.size) for e in exp_shards]
    slots = [G.guarded(per * B) for _ in range(2)]
    cks = torch.zeros(exp_cks.size, dtype=torch.int64, device="cuda")
    received = torch.empty(exp_stream.size, dtype=torch.uint8, device="cuda")
    first, i = 0, 0
    while first < exp_cks.size:
        m = RoleMover(descs, B, first_bucket=first, n_buckets=per)
        got = m.attach_shards(planes, r, D, outs=[o[1] for o in outs])
        assert [g.numel() for g in got] == [e.size for e in exp_shards]
        whole, slot = slots[i % 2]
        slot.fill_(0x77)
        launches = binding.tm_launch_count()
        m.pack_emit(slot, cks[first:first + m.n_buckets])
        torch.cuda.synchronize()
        assert binding.tm_launch_count() == launches + 1 and m.status() == 0
        assert G.guards_intact(whole, per * B) and bool((slot[m.total_bytes:] == 0x77).all())
        lo = m.plan.stream_begin
        received[lo:lo + m.total_bytes].copy_(slot[:m.total_bytes])
        first += per
        i += 1
    assert np.array_equal(received.cpu().numpy(), exp_stream)
    assert np.array_equal(G.u64(cks), exp_cks)
    for (whole, out), e in zip(outs, exp_shards):
        assert np.array_equal(out.cpu().numpy(), e), G._first_diff(out.cpu().numpy(), e)
        assert G.guards_intact(whole, e.size)


@pytest.mark.parametrize("misalign", [0, 2, 6, 10])
def test_pack_emit_every_output_alignment(oracle_mod, misalign):
    # one bulk tensor, shard boundaries mid-stage; shard output at every 2-byte-granular alignment class
    n = 3 * 32768 + 4100
    arena = torch.randint(0, 256, (4 * n + 64,), dtype=torch.uint8, device="cuda",
                          generator=torch.Generator("cuda").manual_seed(misalign + 1))
    for src_mis in (0, 4):
        t = arena[src_mis:src_mis + 4 * n]
        spec = layouts.TensorSpec("t", n, torch.float32, 1, 0)
        state = layouts.RoleState("one", [spec], [t], 1 << 20, 0, 1, arena)
        host = G.host_tensors(state)
        exp_stream, exp_cks = oracle_mod.pack(host, 1 << 20)
        for r, D in ((0, 1), (1, 3), (6, 7)):
            expect = oracle_mod.shard(host, [4 * n], 4, r, D)
            m = RoleMover(state.descs(), 1 << 20)
            whole, out = G.guarded(expect.size + 16)
            out = out[misalign:misalign + expect.size]
            m.attach_shards([(0, 1)], r, D, outs=[out])
            wb, buckets = G.guarded(m.total_bytes)
            cks = m.alloc_checksums()
            m.pack_emit(buckets, cks)
            torch.cuda.synchronize()
            assert m.status() == 0
            assert np.array_equal(buckets.cpu().numpy(), exp_stream) and np.array_equal(G.u64(cks), exp_cks)
            assert np.array_equal(out.cpu().numpy(), expect), (src_mis, r, D, G._first_diff(out.cpu().numpy(), expect))
            assert bool((whole[:G.GUARD + misalign] == G.GUARD_BYTE).all())
            assert bool((whole[G.GUARD + misalign + expect.size:] == G.GUARD_BYTE).all())
            assert G.guards_intact(wb, m.total_bytes)


def test_shard_plan_extract_and_insert_match_the_oracle(oracle_mod):
    cfg = layouts.role_config(0)
    st0 = layouts.materialize(cfg, "cuda")
    adv = layouts.materialize_adversarial(layouts.adversarial_specs(400, max_log2=17), "cuda", seed=31)
    cases = [
        (st0, [st0.plane_indices(p) for p in (layouts.PLANE_MASTER, layouts.PLANE_M, layouts.PLANE_V)], 1, 2),
        (adv, [adv.elem_size_indices(e) for e in (4, 2, 8)], 17, 64),
        (adv, [adv.elem_size_indices(e) for e in (8, 4)], 10 ** 9 - 1, 10 ** 9),    # one-element shards
        (adv, [adv.elem_size_indices(e) for e in (8, 4)], 0, 10 ** 9),              # empty shards: no launch
    ]
    for st, planes, r, D in cases:
        plane_descs = [st.descs_of(idx) for idx in planes]
        host = [[st.host_bytes(i) for i in idx] for idx in planes]
        expect = [oracle_mod.shard(h, [x.size for x in h], st.specs[idx[0]].elem_size, r, D)
                  for h, idx in zip(host, planes)]
        bufs = [G.guarded(e.size + 16) for e in expect]
        flats = [b[1][2 * p:2 * p + e.size] for p, (b, e) in enumerate(zip(bufs, expect))]   # 2-byte-granular outputs
        sp = ShardPlanMover(plane_descs, r, D, flats=flats)
        assert sp.out_bytes == [e.size for e in expect]
        launches = binding.tm_launch_count()
        for _ in range(3):                                   # reuse: no host work between launches
            sp.extract()
        torch.cuda.synchronize()
        assert binding.tm_launch_count() == launches + (3 if any(sp.out_bytes) else 0)
        if any(sp.out_bytes):
            assert sp.status() == 0
        for p, ((whole, _), f, e) in enumerate(zip(bufs, flats, expect)):
            assert np.array_equal(f.cpu().numpy(), e)
            assert bool((whole[:G.GUARD + 2 * p] == G.GUARD_BYTE).all())
            assert bool((whole[G.GUARD + 2 * p + e.size:] == G.GUARD_BYTE).all())
        # insert: new data into [lo, hi) of every plane, everything else untouched
        gen = torch.Generator("cuda").manual_seed(r + 7)
        data = [torch.randint(0, 256, (e.size,), dtype=torch.uint8, device="cuda", generator=gen) for e in expect]
        before = st.arena.clone() if st.arena is not None else None
        sp.rebind(data)
        sp.insert()
        torch.cuda.synchronize()
        for idx, h, d in zip(planes, host, data):
            hh = [x.copy() for x in h]
            oracle_mod.shard_insert(hh, [x.size for x in hh], st.specs[idx[0]].elem_size, r, D, d.cpu().numpy())
            for i, x in zip(idx, hh):
                assert np.array_equal(st.host_bytes(i), x)
        if before is not None:
            mask = torch.ones_like(before, dtype=torch.bool)
            for idx in planes:
                for i in idx:
                    o = st.tensors[i].data_ptr() - st.arena.data_ptr()
                    mask[o:o + st.specs[i].nbytes] = False
            assert torch.equal(st.arena[mask], before[mask])
    dup = [st0.descs_of(st0.plane_indices(layouts.PLANE_M))[:2] * 2]          # the same tensors twice: insert refused
    sp = ShardPlanMover(dup, 0, 1)
    launches = binding.tm_launch_count()
    with pytest.raises(binding.TmError) as e:
        sp.insert()
    assert e.value.status == binding.TM_ERR_OVERLAP and binding.tm_launch_count() == launches


def test_buckets_in_pinned_host_memory(oracle_mod):
    """Host-memory tier: the packed buffer is mapped pinned host memory, so pack writes the buckets
    over PCIe itself and unpack + verify reads them from there; tensors and checksums stay on the GPU."""
    for state, B in ((layouts.materialize(layouts.role_config(0), "cuda"), 1 << 20),
                     (layouts.materialize_adversarial(layouts.adversarial_specs(300, max_log2=16), "cuda", seed=3), 1 << 18)):
        host = G.host_tensors(state)
        exp_stream, exp_cks = oracle_mod.pack(host, B)
        m = RoleMover(state.descs(), B)
        pinned = torch.full((m.total_bytes + 2 * G.GUARD,), G.GUARD_BYTE, dtype=torch.uint8).pin_memory()
        assert pinned.data_ptr() % 256 == 0
        hb = pinned[G.GUARD:G.GUARD + m.total_bytes]
        cks = m.alloc_checksums()
        m.pack(hb, cks)
        torch.cuda.synchronize()
        assert m.status() == 0
        assert np.array_equal(hb.numpy(), exp_stream) and np.array_equal(G.u64(cks), exp_cks)
        assert bool((pinned[:G.GUARD] == G.GUARD_BYTE).all()) and bool((pinned[G.GUARD + m.total_bytes:] == G.GUARD_BYTE).all())
        target = layouts.blank_like(state)
        um = RoleMover(target.descs(), B)
        got = um.alloc_checksums()
        um.unpack_verify(hb, got)
        torch.cuda.synchronize()
        assert um.status() == 0 and np.array_equal(G.u64(got), exp_cks)
        for k in range(len(host)):
            assert np.array_equal(target.host_bytes(k), host[k])


def test_ring_kernel_waits_made_to_expire_leave_everything_in_bounds(oracle_mod):
    """The ring kernels' own producer, store and consumer waits are made to run out in the middle of
    real work: with a limit of 1 ns (below the timer's resolution: a wait that is not satisfied at
    once gives up at once — loads are then still in flight when the roles give up) and of 2 µs (about a
    load's latency: some waits expire, some do not).  Every launch must return, report TM_ERR_TIMEOUT
    through the status word (or finish), write nothing out of bounds, and leave the device fit for
    the next, normal launch, which must be exact."""
    cfg = layouts.role_config(0)
    state = layouts.materialize(cfg, "cuda")
    exp_stream, exp_cks = oracle_mod.pack(G.host_tensors(state), cfg.bucket_bytes)
    seen = {}
    for limit in (1, 2000):
        try:
            binding.tm_options_set(wait_limit_ns=limit)
            hasty = RoleMover(state.descs(), cfg.bucket_bytes)
        finally:
            binding.tm_options_set()
        whole, buckets = G.guarded(hasty.total_bytes)
        cks = hasty.alloc_checksums()
        seen[limit] = set()
        for _ in range(5):
            hasty.pack(buckets, cks)
            seen[limit].add(hasty.status())
            assert G.guards_intact(whole, hasty.total_bytes)
        assert seen[limit] <= {0, binding.TM_ERR_TIMEOUT}
        if seen[limit] == {0}:                                    # every wait happened to succeed at once
            assert np.array_equal(buckets.cpu().numpy(), exp_stream)
    assert binding.TM_ERR_TIMEOUT in seen[1]                      # the give-up paths really ran
    normal = RoleMover(state.descs(), cfg.bucket_bytes)
    normal.pack(buckets, cks)
    torch.cuda.synchronize()
    assert normal.status() == 0 and G.guards_intact(whole, normal.total_bytes)
    assert np.array_equal(buckets.cpu().numpy(), exp_stream) and np.array_equal(G.u64(cks), exp_cks)
    # the same for the receiving side and the shard gather, on a layout whose tensors are misaligned
    # (re-aligned stages, out ring): targets live in one arena, so a stray write would show
    adv = layouts.materialize_adversarial(layouts.adversarial_specs(300, max_log2=17), "cuda", seed=41)
    host = G.host_tensors(adv)
    stream_a, cks_a = oracle_mod.pack(host, 1 << 20)
    received = torch.from_numpy(stream_a).cuda()
    target = layouts.blank_like(adv)
    idx = adv.elem_size_indices(4)
    exp_shard = oracle_mod.shard([host[i] for i in idx], [host[i].size for i in idx], 4, 3, 5)
    sw, sout = G.guarded(exp_shard.size)
    got = torch.zeros(cks_a.size, dtype=torch.int64, device="cuda")
    seen = set()
    for limit in (1, 2000):
        try:
            binding.tm_options_set(wait_limit_ns=limit)
            hasty_rx = RoleMover(target.descs(), 1 << 20)
            hasty_sp = ShardPlanMover([adv.descs_of(idx)], 3, 5, flats=[sout])
        finally:
            binding.tm_options_set()
        for _ in range(5):
            hasty_rx.unpack_verify(received, got)
            hasty_sp.extract()
            seen |= {hasty_rx.status(), hasty_sp.status()}
            assert G.guards_intact(sw, exp_shard.size)
    assert seen <= {0, binding.TM_ERR_TIMEOUT} and binding.TM_ERR_TIMEOUT in seen
    covered = torch.zeros(target.arena.numel(), dtype=torch.bool, device="cuda")
    for t, spec in zip(target.tensors, target.specs):
        o = t.data_ptr() - target.arena.data_ptr()
        covered[o:o + spec.nbytes] = True
    assert bool((target.arena[~covered] == 0xA5).all())          # nothing written between the tensors
    rx = RoleMover(target.descs(), 1 << 20)
    rx.unpack_verify(received, got)
    sp = ShardPlanMover([adv.descs_of(idx)], 3, 5, flats=[sout])
    sp.extract()
    torch.cuda.synchronize()
    assert rx.status() == 0 and sp.status() == 0 and np.array_equal(G.u64(got), cks_a)
    for k in range(len(host)):
        assert np.array_equal(target.host_bytes(k), host[k])
    assert np.array_equal(sout.cpu().numpy(), exp_shard) and G.guards_intact(sw, exp_shard.size)


def test_step_captured_in_a_cuda_graph_replays_exactly(oracle_mod):
    """pack, checksum, unpack+verify and the plan-based shard extract enqueue only stream work once
    their plans are uploaded, so the whole step can be captured in a CUDA graph.  The replayed graph
    must give the oracle's results for whatever the source tensors hold at replay time."""
    cfg = layouts.role_config(0)
    state = layouts.materialize(cfg, "cuda")
    target = layouts.blank_like(state)
    mover, unmover = RoleMover(state.descs(), cfg.bucket_bytes), RoleMover(target.descs(), cfg.bucket_bytes)
    whole, buckets = G.guarded(mover.total_bytes)
    fused, alone, received = mover.alloc_checksums(), mover.alloc_checksums(), mover.alloc_checksums()
    planes = [target.descs_of(target.plane_indices(p)) for p in (layouts.PLANE_MASTER, layouts.PLANE_M, layouts.PLANE_V)]
    sp = ShardPlanMover(planes, cfg.shard_r, cfg.shard_D)

    def step():
        mover.pack(buckets, fused)
        mover.checksum(buckets, alone)
        unmover.unpack_verify(buckets, received)
        sp.extract()

    step()                                   # first launches outside the capture (one-time kernel attributes)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for trial in range(2):
        for t in state.tensors:              # new contents: the graph must read the tensors, not a snapshot
            layouts.tensor_bytes(t).random_(0, 256, generator=torch.Generator("cuda").manual_seed(trial * 7919 + t.numel()))
        buckets.fill_(0xEE)
        launches = binding.tm_launch_count()
        graph.replay()
        torch.cuda.synchronize()
        assert binding.tm_launch_count() == launches          # replayed by the driver, not launched by the library
        host = G.host_tensors(state)
        exp_stream, exp_cks = oracle_mod.pack(host, cfg.bucket_bytes)
        assert np.array_equal(buckets.cpu().numpy(), exp_stream) and G.guards_intact(whole, mover.total_bytes)
        for c in (fused, alone, received):
            assert np.array_equal(G.u64(c), exp_cks)
        for k in range(len(host)):
            assert np.array_equal(target.host_bytes(k), host[k])
        idxs = [state.plane_indices(p) for p in (layouts.PLANE_MASTER, layouts.PLANE_M, layouts.PLANE_V)]
        for idx, out in zip(idxs, sp.flats):
            sub = [host[i] for i in idx]
            assert np.array_equal(out.cpu().numpy(), oracle_mod.shard(sub, [h.size for h in sub], 4, cfg.shard_r, cfg.shard_D))
    assert mover.status() == 0 and unmover.status() == 0 and sp.status() == 0


@pytest.mark.parametrize("case", ["cfg0", "adv", "adv-ranges"])
def test_unpack_emit_gives_tensors_checksums_and_shards_from_one_read(oracle_mod, case):
    """The joiner's fused form: one launch over the received buckets scatters the tensors, recomputes
    the checksums of what arrived and fills the flat shard buffers."""
    if case == "cfg0":
        cfg = layouts.role_config(0)
        state = layouts.materialize(cfg, "cuda")
        P = len(cfg.model)
        planes, r, D, B = [(P, P), (2 * P, P), (3 * P, P)], 1, 2, cfg.bucket_bytes
    else:
        state, planes = _adversarial_by_elem_size(600, 18, seed=23)      # destinations at 2-byte-granular addresses
        r, D, B = 5, 7, 1 << 20
    host = G.host_tensors(state)
    exp_stream, exp_cks = oracle_mod.pack(host, B)
    exp_shards = _expected_shards(oracle_mod, host, state, planes, r, D)
    received = torch.from_numpy(exp_stream).cuda()
    received[7] ^= 0x40 if exp_stream.size > 7 else 0                     # damaged on the way: checksums must show it
    exp_received = oracle_mod.checksum(received.cpu().numpy(), B)
    target = layouts.blank_like(state)
    outs = [G.guarded(e.size + 16) for e in exp_shards]
    flats = [o[1][2 * p:2 * p + e.size] for p, (o, e) in enumerate(zip(outs, exp_shards))]
    got = torch.zeros(exp_cks.size, dtype=torch.int64, device="cuda")
    per = exp_cks.size if case != "adv-ranges" else 3
    first, launches = 0, binding.tm_launch_count()
    while first < exp_cks.size:
        m = RoleMover(target.descs(), B, first_bucket=first, n_buckets=per) if case == "adv-ranges" else \
            RoleMover(target.descs(), B)
        m.attach_shards(planes, r, D, outs=flats)
        lo = m.plan.stream_begin
        m.unpack_emit(received[lo:lo + m.total_bytes], got[first:first + m.n_buckets])
        torch.cuda.synchronize()
        assert m.status() == 0
        first += per
    assert binding.tm_launch_count() == launches + -(-exp_cks.size // per)
    assert np.array_equal(G.u64(got), exp_received) and not np.array_equal(exp_received, exp_cks)
    damaged = oracle_mod.unpack(received.cpu().numpy(), [h.size for h in host])
    if target.arena is not None:
        exp_arena = np.full(target.arena.numel(), 0xA5, dtype=np.uint8)
        for t, h in zip(target.tensors, damaged):
            o = t.data_ptr() - target.arena.data_ptr()
            exp_arena[o:o + h.size] = h
        assert np.array_equal(target.arena.cpu().numpy(), exp_arena)
    else:
        for k, h in enumerate(damaged):
            assert np.array_equal(target.host_bytes(k), h)
    exp_from_received = _expected_shards(oracle_mod, damaged, state, planes, r, D)
    for p, ((whole, _), f, e) in enumerate(zip(outs, flats, exp_from_received)):
        assert np.array_equal(f.cpu().numpy(), e), G._first_diff(f.cpu().numpy(), e)
        assert bool((whole[:G.GUARD + 2 * p] == G.GUARD_BYTE).all())
        assert bool((whole[G.GUARD + 2 * p + e.size:] == G.GUARD_BYTE).all())


@pytest.mark.parametrize("opts", [
    dict(chunk_bytes=8192, shard_chunk_bytes=4096, small_bytes=1024, group_bytes=4096, group_max=4),
    dict(ring_ctas_per_sm=2, ctas_per_sm=8, cksum_tile_bytes=4096),
    dict(chunk_bytes=1 << 30, shard_chunk_bytes=1 << 30, small_bytes=1 << 20, group_bytes=1 << 22, group_max=1024),
])
def test_results_do_not_depend_on_the_tuning_values(oracle_mod, opts):
    """The tuning values change how the work is cut and spread, never what is computed: with tiny
    pieces, with huge pieces and with two blocks per SM every result still equals the oracle's."""
    state, planes = _adversarial_by_elem_size(500, 17, seed=29)
    B = 1 << 19
    host = G.host_tensors(state)
    exp_stream, exp_cks = oracle_mod.pack(host, B)
    exp_shards = _expected_shards(oracle_mod, host, state, planes, 3, 5)
    try:
        binding.tm_options_set(**opts)
        mover = RoleMover(state.descs(), B)
        outs = mover.attach_shards(planes, 3, 5)
        target = layouts.blank_like(state)
        unmover = RoleMover(target.descs(), B)
        sp = ShardPlanMover([state.descs_of(list(range(f, f + c))) for f, c in planes], 3, 5)
        whole, buckets = G.guarded(mover.total_bytes)
        fused, alone, got = mover.alloc_checksums(), mover.alloc_checksums(), mover.alloc_checksums()
        mover.pack_emit(buckets, fused)
        mover.checksum(buckets, alone)            # reads the tile size in force now
    finally:
        binding.tm_options_set()
    unmover.unpack_verify(buckets, got)
    sp.extract()
    torch.cuda.synchronize()
    assert mover.status() == 0 and unmover.status() == 0 and sp.status() == 0 and G.guards_intact(whole, mover.total_bytes)
    assert np.array_equal(buckets.cpu().numpy(), exp_stream)
    for c in (fused, alone, got):
        assert np.array_equal(G.u64(c), exp_cks)
    for out, flat, e in zip(outs, sp.flats, exp_shards):
        assert np.array_equal(out.cpu().numpy(), e) and np.array_equal(flat.cpu().numpy(), e)
    exp_arena = np.full(target.arena.numel(), 0xA5, dtype=np.uint8)
    for t, h in zip(target.tensors, host):
        o = t.data_ptr() - target.arena.data_ptr()
        exp_arena[o:o + h.size] = h
    assert np.array_equal(target.arena.cpu().numpy(), exp_arena)


@pytest.mark.parametrize("seed", range(24))
def test_random_layouts_through_the_fused_forms(oracle_mod, seed):
    """Random small roles whose tensor sizes sit around the cuts that matter (16-byte vector, 2 KiB
    bulk threshold, 8 KiB item threshold, 32 KiB stage, 256 KiB chunk), at random 2-byte-granular
    addresses, with random bucket sizes, ranges, shard ranks and output alignments: the sender's fused
    form (range plans through a slot) and the receiver's fused form must both equal the oracle."""
    rng = np.random.default_rng(7000 + seed)
    cuts = [16, 2048, 8192, 32768, 65536, 262144]
    e = int(rng.choice([2, 4, 8]))
    n = int(rng.integers(1, 7))
    numels = []
    for _ in range(n):
        base = int(rng.choice(cuts)) * int(rng.integers(1, 4)) + int(rng.integers(-40, 41)) * 2
        numels.append(max(1, base // e))
    dtype = {2: torch.bfloat16, 4: torch.float32, 8: torch.int64}[e]
    specs = [layouts.TensorSpec(f"t{k}", m, dtype, 1, k) for k, m in enumerate(numels)]
    state = layouts.materialize_adversarial(specs, "cuda", seed=seed)
    target = layouts.blank_like(state)
    B = 256 * int(rng.choice([1, 3, 64, 1000, 4096]))
    host = G.host_tensors(state)
    exp_stream, exp_cks = oracle_mod.pack(host, B)
    D = int(rng.integers(1, 6))
    r = int(rng.integers(0, D))
    expect = oracle_mod.shard(host, [h.size for h in host], e, r, D)
    per = int(rng.integers(1, exp_cks.size + 1))
    mis = 2 * int(rng.integers(0, 8))
    tx_whole, tx_out = G.guarded(expect.size + 16)
    rx_whole, rx_out = G.guarded(expect.size + 16)
    tx_flat, rx_flat = tx_out[mis:mis + expect.size], rx_out[mis:mis + expect.size]
    slot_whole, slot = G.guarded(per * B)
    cks = torch.zeros(exp_cks.size, dtype=torch.int64, device="cuda")
    got = torch.zeros(exp_cks.size, dtype=torch.int64, device="cuda")
    stream_seen = torch.empty(exp_stream.size, dtype=torch.uint8, device="cuda")
    first = 0
    while first < exp_cks.size:
        tx = RoleMover(state.descs(), B, first_bucket=first, n_buckets=per)
        rx = RoleMover(target.descs(), B, first_bucket=first, n_buckets=per)
        tx.attach_shards([(0, n)], r, D, outs=[tx_flat])
        rx.attach_shards([(0, n)], r, D, outs=[rx_flat])
        slot.fill_(0x3C)
        tx.pack_emit(slot, cks[first:first + tx.n_buckets])
        rx.unpack_emit(slot[:rx.total_bytes], got[first:first + rx.n_buckets])
        torch.cuda.synchronize()
        assert tx.status() == 0 and rx.status() == 0 and G.guards_intact(slot_whole, per * B)
        stream_seen[tx.plan.stream_begin:tx.plan.stream_begin + tx.total_bytes] = slot[:tx.total_bytes]
        first += per
    ctx = (numels, e, B, per, r, D, mis)
    assert np.array_equal(stream_seen.cpu().numpy(), exp_stream), ctx
    assert np.array_equal(G.u64(cks), exp_cks) and np.array_equal(G.u64(got), exp_cks), ctx
    assert np.array_equal(tx_flat.cpu().numpy(), expect) and np.array_equal(rx_flat.cpu().numpy(), expect), ctx
    for whole in (tx_whole, rx_whole):
        assert bool((whole[:G.GUARD + mis] == G.GUARD_BYTE).all()) and bool((whole[G.GUARD + mis + expect.size:] == G.GUARD_BYTE).all()), ctx
    exp_arena = np.full(target.arena.numel(), 0xA5, dtype=np.uint8)
    for t, h in zip(target.tensors, host):
        o = t.data_ptr() - target.arena.data_ptr()
        exp_arena[o:o + h.size] = h
    assert np.array_equal(target.arena.cpu().numpy(), exp_arena), ctx
