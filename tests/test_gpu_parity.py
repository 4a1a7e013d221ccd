"""GPU parity: the CUDA path, called through the C-ABI binding, must equal the CPU oracle bit for
bit — every packed byte, every padding byte, every checksum, every unpacked tensor byte and every
shard byte.  Integer and byte work only, so the bar is exact equality (no tolerance)."""
import numpy as np
import pytest
import torch

from paper_2412_12636_b200 import binding, layouts
from paper_2412_12636_b200.mover import RoleMover, ShardExtractor

import gpu_util as G

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _cuda():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    binding.load_library()   # fails loudly if the CUDA library is not built
    torch.cuda.set_device(0)
    yield


# ------------------------------------------------------------------ tiny and awkward layouts


@pytest.mark.parametrize("seed", range(8))
@pytest.mark.parametrize("B", [256, 512, 768, 1024, 1 << 20])
def test_odd_layouts_pack_checksum_unpack(oracle_mod, seed, B):
    specs = layouts.odd_specs(seed, n_tensors=3 + seed)
    state = layouts.materialize_adversarial(specs, "cuda", seed=seed)   # 2-byte-granular addresses
    G.check_pack_against_oracle(oracle_mod, state, B)


@pytest.mark.parametrize("numel", [1, 2, 7, 8, 9, 127, 128, 129, 4095, 4096, 4097, 32767, 32768, 32769, 65535, 65537,
                                   3 * 32768 + 5, 131071, 131072, 131073, 2 * 131072 + 3])
@pytest.mark.parametrize("misalign", [0, 2, 4, 6, 8, 10, 12, 14])
def test_single_tensor_every_alignment(oracle_mod, numel, misalign):
    # bf16 elements: sizes around the vector (16 B), small-piece (8 KiB), ring-stage (32 KiB) and chunk (256 KiB) cuts
    arena = torch.randint(0, 256, (2 * numel + 64,), dtype=torch.uint8, device="cuda",
                          generator=torch.Generator("cuda").manual_seed(numel * 16 + misalign))
    t = arena[misalign:misalign + 2 * numel]
    spec = layouts.TensorSpec("t", numel, torch.bfloat16, 0, 0)
    state = layouts.RoleState("one", [spec], [t], 1 << 20, 0, 1, arena)
    G.check_pack_against_oracle(oracle_mod, state, 4096)


def test_tensor_straddles_many_buckets_and_exact_fit(oracle_mod):
    gen = torch.Generator("cuda").manual_seed(5)
    a = torch.randint(0, 256, (10 * 4096,), dtype=torch.uint8, device="cuda", generator=gen)   # exactly 10 buckets
    b = torch.randint(0, 256, (4096 + 2,), dtype=torch.uint8, device="cuda", generator=gen)
    specs = [layouts.TensorSpec("a", a.numel() // 2, torch.bfloat16, 0, 0),
             layouts.TensorSpec("b", b.numel() // 2, torch.bfloat16, 0, 1)]
    state = layouts.RoleState("straddle", specs, [a, b], 4096, 0, 1)
    mover, _, stream = G.check_pack_against_oracle(oracle_mod, state, 4096)
    assert mover.n_buckets == 12 and stream.size == 11 * 4096 + 256
    one = layouts.RoleState("fit", specs[:1], [a], 4096, 0, 1)
    mover, _, stream = G.check_pack_against_oracle(oracle_mod, one, 4096)
    assert mover.n_buckets == 10 and stream.size == 10 * 4096


# ------------------------------------------------------------------ config 0 and a small adversarial set, full compare


def test_config0_full(oracle_mod):
    cfg = layouts.role_config(0)
    state = layouts.materialize(cfg, "cuda")
    mover, _, _ = G.check_pack_against_oracle(oracle_mod, state)
    assert (mover.total_bytes, mover.n_buckets) == (25_790_464, 25)
    for plane in (layouts.PLANE_MASTER, layouts.PLANE_M, layouts.PLANE_V):
        exp = G.check_shard_against_oracle(oracle_mod, state, state.plane_indices(plane), cfg.shard_r, cfg.shard_D)
        assert exp.size == 921_088 * 4


def test_small_adversarial_full(oracle_mod):
    # same recipe as config 4 (log-uniform sizes, mixed dtypes, 2-byte-granular addresses), scaled to
    # what the oracle packs in seconds: several chunks per large tensor, many sub-vector tensors
    specs = layouts.adversarial_specs(3000, max_log2=18)
    state = layouts.materialize_adversarial(specs, "cuda")
    G.check_pack_against_oracle(oracle_mod, state, 1 << 20)
    for e in (4, 2, 8):
        idx = state.elem_size_indices(e)
        flat = np.concatenate([state.host_bytes(i) for i in idx])
        parts = []
        for r in range(0, 64):
            ex = ShardExtractor(state.descs_of(idx), r, 64)
            out = ex.alloc_out()
            ex.extract(out)
            parts.append(out.cpu().numpy())
        assert np.array_equal(np.concatenate(parts), flat)            # exact union coverage
        for r in (0, 17, 63):
            G.check_shard_against_oracle(oracle_mod, state, idx, r, 64, out_misalign=2 * (r % 8))


def test_shard_edge_cases(oracle_mod):
    specs = layouts.odd_specs(3, n_tensors=12)
    state = layouts.materialize_adversarial(specs, "cuda", seed=3)
    for e in (2, 4, 8):
        idx = state.elem_size_indices(e)
        if not idx:
            continue
        n_elems = sum(state.specs[i].numel for i in idx)
        for D in (1, 2, 3, n_elems, n_elems + 5):          # D > N gives empty shards
            for r in sorted({0, D // 2, D - 1}):
                G.check_shard_against_oracle(oracle_mod, state, idx, r, D, out_misalign=2 * (r % 3))


@pytest.mark.parametrize("nbytes,B", [(1, 256), (7, 256), (8, 256), (15, 256), (16, 256), (17, 256), (255, 256),
                                      (256, 256), (257, 256), (4099, 1024), (65536 + 3, 4096), (1 << 20, 1 << 20),
                                      ((1 << 20) + 24, 1 << 19), (3 * (1 << 20) + 1001, 768 * 1024)])
def test_checksum_ragged_inputs(oracle_mod, nbytes, B):
    data = torch.randint(0, 256, (nbytes,), dtype=torch.uint8, device="cuda",
                         generator=torch.Generator("cuda").manual_seed(nbytes))
    nb = -(-nbytes // B)
    out = torch.full((nb + 2,), -1, dtype=torch.int64, device="cuda")
    binding.tm_checksum(data.data_ptr(), nbytes, B, out[1:].data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert np.array_equal(G.u64(out[1:1 + nb]), oracle_mod.checksum(data.cpu().numpy(), B))
    assert int(out[0]) == -1 and int(out[-1]) == -1


def test_checksum_constant_words_on_device():
    c, n = 0x3F8000003F800000, 1 << 17      # fp32 1.0 pairs; closed form c * n^2 mod 2^64
    data = torch.ones(2 * n, dtype=torch.float32, device="cuda")
    out = torch.zeros(1, dtype=torch.int64, device="cuda")
    binding.tm_checksum(data.data_ptr(), 8 * n, 8 * n, out.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert int(G.u64(out)[0]) == (c * n * n) % (1 << 64)


# ------------------------------------------------------------------ failure reporting without faulting anything


def test_corruption_is_detected_and_bad_arguments_are_refused(oracle_mod):
    cfg = layouts.role_config(0)
    state = layouts.materialize(cfg, "cuda")
    mover, buckets, cks = G.gpu_pack(state)
    host = buckets.cpu()
    host[3 * cfg.bucket_bytes + 12345] ^= 0x10             # flip one bit of the host copy
    received = host.cuda()
    again = mover.alloc_checksums()
    mover.checksum(received, again)
    torch.cuda.synchronize()
    bad = np.flatnonzero(G.u64(again) != cks)
    assert bad.tolist() == [3]
    s = torch.cuda.current_stream().cuda_stream
    launches = binding.tm_launch_count()
    with pytest.raises(binding.TmError) as e:              # packed buffer too small
        binding.tm_state_pack(mover.plan, buckets.data_ptr(), mover.total_bytes - 256, None, s)
    assert e.value.status == binding.TM_ERR_CAPACITY
    with pytest.raises(binding.TmError) as e:              # packed buffer overlaps a source tensor
        t = state.tensors[0]
        binding.tm_state_pack(mover.plan, t.data_ptr(), 1 << 40, None, s)
    assert e.value.status == binding.TM_ERR_OVERLAP
    with pytest.raises(binding.TmError) as e:              # misaligned packed buffer
        binding.tm_state_unpack(mover.plan, buckets.data_ptr() + 16, mover.total_bytes, s)
    assert e.value.status == binding.TM_ERR_ALIGN
    dup = [state.descs()[0], state.descs()[0]]             # two unpack targets are the same tensor
    m2 = RoleMover(dup, 1 << 20)
    with pytest.raises(binding.TmError) as e:
        m2.unpack(buckets)
    assert e.value.status == binding.TM_ERR_OVERLAP
    assert binding.tm_launch_count() == launches           # nothing was launched by the refused calls
    torch.cuda.synchronize()


def test_repeated_runs_are_identical():
    specs = layouts.adversarial_specs(500, max_log2=16)
    state = layouts.materialize_adversarial(specs, "cuda")
    _, b1, c1 = G.gpu_pack(state, 1 << 18)
    first = b1.clone()
    _, b2, c2 = G.gpu_pack(state, 1 << 18)
    assert torch.equal(first, b2) and np.array_equal(c1, c2)


@pytest.mark.parametrize("wave_bytes", [1 << 20, 3 << 20, 1 << 30])
def test_wave_by_wave_pack_equals_single_plan_and_oracle(oracle_mod, wave_bytes):
    from paper_2412_12636_b200.mover import WaveMover
    cfg = layouts.role_config(0)
    state = layouts.materialize(cfg, "cuda")
    exp_stream, exp_cks = oracle_mod.pack(G.host_tensors(state), cfg.bucket_bytes)
    wm = WaveMover(state.descs(), cfg.bucket_bytes, wave_bytes)
    assert (wm.total_bytes, wm.n_buckets) == (exp_stream.size, exp_cks.size)
    assert wm.n_waves == -(-wm.n_buckets // max(1, wave_bytes // cfg.bucket_bytes))
    whole, buckets = G.guarded(wm.total_bytes)
    cks = torch.zeros(wm.n_buckets, dtype=torch.int64, device="cuda")
    for i in reversed(range(wm.n_waves)):             # order does not matter: waves are independent
        wm.pack_wave(i, buckets, cks)
    torch.cuda.synchronize()
    assert G.guards_intact(whole, wm.total_bytes)
    assert np.array_equal(buckets.cpu().numpy(), exp_stream)
    assert np.array_equal(G.u64(cks), exp_cks)


@pytest.mark.parametrize("e", [4, 2, 8])
def test_shard_insert_matches_oracle_and_inverts_extract(oracle_mod, e):
    specs = layouts.adversarial_specs(400, max_log2=17)
    state = layouts.materialize_adversarial(specs, "cuda", seed=11)
    idx = state.elem_size_indices(e)
    descs = state.descs_of(idx)
    sizes = [d[1] for d in descs]
    before = state.arena.clone()
    for r, D, mis in ((0, 1, 0), (3, 7, 2), (63, 64, 6), (5, 3 * sum(sizes), 0)):   # last: empty or 1-element shards
        ex = ShardExtractor(descs, r, D)
        gen = torch.Generator("cuda").manual_seed(r * 1000 + D)
        whole = torch.randint(0, 256, (ex.out_bytes + 16,), dtype=torch.uint8, device="cuda", generator=gen)
        data = whole[mis:mis + ex.out_bytes]
        host = [state.host_bytes(i).copy() for i in idx]
        assert oracle_mod.shard_insert(host, sizes, e, r, D, data.cpu().numpy()) == ex.hi - ex.lo
        assert ex.insert(data) == ex.hi - ex.lo
        torch.cuda.synchronize()
        for i, h in zip(idx, host):
            assert np.array_equal(state.host_bytes(i), h), f"tensor {i} after insert r={r} D={D}"
        out = ex.alloc_out()
        ex.extract(out)
        torch.cuda.synchronize()
        assert torch.equal(out, data)                       # extract(insert(x)) == x
    # nothing outside the plane's tensors changed (gaps, tensors of other element sizes)
    mask = torch.ones_like(before, dtype=torch.bool)
    base = state.arena.data_ptr()
    for i in idx:
        o = state.tensors[i].data_ptr() - base
        mask[o:o + state.specs[i].nbytes] = False
    assert torch.equal(state.arena[mask], before[mask])


def test_role_delta_pack_of_a_descriptor_subset(oracle_mod):
    # A standby warmed as a middle stage that is promoted to a first/last stage only needs the extra
    # layers' parameters and optimizer state (paper §6): pack just those descriptors.
    cfg = layouts.role_config(0)
    state = layouts.materialize(cfg, "cuda")
    delta = [i for i, s in enumerate(state.specs) if ".embedding" in s.name or ".final_ln" in s.name]
    assert len(delta) == 12
    sub = state.subset(delta, "tiny-gpt-first-stage-delta")
    mover, _, stream = G.check_pack_against_oracle(oracle_mod, sub, 256 * 1024)
    assert stream.size == sum(-(-s.nbytes // 256) * 256 for s in sub.specs)


def test_expired_device_wait_is_reported_not_hung():
    # a wait that nothing completes: the kernel gives up after 50 ms, records the status and returns
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    assert binding.tm_workspace_status(ws.data_ptr(), s) == 0
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    binding.tm_selftest_bounded_wait(ws.data_ptr(), 50_000_000, s)
    t1.record()
    assert binding.tm_workspace_status(ws.data_ptr(), s) == binding.TM_ERR_TIMEOUT
    assert 40.0 < t0.elapsed_time(t1) < 1000.0
    # the context is still usable: a real operation right after
    data = torch.ones(1 << 16, dtype=torch.int64, device="cuda")
    out = torch.zeros(1, dtype=torch.int64, device="cuda")
    binding.tm_checksum(data.data_ptr(), 8 << 16, 8 << 16, out.data_ptr(), s)
    torch.cuda.synchronize()
    assert int(G.u64(out)[0]) == (1 << 32)               # c * n^2 with c = 1, n = 2^16


def test_multi_plane_shard_extract_matches_oracle_per_plane(oracle_mod):
    from paper_2412_12636_b200.mover import MultiShardExtractor
    cfg = layouts.role_config(0)
    state = layouts.materialize(cfg, "cuda")
    adv = layouts.materialize_adversarial(layouts.adversarial_specs(300, max_log2=16), "cuda", seed=5)
    cases = [
        (state, [state.plane_indices(p) for p in (layouts.PLANE_MASTER, layouts.PLANE_M, layouts.PLANE_V)], 1, 2),
        (adv, [adv.elem_size_indices(e) for e in (4, 2, 8)], 17, 64),        # mixed element sizes in one call
        (adv, [adv.elem_size_indices(e) for e in (8, 4)], 10 ** 9 - 1, 10 ** 9),   # D > N: one-element shards
        (adv, [adv.elem_size_indices(e) for e in (8, 4)], 0, 10 ** 9),             # D > N: empty shards, no launch
    ]
    for st, planes, r, D in cases:
        ms = MultiShardExtractor([st.descs_of(idx) for idx in planes], r, D)
        bufs = [G.guarded(n) for n in ms.out_bytes]
        got = ms.extract([b[1] for b in bufs])
        torch.cuda.synchronize()
        if any(ms.out_bytes):
            assert binding.tm_workspace_status(ms.workspace.data_ptr(), torch.cuda.current_stream().cuda_stream) == 0
        for idx, (whole, out), n_el, nbytes in zip(planes, bufs, got, ms.out_bytes):
            e = st.specs[idx[0]].elem_size
            host = [st.host_bytes(i) for i in idx]
            expect = oracle_mod.shard(host, [h.size for h in host], e, r, D)
            assert n_el * e == expect.size == nbytes
            assert np.array_equal(out.cpu().numpy(), expect)
            assert G.guards_intact(whole, nbytes)


def test_two_streams_run_independent_plans_concurrently(oracle_mod):
    specs_a = layouts.adversarial_specs(600, max_log2=17)
    a = layouts.materialize_adversarial(specs_a, "cuda", seed=21)
    b = layouts.materialize(layouts.role_config(0), "cuda")
    exp_a, cks_a = oracle_mod.pack(G.host_tensors(a), 1 << 20)
    exp_b, cks_b = oracle_mod.pack(G.host_tensors(b), 1 << 20)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    ma, mb = RoleMover(a.descs(), 1 << 20, stream=s1), RoleMover(b.descs(), 1 << 20, stream=s2)
    ba, bb = ma.alloc_buckets(), mb.alloc_buckets()
    ca, cb = ma.alloc_checksums(), mb.alloc_checksums()
    ta, tb = layouts.blank_like(a), layouts.blank_like(b)
    ua, ub = RoleMover(ta.descs(), 1 << 20, stream=s1), RoleMover(tb.descs(), 1 << 20, stream=s2)
    torch.cuda.synchronize()
    for _ in range(5):                       # interleave enqueues on the two streams
        ma.pack(ba, ca, stream=s1)
        mb.pack(bb, cb, stream=s2)
        ua.unpack(ba, stream=s1)
        ub.unpack(bb, stream=s2)
    torch.cuda.synchronize()
    assert np.array_equal(ba.cpu().numpy(), exp_a) and np.array_equal(G.u64(ca), cks_a)
    assert np.array_equal(bb.cpu().numpy(), exp_b) and np.array_equal(G.u64(cb), cks_b)
    for k in range(0, len(a.tensors), 37):
        assert np.array_equal(ta.host_bytes(k), a.host_bytes(k))
    for k in range(len(b.tensors)):
        assert np.array_equal(tb.host_bytes(k), b.host_bytes(k))
    assert ma.status(s1) == 0 and mb.status(s2) == 0


def test_bounded_staging_ring_reproduces_the_stream(oracle_mod):
    # two staging slots of 2 MiB stand for the recycled transfer channel (paper §8.5): every wave is
    # packed into a slot, "sent" (copied out), and the slot is reused; the receiver's copy must be the
    # complete stream, and the checksums the complete list
    from paper_2412_12636_b200.mover import WaveMover
    cfg = layouts.role_config(0)
    state = layouts.materialize(cfg, "cuda")
    exp_stream, exp_cks = oracle_mod.pack(G.host_tensors(state), cfg.bucket_bytes)
    wm = WaveMover(state.descs(), cfg.bucket_bytes, 2 << 20)
    slots = [G.guarded(2 << 20) for _ in range(2)]
    cks = torch.zeros(wm.n_buckets, dtype=torch.int64, device="cuda")
    received = torch.empty(wm.total_bytes, dtype=torch.uint8, device="cuda")
    for i in range(wm.n_waves):
        whole, slot = slots[i % 2]
        slot.fill_(0x77)                                   # stale contents of the recycled slot
        n = wm.pack_wave_into(i, slot, cks)
        assert n == wm.wave_bytes(i) <= slot.numel()
        begin, end = wm.wave_span(i)
        received[begin:end].copy_(slot[:n])
        torch.cuda.synchronize()
        assert G.guards_intact(whole, 2 << 20)
        assert bool((slot[n:] == 0x77).all())              # nothing written past the wave
    assert np.array_equal(received.cpu().numpy(), exp_stream)
    assert np.array_equal(G.u64(cks), exp_cks)


def test_pack_emit_gives_the_stream_and_the_shards_in_one_launch(oracle_mod):
    cases = []
    cfg = layouts.role_config(0)
    st0 = layouts.materialize(cfg, "cuda")
    P = len(cfg.model)
    cases.append((st0, [(P, P), (2 * P, P), (3 * P, P)], 1, 2, cfg.bucket_bytes))
    cases.append((st0, [(P, P), (3 * P, P)], 2, 3, 256 * 1024))                    # mid-tensor bounds, two planes
    specs = sorted(layouts.adversarial_specs(500, max_log2=17), key=lambda s: s.elem_size)   # runs per element size
    adv = layouts.materialize_adversarial(specs, "cuda", seed=9)
    runs, k = [], 0
    for e in (2, 4, 8):
        n = sum(1 for s in specs if s.elem_size == e)
        runs.append((k, n))
        k += n
    cases.append((adv, runs, 5, 7, 1 << 20))
    cases.append((adv, runs[1:2], 63, 64, 1 << 20))
    for state, planes, r, D, B in cases:
        host = G.host_tensors(state)
        exp_stream, exp_cks = oracle_mod.pack(host, B)
        mover = RoleMover(state.descs(), B)
        outs = mover.attach_shards(planes, r, D)
        whole, buckets = G.guarded(mover.total_bytes)
        cks = mover.alloc_checksums()
        launches = binding.tm_launch_count()
        mover.pack_emit(buckets, cks)
        torch.cuda.synchronize()
        assert binding.tm_launch_count() == launches + 1
        assert mover.status() == 0 and G.guards_intact(whole, mover.total_bytes)
        assert np.array_equal(buckets.cpu().numpy(), exp_stream)
        assert np.array_equal(G.u64(cks), exp_cks)
        for (first, count), out in zip(planes, outs):
            e = state.specs[first].elem_size
            sub = host[first:first + count]
            expect = oracle_mod.shard(sub, [h.size for h in sub], e, r, D)
            assert np.array_equal(out.cpu().numpy(), expect), (first, count, r, D)
    # argument checks: overlapping or descending planes, unattached plan
    plain = RoleMover(st0.descs(), 1 << 20)
    with pytest.raises(binding.TmError) as ex:
        binding.tm_state_pack_emit(plain.plan, 1 << 40, 1 << 40, None, 0)
    assert ex.value.status == binding.TM_ERR_STATE
    with pytest.raises(binding.TmError) as ex:
        binding.tm_plan_attach_shards(plain.plan, [(2 * P, P), (P, P)], 0, 2, None, None, None, 0, 0)
    assert ex.value.status == binding.TM_ERR_ARG
    with pytest.raises(binding.TmError) as ex:
        binding.tm_plan_attach_shards(plain.plan, [(0, 2 * P)], 0, 2, None, None, None, 0, 0)   # bf16 + fp32 in one plane
    assert ex.value.status == binding.TM_ERR_DTYPE
