"""Leaver -> joiner transfer on one GPU through the loopback transport: the role is packed wave by
wave into a small ring of slots, copied into the receiver's ring, unpacked and verified there, with
all four stages overlapping.  The receiver's tensors and both sides' checksums must equal the CPU
oracle's; a wave damaged in flight must be detected, re-requested and repaired."""
import numpy as np
import pytest
import torch

from paper_2412_12636_b200 import binding, layouts, transfer

import gpu_util as G

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _cuda():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    binding.load_library()
    torch.cuda.set_device(0)
    yield


def _flip_on_host(hits, seen):
    """after_recv hook: for every (round-trip count, wave) in `hits`, copy the arrived slot to the host,
    flip one bit of the host copy, and copy it back — on the stream the slot arrived on."""
    def hook(rx, wave, d_slot, nbytes, stream):
        seen[wave] = seen.get(wave, 0) + 1
        byte = hits.get((seen[wave], wave))
        if byte is None:
            return
        off = d_slot - rx.ring.data_ptr()
        view = rx.ring[off:off + nbytes]
        with torch.cuda.stream(torch.cuda.ExternalStream(stream)):
            host = view.cpu()
            host[byte % nbytes] ^= 0x20
            view.copy_(host)
    return hook


def _check_receiver(oracle, state, target, tx, rx, B):
    host = G.host_tensors(state)
    _, exp_cks = oracle.pack(host, B)
    assert np.array_equal(G.u64(tx.checksums), exp_cks) and np.array_equal(G.u64(rx.checksums), exp_cks)
    assert np.array_equal(G.u64(rx.peer_checksums), exp_cks)
    if target.arena is not None:
        exp_arena = np.full(target.arena.numel(), 0xA5, dtype=np.uint8)
        for t, h in zip(target.tensors, host):
            o = t.data_ptr() - target.arena.data_ptr()
            exp_arena[o:o + h.size] = h
        assert np.array_equal(target.arena.cpu().numpy(), exp_arena)
    else:
        for k, h in enumerate(host):
            assert np.array_equal(target.host_bytes(k), h), f"tensor {k}"


@pytest.mark.parametrize("per_wave,n_slots", [(1, 2), (3, 2), (4, 3), (64, 1)])
def test_loopback_transfer_config0(oracle_mod, per_wave, n_slots):
    cfg = layouts.role_config(0)
    state = layouts.materialize(cfg, "cuda")
    target = layouts.blank_like(state)
    tx, rx, ms = transfer.loopback_transfer(state.descs(), target.descs(), cfg.bucket_bytes, per_wave, n_slots)
    n_waves = -(-25 // per_wave)
    assert tx.n_waves == rx.n_waves == n_waves and tx.ring_bytes == n_slots * per_wave * cfg.bucket_bytes
    for side in (tx, rx):
        assert side.stats["rounds"] == 1 and side.stats["waves"] == n_waves and side.stats["bad_buckets"] == 0
        assert side.stats["bytes"] == 25_790_464
    _check_receiver(oracle_mod, state, target, tx, rx, cfg.bucket_bytes)


def test_loopback_transfer_adversarial_layout(oracle_mod):
    state = layouts.materialize_adversarial(layouts.adversarial_specs(800, max_log2=17), "cuda", seed=17)
    target = layouts.blank_like(state)
    tx, rx, _ = transfer.loopback_transfer(state.descs(), target.descs(), 1 << 18, 3, 2)
    assert rx.stats["rounds"] == 1
    _check_receiver(oracle_mod, state, target, tx, rx, 1 << 18)


def test_wave_damaged_in_flight_is_detected_and_sent_again(oracle_mod):
    cfg = layouts.role_config(0)
    state = layouts.materialize(cfg, "cuda")
    target = layouts.blank_like(state)
    seen = {}
    # wave 2 arrives damaged in round 1 (bucket 7 of the stream), wave 5 in rounds 1 and 2
    hits = {(1, 2): 1 * cfg.bucket_bytes + 12345, (1, 5): 77, (2, 5): 2 * cfg.bucket_bytes + 5}
    tx, rx, _ = transfer.loopback_transfer(state.descs(), target.descs(), cfg.bucket_bytes, 3, 2, max_rounds=4,
                                           after_recv=_flip_on_host(hits, seen))
    for side in (tx, rx):
        assert side.stats["rounds"] == 3 and side.stats["waves"] == 9 + 2 + 1 and side.stats["waves_again"] == 3
    assert rx.stats["bad_buckets"] == 3 and rx.stats["first_bad_bucket"] == 7
    assert seen[2] == 2 and seen[5] == 3 and seen[0] == 1
    _check_receiver(oracle_mod, state, target, tx, rx, cfg.bucket_bytes)


def test_transfer_reports_failure_when_damage_persists(oracle_mod):
    cfg = layouts.role_config(0)
    state = layouts.materialize(cfg, "cuda")
    target = layouts.blank_like(state)
    hits = {(k, 1): 3 for k in range(1, 6)}
    with pytest.raises(binding.TmError) as e:
        transfer.loopback_transfer(state.descs(), target.descs(), cfg.bucket_bytes, 5, 2, max_rounds=2,
                                   after_recv=_flip_on_host(hits, {}))
    assert e.value.status == binding.TM_ERR_VERIFY and e.value.stats["rounds"] == 2
    # the context is fine afterwards
    tx, rx, _ = transfer.loopback_transfer(state.descs(), target.descs(), cfg.bucket_bytes, 5, 2)
    _check_receiver(oracle_mod, state, target, tx, rx, cfg.bucket_bytes)


@pytest.mark.parametrize("seed,B,per_wave,n_slots", [(0, 256, 1, 2), (1, 768, 5, 3), (2, 512, 2, 1), (3, 4096, 3, 2)])
def test_loopback_transfer_tiny_buckets_and_odd_sizes(oracle_mod, seed, B, per_wave, n_slots):
    # sub-vector tensors at 2-byte-granular addresses, buckets of a few hundred bytes, many waves
    specs = layouts.odd_specs(seed, n_tensors=6 + seed)
    state = layouts.materialize_adversarial(specs, "cuda", seed=seed)
    target = layouts.blank_like(state)
    tx, rx, _ = transfer.loopback_transfer(state.descs(), target.descs(), B, per_wave, n_slots)
    assert rx.stats["rounds"] == 1 and tx.n_waves == -(-tx.n_buckets // per_wave)
    _check_receiver(oracle_mod, state, target, tx, rx, B)


@pytest.mark.parametrize("case", ["cfg0", "adversarial"])
def test_receiver_fills_its_shards_while_the_role_arrives(oracle_mod, case):
    """With shards attached to the receiving endpoint, every wave's unpack also writes its part of the
    joiner's flat slices; a wave damaged in flight first writes damaged shard bytes, and its repeat
    repairs them along with the tensors."""
    if case == "cfg0":
        cfg = layouts.role_config(0)
        state = layouts.materialize(cfg, "cuda")
        P = len(cfg.model)
        planes, r, D, B, per_wave = [(P, P), (2 * P, P), (3 * P, P)], 1, 2, cfg.bucket_bytes, 3
    else:
        specs = sorted(layouts.adversarial_specs(600, max_log2=17), key=lambda s: s.elem_size)
        state = layouts.materialize_adversarial(specs, "cuda", seed=19)
        planes, k = [], 0
        for e in (2, 4, 8):
            c = sum(1 for s in specs if s.elem_size == e)
            planes.append((k, c))
            k += c
        r, D, B, per_wave = 4, 9, 1 << 18, 4
    target = layouts.blank_like(state)
    host = G.host_tensors(state)
    n_waves = -(-oracle_mod.layout([h.size for h in host], B)[2] // per_wave)
    hits = {(1, w): 1000 + 37 * w for w in range(0, n_waves, 2)}        # every second wave arrives damaged once
    tx, rx, _ = transfer.loopback_transfer(state.descs(), target.descs(), B, per_wave, 2, max_rounds=3,
                                           after_recv=_flip_on_host(hits, {}), recv_shards=(planes, r, D))
    assert rx.stats["rounds"] == 2 and rx.stats["waves_again"] == len(hits)
    _check_receiver(oracle_mod, state, target, tx, rx, B)
    for (first, count), out in zip(planes, rx.shard_outs):
        sub = host[first:first + count]
        expect = oracle_mod.shard(sub, [h.size for h in sub], state.specs[first].elem_size, r, D)
        assert np.array_equal(out.cpu().numpy(), expect), (first, count)


TWO_PROCESS_WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["TM_ROOT"])
sys.path.insert(0, os.path.join(os.environ["TM_ROOT"], "tests"))
import numpy as np, torch, torch.distributed as dist
import oracle
from paper_2412_12636_b200 import binding, layouts, transfer
dist.init_process_group("gloo")
rank = dist.get_rank()
torch.cuda.set_device(0)
binding.load_library()
cfg = layouts.role_config(0)
B, per_wave, n_slots = cfg.bucket_bytes, 3, 2
state = layouts.materialize(cfg, "cuda")                     # same seed in both processes
host = [state.host_bytes(k) for k in range(len(state.tensors))]
_, exp_cks = oracle.pack(host, B)
streams = [torch.cuda.Stream(), torch.cuda.Stream()]
if rank == 0:                                                # the leaver's process
    ep = transfer.Endpoint(state.descs(), B, per_wave, n_slots, receiver=False)
    sent = {}
    def damage(wave, host_slot):                             # wave 4 leaves damaged the first time
        sent[wave] = sent.get(wave, 0) + 1
        if wave == 4 and sent[wave] == 1:
            host_slot[4321] ^= 0x08
    tr = transfer.HostRelayTransport(1, [ep.ring, ep.checksums], ep.slot_bytes, per_wave, damage=damage)
    stats = ep.run(tr.transport, streams[0], streams[1], 3)
    result = {"rank": 0, "stats": stats, "checksums_ok": bool(np.array_equal(ep.checksums.cpu().numpy().view(np.uint64), exp_cks))}
else:                                                        # the joiner's process
    target = layouts.blank_like(state)
    ep = transfer.Endpoint(target.descs(), B, per_wave, n_slots, receiver=True)
    tr = transfer.HostRelayTransport(0, [ep.ring, ep.checksums, ep.peer_checksums], ep.slot_bytes, per_wave)
    stats = ep.run(tr.transport, streams[0], streams[1], 3)
    torch.cuda.synchronize()
    result = {"rank": 1, "stats": stats,
              "tensors_ok": all(np.array_equal(target.host_bytes(k), host[k]) for k in range(len(host))),
              "checksums_ok": bool(np.array_equal(ep.checksums.cpu().numpy().view(np.uint64), exp_cks))}
dist.barrier()
print(json.dumps(result))
dist.destroy_process_group()
"""


def test_leaver_and_joiner_in_two_processes(tmp_path):
    """The two sides as two processes (gloo ranks 0 and 1) that share this GPU: each runs its endpoint
    with the library's kernels, slots cross between the processes through pinned host memory.  No
    kernel of one process waits for the other — only the host threads block in send / recv — so the
    processes may time-share the device.  One wave is damaged on the way and must be repaired."""
    import json, os, socket, subprocess, sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    script = tmp_path / "worker.py"
    script.write_text(TWO_PROCESS_WORKER)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, TM_ROOT=root, RANK=str(rank), LOCAL_RANK="0", WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=300)
        assert p.returncode == 0, err[-3000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    tx, rx = sorted(outs, key=lambda o: o["rank"])
    for o in (tx, rx):
        assert o["stats"]["rounds"] == 2 and o["stats"]["waves"] == 9 + 1 and o["stats"]["waves_again"] == 1
        assert o["checksums_ok"]
    assert rx["tensors_ok"] and rx["stats"]["bad_buckets"] == 1 and rx["stats"]["first_bad_bucket"] == 12


def test_many_short_transfers_in_a_row(oracle_mod):
    """Hundreds of waves of a few hundred bytes each: the hand-shakes between the two host threads (post,
    match, take) follow one another as fast as they can, which is where a lost wake-up would show as
    a partner time-out."""
    specs = layouts.odd_specs(5, n_tensors=10)
    state = layouts.materialize_adversarial(specs, "cuda", seed=5)
    host = G.host_tensors(state)
    _, exp_cks = oracle_mod.pack(host, 256)
    for i in range(120):
        target = layouts.blank_like(state)
        tx, rx, _ = transfer.loopback_transfer(state.descs(), target.descs(), 256, 1 + i % 3, 1 + i % 4)
        assert rx.stats["rounds"] == 1 and np.array_equal(G.u64(rx.checksums), exp_cks)
        if i % 20 == 0:
            _check_receiver(oracle_mod, state, target, tx, rx, 256)
