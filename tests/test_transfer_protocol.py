"""The leaver -> joiner transfer protocol on CPU.  The loops that order the steps, assign slots,
count rounds and re-request damaged waves are the library's own (tm_xfer_run_sender /
tm_xfer_run_receiver); here their steps are played by the CPU oracle over host memory, first by two
threads of one process, then by two processes that talk through torch.distributed (gloo, world
size 2) with the same transport class that carries slots between two GPUs."""
import os
import queue
import socket
import subprocess
import sys
import threading

import numpy as np
import pytest

from paper_2412_12636_b200 import binding, transfer

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _role(seed, n=9):
    rng = np.random.default_rng(seed)
    return [rng.integers(0, 256, 2 * int(rng.integers(1, 3000)), dtype=np.uint8) for _ in range(n)]


def _in_process_transfer(oracle, n_slots, per_wave, damage, max_rounds=3, B=1024):
    """Sender and receiver threads; `damage` maps (round, wave) -> byte index to flip on arrival."""
    tensors = _role(7)
    sizes = [t.size for t in tensors]
    exp_stream, exp_cks = oracle.pack(tensors, B)
    nb = exp_cks.size
    n_waves = -(-nb // per_wave)
    span = lambda w: (w * per_wave * B, min((w + 1) * per_wave * B, exp_stream.size))
    wire, reports = queue.Queue(), queue.Queue()
    tx_slots = [None] * n_slots
    rx_slots = [None] * n_slots
    received = np.zeros_like(exp_stream)
    mine, peer = np.zeros(nb, np.uint64), np.zeros(nb, np.uint64)
    order, rounds = [], {"tx": 0, "rx": 0}

    def pack(w, slot):
        lo, hi = span(w)
        tx_slots[slot] = (oracle.pack_range(tensors, sizes, lo, hi), oracle.checksum(exp_stream[lo:hi], B))
        order.append(("pack", w, slot))

    def send(w, slot):
        wire.put((w, tx_slots[slot][0].copy(), tx_slots[slot][1].copy()))

    def recv_report():
        rounds["tx"] += 1
        return reports.get(timeout=30)

    def recv(w, slot):
        got_w, data, cks = wire.get(timeout=30)
        assert got_w == w
        hit = damage.get((rounds["rx"], w))
        if hit is not None:
            data[hit] ^= 0x04
        rx_slots[slot] = data
        peer[w * per_wave:w * per_wave + cks.size] = cks

    def unpack_verify(w, slot):
        lo, hi = span(w)
        received[lo:hi] = rx_slots[slot]
        c = oracle.checksum(rx_slots[slot], B)
        mine[w * per_wave:w * per_wave + c.size] = c

    def bad_waves(waves):
        rounds["rx"] += 1
        return [w for w in waves if not np.array_equal(mine[w * per_wave:(w + 1) * per_wave], peer[w * per_wave:(w + 1) * per_wave])]

    out = {}
    t = threading.Thread(target=lambda: out.__setitem__("rx", transfer.run_protocol(
        False, n_waves, n_slots, max_rounds, recv=recv, unpack_verify=unpack_verify, bad_waves=bad_waves,
        send_report=lambda ws: reports.put(list(ws)))))
    t.start()
    out["tx"] = transfer.run_protocol(True, n_waves, n_slots, max_rounds, pack=pack, send=send, recv_report=recv_report)
    t.join(timeout=60)
    return out, received, exp_stream, order, n_waves, sizes, tensors


def test_clean_transfer_uses_slots_round_robin(oracle_mod):
    out, received, exp_stream, order, n_waves, sizes, tensors = _in_process_transfer(oracle_mod, 3, 2, {})
    for side in ("tx", "rx"):
        rc, st = out[side]
        assert rc == binding.TM_OK and st["rounds"] == 1 and st["waves"] == n_waves and st["waves_again"] == 0
    assert order == [("pack", w, w % 3) for w in range(n_waves)]
    assert np.array_equal(received, exp_stream)
    for got, t in zip(oracle_mod.unpack(received, sizes), tensors):
        assert np.array_equal(got, t)


def test_damaged_waves_are_requested_again_until_clean(oracle_mod):
    damage = {(0, 1): 5, (0, 4): 900, (1, 4): 17}          # wave 4 arrives damaged twice
    out, received, exp_stream, order, n_waves, _, _ = _in_process_transfer(oracle_mod, 2, 2, damage)
    for side in ("tx", "rx"):
        rc, st = out[side]
        assert rc == binding.TM_OK and st["rounds"] == 3 and st["waves"] == n_waves + 3 and st["waves_again"] == 3
    # round 2 re-sends waves 1 and 4 in slots 0 and 1, round 3 wave 4 in slot 0
    assert order[n_waves:] == [("pack", 1, 0), ("pack", 4, 1), ("pack", 4, 0)]
    assert np.array_equal(received, exp_stream)


def test_transfer_gives_up_after_the_last_round(oracle_mod):
    damage = {(r, 2): 3 for r in range(5)}
    out, received, exp_stream, *_ = _in_process_transfer(oracle_mod, 2, 2, damage, max_rounds=2)
    assert out["tx"][0] == binding.TM_ERR_VERIFY and out["rx"][0] == binding.TM_ERR_VERIFY
    assert out["rx"][1]["rounds"] == 2 and not np.array_equal(received, exp_stream)


def test_protocol_rejects_nonsense():
    ok = lambda *a: None
    rc, _ = transfer.run_protocol(True, 4, 2, 3, pack=ok, send=ok, recv_report=lambda: [7])      # wave that does not exist
    assert rc == binding.TM_ERR_TRANSPORT
    rc, _ = transfer.run_protocol(True, 4, 2, 3, pack=ok, send=ok, recv_report=lambda: [1, 1])   # named twice
    assert rc == binding.TM_ERR_TRANSPORT
    calls = []
    rc, st = transfer.run_protocol(True, 4, 2, 3, pack=lambda w, s: calls.append(w), send=lambda w, s: 1 / 0,
                                   recv_report=lambda: [])
    assert rc == binding.TM_ERR_TRANSPORT and calls == [0]                                       # a failing step ends the run
    rc, _ = transfer.run_protocol(True, 0, 2, 3, pack=ok, send=ok, recv_report=lambda: [])
    assert rc == binding.TM_ERR_ARG
    rc, _ = transfer.run_protocol(False, 4, 2, 3, recv=ok)                                       # receiver without its steps
    assert rc == binding.TM_ERR_ARG


WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["TM_ROOT"])
import numpy as np, torch, torch.distributed as dist
import oracle
from paper_2412_12636_b200 import binding, transfer
dist.init_process_group("gloo")
rank = dist.get_rank()
B, per_wave, n_slots = 1024, 2, 2
rng = np.random.default_rng(7)
tensors = [rng.integers(0, 256, 2 * int(rng.integers(1, 3000)), dtype=np.uint8) for _ in range(9)]
sizes = [t.size for t in tensors]
exp_stream, exp_cks = oracle.pack(tensors, B)
nb = exp_cks.size
n_waves = -(-nb // per_wave)
span = lambda w: (w * per_wave * B, min((w + 1) * per_wave * B, exp_stream.size))
nbk = lambda w: min(per_wave, nb - w * per_wave)
ring = torch.zeros(n_slots * per_wave * B, dtype=torch.uint8)          # host "ring": gloo moves host tensors
cks = torch.zeros(nb, dtype=torch.int64)
peer = torch.zeros(nb, dtype=torch.int64)
tr = transfer.TorchDistTransport(1 - rank, [ring, cks, peer])
t = tr.transport
slot = lambda s: ring[s * per_wave * B:(s + 1) * per_wave * B]
state = {"round": 0}
if rank == 0:                                                          # the leaver
    def pack(w, s):
        lo, hi = span(w)
        data = oracle.pack_range(tensors, sizes, lo, hi)
        slot(s)[:hi - lo] = torch.from_numpy(data)
        cks[w * per_wave:w * per_wave + nbk(w)] = torch.from_numpy(oracle.checksum(data, B).view(np.int64))
    def send(w, s):
        lo, hi = span(w)
        buf = slot(s)
        if state["round"] == 0 and w == 2:                             # damage what goes on the wire, once
            buf = buf.clone(); buf[11] ^= 1
            ring2 = buf
            tr.owners.append(ring2)
            rc = t.send(None, w, ring2.data_ptr(), hi - lo, cks[w * per_wave:].data_ptr(), nbk(w), None)
            tr.owners.pop()
            return rc
        return t.send(None, w, buf.data_ptr(), hi - lo, cks[w * per_wave:].data_ptr(), nbk(w), None)
    def recv_report():
        import ctypes
        arr = (ctypes.c_uint32 * n_waves)(); n = ctypes.c_uint32()
        assert t.recv_report(None, arr, n_waves, ctypes.byref(n)) == 0
        state["round"] += 1
        return [arr[i] for i in range(n.value)]
    rc, st = transfer.run_protocol(True, n_waves, n_slots, 3, pack=pack, send=send, recv_report=recv_report)
    result = {"rank": 0, "rc": rc, "stats": st}
else:                                                                  # the joiner
    received = np.zeros_like(exp_stream)
    def recv(w, s):
        lo, hi = span(w)
        return t.recv(None, w, slot(s).data_ptr(), hi - lo, peer[w * per_wave:].data_ptr(), nbk(w), None)
    def unpack_verify(w, s):
        lo, hi = span(w)
        data = slot(s)[:hi - lo].numpy()
        received[lo:hi] = data
        cks[w * per_wave:w * per_wave + nbk(w)] = torch.from_numpy(oracle.checksum(data, B).view(np.int64))
    def bad_waves(ws):
        return [w for w in ws if not torch.equal(cks[w * per_wave:w * per_wave + nbk(w)], peer[w * per_wave:w * per_wave + nbk(w)])]
    def send_report(ws):
        import ctypes
        arr = (ctypes.c_uint32 * max(1, len(ws)))(*ws)
        return t.send_report(None, arr, len(ws))
    rc, st = transfer.run_protocol(False, n_waves, n_slots, 3, recv=recv, unpack_verify=unpack_verify,
                                   bad_waves=bad_waves, send_report=send_report)
    back = oracle.unpack(received, sizes)
    result = {"rank": 1, "rc": rc, "stats": st, "stream_ok": bool(np.array_equal(received, exp_stream)),
              "tensors_ok": all(np.array_equal(a, b) for a, b in zip(back, tensors)),
              "checksums_ok": bool(np.array_equal(cks.numpy().view(np.uint64), exp_cks))}
dist.barrier()
print(json.dumps(result))
dist.destroy_process_group()
"""


def test_two_gloo_ranks_transfer_a_role_and_repair_a_damaged_wave(tmp_path):
    import json
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, TM_ROOT=ROOT, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=240)
        assert p.returncode == 0, err[-3000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    tx, rx = sorted(outs, key=lambda o: o["rank"])
    assert tx["rc"] == 0 and rx["rc"] == 0
    for o in (tx, rx):
        assert o["stats"]["rounds"] == 2 and o["stats"]["waves_again"] == 1
    assert rx["stream_ok"] and rx["tensors_ok"] and rx["checksums_ok"]
