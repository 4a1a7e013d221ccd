"""Leaver -> joiner transfer of a role through a bounded ring of staging slots: thin owners of the
library's tm_xfer objects and transports.  The protocol (slot assignment, rounds, re-request of damaged
waves) and every data-path step run inside the library; this module allocates the ring, scratch and
checksum arrays with PyTorch and marshals arguments.

Transports: `Loopback` (both sides in one process on one GPU, the library's own),
`TorchDistTransport`, which moves whole slots with torch.distributed send / recv (NCCL between two
GPUs; gloo between two CPU processes in the protocol tests), and `HostRelayTransport`, which relays
slots through pinned host memory between two processes (also two that share one GPU).
"""
from __future__ import annotations

import ctypes
from typing import Callable, Dict, Optional, Sequence, Tuple

import torch

from . import binding
from .binding import _check, _p, _u32, _u64


def _stream_handle(stream) -> int:
    return stream.cuda_stream if stream is not None else torch.cuda.current_stream().cuda_stream


class Endpoint:
    """One side of a transfer: the role's tensors cut into waves of `buckets_per_wave` whole buckets, a
    ring of `n_slots` staging slots, the scratch for the waves' work lists, and the checksum arrays."""

    def __init__(self, descs: Sequence[Tuple[int, int, int, int]], bucket_bytes: int, buckets_per_wave: int,
                 n_slots: int, receiver: bool, device="cuda", stream=None):
        L = binding.load_library()
        self._h = _p()
        arr = binding.make_descs(descs)
        _check(L.tm_xfer_create(arr, len(arr), bucket_bytes, buckets_per_wave, n_slots, ctypes.byref(self._h)),
               "tm_xfer_create")
        nw, sb, rb, wb, nb = _u32(), _u64(), _u64(), _u64(), _u64()
        _check(L.tm_xfer_query(self._h, ctypes.byref(nw), ctypes.byref(sb), ctypes.byref(rb), ctypes.byref(wb),
                               ctypes.byref(nb)), "tm_xfer_query")
        self.n_waves, self.slot_bytes, self.ring_bytes = nw.value, sb.value, rb.value
        self.workspace_bytes, self.n_buckets = wb.value, nb.value
        self.n_slots, self.receiver = n_slots, receiver
        self.device = torch.device(device)
        self.ring = torch.empty(self.ring_bytes, dtype=torch.uint8, device=self.device)
        self.workspace = torch.empty(self.workspace_bytes, dtype=torch.uint8, device=self.device)
        self.checksums = torch.zeros(self.n_buckets, dtype=torch.int64, device=self.device)
        self.peer_checksums = torch.zeros(self.n_buckets, dtype=torch.int64, device=self.device) if receiver else None
        _check(L.tm_xfer_bind(self._h, self.ring.data_ptr(), self.ring_bytes, self.workspace.data_ptr(),
                              self.workspace_bytes, self.checksums.data_ptr(),
                              self.peer_checksums.data_ptr() if receiver else None, _stream_handle(stream)),
               "tm_xfer_bind")

    def attach_shards(self, planes: Sequence[Tuple[int, int]], r: int, D: int, elem_sizes: Sequence[int], stream=None):
        """Shards filled during the transfer: `planes` = (first descriptor, count) runs of the role,
        `elem_sizes` their element sizes.  Allocates and returns the flat outputs (uint8 tensors)."""
        L = binding.load_library()
        n = len(planes)
        first = (_u64 * n)(*[p[0] for p in planes])
        count = (_u64 * n)(*[p[1] for p in planes])
        got, need = (_u64 * n)(), _u64()
        _check(L.tm_xfer_attach_shards(self._h, first, count, n, r, D, None, None, got, None, 0, ctypes.byref(need), 0),
               "tm_xfer_attach_shards")
        sizes = [g * e for g, e in zip(got, elem_sizes)]
        self.shard_outs = [torch.empty(max(s, 1), dtype=torch.uint8, device=self.device)[:s] for s in sizes]
        self.shard_workspace = torch.empty(max(need.value, 256), dtype=torch.uint8, device=self.device)
        outs = (_p * n)(*[o.data_ptr() for o in self.shard_outs])
        caps = (_u64 * n)(*sizes)
        _check(L.tm_xfer_attach_shards(self._h, first, count, n, r, D, outs, caps, None, self.shard_workspace.data_ptr(),
                                       self.shard_workspace.numel(), None, _stream_handle(stream)), "tm_xfer_attach_shards")
        return self.shard_outs

    def run(self, transport: "binding.TmTransport", work_stream, wire_stream, max_rounds: int = 3) -> Dict[str, int]:
        """Sender: packs on `work_stream`, sends on `wire_stream`.  Receiver: unpacks + verifies on
        `work_stream`, receives on `wire_stream`.  Blocks until the last report has been exchanged;
        returns the statistics.  Raises TmError (TM_ERR_VERIFY, TM_ERR_TRANSPORT, ...) on failure, with
        the statistics in the exception's `stats` attribute."""
        L = binding.load_library()
        stats = binding.TmXferStats()
        fn = L.tm_xfer_receive if self.receiver else L.tm_xfer_send
        rc = fn(self._h, ctypes.byref(transport), _stream_handle(work_stream), _stream_handle(wire_stream), max_rounds,
                ctypes.byref(stats))
        self.stats = stats.as_dict()
        if rc != binding.TM_OK:
            try:
                _check(rc, "tm_xfer_receive" if self.receiver else "tm_xfer_send")
            except binding.TmError as e:
                e.stats = self.stats
                raise
        return self.stats

    def close(self) -> None:
        if self._h:
            binding.load_library().tm_xfer_destroy(self._h)
            self._h = _p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Loopback:
    """The library's same-GPU transport (device-to-device copies between the two rings); the two sides
    run in two host threads of one process."""

    def __init__(self):
        self._h = _p()
        self.transport = binding.TmTransport()
        _check(binding.load_library().tm_loopback_create(ctypes.byref(self._h), ctypes.byref(self.transport)),
               "tm_loopback_create")

    def close(self) -> None:
        if self._h:
            binding.load_library().tm_loopback_destroy(self._h)
            self._h = _p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def wrap_transport(inner: "binding.TmTransport", after_recv: Optional[Callable] = None) -> "binding.TmTransport":
    """A transport that forwards to `inner` and calls after_recv(wave, d_slot, nbytes, stream) once the
    inner recv has been enqueued (fault injection in tests: damage what arrived).  The returned
    structure keeps its callbacks alive."""
    def recv(ctx, wave, d_slot, nbytes, d_cks, n_cks, stream):
        rc = inner.recv(inner.ctx, wave, d_slot, nbytes, d_cks, n_cks, stream)
        if rc == 0 and after_recv is not None:
            after_recv(wave, d_slot, nbytes, stream)
        return rc
    t = binding.TmTransport()
    t.ctx = inner.ctx
    t.send, t.send_report, t.recv_report = inner.send, inner.send_report, inner.recv_report
    t.recv = binding.RECV_FN(recv)
    t._keep = (inner, recv)
    return t


def _as_tensor(ptr: int, nbytes: int, dtype, owner: torch.Tensor) -> torch.Tensor:
    """View of [ptr, ptr + nbytes) inside `owner` (a uint8 or int64 tensor that contains the range)."""
    off = ptr - owner.data_ptr()
    assert 0 <= off and off + nbytes <= owner.numel() * owner.element_size(), "address outside the owning buffer"
    flat = owner.view(torch.uint8).reshape(-1)[off:off + nbytes]
    return flat.view(dtype)


class TorchDistTransport:
    """Whole slots and their checksums travel with torch.distributed send / recv between rank `me` and
    rank `peer`; reports are small tensors sent the other way.  With the NCCL backend the slot is
    sent from and received into device memory (the data lands in the receiver's own HBM, where the
    unpack kernel reads it); with gloo the buffers are host tensors.  `owners` are the tensors the raw
    addresses handed to the callbacks point into (ring, checksum arrays)."""

    def __init__(self, peer: int, owners: Sequence[torch.Tensor], report_device="cpu", group=None):
        import torch.distributed as dist
        self.dist, self.peer, self.owners, self.group = dist, peer, list(owners), group
        self.report_device = torch.device(report_device)
        self.transport = binding.TmTransport()
        self._cb = (binding.SEND_FN(self._send), binding.RECV_FN(self._recv),
                    binding.SEND_REPORT_FN(self._send_report), binding.RECV_REPORT_FN(self._recv_report))
        self.transport.ctx = None
        self.transport.send, self.transport.recv, self.transport.send_report, self.transport.recv_report = self._cb

    def _view(self, ptr: int, nbytes: int, dtype):
        for o in self.owners:
            base = o.data_ptr()
            if base <= ptr and ptr + nbytes <= base + o.numel() * o.element_size():
                return _as_tensor(ptr, nbytes, dtype, o)
        raise ValueError("address outside every registered buffer")

    def _on(self, stream):
        import contextlib
        if stream and torch.cuda.is_available():
            return torch.cuda.stream(torch.cuda.ExternalStream(stream))
        return contextlib.nullcontext()

    def _send(self, ctx, wave, d_slot, nbytes, d_cks, n_cks, stream):
        try:
            with self._on(stream):
                self.dist.send(self._view(d_slot, nbytes, torch.uint8), self.peer, group=self.group, tag=2 * wave)
                self.dist.send(self._view(d_cks, 8 * n_cks, torch.int64), self.peer, group=self.group, tag=2 * wave + 1)
            return 0
        except Exception:
            return binding.TM_ERR_TRANSPORT

    def _recv(self, ctx, wave, d_slot, nbytes, d_cks, n_cks, stream):
        try:
            with self._on(stream):
                self.dist.recv(self._view(d_slot, nbytes, torch.uint8), self.peer, group=self.group, tag=2 * wave)
                self.dist.recv(self._view(d_cks, 8 * n_cks, torch.int64), self.peer, group=self.group, tag=2 * wave + 1)
            return 0
        except Exception:
            return binding.TM_ERR_TRANSPORT

    def _send_report(self, ctx, waves, n):
        try:
            msg = torch.tensor([n] + [waves[i] for i in range(n)], dtype=torch.int64, device=self.report_device)
            self.dist.send(torch.tensor([msg.numel()], dtype=torch.int64, device=self.report_device), self.peer, group=self.group)
            self.dist.send(msg, self.peer, group=self.group)
            return 0
        except Exception:
            return binding.TM_ERR_TRANSPORT

    def _recv_report(self, ctx, waves, capacity, n):
        try:
            size = torch.zeros(1, dtype=torch.int64, device=self.report_device)
            self.dist.recv(size, self.peer, group=self.group)
            msg = torch.zeros(int(size.item()), dtype=torch.int64, device=self.report_device)
            self.dist.recv(msg, self.peer, group=self.group)
            count = int(msg[0].item())
            if count > capacity or count != msg.numel() - 1:
                return binding.TM_ERR_TRANSPORT
            for i in range(count):
                waves[i] = int(msg[1 + i].item())
            n[0] = count
            return 0
        except Exception:
            return binding.TM_ERR_TRANSPORT


class HostRelayTransport(TorchDistTransport):
    """Slots travel through pinned host memory: the sender copies a slot device -> host on the given
    stream, waits for it and sends the host buffer with torch.distributed (any backend that moves CPU
    tensors, e.g. gloo); the receiver receives into pinned host memory and copies host -> device on
    its stream.  For two processes without a GPU-to-GPU link between them — also two processes that
    share one GPU.  `device_owners` are the endpoint's device tensors the raw addresses point into
    (ring, checksums, peer checksums); `damage(wave, host_slot)` (optional) may alter the host copy
    before it is sent."""

    def __init__(self, peer: int, device_owners: Sequence[torch.Tensor], slot_bytes: int, max_checksums: int,
                 group=None, damage: Optional[Callable] = None):
        self.host_slot = torch.empty(slot_bytes, dtype=torch.uint8, pin_memory=True)
        self.host_cks = torch.empty(max_checksums, dtype=torch.int64, pin_memory=True)
        self.damage = damage
        super().__init__(peer, list(device_owners), report_device="cpu", group=group)

    def _send(self, ctx, wave, d_slot, nbytes, d_cks, n_cks, stream):
        try:
            st = torch.cuda.ExternalStream(stream) if stream else torch.cuda.current_stream()
            with torch.cuda.stream(st):
                self.host_slot[:nbytes].copy_(self._view(d_slot, nbytes, torch.uint8), non_blocking=True)
                self.host_cks[:n_cks].copy_(self._view(d_cks, 8 * n_cks, torch.int64), non_blocking=True)
            st.synchronize()
            if self.damage is not None:
                self.damage(wave, self.host_slot[:nbytes])
            self.dist.send(self.host_slot[:nbytes], self.peer, group=self.group, tag=2 * wave)
            self.dist.send(self.host_cks[:n_cks], self.peer, group=self.group, tag=2 * wave + 1)
            return 0
        except Exception:
            return binding.TM_ERR_TRANSPORT

    def _recv(self, ctx, wave, d_slot, nbytes, d_cks, n_cks, stream):
        try:
            st = torch.cuda.ExternalStream(stream) if stream else torch.cuda.current_stream()
            st.synchronize()      # the previous copies out of the host staging buffers have finished
            self.dist.recv(self.host_slot[:nbytes], self.peer, group=self.group, tag=2 * wave)
            self.dist.recv(self.host_cks[:n_cks], self.peer, group=self.group, tag=2 * wave + 1)
            with torch.cuda.stream(st):
                self._view(d_slot, nbytes, torch.uint8).copy_(self.host_slot[:nbytes], non_blocking=True)
                self._view(d_cks, 8 * n_cks, torch.int64).copy_(self.host_cks[:n_cks], non_blocking=True)
            return 0
        except Exception:
            return binding.TM_ERR_TRANSPORT


def run_protocol(sender: bool, n_waves: int, n_slots: int, max_rounds: int, **steps) -> Tuple[int, Dict[str, int]]:
    """Runs the library's protocol loop (tm_xfer_run_sender / tm_xfer_run_receiver) over caller-supplied
    steps — Python callables named like the fields of tm_xfer_hooks (pack, send, recv_report for a
    sender; recv, unpack_verify, bad_waves, send_report for a receiver).  Returns (status, statistics).
    A step returns None or 0 on success; bad_waves(waves) returns the list of damaged waves;
    recv_report() returns the list of waves to send again."""
    L = binding.load_library()

    def step(fn):
        def cb(ctx, wave, slot):
            try:
                return int(fn(wave, slot) or 0)
            except Exception:
                return binding.TM_ERR_TRANSPORT
        return binding.STEP_FN(cb)

    def recv_report_cb(ctx, waves, capacity, n):
        try:
            got = list(steps["recv_report"]())
            if len(got) > capacity:
                return binding.TM_ERR_TRANSPORT
            for i, w in enumerate(got):
                waves[i] = w
            n[0] = len(got)
            return 0
        except Exception:
            return binding.TM_ERR_TRANSPORT

    def bad_waves_cb(ctx, waves, n_w, bad, n_bad):
        try:
            got = list(steps["bad_waves"]([waves[i] for i in range(n_w)]))
            for i, w in enumerate(got):
                bad[i] = w
            n_bad[0] = len(got)
            return 0
        except Exception:
            return binding.TM_ERR_TRANSPORT

    def send_report_cb(ctx, waves, n):
        try:
            return int(steps["send_report"]([waves[i] for i in range(n)]) or 0)
        except Exception:
            return binding.TM_ERR_TRANSPORT

    h = binding.TmXferHooks()
    keep = []
    for name in ("pack", "send", "recv", "unpack_verify"):
        if name in steps:
            cb = step(steps[name])
            keep.append(cb)
            setattr(h, name, cb)
    if "recv_report" in steps:
        keep.append(binding.RECV_REPORT_FN(recv_report_cb))
        h.recv_report = keep[-1]
    if "bad_waves" in steps:
        keep.append(binding.BAD_WAVES_FN(bad_waves_cb))
        h.bad_waves = keep[-1]
    if "send_report" in steps:
        keep.append(binding.SEND_REPORT_FN(send_report_cb))
        h.send_report = keep[-1]
    stats = binding.TmXferStats()
    fn = L.tm_xfer_run_sender if sender else L.tm_xfer_run_receiver
    rc = fn(n_waves, n_slots, max_rounds, ctypes.byref(h), ctypes.byref(stats))
    return rc, stats.as_dict()


def loopback_transfer(send_descs, recv_descs, bucket_bytes: int, buckets_per_wave: int, n_slots: int,
                      max_rounds: int = 3, after_recv: Optional[Callable] = None, device="cuda",
                      recv_shards: Optional[Tuple[Sequence[Tuple[int, int]], int, int]] = None):
    """Moves a role from `send_descs` to `recv_descs` on one GPU: two endpoints, the loopback
    transport, four streams, the receiver in a second host thread.  `after_recv(rx, wave, d_slot,
    nbytes, stream)` is called on the receiving side after every recv has been enqueued (tests damage
    the arrived slot there).  `recv_shards` = (planes, r, D) makes the receiver fill its flat shards
    while it unpacks (rx.shard_outs).  Returns (sender endpoint, receiver endpoint, elapsed device milliseconds
    between the first pack and the last unpack)."""
    import threading
    tx = Endpoint(send_descs, bucket_bytes, buckets_per_wave, n_slots, receiver=False, device=device)
    rx = Endpoint(recv_descs, bucket_bytes, buckets_per_wave, n_slots, receiver=True, device=device)
    if recv_shards is not None:      # (planes, r, D): the receiver also fills its flat shards
        planes, r, D = recv_shards
        rx.attach_shards(planes, r, D, [recv_descs[f][2] for f, _ in planes])
    lb = Loopback()
    rx_transport = lb.transport
    if after_recv is not None:
        rx_transport = wrap_transport(lb.transport, lambda *a: after_recv(rx, *a))
    streams = [torch.cuda.Stream(device=device) for _ in range(4)]
    device_index = tx.ring.device.index          # the receiving thread must work on the same GPU
    torch.cuda.synchronize()
    begin, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    errors = []

    def receive():
        try:
            torch.cuda.set_device(device_index)
            rx.run(rx_transport, streams[2], streams[3], max_rounds)
        except Exception as e:          # reported by the caller's thread
            errors.append(e)

    t = threading.Thread(target=receive)
    begin.record(streams[0])
    t.start()
    try:
        tx.run(lb.transport, streams[0], streams[1], max_rounds)
    except Exception as e:
        errors.append(e)
    t.join()
    end.record(streams[2])
    torch.cuda.synchronize()
    lb.close()
    if errors:
        raise errors[0]
    return tx, rx, begin.elapsed_time(end)
