"""Convenience owners of device buffers around the C-ABI calls.  PyTorch supplies device memory
and streams only; all data movement and checksum arithmetic happens inside the library."""
from __future__ import annotations

from typing import Optional, Sequence, Tuple

import torch

from . import binding


def _stream_handle(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


class RoleMover:
    """A packed-stream plan for one role's tensors with its uploaded work list."""

    def __init__(self, descs: Sequence[Tuple[int, int, int, int]], bucket_bytes: int, device="cuda",
                 stream: Optional[torch.cuda.Stream] = None, first_bucket: Optional[int] = None,
                 n_buckets: Optional[int] = None):
        self.device = torch.device(device)
        self.plan = binding.Plan(descs, bucket_bytes, first_bucket, n_buckets)
        self._elem_sizes = [d[2] for d in descs]
        self.total_bytes = self.plan.total_bytes
        self.n_buckets = self.plan.n_buckets
        self.bucket_bytes = bucket_bytes
        self.workspace = torch.empty(self.plan.workspace_bytes, dtype=torch.uint8, device=self.device)
        self.plan.upload(self.workspace.data_ptr(), self.workspace.numel(), _stream_handle(stream))

    def alloc_buckets(self) -> torch.Tensor:
        return torch.empty(self.total_bytes, dtype=torch.uint8, device=self.device)

    def alloc_checksums(self) -> torch.Tensor:
        # uint64 values carried in an int64 tensor (bit pattern)
        return torch.empty(self.n_buckets, dtype=torch.int64, device=self.device)

    def pack(self, buckets: torch.Tensor, checksums: Optional[torch.Tensor] = None,
             stream: Optional[torch.cuda.Stream] = None) -> None:
        binding.tm_state_pack(self.plan, buckets.data_ptr(), buckets.numel() * buckets.element_size(),
                              None if checksums is None else checksums.data_ptr(), _stream_handle(stream))

    def attach_shards(self, planes: Sequence[Tuple[int, int]], r: int, D: int,
                      stream: Optional[torch.cuda.Stream] = None, outs: Optional[Sequence[torch.Tensor]] = None):
        """Prepares pack_emit: `planes` = (first descriptor, count) runs of this role's descriptors.
        Returns the shard output buffers (one uint8 tensor per plane): `outs` if given (range plans of
        one role share them), freshly allocated otherwise."""
        elems, need = binding.tm_plan_attach_shards(self.plan, planes, r, D, None, None, None, 0, 0)
        sizes = []
        for (first, count), n in zip(planes, elems):
            sizes.append(n * self._elem_sizes[first])
        self.emit_outs = list(outs) if outs is not None else \
            [torch.empty(max(n, 1), dtype=torch.uint8, device=self.device)[:n] for n in sizes]
        self.emit_workspace = torch.empty(need, dtype=torch.uint8, device=self.device)
        binding.tm_plan_attach_shards(self.plan, planes, r, D, [o.data_ptr() for o in self.emit_outs], sizes,
                                      self.emit_workspace.data_ptr(), need, _stream_handle(stream))
        return self.emit_outs

    def pack_emit(self, buckets: torch.Tensor, checksums: Optional[torch.Tensor] = None,
                  stream: Optional[torch.cuda.Stream] = None) -> None:
        """pack + the attached shards in one launch."""
        binding.tm_state_pack_emit(self.plan, buckets.data_ptr(), buckets.numel() * buckets.element_size(),
                                   None if checksums is None else checksums.data_ptr(), _stream_handle(stream))

    def unpack_emit(self, buckets: torch.Tensor, checksums: torch.Tensor,
                    stream: Optional[torch.cuda.Stream] = None) -> None:
        """unpack + verify + the attached shards from one read of the received buckets."""
        binding.tm_state_unpack_emit(self.plan, buckets.data_ptr(), buckets.numel() * buckets.element_size(),
                                     checksums.data_ptr(), _stream_handle(stream))

    def unpack(self, buckets: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
        binding.tm_state_unpack(self.plan, buckets.data_ptr(), buckets.numel() * buckets.element_size(),
                                _stream_handle(stream))

    def unpack_verify(self, buckets: torch.Tensor, checksums: torch.Tensor,
                      stream: Optional[torch.cuda.Stream] = None) -> None:
        """Unpack and, in the same pass, the per-bucket checksums of the buckets as received."""
        binding.tm_state_unpack_verify(self.plan, buckets.data_ptr(), buckets.numel() * buckets.element_size(),
                                       checksums.data_ptr(), _stream_handle(stream))

    def checksum(self, buckets: torch.Tensor, checksums: torch.Tensor,
                 stream: Optional[torch.cuda.Stream] = None) -> None:
        binding.tm_checksum(buckets.data_ptr(), self.total_bytes, self.bucket_bytes, checksums.data_ptr(),
                            _stream_handle(stream))

    def status(self, stream: Optional[torch.cuda.Stream] = None) -> int:
        return self.plan.status(_stream_handle(stream))


class ShardExtractor:
    """Shard r of D of one plane (tensors of one element size) through the one-shot calls, which
    build and upload the work list on every call; owns the scratch workspace they need."""

    def __init__(self, plane_descs: Sequence[Tuple[int, int, int, int]], r: int, D: int, device="cuda"):
        self.device = torch.device(device)
        self.descs = binding.make_descs(plane_descs)
        self.r, self.D = r, D
        self.elem_size = plane_descs[0][2]
        n_elems = sum(d[1] for d in plane_descs) // self.elem_size
        self.lo, self.hi = binding.tm_shard_bounds(n_elems, r, D)
        self.out_bytes = (self.hi - self.lo) * self.elem_size
        ws = binding.tm_shard_workspace(self.descs, r, D)
        self.workspace = torch.empty(ws, dtype=torch.uint8, device=self.device)

    def alloc_out(self) -> torch.Tensor:
        return torch.empty(self.out_bytes, dtype=torch.uint8, device=self.device)

    def extract(self, out: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> int:
        return binding.tm_shard_extract(self.descs, self.r, self.D, out.data_ptr(),
                                        out.numel() * out.element_size(), self.workspace.data_ptr(),
                                        self.workspace.numel(), _stream_handle(stream))

    def insert(self, data: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> int:
        """Writes `data` (this shard) into the plane's tensors; the inverse of extract."""
        return binding.tm_shard_insert(self.descs, self.r, self.D, data.data_ptr(),
                                       data.numel() * data.element_size(), self.workspace.data_ptr(),
                                       self.workspace.numel(), _stream_handle(stream))


class MultiShardExtractor:
    """Shard r of D of several planes (each with its own element size) in one launch, through the
    one-shot call tm_shard_extract_planes."""

    def __init__(self, planes: Sequence[Sequence[Tuple[int, int, int, int]]], r: int, D: int, device="cuda"):
        import ctypes
        self.device = torch.device(device)
        self.r, self.D, self.n_planes = r, D, len(planes)
        self._descs = binding.make_descs([d for plane in planes for d in plane])
        self._counts = (ctypes.c_uint64 * self.n_planes)(*[len(p) for p in planes])
        self.out_bytes = []
        ws = 0
        for plane in planes:
            e = plane[0][2]
            lo, hi = binding.tm_shard_bounds(sum(d[1] for d in plane) // e, r, D)
            self.out_bytes.append((hi - lo) * e)
            ws += binding.tm_shard_workspace(plane, r, D)
        self.workspace = torch.empty(ws, dtype=torch.uint8, device=self.device)
        self._got = (ctypes.c_uint64 * self.n_planes)()

    def alloc_outs(self):
        return [torch.empty(n, dtype=torch.uint8, device=self.device) for n in self.out_bytes]

    def extract(self, outs: Sequence[torch.Tensor], stream: Optional[torch.cuda.Stream] = None):
        import ctypes
        ptrs = (ctypes.c_void_p * self.n_planes)(*[o.data_ptr() for o in outs])
        caps = (ctypes.c_uint64 * self.n_planes)(*[o.numel() * o.element_size() for o in outs])
        L = binding.load_library()
        binding._check(L.tm_shard_extract_planes(self._descs, self._counts, self.n_planes, self.r, self.D, ptrs,
                                                 caps, self._got, self.workspace.data_ptr(),
                                                 self.workspace.numel(), _stream_handle(stream)),
                       "tm_shard_extract_planes")
        return list(self._got)


class ShardPlanMover:
    """Shard r of D of several planes as a reusable plan (tm_shard_plan_*): the work list is built and
    uploaded once, bound to flat buffers that this object owns (or is given); extract and insert are
    then one kernel launch each with no host work."""

    def __init__(self, planes: Sequence[Sequence[Tuple[int, int, int, int]]], r: int, D: int, device="cuda",
                 flats: Optional[Sequence[torch.Tensor]] = None, stream: Optional[torch.cuda.Stream] = None):
        self.device = torch.device(device)
        self.plan = binding.ShardPlan(planes, r, D)
        self.out_bytes = self.plan.out_bytes
        self.workspace = torch.empty(max(self.plan.workspace_bytes, 256), dtype=torch.uint8, device=self.device)
        self.flats = list(flats) if flats is not None else \
            [torch.empty(n, dtype=torch.uint8, device=self.device) for n in self.out_bytes]
        self.rebind(self.flats, stream)

    def rebind(self, flats: Sequence[torch.Tensor], stream: Optional[torch.cuda.Stream] = None) -> None:
        self.flats = list(flats)
        self.plan.bind([f.data_ptr() for f in self.flats], [f.numel() * f.element_size() for f in self.flats],
                       self.workspace.data_ptr(), self.workspace.numel(), _stream_handle(stream))

    def extract(self, stream: Optional[torch.cuda.Stream] = None) -> None:
        self.plan.extract(_stream_handle(stream))

    def insert(self, stream: Optional[torch.cuda.Stream] = None) -> None:
        self.plan.insert(_stream_handle(stream))

    def status(self, stream: Optional[torch.cuda.Stream] = None) -> int:
        return self.plan.status(_stream_handle(stream))


class WaveMover:
    """The same role cut into waves of whole buckets, one range plan (tm_plan_create_range) per wave.

    Wave i packs stream bytes [begin_i, end_i) and produces the checksums of its own buckets, so
    waves can be packed one after another — into slices of one full-size buffer, or into a small
    ring of staging slots when the packed copy must not take a second role's worth of memory (the
    paper's §8.5 rule: the transfer channel is a bounded, recycled buffer).  The concatenation of the
    waves' streams and checksum lists equals what a single plan produces."""

    def __init__(self, descs: Sequence[Tuple[int, int, int, int]], bucket_bytes: int, wave_bytes: int,
                 device="cuda", stream: Optional[torch.cuda.Stream] = None):
        per_wave = max(1, wave_bytes // bucket_bytes)
        arr = binding.make_descs(descs)
        self.movers = []
        first = 0
        while True:
            m = RoleMover.__new__(RoleMover)
            m.device = torch.device(device)
            m.plan = binding.Plan(arr, bucket_bytes, first, per_wave)
            m._elem_sizes = [d[2] for d in descs]
            m.total_bytes, m.n_buckets, m.bucket_bytes = m.plan.total_bytes, m.plan.n_buckets, bucket_bytes
            m.workspace = torch.empty(m.plan.workspace_bytes, dtype=torch.uint8, device=m.device)
            m.plan.upload(m.workspace.data_ptr(), m.workspace.numel(), _stream_handle(stream))
            self.movers.append(m)
            first += per_wave
            if first >= m.plan.whole_buckets:
                break
        p0 = self.movers[0].plan
        self.total_bytes, self.n_buckets, self.bucket_bytes = p0.whole_bytes, p0.whole_buckets, bucket_bytes
        self.n_waves = len(self.movers)
        # tensors touched by each wave, from the stream offsets the planner reports
        offsets = p0.offsets()
        self.tensor_ranges = []
        k = 0
        for m in self.movers:
            lo, hi = m.plan.stream_begin, m.plan.stream_begin + m.plan.total_bytes
            while k < len(descs) and offsets[k] + descs[k][1] <= lo:
                k += 1
            j = k
            while j < len(descs) and offsets[j] < hi:
                j += 1
            self.tensor_ranges.append((k, j))

    def wave_span(self, i: int) -> Tuple[int, int]:
        """(stream_begin, stream_end) of wave i in the complete stream."""
        p = self.movers[i].plan
        return p.stream_begin, p.stream_begin + p.total_bytes

    def wave_buckets(self, i: int) -> Tuple[int, int]:
        """(first bucket, bucket count) of wave i."""
        p = self.movers[i].plan
        return p.first_bucket, p.n_buckets

    def wave_bytes(self, i: int) -> int:
        return self.movers[i].plan.total_bytes

    def pack_wave_into(self, i: int, slot: torch.Tensor, checksums: Optional[torch.Tensor],
                       stream: Optional[torch.cuda.Stream] = None) -> int:
        """Packs wave i into a staging slot (any 256-byte-aligned buffer of at least wave_bytes(i)
        bytes) — the bounded-channel mode: the caller ships the slot and reuses it for a later wave.
        `checksums` is the full per-bucket array of the role.  Returns the bytes written."""
        first, count = self.wave_buckets(i)
        cks = None if checksums is None else checksums[first:first + count]
        self.movers[i].pack(slot, cks, stream)
        return self.wave_bytes(i)

    def pack_wave(self, i: int, buckets: torch.Tensor, checksums: Optional[torch.Tensor],
                  stream: Optional[torch.cuda.Stream] = None) -> None:
        """Packs wave i into its slice of the full-size `buckets` / `checksums` tensors."""
        begin, end = self.wave_span(i)
        self.pack_wave_into(i, buckets[begin:end], checksums, stream)
