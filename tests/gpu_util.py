"""Shared helpers of the GPU parity tests: run the CUDA path through the C-ABI binding and compare
with the CPU oracle on the same seeded inputs, byte for byte."""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np
import torch

from paper_2412_12636_b200 import binding, layouts
from paper_2412_12636_b200.mover import RoleMover, ShardExtractor

GUARD = 512          # guard band (bytes) on both sides of every output buffer
GUARD_BYTE = 0xC3


def guarded(nbytes: int, device="cuda"):
    """(whole buffer, payload view) with guard bands; payload is 256-byte aligned."""
    whole = torch.full((nbytes + 2 * GUARD,), GUARD_BYTE, dtype=torch.uint8, device=device)
    assert whole.data_ptr() % 256 == 0
    return whole, whole[GUARD:GUARD + nbytes]


def guards_intact(whole: torch.Tensor, nbytes: int) -> bool:
    return bool((whole[:GUARD] == GUARD_BYTE).all()) and bool((whole[GUARD + nbytes:] == GUARD_BYTE).all())


def u64(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint64)


def host_tensors(state: layouts.RoleState) -> List[np.ndarray]:
    return [state.host_bytes(k) for k in range(len(state.tensors))]


def gpu_pack(state: layouts.RoleState, bucket_bytes: Optional[int] = None):
    """Returns (mover, packed stream on device, fused checksums (np.uint64))."""
    B = bucket_bytes or state.bucket_bytes
    mover = RoleMover(state.descs(), B)
    whole, buckets = guarded(mover.total_bytes)
    cks = mover.alloc_checksums()
    mover.pack(buckets, cks)
    torch.cuda.synchronize()
    assert guards_intact(whole, mover.total_bytes), "pack wrote outside the packed buffer"
    assert mover.status() == 0
    return mover, buckets, u64(cks)


def check_pack_against_oracle(oracle, state: layouts.RoleState, bucket_bytes: Optional[int] = None):
    """Full byte-for-byte comparison of pack, fused and stand-alone checksum, and unpack."""
    B = bucket_bytes or state.bucket_bytes
    host = host_tensors(state)
    exp_stream, exp_cks = oracle.pack(host, B)
    mover, buckets, cks = gpu_pack(state, B)
    assert mover.total_bytes == exp_stream.size and mover.n_buckets == exp_cks.size
    got = buckets.cpu().numpy()
    assert np.array_equal(got, exp_stream), _first_diff(got, exp_stream)
    assert np.array_equal(cks, exp_cks)
    # stand-alone checksum over the packed stream
    alone = mover.alloc_checksums()
    mover.checksum(buckets, alone)
    torch.cuda.synchronize()
    assert np.array_equal(u64(alone), exp_cks)
    # unpack into fresh tensors (0xA5-filled), including everything around them
    target = layouts.blank_like(state)
    tm = RoleMover(target.descs(), B)
    tm.unpack(buckets)
    torch.cuda.synchronize()
    exp_tensors = oracle.unpack(exp_stream, [s.nbytes for s in state.specs])
    if target.arena is not None:
        exp_arena = np.full(target.arena.numel(), 0xA5, dtype=np.uint8)
        base = target.arena.data_ptr()
        for t, e in zip(target.tensors, exp_tensors):
            o = t.data_ptr() - base
            exp_arena[o:o + e.size] = e
        got_arena = target.arena.cpu().numpy()
        assert np.array_equal(got_arena, exp_arena), _first_diff(got_arena, exp_arena)
    else:
        for k, e in enumerate(exp_tensors):
            assert np.array_equal(target.host_bytes(k), e), f"tensor {k} differs after unpack"
    # unpack + verify in one pass: same tensors, and the checksums of the stream as received — also
    # when a padding byte (which unpack ignores) arrives corrupted
    received = buckets.clone()
    covered = np.zeros(exp_stream.size, dtype=bool)
    off = mover.plan.offsets()
    for o, spec in zip(off, state.specs):
        covered[o:o + spec.nbytes] = True
    pad_positions = np.flatnonzero(~covered)
    if pad_positions.size:
        received[int(pad_positions[pad_positions.size // 2])] = 0x5A
    exp_received = oracle.checksum(received.cpu().numpy(), B)
    target2 = layouts.blank_like(state)
    tm2 = RoleMover(target2.descs(), B)
    got_cks = tm2.alloc_checksums()
    tm2.unpack_verify(received, got_cks)
    torch.cuda.synchronize()
    assert tm2.status() == 0
    assert np.array_equal(u64(got_cks), exp_received)
    if pad_positions.size:
        assert not np.array_equal(exp_received, exp_cks)
    if target2.arena is not None:
        assert torch.equal(target2.arena, target.arena)
    else:
        for a, b in zip(target2.tensors, target.tensors):
            assert torch.equal(layouts.tensor_bytes(a), layouts.tensor_bytes(b))
    return mover, buckets, exp_stream


def check_shard_against_oracle(oracle, state: layouts.RoleState, indices: Sequence[int], r: int, D: int,
                               out_misalign: int = 0):
    """One shard of the plane made of tensors `indices` (common element size), vs the oracle."""
    descs = state.descs_of(indices)
    e = descs[0][2]
    host = [state.host_bytes(i) for i in indices]
    expect = oracle.shard(host, [h.size for h in host], e, r, D)
    ex = ShardExtractor(descs, r, D)
    assert ex.out_bytes == expect.size
    whole, out = guarded(ex.out_bytes + 16)
    out = out[out_misalign:out_misalign + ex.out_bytes]
    n = ex.extract(out)
    torch.cuda.synchronize()
    assert n * e == expect.size
    assert np.array_equal(out.cpu().numpy(), expect), _first_diff(out.cpu().numpy(), expect)
    tail = whole[GUARD + out_misalign + ex.out_bytes:]
    assert bool((whole[:GUARD + out_misalign] == GUARD_BYTE).all()) and bool((tail == GUARD_BYTE).all())
    if ex.out_bytes:
        assert binding.tm_workspace_status(ex.workspace.data_ptr(), torch.cuda.current_stream().cuda_stream) == 0
    return expect


def _first_diff(a: np.ndarray, b: np.ndarray) -> str:
    if a.size != b.size:
        return f"sizes differ: {a.size} vs {b.size}"
    d = np.flatnonzero(a != b)
    if d.size == 0:
        return "equal"
    i = int(d[0])
    return f"{d.size} bytes differ, first at {i} (0x{i:x}): got {a[i]} expected {b[i]}; last at {int(d[-1])}"
