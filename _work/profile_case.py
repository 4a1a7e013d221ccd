"""Small, self-ending case for profiler captures: a reduced role layout (a few GB on the device,
still far larger than the L2) on which each operation is launched a few times.

    python -m paper_2412_12636_b200.profile_case --workload cfg3 --layers 1 --reps 3

Prints the algorithmic bytes of each operation so that captured DRAM traffic can be compared."""
from __future__ import annotations

import argparse
import json

import torch

from . import binding, layouts
from .mover import MultiShardExtractor, RoleMover


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="cfg3", choices=["cfg0", "cfg1", "cfg2", "cfg3"])
    ap.add_argument("--layers", type=int, default=1)
    ap.add_argument("--reps", type=int, default=3)
    args = ap.parse_args()
    binding.load_library()
    torch.cuda.set_device(0)
    cfg = layouts.role_config(int(args.workload[3]), layers=args.layers)
    state = layouts.materialize(cfg, "cuda")
    target = layouts.blank_like(state)
    mover = RoleMover(state.descs(), cfg.bucket_bytes)
    unmover = RoleMover(target.descs(), cfg.bucket_bytes)
    buckets, fused, alone = mover.alloc_buckets(), mover.alloc_checksums(), mover.alloc_checksums()
    planes = [target.descs_of(target.plane_indices(p)) for p in (layouts.PLANE_MASTER, layouts.PLANE_M, layouts.PLANE_V)]
    multi = MultiShardExtractor(planes, cfg.shard_r, cfg.shard_D)
    outs = multi.alloc_outs()
    received = mover.alloc_checksums()
    for _ in range(args.reps):          # launch order per repetition: pack, checksum, unpack, unpack_verify, shard
        mover.pack(buckets, fused)
        mover.checksum(buckets, alone)
        unmover.unpack(buckets)
        unmover.unpack_verify(buckets, received)
        multi.extract(outs)
    torch.cuda.synchronize()
    assert torch.equal(fused, alone) and torch.equal(fused, received) and mover.status() == 0
    print(json.dumps({"workload": cfg.name, "state_bytes": state.state_bytes, "stream_bytes": mover.total_bytes,
                      "n_buckets": mover.n_buckets,
                      "algorithmic_bytes": {"pack": state.state_bytes + mover.total_bytes + 8 * mover.n_buckets,
                                            "checksum": mover.total_bytes + 8 * mover.n_buckets,
                                            "unpack": 2 * state.state_bytes,
                                            "unpack_verify": 2 * state.state_bytes + 8 * mover.n_buckets,
                                            "shard_three_planes": 2 * sum(multi.out_bytes)},
                      "launches": binding.tm_launch_count()}))


if __name__ == "__main__":
    main()
