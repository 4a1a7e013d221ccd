"""B200-native role-state mover: pack / unpack / shard-extract / checksum of a role's training
state (TrainMover, §7 "State Synchronization").

`paper_2412_12636_b200.binding` is the thin ctypes face of the C-ABI library in `csrc/`
(declared in `include/tm_state.h`); `paper_2412_12636_b200.layouts` generates seeded synthetic
role layouts.  Importing this package does not load the CUDA library; the first use of a binding
attribute does, and fails loudly if it has not been built.
"""

_BINDING_NAMES = (
    "Plan", "ShardPlan", "TmError", "tm_state_pack", "tm_state_unpack", "tm_state_unpack_verify", "tm_state_pack_emit",
    "tm_state_unpack_emit", "tm_plan_attach_shards", "tm_shard_extract", "tm_shard_extract_planes", "tm_shard_insert",
    "tm_shard_extract_static", "tm_checksum", "tm_shard_bounds", "tm_shard_workspace", "tm_options_get", "tm_options_set",
    "tm_launch_count", "load_library", "make_descs",
)


def __getattr__(name):
    if name in _BINDING_NAMES:
        from . import binding
        return getattr(binding, name)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
