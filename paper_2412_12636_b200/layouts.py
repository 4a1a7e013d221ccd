"""Seeded synthetic role layouts: tensor lists and values only.

A "role" is what one machine holds for its (TP, PP, DP) identity (paper §6 "General Standby":
first, middle and last pipeline stages are the role types).  Its training state is, per the
paper's §7 "State Synchronization", model parameters plus optimizer states: here bf16 parameters,
fp32 master weights, Adam m and Adam v.  Gradients are not part of it (§8.5: the leaver's
gradient buffer becomes the transfer channel).

This module only *generates inputs* — names, shapes, dtypes, device tensors and their values — for
both the CUDA library's tests/benchmarks and the CPU oracle's.  It contains none of the method's
arithmetic: no stream offsets, no bucket cuts, no shard bounds, no checksums.

The layouts stand in for the Megatron-LM GPT workloads the paper trains (§8 "Evaluation",
experiment setup); values never change the cost of the path, only shapes, dtypes, count and
alignment do.

Order of tensors (the library never reorders): plane-major — every bf16 parameter in model order,
then every fp32 master weight, then Adam m, then Adam v — so that each fp32 plane is one
contiguous run of descriptors.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

PLANE_PARAM, PLANE_MASTER, PLANE_M, PLANE_V, PLANE_OTHER = 0, 1, 2, 3, 4
PLANE_NAMES = {0: "param_bf16", 1: "master_fp32", 2: "adam_m", 3: "adam_v", 4: "other"}

_ELEM = {torch.bfloat16: 2, torch.float32: 4, torch.int64: 8}


@dataclasses.dataclass(frozen=True)
class TensorSpec:
    name: str
    numel: int
    dtype: torch.dtype
    plane: int
    model_index: int       # position of the tensor in model order (seeds its values)
    is_norm: bool = False  # RMSNorm weight (config 1 sets these to 1.0)

    @property
    def elem_size(self) -> int:
        return _ELEM[self.dtype]

    @property
    def nbytes(self) -> int:
        return self.numel * self.elem_size


@dataclasses.dataclass(frozen=True)
class RoleConfig:
    index: int
    name: str
    seed: int
    bucket_bytes: int
    shard_r: int
    shard_D: int
    model: Tuple[Tuple[str, int, bool], ...]  # (name, numel, is_norm) in model order
    norms_are_one: bool = False

    def specs(self) -> List[TensorSpec]:
        out: List[TensorSpec] = []
        for plane, dtype in ((PLANE_PARAM, torch.bfloat16), (PLANE_MASTER, torch.float32),
                             (PLANE_M, torch.float32), (PLANE_V, torch.float32)):
            for i, (name, numel, is_norm) in enumerate(self.model):
                out.append(TensorSpec(f"{PLANE_NAMES[plane]}.{name}", numel, dtype, plane, i, is_norm))
        return out

    @property
    def n_params(self) -> int:
        return sum(n for _, n, _ in self.model)


def _gpt_model(layers: int, h: int, ffn: int, vocab: int) -> Tuple[Tuple[str, int, bool], ...]:
    m: List[Tuple[str, int, bool]] = [("embedding", vocab * h, False)]
    for l in range(layers):
        p = f"l{l}."
        m += [(p + "ln1.w", h, False), (p + "ln1.b", h, False),
              (p + "qkv.w", 3 * h * h, False), (p + "qkv.b", 3 * h, False),
              (p + "proj.w", h * h, False), (p + "proj.b", h, False),
              (p + "ln2.w", h, False), (p + "ln2.b", h, False),
              (p + "fc1.w", ffn * h, False), (p + "fc1.b", ffn, False),
              (p + "fc2.w", h * ffn, False), (p + "fc2.b", h, False)]
    m += [("final_ln.w", h, False), ("final_ln.b", h, False)]  # output layer tied to the embedding
    return tuple(m)


def _llama_model(layers: int, h: int, q_out: int, kv_out: int, ffn: int, vocab_rows: int,
                 ends: bool) -> Tuple[Tuple[str, int, bool], ...]:
    """Per-rank Llama-style tensors.  q_out / kv_out / ffn are this rank's share of the split
    dimension (column-split q, k, v, gate, up; row-split o, down; norms replicated)."""
    m: List[Tuple[str, int, bool]] = []
    if ends:
        m.append(("embedding", vocab_rows * h, False))
    for l in range(layers):
        p = f"l{l}."
        m += [(p + "input_norm", h, True),
              (p + "q", h * q_out, False), (p + "k", h * kv_out, False), (p + "v", h * kv_out, False),
              (p + "o", q_out * h, False),
              (p + "post_attn_norm", h, True),
              (p + "gate", h * ffn, False), (p + "up", h * ffn, False), (p + "down", ffn * h, False)]
    if ends:
        m += [("final_norm", h, True), ("lm_head", vocab_rows * h, False)]
    return tuple(m)


MiB = 1 << 20


def role_config(index: int, layers: Optional[int] = None) -> RoleConfig:
    """The four model-shaped role layouts (config 4, the adversarial set, is `adversarial_specs`).
    `layers` overrides the number of transformer layers (reduced cases for profiling)."""
    if layers is not None:
        full = role_config(index)
        assert 0 < layers <= {0: 2, 1: 22, 2: 32, 3: 10}[index]

        def layer_of(name: str) -> int:
            head = name.split(".")[0]
            return int(head[1:]) if head[0] == "l" and head[1:].isdigit() else -1
        keep = tuple(t for t in full.model if layer_of(t[0]) < layers)
        return dataclasses.replace(full, name=f"{full.name}-{layers}layers", model=keep)
    if index == 0:   # tiny GPT, TP=1 PP=1 DP=2
        return RoleConfig(0, "tiny-gpt", 0, 1 * MiB, 1, 2, _gpt_model(2, 256, 1024, 1024))
    if index == 1:   # Llama-style 1.1B, TP=1 PP=1; 32 heads / 4 KV heads, head dim 64
        return RoleConfig(1, "llama-1.1b", 1, 64 * MiB, 5, 16,
                          _llama_model(22, 2048, 2048, 256, 5632, 32000, True), norms_are_one=True)
    if index == 2:   # Llama-3-8B at TP=8 (rank 3), PP=1: 1/8 of every split dimension
        return RoleConfig(2, "llama3-8b-tp8", 2, 128 * MiB, 11, 32,
                          _llama_model(32, 4096, 4096 // 8, 1024 // 8, 14336 // 8, 128256 // 8, True))
    if index == 3:   # Llama-3-70B at TP=8 PP=8, stage 5 (a middle stage: blocks only), TP rank 2
        return RoleConfig(3, "llama3-70b-tp8-pp8", 3, 256 * MiB, 7, 24,
                          _llama_model(10, 8192, 8192 // 8, 1024 // 8, 28672 // 8, 0, False))
    raise ValueError(f"no model-shaped role config {index}")


# ----------------------------------------------------------------------------------------------
# values


def _gen(device: torch.device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _tensor_seed(cfg_seed: int, model_index: int, kind: int) -> int:
    return (cfg_seed * 1_000_003 + model_index) * 8 + kind


def _fill_model_tensor(cfg: RoleConfig, spec: TensorSpec, device: torch.device) -> torch.Tensor:
    """master ~ N(0, 0.02); bf16 param = master rounded to nearest-even; m ~ N(0, 1e-3);
    v ~ |N(0, 1e-6)|.  Norm weights are 1.0 in param and master when the config says so."""
    n = spec.numel
    if spec.plane in (PLANE_PARAM, PLANE_MASTER):
        if cfg.norms_are_one and spec.is_norm:
            return torch.ones(n, dtype=spec.dtype, device=device)
        master = torch.empty(n, dtype=torch.float32, device=device)
        master.normal_(0.0, 0.02, generator=_gen(device, _tensor_seed(cfg.seed, spec.model_index, 1)))
        return master if spec.plane == PLANE_MASTER else master.to(torch.bfloat16)
    t = torch.empty(n, dtype=torch.float32, device=device)
    if spec.plane == PLANE_M:
        t.normal_(0.0, 1e-3, generator=_gen(device, _tensor_seed(cfg.seed, spec.model_index, 2)))
    else:
        t.normal_(0.0, 1e-6, generator=_gen(device, _tensor_seed(cfg.seed, spec.model_index, 3)))
        t.abs_()
    return t


@dataclasses.dataclass
class RoleState:
    """Device (or CPU) tensors of one role plus their specs, in descriptor order."""
    name: str
    specs: List[TensorSpec]
    tensors: List[torch.Tensor]          # 1-D; uint8 views for the adversarial arena
    bucket_bytes: int
    shard_r: int
    shard_D: int
    arena: Optional[torch.Tensor] = None  # keeps the adversarial arena alive

    def descs(self) -> List[Tuple[int, int, int, int]]:
        """(address, nbytes, elem_size, plane) per tensor."""
        return [(t.data_ptr(), s.nbytes, s.elem_size, s.plane) for s, t in zip(self.specs, self.tensors)]

    def descs_of(self, indices: Sequence[int]) -> List[Tuple[int, int, int, int]]:
        """Descriptors of a subset of the tensors, in the order given."""
        return [(self.tensors[i].data_ptr(), self.specs[i].nbytes, self.specs[i].elem_size, self.specs[i].plane)
                for i in indices]

    def subset(self, indices: Sequence[int], name: Optional[str] = None) -> "RoleState":
        """The same tensors restricted to `indices` (order kept) — e.g. the role delta between a middle
        and a first/last pipeline stage: embedding / output layer and their optimizer state."""
        return RoleState(name or f"{self.name}-subset", [self.specs[i] for i in indices],
                         [self.tensors[i] for i in indices], self.bucket_bytes, self.shard_r, self.shard_D,
                         self.arena)

    def plane_indices(self, plane: int) -> List[int]:
        return [i for i, s in enumerate(self.specs) if s.plane == plane]

    def elem_size_indices(self, elem_size: int) -> List[int]:
        return [i for i, s in enumerate(self.specs) if s.elem_size == elem_size]

    def host_bytes(self, k: int) -> np.ndarray:
        """Bytes of tensor k as a numpy uint8 array on the host."""
        return tensor_bytes(self.tensors[k]).cpu().numpy()

    @property
    def state_bytes(self) -> int:
        return sum(s.nbytes for s in self.specs)


def tensor_bytes(t: torch.Tensor) -> torch.Tensor:
    return t if t.dtype == torch.uint8 else t.view(torch.uint8)


def materialize(cfg: RoleConfig, device) -> RoleState:
    """One separate allocation per tensor, so that packing really gathers."""
    device = torch.device(device)
    specs = cfg.specs()
    tensors = [_fill_model_tensor(cfg, s, device) for s in specs]
    return RoleState(cfg.name, specs, tensors, cfg.bucket_bytes, cfg.shard_r, cfg.shard_D)


def blank_like(state: RoleState) -> RoleState:
    """Same tensor list, freshly allocated and filled with 0xA5 bytes (an unpack target)."""
    if state.arena is not None:
        arena = torch.full_like(state.arena, 0xA5)
        base = state.arena.data_ptr()
        tensors = []
        for s, t in zip(state.specs, state.tensors):
            o = t.data_ptr() - base
            tensors.append(arena[o:o + s.nbytes])
        return RoleState(state.name, state.specs, tensors, state.bucket_bytes, state.shard_r,
                         state.shard_D, arena)
    tensors = []
    for t in state.tensors:
        b = torch.full((t.numel() * t.element_size(),), 0xA5, dtype=torch.uint8, device=t.device)
        tensors.append(b.view(t.dtype))
    return RoleState(state.name, state.specs, tensors, state.bucket_bytes, state.shard_r, state.shard_D)


# ----------------------------------------------------------------------------------------------
# config 4: adversarial descriptor set

ADVERSARIAL_SEED = 4
ADVERSARIAL_BUCKET = 8 * MiB
ADVERSARIAL_D = 64
_ADV_DTYPES = (torch.bfloat16, torch.float32, torch.int64)


def adversarial_specs(n_tensors: int = 200_000, seed: int = ADVERSARIAL_SEED,
                      max_log2: int = 22) -> List[TensorSpec]:
    """numel = floor(2^(max_log2*u)), u ~ U[0,1), clipped to [1, 2^max_log2]; dtype i.i.d. uniform
    over {bf16, fp32, int64}.  The first k specs of a larger set equal the smaller set's."""
    rng = np.random.Generator(np.random.PCG64(seed))
    u = rng.random(n_tensors)
    numel = np.clip(np.floor(np.exp2(max_log2 * u)).astype(np.int64), 1, 1 << max_log2)
    dt = np.random.Generator(np.random.PCG64(seed + 104729)).integers(0, 3, n_tensors)
    specs = []
    for i in range(n_tensors):
        dtype = _ADV_DTYPES[int(dt[i])]
        plane = {torch.bfloat16: PLANE_PARAM, torch.float32: PLANE_MASTER, torch.int64: PLANE_OTHER}[dtype]
        specs.append(TensorSpec(f"adv{i}", int(numel[i]), dtype, plane, i))
    return specs


def adversarial_offsets(specs: Sequence[TensorSpec], seed: int = ADVERSARIAL_SEED) -> Tuple[np.ndarray, int]:
    """Arena byte offset of each tensor: consecutive, separated by a random even gap in [0, 256),
    so base addresses have random 2-byte alignment.  Returns (offsets, arena size)."""
    rng = np.random.Generator(np.random.PCG64(seed + 7919))
    gaps = 2 * rng.integers(0, 128, len(specs))
    offs = np.zeros(len(specs), dtype=np.int64)
    pos = 16  # slack before the first tensor
    for i, s in enumerate(specs):
        pos += int(gaps[i])
        offs[i] = pos
        pos += s.nbytes
    return offs, pos + 16


def materialize_adversarial(specs: Sequence[TensorSpec], device, seed: int = ADVERSARIAL_SEED,
                            wave: int = 0) -> RoleState:
    """All tensors live in one uint8 arena at 2-byte-granular addresses.  Values: bf16 / fp32
    ~ N(0, 0.02); int64 ("step counters") uniform in [0, 2^31).  One value pool per dtype, seeded
    by (seed, wave), consumed in tensor order."""
    device = torch.device(device)
    specs = list(specs)
    offs, size = adversarial_offsets(specs, seed + 31 * wave)
    arena = torch.zeros(size, dtype=torch.uint8, device=device)
    totals: Dict[torch.dtype, int] = {d: 0 for d in _ADV_DTYPES}
    for s in specs:
        totals[s.dtype] += s.numel
    pools: Dict[torch.dtype, torch.Tensor] = {}
    base_seed = seed * 7_368_787 + wave
    if totals[torch.float32]:
        p = torch.empty(totals[torch.float32], dtype=torch.float32, device=device)
        p.normal_(0.0, 0.02, generator=_gen(device, base_seed * 4 + 1))
        pools[torch.float32] = p.view(torch.uint8)
    if totals[torch.bfloat16]:
        p = torch.empty(totals[torch.bfloat16], dtype=torch.float32, device=device)
        p.normal_(0.0, 0.02, generator=_gen(device, base_seed * 4 + 2))
        pools[torch.bfloat16] = p.to(torch.bfloat16).view(torch.uint8)
    if totals[torch.int64]:
        p = torch.randint(0, 1 << 31, (totals[torch.int64],), dtype=torch.int64, device=device,
                          generator=_gen(device, base_seed * 4 + 3))
        pools[torch.int64] = p.view(torch.uint8)
    cursor = {d: 0 for d in _ADV_DTYPES}
    tensors = []
    for s, o in zip(specs, offs):
        o = int(o)
        view = arena[o:o + s.nbytes]
        c = cursor[s.dtype]
        view.copy_(pools[s.dtype][c:c + s.nbytes])
        cursor[s.dtype] = c + s.nbytes
        tensors.append(view)
    return RoleState(f"adversarial-{len(specs)}", specs, tensors, ADVERSARIAL_BUCKET, 0,
                     ADVERSARIAL_D, arena)


def odd_specs(seed: int, n_tensors: int = 8) -> List[TensorSpec]:
    """Tiny layout with awkward sizes (1, 3, 127, 129, 255, 257, ... elements), mixed dtypes."""
    rng = np.random.Generator(np.random.PCG64(1000 + seed))
    sizes = [1, 3, 127, 129, 255, 257, 511, 513, 1000, 4097, 65, 31]
    specs = []
    for i in range(n_tensors):
        numel = int(sizes[int(rng.integers(0, len(sizes)))])
        dtype = _ADV_DTYPES[int(rng.integers(0, 3))]
        plane = {torch.bfloat16: PLANE_PARAM, torch.float32: PLANE_MASTER, torch.int64: PLANE_OTHER}[dtype]
        specs.append(TensorSpec(f"odd{i}", numel, dtype, plane, i))
    return specs
