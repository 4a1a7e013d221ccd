"""Host-only checks of the synthetic role layouts and of the oracle's layout arithmetic at the
full sizes of the four model-shaped configs (sizes only, no data).  Expected numbers were worked
out independently from the model shapes (parameter counts, 14 bytes of state per parameter)."""
import numpy as np
import pytest
import torch

from paper_2412_12636_b200 import layouts

# index: (tensors per plane, parameters N, stream bytes T, buckets, last bucket bytes, shard lo, hi)
EXPECT = {
    0: (27, 1_842_176, 25_790_464, 25, 624_640, 921_088, 1_842_176),
    1: (201, 1_100_048_384, 15_400_677_376, 230, 32_747_520, 343_765_120, 412_518_144),
    2: (291, 1_004_015_616, 14_056_218_624, 105, 97_574_912, 345_130_368, 376_505_856),
    3: (90, 1_069_711_360, 14_975_959_040, 56, 212_008_960, 311_999_146, 356_570_453),
}


@pytest.mark.parametrize("idx", [0, 1, 2, 3])
def test_config_sizes_and_oracle_layout(oracle_mod, idx):
    per_plane, N, T, nb, last, lo, hi = EXPECT[idx]
    cfg = layouts.role_config(idx)
    specs = cfg.specs()
    assert len(cfg.model) == per_plane and len(specs) == 4 * per_plane
    assert cfg.n_params == N
    assert sum(s.nbytes for s in specs) == 14 * N == T     # every tensor is a multiple of 256 bytes
    # plane-major order: bf16 params, then fp32 master, m, v
    assert [s.plane for s in specs] == sorted(s.plane for s in specs)
    off, total, n_buckets = oracle_mod.layout([s.nbytes for s in specs], cfg.bucket_bytes)
    assert (total, n_buckets) == (T, nb)
    assert total - (nb - 1) * cfg.bucket_bytes == last
    assert int(off[per_plane]) == 2 * N                     # the master plane starts after the bf16 plane
    assert oracle_mod.shard_bounds(N, cfg.shard_r, cfg.shard_D) == (lo, hi)


def test_tiny_config_values_follow_the_recipe():
    cfg = layouts.role_config(0)
    st = layouts.materialize(cfg, "cpu")
    again = layouts.materialize(cfg, "cpu")
    P = len(cfg.model)
    for k in (0, 3, P + 3, 2 * P + 3, 3 * P + 3):
        assert torch.equal(st.tensors[k], again.tensors[k])          # seeded
    master, param = st.tensors[P + 3], st.tensors[3]
    assert param.dtype == torch.bfloat16 and torch.equal(param, master.to(torch.bfloat16))
    assert abs(float(master.std()) - 0.02) < 2e-3
    assert abs(float(st.tensors[2 * P + 3].std()) - 1e-3) < 1e-4
    assert float(st.tensors[3 * P + 3].min()) >= 0.0
    one = layouts.role_config(1)
    spec = [s for s in one.specs() if s.is_norm][0]
    assert torch.all(layouts._fill_model_tensor(one, spec, torch.device("cpu")) == 1.0)


def test_adversarial_specs_distribution_and_alignment():
    specs = layouts.adversarial_specs(20_000)
    numel = np.array([s.numel for s in specs])
    assert numel.min() >= 1 and numel.max() <= 1 << 22
    # log-uniform: about half the tensors below 2^11 elements
    assert 0.45 < np.mean(numel < 2048) < 0.55
    assert {s.elem_size for s in specs} == {2, 4, 8}
    assert layouts.adversarial_specs(100) == specs[:100]              # prefix property
    small = layouts.materialize_adversarial(specs[:300], "cpu")
    addr = np.array([t.data_ptr() for t in small.tensors])
    assert np.all(addr % 2 == 0) and len(set(addr % 16)) == 8        # every even residue occurs
    ends = addr + np.array([s.nbytes for s in small.specs])
    assert np.all(addr[1:] >= ends[:-1])                              # disjoint
    blank = layouts.blank_like(small)
    assert all(int(t[0]) == 0xA5 for t in blank.tensors[:5])
    assert [t.data_ptr() - blank.arena.data_ptr() for t in blank.tensors] == \
           [t.data_ptr() - small.arena.data_ptr() for t in small.tensors]
