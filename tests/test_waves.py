"""Host-only: waves tile the complete stream, and packing the waves one after another with the
oracle gives the complete stream and the complete checksum list."""
import numpy as np
import pytest

from paper_2412_12636_b200 import waves


@pytest.mark.parametrize("seed,B,budget", [(0, 256, 1024), (1, 512, 512), (2, 1024, 5000), (3, 768, 100000)])
def test_waves_reproduce_the_whole_stream(oracle_mod, seed, B, budget):
    rng = np.random.default_rng(seed)
    tensors = [rng.integers(1, 256, 2 * int(rng.integers(1, 1500)), dtype=np.uint8) for _ in range(25)]
    sizes = [t.size for t in tensors]
    off, T, nb = oracle_mod.layout(sizes, B)
    off = [int(x) for x in off]
    whole, cks = oracle_mod.pack(tensors, B)
    ws = waves.cut_waves(sizes, off, T, B, budget)
    assert ws[0].stream_begin == 0 and ws[-1].stream_end == T
    assert sum(w.n_buckets for w in ws) == nb
    got_stream, got_cks = [], []
    for a, b in zip(ws, ws[1:]):
        assert a.stream_end == b.stream_begin and a.stream_end % B == 0
    for w in ws:
        pieces = [tensors[p.tensor][p.byte_start:p.byte_start + p.nbytes] for p in w.parts]
        assert all(p.byte_start % 256 == 0 for p in w.parts)
        s, c = oracle_mod.pack(pieces, B)
        assert s.size == w.stream_end - w.stream_begin
        got_stream.append(s)
        got_cks.append(c)
    assert np.array_equal(np.concatenate(got_stream), whole)
    assert np.array_equal(np.concatenate(got_cks), cks)
