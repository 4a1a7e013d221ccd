"""Mutation check of the oracle's pins.  Each mutant is a copy of oracle/tm_oracle.cpp with one
plausible mistake planted (a dropped term, a wrong sign or index, a swapped byte order, a wrong
rounding); it is compiled on the CPU and the pin tests of test_oracle_pins.py are run against it.
Every mutant must be caught by at least one pin — otherwise the pins would let that mistake through
in the real oracle.  Nothing here touches the GPU."""
import itertools
import os
import subprocess

import pytest

import test_oracle_pins as pins

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "tm_oracle.cpp")

# (name, text to find, replacement); the text must occur exactly `count` times (default 1)
MUTANTS = [
    ("weight_2i", "C += w * (2 * i + 1);", "C += w * (2 * i);"),
    ("weight_2i_plus_2", "C += w * (2 * i + 1);", "C += w * (2 * i + 2);"),
    ("weight_i_plus_1", "C += w * (2 * i + 1);", "C += w * (i + 1);"),
    ("big_endian_words", "w |= byte << (8 * b);", "w |= byte << (8 * (7 - b));"),
    ("ragged_tail_dropped", "uint64_t n = (L + 7) / 8;", "uint64_t n = L / 8;"),
    ("index_not_restarted", "out[j] = checksum_one(bytes + begin, end - begin);",
     "out[j] = checksum_one(bytes, end) - (j == 0 ? 0 : checksum_one(bytes, begin));"),
    ("align_128", "uint64_t rem = x % 256;\n  if (rem == 0) return x;\n  return x + (256 - rem);",
     "uint64_t rem = x % 128;\n  if (rem == 0) return x;\n  return x + (128 - rem);"),
    ("bucket_count_plus_one", "*n_buckets = (T + B - 1) / B;", "*n_buckets = (T + B) / B;"),   # memory-safe: over-counts
    ("total_not_padded", "uint64_t T = round_up_256(pos);\n  if (total != NULL)", "uint64_t T = pos;\n  if (total != NULL)"),
    ("padding_not_zero", "for (uint64_t i = 0; i < T; ++i) out[i] = 0;", "for (uint64_t i = 0; i < T; ++i) out[i] = 1;"),
    ("pack_reversed_bytes", "out[pos + j] = src[j];", "out[pos + j] = src[nbytes[k] - 1 - j];"),
    ("pack_range_off_by_one", "if (s >= lo && s < hi) out[s - lo] = ptrs[k][j];",
     "if (s > lo && s < hi) out[s - lo] = ptrs[k][j];"),
    ("unpack_swapped_pairs", "dst[j] = stream[pos + j];", "dst[j] = stream[pos + (j ^ 1)];"),
    ("shard_lo_ceil", "*lo = (uint64_t)(a / D);", "*lo = (uint64_t)((a + D - 1) / D);"),
    ("shard_hi_plus_one_rank", "unsigned __int128 b = ((unsigned __int128)r + 1) * (unsigned __int128)N;",
     "unsigned __int128 b = ((unsigned __int128)r + 2) * (unsigned __int128)N;"),
    ("shard_64_bit_product", "unsigned __int128 a = (unsigned __int128)r * (unsigned __int128)N;",
     "unsigned __int128 a = (uint64_t)((uint64_t)r * N);"),
    ("shard_element_bytes_swapped", "out[(g - lo) * e + b] = ptrs[k][idx * e + b];",
     "out[(g - lo) * e + b] = ptrs[k][idx * e + (e - 1 - b)];"),
    ("shard_range_inclusive", "if (g >= lo && g < hi) {\n        if (ptrs[k] == NULL) return ORC_ERR_ARG;\n        for (uint32_t b = 0; b < e; ++b) out",
     "if (g > lo && g < hi) {\n        if (ptrs[k] == NULL) return ORC_ERR_ARG;\n        for (uint32_t b = 0; b < e; ++b) out"),
    ("insert_element_bytes_swapped", "ptrs[k][idx * e + b] = in[(g - lo) * e + b];",
     "ptrs[k][idx * e + b] = in[(g - lo) * e + (e - 1 - b)];"),
]


def _expand(fn):
    """All parameter combinations of a (possibly parametrized) pin test, as keyword dictionaries."""
    axes = []
    for mark in getattr(fn, "pytestmark", []):
        if mark.name == "parametrize":
            names = [n.strip() for n in mark.args[0].split(",")]
            values = [v if isinstance(v, (tuple, list)) and len(names) > 1 else (v,) for v in mark.args[1]]
            axes.append([dict(zip(names, v)) for v in values])
    for combo in itertools.product(*axes):
        kw = {}
        for d in combo:
            kw.update(d)
        yield kw


def run_all_pins(oracle_mod):
    """Runs every pin; returns the names of the pins that failed."""
    failed = []
    for name in sorted(dir(pins)):
        fn = getattr(pins, name)
        if not (name.startswith("test_") and callable(fn)):
            continue
        for kw in _expand(fn):
            try:
                fn(oracle_mod, **kw)
            except (AssertionError, oracle_mod.OracleError, ValueError, IndexError):
                failed.append(name)
                break
    return failed


def test_the_real_oracle_passes_this_runner(oracle_mod):
    assert run_all_pins(oracle_mod) == []


@pytest.mark.parametrize("name,find,replace", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_every_planted_mistake_is_caught(oracle_mod, tmp_path, name, find, replace):
    src = open(SRC).read()
    assert src.count(find) == 1, f"mutant {name}: pattern occurs {src.count(find)} times"
    mutant_cpp = tmp_path / f"{name}.cpp"
    mutant_so = tmp_path / f"{name}.so"
    mutant_cpp.write_text(src.replace(find, replace))
    subprocess.run(["g++", "-std=c++17", "-O1", "-fPIC", "-shared", "-o", str(mutant_so), str(mutant_cpp)], check=True)
    with oracle_mod.use_library(str(mutant_so)):
        failed = run_all_pins(oracle_mod)
    assert failed, f"no pin noticed the planted mistake '{name}'"
