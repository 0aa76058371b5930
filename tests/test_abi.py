"""GPU-free checks of the C boundary: the library builds, loads, and exports every symbol include/resist.h
declares; its splitmix64 agrees with the published vector and the other two writers."""
import os
import re

import numpy as np

import oracle
import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    src = open(os.path.join(ROOT, "include", "resist.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(resist_[a-z0-9_]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    import paper_2107_00961_b200 as m
    L = m.lib()
    syms = declared_symbols()
    assert "resist_init" in syms and "resist_partition" in syms and "resist_local_step" in syms
    assert "resist_aggregate" in syms and "resist_eval" in syms
    for s in syms:
        assert hasattr(L, s), s
    assert sorted(m.EXPORTS) == [s for s in syms if s in m.EXPORTS] and set(syms) <= set(m.EXPORTS)


def test_library_splitmix64_matches_published_vector_and_other_writers():
    import paper_2107_00961_b200 as m
    g = [int(l) for l in open(os.path.join(ROOT, "tests", "golden", "splitmix64_seed1234567.txt")) if l.strip() and not l.startswith("#")]
    np.testing.assert_array_equal(m.resist_splitmix64(1234567, len(g)), np.array(g, dtype=np.uint64))
    for seed in (0, 1, 2 ** 64 - 1):
        w = m.resist_splitmix64(seed, 1000)
        np.testing.assert_array_equal(w, oracle.splitmix64(seed, 1000))
        np.testing.assert_array_equal(w, synth.splitmix64_words(seed, 1000))


def test_no_cpu_fallback_without_a_device():
    import torch
    import paper_2107_00961_b200 as m
    if torch.cuda.is_available():
        return
    try:
        m.Context(synth.tiny_arch().to_int32())
    except RuntimeError as e:
        assert "CUDA" in str(e)
    else:
        raise AssertionError("a context must not be creatable without a GPU")
