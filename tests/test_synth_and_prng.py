"""The three splitmix64 writers (input generator, oracle; the CUDA library's is checked in the GPU-free
ABI test) against the generator's published test vector, and sanity of the synthetic inputs."""
import os

import numpy as np

import oracle
import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "splitmix64_seed1234567.txt")


def golden_words():
    with open(GOLDEN) as f:
        return np.array([int(l) for l in f if l.strip() and not l.startswith("#")], dtype=np.uint64)


def test_splitmix64_published_vector():
    g = golden_words()
    np.testing.assert_array_equal(synth.splitmix64_words(1234567, len(g)), g)
    np.testing.assert_array_equal(oracle.splitmix64(1234567, len(g)), g)


def test_splitmix64_writers_agree_on_edge_seeds():
    for seed in (0, 1, 2 ** 64 - 1, 0x5EED0002):
        np.testing.assert_array_equal(synth.splitmix64_words(seed, 1000), oracle.splitmix64(seed, 1000))
    np.testing.assert_array_equal(synth.splitmix64_words(7, 10, skip=5), oracle.splitmix64(7, 15)[5:])


def test_normals_and_labels_look_right():
    z = synth.standard_normal(42, 200001)
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1) < 0.01 and z.shape == (200001,)
    c = synth.config(2)
    x, y = synth.batch(c, 0, 0, 0, B=16)
    assert x.shape == (16, 32, 32, 3) and y.shape == (16,) and y.min() >= 0 and y.max() < 10
    np.testing.assert_array_equal(x, synth.round_to_bf16(x))          # bf16 configs get bf16-exact pixels
    x2, _ = synth.batch(c, 0, 0, 1, B=16)
    assert not np.array_equal(x, x2)


def test_param_layout_matches_oracle_layout_and_init_scale():
    for cfg in (1, 2, 3, 4):
        arch = synth.config(cfg).arch
        ts, n, nb = synth.param_layout(arch)
        assert (n, nb) == oracle.param_count(arch.to_int32())
        r = oracle.block_ranges(arch.to_int32())
        for b in range(len(arch.blocks)):
            mine = [t for t in ts if t.block == b]
            assert mine[0].offset == r[b, 0] and mine[-1].offset + mine[-1].size == r[b, 1]
    p, buf = synth.init_params(synth.config(2).arch, 5)
    t = [t for t in synth.param_layout(synth.config(2).arch)[0] if t.name == "block20.conv1"][0]
    w = p[t.offset:t.offset + t.size]
    assert abs(w.std() - np.sqrt(2.0 / (9 * 32))) < 0.005


def test_bf16_rounding_helper_matches_torch():
    import torch
    x = synth.standard_normal(3, 10000).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16)
    np.testing.assert_array_equal(synth.round_to_bf16(x), ref.to(torch.float32).numpy())
    np.testing.assert_array_equal(synth.bf16_bits(x), ref.view(torch.int16).numpy().view(np.uint16))
