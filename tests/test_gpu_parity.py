"""GPU parity: the CUDA library, called through its C boundary, against the CPU oracle on the same seeded inputs.

Tolerances: partitions and the reassembly are bit-exact; the fp32 path is within 1e-4 max relative error
(elements below 1e-3 of their tensor's scale are compared against that scale); the bf16 path is within 2e-2
normalised max-abs error of the fp32 oracle.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
from parity import LR, MOM, max_rel_err, norm_max_abs, per_tensor, run_protocol_both, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lib_mod():
    import paper_2107_00961_b200 as m
    m.lib()
    return m


def small_bottleneck_arch(policy="paper_section3"):
    return synth.Arch(20, 20, 3, 7, 7, 2, 8, 1, 1,
                      synth._stack(synth.BOTTLENECK, 8, (1, 2, 3, 1), (16, 32, 64, 128), (8, 8, 16, 32), policy))


def check_fp32(out, arch, tol=1e-4):
    np.testing.assert_array_equal(out["mask_gpu"], out["mask_cpu"])
    for rec in out["steps"]:
        for s, r in enumerate(rec["subs"]):
            assert max_rel_err(r["logits_gpu"], r["logits_cpu"]) < tol
            assert abs(rec["loss_gpu"][s] - r["loss_cpu"]) < tol * max(1.0, abs(r["loss_cpu"]))
            v, name = per_tensor(arch, r["grads_gpu"], r["grads_cpu"], max_rel_err)
            assert v < tol, ("grads", name, v)
            v, name = per_tensor(arch, r["params_gpu"], r["params_cpu"], max_rel_err)
            assert v < tol, ("params", name, v)
            assert max_rel_err(r["bufs_gpu"], r["bufs_cpu"]) < tol
    np.testing.assert_array_equal(out["global_gpu"], out["global_from_gpu_subs"])          # reassembly: bit-exact
    np.testing.assert_array_equal(out["global_buf_gpu"], out["global_buf_from_gpu_subs"])
    v, name = per_tensor(arch, out["global_gpu"], out["global_cpu"], max_rel_err)
    assert v < tol, ("global", name, v)


@pytest.mark.parametrize("grouped", [False, True])
def test_config1_tiny_fp32_round(lib_mod, grouped):
    c = synth.config(1)
    out = run_protocol_both(c.arch, c.S, c.batch, c.local_steps, 5, "f32", 0, grouped, lib_mod, policy_seed=c.round_seed(0))
    check_fp32(out, c.arch)
    assert out["info"]["kernel_launches"] > 0 and out["info"]["conv_flops"] > 0


def test_grouped_and_single_steps_agree_bitwise(lib_mod):
    c = synth.config(1)
    a = run_protocol_both(c.arch, 2, 8, 2, 9, "f32", 0, False, lib_mod)
    b = run_protocol_both(c.arch, 2, 8, 2, 9, "f32", 0, True, lib_mod)
    np.testing.assert_array_equal(a["global_gpu"], b["global_gpu"])
    # and the same call twice gives the same bits (fixed-order reductions)
    c2 = run_protocol_both(c.arch, 2, 8, 2, 9, "f32", 0, True, lib_mod)
    np.testing.assert_array_equal(b["global_gpu"], c2["global_gpu"])
    np.testing.assert_array_equal(b["steps"][-1]["subs"][1]["grads_gpu"], c2["steps"][-1]["subs"][1]["grads_gpu"])


@pytest.mark.parametrize("grouped", [False, True])
def test_bottleneck_imagenet_stem_fp32(lib_mod, grouped):
    arch = small_bottleneck_arch()
    out = run_protocol_both(arch, 2, 6, 2, 13, "f32", 0, grouped, lib_mod)
    check_fp32(out, arch)


def test_fp32_ragged_sizes_span_tiles(lib_mod):
    # 3-stage basic net at 20x12 input, batch 5: M = 1200, 300, 75 rows: several 64-row tiles and ragged tails
    arch = synth.Arch(20, 12, 3, 11, 3, 1, 24, 0, 0, synth._stack(synth.BASIC, 24, (2, 3, 2), (24, 40, 72), (24, 40, 72), "stage_first_shared"))
    out = run_protocol_both(arch, 3, 5, 1, 21, "f32", 0, True, lib_mod)
    check_fp32(out, arch)


def check_bf16(out, arch, tol=2e-2):
    np.testing.assert_array_equal(out["mask_gpu"], out["mask_cpu"])
    for rec in out["steps"]:
        for s, r in enumerate(rec["subs"]):
            assert norm_max_abs(r["logits_gpu"], r["logits_cpu"]) < tol
            v, name = per_tensor(arch, r["grads_gpu"], r["grads_cpu"], norm_max_abs)
            assert v < tol, ("grads", name, v)
            v, name = per_tensor(arch, r["params_gpu"], r["params_cpu"], norm_max_abs)
            assert v < tol, ("params", name, v)
    np.testing.assert_array_equal(out["global_gpu"], out["global_from_gpu_subs"])
    np.testing.assert_array_equal(out["global_buf_gpu"], out["global_buf_from_gpu_subs"])


@pytest.mark.parametrize("backend", [1, 0])
def test_tiny_bf16_against_fp32_oracle(lib_mod, backend):
    c = synth.config(1)
    out = run_protocol_both(c.arch, 2, 8, 1, 5, "bf16", 0, True, lib_mod, conv_backend=backend)
    check_bf16(out, c.arch)


@pytest.mark.parametrize("backend", [1, 0])
def test_resnet110_bf16_reduced_batch(lib_mod, backend):
    # configuration 2's network and S at batch 8 (the oracle finishes in seconds); one local step
    c = synth.config(2)
    out = run_protocol_both(c.arch, c.S, 8, 1, 31, "bf16", 0, True, lib_mod, policy_seed=c.round_seed(0), conv_backend=backend)
    check_bf16(out, c.arch)
    # against the oracle that rounds storage to bf16 at the same points the agreement is much tighter
    out_q = run_protocol_both(c.arch, c.S, 8, 1, 31, "bf16", 1, True, lib_mod, policy_seed=c.round_seed(0), conv_backend=backend)
    check_bf16(out_q, c.arch, tol=1e-2)


def test_eval_matches_oracle(lib_mod):
    for arch in (synth.tiny_arch(), small_bottleneck_arch()):
        a = arch.to_int32()
        p, buf = synth.perturbed_params(arch, 3)
        buf = (buf + 0.1 * np.abs(synth.standard_normal(5, buf.size))).astype(np.float32)
        ctx = lib_mod.Context(a, dtype=lib_mod.F32)
        ctx.set_params(p, buf)
        ctx.partition(1, 2)
        B = 5
        x = synth.standard_normal(8, B * arch.in_h * arch.in_w * arch.in_c).astype(np.float32).reshape(B, arch.in_h, arch.in_w, arch.in_c)
        y = (synth.splitmix64_words(9, B) % np.uint64(arch.classes)).astype(np.int32)
        logits, loss, correct = ctx.eval(to_dev(x, torch.float32), to_dev(y, None))
        ref = oracle.evaluate(a, p, buf, 2, x, y)
        assert max_rel_err(logits.cpu().numpy(), ref["logits"]) < 1e-4
        assert abs(loss.item() - ref["loss"]) < 1e-4 * max(1, abs(ref["loss"]))
        assert correct.item() == ref["correct"]


def test_min_depth_partition_and_partial_sharing(lib_mod):
    arch = synth.Arch(8, 8, 3, 10, 3, 1, 8, 0, 0, synth._stack(synth.BASIC, 8, (6,), (8,), (8,), "stage_first_shared"))
    a = arch.to_int32()
    ctx = lib_mod.Context(a, dtype=lib_mod.F32, min_depth=3)
    for seed in (5, 6, 7):
        np.testing.assert_array_equal(ctx.partition(seed, 2), oracle.partition(a, seed, 2, min_depth=3))
    out_mask = ctx.partition(5, 2)
    assert any(m == 3 for m in out_mask[1:])          # one block sits in both sub-ResNets (Fig. 1)


def test_partition_bit_exact_on_all_configs(lib_mod):
    for cfg in (1, 2, 3, 4):
        c = synth.config(cfg)
        a = c.arch.to_int32()
        ctx = lib_mod.Context(a, dtype=lib_mod.F32)
        for t in range(4):
            np.testing.assert_array_equal(ctx.partition(c.round_seed(t), c.S), oracle.partition(a, c.round_seed(t), c.S))
        ctx.close()


def test_reassembly_stress_bit_exact(lib_mod):
    # ResNet-101 parameter set, S in {2,4,8}: working copies = global + N(0,1e-3) deltas; aggregate must equal
    # the oracle bit for bit; single-owner blocks are copies
    c = synth.config(5)
    a = c.arch.to_int32()
    ctx = lib_mod.Context(a, dtype=lib_mod.BF16)
    p0, b0 = ctx.get_params(-1)
    n = ctx.n_params
    for S in (2, 4, 8):
        mask = ctx.partition(c.round_seed(S), S)
        np.testing.assert_array_equal(mask, oracle.partition(a, c.round_seed(S), S))
        subs = []
        for s in range(S):
            w, _ = ctx.get_params(s)
            subs.append(w)
        # the scatter copied the held blocks bit for bit
        r = oracle.block_ranges(a)
        for s in range(S):
            held = np.ones(n, bool)
            for b in range(len(c.arch.blocks)):
                if not (mask[b] >> s & 1):
                    held[r[b, 0]:r[b, 1]] = False
            np.testing.assert_array_equal(subs[s][held], p0[held])
        ctx.aggregate()
        g, gb = ctx.get_params(-1)
        np.testing.assert_array_equal(g, p0)           # identical copies: the identity
        np.testing.assert_array_equal(gb, b0)
    ctx.close()


def test_error_paths(lib_mod):
    a = synth.tiny_arch().to_int32()
    ctx = lib_mod.Context(a, dtype=lib_mod.F32)
    x = torch.zeros(4, 8, 8, 3, device="cuda")
    y = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(lib_mod.ResistError) as e:
        ctx.local_step(0, x, y, 0.1)
    assert e.value.code == -2                           # step before partition
    with pytest.raises(lib_mod.ResistError) as e:
        ctx.aggregate()
    assert e.value.code == -2
    with pytest.raises(lib_mod.ResistError) as e:
        ctx.partition(1, 4)                             # S > P without a minimum depth
    assert e.value.code == -1
    with pytest.raises(lib_mod.ResistError):
        ctx.partition(1, 33)
    ctx.partition(1, 2)
    with pytest.raises(lib_mod.ResistError) as e:
        ctx.local_step(2, x, y, 0.1)                    # subnet >= S
    assert e.value.code == -1
    with pytest.raises(lib_mod.ResistError):
        ctx.local_step(0, x[:1], y[:1], 0.1)            # B < 2
    ctx.local_step(0, x, y, 0.1)                        # and the context still works
    torch.cuda.synchronize()
    bad = a.copy()
    bad[10 + 2] = 5                                     # first block's cin no longer matches the stem
    with pytest.raises(lib_mod.ResistError):
        lib_mod.Context(bad, dtype=lib_mod.F32)
