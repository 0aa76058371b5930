"""Pins for the oracle's sub-ResNet step, evaluation, reassembly and partition (CPU only).

The whole step is checked against torch.nn.functional + autograd in fp64 (library routines strung
together in this file, independently of the oracle), against central finite differences of the
oracle's own loss, against the paper's statements (absent block = identity map, Appendix B;
single owner = copy, Sec. 2.3; the one-step identity for the aggregated weights, Appendix B),
and against closed forms (SGD with momentum on a fixed gradient).
"""
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ an independent fp64 restatement with autograd
def torch_net(arch, params, images, labels, present, train=True, buffers=None, S=1, eps=1e-5):
    ts, n, _ = synth.param_layout(arch)
    P = {t.name: params[t.offset:t.offset + t.size].reshape(t.shape) for t in ts}
    bufs = {}
    if buffers is not None:
        o = 0
        for t in ts:
            if t.kind == "gamma":
                c = t.size
                bufs[t.name[:-6]] = (buffers[o:o + c], buffers[o + c:o + 2 * c])
                o += 2 * c

    def conv(x, name, stride):
        w = P[name].permute(0, 3, 1, 2)
        return F.conv2d(x, w, stride=stride, padding=(w.shape[-1] - 1) // 2)

    def bn(x, name):
        if train:
            return F.relu(F.batch_norm(x, None, None, P[name + ".gamma"], P[name + ".beta"], training=True, eps=eps))
        rm, rv = bufs[name]
        return F.relu(F.batch_norm(x, rm, rv, P[name + ".gamma"], P[name + ".beta"], training=False, eps=eps))

    x = conv(images.permute(0, 3, 1, 2), "stem.conv", arch.stem_stride)
    if arch.stem_bn_relu:
        x = bn(x, "stem.bn")
    if arch.stem_maxpool:
        x = F.max_pool2d(x, 3, 2, 1)
    for i, b in enumerate(arch.blocks):
        if not present[i]:
            continue
        p = f"block{i}"
        scale = (1.0 / S) if (not train and b.partitionable) else 1.0
        a1 = bn(x, p + ".bn1")
        sc = conv(a1, p + ".proj", b.stride) if b.has_projection else x
        if b.kind == synth.BASIC:
            z = conv(bn(conv(a1, p + ".conv1", b.stride), p + ".bn2"), p + ".conv2", 1)
        else:
            z = conv(bn(conv(a1, p + ".conv1", 1), p + ".bn2"), p + ".conv2", b.stride)
            z = conv(bn(z, p + ".bn3"), p + ".conv3", 1)
        x = sc + scale * z
    x = bn(x, "final.bn").mean(dim=(2, 3))
    logits = x @ P["head.w"].T + P["head.b"]
    return logits, F.cross_entropy(logits, labels)


def small_bottleneck_arch():
    """A 4-stage bottleneck net with an ImageNet-style stem (7x7 s2 conv, BN, ReLU, max-pool), small enough
    for fp64 autograd: covers the stem BN, the pool, strided 3x3 and projection shortcuts."""
    return synth.Arch(20, 20, 3, 7, 7, 2, 4, 1, 1,
                      synth._stack(synth.BOTTLENECK, 4, (1, 2, 3, 1), (8, 16, 32, 64), (2, 4, 8, 16), "paper_section3"))


def case(arch, B, seed, dtype=np.float64):
    p, buf = synth.perturbed_params(arch, seed)
    n = B * arch.in_h * arch.in_w * arch.in_c
    x = synth.standard_normal(seed + 1, n).reshape(B, arch.in_h, arch.in_w, arch.in_c)
    y = (synth.splitmix64_words(seed + 2, B) % np.uint64(arch.classes)).astype(np.int32)
    return p.astype(dtype), buf.astype(dtype), x.astype(dtype), y


@pytest.mark.parametrize("which", ["tiny_full", "tiny_sub", "bottleneck_full", "bottleneck_sub"])
def test_step_matches_autograd(which):
    arch = synth.tiny_arch() if which.startswith("tiny") else small_bottleneck_arch()
    B = 4
    p, buf, x, y = case(arch, B, 11)
    present = np.ones(len(arch.blocks), dtype=np.uint8)
    if which.endswith("sub"):
        for i, b in enumerate(arch.blocks):
            if b.partitionable and i % 2 == 1:
                present[i] = 0
        assert present.sum() < len(arch.blocks)
    tp = torch.from_numpy(p.copy()).requires_grad_()
    logits, loss = torch_net(arch, tp, torch.from_numpy(x), torch.from_numpy(y).long(), present)
    loss.backward()
    out = oracle.step(arch.to_int32(), present, p.copy(), np.zeros_like(p), buf.copy(), x, y, do_update=False)
    np.testing.assert_allclose(out["logits"], logits.detach().numpy(), rtol=1e-9, atol=1e-10)
    assert abs(out["loss"] - loss.item()) < 1e-10
    g_ref = tp.grad.numpy()
    scale = np.abs(g_ref).max()
    np.testing.assert_allclose(out["grads"], g_ref, rtol=1e-7, atol=1e-9 * scale)
    # absent blocks receive exactly zero gradient
    rng = oracle.block_ranges(arch.to_int32())
    for i in np.nonzero(present == 0)[0]:
        assert not out["grads"][rng[i, 0]:rng[i, 1]].any()


def test_step_gradient_by_finite_differences():
    arch = synth.tiny_arch()
    p, buf, x, y = case(arch, 4, 5)
    present = np.array([1, 1, 1, 0, 1, 1], dtype=np.uint8)
    a = arch.to_int32()
    g = oracle.step(a, present, p.copy(), np.zeros_like(p), None, x, y, do_update=False)["grads"]
    ts, n, _ = synth.param_layout(arch)
    rs = np.random.default_rng(0)
    h = 1e-6
    for t in ts:
        if t.block == 3:
            continue
        for i in rs.choice(t.size, size=min(3, t.size), replace=False):
            j = t.offset + int(i)
            pp, pm = p.copy(), p.copy()
            pp[j] += h
            pm[j] -= h
            lp = oracle.step(a, present, pp, np.zeros_like(p), None, x, y, do_update=False)["loss"]
            lm = oracle.step(a, present, pm, np.zeros_like(p), None, x, y, do_update=False)["loss"]
            fd = (lp - lm) / (2 * h)
            assert abs(fd - g[j]) < 1e-6 * max(1.0, abs(fd)) + 2e-7, (t.name, i, fd, g[j])


def test_absent_block_is_identity_bit_exact():
    # Appendix B: an absent block contributes its term times M = 0.  So the sub-ResNet's logits equal the
    # full net's logits when the absent blocks' last convolution is zero: bit for bit, in fp32.
    arch = synth.tiny_arch()
    p, buf, x, y = case(arch, 8, 3, np.float32)
    present = np.array([1, 0, 1, 1, 1, 0], dtype=np.uint8)
    ts, _, _ = synth.param_layout(arch)
    pz = p.copy()
    for t in ts:
        if t.name in ("block1.conv2", "block5.conv2"):
            pz[t.offset:t.offset + t.size] = 0
    a = arch.to_int32()
    sub = oracle.step(a, present, p.copy(), np.zeros_like(p), None, x, y, do_update=False)
    full = oracle.step(a, np.ones(6, np.uint8), pz, np.zeros_like(p), None, x, y, do_update=False)
    np.testing.assert_array_equal(sub["logits"], full["logits"])
    assert sub["loss"] == full["loss"]


def test_gamma_zero_block_outputs_its_shortcut():
    arch = synth.tiny_arch()
    p, buf, x, y = case(arch, 4, 9)
    ts, _, _ = synth.param_layout(arch)
    pz = p.copy()
    for t in ts:                       # gamma2 = beta2 = 0 => relu(bn2(.)) = 0 => conv2 output 0 => out = shortcut
        if t.name in ("block1.bn2.gamma", "block1.bn2.beta"):
            pz[t.offset:t.offset + t.size] = 0
    a = arch.to_int32()
    l1 = oracle.step(a, np.ones(6, np.uint8), pz, np.zeros_like(p), None, x, y, do_update=False)["logits"]
    l2 = oracle.step(a, np.array([1, 0, 1, 1, 1, 1], np.uint8), p.copy(), np.zeros_like(p), None, x, y, do_update=False)["logits"]
    np.testing.assert_allclose(l1, l2, rtol=1e-12, atol=1e-12)


def test_uniform_logits_loss_is_log_classes():
    arch = synth.tiny_arch()
    p, buf, x, y = case(arch, 4, 2)
    ts, _, _ = synth.param_layout(arch)
    for t in ts:
        if t.name.startswith("head"):
            p[t.offset:t.offset + t.size] = 0
    out = oracle.step(arch.to_int32(), np.ones(6, np.uint8), p, np.zeros_like(p), None, x, y, do_update=False)
    assert abs(out["loss"] - np.log(10.0)) < 1e-12


def test_sgd_momentum_closed_form():
    # With the head as the only moving part on a fixed batch the gradient still changes, so pin the update
    # rule itself: first step v = g (momentum restarted), w1 = w0 - lr*g; second step v = mu*g1 + g2.
    arch = synth.tiny_arch()
    p0, buf, x, y = case(arch, 4, 4)
    a = arch.to_int32()
    ones = np.ones(6, np.uint8)
    g1 = oracle.step(a, ones, p0.copy(), np.zeros_like(p0), None, x, y, do_update=False)["grads"]
    p, v = p0.copy(), np.zeros_like(p0)
    oracle.step(a, ones, p, v, None, x, y, lr=0.05, mu=0.9, do_update=True)
    np.testing.assert_allclose(v, g1, rtol=0, atol=0)
    np.testing.assert_allclose(p, p0 - 0.05 * g1, rtol=1e-15, atol=1e-18)
    g2 = oracle.step(a, ones, p.copy(), np.zeros_like(p0), None, x, y, do_update=False)["grads"]
    p1 = p.copy()
    oracle.step(a, ones, p, v, None, x, y, lr=0.05, mu=0.9, do_update=True)
    np.testing.assert_allclose(v, 0.9 * g1 + g2, rtol=1e-14, atol=1e-18)
    np.testing.assert_allclose(p, p1 - 0.05 * (0.9 * g1 + g2), rtol=1e-14, atol=1e-18)
    # weight decay enters the gradient: g + wd*w
    p, v = p0.copy(), np.zeros_like(p0)
    oracle.step(a, ones, p, v, None, x, y, lr=0.05, mu=0.9, wd=0.01, do_update=True)
    np.testing.assert_allclose(v, g1 + 0.01 * p0, rtol=1e-14, atol=1e-18)


def test_absent_blocks_are_not_updated():
    arch = synth.tiny_arch()
    p0, buf0, x, y = case(arch, 4, 6)
    present = np.array([1, 0, 1, 1, 1, 0], np.uint8)
    p, v, buf = p0.copy(), np.zeros_like(p0), buf0.copy()
    oracle.step(arch.to_int32(), present, p, v, buf, x, y, wd=0.1)
    r = oracle.block_ranges(arch.to_int32())
    for i in (1, 5):
        np.testing.assert_array_equal(p[r[i, 0]:r[i, 1]], p0[r[i, 0]:r[i, 1]])
        np.testing.assert_array_equal(buf[r[i, 2]:r[i, 3]], buf0[r[i, 2]:r[i, 3]])
    assert (p[r[0, 0]:r[0, 1]] != p0[r[0, 0]:r[0, 1]]).any()


def test_eval_matches_library_with_one_over_S_scaling():
    for arch in (synth.tiny_arch(), small_bottleneck_arch()):
        p, buf, x, y = case(arch, 3, 21)
        buf = buf + 0.1 * np.abs(synth.standard_normal(77, buf.size))
        S = 4
        ref_logits, ref_loss = torch_net(arch, torch.from_numpy(p), torch.from_numpy(x), torch.from_numpy(y).long(),
                                         np.ones(len(arch.blocks)), train=False, buffers=torch.from_numpy(buf), S=S)
        out = oracle.evaluate(arch.to_int32(), p, buf, S, x, y)
        np.testing.assert_allclose(out["logits"], ref_logits.numpy(), rtol=1e-9, atol=1e-10)
        assert abs(out["loss"] - ref_loss.item()) < 1e-10
        assert out["correct"] == int((ref_logits.argmax(1).numpy() == y).sum())


# ------------------------------------------------------------------ reassembly
def test_aggregate_single_owner_is_a_bit_copy_and_identical_copies_are_identity():
    arch = synth.tiny_arch()
    a = arch.to_int32()
    n, nb = oracle.param_count(a)
    rs = np.random.default_rng(1)
    for S in (2, 4, 8):
        mask = oracle.partition(a, 99, min(S, 3)) if S <= 3 else None
        if mask is None:
            # S > P = 3 is refused without a minimum depth: build a legal mask by hand (blocks 1,3,5 single-owner)
            allm = np.uint32((1 << S) - 1)
            mask = np.array([allm, 1, allm, 2, allm, 4], dtype=np.uint32)
        subs = [rs.standard_normal(n).astype(np.float32) for _ in range(S)]
        sbuf = [rs.standard_normal(nb).astype(np.float32) for _ in range(S)]
        g, gb = np.zeros(n, np.float32), np.zeros(nb, np.float32)
        oracle.aggregate(a, mask, subs, sbuf, g, gb)
        r = oracle.block_ranges(a)
        for b in range(len(arch.blocks)):
            owners = [s for s in range(S) if mask[b] >> s & 1]
            if len(owners) == 1:
                np.testing.assert_array_equal(g[r[b, 0]:r[b, 1]], subs[owners[0]][r[b, 0]:r[b, 1]])
                np.testing.assert_array_equal(gb[r[b, 2]:r[b, 3]], sbuf[owners[0]][r[b, 2]:r[b, 3]])
        # shared parameters: the mean over all S (Appendix B), here against fp64
        shared = np.ones(n, bool)
        for b in range(len(arch.blocks)):
            if bin(int(mask[b])).count("1") != S:
                shared[r[b, 0]:r[b, 1]] = False
        ref = np.mean(np.stack(subs).astype(np.float64), axis=0)
        np.testing.assert_allclose(g[shared], ref[shared], rtol=2e-6, atol=1e-6)   # values are O(1): a few fp32 ulps
        # identical copies: averaging is the identity, exactly, for power-of-two counts
        same = [subs[0].copy() for _ in range(S)]
        g2 = np.zeros(n, np.float32)
        oracle.aggregate(a, mask, same, None, g2, None)
        np.testing.assert_array_equal(g2, subs[0])


def test_aggregate_partial_sharing_counts():
    # the starred block of Fig. 1: a block held by 2 of 3 sub-ResNets is the mean of exactly those two
    arch = synth.tiny_arch()
    a = arch.to_int32()
    n, _ = oracle.param_count(a)
    mask = np.array([7, 0b011, 7, 0b100, 7, 0b101], dtype=np.uint32)
    rs = np.random.default_rng(3)
    subs = [rs.standard_normal(n) for _ in range(3)]
    g = np.full(n, np.nan)
    oracle.aggregate(a, mask, subs, None, g, None)
    r = oracle.block_ranges(a)
    np.testing.assert_allclose(g[r[1, 0]:r[1, 1]], 0.5 * (subs[0] + subs[1])[r[1, 0]:r[1, 1]], rtol=1e-12, atol=1e-14)
    np.testing.assert_array_equal(g[r[3, 0]:r[3, 1]], subs[2][r[3, 0]:r[3, 1]])
    np.testing.assert_allclose(g[r[5, 0]:r[5, 1]], 0.5 * (subs[0] + subs[2])[r[5, 0]:r[5, 1]], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(g[:r[0, 0]], ((subs[0] + subs[1] + subs[2]) / 3)[:r[0, 0]], rtol=1e-12, atol=1e-14)


def test_one_step_identity_ties_partition_step_and_aggregate():
    # Appendix B: with one local step of plain SGD, W_{t+1} - W_t = -eta * sum_v g_v / sum_v M_v per block.
    arch = synth.tiny_arch()
    a = arch.to_int32()
    S, lr = 2, 0.1
    p0, buf0, _, _ = case(arch, 4, 31)
    mask = oracle.partition(a, 1234, S)
    subs, grads = [], []
    for s in range(S):
        _, _, x, y = case(arch, 6, 100 + s)
        p, v = p0.copy(), np.zeros_like(p0)
        out = oracle.step(a, oracle.present_of(mask, s), p, v, None, x, y, lr=lr, mu=0.0)
        subs.append(p)
        grads.append(out["grads"])
    g = p0.copy()
    oracle.aggregate(a, mask, subs, None, g, None)
    n, _ = oracle.param_count(a)
    count = np.full(n, S, dtype=np.float64)
    r = oracle.block_ranges(a)
    for b in range(len(arch.blocks)):
        count[r[b, 0]:r[b, 1]] = bin(int(mask[b])).count("1")
    np.testing.assert_allclose(g - p0, -lr * (grads[0] + grads[1]) / count, rtol=1e-9, atol=1e-13)


def test_S1_is_plain_sgd_and_no_partitionable_block_is_local_sgd():
    arch = synth.tiny_arch()
    a = arch.to_int32()
    mask = oracle.partition(a, 7, 1)
    assert (mask == 1).all()
    none = synth.tiny_arch("none").to_int32()
    mask = oracle.partition(none, 7, 4)
    assert (mask == 15).all()


# ------------------------------------------------------------------ partition
def test_partition_invariants():
    for cfg in (1, 2, 3, 4):
        c = synth.config(cfg)
        a = c.arch.to_int32()
        P = c.arch.num_partitionable
        for t in range(5):
            mask = oracle.partition(a, c.round_seed(t), c.S)
            allm = (1 << c.S) - 1
            sizes = np.zeros(c.S, int)
            for b, blk in enumerate(c.arch.blocks):
                if blk.partitionable:
                    assert bin(int(mask[b])).count("1") == 1          # exactly one sub-ResNet
                    sizes[int(mask[b]).bit_length() - 1] += 1
                else:
                    assert mask[b] == allm                             # shared blocks are in all of them
            assert set(sizes) <= {P // c.S, -(-P // c.S)} and sizes.sum() == P


def test_resnet101_has_22_partitionable_blocks_and_resnet50_has_five():
    # Sec. 2.6 counts five partitionable blocks for ResNet-50 (its third section has six blocks)
    assert synth.resnet101_arch().num_partitionable == 22
    assert synth.resnet101_arch(depths=(3, 4, 6, 3)).num_partitionable == 5


def test_partition_is_uniform_over_arrangements_brute_force():
    # P = 3 partitionable blocks, S = 3: each of the 3! assignments should appear ~1/6 of the time
    arch = synth.tiny_arch()
    a = arch.to_int32()
    counts = {}
    N = 30000
    seeds = synth.splitmix64_words(424242, N)
    for sd in seeds:
        m = oracle.partition(a, int(sd), 3)
        key = (int(m[1]), int(m[3]), int(m[5]))
        counts[key] = counts.get(key, 0) + 1
    assert len(counts) == 6
    for v in counts.values():
        assert abs(v - N / 6) < 5 * np.sqrt(N * (1 / 6) * (5 / 6))


def test_partition_follows_the_stated_shuffle_and_deal():
    # brute force in Python, from the published splitmix64 words: Fisher-Yates from the end, j = word mod (i+1),
    # then position j of the permutation goes to sub-ResNet j mod S.
    c = synth.config(2)
    a = c.arch.to_int32()
    ids = [i for i, b in enumerate(c.arch.blocks) if b.partitionable]
    seed = 0xDEADBEEF
    words = synth.splitmix64_words(seed, len(ids) - 1)
    k = 0
    for i in range(len(ids) - 1, 0, -1):
        j = int(words[k]) % (i + 1)
        k += 1
        ids[i], ids[j] = ids[j], ids[i]
    expect = np.full(len(c.arch.blocks), 15, dtype=np.uint32)
    for j, b in enumerate(ids):
        expect[b] = 1 << (j % 4)
    np.testing.assert_array_equal(oracle.partition(a, seed, 4), expect)


def test_partition_rejects_more_subnets_than_blocks_and_min_depth_tops_up():
    a = synth.tiny_arch().to_int32()
    with pytest.raises(ValueError):
        oracle.partition(a, 1, 4)
    # Fig. 1: five partitionable blocks, S = 2, equal depth 3: one block ends up in both sub-ResNets
    arch = synth.Arch(8, 8, 3, 10, 3, 1, 8, 0, 0, synth._stack(synth.BASIC, 8, (6,), (8,), (8,), "stage_first_shared"))
    m = oracle.partition(arch.to_int32(), 5, 2, min_depth=3)
    held = [sum(1 for b in range(1, 6) if m[b] >> s & 1) for s in range(2)]
    assert held == [3, 3]
    assert sum(1 for b in range(1, 6) if m[b] == 3) == 1 and all(m[b] != 0 for b in range(1, 6))


def test_table1_parameter_accounting_within_two_percent():
    # Table 1: bytes per round = S sub-ResNets x 2 directions x 4 B x params(sub-ResNet).  Local SGD moves
    # the full net.  ResNet101 with only the 22 non-strided third-section blocks partitioned.
    rows = {}
    with open(os.path.join(GOLDEN, "table1_comm_gb.txt")) as f:
        for line in f:
            if line.startswith("#"):
                continue
            k, *v = line.split()
            rows[k] = [float(z) for z in v]
    for classes, key in ((1000, "local_sgd"), (100, "resist")):
        arch = synth.resnet101_arch(classes=classes)
        a = arch.to_int32()
        n, _ = oracle.param_count(a)
        r = oracle.block_ranges(a)
        part = sum(int(r[b, 1] - r[b, 0]) for b, blk in enumerate(arch.blocks) if blk.partitionable)
        for S, paper in zip((2, 4, 8), rows[key]):
            sub = n if key == "local_sgd" else (n - part) + part / S
            gib = S * 2 * 4 * sub / 2 ** 30
            assert abs(gib - paper) / paper < 0.021, (key, S, gib, paper)


def test_deeper_descriptors_partition_counts():
    """ResNet-152 and ResNet-200 (appendix on deeper architectures) in the usual layouts: 36 blocks in the third section, of which the
    strided first stays shared (Sec. 2.2), so P = 35 for both; every sub-ResNet of S = 4 gets 8 or 9 of them."""
    for arch, nblocks in ((synth.resnet152_arch(), 50), (synth.resnet200_arch(), 66)):
        assert len(arch.blocks) == nblocks and arch.num_partitionable == 35
        a = arch.to_int32()
        mask = oracle.partition(a, 12345, 4)
        part = [b for b, blk in enumerate(arch.blocks) if blk.partitionable]
        assert all(bin(int(mask[b])).count("1") == 1 for b in part)
        assert all(int(mask[b]) == 0xF for b in range(nblocks) if b not in part)
        sizes = [sum(1 for b in part if mask[b] >> s & 1) for s in range(4)]
        assert sorted(sizes) == [8, 9, 9, 9]
