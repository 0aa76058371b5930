"""Seeded synthetic workloads: architecture descriptors, parameter layout and input generators.

This module serves both the CPU oracle's tests and the CUDA library's tests and benchmark.
It holds no arithmetic of the method itself (no partition, no layer math, no update rule,
no averaging): only *what the inputs are*.  The images stand in for CIFAR-10/100 (32x32x3)
and ILSVRC2012 (224x224x3), which the paper trains on (Sec. 5) and which are not needed for
a throughput and parity study: i.i.d. N(0,1) pixels, uniform labels, He-normal weights.

Random numbers come from the splitmix64 generator (Steele, Lea, Flood 2014), written here in
vectorised numpy: word i of a stream seeded with `seed` is mix(seed + (i+1)*GAMMA).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Tuple

import numpy as np

GAMMA = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)

BASIC, BOTTLENECK = 0, 1
ARCH_HEADER_INTS = 10
BLOCK_INTS = 8


def splitmix64_words(seed: int, n: int, skip: int = 0) -> np.ndarray:
    """Words skip .. skip+n-1 of the splitmix64 stream seeded with `seed` (uint64 array)."""
    with np.errstate(over="ignore"):
        idx = np.arange(skip + 1, skip + n + 1, dtype=np.uint64)
        z = np.uint64(seed & 0xFFFFFFFFFFFFFFFF) + idx * GAMMA
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


def uniform01(seed: int, n: int, skip: int = 0) -> np.ndarray:
    """Doubles in [0,1): the top 53 bits of each word times 2^-53."""
    return (splitmix64_words(seed, n, skip) >> np.uint64(11)).astype(np.float64) * (2.0 ** -53)


def standard_normal(seed: int, n: int) -> np.ndarray:
    """n standard normals by Box-Muller in double; one (u1,u2) pair per two variates,
    cosine branch first, then sine."""
    pairs = (n + 1) // 2
    u = uniform01(seed, 2 * pairs)
    u1, u2 = u[0::2], u[1::2]
    r = np.sqrt(-2.0 * np.log1p(-u1))
    out = np.empty(2 * pairs, dtype=np.float64)
    out[0::2] = r * np.cos(2.0 * np.pi * u2)
    out[1::2] = r * np.sin(2.0 * np.pi * u2)
    return out[:n]


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """float32 array rounded to the nearest bf16 (ties to even), returned as float32."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (b >> np.uint32(16)) & np.uint32(1)
    with np.errstate(over="ignore"):
        r = (b + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 array -> uint16 array of bf16 bit patterns (round to nearest even)."""
    return (round_to_bf16(x).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


@dataclass
class Block:
    kind: int            # BASIC or BOTTLENECK
    stage: int           # 0-based section index
    cin: int
    cmid: int            # bottleneck width (basic: = cout)
    cout: int
    stride: int
    has_projection: int  # 1x1 strided conv on the skip path
    partitionable: int   # 1: dealt to exactly one sub-ResNet per round; 0: held by all


@dataclass
class Arch:
    in_h: int
    in_w: int
    in_c: int
    classes: int
    stem_k: int
    stem_stride: int
    stem_cout: int
    stem_bn_relu: int
    stem_maxpool: int
    blocks: List[Block] = field(default_factory=list)

    def to_int32(self) -> np.ndarray:
        """Flat descriptor: 10 header ints then 8 ints per block (the order of the fields above)."""
        out = [self.in_h, self.in_w, self.in_c, self.classes, self.stem_k, self.stem_stride,
               self.stem_cout, self.stem_bn_relu, self.stem_maxpool, len(self.blocks)]
        for b in self.blocks:
            out += [b.kind, b.stage, b.cin, b.cmid, b.cout, b.stride, b.has_projection, b.partitionable]
        return np.asarray(out, dtype=np.int32)

    @property
    def num_partitionable(self) -> int:
        return sum(b.partitionable for b in self.blocks)


def _stack(kind: int, stem_cout: int, depths, widths, mids, policy: str) -> List[Block]:
    """policy 'stage_first_shared': every block but the first of each stage is partitionable.
    policy 'paper_section3': only the non-first blocks of the third stage are (Sec. 2.2)."""
    blocks: List[Block] = []
    cin = stem_cout
    for st, (d, w, m) in enumerate(zip(depths, widths, mids)):
        for i in range(d):
            stride = 2 if (i == 0 and st > 0) else 1
            proj = 1 if (i == 0 and (stride != 1 or cin != w)) else 0
            if policy == "stage_first_shared":
                part = 1 if i > 0 else 0
            elif policy == "paper_section3":
                part = 1 if (st == 2 and i > 0) else 0
            elif policy == "none":
                part = 0
            else:
                raise ValueError(policy)
            blocks.append(Block(kind, st, cin, m, w, stride, proj, part))
            cin = w
    return blocks


def tiny_arch(policy: str = "stage_first_shared") -> Arch:
    w = (8, 16, 32)
    return Arch(8, 8, 3, 10, 3, 1, 8, 0, 0, _stack(BASIC, 8, (2, 2, 2), w, w, policy))


def resnet110_arch(policy: str = "stage_first_shared") -> Arch:
    w = (16, 32, 64)
    return Arch(32, 32, 3, 10, 3, 1, 16, 0, 0, _stack(BASIC, 16, (18, 18, 18), w, w, policy))


def wide_cifar_arch(policy: str = "paper_section3", depths=(3, 4, 23, 3)) -> Arch:
    mids = (64, 128, 256, 512)
    w = tuple(4 * m for m in mids)
    return Arch(32, 32, 3, 100, 3, 1, 64, 0, 0, _stack(BOTTLENECK, 64, depths, w, mids, policy))


def resnet101_arch(policy: str = "paper_section3", depths=(3, 4, 23, 3), classes: int = 1000,
                   in_hw: int = 224) -> Arch:
    w = (256, 512, 1024, 2048)
    mids = tuple(x // 4 for x in w)
    return Arch(in_hw, in_hw, 3, classes, 7, 2, 64, 1, 1, _stack(BOTTLENECK, 64, depths, w, mids, policy))


def resnet152_arch(policy: str = "paper_section3", classes: int = 1000, in_hw: int = 224) -> Arch:
    """The deeper variants of the appendix on deeper architectures: the extra blocks go to the third section ([3,8,36,3] and, below,
    [3,24,36,3] in the usual layouts), so the share of partitioned blocks grows (P = 35 for both: 36 blocks in section 3, minus the strided one)."""
    return resnet101_arch(policy, (3, 8, 36, 3), classes, in_hw)


def resnet200_arch(policy: str = "paper_section3", classes: int = 1000, in_hw: int = 224) -> Arch:
    return resnet101_arch(policy, (3, 24, 36, 3), classes, in_hw)


@dataclass
class Config:
    cfg: int
    name: str
    arch: Arch
    S: int
    batch: int
    local_steps: int
    rounds: int
    dtype: str           # "f32" or "bf16"
    lr: float = 0.1
    momentum: float = 0.9

    @property
    def data_seed(self) -> int:
        return 0xD47A0000 + self.cfg

    @property
    def init_seed(self) -> int:
        return 0x1417 + self.cfg

    def round_seed(self, t: int) -> int:
        return int(splitmix64_words((0x5EED0000 + self.cfg) ^ t, 1)[0])


def config(cfg: int) -> Config:
    if cfg == 1:
        return Config(1, "tiny-resnet-f32", tiny_arch(), 2, 8, 2, 1, "f32")
    if cfg == 2:
        return Config(2, "cifar-resnet110-bf16", resnet110_arch(), 4, 128, 50, 4, "bf16")
    if cfg == 3:
        return Config(3, "wide-cifar-bottleneck-bf16", wide_cifar_arch(), 8, 128, 50, 2, "bf16")
    if cfg == 4:
        return Config(4, "imagenet-resnet101-bf16", resnet101_arch(), 4, 64, 20, 1, "bf16")
    if cfg == 5:
        return Config(5, "resnet101-reassembly-stress", resnet101_arch(), 4, 32, 1, 1, "bf16")
    raise ValueError(cfg)


# ---------------------------------------------------------------------------------------------
# Flat parameter layout (an interface shared by every implementation, restated in each):
#   stem conv [Cout][k][k][Cin]; (stem BN gamma, beta if present);
#   per block, in network order:
#     basic:      bn1 g,b | conv1 [Cout][3][3][Cin] | bn2 g,b | conv2 [Cout][3][3][Cout] | (proj [Cout][1][1][Cin])
#     bottleneck: bn1 g,b | conv1 [Cmid][1][1][Cin] | bn2 g,b | conv2 [Cmid][3][3][Cmid] | bn3 g,b |
#                 conv3 [Cout][1][1][Cmid] | (proj [Cout][1][1][Cin])
#   final BN g,b | head W [classes][C] | head bias [classes].
# Buffers: for every BN in the same order, running mean [C] then running var [C].
# ---------------------------------------------------------------------------------------------
@dataclass
class Tensor:
    name: str
    kind: str            # "conv", "gamma", "beta", "head_w", "head_b"
    shape: Tuple[int, ...]
    offset: int
    block: int           # block index, -1 for stem / final BN / head

    @property
    def size(self) -> int:
        return int(np.prod(self.shape))


def param_layout(arch: Arch) -> Tuple[List[Tensor], int, int]:
    """Returns (tensors, n_params, n_buffers)."""
    ts: List[Tensor] = []
    off = 0
    nbuf = 0

    def add(name, kind, shape, blk):
        nonlocal off
        t = Tensor(name, kind, tuple(shape), off, blk)
        ts.append(t)
        off += t.size

    def bn(name, c, blk):
        nonlocal nbuf
        add(name + ".gamma", "gamma", (c,), blk)
        add(name + ".beta", "beta", (c,), blk)
        nbuf += 2 * c

    add("stem.conv", "conv", (arch.stem_cout, arch.stem_k, arch.stem_k, arch.in_c), -1)
    if arch.stem_bn_relu:
        bn("stem.bn", arch.stem_cout, -1)
    c = arch.stem_cout
    for i, b in enumerate(arch.blocks):
        p = f"block{i}"
        if b.kind == BASIC:
            bn(p + ".bn1", b.cin, i)
            add(p + ".conv1", "conv", (b.cout, 3, 3, b.cin), i)
            bn(p + ".bn2", b.cout, i)
            add(p + ".conv2", "conv", (b.cout, 3, 3, b.cout), i)
        else:
            bn(p + ".bn1", b.cin, i)
            add(p + ".conv1", "conv", (b.cmid, 1, 1, b.cin), i)
            bn(p + ".bn2", b.cmid, i)
            add(p + ".conv2", "conv", (b.cmid, 3, 3, b.cmid), i)
            bn(p + ".bn3", b.cmid, i)
            add(p + ".conv3", "conv", (b.cout, 1, 1, b.cmid), i)
        if b.has_projection:
            add(p + ".proj", "conv", (b.cout, 1, 1, b.cin), i)
        c = b.cout
    bn("final.bn", c, -1)
    add("head.w", "head_w", (arch.classes, c), -1)
    add("head.b", "head_b", (arch.classes,), -1)
    return ts, off, nbuf


def init_params(arch: Arch, seed: int) -> Tuple[np.ndarray, np.ndarray]:
    """He-normal N(0, 2/fan_in) for conv and head weights (fan_in = kh*kw*Cin), gamma 1, beta 0,
    bias 0; one normal stream consumed in flat parameter order.  Buffers: mean 0, var 1."""
    ts, n, nbuf = param_layout(arch)
    n_rand = sum(t.size for t in ts if t.kind in ("conv", "head_w"))
    z = standard_normal(seed, n_rand)
    p = np.zeros(n, dtype=np.float32)
    k = 0
    for t in ts:
        if t.kind == "conv":
            fan_in = t.shape[1] * t.shape[2] * t.shape[3]
        elif t.kind == "head_w":
            fan_in = t.shape[1]
        elif t.kind == "gamma":
            p[t.offset:t.offset + t.size] = 1.0
            continue
        else:
            continue
        p[t.offset:t.offset + t.size] = (z[k:k + t.size] * np.sqrt(2.0 / fan_in)).astype(np.float32)
        k += t.size
    buf = np.zeros(nbuf, dtype=np.float32)
    # running variance starts at one: buffers are [mean C | var C] per BN
    o = 0
    for t in ts:
        if t.kind == "gamma":
            c = t.size
            buf[o + c:o + 2 * c] = 1.0
            o += 2 * c
    return p, buf


def perturbed_params(arch: Arch, seed: int, scale: float = 0.1) -> Tuple[np.ndarray, np.ndarray]:
    """init_params with gamma, beta and head bias moved off their trivial values, so that tests
    exercise every term (a test at gamma=1, beta=0 cannot see a dropped beta)."""
    p, buf = init_params(arch, seed)
    ts, n, _ = param_layout(arch)
    z = standard_normal(seed ^ 0xABCDEF, n)
    for t in ts:
        if t.kind in ("gamma", "beta", "head_b"):
            p[t.offset:t.offset + t.size] += (scale * z[t.offset:t.offset + t.size]).astype(np.float32)
    return p, buf


def batch(cfg: Config, rnd: int, step: int, subnet: int, B: int | None = None,
          as_bf16: bool | None = None) -> Tuple[np.ndarray, np.ndarray]:
    """A fresh batch for (round, step, sub-ResNet): NHWC float32 images ~ N(0,1), int32 labels."""
    B = cfg.batch if B is None else B
    a = cfg.arch
    seed = int(splitmix64_words(cfg.data_seed, 1, skip=(rnd * 100003 + step) * 64 + subnet)[0])
    n = B * a.in_h * a.in_w * a.in_c
    x = standard_normal(seed, n).astype(np.float32).reshape(B, a.in_h, a.in_w, a.in_c)
    if as_bf16 if as_bf16 is not None else (cfg.dtype == "bf16"):
        x = round_to_bf16(x)
    y = (splitmix64_words(seed ^ 0x1ABE1, B) % np.uint64(a.classes)).astype(np.int32)
    return x, y
