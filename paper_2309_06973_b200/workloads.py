"""Seeded synthetic CNN workloads: shapes, channel-group wiring and weight values.

This module only *describes* networks and draws their parameters.  It holds none
of the pruning method's arithmetic (no thresholding, masking, detection,
propagation or compaction), so both the CPU oracle's tests and the CUDA path can
take their inputs from it without sharing anything else.

A workload is a list of weight tensors in OIHW layout, the BatchNorm vectors
that follow them, the channel groups that tie tensor axes together (the set of
channels an output axis shares with the input axes that read it, including
every tensor coupled through a residual add), a list of prune counts ``k`` and
a small op list that a test can interpret to run the network forward.

The five named workloads stand in for the networks the paper evaluates
(Section IV, Table II: VGG-16 on CIFAR-10 with 14.72 M parameters, ResNet-50
with 25.56 M) by shape, size and value distribution only; no trained weights or
dataset items are involved.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np

F32 = 0
BF16 = 1

SCOPE_GLOBAL = 0
SCOPE_PER_TENSOR = 1

GROUP_FROZEN = 1


@dataclass
class TensorSpec:
    name: str
    O: int
    I: int            # columns of the [O][I][KH][KW] array; FC: C_in * in_spatial
    KH: int
    KW: int
    out_group: int
    in_group: int
    in_spatial: int = 1
    prunable: bool = True
    has_bias: bool = False
    stride: int = 1
    pad: int = 0

    @property
    def numel(self) -> int:
        return self.O * self.I * self.KH * self.KW


@dataclass
class BNSpec:
    name: str
    C: int
    tensor: int       # index of the conv whose output it normalises
    group: int
    eps: float = 1e-5


@dataclass
class GroupSpec:
    C: int
    flags: int = 0


@dataclass
class Workload:
    name: str
    seed: int
    scope: int
    tensors: List[TensorSpec]
    bns: List[BNSpec]
    groups: List[GroupSpec]
    ops: List[tuple]
    input_hw: int
    # values (filled by the generator)
    weights: List[np.ndarray] = field(default_factory=list)       # fp32, shape (O, I, KH, KW)
    biases: List[Optional[np.ndarray]] = field(default_factory=list)
    bn_params: List[Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]] = field(default_factory=list)
    ks: Optional[np.ndarray] = None   # uint64, shape (n_k, n_segments)
    planted: List[np.ndarray] = field(default_factory=list)        # zeroed filter indices per tensor

    @property
    def n_prunable(self) -> int:
        return sum(t.numel for t in self.tensors if t.prunable)

    @property
    def n_params(self) -> int:
        n = sum(t.numel for t in self.tensors)
        n += sum(t.O for t in self.tensors if t.has_bias)
        n += sum(2 * b.C for b in self.bns)          # affine gamma, beta
        return n

    def segments(self) -> List[List[int]]:
        """Tensor indices per ranking segment, in descriptor order."""
        pr = [i for i, t in enumerate(self.tensors) if t.prunable]
        if self.scope == SCOPE_GLOBAL:
            return [pr]
        return [[i] for i in pr]

    def weights_as(self, dtype: int) -> List[np.ndarray]:
        """The weight arrays as stored words: float32, or uint16 holding bf16."""
        if dtype == F32:
            return [w.copy() for w in self.weights]
        return [f32_to_bf16_bits(w) for w in self.weights]


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even conversion of float32 to bf16 storage words."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    nan = (u & 0x7FFFFFFF) > 0x7F800000
    r = (u + (0x7FFF + ((u >> 16) & 1))) >> 16
    r = np.where(nan, (u >> 16) | 0x40, r)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32)


# --------------------------------------------------------------------------
# integer prune counts
# --------------------------------------------------------------------------

def k_fraction(n: int, p: int, q: int) -> int:
    """floor(n * p / q) in integers."""
    return (n * p) // q


def k_iterative(n: int, rounds: List[int]) -> List[int]:
    """Cumulative prune counts when each round removes ceil(remaining / 5)."""
    out, rem, r = [], n, 0
    want = set(rounds)
    while r < max(rounds):
        rem = rem - (rem + 4) // 5
        r += 1
        if r in want:
            out.append(n - rem)
    return out


# --------------------------------------------------------------------------
# architecture builders
# --------------------------------------------------------------------------

class _Builder:
    def __init__(self):
        self.tensors: List[TensorSpec] = []
        self.bns: List[BNSpec] = []
        self.groups: List[GroupSpec] = []
        self.ops: List[tuple] = []

    def group(self, C, frozen=False) -> int:
        self.groups.append(GroupSpec(C, GROUP_FROZEN if frozen else 0))
        return len(self.groups) - 1

    def conv_bn(self, name, src, dst, gin, gout, k, stride, pad, relu=True):
        """conv (no bias) + BN (+ ReLU) from activation `src` to activation `dst`."""
        cin, cout = self.groups[gin].C, self.groups[gout].C
        t = len(self.tensors)
        self.tensors.append(TensorSpec(name, cout, cin, k, k, gout, gin, stride=stride, pad=pad))
        b = len(self.bns)
        self.bns.append(BNSpec(name + ".bn", cout, t, gout))
        self.ops.append(("conv", t, src, dst, stride, pad))
        self.ops.append(("bn", b, dst, dst))
        if relu:
            self.ops.append(("relu", dst, dst))
        return t

    def fc(self, name, src, dst, gin, gout, in_spatial=1):
        cin, cout = self.groups[gin].C, self.groups[gout].C
        t = len(self.tensors)
        self.tensors.append(TensorSpec(name, cout, cin * in_spatial, 1, 1, gout, gin,
                                       in_spatial=in_spatial, has_bias=True))
        self.ops.append(("fc", t, src, dst))
        return t


def _plain_chain(name, widths, n_classes, seed, scope, input_hw):
    b = _Builder()
    g = b.group(3, frozen=True)
    act = "x"
    for li, w in enumerate(widths):
        gn = b.group(w)
        b.conv_bn(f"conv{li}", act, f"a{li}", g, gn, 3, 1, 1)
        g, act = gn, f"a{li}"
    b.ops.append(("gap", act, "pool"))
    gc = b.group(n_classes, frozen=True)
    b.fc("fc", "pool", "out", g, gc)
    return Workload(name, seed, scope, b.tensors, b.bns, b.groups, b.ops, input_hw)


def _vgg16(seed, scope):
    widths = [64, 64, "M", 128, 128, "M", 256, 256, 256, "M", 512, 512, 512, "M", 512, 512, 512, "M"]
    b = _Builder()
    g = b.group(3, frozen=True)
    act, li = "x", 0
    for w in widths:
        if w == "M":
            b.ops.append(("maxpool", act, act + "p", 2, 2, 0))
            act = act + "p"
            continue
        gn = b.group(w)
        b.conv_bn(f"conv{li}", act, f"a{li}", g, gn, 3, 1, 1)
        g, act, li = gn, f"a{li}", li + 1
    b.ops.append(("gap", act, "pool"))
    gc = b.group(10, frozen=True)
    b.fc("fc", "pool", "out", g, gc)
    return Workload("vgg16", seed, scope, b.tensors, b.bns, b.groups, b.ops, 32)


def _resnet_basic(seed, scope, n_blocks=9, widths=(16, 32, 64), n_classes=10):
    """CIFAR ResNet with two-conv blocks; a 1x1 stride-2 projection opens each new stage."""
    b = _Builder()
    gi = b.group(3, frozen=True)
    stream = b.group(widths[0])
    b.conv_bn("stem", "x", "s0", gi, stream, 3, 1, 1)
    act, uid = "s0", 0
    for si, w in enumerate(widths):
        for bi in range(n_blocks):
            first = si > 0 and bi == 0
            new_stream = b.group(w) if first else stream
            stride = 2 if first else 1
            inner = b.group(w)
            nm = f"l{si}.{bi}"
            b.conv_bn(nm + ".conv1", act, nm + ".h", stream, inner, 3, stride, 1)
            b.conv_bn(nm + ".conv2", nm + ".h", nm + ".r", inner, new_stream, 3, 1, 1, relu=False)
            skip = act
            if first:
                b.conv_bn(nm + ".proj", act, nm + ".sk", stream, new_stream, 1, stride, 0, relu=False)
                skip = nm + ".sk"
            b.ops.append(("add", nm + ".r", skip, nm + ".o"))
            b.ops.append(("relu", nm + ".o", nm + ".o"))
            act, stream, uid = nm + ".o", new_stream, uid + 1
    b.ops.append(("gap", act, "pool"))
    gc = b.group(n_classes, frozen=True)
    b.fc("fc", "pool", "out", stream, gc)
    return Workload("resnet56", seed, scope, b.tensors, b.bns, b.groups, b.ops, 32)


def _resnet_bottleneck(name, seed, scope, blocks, n_classes=1000):
    """ImageNet ResNet with 1x1-3x3-1x1 blocks, expansion 4, projection in each stage's first block."""
    b = _Builder()
    gi = b.group(3, frozen=True)
    stream = b.group(64)
    b.conv_bn("stem", "x", "s0", gi, stream, 7, 2, 3)
    b.ops.append(("maxpool", "s0", "s0p", 3, 2, 1))
    act = "s0p"
    for si, nb in enumerate(blocks):
        width = 64 << si
        for bi in range(nb):
            first = bi == 0
            stride = 2 if (first and si > 0) else 1
            new_stream = b.group(width * 4) if first else stream
            g1, g2 = b.group(width), b.group(width)
            nm = f"l{si}.{bi}"
            b.conv_bn(nm + ".conv1", act, nm + ".h1", stream, g1, 1, 1, 0)
            b.conv_bn(nm + ".conv2", nm + ".h1", nm + ".h2", g1, g2, 3, stride, 1)
            b.conv_bn(nm + ".conv3", nm + ".h2", nm + ".r", g2, new_stream, 1, 1, 0, relu=False)
            skip = act
            if first:
                b.conv_bn(nm + ".proj", act, nm + ".sk", stream, new_stream, 1, stride, 0, relu=False)
                skip = nm + ".sk"
            b.ops.append(("add", nm + ".r", skip, nm + ".o"))
            b.ops.append(("relu", nm + ".o", nm + ".o"))
            act, stream = nm + ".o", new_stream
    b.ops.append(("gap", act, "pool"))
    gc = b.group(n_classes, frozen=True)
    b.fc("fc", "pool", "out", stream, gc)
    return Workload(name, seed, scope, b.tensors, b.bns, b.groups, b.ops, 64)


# --------------------------------------------------------------------------
# value generators
# --------------------------------------------------------------------------

def _draw(wl: Workload, he_scaled: bool, lognormal_sigma: float, planted_frac: float,
          planted_mode: str = "per_conv"):
    """Fill a workload with seeded values.

    Order of draws (fixed, so a seed names one model): for every tensor in
    descriptor order its Gaussian values, then its per-filter log-normal factors;
    then the planted zero filters; then per BN gamma, beta, mean, var.
    """
    rng = np.random.default_rng(wl.seed)
    wl.weights, wl.biases, wl.bn_params, wl.planted = [], [], [], []
    for t in wl.tensors:
        fan_in = t.I * t.KH * t.KW
        w = rng.standard_normal((t.O, t.I, t.KH, t.KW), dtype=np.float32)
        if he_scaled:
            w *= np.float32(np.sqrt(2.0 / fan_in))
        if lognormal_sigma > 0:
            z = rng.standard_normal(t.O)
            w *= np.exp(lognormal_sigma * z).astype(np.float32)[:, None, None, None]
        wl.weights.append(np.ascontiguousarray(w))
        wl.biases.append(np.zeros(t.O, np.float32) if t.has_bias else None)
    # planted all-zero filters
    if planted_mode == "per_conv":
        for ti, t in enumerate(wl.tensors):
            is_conv = not t.has_bias
            n0 = int(planted_frac * t.O) if is_conv else 0
            idx = np.sort(rng.permutation(t.O)[:n0]).astype(np.int64)
            wl.weights[ti][idx] = 0.0
            wl.planted.append(idx)
    elif planted_mode == "per_stream":
        # the same channel indices are zeroed in every producer of a residual stream
        producers = {}
        for ti, t in enumerate(wl.tensors):
            producers.setdefault(t.out_group, []).append(ti)
        wl.planted = [np.zeros(0, np.int64) for _ in wl.tensors]
        for g, tis in sorted(producers.items()):
            if len(tis) < 2 or (wl.groups[g].flags & GROUP_FROZEN):
                continue
            C = wl.groups[g].C
            idx = np.sort(rng.permutation(C)[: int(planted_frac * C)]).astype(np.int64)
            for ti in tis:
                wl.weights[ti][idx] = 0.0
                wl.planted[ti] = idx
    else:
        wl.planted = [np.zeros(0, np.int64) for _ in wl.tensors]
    for b in wl.bns:
        gamma = rng.uniform(0.5, 1.5, b.C).astype(np.float32)
        beta = (0.1 * rng.standard_normal(b.C)).astype(np.float32)
        mean = (0.1 * rng.standard_normal(b.C)).astype(np.float32)
        var = rng.uniform(0.5, 1.5, b.C).astype(np.float32)
        wl.bn_params.append((gamma, beta, mean, var))
    return wl


def _set_ks(wl: Workload, per_segment_ks):
    """per_segment_ks(n) -> list of k for a segment of n weights."""
    segs = wl.segments()
    cols = [per_segment_ks(sum(wl.tensors[i].numel for i in s)) for s in segs]
    wl.ks = np.array(cols, dtype=np.uint64).T.copy()      # (n_k, n_segments)
    return wl


def toy(seed=0):
    """Four 3x3 convs 3-16-32-32-64 with BN, global pooling, FC to 10 classes; 90 % global sparsity."""
    wl = _plain_chain("toy", [16, 32, 32, 64], 10, seed, SCOPE_GLOBAL, 32)
    _draw(wl, he_scaled=False, lognormal_sigma=1.0, planted_frac=0.25)
    return _set_ks(wl, lambda n: [k_fraction(n, 9, 10)])


def vgg16(seed=1):
    """VGG-16 with CIFAR shapes (13 convs + one linear layer); 95 % sparsity per tensor."""
    wl = _vgg16(seed, SCOPE_PER_TENSOR)
    _draw(wl, he_scaled=True, lognormal_sigma=0.0, planted_frac=0.30)
    return _set_ks(wl, lambda n: [k_fraction(n, 19, 20)])


def resnet56(seed=2):
    """ResNet-56 with CIFAR shapes; ten variants, each round pruning a fifth of what remains."""
    wl = _resnet_basic(seed, SCOPE_GLOBAL)
    _draw(wl, he_scaled=True, lognormal_sigma=0.0, planted_frac=0.20, planted_mode="per_stream")
    return _set_ks(wl, lambda n: k_iterative(n, list(range(1, 11))))


def resnet50(seed=3):
    """ResNet-50 with ImageNet shapes; global sparsity 80 %, 90 %, 98 %."""
    wl = _resnet_bottleneck("resnet50", seed, SCOPE_GLOBAL, [3, 4, 6, 3])
    _draw(wl, he_scaled=True, lognormal_sigma=0.5, planted_frac=0.10)
    return _set_ks(wl, lambda n: [k_fraction(n, 4, 5), k_fraction(n, 9, 10), k_fraction(n, 49, 50)])


def resnet152(seed=4):
    """ResNet-152 with ImageNet shapes; eight variants at sparsity 1 - 0.8^r, r = 3..10."""
    wl = _resnet_bottleneck("resnet152", seed, SCOPE_GLOBAL, [3, 8, 36, 3])
    _draw(wl, he_scaled=True, lognormal_sigma=1.0, planted_frac=0.0, planted_mode="none")
    return _set_ks(wl, lambda n: k_iterative(n, list(range(3, 11))))


def chain(widths, seed=0, kernel=3, n_classes=4, planted_frac=0.25):
    """A small plain chain of convs for tests (the setting of the paper's Algorithm 1)."""
    wl = _plain_chain("chain", list(widths), n_classes, seed, SCOPE_GLOBAL, 8)
    if kernel != 3:
        for t in wl.tensors:
            if not t.has_bias:
                t.KH = t.KW = kernel
                t.pad = kernel // 2
        wl.ops = [(o[0], o[1], o[2], o[3], o[4], kernel // 2) if o[0] == "conv" else o for o in wl.ops]
    _draw(wl, he_scaled=True, lognormal_sigma=0.5, planted_frac=planted_frac)
    return _set_ks(wl, lambda n: [k_fraction(n, 1, 2)])


def small_resnet(seed=0, bottleneck=True):
    """A two-stage residual net small enough for exhaustive checks."""
    if bottleneck:
        wl = _resnet_bottleneck("small_bottleneck", seed, SCOPE_GLOBAL, [2, 2], n_classes=8)
        # shrink the widths by 8 so the whole model is a few thousand weights
        wl = _shrink(wl, 8)
    else:
        wl = _resnet_basic(seed, SCOPE_GLOBAL, n_blocks=2, widths=(8, 16), n_classes=6)
        wl.name = "small_basic"
    _draw(wl, he_scaled=True, lognormal_sigma=0.5, planted_frac=0.25, planted_mode="per_stream")
    return _set_ks(wl, lambda n: k_iterative(n, [2, 5, 8]))


def _shrink(wl: Workload, f: int) -> Workload:
    for g in wl.groups:
        if not (g.flags & GROUP_FROZEN):
            g.C = max(2, g.C // f)
    for t in wl.tensors:
        t.O = wl.groups[t.out_group].C
        t.I = wl.groups[t.in_group].C * t.in_spatial
    for b in wl.bns:
        b.C = wl.groups[b.group].C
    return wl


def freeze_streams(wl: Workload) -> Workload:
    """Mark every channel group that more than one layer writes (a residual stream: the stem or a projection plus
    the last conv of every block on it) as frozen, so that only plain layer-to-layer connections are pruned -
    the paper's own setting, which leaves skip connections and downsampling layers alone (Section IV-B-2)."""
    writers = [0] * len(wl.groups)
    for t in wl.tensors:
        writers[t.out_group] += 1
    for g, n in zip(wl.groups, writers):
        if n > 1:
            g.flags |= GROUP_FROZEN
    return wl


BY_NAME = {"toy": toy, "vgg16": vgg16, "resnet56": resnet56, "resnet50": resnet50, "resnet152": resnet152}
