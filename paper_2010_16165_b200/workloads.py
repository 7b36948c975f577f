"""Seeded synthetic workloads: network descriptors, parameters and inputs.

This module only *describes* networks (a flat, topologically ordered node list)
and draws random parameters and inputs for them.  It contains none of the
method's arithmetic (no convolution, folding, scoring, fusion or pruning), so
that the CPU oracle and the CUDA library can both be fed from it without
sharing any computation.

Networks follow Table II of the paper (ResNet-20/32 on 32x32 inputs,
ResNet-18/34 on 224x224 inputs) extended to the deeper CIFAR-shaped and the
bottleneck ImageNet-shaped variants that the workload list asks for.

Node fields (one dict per node, mirrored by ``fp_node`` in the C header):
    op        one of the OP_* codes below
    in0, in1  producer node ids, -1 = network input (in1 only for ADD)
    K, C      output / input channels (CONV, FC); channels (BN, pools)
    R, S, stride, pad   window geometry (CONV, MAXPOOL; SHORTCUT_A uses stride)
    pad_lo    SHORTCUT_A: zero channels placed before the copied ones
    w_off     element offset of the KCRS (CONV) or KC (FC) fp32 weights
    b_off     element offset of the fp32 bias (FC), -1 = none
    bn_off    element offset of [gamma|beta|mean|var] (4*K fp32) in ``bn``
    block_id  index of the residual building block the node belongs to (-1 = none)
    aggressive  1 = fuse this block the paper's way (Sec. IV-B), 0 = keep the add
"""
from __future__ import annotations

import numpy as np

OP_CONV, OP_BN, OP_RELU, OP_ADD, OP_SHORTCUT_A, OP_MAXPOOL, OP_GAVGPOOL, OP_FC, OP_CONCAT = range(9)
OP_NAMES = ["conv", "bn", "relu", "add", "shortcut_a", "maxpool", "gavgpool", "fc", "concat"]

BASE_SEED = 20201016


class Net:
    """A descriptor under construction: node list + sizes of the parameter arrays."""

    def __init__(self, in_C, in_H, in_W, name=""):
        self.name = name
        self.in_C, self.in_H, self.in_W = in_C, in_H, in_W
        self.nodes = []
        self.n_weights = 0
        self.n_bn = 0
        self.bn_eps = 1e-5

    def _add(self, **kw):
        node = dict(op=0, in0=-1, in1=-1, K=0, C=0, R=0, S=0, stride=1, pad=0, pad_lo=0,
                    w_off=-1, b_off=-1, bn_off=-1, block_id=-1, aggressive=0)
        node.update(kw)
        self.nodes.append(node)
        return len(self.nodes) - 1

    def conv(self, src, K, C, R, stride, pad, block=-1, aggressive=0):
        off = self.n_weights
        self.n_weights += K * C * R * R
        return self._add(op=OP_CONV, in0=src, K=K, C=C, R=R, S=R, stride=stride, pad=pad,
                         w_off=off, block_id=block, aggressive=aggressive)

    def bn(self, src, K, block=-1, aggressive=0):
        off = self.n_bn
        self.n_bn += 4 * K
        return self._add(op=OP_BN, in0=src, K=K, C=K, bn_off=off, block_id=block, aggressive=aggressive)

    def relu(self, src, block=-1, aggressive=0):
        return self._add(op=OP_RELU, in0=src, block_id=block, aggressive=aggressive)

    def add(self, main, shortcut, block=-1, aggressive=0):
        return self._add(op=OP_ADD, in0=main, in1=shortcut, block_id=block, aggressive=aggressive)

    def shortcut_a(self, src, C, K, stride, pad_lo=0, block=-1, aggressive=0):
        return self._add(op=OP_SHORTCUT_A, in0=src, C=C, K=K, stride=stride, pad_lo=pad_lo,
                         block_id=block, aggressive=aggressive)

    def concat(self, a, b, Ka, Cb):
        """Channel concatenation [a ; b]: a = the (BN / ReLU of a) convolution's output with Ka channels, b = that
        convolution's input with Cb channels (the concatenation structure of Sec. IV-B.1)."""
        return self._add(op=OP_CONCAT, in0=a, in1=b, K=Ka + Cb, C=Cb)

    def maxpool(self, src, C, R=3, stride=2, pad=1):
        return self._add(op=OP_MAXPOOL, in0=src, K=C, C=C, R=R, S=R, stride=stride, pad=pad)

    def gavgpool(self, src, C):
        return self._add(op=OP_GAVGPOOL, in0=src, K=C, C=C)

    def fc(self, src, K, C):
        off = self.n_weights
        self.n_weights += K * C
        boff = self.n_weights
        self.n_weights += K
        return self._add(op=OP_FC, in0=src, K=K, C=C, w_off=off, b_off=boff)

    # ---- derived views -------------------------------------------------------------
    def conv_ids(self):
        return [i for i, n in enumerate(self.nodes) if n["op"] == OP_CONV]

    def n_convs(self):
        return len(self.conv_ids())

    def n_classes(self):
        return [n for n in self.nodes if n["op"] == OP_FC][-1]["K"]


def _basic_block(net, x, C, K, stride, shortcut, block, aggressive, pad_lo=0):
    """conv3x3-bn-relu-conv3x3-bn-(+shortcut)-relu.  shortcut in {'id','A','proj'}."""
    kw = dict(block=block, aggressive=aggressive)
    h = net.conv(x, K, C, 3, stride, 1, **kw)
    h = net.bn(h, K, **kw)
    h = net.relu(h, **kw)
    h = net.conv(h, K, K, 3, 1, 1, **kw)
    h = net.bn(h, K, **kw)
    if shortcut == "id":
        sc = x
    elif shortcut == "A":
        sc = net.shortcut_a(x, C, K, stride, pad_lo=pad_lo, **kw)
    else:
        sc = net.conv(x, K, C, 1, stride, 0, **kw)
        sc = net.bn(sc, K, **kw)
    y = net.add(h, sc, **kw)
    return net.relu(y, **kw)


def _bottleneck(net, x, C, width, stride, project, block, aggressive=0):
    """1x1-3x3(stride)-1x1 bottleneck, expansion 4; stride sits on the 3x3 conv."""
    kw = dict(block=block, aggressive=aggressive)
    K = 4 * width
    h = net.relu(net.bn(net.conv(x, width, C, 1, 1, 0, **kw), width, **kw), **kw)
    h = net.relu(net.bn(net.conv(h, width, width, 3, stride, 1, **kw), width, **kw), **kw)
    h = net.bn(net.conv(h, K, width, 1, 1, 0, **kw), K, **kw)
    if project:
        sc = net.bn(net.conv(x, K, C, 1, stride, 0, **kw), K, **kw)
    else:
        sc = x
    return net.relu(net.add(h, sc, **kw), **kw)


def _aggr(aggressive, block):
    """aggressive may be a bool, or a set/list of block ids (fusion option x/n of the paper)."""
    if isinstance(aggressive, (set, list, tuple, frozenset)):
        return 1 if block in aggressive else 0
    return 1 if aggressive else 0


def resnet_cifar(n_per_stage, widths=(16, 32, 64), in_hw=32, n_classes=10, aggressive=False,
                 pad_lo_centered=False, name=None):
    """CIFAR-shaped ResNet-(6n+2) with option-A shortcuts (Table II, ResNet-20/32 columns)."""
    net = Net(3, in_hw, in_hw, name or f"resnet{6 * n_per_stage + 2}")
    x = net.relu(net.bn(net.conv(-1, widths[0], 3, 3, 1, 1), widths[0]))
    C = widths[0]
    block = 0
    for si, K in enumerate(widths):
        for bi in range(n_per_stage):
            first = (bi == 0 and si > 0)
            pad_lo = (K - C) // 2 if (first and pad_lo_centered) else 0
            x = _basic_block(net, x, C, K, 2 if first else 1, "A" if first else "id", block,
                             _aggr(aggressive, block), pad_lo)
            C = K
            block += 1
    x = net.gavgpool(x, C)
    net.fc(x, n_classes, C)
    net.n_blocks = block
    return net


def resnet_imagenet_basic(layers=(2, 2, 2, 2), widths=(64, 128, 256, 512), in_hw=224, n_classes=1000,
                          aggressive=False, name=None, stem_k=7):
    """ImageNet-shaped ResNet-18/34 (Table II): 7x7/2 stem, 3x3/2 maxpool, projection shortcuts."""
    net = Net(3, in_hw, in_hw, name or f"resnet{2 * sum(layers) + 2}")
    x = net.relu(net.bn(net.conv(-1, widths[0], 3, stem_k, 2, stem_k // 2), widths[0]))
    x = net.maxpool(x, widths[0])
    C = widths[0]
    block = 0
    for si, K in enumerate(widths):
        for bi in range(layers[si]):
            first = (bi == 0 and si > 0)
            x = _basic_block(net, x, C, K, 2 if first else 1, "proj" if first else "id", block,
                             _aggr(aggressive, block))
            C = K
            block += 1
    x = net.gavgpool(x, C)
    net.fc(x, n_classes, C)
    net.n_blocks = block
    return net


def resnet_imagenet_bottleneck(layers=(3, 4, 6, 3), widths=(64, 128, 256, 512), in_hw=224,
                               n_classes=1000, name=None, stem_k=7, stem_width=64, aggressive=False):
    """ImageNet-shaped ResNet-50: bottleneck blocks, projection on the first block of every stage."""
    net = Net(3, in_hw, in_hw, name or f"resnet{3 * sum(layers) + 2}")
    x = net.relu(net.bn(net.conv(-1, stem_width, 3, stem_k, 2, stem_k // 2), stem_width))
    x = net.maxpool(x, stem_width)
    C = stem_width
    block = 0
    for si, wd in enumerate(widths):
        for bi in range(layers[si]):
            first = bi == 0
            x = _bottleneck(net, x, C, wd, 2 if (first and si > 0) else 1, first, block, _aggr(aggressive, block))
            C = 4 * wd
            block += 1
    x = net.gavgpool(x, C)
    net.fc(x, n_classes, C)
    net.n_blocks = block
    return net


# ---------------------------------------------------------------------------------------
# parameters and inputs
# ---------------------------------------------------------------------------------------

def bf16_round(a):
    """Round an fp32 array to the nearest bf16-representable value (ties to even), as fp32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def make_params(net, rng):
    """Draw weights and BN statistics in descriptor order (see module docstring of the recipe).

    Per CONV node (in node order) W ~ N(0, 2/(C*R*S)) followed immediately by the BN
    that normalises it: gamma ~ U(0.5,1.5), beta ~ N(0,0.1), mean ~ N(0,0.1),
    var ~ U(0.5,1.5).  Then the FC weight ~ N(0, 2/C), FC bias 0.  Values are drawn in
    fp64 and cast to fp32.
    """
    weights = np.zeros(net.n_weights, dtype=np.float32)
    bn = np.zeros(net.n_bn, dtype=np.float32)
    consumers = {}
    for i, n in enumerate(net.nodes):
        if n["op"] == OP_BN:
            consumers[n["in0"]] = i
    for i, n in enumerate(net.nodes):
        if n["op"] == OP_CONV:
            cnt = n["K"] * n["C"] * n["R"] * n["S"]
            std = np.sqrt(2.0 / (n["C"] * n["R"] * n["S"]))
            weights[n["w_off"]:n["w_off"] + cnt] = (rng.standard_normal(cnt) * std).astype(np.float32)
            if i in consumers:
                b = net.nodes[consumers[i]]
                K, o = b["K"], b["bn_off"]
                bn[o:o + K] = rng.uniform(0.5, 1.5, K)
                bn[o + K:o + 2 * K] = rng.standard_normal(K) * 0.1
                bn[o + 2 * K:o + 3 * K] = rng.standard_normal(K) * 0.1
                bn[o + 3 * K:o + 4 * K] = rng.uniform(0.5, 1.5, K)
    for n in net.nodes:
        if n["op"] == OP_FC:
            cnt = n["K"] * n["C"]
            weights[n["w_off"]:n["w_off"] + cnt] = (rng.standard_normal(cnt) * np.sqrt(2.0 / n["C"])).astype(np.float32)
    return weights, bn


def make_input(net, batch, rng, bf16=False):
    x = rng.standard_normal((batch, net.in_C, net.in_H, net.in_W)).astype(np.float32)
    return bf16_round(x) if bf16 else x


class Workload:
    """A network + parameters + input + pruning request, all seeded."""

    def __init__(self, name, net, batch, seed, in_bf16, ratios=None, ratio_spec="", compute="bf16"):
        self.name, self.net, self.batch, self.seed = name, net, batch, seed
        rng = np.random.default_rng(seed)
        self.weights, self.bn = make_params(net, rng)
        self.in_bf16 = in_bf16
        self._rng = rng
        self._x = None
        nc = net.n_convs()
        if callable(ratios):
            # ratios drawn after the input in the stream order: materialise the input first
            _ = self.x
            ratios = ratios(net, self._rng)
        self.ratios = np.zeros(nc) if ratios is None else np.asarray(ratios, dtype=np.float64)
        self.ratio_spec = ratio_spec
        self.compute = compute

    @property
    def x(self):
        if self._x is None:
            self._x = make_input(self.net, self.batch, self._rng, self.in_bf16)
        return self._x


def uniform_ratios(p):
    return lambda net, rng: np.full(net.n_convs(), float(p))


def drawn_ratios(lo, hi):
    return lambda net, rng: rng.uniform(lo, hi, net.n_convs())


def inner_bottleneck_ratios(p):
    """Prune only the first two convs (1x1 reduce, 3x3) of every bottleneck block."""
    def f(net, rng):
        r = np.zeros(net.n_convs())
        per_block = {}
        for ci, nid in enumerate(net.conv_ids()):
            b = net.nodes[nid]["block_id"]
            if b >= 0:
                per_block.setdefault(b, []).append(ci)
        for b, cis in per_block.items():
            for ci in cis[:2]:
                r[ci] = p
        return r
    return f


def workload(config, batch=None, prune=None, aggressive=False):
    """The five benchmark-shaped workloads (``config`` 1..5) and the two other networks of the paper's Table II
    (6: ResNet-32, 7: ResNet-34); batch/prune override the defaults."""
    seed = BASE_SEED + config
    if config == 1:
        net = resnet_cifar(3, aggressive=aggressive)
        p = 0.3 if prune is None else prune
        return Workload(f"resnet20_b{batch or 8}_p{p}", net, batch or 8, seed, False, uniform_ratios(p), f"uniform {p}")
    if config == 2:
        net = resnet_cifar(9, aggressive=aggressive)
        p = 0.3 if prune is None else prune
        return Workload(f"resnet56_b{batch or 256}_p{p}", net, batch or 256, seed, True, uniform_ratios(p), f"uniform {p}")
    if config == 3:
        net = resnet_cifar(18, aggressive=aggressive)
        return Workload(f"resnet110_b{batch or 1024}_pU(0.2,0.6)", net, batch or 1024, seed, True,
                        drawn_ratios(0.2, 0.6), "U(0.2,0.6) per conv")
    if config == 4:
        net = resnet_imagenet_basic(aggressive=aggressive)
        p = 0.3 if prune is None else prune
        return Workload(f"resnet18_b{batch or 64}_p{p}", net, batch or 64, seed, True, uniform_ratios(p), f"uniform {p}")
    if config == 5:
        net = resnet_imagenet_bottleneck()
        p = 0.4 if prune is None else prune
        return Workload(f"resnet50_b{batch or 128}_inner{p}", net, batch or 128, seed, True,
                        inner_bottleneck_ratios(p), f"inner bottleneck {p}")
    if config == 6:      # the paper's second CIFAR model (Table II), shaped like config 2
        net = resnet_cifar(5, aggressive=aggressive)
        p = 0.3 if prune is None else prune
        return Workload(f"resnet32_b{batch or 256}_p{p}", net, batch or 256, seed, True, uniform_ratios(p), f"uniform {p}")
    if config == 7:      # the paper's second ImageNet model (Table II), shaped like config 4
        net = resnet_imagenet_basic((3, 4, 6, 3), aggressive=aggressive)
        p = 0.3 if prune is None else prune
        return Workload(f"resnet34_b{batch or 64}_p{p}", net, batch or 64, seed, True, uniform_ratios(p), f"uniform {p}")
    raise ValueError("config must be 1..7")


def tiny_cifar(n_per_stage=1, widths=(8, 16, 24), in_hw=8, batch=2, seed=7, aggressive=False, p=0.0,
               pad_lo_centered=False):
    """Small CIFAR-style net for unit tests (odd widths allowed)."""
    net = resnet_cifar(n_per_stage, widths, in_hw, n_classes=5, aggressive=aggressive,
                       pad_lo_centered=pad_lo_centered, name="tiny_cifar")
    return Workload("tiny_cifar", net, batch, seed, False, uniform_ratios(p), f"uniform {p}")


def tiny_imagenet_basic(layers=(1, 1, 1), widths=(8, 12, 20), in_hw=32, batch=2, seed=11, aggressive=False,
                        p=0.0, stem_k=7):
    net = resnet_imagenet_basic(layers, widths, in_hw, n_classes=7, aggressive=aggressive,
                                name="tiny_imagenet_basic", stem_k=stem_k)
    return Workload("tiny_imagenet_basic", net, batch, seed, False, uniform_ratios(p), f"uniform {p}")


def concat_net(growth=(6, 10, 5), stem=8, in_hw=12, n_classes=4, name="concat_net"):
    """A small network of concatenation structures (DenseNet-like growth): x <- concat(relu(bn(conv3x3(x))), x)."""
    net = Net(3, in_hw, in_hw, name)
    x = net.relu(net.bn(net.conv(-1, stem, 3, 3, 1, 1), stem))
    C = stem
    for g in growth:
        h = net.relu(net.bn(net.conv(x, g, C, 3, 1, 1), g))
        x = net.concat(h, x, g, C)
        C += g
    x = net.gavgpool(x, C)
    net.fc(x, n_classes, C)
    net.n_blocks = 0
    return net


def tiny_concat(batch=3, seed=19, p=0.0, **kw):
    return Workload("tiny_concat", concat_net(**kw), batch, seed, False, uniform_ratios(p), f"uniform {p}")


def tiny_bottleneck(layers=(1, 2), widths=(4, 8), in_hw=32, batch=2, seed=13, p=0.0, aggressive=False):
    net = resnet_imagenet_bottleneck(layers, widths, in_hw, n_classes=6, name="tiny_bottleneck", stem_width=8,
                                     aggressive=aggressive)
    return Workload("tiny_bottleneck", net, batch, seed, False, inner_bottleneck_ratios(p), f"inner {p}")
