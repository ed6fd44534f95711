"""Layer lists of the synthetic workloads (descriptions only, no arithmetic of the step).

A network is a list of `Layer` records in execution order.  `src` is the index
of the layer whose output a layer consumes and `add_from` (for "add") the index
of the second operand; index -1 denotes the network input.  A stage is a
contiguous index range [first, last]; references to `first - 1` are then the
stage's own input tensor.

Workloads follow the models the paper trains (MobileNetV2 and ResNet50 among
them, Section 5.1) at the shapes of its CIFAR-10 / Mini-ImageNet inputs; all
tensors are synthetic.
"""
from collections import namedtuple

Layer = namedtuple("Layer", "op c_in c_out k stride pad src add_from")

# integer codes shared with the C header's enum (values fixed by that header)
OPS = {"conv": 0, "dwconv": 1, "bn": 2, "relu6": 3, "relu": 4, "add": 5, "gap": 6, "linear": 7, "silu": 8, "se": 9}


class _Builder:
    def __init__(self):
        self.layers = []

    def _push(self, op, c_in, c_out, k=0, stride=1, pad=0, src=None, add_from=-1):
        if src is None:
            src = len(self.layers) - 1
        self.layers.append(Layer(op, c_in, c_out, k, stride, pad, src, add_from))
        return len(self.layers) - 1

    @property
    def last(self):
        return len(self.layers) - 1

    def conv(self, c_in, c_out, k, stride=1, pad=None, src=None):
        return self._push("conv", c_in, c_out, k, stride, (k - 1) // 2 if pad is None else pad, src)

    def dwconv(self, c, stride=1, src=None, k=3):
        return self._push("dwconv", c, c, k, stride, (k - 1) // 2, src)

    def silu(self, c):
        return self._push("silu", c, c)

    def se(self, c, squeeze):
        """Squeeze-excite over c channels with `squeeze` hidden units (kept in the record's k field)."""
        return self._push("se", c, c, squeeze)

    def bn(self, c):
        return self._push("bn", c, c)

    def relu6(self, c):
        return self._push("relu6", c, c)

    def relu(self, c):
        return self._push("relu", c, c)

    def add(self, c, src, add_from):
        return self._push("add", c, c, src=src, add_from=add_from)

    def gap(self, c):
        return self._push("gap", c, c)

    def linear(self, c_in, c_out):
        return self._push("linear", c_in, c_out)


def inverted_residual(b, c_in, c_out, stride, t, use_bn=True, act="relu6"):
    """Append one MobileNetV2 inverted-residual block to builder `b`; returns its last index."""
    x = b.last                      # block input (may be -1: network input)
    hid = c_in * t
    def _post(c, with_act):
        if use_bn:
            b.bn(c)
        if with_act and act:
            getattr(b, act)(c)
    if t != 1:
        b.conv(c_in, hid, 1)
        _post(hid, True)
    b.dwconv(hid, stride)
    _post(hid, True)
    b.conv(hid, c_out, 1)
    _post(c_out, False)
    if stride == 1 and c_in == c_out:
        b.add(c_out, src=b.last, add_from=x)
    return b.last


def mbconv(b, c_in, c_out, stride, t, k, se_ratio=0.25):
    """Append one EfficientNet MBConv block: 1x1 expand + BN + SiLU, k x k depthwise + BN + SiLU, squeeze-excite with
    max(1, c_in * se_ratio) hidden units, 1x1 project + BN, residual add when the shapes allow."""
    x = b.last
    hid = c_in * t
    if t != 1:
        b.conv(c_in, hid, 1); b.bn(hid); b.silu(hid)
    b.dwconv(hid, stride, k=k); b.bn(hid); b.silu(hid)
    b.se(hid, max(1, int(c_in * se_ratio)))
    b.conv(hid, c_out, 1); b.bn(c_out)
    if stride == 1 and c_in == c_out:
        b.add(c_out, src=b.last, add_from=x)
    return b.last


def mbconv_net(c_in, blocks):
    """A stage of MBConv blocks [(c_out, stride, expand, kernel)]."""
    b = _Builder()
    for c_out, stride, t, k in blocks:
        mbconv(b, c_in, c_out, stride, t, k)
        c_in = c_out
    return b.layers


def efficientnet_b1_stage_net():
    """EfficientNet-B1-style stage (the paper's third vision workload, Section 5.1): the 5x5 and the first 3x3 MBConv6 groups,
    24 -> 40 (stride 2, then two more) -> 80 (stride 2, then one more), for a 56x56x24 input."""
    return mbconv_net(24, [(40, 2, 6, 5), (40, 1, 6, 5), (40, 1, 6, 5), (80, 2, 6, 3), (80, 1, 6, 3)])


def block_net(c=16, t=6):
    """Config 1: a single inverted-residual block c -> t*c -> c, stride 1, with residual."""
    b = _Builder()
    inverted_residual(b, c, c, 1, t)
    return b.layers


def bnfree_net(c=4, t=2, act="relu6"):
    """A BatchNorm-free inverted-residual block (for the gradient-accumulation invariant)."""
    b = _Builder()
    inverted_residual(b, c, c, 1, t, use_bn=False, act=act)
    return b.layers


def stage_net_mbv2_4blocks():
    """Config 2: 24->24 (x2, s1), 24->32 (s2), 32->32 (s1), expand ratio 6, input 56x56x24."""
    b = _Builder()
    for c_in, c_out, s in [(24, 24, 1), (24, 24, 1), (24, 32, 2), (32, 32, 1)]:
        inverted_residual(b, c_in, c_out, s, 6)
    return b.layers


_MBV2_TABLE = [(1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2),
               (6, 96, 3, 1), (6, 160, 3, 2), (6, 320, 1, 1)]


def _mobilenetv2(classes=1000, width_table=_MBV2_TABLE, stem_c=32, head_c=1280):
    b = _Builder()
    unit_last = []
    b.conv(3, stem_c, 3, 2)
    b.bn(stem_c)
    b.relu6(stem_c)
    unit_last.append(b.last)
    c_in = stem_c
    for t, c, n, s in width_table:
        for i in range(n):
            inverted_residual(b, c_in, c, s if i == 0 else 1, t)
            unit_last.append(b.last)
            c_in = c
    b.conv(c_in, head_c, 1)
    b.bn(head_c)
    b.relu6(head_c)
    b.gap(head_c)
    b.linear(head_c, classes)
    unit_last.append(b.last)
    return b.layers, unit_last


def mobilenetv2_net(classes=1000):
    """Config 3: MobileNetV2 width 1.0: stem, 17 inverted-residual blocks, 1x1 to 1280, GAP, linear."""
    return _mobilenetv2(classes)[0]


def mobilenetv2_units(classes=1000):
    """Last layer index of each of the 19 block-level units (stem, 17 blocks, head)."""
    return _mobilenetv2(classes)[1]


def bottleneck_net(c_in, groups):
    """ResNet bottleneck groups [(mid, c_out, n_blocks, first_stride)]: 1x1 -> 3x3 (carries the
    stride) -> 1x1, BN after each conv, ReLU after the first two and after the residual add;
    the first block of a group has a 1x1 conv + BN shortcut."""
    b = _Builder()
    for mid, c_out, n, s0 in groups:
        for i in range(n):
            s = s0 if i == 0 else 1
            x = b.last
            b.conv(c_in, mid, 1); b.bn(mid); b.relu(mid)
            b.conv(mid, mid, 3, s); b.bn(mid); b.relu(mid)
            b.conv(mid, c_out, 1); main = b.bn(c_out)
            if i == 0:
                b.conv(c_in, c_out, 1, s, pad=0, src=x); sc = b.bn(c_out)
                b.add(c_out, src=sc, add_from=main)
            else:
                b.add(c_out, src=main, add_from=x)
            b.relu(c_out)
            c_in = c_out
    return b.layers


def resnet50_c2c3_net():
    """Config 4: ResNet-50 conv2_x (3 bottlenecks, 64->256) and conv3_x (4, ->512, stride 2 on the 3x3)."""
    return bottleneck_net(64, [(64, 256, 3, 1), (128, 512, 4, 2)])


def small_mobilenet(classes=10):
    """A shrunken MobileNetV2-shaped network (stem, 4 blocks, head) for tests."""
    return _mobilenetv2(classes, [(1, 8, 1, 1), (2, 8, 2, 2), (2, 16, 1, 1)], stem_c=8, head_c=32)


def single_unit_net(kind, c_in, c_out, k=1, stride=1, bn=False, act=None, se=0):
    """One conv (or depthwise conv) layer, optionally followed by BatchNorm and an activation: the
    smallest stage that exercises one contraction / stencil kernel path in both directions."""
    b = _Builder()
    if kind == "dwconv":
        b.dwconv(c_in, stride, k=k if k > 1 else 3)
    else:
        b.conv(c_in, c_out, k, stride, pad=(k - 1) // 2)
    if bn:
        b.bn(c_out)
    if act:
        getattr(b, act)(c_out)
    if se:
        b.se(c_out, se)
    return b.layers


def head_net(c, classes, bn_conv=0):
    """Classifier head: [1x1 conv to bn_conv channels + BatchNorm,] global average pool, linear."""
    b = _Builder()
    if bn_conv:
        b.conv(c, bn_conv, 1)
        b.bn(bn_conv)
        c = bn_conv
    b.gap(c)
    b.linear(c, classes)
    return b.layers


def out_shape(net, first, last, in_h, in_w):
    """(h, w, c) of every layer's output in [first, last], keyed by layer index."""
    shp = {first - 1: (in_h, in_w, net[first].c_in)}
    for i in range(first, last + 1):
        L = net[i]
        h, w, c = shp[L.src]
        if L.op in ("conv", "dwconv"):
            assert c == L.c_in, (i, c, L)
            shp[i] = ((h + 2 * L.pad - L.k) // L.stride + 1, (w + 2 * L.pad - L.k) // L.stride + 1, L.c_out)
        elif L.op == "gap":
            shp[i] = (1, 1, c)
        elif L.op == "linear":
            shp[i] = (1, 1, L.c_out)
        else:
            shp[i] = (h, w, c)
    return shp


def forward_macs(net, first, last, in_h, in_w):
    """Multiply-accumulates per sample of each layer in [first, last]."""
    shp = out_shape(net, first, last, in_h, in_w)
    macs = {}
    for i in range(first, last + 1):
        L = net[i]
        h, w, c = shp[i]
        if L.op == "conv":
            macs[i] = h * w * L.c_out * L.c_in * L.k * L.k
        elif L.op == "dwconv":
            macs[i] = h * w * L.c_out * L.k * L.k
        elif L.op == "linear":
            macs[i] = L.c_in * L.c_out
        else:
            macs[i] = 0
    return macs


def partition_units(net, unit_last, n_stages, in_h, in_w):
    """Cut the unit sequence into `n_stages` contiguous stages that minimise the largest
    stage's forward MACs (the FLOPs-proportional split of Section 3.4's re-planning).
    Returns a list of (first_layer, last_layer)."""
    macs = forward_macs(net, 0, len(net) - 1, in_h, in_w)
    unit_first = [0] + [u + 1 for u in unit_last[:-1]]
    cost = [sum(macs[i] for i in range(f, l + 1)) for f, l in zip(unit_first, unit_last)]
    n = len(cost)
    pre = [0]
    for c in cost:
        pre.append(pre[-1] + c)
    INF = float("inf")
    best = [[INF] * (n + 1) for _ in range(n_stages + 1)]
    arg = [[0] * (n + 1) for _ in range(n_stages + 1)]
    best[0][0] = 0
    for p in range(1, n_stages + 1):
        for j in range(p, n + 1):
            for i in range(p - 1, j):
                v = max(best[p - 1][i], pre[j] - pre[i])
                if v < best[p][j]:
                    best[p][j], arg[p][j] = v, i
    cuts, j = [], n
    for p in range(n_stages, 0, -1):
        i = arg[p][j]
        cuts.append((unit_first[i], unit_last[j - 1]))
        j = i
    return cuts[::-1]
