"""Layer tables and seeded random weights for the CNN trunks the workloads use.

Input description only: shapes, strides, graph wiring and random numbers.  No
convolution, erosion or matching arithmetic lives here.

A layer is a plain dict with the keys of the C struct ``dc_layer_desc``:
``kind, kh, kw, sh, sw, ph, pw, cin, cout, relu, in0, in1, out_h, out_w, groups``.
``in0`` / ``in1`` index the producing layer; ``-1`` is the input frame.
Weights are float32, laid out ``[cout][kh][kw][cin / groups]``; biases float32 ``[cout]``.
"""
from __future__ import annotations

import numpy as np

# Layer kind codes: an interface shared with the C header and the oracle.
KIND_CONV, KIND_MAXPOOL, KIND_RELU, KIND_ADD, KIND_CONCAT, KIND_RESIZE_AREA, KIND_LRN, KIND_FC = range(8)


def _layer(kind, in0, out_h, out_w, cin, cout, k=1, s=1, p=0, relu=0, in1=-1, groups=1):
    return dict(kind=kind, kh=k, kw=k, sh=s, sw=s, ph=p, pw=p, cin=cin, cout=cout,
                relu=relu, in0=in0, in1=in1, out_h=out_h, out_w=out_w, groups=groups)


class NetBuilder:
    """Appends layers, tracking each layer's output shape."""

    def __init__(self, height: int, width: int, channels: int = 3):
        self.layers: list[dict] = []
        self.in_shape = (height, width, channels)

    def shape(self, idx: int):
        if idx < 0:
            return self.in_shape
        l = self.layers[idx]
        return (l["out_h"], l["out_w"], l["cout"])

    def conv(self, src: int, cout: int, k: int, s: int = 1, p: int = 0, relu: int = 1, groups: int = 1) -> int:
        h, w, c = self.shape(src)
        assert c % groups == 0 and cout % groups == 0
        oh, ow = (h + 2 * p - k) // s + 1, (w + 2 * p - k) // s + 1
        self.layers.append(_layer(KIND_CONV, src, oh, ow, c, cout, k, s, p, relu, groups=groups))
        return len(self.layers) - 1

    def maxpool(self, src: int, k: int, s: int, p: int = 0) -> int:
        h, w, c = self.shape(src)
        oh, ow = (h + 2 * p - k) // s + 1, (w + 2 * p - k) // s + 1
        self.layers.append(_layer(KIND_MAXPOOL, src, oh, ow, c, c, k, s, p))
        return len(self.layers) - 1

    def add(self, a: int, b: int, relu: int = 1) -> int:
        h, w, c = self.shape(a)
        assert self.shape(b) == (h, w, c)
        self.layers.append(_layer(KIND_ADD, a, h, w, c, c, relu=relu, in1=b))
        return len(self.layers) - 1

    def lrn(self, src: int, radius: int) -> int:
        """Within-channel local response normalisation over a (2 radius + 1)^2 window (Table 2's LRN row)."""
        h, w, c = self.shape(src)
        self.layers.append(_layer(KIND_LRN, src, h, w, c, c, 2 * radius + 1, 1, radius))
        return len(self.layers) - 1

    def concat(self, a: int, b: int) -> int:
        h, w, ca = self.shape(a)
        hb, wb, cb = self.shape(b)
        assert (h, w) == (hb, wb)
        self.layers.append(_layer(KIND_CONCAT, a, h, w, ca, ca + cb, in1=b))
        return len(self.layers) - 1

    def fc(self, src: int, cout: int, relu: int = 0) -> int:
        """Fully connected = a convolution whose kernel covers the whole input map (weights [cout][h][w][cin])."""
        h, w, c = self.shape(src)
        l = _layer(KIND_FC, src, 1, 1, c, cout, 1, 1, 0, relu)
        l["kh"], l["kw"] = h, w
        self.layers.append(l)
        return len(self.layers) - 1

    def resize_area(self, src: int, oh: int, ow: int) -> int:
        h, w, c = self.shape(src)
        self.layers.append(_layer(KIND_RESIZE_AREA, src, oh, ow, c, c))
        return len(self.layers) - 1


def single_conv(h=64, w=64):
    b = NetBuilder(h, w)
    b.conv(-1, 16, 3, 1, 1)
    return b.layers


def small_cnn(h=227, w=227):
    b = NetBuilder(h, w)
    x = b.conv(-1, 32, 3, 1, 1)
    x = b.conv(x, 32, 3, 1, 1)
    x = b.maxpool(x, 2, 2)
    x = b.conv(x, 64, 3, 1, 1)
    x = b.conv(x, 64, 3, 1, 1)
    x = b.maxpool(x, 2, 2)
    b.conv(x, 128, 3, 1, 1)
    return b.layers


def inception_lrn_net(h=64, w=64):
    """A small GoogLeNet-flavoured graph that uses every layer kind of Table 2: convolution, LRN, pooling, two
    branches joined by a channel concatenation, and a fully connected head."""
    b = NetBuilder(h, w)
    x = b.conv(-1, 32, 3, 1, 1)
    x = b.lrn(x, 1)
    x = b.maxpool(x, 2, 2)
    p1 = b.conv(x, 32, 1, 1, 0)
    p2 = b.conv(x, 16, 3, 1, 1)
    p2 = b.conv(p2, 32, 3, 1, 1)
    x = b.concat(p1, p2)
    x = b.conv(x, 64, 3, 1, 1)
    x = b.maxpool(x, 2, 2)
    x = b.lrn(x, 2)
    x = b.maxpool(x, 4, 4)
    b.fc(x, 48)
    return b.layers


def alexnet_trunk(h=227, w=227, grouped=False):
    """AlexNet-shaped trunk.  ``grouped``: the second, fourth and fifth convolutions in two channel groups,
    as in the two-GPU original; the stated workload uses the ungrouped form."""
    g = 2 if grouped else 1
    b = NetBuilder(h, w)
    x = b.conv(-1, 96, 11, 4, 0)
    x = b.maxpool(x, 3, 2)
    x = b.conv(x, 256, 5, 1, 2, groups=g)
    x = b.maxpool(x, 3, 2)
    x = b.conv(x, 384, 3, 1, 1)
    x = b.conv(x, 384, 3, 1, 1, groups=g)
    x = b.conv(x, 256, 3, 1, 1, groups=g)
    b.maxpool(x, 3, 2)
    return b.layers


def resnet50_trunk(h=224, w=224):
    b = NetBuilder(h, w)
    x = b.conv(-1, 64, 7, 2, 3)
    x = b.maxpool(x, 3, 2, 1)
    for stage, (width, blocks) in enumerate(((64, 3), (128, 4), (256, 6), (512, 3))):
        for blk in range(blocks):
            s = 2 if (blk == 0 and stage > 0) else 1
            y = b.conv(x, width, 1, 1, 0)
            y = b.conv(y, width, 3, s, 1)
            y = b.conv(y, width * 4, 1, 1, 0, relu=0)
            sc = b.conv(x, width * 4, 1, s, 0, relu=0) if blk == 0 else x
            x = b.add(y, sc, relu=1)
    return b.layers


def vgg16_trunk(h=224, w=224, src_h=None, src_w=None):
    """13 3x3 convolutions; with ``src_h/src_w`` an area-resize layer comes first."""
    if src_h is not None:
        b = NetBuilder(src_h, src_w)
        x = b.resize_area(-1, h, w)
    else:
        b = NetBuilder(h, w)
        x = -1
    for cout, n in ((64, 2), (128, 2), (256, 3), (512, 3), (512, 3)):
        for _ in range(n):
            x = b.conv(x, cout, 3, 1, 1)
        x = b.maxpool(x, 2, 2)
    return b.layers


def random_weights(layers, seed: int, *, std: float | None = None, bias_std: float = 0.05):
    """He-normal (or fixed-``std``) weights for every conv and fully-connected layer; ``None`` elsewhere.

    The last conv of a residual branch (a conv feeding an add with relu=0) is
    scaled by 0.5 so activations stay tame through deep residual stacks.
    """
    rng = np.random.Generator(np.random.PCG64([seed, 0x3E16]))
    feeds_add = set()
    for l in layers:
        if l["kind"] == KIND_ADD:
            feeds_add.add(l["in0"])
    weights, biases = [], []
    for i, l in enumerate(layers):
        if l["kind"] not in (KIND_CONV, KIND_FC):
            weights.append(None)
            biases.append(None)
            continue
        cin_g = l["cin"] // max(1, l.get("groups", 1))            # a grouped convolution sees cin / groups channels
        fan_in = l["kh"] * l["kw"] * cin_g
        sd = std if std is not None else float(np.sqrt(2.0 / fan_in))
        if i in feeds_add:
            sd *= 0.5
        w = rng.normal(0.0, sd, size=(l["cout"], l["kh"], l["kw"], cin_g)).astype(np.float32)
        bvec = (rng.normal(0.0, bias_std, size=l["cout"]) if bias_std > 0 else np.zeros(l["cout"]))
        weights.append(w)
        biases.append(bvec.astype(np.float32))
    return weights, biases
