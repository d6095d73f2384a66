"""Layer tables (one segment per parameter tensor, dense packing, definition order)
for the five benchmark workloads.

Each entry is ``(name, shape, kind, fan_in)``.  ``kind`` selects the value recipe
used by :mod:`gen.values` ("weight", "scale" for normalisation gains, "shift" for
normalisation shifts and biases, "embed" for tokens/position tables).  Only the
shapes of the published architectures are used; no weights, no data.
"""
from __future__ import annotations

from math import prod

import numpy as np


def _conv(name, cin, cout, k):
    return (name, (cout, cin, k, k), "weight", cin * k * k)


def _norm(name, c):
    return [(name + ".gain", (c,), "scale", 0), (name + ".shift", (c,), "shift", 0)]


def toy10():
    """Ten layers of the sizes the small benchmark configuration lists."""
    sizes = [4096, 64, 65536, 256, 262144, 512, 262144, 512, 131072, 10]
    return [(f"layer{i}", (s,), "weight", 0) for i, s in enumerate(sizes)]


def resnet20_cifar():
    """3x3 stem, three stages of three two-conv residual blocks at 16/32/64 channels,
    parameter-free shortcuts, a normalisation pair after every conv, 64x10 classifier."""
    t = [_conv("stem.conv", 3, 16, 3)] + _norm("stem.norm", 16)
    cin = 16
    for s, c in enumerate((16, 32, 64)):
        for b in range(3):
            t.append(_conv(f"s{s}.b{b}.conv1", cin, c, 3)); t += _norm(f"s{s}.b{b}.norm1", c)
            t.append(_conv(f"s{s}.b{b}.conv2", c, c, 3)); t += _norm(f"s{s}.b{b}.norm2", c)
            cin = c
    t.append(("fc.weight", (10, 64), "weight", 64))
    t.append(("fc.bias", (10,), "shift", 0))
    return t


def resnet18_imagenet():
    """7x7 stem, four stages (64/128/256/512) of two two-conv blocks, 1x1 projection
    shortcut in the first block of stages 2-4, 512x1000 classifier."""
    t = [_conv("stem.conv", 3, 64, 7)] + _norm("stem.norm", 64)
    cin = 64
    for s, c in enumerate((64, 128, 256, 512)):
        for b in range(2):
            t.append(_conv(f"s{s}.b{b}.conv1", cin, c, 3)); t += _norm(f"s{s}.b{b}.norm1", c)
            t.append(_conv(f"s{s}.b{b}.conv2", c, c, 3)); t += _norm(f"s{s}.b{b}.norm2", c)
            if b == 0 and cin != c:
                t.append(_conv(f"s{s}.b{b}.proj", cin, c, 1)); t += _norm(f"s{s}.b{b}.projnorm", c)
            cin = c
    t.append(("fc.weight", (1000, 512), "weight", 512))
    t.append(("fc.bias", (1000,), "shift", 0))
    return t


def vgg16():
    """Thirteen 3x3 convs with bias, then 25088x4096, 4096x4096, 4096x1000 with bias."""
    t = []
    cin = 3
    for i, c in enumerate((64, 64, 128, 128, 256, 256, 256, 512, 512, 512, 512, 512, 512)):
        t.append(_conv(f"conv{i}.weight", cin, c, 3))
        t.append((f"conv{i}.bias", (c,), "shift", 0))
        cin = c
    for i, (fi, fo) in enumerate(((25088, 4096), (4096, 4096), (4096, 1000))):
        t.append((f"fc{i}.weight", (fo, fi), "weight", fi))
        t.append((f"fc{i}.bias", (fo,), "shift", 0))
    return t


def vit_b16():
    """Class token, 197x768 position table, 16x16x3 patch projection, 12 blocks of
    {norm; qkv 768x2304; out 768x768; norm; mlp 768x3072; 3072x768}, final norm, 768x1000 head."""
    d, h = 768, 3072
    t = [("cls", (d,), "embed", 0), ("pos", (197, d), "embed", 0),
         ("patch.weight", (d, 3 * 16 * 16), "weight", 3 * 16 * 16), ("patch.bias", (d,), "shift", 0)]
    for b in range(12):
        t += _norm(f"blk{b}.norm1", d)
        t += [(f"blk{b}.qkv.weight", (3 * d, d), "weight", d), (f"blk{b}.qkv.bias", (3 * d,), "shift", 0)]
        t += [(f"blk{b}.out.weight", (d, d), "weight", d), (f"blk{b}.out.bias", (d,), "shift", 0)]
        t += _norm(f"blk{b}.norm2", d)
        t += [(f"blk{b}.mlp1.weight", (h, d), "weight", d), (f"blk{b}.mlp1.bias", (h,), "shift", 0)]
        t += [(f"blk{b}.mlp2.weight", (d, h), "weight", h), (f"blk{b}.mlp2.bias", (d,), "shift", 0)]
    t += _norm("final.norm", d)
    t += [("head.weight", (1000, d), "weight", d), ("head.bias", (1000,), "shift", 0)]
    return t


TABLES = {
    "toy10": toy10,
    "resnet20_cifar": resnet20_cifar,
    "resnet18_imagenet": resnet18_imagenet,
    "vgg16": vgg16,
    "vit_b16": vit_b16,
}


def layer_sizes(table):
    return [int(prod(shape)) for _, shape, _, _ in table]


def layer_offsets(table):
    """int64 array of K+1 offsets into the flat vector (offsets[0]=0, offsets[K]=n)."""
    off = np.zeros(len(table) + 1, dtype=np.int64)
    np.cumsum(layer_sizes(table), out=off[1:])
    return off
