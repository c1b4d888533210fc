"""Workload recipes: layer lists for the synthetic networks.

A layer is a dict with the fields of the C descriptor: op ('conv', 'dwconv', 'fc',
'maxpool', 'gavgpool'), act ('none', 'relu', 'relu6'), cin, cout, kh, kw, stride, pad,
groups, src (index of the producing layer, -1 = network input), res_src (-2 = none,
-1 = network input, else layer index added before the activation) and pool (0, or 2
for a fused 2x2/2 max-pool after the activation).  No shapes are computed here: each
consumer infers them itself.
"""
from __future__ import annotations


def _layer(op, cin, cout, k=1, stride=1, pad=None, act="none", groups=1, src=None,
           res_src=-2, pool=0):
    return dict(op=op, act=act, cin=cin, cout=cout, kh=k, kw=k, stride=stride,
                pad=(k // 2 if pad is None else pad), groups=groups, src=src,
                res_src=res_src, pool=pool)


def _finish(layers):
    for i, l in enumerate(layers):
        if l["src"] is None:
            l["src"] = i - 1
    return layers


def conv_chain(depth: int, c: int, k: int, act="relu", cin=None):
    """`depth` identical convs C->C, kernel k, pad k//2, bias + activation each."""
    return _finish([_layer("conv", (cin if (cin and i == 0) else c), c, k, act=act)
                    for i in range(depth)])


def vgg16(classes=1000):
    """13 conv3x3 + bias + ReLU in five stages, 2x2 max-pool fused after each stage,
    then FC 25088-4096-4096-classes (ReLU after the two hidden ones)."""
    L, cin = [], 3
    for width, reps in ((64, 2), (128, 2), (256, 3), (512, 3), (512, 3)):
        for r in range(reps):
            L.append(_layer("conv", cin, width, 3, act="relu",
                            pool=2 if r == reps - 1 else 0))
            cin = width
    L.append(_layer("fc", 7 * 7 * 512, 4096, act="relu"))
    L.append(_layer("fc", 4096, 4096, act="relu"))
    L.append(_layer("fc", 4096, classes))
    return _finish(L)


def vgg19(classes=1000):
    """VGG-19 (the paper's Table 2 workload): 16 conv3x3 + bias + ReLU in five stages (2, 2, 4, 4, 4), 2x2 max-pool
    fused after each stage, then the same three fully connected layers as VGG-16."""
    L, cin = [], 3
    for width, reps in ((64, 2), (128, 2), (256, 4), (512, 4), (512, 4)):
        for r in range(reps):
            L.append(_layer("conv", cin, width, 3, act="relu", pool=2 if r == reps - 1 else 0))
            cin = width
    L.append(_layer("fc", 7 * 7 * 512, 4096, act="relu"))
    L.append(_layer("fc", 4096, 4096, act="relu"))
    L.append(_layer("fc", 4096, classes))
    return _finish(L)


def resnet18(classes=1000):
    """ResNet-18 (Table 2): 7x7/2 stem + 3x3/2 max-pool, basic blocks [2,2,2,2] of two 3x3 convolutions (stride on the
    first; list order per block: first 3x3, 1x1/2 projection if any, second 3x3 + add + ReLU), global average pool, FC:
    20 convolutions."""
    L = [_layer("conv", 3, 64, 7, stride=2, pad=3, act="relu"),
         _layer("maxpool", 64, 64, 3, stride=2, pad=1)]
    cin, block_in = 64, 1
    for stage, width in enumerate((64, 128, 256, 512)):
        for b in range(2):
            s = 2 if (b == 0 and stage > 0) else 1
            L.append(_layer("conv", cin, width, 3, stride=s, act="relu", src=block_in))
            first = len(L) - 1
            skip = block_in
            if s == 2:
                L.append(_layer("conv", cin, width, 1, stride=s, pad=0, src=block_in))
                skip = len(L) - 1
            L.append(_layer("conv", width, width, 3, act="relu", src=first, res_src=skip))
            block_in, cin = len(L) - 1, width
    L.append(_layer("gavgpool", cin, cin))
    L.append(_layer("fc", cin, classes))
    return _finish(L)


def alexnet(classes=1000):
    """AlexNet in its single-tower form (the variant whose operation count matches Table 2): 11x11/4 pad 2 -> 64,
    3x3/2 max-pool, 5x5 pad 2 -> 192, 3x3/2 max-pool, three 3x3 (384, 256, 256), 3x3/2 max-pool, FC 9216-4096-4096-classes;
    bias + ReLU after every convolution and hidden FC."""
    L = [_layer("conv", 3, 64, 11, stride=4, pad=2, act="relu"), _layer("maxpool", 64, 64, 3, stride=2, pad=0),
         _layer("conv", 64, 192, 5, pad=2, act="relu"), _layer("maxpool", 192, 192, 3, stride=2, pad=0),
         _layer("conv", 192, 384, 3, act="relu"), _layer("conv", 384, 256, 3, act="relu"), _layer("conv", 256, 256, 3, act="relu"),
         _layer("maxpool", 256, 256, 3, stride=2, pad=0),
         _layer("fc", 6 * 6 * 256, 4096, act="relu"), _layer("fc", 4096, 4096, act="relu"), _layer("fc", 4096, classes)]
    return _finish(L)


def resnet50(classes=1000):
    """7x7/2 stem + 3x3/2 max-pool, bottlenecks [3,4,6,3] (stride on the 3x3; list
    order per block: reduce, 3x3, projection if any, expand + add + ReLU), global
    average pool, FC."""
    L = [_layer("conv", 3, 64, 7, stride=2, pad=3, act="relu"),
         _layer("maxpool", 64, 64, 3, stride=2, pad=1)]
    cin, block_in = 64, 1
    for stage, (reps, width) in enumerate(((3, 64), (4, 128), (6, 256), (3, 512))):
        for b in range(reps):
            s = 2 if (b == 0 and stage > 0) else 1
            L.append(_layer("conv", cin, width, 1, act="relu", src=block_in))
            L.append(_layer("conv", width, width, 3, stride=s, act="relu"))
            mid = len(L) - 1
            skip = block_in
            if b == 0:
                L.append(_layer("conv", cin, 4 * width, 1, stride=s, pad=0, src=block_in))
                skip = len(L) - 1
            L.append(_layer("conv", width, 4 * width, 1, act="relu", src=mid, res_src=skip))
            block_in, cin = len(L) - 1, 4 * width
    L.append(_layer("gavgpool", cin, cin))
    L.append(_layer("fc", cin, classes))
    return _finish(L)


def mobilenet_v2(classes=1000):
    """3x3/2 stem 32, 17 inverted-residual blocks (first one without expansion),
    1x1 -> 1280, global average pool, FC."""
    L = [_layer("conv", 3, 32, 3, stride=2, act="relu6")]
    cin = 32
    for t, c, reps, s in ((1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2),
                          (6, 96, 3, 1), (6, 160, 3, 2), (6, 320, 1, 1)):
        for b in range(reps):
            st = s if b == 0 else 1
            block_in, hid = len(L) - 1, cin * t
            if t != 1:
                L.append(_layer("conv", cin, hid, 1, act="relu6"))
            L.append(_layer("dwconv", hid, hid, 3, stride=st, act="relu6", groups=hid))
            L.append(_layer("conv", hid, c, 1,
                            res_src=block_in if (st == 1 and cin == c) else -2))
            cin = c
    L.append(_layer("conv", cin, 1280, 1, act="relu6"))
    L.append(_layer("gavgpool", 1280, 1280))
    L.append(_layer("fc", 1280, classes))
    return _finish(L)


def two_layer_group():
    """Two conv3x3 16->16 + bias + ReLU (the smallest fusion group)."""
    return conv_chain(2, 16, 3)
