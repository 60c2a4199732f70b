"""Layer-shape lists for the five benchmark configurations.

Each layer is a plain dict whose keys mirror the C descriptor
(`nnv_layer_desc_t`): op, C, K, R, S, stride, pad, groups, H, W (input size),
in0, in1 (producer layer indices, -1 = model input / no residual), act,
has_bias.  Layers are listed in topological order (producers first).

The shapes follow the public architectures the paper evaluates (its Table 4
lists ResNet-18/50, MobileNetV2, VGG-class models); weights are synthetic.
"""

OP_CONV, OP_MAXPOOL, OP_GAVGPOOL = 0, 1, 2
ACT_NONE, ACT_RELU, ACT_RELU6 = 0, 1, 2


def out_hw(L):
    """Output height/width of a layer (floor convention)."""
    if L["op"] == OP_GAVGPOOL:
        return 1, 1
    oh = (L["H"] + 2 * L["pad"] - L["R"]) // L["stride"] + 1
    ow = (L["W"] + 2 * L["pad"] - L["S"]) // L["stride"] + 1
    return oh, ow


class _Net:
    def __init__(self, C, H, W):
        self.layers = []
        self.shape = {-1: (C, H, W)}

    def _push(self, L):
        self.layers.append(L)
        i = len(self.layers) - 1
        oh, ow = out_hw(L)
        self.shape[i] = (L["K"], oh, ow)
        return i

    def conv(self, src, K, R, stride=1, pad=None, groups=1, act=ACT_RELU, add=-1, bias=0):
        C, H, W = self.shape[src]
        if pad is None:
            pad = R // 2
        return self._push(dict(op=OP_CONV, C=C, K=K, R=R, S=R, stride=stride, pad=pad,
                               groups=groups, H=H, W=W, in0=src, in1=add, act=act,
                               has_bias=bias))

    def maxpool(self, src, R, stride, pad):
        C, H, W = self.shape[src]
        return self._push(dict(op=OP_MAXPOOL, C=C, K=C, R=R, S=R, stride=stride, pad=pad,
                               groups=1, H=H, W=W, in0=src, in1=-1, act=ACT_NONE, has_bias=0))

    def gavgpool(self, src):
        C, H, W = self.shape[src]
        return self._push(dict(op=OP_GAVGPOOL, C=C, K=C, R=H, S=W, stride=1, pad=0,
                               groups=1, H=H, W=W, in0=src, in1=-1, act=ACT_NONE, has_bias=0))


def cfg1():
    """One 3x3 conv, 64->64, stride 1, pad 1, 56x56."""
    n = _Net(64, 56, 56)
    n.conv(-1, 64, 3)
    return n.layers


def cfg2_resnet18():
    """ResNet-18-shaped stack: 20 convs, 11,166,912 weights."""
    n = _Net(3, 224, 224)
    x = n.conv(-1, 64, 7, stride=2, pad=3)
    x = n.maxpool(x, 3, 2, 1)
    width = 64
    for stage, K in enumerate((64, 128, 256, 512)):
        for blk in range(2):
            stride = 2 if (stage > 0 and blk == 0) else 1
            y = n.conv(x, K, 3, stride=stride)
            if stride != 1 or width != K:
                sc = n.conv(x, K, 1, stride=stride, pad=0, act=ACT_NONE)
            else:
                sc = x
            x = n.conv(y, K, 3, add=sc)
            width = K
    return n.layers


def cfg4_resnet50():
    """ResNet-50-shaped bottleneck stack: 53 convs, stride on the 3x3."""
    n = _Net(3, 224, 224)
    x = n.conv(-1, 64, 7, stride=2, pad=3)
    x = n.maxpool(x, 3, 2, 1)
    width = 64
    for stage, (mid, out, nblk) in enumerate(((64, 256, 3), (128, 512, 4),
                                              (256, 1024, 6), (512, 2048, 3))):
        for blk in range(nblk):
            stride = 2 if (stage > 0 and blk == 0) else 1
            a = n.conv(x, mid, 1, pad=0)
            b = n.conv(a, mid, 3, stride=stride)
            if blk == 0:
                sc = n.conv(x, out, 1, stride=stride, pad=0, act=ACT_NONE)
            else:
                sc = x
            x = n.conv(b, out, 1, pad=0, add=sc)
            width = out
    del width
    return n.layers


def cfg3_mobilenetv2():
    """MobileNetV2-1.0-shaped stack: 52 convs (1x1 GEMMs + depthwise 3x3)."""
    n = _Net(3, 224, 224)
    x = n.conv(-1, 32, 3, stride=2, act=ACT_RELU6)
    cin = 32
    for t, c, reps, s in ((1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2),
                          (6, 96, 3, 1), (6, 160, 3, 2), (6, 320, 1, 1)):
        for r in range(reps):
            stride = s if r == 0 else 1
            h = x
            if t != 1:
                h = n.conv(h, cin * t, 1, pad=0, act=ACT_RELU6)
            h = n.conv(h, cin * t, 3, stride=stride, groups=cin * t, act=ACT_RELU6)
            res = x if (stride == 1 and cin == c) else -1
            x = n.conv(h, c, 1, pad=0, act=ACT_NONE, add=res)
            cin = c
    n.conv(x, 1280, 1, pad=0, act=ACT_RELU6)
    return n.layers


def cfg5_vgg16():
    """VGG-16-shaped stack: 13 3x3 convs, 2x2 max-pools between stages."""
    n = _Net(3, 224, 224)
    x = -1
    stages = ((64, 2), (128, 2), (256, 3), (512, 3), (512, 3))
    for si, (K, reps) in enumerate(stages):
        for _ in range(reps):
            x = n.conv(x, K, 3)
        if si + 1 < len(stages):
            x = n.maxpool(x, 2, 2, 0)
    return n.layers


def tiny_net(C=5, H=9, W=7):
    """A small ragged network touching every op kind; used by fast tests."""
    n = _Net(C, H, W)
    a = n.conv(-1, 12, 3)                                   # dense 3x3 s1 (Winograd-eligible)
    b = n.conv(a, 12, 3, add=a)                             # residual
    c = n.conv(b, 12, 3, groups=12, act=ACT_RELU6)          # depthwise
    d = n.conv(c, 20, 1, pad=0, act=ACT_NONE, bias=1)       # 1x1 with bias
    e = n.maxpool(d, 3, 2, 1)
    f = n.conv(e, 9, 3, stride=2)                           # strided dense 3x3
    g = n.conv(f, 16, 1, stride=2, pad=0)                   # strided 1x1
    n.gavgpool(g)
    return n.layers


CONFIGS = {
    "cfg1": cfg1,
    "cfg2_resnet18": cfg2_resnet18,
    "cfg3_mobilenetv2": cfg3_mobilenetv2,
    "cfg4_resnet50": cfg4_resnet50,
    "cfg5_vgg16": cfg5_vgg16,
}


def conv_layers(layers):
    return [i for i, L in enumerate(layers) if L["op"] == OP_CONV]


def weight_count(layers):
    return sum(L["K"] * (L["C"] // L["groups"]) * L["R"] * L["S"]
               for L in layers if L["op"] == OP_CONV)
