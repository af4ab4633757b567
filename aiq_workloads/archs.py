"""Architecture tables for the networks the paper evaluates (Section 3).

An architecture is a dict::

    {"name": str, "in_c": int, "in_h": int, "in_w": int, "n_classes": int,
     "layers": [layer, ...]}

and a layer is a dict with the keys

    name      label used in reports
    kind      "conv" (dense k x k), "dw" (depthwise k x k) or "fc"
    cin, cout channel counts ("dw": cin == cout)
    k, stride, pad
    act       "none", "relu" or "relu6", applied after bias and residual add
    input     index of the layer whose output feeds this one, -1 = network input
    residual  index of the layer whose output is added before `act`, -1 = none
    has_bn    True when the layer is followed by batch normalisation

The list order is the order of the scheme vector q = (q_1 .. q_L) of Section 2.1:
one bit-width per weight tensor.  An "fc" layer consumes the global average pool
of its input layer's output.  Only shapes and wiring live here; no arithmetic.
"""


def _conv(name, cin, cout, k, stride, act, inp, residual=-1, kind="conv"):
    return dict(name=name, kind=kind, cin=cin, cout=cout, k=k, stride=stride,
                pad=k // 2, act=act, input=inp, residual=residual, has_bn=True)


def _fc(name, cin, cout, inp):
    return dict(name=name, kind="fc", cin=cin, cout=cout, k=1, stride=1, pad=0,
                act="none", input=inp, residual=-1, has_bn=False)


def resnet20(channels=(16, 32, 64), n_classes=10, in_hw=32, name="resnet20", stem=None):
    """CIFAR ResNet-20 with 1x1 projection shortcuts where shape changes.

    Stem conv3x3 (`stem` channels, default channels[0]), three stages of three basic
    blocks, global average pool, linear classifier.  Scheme order: stem; per block conv1,
    conv2, then the block's projection (if any); classifier last.
    """
    stem = channels[0] if stem is None else stem
    layers = [_conv("stem", 3, stem, 3, 1, "relu", -1)]
    prev = 0            # index of the layer producing the current block input
    cin = stem
    for si, c in enumerate(channels):
        for b in range(3):
            stride = 2 if (si > 0 and b == 0) else 1
            need_proj = stride != 1 or cin != c
            i1 = len(layers)
            i2 = i1 + 1
            ip = i1 + 2
            layers.append(_conv(f"s{si + 1}.b{b}.c1", cin, c, 3, stride, "relu", prev))
            layers.append(_conv(f"s{si + 1}.b{b}.c2", c, c, 3, 1, "relu", i1,
                                residual=ip if need_proj else prev))
            if need_proj:
                layers.append(_conv(f"s{si + 1}.b{b}.proj", cin, c, 1, stride, "none", prev))
            prev = i2
            cin = c
    layers.append(_fc("fc", cin, n_classes, prev))
    return dict(name=name, in_c=3, in_h=in_hw, in_w=in_hw, n_classes=n_classes, layers=layers)


def heavy_early_resnet20(n_classes=10, in_hw=32):
    """HeavyEarlyResNet20 (Section 4.5): ResNet-20 with the channel progression reversed,
    channel groups (64, 32, 16, 16) for (stem, stage 1, stage 2, stage 3) instead of
    (16, 16, 32, 64).  The first block of stage 1 then changes the width (64 -> 32) at
    stride 1 and gets a projection shortcut like every other shape change."""
    return resnet20(channels=(32, 16, 16), n_classes=n_classes, in_hw=in_hw, name="heavy_early_resnet20", stem=64)


def plain_convnet20(n_classes=10, in_hw=32, width=64):
    """PlainConvNet20 (Section 4.5): 20 convolution layers of 64 channels, no shortcuts, then
    the classifier (21 weight tensors, as in Table 1).  The paper does not say where the
    network reduces resolution; reading: stride 2 at layers 7 and 13, where ResNet-20 starts
    its second and third stage, so that depth and cost stay comparable."""
    layers = []
    cin = 3
    for i in range(20):
        stride = 2 if i in (7, 13) else 1
        layers.append(_conv(f"f{3 * i}", cin, width, 3, stride, "relu", i - 1))
        cin = width
    layers.append(_fc("cls", width, n_classes, 19))
    return dict(name="plain_convnet20", in_c=3, in_h=in_hw, in_w=in_hw, n_classes=n_classes, layers=layers)


_MBV2_CFG = [(1, 16, 1), (6, 24, 2), (6, 32, 3), (6, 64, 4), (6, 96, 3), (6, 160, 3), (6, 320, 1)]


def mobilenet_v2(variant="cifar"):
    """MobileNetV2, width 1.0.

    variant "cifar":    32x32 input, stem stride 1, stage strides (1,1,1,2,1,2,1), 10 classes.
    variant "imagenet": 224x224 input, stem stride 2, stage strides (1,2,2,2,1,2,1), 1000 classes.
    """
    if variant == "cifar":
        hw, stem_stride, strides, n_classes = 32, 1, (1, 1, 1, 2, 1, 2, 1), 10
    elif variant == "imagenet":
        hw, stem_stride, strides, n_classes = 224, 2, (1, 2, 2, 2, 1, 2, 1), 1000
    else:
        raise ValueError(variant)
    layers = [_conv("stem", 3, 32, 3, stem_stride, "relu6", -1)]
    prev, cin, bi = 0, 32, 0
    for (t, c, n), s0 in zip(_MBV2_CFG, strides):
        for i in range(n):
            stride = s0 if i == 0 else 1
            hid = cin * t
            src = prev
            if t != 1:
                layers.append(_conv(f"b{bi}.expand", cin, hid, 1, 1, "relu6", src))
                src = len(layers) - 1
            layers.append(_conv(f"b{bi}.dw", hid, hid, 3, stride, "relu6", src, kind="dw"))
            src = len(layers) - 1
            use_res = stride == 1 and cin == c
            layers.append(_conv(f"b{bi}.project", hid, c, 1, 1, "none", src,
                                residual=prev if use_res else -1))
            prev = len(layers) - 1
            cin = c
            bi += 1
    layers.append(_conv("head", cin, 1280, 1, 1, "relu6", prev))
    layers.append(_fc("fc", 1280, n_classes, len(layers) - 1))
    return dict(name=f"mobilenet_v2_{variant}", in_c=3, in_h=hw, in_w=hw,
                n_classes=n_classes, layers=layers)


def tiny_net(in_c=3, hw=8, n_classes=5):
    """A small network touching every layer kind and wiring form (test workload)."""
    layers = [
        _conv("stem", in_c, 8, 3, 1, "relu", -1),
        _conv("b0.c1", 8, 16, 3, 2, "relu", 0),
        _conv("b0.c2", 16, 16, 3, 1, "relu", 1, residual=3),
        _conv("b0.proj", 8, 16, 1, 2, "none", 0),
        _conv("b1.expand", 16, 48, 1, 1, "relu6", 2),
        _conv("b1.dw", 48, 48, 3, 1, "relu6", 4, kind="dw"),
        _conv("b1.project", 48, 16, 1, 1, "none", 5, residual=2),
        _conv("b2.dw", 16, 16, 3, 2, "relu6", 6, kind="dw"),
        _conv("b2.project", 16, 24, 1, 1, "none", 7),
        _fc("fc", 24, n_classes, 8),
    ]
    return dict(name="tiny_net", in_c=in_c, in_h=hw, in_w=hw, n_classes=n_classes, layers=layers)


def depthwise_stack(hw, channels=96, n_classes=7):
    """A short network around two depthwise layers (test workload): stem 3x3, depthwise 3x3 at
    stride 2, pointwise, depthwise 3x3 at stride 1 with a shortcut from its own input,
    classifier.  `hw` sets the image size, so the depthwise layers see any output height."""
    c = channels
    layers = [
        _conv("stem", 3, c, 3, 1, "relu6", -1),
        _conv("dw.s2", c, c, 3, 2, "relu6", 0, kind="dw"),
        _conv("pw", c, c, 1, 1, "none", 1),
        _conv("dw.s1", c, c, 3, 1, "relu6", 2, residual=2, kind="dw"),
        _fc("fc", c, n_classes, 3),
    ]
    return dict(name=f"depthwise_stack_{hw}", in_c=3, in_h=hw, in_w=hw, n_classes=n_classes, layers=layers)


def pointwise_stack(cin, cout, hw=8, n_classes=6):
    """A short network around one pointwise (1x1) convolution (test workload): stem 3x3 to `cin`
    channels, pointwise `cin` -> `cout`, classifier.  Lets a test reach any channel pair of the
    pointwise layers of MobileNetV2 without the 50 layers around them."""
    layers = [
        _conv("stem", 3, cin, 3, 1, "relu6", -1),
        _conv("pw", cin, cout, 1, 1, "relu6", 0),
        _fc("fc", cout, n_classes, 1),
    ]
    return dict(name=f"pointwise_stack_{cin}_{cout}", in_c=3, in_h=hw, in_w=hw, n_classes=n_classes, layers=layers)


def inverted_residual_stack(cin, cout, hw=8, stride=1, t=6, n_classes=6):
    """A short network around one MobileNetV2 inverted-residual block (test workload): stem 3x3
    to `cin` channels, expansion 1x1 to t * cin, depthwise 3x3 at `stride`, projection 1x1 to
    `cout` with the shortcut from the block's input when stride is 1 and cin == cout, classifier."""
    hid = cin * t
    layers = [
        _conv("stem", 3, cin, 3, 1, "relu6", -1),
        _conv("b.expand", cin, hid, 1, 1, "relu6", 0),
        _conv("b.dw", hid, hid, 3, stride, "relu6", 1, kind="dw"),
        _conv("b.project", hid, cout, 1, 1, "none", 2, residual=0 if (stride == 1 and cin == cout) else -1),
        _fc("fc", cout, n_classes, 3),
    ]
    return dict(name=f"inverted_residual_stack_{cin}_{cout}_{hw}_s{stride}", in_c=3, in_h=hw, in_w=hw,
                n_classes=n_classes, layers=layers)


def conv_layer_indices(arch):
    """Indices of every layer that is not the classifier (the sweep candidates)."""
    return [i for i, l in enumerate(arch["layers"]) if l["kind"] != "fc"]
