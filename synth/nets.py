"""Network tables: each network is a list of `Layer` descriptors plus a model config dict.

A descriptor mirrors the C struct `ftp_layer_desc` field by field.  `unit` is the
partition unit (the paper's "layer": what the profile, the partition optimiser and
run_stage(a, b) index); a residual connection never crosses a unit edge.

Activations are channels-last: (N, H, W, C); a 1-D signal is H == 1.
Canonical parameter order inside an op (an interface convention, restated on each side):
  CONV1D / CONV2D / FC : W[kh][kw][cin][cout] (FC: kh = kw = 1), then bias[cout] if has_bias
  DWCONV3x3           : W[3][3][c]
  BN                  : gamma[c], beta[c]           (state: running_mean[c], running_var[c])
"""
from collections import namedtuple

Layer = namedtuple("Layer", "unit kind cin cout k stride pad act has_bias residual_src")

KIND = dict(CONV1D=0, CONV2D=1, DWCONV3x3=2, BN=3, ACT=4, ADD_RESIDUAL=5, MAXPOOL2=6, GAP=7, FC=8,
            SOFTMAX_CE=9)
ACT = dict(NONE=0, RELU=1, RELU6=2)


def _L(unit, kind, cin=0, cout=0, k=0, stride=1, pad=0, act="NONE", has_bias=0, residual_src=-1):
    return Layer(unit, KIND[kind], cin, cout, k, stride, pad, ACT[act], has_bias, residual_src)


def num_units(layers):
    return layers[-1].unit + 1


def config(batch, in_c, in_h, in_w, n_classes, precision=0, max_stages=5, lr=0.01, momentum=0.0,
           weight_decay=0.0, bn_eps=1e-5, bn_momentum=0.1):
    return dict(batch=batch, in_c=in_c, in_h=in_h, in_w=in_w, n_classes=n_classes,
                precision=precision, max_stages=max_stages, lr=lr, momentum=momentum,
                weight_decay=weight_decay, bn_eps=bn_eps, bn_momentum=bn_momentum)


def har_cnn(batch=32, in_c=9, t=128, width=64, n_classes=6):
    """3 x [conv1d k5 pad2 + bias + ReLU], global average pool, FC, softmax cross-entropy."""
    ls = []
    c = in_c
    for u in range(3):
        ls.append(_L(u, "CONV1D", c, width, 5, 1, 2, "RELU", 1))
        c = width
    ls.append(_L(3, "GAP", c, c))
    ls.append(_L(4, "FC", c, n_classes, 1, 1, 0, "NONE", 1))
    ls.append(_L(4, "SOFTMAX_CE", n_classes, n_classes))
    return ls, config(batch, in_c, 1, t, n_classes, precision=0, lr=0.01)


def _inverted_residual(ls, unit, cin, cout, expand, stride):
    src = len(ls) - 1                      # op whose output is the block input
    hidden = cin * expand
    if expand != 1:
        ls.append(_L(unit, "CONV2D", cin, hidden, 1, 1, 0))
        ls.append(_L(unit, "BN", hidden, hidden, act="RELU6"))
    ls.append(_L(unit, "DWCONV3x3", hidden, hidden, 3, stride, 1))
    ls.append(_L(unit, "BN", hidden, hidden, act="RELU6"))
    ls.append(_L(unit, "CONV2D", hidden, cout, 1, 1, 0))
    ls.append(_L(unit, "BN", cout, cout, act="NONE"))
    if stride == 1 and cin == cout:
        ls.append(_L(unit, "ADD_RESIDUAL", cout, cout, residual_src=src))


def mobilenetv2(batch, hw, n_classes, precision, cifar, table=None, stem_c=32, last_c=1280,
                lr=0.01, momentum=0.9, weight_decay=4e-5, in_c=3):
    """MobileNetV2, width 1.0.  `cifar` selects stride 1 for the stem and the 24-channel group."""
    if table is None:
        table = [(1, 16, 1, 1), (6, 24, 2, 1 if cifar else 2), (6, 32, 3, 2), (6, 64, 4, 2),
                 (6, 96, 3, 1), (6, 160, 3, 2), (6, 320, 1, 1)]
    ls = [_L(0, "CONV2D", in_c, stem_c, 3, 1 if cifar else 2, 1), _L(0, "BN", stem_c, stem_c, act="RELU6")]
    unit, c = 1, stem_c
    for t, cout, n, s in table:
        for i in range(n):
            _inverted_residual(ls, unit, c, cout, t, s if i == 0 else 1)
            c = cout
            unit += 1
    ls.append(_L(unit, "CONV2D", c, last_c, 1, 1, 0))
    ls.append(_L(unit, "BN", last_c, last_c, act="RELU6"))
    unit += 1
    ls.append(_L(unit, "GAP", last_c, last_c))
    ls.append(_L(unit, "FC", last_c, n_classes, 1, 1, 0, "NONE", 1))
    ls.append(_L(unit, "SOFTMAX_CE", n_classes, n_classes))
    return ls, config(batch, in_c, hw, hw, n_classes, precision, lr=lr, momentum=momentum,
                      weight_decay=weight_decay)


def continual_mbv2(batch=8, hw=28, n_classes=10, precision=0):
    """The continuous-learning shape of Sec. IV-F ("Continuous Learning Evaluation"): MobileNetV2 on 28 x 28 x 1 images at batch 8 with the learning rate
    scaled to that batch (0.1 * 8 / 128 = 0.00625); strides as in the 32 x 32 variant (final map 4 x 4)."""
    return mobilenetv2(batch, hw, n_classes, precision, True, lr=0.00625, in_c=1)


def tiny_mbv2(batch=4, hw=8, n_classes=5, precision=0, momentum=0.9, weight_decay=4e-5):
    """A 4-block MobileNetV2-shaped net small enough for finite differences and brute force."""
    table = [(1, 8, 1, 1), (6, 8, 2, 1), (6, 16, 1, 2)]
    return mobilenetv2(batch, hw, n_classes, precision, True, table, stem_c=8, last_c=32,
                       momentum=momentum, weight_decay=weight_decay)


def vgg16(batch=256, hw=32, n_classes=10, precision=1, plan=None, lr=0.01, momentum=0.9,
          weight_decay=4e-5):
    """13 x [conv3x3 pad1 + BN + ReLU] with 2x2 max-pool closing each group, then FC."""
    if plan is None:
        plan = [64, 64, "M", 128, 128, "M", 256, 256, 256, "M", 512, 512, 512, "M", 512, 512, 512, "M"]
    ls, unit, c = [], -1, 3
    for p in plan:
        if p == "M":
            ls.append(_L(unit, "MAXPOOL2", c, c, 2, 2, 0))
        else:
            unit += 1
            ls.append(_L(unit, "CONV2D", c, p, 3, 1, 1))
            ls.append(_L(unit, "BN", p, p, act="RELU"))
            c = p
    unit += 1
    ls.append(_L(unit, "FC", c, n_classes, 1, 1, 0, "NONE", 1))   # spatial size is 1x1 here
    ls.append(_L(unit, "SOFTMAX_CE", n_classes, n_classes))
    return ls, config(batch, 3, hw, hw, n_classes, precision, lr=lr, momentum=momentum,
                      weight_decay=weight_decay)


def tiny_vgg(batch=4, hw=4, n_classes=3, precision=0):
    return vgg16(batch, hw, n_classes, precision, plan=[8, "M", 8, "M"], momentum=0.9)


def param_shapes(l):
    """Shapes of the trainable arrays of one op, in canonical order."""
    k = l.kind
    if k == KIND["CONV1D"]:
        s = [(1, l.k, l.cin, l.cout)]
    elif k == KIND["CONV2D"]:
        s = [(l.k, l.k, l.cin, l.cout)]
    elif k == KIND["FC"]:
        s = [(1, 1, l.cin, l.cout)]
    elif k == KIND["DWCONV3x3"]:
        return [(3, 3, l.cin)]
    elif k == KIND["BN"]:
        return [(l.cin,), (l.cin,)]
    else:
        return []
    if l.has_bias:
        s.append((l.cout,))
    return s


def state_shapes(l):
    """Shapes of the non-trainable arrays (BN running mean, running variance)."""
    return [(l.cin,), (l.cin,)] if l.kind == KIND["BN"] else []
