"""Op lists of the pre-activation bottleneck ResNets the benchmark configurations name.

An op is the tuple (kind, src0, src1, c_in, c_out, ksize, stride, pad, eps);
src = index of the producing op, -1 = the network input.  Inside a block the
order is BNRELU, CONV1x1, BNRELU, CONV3x3, BNRELU, CONV1x1, [projection CONV1x1], ADD.
The stride of a down-sampling block sits on its first 1x1 conv and on the
projection, which reads the raw block input; there is no BN after the stem.
"""
from collections import namedtuple

CONV, BNRELU, ADD, MAXPOOL, HEAD, BN, RELU = 1, 2, 3, 4, 5, 6, 7
Op = namedtuple("Op", "kind src0 src1 c_in c_out ksize stride pad eps")
EPS = 1e-5


def _bottleneck_stages(ops, t, c_t, widths, blocks, first_stride, outs=None):
    """widths = bottleneck channels per stage; outs = block output channels per stage (default 4 x width)."""
    for si, (w, nb) in enumerate(zip(widths, blocks)):
        co = 4 * w if outs is None else outs[si]
        for bi in range(nb):
            s = first_stride[si] if bi == 0 else 1
            ops.append(Op(BNRELU, t, -1, c_t, c_t, 0, 1, 0, EPS)); a1 = len(ops) - 1
            ops.append(Op(CONV, a1, -1, c_t, w, 1, s, 0, 0.0)); c1 = len(ops) - 1
            ops.append(Op(BNRELU, c1, -1, w, w, 0, 1, 0, EPS)); a2 = len(ops) - 1
            ops.append(Op(CONV, a2, -1, w, w, 3, 1, 1, 0.0)); c2 = len(ops) - 1
            ops.append(Op(BNRELU, c2, -1, w, w, 0, 1, 0, EPS)); a3 = len(ops) - 1
            ops.append(Op(CONV, a3, -1, w, co, 1, 1, 0, 0.0)); c3 = len(ops) - 1
            short = t
            if bi == 0:
                ops.append(Op(CONV, t, -1, c_t, co, 1, s, 0, 0.0)); short = len(ops) - 1
            ops.append(Op(ADD, c3, short, co, co, 0, 1, 0, 0.0)); t = len(ops) - 1
            c_t = co
    return t, c_t


def resnet_v2_cifar(n, widths=(16, 32, 64), n_classes=10, in_ch=3, outs=None):
    """Depth 9n+2: 3x3 stem to widths[0] channels, three stages of n bottleneck blocks.

    outs = block output channels per stage.  The default (4 x width: 64/128/256 from widths 16/32/64) is the
    benchmark's instance; widths (16, 64, 128) with outs (64, 128, 256) is the chaining rule of the Keras example
    the paper takes its definitions from (a stage's bottleneck width = the previous stage's output)."""
    ops = [Op(CONV, -1, -1, in_ch, widths[0], 3, 1, 1, 0.0)]
    t, c_t = _bottleneck_stages(ops, 0, widths[0], widths, (n,) * len(widths), (1,) + (2,) * (len(widths) - 1), outs)
    ops.append(Op(BNRELU, t, -1, c_t, c_t, 0, 1, 0, EPS))
    ops.append(Op(HEAD, len(ops) - 1, -1, c_t, n_classes, 0, 1, 0, 0.0))
    return ops


def resnet_v1_cifar(n, widths=(16, 32, 64), n_classes=10, in_ch=3):
    """Post-activation (v1) basic-block ResNet of depth 6n+2, the Keras example's definition: 3x3 stem conv, BN, ReLU;
    per block conv3x3 (stride 2 in the first block of stages 2 and 3), BN, ReLU, conv3x3, BN, ADD with the shortcut
    (a 1x1 stride-2 convolution of the block input where the shape changes, identity elsewhere), ReLU; then the head.
    Convolution biases are left out: in front of a BN they are absorbed by its shift."""
    ops = [Op(CONV, -1, -1, in_ch, widths[0], 3, 1, 1, 0.0)]
    ops.append(Op(BNRELU, 0, -1, widths[0], widths[0], 0, 1, 0, EPS))
    t, c_t = 1, widths[0]
    for si, w in enumerate(widths):
        for bi in range(n):
            s = 2 if (si > 0 and bi == 0) else 1
            ops.append(Op(CONV, t, -1, c_t, w, 3, s, 1, 0.0)); c1 = len(ops) - 1
            ops.append(Op(BNRELU, c1, -1, w, w, 0, 1, 0, EPS)); a1 = len(ops) - 1
            ops.append(Op(CONV, a1, -1, w, w, 3, 1, 1, 0.0)); c2 = len(ops) - 1
            ops.append(Op(BN, c2, -1, w, w, 0, 1, 0, EPS)); b2 = len(ops) - 1
            short = t
            if s != 1 or c_t != w:
                ops.append(Op(CONV, t, -1, c_t, w, 1, s, 0, 0.0)); short = len(ops) - 1
            ops.append(Op(ADD, b2, short, w, w, 0, 1, 0, 0.0)); ad = len(ops) - 1
            ops.append(Op(RELU, ad, -1, w, w, 0, 1, 0, 0.0)); t = len(ops) - 1
            c_t = w
    ops.append(Op(HEAD, t, -1, c_t, n_classes, 0, 1, 0, 0.0))
    return ops


def vgg16_cifar(widths=(64, 128, 256, 512, 512), convs=(2, 2, 3, 3, 3), fc=4096, n_classes=10, in_ch=3):
    """VGG-16 laid out for 32x32 inputs: five groups of 3x3 convolutions (pad 1) each followed by ReLU, a 2x2 stride-2
    max-pool after every group (32 -> 1 pixel), two hidden fully connected layers with ReLU (1x1 convolutions on the 1x1
    map) and the classifier (the head's mean over one pixel is the identity).  13 + 3 weight layers, no batch norm.
    Biases are left out: the op list has no bias term for convolutions."""
    ops, t, c_t = [], -1, in_ch
    for w, k in zip(widths, convs):
        for _ in range(k):
            ops.append(Op(CONV, t, -1, c_t, w, 3, 1, 1, 0.0)); t = len(ops) - 1
            ops.append(Op(RELU, t, -1, w, w, 0, 1, 0, 0.0)); t = len(ops) - 1
            c_t = w
        ops.append(Op(MAXPOOL, t, -1, c_t, c_t, 2, 2, 0, 0.0)); t = len(ops) - 1
    for _ in range(2):
        ops.append(Op(CONV, t, -1, c_t, fc, 1, 1, 0, 0.0)); t = len(ops) - 1
        ops.append(Op(RELU, t, -1, fc, fc, 0, 1, 0, 0.0)); t = len(ops) - 1
        c_t = fc
    ops.append(Op(HEAD, t, -1, c_t, n_classes, 0, 1, 0, 0.0))
    return ops


def resnet_v2_imagenet(blocks=(3, 8, 36, 3), widths=(64, 128, 256, 512), n_classes=1000, in_ch=3):
    """7x7 stride-2 stem, 3x3 stride-2 max-pool, four bottleneck stages."""
    ops = [Op(CONV, -1, -1, in_ch, widths[0], 7, 2, 3, 0.0),
           Op(MAXPOOL, 0, -1, widths[0], widths[0], 3, 2, 1, 0.0)]
    t, c_t = _bottleneck_stages(ops, 1, widths[0], widths, blocks, (1,) + (2,) * (len(widths) - 1))
    ops.append(Op(BNRELU, t, -1, c_t, c_t, 0, 1, 0, EPS))
    ops.append(Op(HEAD, len(ops) - 1, -1, c_t, n_classes, 0, 1, 0, 0.0))
    return ops


def default_cuts(n_ops, P):
    """Equal op counts per partition: cut p at floor(p*K/P)."""
    return [(p * n_ops) // P for p in range(1, P)]


# name -> (ops builder, input (H, W, C), batch B, micro-batches M, partitions P)
CONFIGS = {
    "r11":   (lambda: resnet_v2_cifar(1), (32, 32, 3), 8, 2, 2),
    "r110":  (lambda: resnet_v2_cifar(12), (32, 32, 3), 128, 4, 4),
    "r1001": (lambda: resnet_v2_cifar(111), (32, 32, 3), 128, 8, 8),
    "r152":  (lambda: resnet_v2_imagenet(), (224, 224, 3), 64, 4, 4),
    # the ~30 M-parameter width variant of ResNet-1001 (Section 6.3 quotes that size) and a short net of the same widths
    "r1001k": (lambda: resnet_v2_cifar(111, (16, 64, 128), outs=(64, 128, 256)), (32, 32, 3), 128, 8, 8),
    "r20k":   (lambda: resnet_v2_cifar(2, (16, 64, 128), outs=(64, 128, 256)), (32, 32, 3), 16, 2, 2),
    # the paper's ResNet-110 is the post-activation (v1) basic-block net, depth 6n+2 with n = 18; a short one for tests
    "r110v1": (lambda: resnet_v1_cifar(18), (32, 32, 3), 128, 4, 4),
    "r8v1":   (lambda: resnet_v1_cifar(1), (32, 32, 3), 8, 2, 2),
    # the paper's third model and a narrow copy of it for tests
    "vgg16":  (lambda: vgg16_cifar(), (32, 32, 3), 128, 4, 4),
    "vgg16s": (lambda: vgg16_cifar(widths=(16, 16, 32, 32, 64), fc=64), (32, 32, 3), 8, 2, 2),
}


def config(name):
    build, hwc, B, M, P = CONFIGS[name]
    ops = build()
    return dict(name=name, ops=ops, in_hwc=hwc, B=B, M=M, P=P, cuts=default_cuts(len(ops), P))


def conv_sweep_shapes():
    """The convolution micro-benchmark sweep: (ksize, stride, c_in, c_out, H) at batch 128.

    The cross product of the channel pair at each resolution for 1x1 and 3x3
    (pad 1) convolutions, plus the four stride-2 transitions.
    """
    out = []
    for H, (a, b) in ((32, (16, 64)), (16, (32, 128)), (8, (64, 256))):
        for k in (1, 3):
            for ci in (a, b):
                for co in (a, b):
                    out.append((k, 1, ci, co, H))
    out += [(1, 2, 64, 32, 32), (1, 2, 64, 128, 32), (1, 2, 128, 64, 16), (1, 2, 128, 256, 16)]
    return out
