"""Layer lists and stage splits of the benchmark networks.

A network is a flat list of `Layer` records and, per layer, the index of the
pipeline stage it belongs to (non-decreasing).  A stage starts with the layer
that owns its weights (FC or CONV2D); normalisation, skip add, activation and
pooling that follow ride in the same stage, as the paper groups a convolution
with its normalisation and activation (Section 2.1).  Stage `src` fields name
an earlier stage whose output for the same sample is read (-1: the stage just
before, or the network input for stage 0).
"""
from dataclasses import dataclass, field
from enum import IntEnum
from typing import List, Tuple


class OP(IntEnum):
    FC = 0
    CONV2D = 1
    GROUPNORM = 2
    RELU = 3
    MAXPOOL = 4
    AVGPOOL_GLOBAL = 5
    ADD_SKIP = 6
    SOFTMAX_CE = 7


SKIP_IDENTITY = 0      # same shape
SKIP_SUBSAMPLE_PAD = 1  # every second pixel, new channels filled with zeros
SKIP_PRENORM = 2        # flag, added to one of the above: the skip input joins the convolution output BEFORE the
                        # normalisation, and it is the source stage's own convolution output after ITS such
                        # addition (the running sum of a pre-activation residual network)

FLAG_SC = 1
FLAG_LWP = 2
FLAG_LWP_WFORM = 4
FLAG_CONV_BF16 = 8


@dataclass
class Layer:
    op: int
    c_in: int = 0
    c_out: int = 0
    k: int = 0
    stride: int = 1
    pad: int = 0
    groups: int = 0
    src: int = -1
    skip_mode: int = 0

    def astuple(self):
        return (int(self.op), self.c_in, self.c_out, self.k, self.stride,
                self.pad, self.groups, self.src, self.skip_mode)


@dataclass
class Workload:
    name: str
    layers: List[Layer]
    stage_of_layer: List[int]
    in_shape: Tuple[int, int, int]
    n_classes: int
    lr: float
    momentum: float
    ticks: int
    seed: int
    flags: int = FLAG_SC | FLAG_LWP
    notes: str = ""

    @property
    def n_stages(self):
        return self.stage_of_layer[-1] + 1

    @property
    def sample_elems(self):
        c, h, w = self.in_shape
        return c * h * w


class _Builder:
    def __init__(self):
        self.layers, self.stage_of = [], []
        self.stage = -1

    def new_stage(self):
        self.stage += 1
        return self.stage

    def add(self, layer):
        self.layers.append(layer)
        self.stage_of.append(self.stage)

    def fc(self, c_in, c_out, relu=True, loss=False, src=-1):
        s = self.new_stage()
        self.add(Layer(OP.FC, c_in, c_out, src=src))
        if relu:
            self.add(Layer(OP.RELU))
        if loss:
            self.add(Layer(OP.SOFTMAX_CE))
        return s

    def conv(self, c_in, c_out, k, stride, pad, groups, relu=True, src=-1,
             skip=None, skip_mode=SKIP_IDENTITY, pool=None, avgpool=False):
        s = self.new_stage()
        self.add(Layer(OP.CONV2D, c_in, c_out, k, stride, pad, src=src))
        if skip is not None and skip_mode & SKIP_PRENORM:
            self.add(Layer(OP.ADD_SKIP, src=skip, skip_mode=skip_mode))
        self.add(Layer(OP.GROUPNORM, c_out, c_out, groups=groups))
        if skip is not None and not skip_mode & SKIP_PRENORM:
            self.add(Layer(OP.ADD_SKIP, src=skip, skip_mode=skip_mode))
        if relu:
            self.add(Layer(OP.RELU))
        if pool is not None:
            pk, ps, pp = pool
            self.add(Layer(OP.MAXPOOL, k=pk, stride=ps, pad=pp))
        if avgpool:
            self.add(Layer(OP.AVGPOOL_GLOBAL))
        return s


def mlp(sizes, name="mlp", lr=0.01, momentum=0.9, ticks=64, seed=0,
        flags=FLAG_SC | FLAG_LWP):
    """FC sizes[0]->...->sizes[-1], ReLU between, softmax cross-entropy last."""
    b = _Builder()
    n = len(sizes) - 1
    for q in range(n):
        last = q == n - 1
        b.fc(sizes[q], sizes[q + 1], relu=not last, loss=last)
    return Workload(name, b.layers, b.stage_of, (sizes[0], 1, 1), sizes[-1],
                    lr, momentum, ticks, seed, flags)


def _vgg11():
    b = _Builder()
    chans = [64, 128, 256, 256, 512, 512, 512, 512]
    pool_after = {1, 2, 4, 6, 8}
    c_in = 3
    for q, c in enumerate(chans, start=1):
        b.conv(c_in, c, 3, 1, 1, 32,
               pool=(2, 2, 0) if q in pool_after else None)
        c_in = c
    b.fc(512, 10, relu=False, loss=True)
    return Workload("vgg11", b.layers, b.stage_of, (3, 32, 32), 10,
                    0.01, 0.9, 2048, 2)


def _resnet20(widths=(16, 32, 64), blocks=3, groups=8, hw=32, n_classes=10,
              name="resnet20", lr=0.01, ticks=4096, seed=3):
    b = _Builder()
    prev = b.conv(3, widths[0], 3, 1, 1, groups)
    c_in = widths[0]
    n_blocks = len(widths) * blocks
    done = 0
    for g, c in enumerate(widths):
        for q in range(blocks):
            down = g > 0 and q == 0
            b.conv(c_in, c, 3, 2 if down else 1, 1, groups)
            done += 1
            prev = b.conv(c, c, 3, 1, 1, groups, skip=prev,
                          skip_mode=SKIP_SUBSAMPLE_PAD if down else SKIP_IDENTITY,
                          avgpool=(done == n_blocks))
            c_in = c
    b.fc(c_in, n_classes, relu=False, loss=True)
    return Workload(name, b.layers, b.stage_of, (3, hw, hw), n_classes,
                    lr, 0.9, ticks, seed)


def _resnet50(depths=(3, 4, 6, 3), base=64, hw=224, n_classes=1000,
              groups=32, name="resnet50", ticks=512, seed=4,
              flags=FLAG_SC | FLAG_LWP | FLAG_CONV_BF16, relu=True):
    """relu=False leaves the activation out of every stage after the stem (a
    network that is smooth in its weights; the stem keeps ReLU and max-pool)."""
    b = _Builder()
    prev = b.conv(3, base, 7, 2, 3, groups, pool=(3, 2, 1))
    c_in = base
    n_blocks = sum(depths)
    done = 0
    for g, depth in enumerate(depths):
        w = base * (2 ** g)
        for q in range(depth):
            stride = 2 if (g > 0 and q == 0) else 1
            block_in = prev
            if q == 0:
                # projection shortcut: 1x1 conv + GN, no activation
                skip = b.conv(c_in, 4 * w, 1, stride, 0, groups, relu=False,
                              src=block_in)
            else:
                skip = block_in
            b.conv(c_in, w, 1, 1, 0, groups, src=block_in, relu=relu)
            b.conv(w, w, 3, stride, 1, groups, relu=relu)
            done += 1
            prev = b.conv(w, 4 * w, 1, 1, 0, groups, skip=skip, relu=relu,
                          avgpool=(done == n_blocks))
            c_in = 4 * w
    b.fc(c_in, n_classes, relu=False, loss=True)
    return Workload(name, b.layers, b.stage_of, (3, hw, hw), n_classes,
                    0.005, 0.9, ticks, seed, flags)


def tiny_cnn(seed=11, ticks=24, flags=FLAG_SC | FLAG_LWP):
    """3 conv stages (one pooled) + FC on 3x8x8 inputs: a few hundred weights."""
    b = _Builder()
    b.conv(3, 4, 3, 1, 1, 2, pool=(2, 2, 0))
    b.conv(4, 6, 3, 1, 1, 3)
    b.conv(6, 6, 3, 2, 1, 3)
    b.fc(6 * 2 * 2, 5, relu=False, loss=True)
    return Workload("tiny_cnn", b.layers, b.stage_of, (3, 8, 8), 5,
                    0.02, 0.9, ticks, seed, flags)


def tail_cnn(seed=14, ticks=40, flags=FLAG_SC | FLAG_LWP):
    """The tail of a VGG-style net in small: 3x3 convolutions on 4x4 and 2x2 images with
    32..64 channels (a handful of output pixels per weight: weight-streaming stages)."""
    b = _Builder()
    b.conv(3, 32, 3, 1, 1, 8, pool=(2, 2, 0))         # 8x8 -> 4x4
    b.conv(32, 64, 3, 1, 1, 8)                        # 4x4
    b.conv(64, 64, 3, 1, 1, 16, pool=(2, 2, 0))       # 4x4 -> 2x2
    b.conv(64, 32, 3, 1, 1, 4)                        # 2x2
    b.conv(32, 32, 3, 1, 1, 8, pool=(2, 2, 0))        # 2x2 -> 1x1
    b.fc(32, 6, relu=False, loss=True)
    return Workload("tail_cnn", b.layers, b.stage_of, (3, 8, 8), 6,
                    0.01, 0.9, ticks, seed, flags)


def tiny_resnet(seed=12, ticks=40, flags=FLAG_SC | FLAG_LWP, bottleneck=False, relu=True):
    """Small residual nets that reach every skip form the big ones use."""
    if bottleneck:
        return _resnet50(depths=(1, 2), base=8, hw=16, n_classes=7, groups=4,
                         name="tiny_bottleneck", ticks=ticks, seed=seed,
                         flags=flags, relu=relu)
    return _resnet20(widths=(4, 8), blocks=1, groups=2, hw=8, n_classes=5,
                     name="tiny_resnet", lr=0.02, ticks=ticks, seed=seed)


def preact_resnet(widths=(8, 16), blocks=2, groups=4, hw=16, n_classes=10, name="preact_resnet",
                  lr=0.01, ticks=48, seed=15, flags=FLAG_SC | FLAG_LWP, relu=True):
    """Pre-activation residual network (normalisation and ReLU BEFORE each convolution, the layout the
    paper trains: Section 4, Experiment Details) in stages of convolution -> (+ running sum) ->
    normalisation -> ReLU: a stage's normalisation and ReLU are the pre-activation of the next
    convolution, and the residual sum runs along the convolution outputs.  Basic blocks of two 3x3
    convolutions; parameter-free shortcut (every second pixel, zero channels) where the width changes."""
    b = _Builder()
    prev = b.conv(3, widths[0], 3, 1, 1, groups, relu=relu)      # stem; its output sum starts the residual stream
    c_in = widths[0]
    n_blocks, done = len(widths) * blocks, 0
    for g, c in enumerate(widths):
        for q in range(blocks):
            down = g > 0 and q == 0
            b.conv(c_in, c, 3, 2 if down else 1, 1, groups, relu=relu)
            done += 1
            prev = b.conv(c, c, 3, 1, 1, groups, relu=relu, skip=prev,
                          skip_mode=(SKIP_SUBSAMPLE_PAD if down else SKIP_IDENTITY) | SKIP_PRENORM,
                          avgpool=(done == n_blocks))
            c_in = c
    b.fc(c_in, n_classes, relu=False, loss=True)
    return Workload(name, b.layers, b.stage_of, (3, hw, hw), n_classes, lr, 0.9, ticks, seed, flags)


def tall_bottleneck(seed=13, ticks=48, lr=0.001, flags=FLAG_SC | FLAG_LWP | FLAG_CONV_BF16, relu=True):
    """Few channels on large images: the ResNet-50 stage kinds (7x7/2 stem with
    3x3/2 max-pool, two bottleneck blocks with projection shortcuts, the second
    one strided) at 8..64 channels on 3x256x256 inputs.  The stem's output has
    16384 pixels and the first block's 4096, so the shapes only large images
    reach (weight gradients contracting over thousands of pixels, normalisation
    groups cut into several pieces per channel) are met by a net whose CPU
    evaluation takes a fraction of a second per tick."""
    wl = _resnet50(depths=(1, 1), base=8, hw=256, n_classes=7, groups=4,
                   name="tall_bottleneck", ticks=ticks, seed=seed, flags=flags, relu=relu)
    wl.lr = lr
    return wl


WORKLOAD_NAMES = ["mlp4", "mlp16x2048", "vgg11", "resnet20", "resnet50"]


def workload(name):
    """The five benchmark workloads, by name."""
    if name == "mlp4":
        return mlp([784, 256, 256, 256, 10], "mlp4", 0.01, 0.9, 256, 0)
    if name == "mlp16x2048":
        return mlp([2048] * 16 + [10], "mlp16x2048", 0.005, 0.9, 4096, 1)
    if name == "vgg11":
        return _vgg11()
    if name == "resnet20":
        return _resnet20()
    if name == "resnet50":
        return _resnet50()
    if name == "resnet50_112":
        # the same 54 stages on 112x112 images: a quarter of the activation
        # memory, for profiler captures that replay kernels many times
        return _resnet50(hw=112, name="resnet50_112")
    raise KeyError(name)


def param_sizes(wl):
    """[(kind, count, fan_in)] per parameter tensor, in layer order."""
    out = []
    for L in wl.layers:
        if L.op == OP.FC:
            out.append(("weight", L.c_in * L.c_out, L.c_in))
            out.append(("zeros", L.c_out, 0))
        elif L.op == OP.CONV2D:
            out.append(("weight", L.c_out * L.c_in * L.k * L.k, L.c_in * L.k * L.k))
        elif L.op == OP.GROUPNORM:
            out.append(("ones", L.c_out, 0))
            out.append(("zeros", L.c_out, 0))
    return out


def infer_shapes(wl):
    """Output shape (c, h, w) of every stage; bookkeeping only."""
    shapes = []
    cur = None
    for L, s in zip(wl.layers, wl.stage_of_layer):
        if L.op in (OP.FC, OP.CONV2D):
            if L.src >= 0:
                cur = shapes[L.src]
            elif s == 0:
                cur = wl.in_shape
            else:
                cur = shapes[s - 1]
            if L.op == OP.FC:
                assert cur[0] * cur[1] * cur[2] == L.c_in, (s, cur, L.c_in)
                cur = (L.c_out, 1, 1)
            else:
                assert cur[0] == L.c_in, (s, cur, L.c_in)
                h = (cur[1] + 2 * L.pad - L.k) // L.stride + 1
                w = (cur[2] + 2 * L.pad - L.k) // L.stride + 1
                cur = (L.c_out, h, w)
            shapes.append(cur)
        elif L.op == OP.MAXPOOL:
            h = (cur[1] + 2 * L.pad - L.k) // L.stride + 1
            w = (cur[2] + 2 * L.pad - L.k) // L.stride + 1
            cur = (cur[0], h, w)
            shapes[s] = cur
        elif L.op == OP.AVGPOOL_GLOBAL:
            cur = (cur[0], 1, 1)
            shapes[s] = cur
    return shapes


def work_per_tick(wl):
    """Bookkeeping for benchmarks: what one steady-state tick has to touch.

    Returns a dict with `params`; forward multiply-accumulates per tick split
    into `macs_fc`, `macs_conv_f32` (CUDA cores) and `macs_conv_bf16` (tensor
    cores: every conv of a bfloat16 workload whose channel counts are multiples
    of 8 and whose input is not the network input); and `act_elems`, the
    activation elements a tick moves at least once: per stage 3 x input
    (forward read, weight-gradient read, data gradient written) + 2 x head
    output (written forward, read backward) + 2 x stage output (written forward,
    its gradient read backward)."""
    shapes = infer_shapes(wl)
    out = dict(params=0, macs_fc=0, macs_conv_f32=0, macs_conv_bf16=0, act_elems=0)
    bf16 = bool(wl.flags & FLAG_CONV_BF16)
    for L, s in zip(wl.layers, wl.stage_of_layer):
        if L.op not in (OP.FC, OP.CONV2D):
            if L.op == OP.GROUPNORM:
                out["params"] += 2 * L.c_out
            continue
        src = L.src if L.src >= 0 else s - 1
        cin = wl.in_shape if src < 0 else shapes[src]
        a_in = cin[0] * cin[1] * cin[2]
        a_out = shapes[s][0] * shapes[s][1] * shapes[s][2]
        if L.op == OP.FC:
            out["params"] += L.c_in * L.c_out + L.c_out
            out["macs_fc"] += L.c_in * L.c_out
            a_head = L.c_out
        else:
            h = (cin[1] + 2 * L.pad - L.k) // L.stride + 1
            w = (cin[2] + 2 * L.pad - L.k) // L.stride + 1
            a_head = L.c_out * h * w
            macs = a_head * L.c_in * L.k * L.k
            out["params"] += L.c_out * L.c_in * L.k * L.k
            tc = bf16 and src >= 0 and L.c_in % 8 == 0 and L.c_out % 8 == 0
            out["macs_conv_bf16" if tc else "macs_conv_f32"] += macs
        out["act_elems"] += 3 * a_in + 2 * a_head + 2 * a_out
    return out
