"""Seeded synthetic workloads: layer shapes and random tensors only.

This module holds no arithmetic of the quantization method.  It describes the
networks whose *shapes* the paper evaluates on (Section 4: GoogLeNet v1,
ResNet-50, MobileNet v1; VGG is named in the introduction) as flat lists of
layer records, and draws every float tensor from a counter-based generator
(numpy Philox keyed by (seed, tensor id)), so the CUDA path and the CPU checker
can be fed identical bytes.  The paper's ImageNet images and trained Caffe
weights are not reproduced; these tensors stand in for them.

A network is a dict:
  name, input: (N, H, W, C), input_dist: "normal" | "halfnormal",
  per_channel: weight scales per output channel (1) or per layer (0),
  buffers: {buffer name: (H, W, channel pitch)},
  nodes: list of dicts, in execution order.  Nodes that write the same `dst`
         buffer form a concat group and are listed consecutively.
Conv node keys: name, op="conv", src, dst, dst_c_offset, C (= pitch of src),
  C_real (channels that carry data; the rest of the pitch is zero padding), K, R, S,
  stride, pad, groups, relu, symmetric, residual (buffer name or None),
  w_std, b_std, tid (tensor id for the generator).
Pool node keys: name, op="maxpool", src, dst, R, S, stride, pad.
"""
import math

import numpy as np


def rng_for(seed: int, tensor_id: int) -> np.random.Generator:
    """Counter-based stream: Philox-4x64 keyed by (seed, tensor id)."""
    return np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), int(tensor_id)]))


def out_size(h, r, stride, pad):
    return (h + 2 * pad - r) // stride + 1


def pad16(c):
    return (c + 15) // 16 * 16


class _Builder:
    def __init__(self, name, input_shape, input_dist, per_channel, w_std=None):
        self.net = dict(name=name, input=tuple(input_shape), input_dist=input_dist,
                        per_channel=per_channel, buffers={}, nodes=[])
        n, h, w, c = input_shape
        self.net["buffers"]["input"] = (h, w, c)
        self.tid = 100
        self.w_std = w_std

    def buf(self, name, h, w, pitch):
        if name in self.net["buffers"]:
            assert self.net["buffers"][name] == (h, w, pitch)
        else:
            self.net["buffers"][name] = (h, w, pitch)

    def conv(self, name, src, dst, K, R, S=None, stride=1, pad=None, groups=1, relu=1,
             symmetric=1, residual=None, dst_c_offset=0, dst_pitch=None, C_real=None):
        S = R if S is None else S
        pad = R // 2 if pad is None else pad
        h, w, cp = self.net["buffers"][src]
        C_real = cp if C_real is None else C_real
        p, q = out_size(h, R, stride, pad), out_size(w, S, stride, pad)
        self.buf(dst, p, q, pad16(K) if dst_pitch is None else dst_pitch)
        fan_in = R * S * (C_real // groups)
        w_std = self.w_std if self.w_std is not None else math.sqrt(2.0 / fan_in)
        self.tid += 4
        self.net["nodes"].append(dict(
            name=name, op="conv", src=src, dst=dst, dst_c_offset=dst_c_offset, C=cp, C_real=C_real,
            K=K, R=R, S=S, stride=stride, pad=pad, groups=groups, relu=relu, symmetric=symmetric,
            residual=residual, w_std=w_std, b_std=0.01, tid=self.tid, H=h, W=w, P=p, Q=q))

    def pool(self, name, src, dst, R, stride, pad):
        h, w, cp = self.net["buffers"][src]
        p, q = out_size(h, R, stride, pad), out_size(w, R, stride, pad)
        self.buf(dst, p, q, cp)
        self.net["nodes"].append(dict(name=name, op="maxpool", src=src, dst=dst, R=R, S=R,
                                      stride=stride, pad=pad, H=h, W=w, P=p, Q=q, C=cp))


def single_conv_cfg():
    """The one-layer case: 1x32x32x16 int8 uniform input, 3x3x16x16 int8 uniform
    weights in [R][S][C][K] order, int32 bias uniform in [-2^12, 2^12], stride 1,
    pad 1, right shift 7, ReLU, seed 0.  Integer tensors are drawn directly."""
    g = rng_for(0, 1)
    x = g.integers(-128, 128, size=(1, 32, 32, 16), dtype=np.int8)
    w = rng_for(0, 2).integers(-128, 128, size=(3, 3, 16, 16), dtype=np.int8)
    bias = rng_for(0, 3).integers(-2**12, 2**12 + 1, size=(16,), dtype=np.int32)
    shift = np.full(16, 7, dtype=np.int32)
    return dict(x=x, w=w, bias=bias, shift=shift, R=3, S=3, stride=(1, 1), pad=(1, 1), relu=1,
                weight_layout=1, K=16)


def resnet50(batch=32, res=224, width=64, blocks=(3, 4, 6, 3), stride_on_3x3=False):
    """ResNet-50 shape: 7x7/2 stem, 3x3/2 max-pool, four stages of bottlenecks
    (1x1 reduce, 3x3, 1x1 expand x4) with the stride on the first 1x1 of a stage
    (or, with stride_on_3x3, on the 3x3 layer: the later variant of the network)
    and a 1x1 projection shortcut on the first block; residual added before the
    final ReLU of each block."""
    b = _Builder("resnet50", (batch, res, res, 3), "normal", per_channel=0)
    b.conv("stem", "input", "stem", width, 7, stride=2, pad=3)
    b.pool("pool1", "stem", "s0", 3, 2, 1)
    cur = "s0"
    for si, nb in enumerate(blocks):
        mid = width << si
        out = mid * 4
        for bi in range(nb):
            s = 2 if (bi == 0 and si > 0) else 1
            tag = "s%db%d" % (si, bi)
            b.conv(tag + "_a", cur, tag + "_a", mid, 1, stride=1 if stride_on_3x3 else s, pad=0)
            b.conv(tag + "_b", tag + "_a", tag + "_b", mid, 3, stride=s if stride_on_3x3 else 1)
            if bi == 0:
                b.conv(tag + "_prj", cur, tag + "_prj", out, 1, stride=s, pad=0, relu=0)
                resid = tag + "_prj"
            else:
                resid = cur
            b.conv(tag + "_c", tag + "_b", tag + "_out", out, 1, pad=0, residual=resid)
            cur = tag + "_out"
    return b.net


def vgg16(batch=64, res=224, widths=(64, 128, 256, 512, 512), reps=(2, 2, 3, 3, 3)):
    """VGG-16 convolution shapes: 13 3x3 convs, 2x2/2 max-pool between stages
    (the pool after the last stage is left out: no conv follows it)."""
    b = _Builder("vgg16", (batch, res, res, 3), "halfnormal", per_channel=0, w_std=0.05)
    cur = "input"
    for si, (wd, rp) in enumerate(zip(widths, reps)):
        for ri in range(rp):
            name = "conv%d_%d" % (si + 1, ri + 1)
            b.conv(name, cur, name, wd, 3)
            cur = name
        if si + 1 < len(widths):
            b.pool("pool%d" % (si + 1), cur, "pool%d" % (si + 1), 2, 2, 0)
            cur = "pool%d" % (si + 1)
    return b.net


INCEPTION_BLOCKS = (
    # tag, c1, c3r, c3, c5r, c5, pool-proj
    ("3a", 64, 96, 128, 16, 32, 32),
    ("3b", 128, 128, 192, 32, 96, 64),
    ("pool", 0, 0, 0, 0, 0, 0),
    ("4a", 192, 96, 208, 16, 48, 64),
    ("4b", 160, 112, 224, 24, 64, 64),
    ("4c", 128, 128, 256, 24, 64, 64),
    ("4d", 112, 144, 288, 32, 64, 64),
    ("4e", 256, 160, 320, 32, 128, 128),
    ("5b", 384, 192, 384, 48, 128, 128),
)


def inception(batch=128, res=28, cin=192, blocks=INCEPTION_BLOCKS):
    """GoogLeNet-style inception blocks chained: 3a, 3b at res x res, a 3x3/2
    max-pool, then 4a..4e and the 5b-shaped block at res/2.  Each block has four
    branches (1x1; 1x1 reduce -> 3x3; 1x1 reduce -> 5x5; 3x3/1 max-pool -> 1x1)
    whose int8 outputs are written side by side into one buffer (concat)."""
    b = _Builder("inception", (batch, res, res, cin), "halfnormal", per_channel=0)
    cur = "input"
    for tag, c1, c3r, c3, c5r, c5, pp in blocks:
        if tag == "pool":
            b.pool("pool3", cur, "pool3", 3, 2, 1)
            cur = "pool3"
            continue
        total = c1 + c3 + c5 + pp
        out = "i" + tag
        b.conv(tag + "_3r", cur, tag + "_3r", c3r, 1, pad=0)
        b.conv(tag + "_5r", cur, tag + "_5r", c5r, 1, pad=0)
        b.pool(tag + "_mp", cur, tag + "_mp", 3, 1, 1)
        b.conv(tag + "_1x1", cur, out, c1, 1, pad=0, dst_pitch=total, dst_c_offset=0)
        b.conv(tag + "_3x3", tag + "_3r", out, c3, 3, dst_pitch=total, dst_c_offset=c1, C_real=c3r)
        b.conv(tag + "_5x5", tag + "_5r", out, c5, 5, dst_pitch=total, dst_c_offset=c1 + c3,
               C_real=c5r)
        b.conv(tag + "_pp", tag + "_mp", out, pp, 1, pad=0, dst_pitch=total,
               dst_c_offset=c1 + c3 + c5)
        cur = out
    return b.net


MOBILENET_BLOCKS = ((64, 1), (128, 2), (128, 1), (256, 2), (256, 1), (512, 2), (512, 1), (512, 1),
                    (512, 1), (512, 1), (512, 1), (1024, 2), (1024, 1))


def mobilenet(batch=256, res=224, width=32, blocks=MOBILENET_BLOCKS):
    """MobileNet-v1 shape: 3x3/2 stem, then 13 blocks of a 3x3 depthwise conv
    followed by a 1x1 pointwise conv; widths scale with `width` / 32."""
    b = _Builder("mobilenet", (batch, res, res, 3), "normal", per_channel=1)
    b.conv("stem", "input", "stem", width, 3, stride=2, pad=1)
    cur, c = "stem", width
    for i, (k, s) in enumerate(blocks):
        k = k * width // 32
        b.conv("dw%d" % (i + 1), cur, "dw%d" % (i + 1), c, 3, stride=s, pad=1, groups=c)
        b.conv("pw%d" % (i + 1), "dw%d" % (i + 1), "pw%d" % (i + 1), k, 1, pad=0)
        cur, c = "pw%d" % (i + 1), k
    return b.net


def gen_input(net, seed=0, batch=None):
    """Float input batch [N, H, W, C]: N(0,1), or |N(0,1)| for ReLU-like data."""
    n, h, w, c = net["input"]
    n = n if batch is None else batch
    x = rng_for(seed, 1).standard_normal(size=(n, h, w, c), dtype=np.float32)
    if net["input_dist"] == "halfnormal":
        x = np.abs(x)
    return x


def gen_weights(node, seed=0):
    """Float weights [K, R, S, C/groups] (zero in padded input channels) and bias [K]."""
    K, R, S, C, g = node["K"], node["R"], node["S"], node["C"], node["groups"]
    cg = C // g
    cg_real = node["C_real"] // g if g == 1 else cg
    w = np.zeros((K, R, S, cg), dtype=np.float32)
    w[..., :cg_real] = rng_for(seed, node["tid"]).standard_normal(
        size=(K, R, S, cg_real), dtype=np.float32) * np.float32(node["w_std"])
    bias = rng_for(seed, node["tid"] + 1).standard_normal(size=(K,), dtype=np.float32) \
        * np.float32(node["b_std"])
    return w, bias


def gen_activation_i8(shape, seed, tensor_id, relu_like=True):
    """int8 activations for stand-alone layer cases: round(|N(0,1)| * 32) clipped
    to [0, 127] (ReLU-like) or round(N(0,1) * 32) clipped to [-127, 127]."""
    x = rng_for(seed, tensor_id).standard_normal(size=shape, dtype=np.float32) * np.float32(32.0)
    if relu_like:
        x = np.abs(x)
    return np.clip(np.rint(x), -127, 127).astype(np.int8)


def conv_macs(node, batch):
    return batch * node["P"] * node["Q"] * node["K"] * node["R"] * node["S"] * (node["C_real"] // node["groups"])


def conv_alg_bytes(node, batch):
    """Bytes the layer must move at least: input once, output once, weights,
    bias, and the residual if any (int8 activations, int32 bias)."""
    cin = node["C_real"]
    b = batch * node["H"] * node["W"] * cin + batch * node["P"] * node["Q"] * node["K"]
    b += node["K"] * node["R"] * node["S"] * (cin // node["groups"]) + 4 * node["K"]
    if node.get("residual"):
        b += batch * node["P"] * node["Q"] * node["K"]
    return b
