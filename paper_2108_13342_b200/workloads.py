"""Seeded synthetic workloads: graph descriptions and input tensors.

This module serves both the CUDA path and the test oracle.  It holds no
arithmetic of the fusion method itself: it only (a) describes operator graphs
as plain data (operator name, input names, output names, attributes) and
(b) draws seeded input values.  Neither the oracle nor the CUDA library is
imported here.

Random values come from a counter-based generator, value_i = f(seed, tensor
index, i), so a tensor's contents do not depend on the order tensors are drawn
in or on how many other tensors exist.

The five workloads follow the evaluation families of the paper (Section 5:
CNN blocks, transformer encoders) at the shapes of the MobileNet/EfficientNet
and BERT-base rows of its Tables 5 and 6; the trained models themselves are
replaced by random weights of the same shapes.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

BASE_SEED = 20210620

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def _splitmix64(x: np.ndarray) -> np.ndarray:
    """Avalanche hash of a uint64 counter (wrap-around arithmetic)."""
    with np.errstate(over="ignore"):
        x = (x + np.uint64(0x9E3779B97F4A7C15)) & _M64
        z = x
        z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _M64
        z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _M64
        return z ^ (z >> np.uint64(31))


def _counter_bits(seed: int, tensor_index: int, n: int, lane: int) -> np.ndarray:
    with np.errstate(over="ignore"):
        key = _splitmix64(np.array([seed * 1000003 + tensor_index * 7919 + lane * 104729],
                                   dtype=np.uint64))[0]
        ctr = np.arange(n, dtype=np.uint64)
        return _splitmix64(ctr ^ key)


def uniform01(seed: int, tensor_index: int, n: int, lane: int = 0) -> np.ndarray:
    """n doubles in [0, 1) with 24 random bits each."""
    bits = _counter_bits(seed, tensor_index, n, lane) >> np.uint64(40)
    return bits.astype(np.float64) / float(1 << 24)


def uniform(seed, tensor_index, shape, lo, hi) -> np.ndarray:
    n = int(np.prod(shape))
    u = uniform01(seed, tensor_index, n)
    return (lo + (hi - lo) * u).astype(np.float32).reshape(shape)


def normal(seed, tensor_index, shape, mean, std) -> np.ndarray:
    """Box-Muller in double on two independent counter streams."""
    n = int(np.prod(shape))
    u1 = uniform01(seed, tensor_index, n, lane=1)
    u2 = uniform01(seed, tensor_index, n, lane=2)
    u1 = (u1 * float(1 << 24) + 1.0) / float((1 << 24) + 1)   # (0, 1): log stays finite
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * math.pi * u2)
    return (mean + std * z).astype(np.float32).reshape(shape)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); result kept as fp32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    b = x.view(np.uint32).astype(np.uint64)
    lsb = (b >> np.uint64(16)) & np.uint64(1)
    b = (b + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return b.astype(np.uint32).view(np.float32).reshape(x.shape)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 storage of values that are already bf16-representable."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> np.uint32(16)).astype(np.uint16).reshape(x.shape)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).reshape(b.shape)


# --------------------------------------------------------------------------
# Graph description (plain data)
# --------------------------------------------------------------------------

@dataclass
class TensorDesc:
    name: str
    shape: tuple
    dtype: str          # "f32" | "bf16"
    kind: str           # "input" | "weight"


@dataclass
class OpDesc:
    op: str
    inputs: list
    outputs: list
    attrs: dict = field(default_factory=dict)


@dataclass
class GraphDesc:
    """Operators in topological order plus the external tensors they read."""
    name: str = ""
    tensors: dict = field(default_factory=dict)     # name -> TensorDesc (externals only)
    ops: list = field(default_factory=list)
    outputs: list = field(default_factory=list)
    _n: int = 0

    def ext(self, name, shape, dtype="f32", kind="input"):
        self.tensors[name] = TensorDesc(name, tuple(int(s) for s in shape), dtype, kind)
        return name

    def add(self, op, inputs, n_out=1, out=None, **attrs):
        if out is None:
            outs = []
            for _ in range(n_out):
                self._n += 1
                outs.append(f"%{self._n}")
        else:
            outs = [out] if isinstance(out, str) else list(out)
        self.ops.append(OpDesc(op, list(inputs), outs, dict(attrs)))
        return outs[0] if len(outs) == 1 else outs

    def mark_output(self, name):
        self.outputs.append(name)
        return name


@dataclass
class Workload:
    graph: GraphDesc
    inputs: dict        # name -> fp32 ndarray (bf16 tensors hold bf16-representable values)
    note: str = ""


class _Draw:
    """Hands out tensor indices in declaration order."""

    def __init__(self, seed):
        self.seed = seed
        self.idx = 0

    def _next(self):
        self.idx += 1
        return self.idx

    def uniform(self, shape, lo, hi):
        return uniform(self.seed, self._next(), shape, lo, hi)

    def normal(self, shape, mean, std):
        return normal(self.seed, self._next(), shape, mean, std)


def causal_mask(s: int) -> np.ndarray:
    """M[i, j] = 0 for j <= i, -1e9 above the diagonal."""
    i = np.arange(s)[:, None]
    j = np.arange(s)[None, :]
    return np.where(j <= i, 0.0, -1e9).astype(np.float32)


# --------------------------------------------------------------------------
# Workload 1: bias + scale + swish + NCHW->NHWC transpose
# --------------------------------------------------------------------------

def swish_transpose(n=1, c=64, h=56, w=56, seed=BASE_SEED) -> Workload:
    d = _Draw(seed)
    g = GraphDesc("swish_transpose")
    g.ext("X", (n, c, h, w))
    g.ext("b", (1, c, 1, 1), kind="weight")
    t = g.add("Add", ["X", "b"])
    t = g.add("MulC", [t], c=0.5)
    s = g.add("Sigmoid", [t])
    y = g.add("Mul", [t, s])
    o = g.add("Transpose", [y], perm=(0, 2, 3, 1), out="Y")
    g.mark_output(o)
    inputs = {"X": d.uniform((n, c, h, w), -1.0, 1.0),
              "b": d.uniform((1, c, 1, 1), -0.5, 0.5)}
    return Workload(g, inputs)


# --------------------------------------------------------------------------
# Workload 2a: scale + causal mask + softmax ; 2b: residual + LayerNorm + GELU
# --------------------------------------------------------------------------

def masked_softmax(batch=8, heads=12, s=128, seed=BASE_SEED) -> Workload:
    d = _Draw(seed + 1)
    g = GraphDesc("masked_softmax")
    g.ext("S", (batch, heads, s, s))
    g.ext("M", (s, s), kind="weight")
    t = g.add("MulC", ["S"], c=1.0 / math.sqrt(64.0))
    t = g.add("Add", [t, "M"])
    o = g.add("Softmax", [t], axis=-1, out="P")
    g.mark_output(o)
    inputs = {"S": d.normal((batch, heads, s, s), 0.0, 1.0), "M": causal_mask(s)}
    return Workload(g, inputs)


def add_layernorm_gelu(rows=1024, hidden=768, seed=BASE_SEED) -> Workload:
    d = _Draw(seed + 2)
    g = GraphDesc("add_layernorm_gelu")
    g.ext("H", (rows, hidden))
    g.ext("R", (rows, hidden))
    g.ext("gamma", (hidden,), kind="weight")
    g.ext("beta", (hidden,), kind="weight")
    z = g.add("Add", ["H", "R"])
    y = g.add("LayerNorm", [z, "gamma", "beta"], axis=-1, eps=1e-5)
    o = g.add("Gelu", [y], approx="erf", out="Y")
    g.mark_output(o)
    inputs = {"H": d.normal((rows, hidden), 0.0, 1.0),
              "R": d.normal((rows, hidden), 0.0, 1.0),
              "gamma": d.normal((hidden,), 1.0, 0.02),
              "beta": d.normal((hidden,), 0.0, 0.02)}
    return Workload(g, inputs)


# --------------------------------------------------------------------------
# Workload 3: GEMM + bias + GELU(tanh) ; GEMM + bias + residual   (bf16)
# --------------------------------------------------------------------------

def ffn_block(m=4096, hidden=768, ffn=3072, seed=BASE_SEED) -> Workload:
    d = _Draw(seed + 3)
    g = GraphDesc("ffn_block")
    g.ext("A", (m, hidden), "bf16")
    g.ext("W1", (hidden, ffn), "bf16", kind="weight")
    g.ext("b1", (ffn,), "f32", kind="weight")
    g.ext("W2", (ffn, hidden), "bf16", kind="weight")
    g.ext("b2", (hidden,), "f32", kind="weight")
    t = g.add("MatMul", ["A", "W1"])
    t = g.add("Add", [t, "b1"])
    t = g.add("Gelu", [t], approx="tanh")
    t = g.add("MatMul", [t, "W2"])
    t = g.add("Add", [t, "b2"])
    o = g.add("Add", [t, "A"], out="Y")
    g.mark_output(o)
    inputs = {"A": round_to_bf16(d.normal((m, hidden), 0.0, 1.0)),
              "W1": round_to_bf16(d.normal((hidden, ffn), 0.0, 0.02)),
              "b1": d.normal((ffn,), 0.0, 0.02),
              "W2": round_to_bf16(d.normal((ffn, hidden), 0.0, 0.02)),
              "b2": d.normal((hidden,), 0.0, 0.02)}
    return Workload(g, inputs)


# --------------------------------------------------------------------------
# Workload 4: MobileNetV2-style inverted residual block, fp32 NHWC
# --------------------------------------------------------------------------

def mbconv_block(n=32, h=56, w=56, cin=24, cexp=144, seed=BASE_SEED) -> Workload:
    d = _Draw(seed + 4)
    g = GraphDesc("mbconv_block")
    g.ext("X", (n, h, w, cin))
    g.ext("W1", (cin, cexp), kind="weight")
    g.ext("s1", (cexp,), kind="weight"); g.ext("t1", (cexp,), kind="weight")
    g.ext("Kd", (3, 3, cexp), kind="weight")
    g.ext("s2", (cexp,), kind="weight"); g.ext("t2", (cexp,), kind="weight")
    g.ext("W3", (cexp, cin), kind="weight")
    g.ext("s3", (cin,), kind="weight"); g.ext("t3", (cin,), kind="weight")
    e = g.add("Conv1x1", ["X", "W1"])
    e = g.add("ScaleShift", [e, "s1", "t1"], axis=-1)
    e = g.add("Clip", [e], lo=0.0, hi=6.0)
    e = g.add("DwConv3x3", [e, "Kd"])
    e = g.add("ScaleShift", [e, "s2", "t2"], axis=-1)
    e = g.add("Clip", [e], lo=0.0, hi=6.0)
    e = g.add("Conv1x1", [e, "W3"])
    e = g.add("ScaleShift", [e, "s3", "t3"], axis=-1)
    o = g.add("Add", [e, "X"], out="Y")
    g.mark_output(o)
    inputs = {"X": d.uniform((n, h, w, cin), 0.0, 1.0),
              "W1": d.normal((cin, cexp), 0.0, math.sqrt(2.0 / cin)),
              "s1": d.uniform((cexp,), 0.5, 1.5), "t1": d.uniform((cexp,), -0.5, 0.5),
              "Kd": d.normal((3, 3, cexp), 0.0, math.sqrt(2.0 / 9.0)),
              "s2": d.uniform((cexp,), 0.5, 1.5), "t2": d.uniform((cexp,), -0.5, 0.5),
              "W3": d.normal((cexp, cin), 0.0, math.sqrt(2.0 / cexp)),
              "s3": d.uniform((cin,), 0.5, 1.5), "t3": d.uniform((cin,), -0.5, 0.5)}
    return Workload(g, inputs)


def cnn_neck(n=8, h=64, w=64, c=32, seed=BASE_SEED) -> Workload:
    """A detection-style feature-pyramid fragment in NHWC fp32 that uses the rest of Table 2's operator set
    around the convolution blocks: a pointwise stem, MaxPool and SpaceToDepth downsampling, nearest-neighbour
    Resize and DepthToSpace upsampling, channel Concat with skip connections, a global AveragePool gate.
    Synthetic shapes in the range of the paper's mobile CNNs (Section 5: 224-416 pixel inputs, stride 4-8 maps)."""
    d = _Draw(seed + 9)
    g = GraphDesc("cnn_neck")
    ins = {}

    def ext(name, shape, lo=None, hi=None, std=None):
        g.ext(name, shape, kind="input" if name == "X" else "weight")
        ins[name] = d.normal(shape, 0.0, std) if std is not None else d.uniform(shape, lo, hi)
        return name

    def conv_bn_relu6(x, cin, cout, tag):
        wn = ext("W" + tag, (cin, cout), std=math.sqrt(2.0 / cin))
        sn = ext("s" + tag, (cout,), 0.5, 1.5); tn = ext("t" + tag, (cout,), -0.5, 0.5)
        e = g.add("Conv1x1", [x, wn])
        e = g.add("ScaleShift", [e, sn, tn], axis=-1)
        return g.add("Clip", [e], lo=0.0, hi=6.0)

    ext("X", (n, h, w, c), 0.0, 1.0)
    stem = conv_bn_relu6("X", c, 2 * c, "0")                              # [n, h, w, 2c]
    p1 = g.add("MaxPool", [stem], kernel=3, stride=2, pad=1)              # [n, h/2, w/2, 2c]
    s2d = g.add("SpaceToDepth", [stem], block=2)                          # [n, h/2, w/2, 8c]
    lat = conv_bn_relu6(s2d, 8 * c, 2 * c, "1")                           # [n, h/2, w/2, 2c]
    mid = g.add("Concat", [p1, lat], axis=3)                              # [n, h/2, w/2, 4c]
    kd = ext("Kd", (3, 3, 4 * c), std=math.sqrt(2.0 / 9.0))
    sd = ext("sd", (4 * c,), 0.5, 1.5); td = ext("td", (4 * c,), -0.5, 0.5)
    dw = g.add("DwConv3x3", [mid, kd])
    dw = g.add("ScaleShift", [dw, sd, td], axis=-1)
    dw = g.add("Clip", [dw], lo=0.0, hi=6.0)                              # [n, h/2, w/2, 4c]
    # squeeze-and-excitation style gate from a global average pool
    gap = g.add("AveragePool", [dw], kernel=h // 2, stride=1, pad=0)      # [n, 1, 1, 4c]
    wg = ext("Wg", (4 * c, 4 * c), std=math.sqrt(1.0 / (4 * c)))
    gate = g.add("Sigmoid", [g.add("Conv1x1", [gap, wg])])                # [n, 1, 1, 4c]
    gated = g.add("Mul", [dw, gate])                                      # broadcast over the image
    up_a = g.add("DepthToSpace", [gated], block=2)                        # [n, h, w, c]
    up_b = g.add("Resize", [conv_bn_relu6(gated, 4 * c, c, "2")], scale=2)   # [n, h, w, c]
    top = g.add("Concat", [up_a, up_b, "X"], axis=3)                      # [n, h, w, 3c]
    y = conv_bn_relu6(top, 3 * c, c, "3")
    y = g.add("Add", [y, "X"], out="Y")
    g.mark_output(y)
    return Workload(g, ins, note="fp32 NHWC")


def mbconv_stack(n=32, hw=56, seed=BASE_SEED, layout="nhwc") -> Workload:
    """A MobileNetV2-shaped stack of inverted-residual blocks in NHWC fp32 (expand 1x1 + BN + ReLU6, depthwise 3x3 + BN +
    ReLU6, project 1x1 + BN, residual where the shapes agree) with the channel progression 16-24-32-64-96-160 and
    expansion 6, MaxPool 3x3 / 2 between the stages (the library's depthwise kernel has stride 1), a 1x1 head, global
    average pool and a classifier: the convolution side of the paper's model zoo (Section 5) as one synthetic graph.
    Expansions beyond 192 channels and projections deeper than 244 exercise the planner's column-block and K splits.

    layout="nchw" describes the same network the way a channels-first exporter writes it: the image X and every
    feature map are [n, c, h, w], batch normalisation scales axis 1, ReLU6 and the residual Add act on channels-first
    tensors, and each operator the library defines channels-last only (the convolutions and the pools) sits between a
    Transpose to NHWC and a Transpose back.  The values are those of the NHWC graph with X transposed (same seeds), so
    the logits agree: the case for inter-block layout selection (Section 4.4.2)."""
    if layout not in ("nhwc", "nchw"):
        raise ValueError("layout is 'nhwc' or 'nchw'")
    cf = layout == "nchw"
    d = _Draw(seed + 11)
    g = GraphDesc("mbconv_stack" + ("_nchw" if cf else ""))
    ins = {}
    cnt = [0]

    def ext(shape, lo=None, hi=None, std=None, name=None):
        cnt[0] += 1
        name = name or "p%d" % cnt[0]
        g.ext(name, shape, kind="input" if name == "X" else "weight")
        ins[name] = d.normal(shape, 0.0, std) if std is not None else d.uniform(shape, lo, hi)
        return name

    def bn(x, c):
        return g.add("ScaleShift", [x, ext((c,), 0.5, 1.5), ext((c,), -0.5, 0.5)], axis=1 if cf else -1)

    def channels_last(kind, ins, **attrs):
        """An operator the library defines on NHWC tensors; in the channels-first graph it is wrapped in Transposes."""
        if not cf:
            return g.add(kind, ins, **attrs)
        y = g.add(kind, [g.add("Transpose", [ins[0]], perm=(0, 2, 3, 1))] + list(ins[1:]), **attrs)
        return g.add("Transpose", [y], perm=(0, 3, 1, 2))

    def block(x, cin, cout, t=6):
        e = cin * t
        y = g.add("Clip", [bn(channels_last("Conv1x1", [x, ext((cin, e), std=math.sqrt(2.0 / cin))]), e)], lo=0.0, hi=6.0)
        y = g.add("Clip", [bn(channels_last("DwConv3x3", [y, ext((3, 3, e), std=math.sqrt(2.0 / 9.0))]), e)], lo=0.0, hi=6.0)
        y = bn(channels_last("Conv1x1", [y, ext((e, cout), std=math.sqrt(1.0 / e))]), cout)
        return g.add("Add", [y, x]) if cin == cout else y

    x = ext((n, 16, hw, hw) if cf else (n, hw, hw, 16), 0.0, 1.0, name="X")
    if cf:
        ins["X"] = np.ascontiguousarray(ins["X"].reshape(n, hw, hw, 16).transpose(0, 3, 1, 2))
    x = block(x, 16, 24); x = block(x, 24, 24)
    x = channels_last("MaxPool", [x], kernel=3, stride=2, pad=1)
    x = block(x, 24, 32); x = block(x, 32, 32); x = block(x, 32, 64)
    x = channels_last("MaxPool", [x], kernel=3, stride=2, pad=1)
    x = block(x, 64, 64); x = block(x, 64, 96); x = block(x, 96, 96); x = block(x, 96, 160)
    x = g.add("Clip", [bn(channels_last("Conv1x1", [x, ext((160, 320), std=math.sqrt(2.0 / 160))]), 320)], lo=0.0, hi=6.0)
    x = channels_last("AveragePool", [x], kernel=hw // 4, stride=1, pad=0)                 # [n, 1, 1, 320] (NHWC)
    if cf:
        x = g.add("Transpose", [x], perm=(0, 2, 3, 1))
    x = g.add("Add", [g.add("Conv1x1", [x, ext((320, 100), std=math.sqrt(1.0 / 320))]), ext((100,), -0.1, 0.1)], out="logits")
    g.mark_output(x)
    return Workload(g, ins, note="fp32 " + layout.upper())


def style_decoder(n=8, hw=64, c=64, seed=BASE_SEED) -> Workload:
    """The decoder half of a style-transfer / image-to-image generator in NHWC fp32: a residual block (pointwise
    convolution, instance normalisation, ReLU, depthwise 3x3, instance normalisation, skip), two transposed
    convolutions with overlapping patches (kernel 4, stride 2, pad 1: each doubles the image) with instance
    normalisation and ReLU, and a pointwise convolution to 4 output channels with Tanh.  Synthetic shapes in the range of
    the paper's image-to-image models (Section 5); it exercises InstanceNormalization and ConvTranspose at sizes where
    they dominate."""
    d = _Draw(seed + 13)
    g = GraphDesc("style_decoder")
    ins = {}
    cnt = [0]

    def ext(shape, lo=None, hi=None, std=None, name=None):
        cnt[0] += 1
        name = name or "p%d" % cnt[0]
        g.ext(name, shape, kind="input" if name == "X" else "weight")
        ins[name] = d.normal(shape, 0.0, std) if std is not None else d.uniform(shape, lo, hi)
        return name

    def inorm(x, ch):
        return g.add("InstanceNorm", [x, ext((ch,), 0.5, 1.5), ext((ch,), -0.5, 0.5)], eps=1e-5)

    x = ext((n, hw, hw, c), -1.0, 1.0, name="X")
    y = g.add("Relu", [inorm(g.add("Conv1x1", [x, ext((c, c), std=math.sqrt(2.0 / c))]), c)])
    y = inorm(g.add("DwConv3x3", [y, ext((3, 3, c), std=math.sqrt(2.0 / 9.0))]), c)
    y = g.add("Add", [y, x])
    ch = c
    for _ in range(2):
        y = g.add("ConvTranspose", [y, ext((ch, 4, 4, ch // 2), std=math.sqrt(2.0 / (4 * ch)))], kernel=4, stride=2, pad=1)
        ch //= 2
        y = g.add("Relu", [inorm(y, ch)])
    y = g.add("Tanh", [g.add("Add", [g.add("Conv1x1", [y, ext((ch, 4), std=math.sqrt(1.0 / ch))]), ext((4,), -0.1, 0.1)])], out="image")
    g.mark_output(y)
    return Workload(g, ins, note="fp32 NHWC")


# --------------------------------------------------------------------------
# Workload 5: transformer encoder as primitive operators (48 per layer)
# --------------------------------------------------------------------------

def _layernorm_primitives(g, x, gamma, beta, eps):
    mu = g.add("ReduceMean", [x], axis=-1, keepdims=1)
    xc = g.add("Sub", [x, mu])
    sq = g.add("Pow", [xc], p=2.0)
    var = g.add("ReduceMean", [sq], axis=-1, keepdims=1)
    ve = g.add("AddC", [var], c=eps)
    sd = g.add("Sqrt", [ve])
    xn = g.add("Div", [xc, sd])
    xs = g.add("Mul", [xn, gamma])
    return g.add("Add", [xs, beta])


def _gelu_erf_primitives(g, x):
    t = g.add("MulC", [x], c=1.0 / math.sqrt(2.0))
    t = g.add("Erf", [t])
    t = g.add("AddC", [t], c=1.0)
    t = g.add("Mul", [x, t])
    return g.add("MulC", [t], c=0.5)


def encoder(layers=12, batch=8, seq=128, hidden=768, heads=12, ffn=3072,
            seed=BASE_SEED) -> Workload:
    d = _Draw(seed + 5)
    hd = hidden // heads
    g = GraphDesc("encoder")
    inputs = {}

    def ext(name, shape, dtype, kind, arr):
        g.ext(name, shape, dtype, kind)
        inputs[name] = round_to_bf16(arr) if dtype == "bf16" else arr
        return name

    x = ext("x", (batch, seq, hidden), "bf16", "input", d.normal((batch, seq, hidden), 0.0, 1.0))
    ext("mask", (seq, seq), "f32", "weight", causal_mask(seq))
    for l in range(layers):
        p = f"L{l}."
        wqkv = ext(p + "Wqkv", (hidden, 3 * hidden), "bf16", "weight", d.normal((hidden, 3 * hidden), 0.0, 0.02))
        bqkv = ext(p + "bqkv", (3 * hidden,), "f32", "weight", d.normal((3 * hidden,), 0.0, 0.02))
        wo = ext(p + "Wo", (hidden, hidden), "bf16", "weight", d.normal((hidden, hidden), 0.0, 0.02))
        bo = ext(p + "bo", (hidden,), "f32", "weight", d.normal((hidden,), 0.0, 0.02))
        g1 = ext(p + "ln1.g", (hidden,), "f32", "weight", d.normal((hidden,), 1.0, 0.02))
        be1 = ext(p + "ln1.b", (hidden,), "f32", "weight", d.normal((hidden,), 0.0, 0.02))
        w1 = ext(p + "W1", (hidden, ffn), "bf16", "weight", d.normal((hidden, ffn), 0.0, 0.02))
        b1 = ext(p + "b1", (ffn,), "f32", "weight", d.normal((ffn,), 0.0, 0.02))
        w2 = ext(p + "W2", (ffn, hidden), "bf16", "weight", d.normal((ffn, hidden), 0.0, 0.02))
        b2 = ext(p + "b2", (hidden,), "f32", "weight", d.normal((hidden,), 0.0, 0.02))
        g2 = ext(p + "ln2.g", (hidden,), "f32", "weight", d.normal((hidden,), 1.0, 0.02))
        be2 = ext(p + "ln2.b", (hidden,), "f32", "weight", d.normal((hidden,), 0.0, 0.02))

        qkv = g.add("MatMul", [x, wqkv])
        qkv = g.add("Add", [qkv, bqkv])
        q, k, v = g.add("Split", [qkv], n_out=3, axis=-1, sizes=(hidden, hidden, hidden))
        hs = []
        for t in (q, k, v):
            t = g.add("Reshape", [t], shape=(batch, seq, heads, hd))
            hs.append(g.add("Transpose", [t], perm=(0, 2, 1, 3)))
        q, k, v = hs
        kt = g.add("Transpose", [k], perm=(0, 1, 3, 2))
        s = g.add("MatMul", [q, kt])
        s = g.add("MulC", [s], c=1.0 / math.sqrt(hd))
        s = g.add("Add", [s, "mask"])
        pr = g.add("Softmax", [s], axis=-1)
        a = g.add("MatMul", [pr, v])
        a = g.add("Transpose", [a], perm=(0, 2, 1, 3))
        a = g.add("Reshape", [a], shape=(batch, seq, hidden))
        o = g.add("MatMul", [a, wo])
        o = g.add("Add", [o, bo])
        o = g.add("Add", [o, x])
        x1 = _layernorm_primitives(g, o, g1, be1, 1e-5)
        f = g.add("MatMul", [x1, w1])
        f = g.add("Add", [f, b1])
        f = _gelu_erf_primitives(g, f)
        f = g.add("MatMul", [f, w2])
        f = g.add("Add", [f, b2])
        f = g.add("Add", [f, x1])
        x = _layernorm_primitives(g, f, g2, be2, 1e-5)
    g.mark_output(x)
    return Workload(g, inputs)


# --------------------------------------------------------------------------
# Workload 6: GPT-2 style decoder as primitive operators (pre-LayerNorm blocks, causal attention,
# GELU in its tanh form spelled out; 53 operators per layer plus a final LayerNorm)
# --------------------------------------------------------------------------

def _gelu_tanh_primitives(g, x):
    x2 = g.add("Mul", [x, x])
    x3 = g.add("Mul", [x2, x])
    t = g.add("MulC", [x3], c=0.044715)
    t = g.add("Add", [x, t])
    t = g.add("MulC", [t], c=math.sqrt(2.0 / math.pi))
    t = g.add("Tanh", [t])
    t = g.add("AddC", [t], c=1.0)
    t = g.add("Mul", [x, t])
    return g.add("MulC", [t], c=0.5)


def decoder(layers=12, batch=8, seq=128, hidden=768, heads=12, ffn=3072, seed=BASE_SEED) -> Workload:
    d = _Draw(seed + 6)
    hd = hidden // heads
    g = GraphDesc("decoder")
    inputs = {}

    def ext(name, shape, dtype, kind, arr):
        g.ext(name, shape, dtype, kind)
        inputs[name] = round_to_bf16(arr) if dtype == "bf16" else arr
        return name

    def vec(name, n, mean):
        return ext(name, (n,), "f32", "weight", d.normal((n,), mean, 0.02))

    x = ext("x", (batch, seq, hidden), "bf16", "input", d.normal((batch, seq, hidden), 0.0, 1.0))
    ext("mask", (seq, seq), "f32", "weight", causal_mask(seq))
    for l in range(layers):
        p = f"L{l}."
        g1, be1 = vec(p + "ln1.g", hidden, 1.0), vec(p + "ln1.b", hidden, 0.0)
        wqkv = ext(p + "Wqkv", (hidden, 3 * hidden), "bf16", "weight", d.normal((hidden, 3 * hidden), 0.0, 0.02))
        bqkv = vec(p + "bqkv", 3 * hidden, 0.0)
        wo = ext(p + "Wo", (hidden, hidden), "bf16", "weight", d.normal((hidden, hidden), 0.0, 0.02))
        bo = vec(p + "bo", hidden, 0.0)
        g2, be2 = vec(p + "ln2.g", hidden, 1.0), vec(p + "ln2.b", hidden, 0.0)
        w1 = ext(p + "W1", (hidden, ffn), "bf16", "weight", d.normal((hidden, ffn), 0.0, 0.02))
        b1 = vec(p + "b1", ffn, 0.0)
        w2 = ext(p + "W2", (ffn, hidden), "bf16", "weight", d.normal((ffn, hidden), 0.0, 0.02))
        b2 = vec(p + "b2", hidden, 0.0)

        h1 = _layernorm_primitives(g, x, g1, be1, 1e-5)
        qkv = g.add("MatMul", [h1, wqkv])
        qkv = g.add("Add", [qkv, bqkv])
        q, k, v = g.add("Split", [qkv], n_out=3, axis=-1, sizes=(hidden, hidden, hidden))
        hs = []
        for t in (q, k, v):
            t = g.add("Reshape", [t], shape=(batch, seq, heads, hd))
            hs.append(g.add("Transpose", [t], perm=(0, 2, 1, 3)))
        q, k, v = hs
        kt = g.add("Transpose", [k], perm=(0, 1, 3, 2))
        s = g.add("MatMul", [q, kt])
        s = g.add("MulC", [s], c=1.0 / math.sqrt(hd))
        s = g.add("Add", [s, "mask"])
        pr = g.add("Softmax", [s], axis=-1)
        a = g.add("MatMul", [pr, v])
        a = g.add("Transpose", [a], perm=(0, 2, 1, 3))
        a = g.add("Reshape", [a], shape=(batch, seq, hidden))
        o = g.add("MatMul", [a, wo])
        o = g.add("Add", [o, bo])
        x = g.add("Add", [x, o])
        h2 = _layernorm_primitives(g, x, g2, be2, 1e-5)
        f = g.add("MatMul", [h2, w1])
        f = g.add("Add", [f, b1])
        f = _gelu_tanh_primitives(g, f)
        f = g.add("MatMul", [f, w2])
        f = g.add("Add", [f, b2])
        x = g.add("Add", [x, f])
    gf, bf = vec("lnf.g", hidden, 1.0), vec("lnf.b", hidden, 0.0)
    x = _layernorm_primitives(g, x, gf, bf, 1e-5)
    g.mark_output(x)
    return Workload(g, inputs)


def by_name(name: str, **kw) -> Workload:
    table = {"swish_transpose": swish_transpose, "masked_softmax": masked_softmax,
             "add_layernorm_gelu": add_layernorm_gelu, "ffn_block": ffn_block,
             "mbconv_block": mbconv_block, "encoder": encoder, "decoder": decoder, "cnn_neck": cnn_neck,
             "mbconv_stack": mbconv_stack, "style_decoder": style_decoder}
    return table[name](**kw)
