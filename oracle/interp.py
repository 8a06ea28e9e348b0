"""Reference interpreter for operator graphs (TEST INFRASTRUCTURE, not product).

This is the oracle the CUDA path is checked against.  It executes the
ORIGINAL graph -- unrewritten, unfused -- one operator at a time in
topological order, every intermediate fully materialised as its own fp64
array.  Operator fusion and index rewriting are exact transformations of that
function (paper Section 1: fusion removes materialisation of intermediates;
Section 4.2: rewriting keeps the mathematical function), so the plain
definition of each operator, composed, is what a fused block must reproduce.

It shares no code with the CUDA library and imports nothing from it; only
tests, the smoke check and the CPU-baseline leg of the benchmark may call it.

Operator semantics follow the ONNX vocabulary the paper classifies in Table 2
(Section 3.1).  Operators the paper uses in Table 4 (Recip, Square, Abs,
BitShift, ReduceSum, ReduceProd, Exp) are included so that both sides of each
rewrite identity can be evaluated.

Pinned by tests/test_oracle_*.py against closed forms, invariants and
brute-force index loops; whole-workload outputs have no printed values in the
paper ("parity unpinned" beyond the per-operator pins and composition).
"""
from __future__ import annotations

import math

import numpy as np

_erf = np.vectorize(math.erf, otypes=[np.float64])


def _axis(a, rank):
    return a + rank if a < 0 else a


# ---- One-to-One operators (Table 2, first row) ---------------------------

def op_add(a, b): return a + b            # multidirectional broadcasting (Table 2: elementwise w/ broadcast)
def op_sub(a, b): return a - b
def op_mul(a, b): return a * b
def op_div(a, b): return a / b
def op_mulc(a, c): return a * float(c)
def op_addc(a, c): return a + float(c)
def op_sigmoid(a): return 1.0 / (1.0 + np.exp(-a))
def op_tanh(a): return np.tanh(a)
def op_erf(a): return _erf(a)
def op_exp(a): return np.exp(a)
def op_log(a): return np.log(a)
def op_sqrt(a): return np.sqrt(a)
def op_abs(a): return np.abs(a)
def op_neg(a): return -a
def op_recip(a): return 1.0 / a
def op_square(a): return a * a
def op_relu(a): return np.maximum(a, 0.0)
def op_clip(a, lo, hi): return np.minimum(np.maximum(a, float(lo)), float(hi))
def op_pow(a, p): return np.power(a, float(p))


def op_bitshift(a, bits, direction="left"):
    """Element-wise shift of integer-valued entries (Table 4, Commutative rows)."""
    ai = np.rint(a).astype(np.int64)
    r = ai << int(bits) if direction == "left" else ai >> int(bits)
    return r.astype(np.float64)


def op_gelu(a, approx="erf"):
    if approx == "erf":
        return 0.5 * a * (1.0 + _erf(a / math.sqrt(2.0)))
    k = math.sqrt(2.0 / math.pi)
    return 0.5 * a * (1.0 + np.tanh(k * (a + 0.044715 * a * a * a)))


def op_scaleshift(x, scale, shift, axis=-1):
    """Inference-time BatchNormalization folded to y = x*scale[c] + shift[c] (Table 2: One-to-One)."""
    ax = _axis(axis, x.ndim)
    shp = [1] * x.ndim
    shp[ax] = x.shape[ax]
    return x * scale.reshape(shp) + shift.reshape(shp)


# ---- Reorganize / Shuffle (Table 2; definitions in Section 3.1) -----------

def op_transpose(x, perm):
    """out[i_0..i_{n-1}] = in[j] with j[perm[k]] = i_k  (Shuffle: permutation of the index tuple)."""
    return np.ascontiguousarray(np.transpose(x, tuple(perm)))


def op_reshape(x, shape):
    """Same row-major element order under new dimensions (Reorganize)."""
    return np.ascontiguousarray(x).reshape(tuple(int(s) for s in shape)).copy()


def op_flatten(x, axis=1):
    ax = _axis(axis, x.ndim)
    lead = int(np.prod(x.shape[:ax])) if ax > 0 else 1
    return op_reshape(x, (lead, -1))


def op_squeeze(x, axes):
    axes = sorted(_axis(a, x.ndim) for a in axes)
    shp = [s for i, s in enumerate(x.shape) if i not in axes]
    return op_reshape(x, shp)


def op_unsqueeze(x, axes):
    rank = x.ndim + len(axes)
    axes = sorted(_axis(a, rank) for a in axes)
    shp = list(x.shape)
    for a in axes:
        shp.insert(a, 1)
    return op_reshape(x, shp)


def op_split(x, axis, sizes):
    ax = _axis(axis, x.ndim)
    outs, start = [], 0
    for s in sizes:
        idx = [slice(None)] * x.ndim
        idx[ax] = slice(start, start + int(s))
        outs.append(np.ascontiguousarray(x[tuple(idx)]))
        start += int(s)
    assert start == x.shape[ax]
    return outs


def op_concat(xs, axis):
    return np.concatenate(xs, axis=_axis(axis, xs[0].ndim))


def op_slice(x, axis, start, end):
    ax = _axis(axis, x.ndim)
    idx = [slice(None)] * x.ndim
    idx[ax] = slice(int(start), int(end))
    return np.ascontiguousarray(x[tuple(idx)])


# ---- One-to-Many -----------------------------------------------------------

def op_expand(x, shape):
    return np.ascontiguousarray(np.broadcast_to(x, tuple(int(s) for s in shape)))


def op_depthtospace(x, block):
    """NHWC, depth-column-row order: y[n, h*b+i, w*b+j, c] = x[n, h, w, (i*b+j)*C' + c] with C' = C / b^2
    (Table 2 lists DepthToSpace under Shuffle)."""
    b = int(block)
    n, h, w, c = x.shape
    cp = c // (b * b)
    y = np.zeros((n, h * b, w * b, cp), dtype=np.float64)
    for i in range(b):
        for j in range(b):
            y[:, i::b, j::b, :] = x[:, :, :, (i * b + j) * cp:(i * b + j + 1) * cp]
    return y


def op_spacetodepth(x, block):
    """Inverse of op_depthtospace: y[n, h, w, (i*b+j)*C + c] = x[n, h*b+i, w*b+j, c]."""
    b = int(block)
    n, h, w, c = x.shape
    y = np.zeros((n, h // b, w // b, b * b * c), dtype=np.float64)
    for i in range(b):
        for j in range(b):
            y[:, :, :, (i * b + j) * c:(i * b + j + 1) * c] = x[:, i::b, j::b, :]
    return y


def op_resize_nearest(x, scale):
    """NHWC nearest-neighbour enlargement by an integer factor: y[n, h, w, c] = x[n, h // s, w // s, c]
    (Table 2 lists Resize / Upsample under One-to-Many)."""
    s = int(scale)
    n, h, w, c = x.shape
    hi = np.arange(h * s) // s
    wi = np.arange(w * s) // s
    return x[:, hi][:, :, wi]


def op_gather(x, indices, axis=0):
    return np.take(x, np.rint(indices).astype(np.int64), axis=_axis(axis, x.ndim))


# ---- Many-to-Many (Table 2) ------------------------------------------------

def op_matmul(a, b):
    """C[..., i, j] = sum_k A[..., i, k] * B[..., k, j], leading dims broadcast."""
    return np.matmul(a, b)


def op_conv1x1(x, w):
    """NHWC pointwise convolution: y[n,h,w,o] = sum_c x[n,h,w,c] * W[c,o]."""
    return np.einsum("nhwc,co->nhwo", x, w)


def op_dwconv3x3(x, k):
    """NHWC depthwise 3x3, stride 1, zero padding 1:
    y[n,h,w,c] = sum_{dh,dw in -1..1} x[n,h+dh,w+dw,c] * K[dh+1,dw+1,c]."""
    n, h, w, c = x.shape
    xp = np.zeros((n, h + 2, w + 2, c), dtype=np.float64)
    xp[:, 1:h + 1, 1:w + 1, :] = x
    y = np.zeros_like(x, dtype=np.float64)
    for dh in range(3):
        for dw in range(3):
            y += xp[:, dh:dh + h, dw:dw + w, :] * k[dh, dw, :]
    return y


def _pool(x, kernel, stride, pad, is_max):
    """NHWC pooling window by window: result[n, i, j, c] reduces x[n, i*s-p : i*s-p+k, j*s-p : j*s-p+k, c]
    restricted to the image.  MaxPool takes the maximum of those elements, AveragePool their mean (elements of
    the padding are neither compared nor counted).  Table 2 lists both under Many-to-Many."""
    k, s, p = int(kernel), int(stride), int(pad)
    n, h, w, c = x.shape
    ho, wo = (h + 2 * p - k) // s + 1, (w + 2 * p - k) // s + 1
    y = np.zeros((n, ho, wo, c), dtype=np.float64)
    for i in range(ho):
        for j in range(wo):
            win = x[:, max(i * s - p, 0):min(i * s - p + k, h), max(j * s - p, 0):min(j * s - p + k, w), :]
            y[:, i, j, :] = win.max(axis=(1, 2)) if is_max else win.mean(axis=(1, 2))
    return y


def op_maxpool(x, kernel, stride=1, pad=0): return _pool(x, kernel, stride, pad, True)
def op_avgpool(x, kernel, stride=1, pad=0): return _pool(x, kernel, stride, pad, False)


def op_convtranspose(x, w, stride, pad=0):
    """NHWC transposed convolution, weights [Cin, k, k, Cout]: every input pixel adds its k x k x Cout patch at
    (h*s, w*s): y[n, h*s+i, w*s+j, o] += sum_c x[n,h,w,c] W[c,i,j,o]; `pad` rows and columns are then cut from every
    border (ONNX pads), leaving (H-1)*s + k - 2*pad rows (Table 2 lists ConvTranspose under Many-to-Many)."""
    s, p = int(stride), int(pad)
    n, h, wd, c = x.shape
    _, k, _, co = w.shape
    y = np.zeros((n, (h - 1) * s + k, (wd - 1) * s + k, co), dtype=np.float64)
    for a in range(h):
        for b in range(wd):
            y[:, a * s:a * s + k, b * s:b * s + k, :] += np.einsum("nc,cijo->nijo", x[:, a, b, :], w)
    return y[:, p:y.shape[1] - p, p:y.shape[2] - p, :] if p else y


def op_softmax(x, axis=-1):
    ax = _axis(axis, x.ndim)
    m = np.max(x, axis=ax, keepdims=True)
    e = np.exp(x - m)
    return e / np.sum(e, axis=ax, keepdims=True)


def op_layernorm(x, gamma, beta, axis=-1, eps=1e-5):
    """Biased variance, eps inside the square root, over the last axis."""
    ax = _axis(axis, x.ndim)
    assert ax == x.ndim - 1
    mu = np.mean(x, axis=ax, keepdims=True)
    xc = x - mu
    var = np.mean(xc * xc, axis=ax, keepdims=True)
    return xc / np.sqrt(var + float(eps)) * gamma + beta


def _reduce(fn, x, axis, keepdims):
    return fn(x, axis=_axis(axis, x.ndim), keepdims=bool(keepdims))


def op_reducesum(x, axis=-1, keepdims=1): return _reduce(np.sum, x, axis, keepdims)
def op_reducemean(x, axis=-1, keepdims=1): return _reduce(np.mean, x, axis, keepdims)
def op_reduceprod(x, axis=-1, keepdims=1): return _reduce(np.prod, x, axis, keepdims)
def op_reducemax(x, axis=-1, keepdims=1): return _reduce(np.max, x, axis, keepdims)


# ---- further One-to-One operators of Table 2 ---------------------------------

def op_sin(x): return np.sin(x)
def op_cos(x): return np.cos(x)
def op_asin(x): return np.arcsin(x)
def op_ceil(x): return np.ceil(x)
def op_floor(x): return np.floor(x)
def op_round(x): return np.rint(x)                         # to nearest, ties to even (ONNX Round)
def op_leakyrelu(x, alpha): return np.where(x > 0, x, float(alpha) * x)
def op_not(x): return np.where(x == 0, 1.0, 0.0)           # on 0 / 1 valued tensors
def op_greater(a, b): return np.where(a > b, 1.0, 0.0)     # multidirectional broadcasting
def op_prelu(x, slope): return np.where(x > 0, x, slope * x)


# ---- further Table 2 operators: Where, Cast (One-to-One); CumSum, InstanceNormalization (Many-to-Many) ----

def op_where(cond, a, b):
    """y = a where cond is non-zero, else b; cond is a 0 / 1 valued tensor; multidirectional broadcasting.
    A selection, not arithmetic: an infinity or NaN in the branch that is not taken leaves no trace."""
    return np.where(np.asarray(cond) != 0, a, b)


def _round_to_bf16(x):
    """Nearest bfloat16 (8 significand bits), ties to even, of the fp32 value nearest to x."""
    bits = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    bits = (bits + 0x7FFF + ((bits >> 16) & 1)) & 0xFFFF0000
    return bits.astype(np.uint32).view(np.float32).astype(np.float64)


def op_cast(x, to):
    """ONNX Cast between the value types a graph here can hold.  "f32": unchanged; "bf16": nearest bfloat16, ties to
    even; "i32": the integer toward zero (the float-to-integer conversion); "bool": 1 where x is non-zero, else 0.
    Integer and boolean results stay stored as floating-point numbers with those values."""
    x = np.asarray(x, dtype=np.float64)
    if to == "f32": return x
    if to == "bf16": return _round_to_bf16(x).reshape(x.shape)
    if to == "i32": return np.trunc(x)
    if to == "bool": return np.where(x != 0, 1.0, 0.0)
    raise ValueError(f"Cast: unknown target {to}")


def op_cumsum(x, axis=-1, exclusive=0, reverse=0):
    """ONNX CumSum along `axis`: y[i] = sum of x[j] over j <= i (j < i when exclusive), counted from the far end
    when reverse."""
    x = np.asarray(x, dtype=np.float64)
    ax = _axis(axis, x.ndim)
    if reverse: x = np.flip(x, ax)
    y = np.cumsum(x, axis=ax)
    if exclusive: y = y - x
    if reverse: y = np.flip(y, ax)
    return y


def op_instancenorm(x, scale, bias, eps=1e-5):
    """ONNX InstanceNormalization on an NHWC tensor: every image n and channel c is normalised by the mean and the
    (biased) variance over its own H x W positions, then scaled and shifted per channel."""
    x = np.asarray(x, dtype=np.float64)
    mean = x.mean(axis=(1, 2), keepdims=True)
    var = ((x - mean) ** 2).mean(axis=(1, 2), keepdims=True)
    return (x - mean) / np.sqrt(var + float(eps)) * np.asarray(scale, dtype=np.float64) + np.asarray(bias, dtype=np.float64)


def op_einsum(a, b, equation):
    """ONNX Einsum of two operands in explicit form ("bhqd,bhkd->bhqk"): the sum over the labels that are missing in
    the result of the products of the operands' elements (the library routine is the definition written out)."""
    return np.einsum(equation, np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64))


# ---- dispatcher -------------------------------------------------------------

def _apply(op, ins, at):
    g = at.get
    if op == "Add": return [op_add(*ins)]
    if op == "Sub": return [op_sub(*ins)]
    if op == "Mul": return [op_mul(*ins)]
    if op == "Div": return [op_div(*ins)]
    if op == "MulC": return [op_mulc(ins[0], at["c"])]
    if op == "AddC": return [op_addc(ins[0], at["c"])]
    if op == "Sigmoid": return [op_sigmoid(ins[0])]
    if op == "Tanh": return [op_tanh(ins[0])]
    if op == "Erf": return [op_erf(ins[0])]
    if op == "Exp": return [op_exp(ins[0])]
    if op == "Log": return [op_log(ins[0])]
    if op == "Sqrt": return [op_sqrt(ins[0])]
    if op == "Abs": return [op_abs(ins[0])]
    if op == "Neg": return [op_neg(ins[0])]
    if op == "Recip": return [op_recip(ins[0])]
    if op == "Square": return [op_square(ins[0])]
    if op == "Relu": return [op_relu(ins[0])]
    if op == "Sin": return [op_sin(ins[0])]
    if op == "Cos": return [op_cos(ins[0])]
    if op == "Asin": return [op_asin(ins[0])]
    if op == "Ceil": return [op_ceil(ins[0])]
    if op == "Floor": return [op_floor(ins[0])]
    if op == "Round": return [op_round(ins[0])]
    if op == "LeakyRelu": return [op_leakyrelu(ins[0], g("alpha", g("c", 0.01)))]
    if op == "Not": return [op_not(ins[0])]
    if op == "Greater": return [op_greater(ins[0], ins[1])]
    if op == "PRelu": return [op_prelu(ins[0], ins[1])]
    if op == "Clip": return [op_clip(ins[0], at["lo"], at["hi"])]
    if op == "Pow": return [op_pow(ins[0], at["p"])]
    if op == "BitShift": return [op_bitshift(ins[0], at["bits"], g("direction", "left"))]
    if op == "Gelu": return [op_gelu(ins[0], g("approx", "erf"))]
    if op == "ScaleShift": return [op_scaleshift(ins[0], ins[1], ins[2], g("axis", -1))]
    if op == "Transpose": return [op_transpose(ins[0], at["perm"])]
    if op == "Reshape": return [op_reshape(ins[0], at["shape"])]
    if op == "Flatten": return [op_flatten(ins[0], g("axis", 1))]
    if op == "Squeeze": return [op_squeeze(ins[0], at["axes"])]
    if op == "Unsqueeze": return [op_unsqueeze(ins[0], at["axes"])]
    if op == "Split": return op_split(ins[0], at["axis"], at["sizes"])
    if op == "Concat": return [op_concat(ins, at["axis"])]
    if op == "Slice": return [op_slice(ins[0], at["axis"], at["start"], at["end"])]
    if op == "Expand": return [op_expand(ins[0], at["shape"])]
    if op == "DepthToSpace": return [op_depthtospace(ins[0], at["block"])]
    if op == "SpaceToDepth": return [op_spacetodepth(ins[0], at["block"])]
    if op == "Resize": return [op_resize_nearest(ins[0], at["scale"])]
    if op == "Gather": return [op_gather(ins[0], ins[1], g("axis", 0))]
    if op == "MatMul": return [op_matmul(ins[0], ins[1])]
    if op == "Conv1x1": return [op_conv1x1(ins[0], ins[1])]
    if op == "DwConv3x3": return [op_dwconv3x3(ins[0], ins[1])]
    if op == "MaxPool": return [op_maxpool(ins[0], at["kernel"], g("stride", 1), g("pad", 0))]
    if op == "AveragePool": return [op_avgpool(ins[0], at["kernel"], g("stride", 1), g("pad", 0))]
    if op == "ConvTranspose": return [op_convtranspose(ins[0], ins[1], g("stride", at["kernel"]), g("pad", 0))]
    if op == "Softmax": return [op_softmax(ins[0], g("axis", -1))]
    if op == "LayerNorm": return [op_layernorm(ins[0], ins[1], ins[2], g("axis", -1), g("eps", 1e-5))]
    if op == "ReduceSum": return [op_reducesum(ins[0], g("axis", -1), g("keepdims", 1))]
    if op == "ReduceMean": return [op_reducemean(ins[0], g("axis", -1), g("keepdims", 1))]
    if op == "ReduceProd": return [op_reduceprod(ins[0], g("axis", -1), g("keepdims", 1))]
    if op == "ReduceMax": return [op_reducemax(ins[0], g("axis", -1), g("keepdims", 1))]
    if op == "Where": return [op_where(ins[0], ins[1], ins[2])]
    if op == "Cast": return [op_cast(ins[0], at["to"])]
    if op == "CumSum": return [op_cumsum(ins[0], g("axis", -1), g("exclusive", 0), g("reverse", 0))]
    if op == "Einsum": return [op_einsum(ins[0], ins[1], at["equation"])]
    if op == "InstanceNorm": return [op_instancenorm(ins[0], ins[1], ins[2], g("eps", 1e-5))]
    raise KeyError(f"oracle: unknown operator {op}")


def run_graph(graph, inputs, keep_all=False):
    """Evaluate `graph` (an object with .ops, .outputs; each op has .op, .inputs,
    .outputs, .attrs) on `inputs` (name -> array).  Returns name -> fp64 array
    for the marked outputs (or every tensor when keep_all)."""
    env = {k: np.asarray(v, dtype=np.float64) for k, v in inputs.items()}
    for o in graph.ops:
        ins = [env[n] for n in o.inputs]
        outs = _apply(o.op, ins, o.attrs)
        assert len(outs) == len(o.outputs), (o.op, len(outs), len(o.outputs))
        for n, v in zip(o.outputs, outs):
            env[n] = np.asarray(v, dtype=np.float64)
    if keep_all:
        return env
    return {n: env[n] for n in graph.outputs}
