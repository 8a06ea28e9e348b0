"""Randomised shapes for the contraction-anchored kernels: bf16 GEMM blocks (both tensor-core kernels, split-K, ragged
edges in M, N and K, both layouts of B, random epilogues), fp32 tall-and-skinny GEMM blocks (split-TF32 kernel) and
fp32 NHWC depthwise / pointwise convolutions, each against the oracle with NaN-poisoned outputs."""
import numpy as np
import pytest

from paper_2108_13342_b200 import binding as B
from paper_2108_13342_b200 import workloads as W
from paper_2108_13342_b200.runtime import Session
from oracle import interp as O
from util import RTOL_BF16, RTOL_F32, close, graph, rnd

pytestmark = pytest.mark.gpu


def _u(seed, i):
    return float(W.uniform(31337 + seed, i, (1,), 0.0, 1.0)[0])


def _pick(seed, i, xs):
    return xs[min(int(_u(seed, i) * len(xs)), len(xs) - 1)]


def _run(wl, rtol, plan_flags=B.PLAN_FUSED):
    ref = O.run_graph(wl.graph, wl.inputs)
    s = Session(wl, plan_flags=plan_flags, rewrite_flags=B.REWRITE_NONE)
    s.workspace[s.g.workspace_zero_bytes():].fill_(0xFF)
    for n in wl.graph.outputs:
        s.buffers[n].fill_(float("nan"))
    for _ in range(2):                      # twice: split-K counters must be back at zero
        s.run()
        assert s.g.status()[0] == 0
        for n in wl.graph.outputs:
            got = s.output(n)
            assert np.isfinite(got).all(), (n, s.g.blocks())
            try:
                close(got, ref[n], rtol)
            except AssertionError as e:
                raise AssertionError(f"{[(b['family'], b['variant'], b['grid']) for b in s.g.blocks()]}: {e}") from None
    return s


def _bf(a):
    return W.round_to_bf16(a)


@pytest.mark.parametrize("seed", range(160))
def test_random_bf16_gemm(seed):
    m = _pick(seed, 1, [1, 7, 64, 129, 256, 300, 512, 777, 1024, 1500])
    n = 8 * (1 + int(_u(seed, 2) * 90))
    k = 8 * (1 + int(_u(seed, 3) * _pick(seed, 4, [8, 40, 300])))
    epi = _pick(seed, 5, ["none", "bias", "bias_gelu", "bias_residual", "bias_relu_f32out"])
    kmajor = _u(seed, 6) < 0.4
    g = graph()
    g.ext("A", (m, k), "bf16")
    ins = {"A": _bf(rnd((m, k), 31, -1, 1))}
    if kmajor:
        g.ext("Bt", (n, k), "bf16"); ins["Bt"] = _bf(rnd((n, k), 32, -0.1, 0.1))
        b = g.add("Transpose", ["Bt"], perm=(1, 0))
    else:
        g.ext("Bm", (k, n), "bf16"); ins["Bm"] = _bf(rnd((k, n), 32, -0.1, 0.1)); b = "Bm"
    t = g.add("MatMul", ["A", b])
    if epi != "none":
        g.ext("bias", (n,), "f32"); ins["bias"] = rnd((n,), 33, -0.5, 0.5)
        t = g.add("Add", [t, "bias"])
    if epi == "bias_gelu":
        t = g.add("Gelu", [t], approx="tanh")
    if epi == "bias_residual":
        g.ext("R", (m, n), "bf16"); ins["R"] = _bf(rnd((m, n), 34, -1, 1))
        t = g.add("Add", [t, "R"])
    if epi == "bias_relu_f32out":
        g.ext("S", (m, n), "f32"); ins["S"] = rnd((m, n), 35, -1, 1)
        t = g.add("Add", [g.add("Relu", [t]), "S"])         # fp32 operand: the block's output is fp32
    g.mark_output(t)
    _run(W.Workload(g, ins), RTOL_BF16)


@pytest.mark.parametrize("seed", range(120))
def test_random_fp32_tall_skinny_gemm(seed):
    m = 512 + int(_u(seed, 1) * 4000)
    k = 4 * (1 + int(_u(seed, 2) * 59))
    n = 4 * (1 + int(_u(seed, 3) * 47))
    epi = _pick(seed, 4, ["none", "scale_shift_clip", "bias_residual", "two_outputs"])
    g = graph()
    g.ext("X", (m, k)); g.ext("Wm", (k, n)); g.ext("s", (n,)); g.ext("t", (n,))
    ins = {"X": rnd((m, k), 41, -1, 1), "Wm": rnd((k, n), 42, -0.5, 0.5), "s": rnd((n,), 43, 0.5, 1.5), "t": rnd((n,), 44, -0.5, 0.5)}
    y = g.add("MatMul", ["X", "Wm"])
    if epi == "scale_shift_clip":
        y = g.add("Clip", [g.add("ScaleShift", [y, "s", "t"], axis=-1)], lo=-1.0, hi=2.0)
    elif epi == "bias_residual":
        g.ext("R", (m, n)); ins["R"] = rnd((m, n), 45, -1, 1)
        y = g.add("Add", [g.add("Add", [y, "t"]), "R"])
    elif epi == "two_outputs":
        y = g.add("Add", [y, "t"], out="Z")
        g.mark_output(y)
        y = g.add("Tanh", [y])
    g.mark_output(y)
    _run(W.Workload(g, ins), RTOL_F32)


@pytest.mark.parametrize("seed", range(100))
def test_random_depthwise_and_pointwise_conv(seed):
    n = _pick(seed, 1, [1, 2, 5, 16, 40])
    h = 4 + int(_u(seed, 2) * 40)
    w = 4 + int(_u(seed, 3) * 40)
    c = 4 * (1 + int(_u(seed, 4) * _pick(seed, 5, [6, 36, 90])))
    co = 4 * (1 + int(_u(seed, 6) * 40))
    g = graph()
    g.ext("X", (n, h, w, c)); g.ext("Kd", (3, 3, c)); g.ext("s", (c,)); g.ext("t", (c,)); g.ext("Wp", (c, co)); g.ext("u", (co,))
    ins = {"X": rnd((n, h, w, c), 51, -1, 1), "Kd": rnd((3, 3, c), 52, -0.5, 0.5), "s": rnd((c,), 53, 0.5, 1.5), "t": rnd((c,), 54, -0.5, 0.5),
           "Wp": rnd((c, co), 55, -0.3, 0.3), "u": rnd((co,), 56, -0.5, 0.5)}
    e = g.add("DwConv3x3", ["X", "Kd"])
    e = g.add("Clip", [g.add("ScaleShift", [e, "s", "t"], axis=-1)], lo=0.0, hi=6.0)
    y = g.add("Conv1x1", [e, "Wp"])
    g.mark_output(g.add("Add", [y, "u"], out="Y"))
    _run(W.Workload(g, ins), RTOL_F32)


@pytest.mark.parametrize("seed", range(60))
def test_random_deep_pointwise_conv(seed):
    """Channel counts beyond what the split-TF32 kernel takes in one pass (K up to 1024): the planner's K slices, with
    slice counts 2-8 or none when K has no suitable divisor, and three kinds of epilogue."""
    # most of these sizes are below the planner's break-even for a split
    plan_flags = B.PLAN_FUSED | (B.PLAN_SPLIT_ALWAYS if seed % 3 else 0)
    n = _pick(seed, 1, [1, 2, 3])
    h = 8 + int(_u(seed, 2) * 40)
    w = 8 + int(_u(seed, 3) * 40)
    c = 4 * (62 + int(_u(seed, 4) * 195))             # 248 .. 1024
    co = 4 * (1 + int(_u(seed, 6) * (47 if seed % 2 else 120)))     # 4 .. 188, or up to 480 (column blocks as well)
    g = graph()
    g.ext("X", (n, h, w, c)); g.ext("Wp", (c, co)); g.ext("s", (co,)); g.ext("t", (co,)); g.ext("R", (n, h, w, co))
    ins = {"X": rnd((n, h, w, c), 61, -1, 1), "Wp": rnd((c, co), 62, -0.1, 0.1), "s": rnd((co,), 63, 0.5, 1.5),
           "t": rnd((co,), 64, -0.5, 0.5), "R": rnd((n, h, w, co), 65, -1, 1)}
    y = g.add("Conv1x1", ["X", "Wp"])
    kind = _pick(seed, 7, ["bias", "bn_clip", "bn_res", "plain"])
    if kind == "bias": y = g.add("Add", [y, "t"])
    elif kind == "bn_clip": y = g.add("Clip", [g.add("ScaleShift", [y, "s", "t"], axis=-1)], lo=-1.0, hi=1.0)
    elif kind == "bn_res": y = g.add("Add", [g.add("ScaleShift", [y, "s", "t"], axis=-1), "R"])
    g.mark_output(y)
    _run(W.Workload(g, ins), 2e-5, plan_flags)


@pytest.mark.parametrize("seed", range(40))
def test_random_attention(seed):
    """Q, K, V sliced out of one packed [B, S, 3*H*D] tensor, heads split by Reshape + Transpose, scores scaled and
    masked, Softmax, P*V stored back to [B, S, H*D]: all index operators fold into operand strides of the two batched
    GEMM blocks."""
    import math
    bsz = _pick(seed, 1, [1, 2, 3, 5])
    s = _pick(seed, 2, [16, 32, 48, 100, 128, 200])
    h = _pick(seed, 3, [1, 2, 3, 12])
    d = _pick(seed, 4, [16, 32, 64, 128])
    qkv = _bf(rnd((bsz, s, 3 * h * d), 5, -1, 1))
    g = graph()
    g.ext("QKV", qkv.shape, "bf16"); g.ext("mask", (s, s), "f32")
    q, k, v = g.add("Split", ["QKV"], n_out=3, axis=-1, sizes=(h * d,) * 3)
    hs = []
    for t in (q, k, v):
        t = g.add("Reshape", [t], shape=(bsz, s, h, d))
        hs.append(g.add("Transpose", [t], perm=(0, 2, 1, 3)))
    q, k, v = hs
    kt = g.add("Transpose", [k], perm=(0, 1, 3, 2))
    sc = g.add("MatMul", [q, kt])
    sc = g.add("MulC", [sc], c=1.0 / math.sqrt(d))
    sc = g.add("Add", [sc, "mask"])
    p = g.add("Softmax", [sc], axis=-1)
    a = g.add("MatMul", [p, v])
    a = g.add("Transpose", [a], perm=(0, 2, 1, 3))
    a = g.add("Reshape", [a], shape=(bsz, s, h * d), out="O")
    g.mark_output(a)
    _run(W.Workload(g, {"QKV": qkv, "mask": W.causal_mask(s)}), RTOL_BF16)
