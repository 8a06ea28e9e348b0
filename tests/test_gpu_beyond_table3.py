"""Fusions that Table 3 forbids (Many-to-Many followed by Many-to-Many), formed only under DNNF_PLAN_BEYOND_TABLE3:
the attention head MatMul -> scale -> + mask -> Softmax -> MatMul as ONE kernel, against the oracle and against the
three-block plan of the paper's rules."""
import math

import numpy as np
import pytest

from paper_2108_13342_b200 import binding as B
from paper_2108_13342_b200 import workloads as W
from util import RTOL_BF16, RTOL_F32, check, close, graph, rnd, run_both

pytestmark = pytest.mark.gpu
BEYOND = B.PLAN_FUSED | B.PLAN_BEYOND_TABLE3


def _bf(x):
    return W.round_to_bf16(x)


def _attention(bsz, sq, h, d, scale=True, mask="causal", seed=5, amp=None):
    # without the 1 / sqrt(d) factor the inputs are drawn smaller, so that the scores stay of order one and the
    # bf16 scores of the three-block plan remain inside the tolerance
    amp = amp if amp is not None else (1.0 if scale else 0.4)
    qkv = _bf(rnd((bsz, sq, 3 * h * d), seed, -amp, amp))
    g = graph()
    g.ext("QKV", qkv.shape, "bf16")
    ins = {"QKV": qkv}
    q, k, v = g.add("Split", ["QKV"], n_out=3, axis=-1, sizes=(h * d,) * 3)
    hs = []
    for t in (q, k, v):
        t = g.add("Reshape", [t], shape=(bsz, sq, h, d))
        hs.append(g.add("Transpose", [t], perm=(0, 2, 1, 3)))
    q, k, v = hs
    sc = g.add("MatMul", [q, g.add("Transpose", [k], perm=(0, 1, 3, 2))])
    if scale:
        sc = g.add("MulC", [sc], c=1.0 / math.sqrt(d))
    if mask == "causal":
        g.ext("mask", (sq, sq), "f32"); ins["mask"] = W.causal_mask(sq)
        sc = g.add("Add", [sc, "mask"])
    elif mask == "per_batch":                       # a padding mask: one row of key biases per batch element
        g.ext("mask", (bsz, 1, 1, sq), "f32")
        m = np.zeros((bsz, 1, 1, sq), np.float32)
        for b in range(bsz):
            m[b, 0, 0, sq - 1 - 3 * b:] = -1e9
        ins["mask"] = m
        sc = g.add("Add", [sc, "mask"])
    p = g.add("Softmax", [sc], axis=-1)
    a = g.add("MatMul", [p, v])
    a = g.add("Transpose", [a], perm=(0, 2, 1, 3))
    a = g.add("Reshape", [a], shape=(bsz, sq, h * d), out="O")
    g.mark_output(a)
    return W.Workload(g, ins)


@pytest.mark.parametrize("cfg", [(8, 128, 12, 64), (2, 32, 3, 64), (1, 100, 2, 64), (3, 200, 2, 64), (2, 256, 1, 64), (2, 128, 2, 128),
                                 (1, 48, 5, 128), (2, 300, 2, 64)])
@pytest.mark.parametrize("scale,mask", [(True, "causal"), (False, None), (True, "per_batch"), (False, "causal")])
def test_attention_head_in_one_kernel(cfg, scale, mask):
    """The first case is the encoder's shape: 8 sequences of 128 tokens, 12 heads of 64.  Key counts that are not a
    multiple of the MMA's granularity, several query tiles, heads of 128.  300 keys are too many for the single-kernel
    form and 100 keys leave the rows of the probabilities unaligned for TMA: those graphs keep the blocks of the
    normal plan."""
    bsz, sq, h, d = cfg
    wl = _attention(bsz, sq, h, d, scale, mask)
    s, got, ref = run_both(wl, BEYOND)
    close(got["O"], ref["O"], RTOL_BF16)
    fams = [b["family"] for b in s.g.blocks() if b["family"] != "alias"]
    if sq <= 256 and sq % 8 == 0:
        assert fams[0] == "attention" and "gemm" not in fams and "row" not in fams, s.g.blocks()
    else:
        assert fams[:3] == ["gemm", "row", "gemm"], s.g.blocks()
    # a second run on the same buffers, and the plan of the paper's rules beside it
    s.buffers["O"].fill_(float("nan"))
    s.run()
    close(s.output("O"), ref["O"], RTOL_BF16)
    assert s.g.status() == (0, -1)
    three, got3, _ = run_both(wl, B.PLAN_FUSED)
    assert [b["family"] for b in three.g.blocks() if b["family"] != "alias"][:3] == ["gemm", "row", "gemm"]
    close(got3["O"], ref["O"], RTOL_BF16)


def test_single_kernel_keeps_fp32_scores():
    """The plan of the paper's rules rounds the scores to bf16 between its blocks.  Unscaled scores of magnitude 9 then
    carry an absolute error of 0.03 into the exponentials and that plan leaves the tolerance; the single kernel holds
    the scores as fp32 in tensor memory and stays inside it."""
    wl = _attention(8, 128, 12, 64, scale=False, mask=None, amp=1.0)
    s, got, ref = run_both(wl, BEYOND)
    close(got["O"], ref["O"], RTOL_BF16)
    _, got3, _ = run_both(wl, B.PLAN_FUSED)
    e1 = np.abs(got["O"] - ref["O"]).max(); e3 = np.abs(got3["O"] - ref["O"]).max()
    assert e1 < 0.25 * e3, (e1, e3)


def test_one_hot_rows():
    """Row 0 of a causal mask attends to one key: its probability is exactly 1 and the output row is V's first row."""
    bsz, sq, h, d = 1, 64, 1, 64
    wl = _attention(bsz, sq, h, d, True, "causal")
    s, got, ref = run_both(wl, BEYOND)
    assert [b["family"] for b in s.g.blocks() if b["family"] != "alias"][0] == "attention"
    close(got["O"], ref["O"], RTOL_BF16)
    v = wl.inputs["QKV"][0, :, 2 * h * d:]
    assert np.array_equal(got["O"][0, 0], v[0])


@pytest.mark.parametrize("which", ["encoder", "decoder"])
def test_whole_graphs_with_single_kernel_attention(which):
    wl = W.encoder(layers=2, batch=2, seq=32, hidden=128, heads=2, ffn=256) if which == "encoder" else \
        W.decoder(layers=2, batch=2, seq=32, hidden=128, heads=2, ffn=256)
    s, got, ref = run_both(wl, BEYOND, B.REWRITE_CANON_MACRO)
    (name,) = wl.graph.outputs
    close(got[name], ref[name], RTOL_BF16)
    fams = [b["family"] for b in s.g.blocks()]
    assert fams.count("attention") == 2, fams
    base = check(wl, RTOL_BF16, B.PLAN_FUSED, B.REWRITE_CANON_MACRO)
    assert s.plan_stats.n_kernels == base.plan_stats.n_kernels - 4


def test_encoder_full_size_one_layer_with_single_kernel_attention():
    wl = W.encoder(layers=1)
    s, got, ref = run_both(wl, BEYOND, B.REWRITE_CANON_MACRO)
    (name,) = wl.graph.outputs
    close(got[name], ref[name], RTOL_BF16)
    assert s.plan_stats.n_kernels == 7


# ---- the inverted-residual block as one kernel ---------------------------------------------------------------------------

def _families(s):
    return [b["family"] for b in s.g.blocks() if b["family"] != "alias"]


@pytest.mark.parametrize("cfg", [(1, 8, 16, 24, 144), (2, 14, 14, 24, 144), (3, 19, 23, 24, 144), (1, 56, 56, 24, 144), (2, 9, 33, 24, 48),
                                 (1, 17, 18, 24, 96), (2, 7, 5, 24, 144), (1, 2, 3, 24, 48), (5, 3, 70, 24, 96)])
def test_inverted_residual_block_as_one_kernel(cfg):
    """Expansion, depthwise filter and projection with their batch-norm / ReLU6 / residual chains in one kernel: same values
    as the oracle at the tolerance of fp32 blocks, on tiles that are ragged in both directions, image borders inside and
    outside a tile, one to several tiles per image."""
    n, h, w, cin, cexp = cfg
    wl = W.mbconv_block(n, h, w, cin, cexp)
    s = check(wl, RTOL_F32, BEYOND | B.PLAN_MBCONV_ALWAYS, expect_blocks=1)
    assert _families(s) == ["mbconv"]
    # the paper's rules keep three kernels
    assert len(_families(check(wl, RTOL_F32, B.PLAN_FUSED, expect_blocks=3))) == 3


def test_inverted_residual_block_full_size():
    """32 images are 896 tiles, six waves: the planner keeps the three kernels unless told otherwise (they are faster
    there); the single kernel is checked on the full size all the same."""
    s = check(W.mbconv_block(), RTOL_F32, BEYOND | B.PLAN_MBCONV_ALWAYS, expect_blocks=1)
    assert _families(s) == ["mbconv"] and s.g.blocks()[0]["grid"] == 148
    s = check(W.mbconv_block(), RTOL_F32, BEYOND, expect_blocks=3)
    assert "mbconv" not in _families(s)
    s = check(W.mbconv_block(n=1), RTOL_F32, BEYOND, expect_blocks=1)       # one image: 28 tiles
    assert _families(s) == ["mbconv"]
    s = check(W.mbconv_block(n=1, h=14, w=14), RTOL_F32, BEYOND, expect_blocks=3)       # two tiles: not worth the set-up
    assert "mbconv" not in _families(s)
    s = check(W.mbconv_block(n=1, h=14, w=14), RTOL_F32, BEYOND | B.PLAN_MBCONV_ALWAYS, expect_blocks=1)
    assert _families(s) == ["mbconv"]


@pytest.mark.parametrize("cout,tail,act", [(32, "none", "clip"), (24, "relu", "relu"), (32, "two_outputs", "clip"), (24, "pixel_gate", "leaky")])
def test_inverted_residual_block_other_chains(cout, tail, act):
    """Chains without a compile-time table (interpreted), a projection without residual, onto 32 channels, with two
    outputs, with an operand that depends on the pixel only."""
    n, h, w, ce = 2, 21, 19, 96
    cin = {"none": 16, "two_outputs": 40}.get(tail, 24)           # 40 input channels: a K with an 8-wide tail
    g = graph("mb"); ins = {}

    def ext(name, shape, lo, hi, seed, kind="weight"):
        g.ext(name, shape, kind=kind); ins[name] = rnd(shape, seed, lo, hi); return name

    def activation(x):
        if act == "clip": return g.add("Clip", [x], lo=0.0, hi=6.0)
        if act == "relu": return g.add("Relu", [x])
        return g.add("LeakyRelu", [x], alpha=0.1)

    ext("X", (n, h, w, cin), 0.0, 1.0, 1, kind="input")
    e = g.add("Conv1x1", ["X", ext("W1", (cin, ce), -0.3, 0.3, 2)])
    e = activation(g.add("ScaleShift", [e, ext("s1", (ce,), 0.5, 1.5, 3), ext("t1", (ce,), -0.5, 0.5, 4)], axis=-1))
    e = g.add("DwConv3x3", [e, ext("Kd", (3, 3, ce), -0.5, 0.5, 5)])
    e = activation(g.add("Add", [e, ext("b2", (ce,), -0.5, 0.5, 6)]))
    e = g.add("Conv1x1", [e, ext("W3", (ce, cout), -0.2, 0.2, 7)])
    e = g.add("ScaleShift", [e, ext("s3", (cout,), 0.5, 1.5, 8), ext("t3", (cout,), -0.5, 0.5, 9)], axis=-1)
    if tail == "relu":
        e = g.add("Relu", [g.add("Add", [e, "X"])])
    elif tail == "two_outputs":
        g.mark_output(e)
        e = g.add("Sigmoid", [e])
    elif tail == "pixel_gate":
        e = g.add("Mul", [g.add("Add", [e, "X"]), ext("P", (n, h, w, 1), 0.5, 1.5, 10, kind="input")])
    g.mark_output(e)
    s = check(W.Workload(g, ins), RTOL_F32, BEYOND | B.PLAN_MBCONV_ALWAYS, expect_blocks=1)       # (12 tiles: below the planner's own bar)
    assert _families(s) == ["mbconv"]


def test_inverted_residual_blocks_that_stay_three_kernels():
    # the expanded tensor is also a graph output; an operand behind the expansion depends on the pixel
    wl = W.mbconv_block(2, 12, 12, 24, 48)
    wl.graph.mark_output(wl.graph.ops[2].outputs[0])                      # the first ReLU6
    s = check(wl, RTOL_F32, BEYOND)
    assert "mbconv" not in _families(s)
    g = graph("mb2"); n, h, w = 1, 10, 10
    g.ext("X", (n, h, w, 24)); g.ext("W1", (24, 48), kind="weight"); g.ext("Kd", (3, 3, 48), kind="weight"); g.ext("W3", (48, 24), kind="weight")
    g.ext("R", (n, h, w, 48))
    e = g.add("Add", [g.add("Conv1x1", ["X", "W1"]), "R"])
    g.mark_output(g.add("Conv1x1", [g.add("Relu", [g.add("DwConv3x3", [e, "Kd"])]), "W3"]))
    ins = {"X": rnd((n, h, w, 24), 1), "W1": rnd((24, 48), 2, -0.3, 0.3), "Kd": rnd((3, 3, 48), 3, -0.5, 0.5), "W3": rnd((48, 24), 4, -0.3, 0.3),
           "R": rnd((n, h, w, 48), 5)}
    s = check(W.Workload(g, ins), RTOL_F32, BEYOND)
    assert "mbconv" not in _families(s)


def test_mobilenet_stack_with_single_kernel_blocks():
    """The MobileNetV2-shaped stack: the inverted-residual blocks whose channel counts fit run as one kernel each, the others
    keep the three kernels of the paper's rules; same logits as the oracle."""
    wl = W.mbconv_stack(n=4, hw=48)
    s = check(wl, 5e-4, BEYOND | B.PLAN_MBCONV_ALWAYS, B.REWRITE_DEFAULT)
    fams = _families(s)
    assert fams.count("mbconv") >= 2, fams
