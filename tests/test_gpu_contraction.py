"""Parity of contraction-anchored blocks (GEMM / pointwise convolution with fused
epilogues, strided operands, permuted stores) with the oracle."""
import numpy as np
import pytest

from paper_2108_13342_b200 import binding as B
from paper_2108_13342_b200 import workloads as W
from util import RTOL_BF16, RTOL_F32, check, close, graph, rnd, run_both

pytestmark = pytest.mark.gpu
FUSED, UNFUSED = B.PLAN_FUSED, B.PLAN_UNFUSED



def _expect_variant(sess, variant):
    """The block must run on the named kernel variant."""
    ok = variant if isinstance(variant, tuple) else (variant,)
    assert sess.g.blocks()[0]["variant"] in ok, sess.g.blocks()

def _bf(x):
    return W.round_to_bf16(x)


@pytest.mark.parametrize("mnk", [(128, 128, 64), (256, 256, 256), (1, 17, 8), (129, 257, 72), (17, 129, 264), (300, 40, 1024),
                                 (512, 768, 768)])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_plain_matmul(mnk, dtype):
    m, n, k = mnk
    a, b = rnd((m, k), 1, -1, 1), rnd((k, n), 2, -1, 1)
    if dtype == "bf16":
        a, b = _bf(a), _bf(b)
    g = graph()
    g.ext("A", (m, k), dtype); g.ext("B", (k, n), dtype)
    g.mark_output(g.add("MatMul", ["A", "B"], out="C"))
    check(W.Workload(g, {"A": a, "B": b}), RTOL_BF16 if dtype == "bf16" else 1e-4)


@pytest.mark.parametrize("cfg", [(256, 64, 128), (129, 72, 136), (512, 768, 3072), (4096, 768, 3072)])
@pytest.mark.parametrize("flags", [FUSED, UNFUSED])
def test_ffn_block(cfg, flags):
    """The last case is the GEMM-anchored configuration at its stated size: 192 and 96 output tiles, i.e. every
    CTA pair of the persistent kernel works through several tiles (accumulator stages alternate across tiles,
    the bias vector is re-staged and the residual tile prefetched per work item)."""
    m, hidden, ffn = cfg
    s = check(W.ffn_block(m, hidden, ffn), RTOL_BF16, flags, expect_blocks=2 if flags == FUSED else 6)
    if flags == FUSED:
        assert [b["family"] for b in s.g.blocks()] == ["gemm", "gemm"]
        assert all(b["variant"] in (1, 3, 5) for b in s.g.blocks()), "expected a tensor-core kernel"


@pytest.mark.parametrize("mnk", [(256, 128, 64), (300, 200, 72), (1000, 328, 264), (257, 136, 8), (512, 2304, 768), (512, 128, 448)])
@pytest.mark.parametrize("kmajor_b", [False, True])
@pytest.mark.parametrize("epi", ["none", "bias_gelu", "bias_residual"])
@pytest.mark.parametrize("kernel", ["pair", "tile"])
def test_pair_gemm_shapes_and_epilogues(mnk, kmajor_b, epi, kernel):
    """The CTA-pair kernel (M >= 256, N >= 128) and the one-tile-per-CTA kernel, which the planner prefers at these
    sizes: ragged edges in M, N and K, both operand layouts for B."""
    m, n, k = mnk
    g = graph()
    g.ext("A", (m, k), "bf16")
    ins = {"A": _bf(rnd((m, k), 31, -1, 1))}
    if kmajor_b:
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
    g.mark_output(t)
    s = check(W.Workload(g, ins), RTOL_BF16, FUSED | (B.PLAN_NO_TILE_GEMM if kernel == "pair" else 0), expect_blocks=1)
    _expect_variant(s, 3 if kernel == "pair" else 5)


@pytest.mark.parametrize("mnk", [(4000, 3000, 776), (2304, 2304, 264), (2500, 1104, 264), (8192, 1024, 128), (5000, 1544, 72)])
@pytest.mark.parametrize("epi", ["none", "bias_gelu", "bias_residual"])
def test_pair_gemm_more_tiles_than_cta_pairs(mnk, epi):
    """More work items than the machine has CTA pairs (and than it has SMs), ragged in M, N and K: the persistent
    loop over work items, with every epilogue.  Two runs on the same buffers."""
    m, n, k = mnk
    g = graph()
    g.ext("A", (m, k), "bf16"); g.ext("Bm", (k, n), "bf16")
    ins = {"A": _bf(rnd((m, k), 51, -1, 1)), "Bm": _bf(rnd((k, n), 52, -0.1, 0.1))}
    t = g.add("MatMul", ["A", "Bm"])
    if epi != "none":
        g.ext("bias", (n,), "f32"); ins["bias"] = rnd((n,), 53, -0.5, 0.5)
        t = g.add("Add", [t, "bias"])
    if epi == "bias_gelu":
        t = g.add("Gelu", [t], approx="tanh")
    if epi == "bias_residual":
        g.ext("R", (m, n), "bf16"); ins["R"] = _bf(rnd((m, n), 54, -1, 1))
        t = g.add("Add", [t, "R"])
    g.mark_output(t)
    wl = W.Workload(g, ins)
    s, got, ref = run_both(wl, FUSED | B.PLAN_NO_TILE_GEMM)
    (name,) = wl.graph.outputs
    close(got[name], ref[name], RTOL_BF16)
    _expect_variant(s, 3)
    s.buffers[name].fill_(float("nan"))
    s.run()
    close(s.output(name), ref[name], RTOL_BF16)
    assert s.g.status()[0] == 0


def _gemm_with_epilogue(m, n, k, epi, seed0):
    g = graph()
    g.ext("A", (m, k), "bf16"); g.ext("Bm", (k, n), "bf16")
    ins = {"A": _bf(rnd((m, k), seed0, -1, 1)), "Bm": _bf(rnd((k, n), seed0 + 1, -0.1, 0.1))}
    t = g.add("MatMul", ["A", "Bm"])
    if epi != "none":
        g.ext("bias", (n,), "f32"); ins["bias"] = rnd((n,), seed0 + 2, -0.5, 0.5)
        t = g.add("Add", [t, "bias"])
    if epi == "bias_gelu":
        t = g.add("Gelu", [t], approx="tanh")
    if epi == "bias_residual":
        g.ext("R", (m, n), "bf16"); ins["R"] = _bf(rnd((m, n), seed0 + 3, -1, 1))
        t = g.add("Add", [t, "R"])
    g.mark_output(t)
    return W.Workload(g, ins)


@pytest.mark.parametrize("mnk", [(512, 128, 2048), (256, 256, 2304), (1024, 768, 3072), (300, 136, 2120), (512, 384, 2056)])
@pytest.mark.parametrize("epi", ["none", "bias_gelu", "bias_residual"])
def test_pair_gemm_split_k(mnk, epi):
    """Few output tiles and a long K: several CTA pairs share a tile (split-K through the workspace).  Three runs in a row
    on the same workspace: the arrival counters must come back to zero by themselves."""
    m, n, k = mnk
    wl = _gemm_with_epilogue(m, n, k, epi, 41)
    s, got, ref = run_both(wl, FUSED | B.PLAN_NO_TILE_GEMM)
    (name,) = wl.graph.outputs
    close(got[name], ref[name], RTOL_BF16)
    assert s.g.blocks()[0]["variant"] == 3 and s.g.workspace_zero_bytes() > 256, (s.g.blocks(), s.g.workspace_zero_bytes())
    for _ in range(2):
        s.run()
        close(s.output(name), ref[name], RTOL_BF16)
        assert s.g.status()[0] == 0


@pytest.mark.parametrize("mnk", [(512, 128, 2048), (256, 256, 2304), (1024, 768, 3072), (1024, 768, 768), (1024, 2304, 768), (300, 136, 2120),
                                 (512, 384, 2056), (129, 72, 1032), (1000, 200, 392), (128, 128, 832)])
@pytest.mark.parametrize("epi", ["none", "bias_gelu", "bias_residual"])
def test_tile_gemm_cluster_split_k(mnk, epi):
    """The one-tile-per-CTA kernel with a cluster of 2 or 4 CTAs per tile (an option: measured slower than no split): each takes a range of the k-tiles, the partial
    sums meet through distributed shared memory and every CTA finishes its own column slice.  Ragged M, N and K, a
    last CTA with fewer k-tiles than the others, both cluster sizes, every epilogue; nothing goes through the
    workspace."""
    m, n, k = mnk
    wl = _gemm_with_epilogue(m, n, k, epi, 71)
    s, got, ref = run_both(wl, FUSED | B.PLAN_CLUSTER_SPLIT_K)
    (name,) = wl.graph.outputs
    close(got[name], ref[name], RTOL_BF16)
    b = s.g.blocks()[0]
    tiles = -(-m // 128) * -(-n // (128 if n > 64 else 64))
    assert b["variant"] == 5 and b["grid"] in (2 * tiles, 4 * tiles) and s.g.workspace_zero_bytes() == 256, (b, tiles)
    s.buffers[name].fill_(float("nan"))
    s.run()
    close(s.output(name), ref[name], RTOL_BF16)
    assert s.g.status() == (0, -1)
    # the same block without the split
    s1, got1, _ = run_both(wl, FUSED | B.PLAN_CLUSTER_SPLIT_K | B.PLAN_NO_SPLIT_K)
    assert s1.g.blocks()[0]["variant"] == 5 and s1.g.blocks()[0]["grid"] == tiles
    close(got1[name], ref[name], RTOL_BF16)


def test_batched_matmul_with_transposed_and_strided_operands():
    # scores = (Q K^T) * scale + mask with Q, K sliced out of one [B,S,3*H*D] tensor -- all index
    # operators fold into operand strides; P V is stored straight into [B,S,H*D]
    bsz, s, h, d = 2, 32, 3, 16
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
    sc = g.add("MulC", [sc], c=0.25)
    sc = g.add("Add", [sc, "mask"])
    p = g.add("Softmax", [sc], axis=-1)
    a = g.add("MatMul", [p, v])
    a = g.add("Transpose", [a], perm=(0, 2, 1, 3))
    a = g.add("Reshape", [a], shape=(bsz, s, h * d), out="O")
    g.mark_output(a)
    wl = W.Workload(g, {"QKV": qkv, "mask": W.causal_mask(s)})
    sess = check(wl, RTOL_BF16, FUSED, expect_blocks=3)
    assert [b["family"] for b in sess.g.blocks()] == ["gemm", "row", "gemm"]
    check(wl, RTOL_BF16, UNFUSED)


def test_matmul_broadcast_weight_over_batch_and_f32_epilogue_operands():
    x = _bf(rnd((3, 40, 64), 7, -1, 1)); w = _bf(rnd((64, 48), 8, -0.2, 0.2))
    g = graph()
    g.ext("X", x.shape, "bf16"); g.ext("Wt", w.shape, "bf16", kind="weight"); g.ext("b", (48,), "f32"); g.ext("R", (3, 40, 48), "bf16")
    t = g.add("MatMul", ["X", "Wt"])
    t = g.add("Add", [t, "b"])
    t = g.add("Relu", [t])
    g.mark_output(g.add("Add", [t, "R"], out="Y"))
    check(W.Workload(g, {"X": x, "Wt": w, "b": rnd((48,), 9), "R": _bf(rnd((3, 40, 48), 10))}), RTOL_BF16, FUSED, expect_blocks=1)


@pytest.mark.parametrize("cfg", [(1, 5, 6, 24, 144), (2, 7, 3, 144, 24), (1, 4, 4, 3, 5)])
def test_conv1x1_with_epilogue(cfg):
    n, h, w, ci, co = cfg
    g = graph()
    g.ext("X", (n, h, w, ci)); g.ext("Wc", (ci, co)); g.ext("s", (co,)); g.ext("t", (co,))
    e = g.add("Conv1x1", ["X", "Wc"])
    e = g.add("ScaleShift", [e, "s", "t"], axis=-1)
    g.mark_output(g.add("Clip", [e], lo=0.0, hi=6.0, out="Y"))
    ins = {"X": rnd((n, h, w, ci), 11, 0, 1), "Wc": rnd((ci, co), 12, -0.5, 0.5), "s": rnd((co,), 13, 0.5, 1.5), "t": rnd((co,), 14, -0.5, 0.5)}
    check(W.Workload(g, ins), RTOL_F32, FUSED, expect_blocks=1)


# fp32 blocks on the tensor cores (split-TF32): tall-and-skinny shapes, ragged M, N and K
@pytest.mark.parametrize("cfg", [(2, 16, 16, 24, 144), (3, 19, 23, 144, 24), (1, 30, 31, 12, 20), (1, 40, 40, 36, 160), (4, 16, 16, 32, 192),
                                 (1, 33, 33, 100, 8), (2, 24, 24, 96, 48),
                                 (1, 29, 89, 32, 124), (1, 40, 40, 16, 100), (1, 40, 40, 16, 96)])
@pytest.mark.parametrize("epi", ["clip", "residual", "affine", "none"])
def test_conv1x1_tensor_core_fp32(cfg, epi):
    n, h, w, ci, co = cfg
    g = graph()
    g.ext("X", (n, h, w, ci)); g.ext("Wc", (ci, co)); g.ext("s", (co,)); g.ext("t", (co,))
    ins = {"X": rnd((n, h, w, ci), 11, -1, 1), "Wc": rnd((ci, co), 12, -0.5, 0.5), "s": rnd((co,), 13, 0.5, 1.5), "t": rnd((co,), 14, -0.5, 0.5)}
    e = g.add("Conv1x1", ["X", "Wc"])
    if epi == "none":
        g.mark_output(e)
    else:
        e = g.add("ScaleShift", [e, "s", "t"], axis=-1)
        if epi == "clip":
            g.mark_output(g.add("Clip", [e], lo=0.0, hi=6.0, out="Y"))
        elif epi == "affine":                  # a projection whose channel count changes: no residual
            g.mark_output(e)
        else:
            g.ext("R", (n, h, w, co)); ins["R"] = rnd((n, h, w, co), 15, -1, 1)
            g.mark_output(g.add("Add", [e, "R"], out="Y"))
    s = check(W.Workload(g, ins), RTOL_F32, FUSED | B.PLAN_NO_SMALL_CONV, expect_blocks=1)     # (few rows would go to the one-tile-per-CTA kernel)
    _expect_variant(s, 4)


def test_matmul_fp32_tall_skinny_uses_tensor_cores():
    m, k, n = 1000, 52, 72
    g = graph()
    g.ext("X", (m, k)); g.ext("Wt", (k, n), kind="weight"); g.ext("b", (n,))
    t = g.add("MatMul", ["X", "Wt"])
    t = g.add("Add", [t, "b"])
    g.mark_output(g.add("Tanh", [t], out="Y"))
    s = check(W.Workload(g, {"X": rnd((m, k), 3, -1, 1), "Wt": rnd((k, n), 4, -0.3, 0.3), "b": rnd((n,), 5)}), RTOL_F32, FUSED | B.PLAN_NO_SMALL_CONV, expect_blocks=1)
    _expect_variant(s, 4)


def test_matmul_fp32_tall_skinny_transposed_weight_and_second_output():
    """fp32 tensor-core kernel with a K-major weight (strided B: split by the strided loader) and a block with two
    outputs (general, transposing epilogue)."""
    m, k, n = 777, 40, 56
    g = graph()
    g.ext("X", (m, k)); g.ext("Wt", (n, k), kind="weight"); g.ext("b", (n,))
    w = g.add("Transpose", ["Wt"], perm=(1, 0))
    t = g.add("MatMul", ["X", w])
    t = g.add("Add", [t, "b"], out="Z")
    g.mark_output(t)
    g.mark_output(g.add("Relu", [t], out="Y"))
    s = check(W.Workload(g, {"X": rnd((m, k), 3, -1, 1), "Wt": rnd((n, k), 4, -0.3, 0.3), "b": rnd((n,), 5)}), RTOL_F32, FUSED | B.PLAN_NO_SMALL_CONV, expect_blocks=1)
    _expect_variant(s, 4)


@pytest.mark.parametrize("cfg", [(1, 5, 6, 8), (2, 7, 9, 144), (1, 1, 1, 4), (1, 3, 1, 12), (2, 30, 17, 24)])
def test_dwconv3x3_with_epilogue(cfg):
    n, h, w, c = cfg
    g = graph()
    g.ext("X", (n, h, w, c)); g.ext("Kd", (3, 3, c)); g.ext("s", (c,)); g.ext("t", (c,))
    e = g.add("DwConv3x3", ["X", "Kd"])
    e = g.add("ScaleShift", [e, "s", "t"], axis=-1)
    g.mark_output(g.add("Clip", [e], lo=0.0, hi=6.0, out="Y"))
    ins = {"X": rnd((n, h, w, c), 21, 0, 1), "Kd": rnd((3, 3, c), 22, -0.5, 0.5), "s": rnd((c,), 23, 0.5, 1.5), "t": rnd((c,), 24, -0.5, 0.5)}
    check(W.Workload(g, ins), RTOL_F32, FUSED, expect_blocks=1)
    check(W.Workload(g, ins), RTOL_F32, UNFUSED, expect_blocks=3)


# shapes with enough tiles for the TMA-tiled depthwise kernel: ragged H and W, several channel blocks, several items per thread
@pytest.mark.parametrize("cfg", [(64, 20, 9, 12), (10, 16, 16, 320), (80, 9, 10, 36), (3, 56, 56, 144), (100, 12, 31, 8)])
def test_dwconv3x3_tma_tiled(cfg):
    n, h, w, c = cfg
    g = graph()
    g.ext("X", (n, h, w, c)); g.ext("Kd", (3, 3, c)); g.ext("s", (c,)); g.ext("t", (c,)); g.ext("R", (n, h, w, c))
    e = g.add("DwConv3x3", ["X", "Kd"])
    e = g.add("ScaleShift", [e, "s", "t"], axis=-1)
    g.mark_output(g.add("Add", [e, "R"], out="Y"))
    ins = {"X": rnd((n, h, w, c), 21, -1, 1), "Kd": rnd((3, 3, c), 22, -0.5, 0.5), "s": rnd((c,), 23, 0.5, 1.5), "t": rnd((c,), 24, -0.5, 0.5),
           "R": rnd((n, h, w, c), 25, -1, 1)}
    s = check(W.Workload(g, ins), RTOL_F32, FUSED, expect_blocks=1)
    _expect_variant(s, -1)
    check(W.Workload(g, ins), RTOL_F32, UNFUSED, expect_blocks=3)


@pytest.mark.parametrize("cfg", [(2, 14, 14, 24, 144), (32, 56, 56, 24, 144), (1, 3, 5, 8, 16)])
@pytest.mark.parametrize("flags", [FUSED, UNFUSED])
def test_mbconv_block(cfg, flags):
    n, h, w, cin, cexp = cfg
    s = check(W.mbconv_block(n, h, w, cin, cexp), RTOL_F32, flags, expect_blocks=3 if flags == FUSED else 9)
    if flags == FUSED:
        assert [b["family"] for b in s.g.blocks()] == ["conv1x1", "dwconv", "conv1x1"]


@pytest.mark.parametrize("flags,rewrite", [(FUSED, B.REWRITE_NONE), (UNFUSED, B.REWRITE_NONE), (FUSED, B.REWRITE_CANON_MACRO)])
def test_encoder_small(flags, rewrite):
    wl = W.encoder(layers=2, batch=2, seq=32, hidden=64, heads=4, ffn=128)
    s, got, ref = run_both(wl, flags, rewrite)
    (name,) = wl.graph.outputs
    close(got[name], ref[name], RTOL_BF16)
    if flags == FUSED:
        assert s.plan_stats.n_kernels <= 2 * 11


@pytest.mark.parametrize("flags,rewrite", [(FUSED, B.REWRITE_NONE), (UNFUSED, B.REWRITE_NONE), (FUSED, B.REWRITE_DEFAULT), (FUSED, B.REWRITE_CANON_MACRO)])
def test_decoder_small(flags, rewrite):
    """GPT-2 style decoder (pre-LayerNorm, GELU by tanh spelled out in primitives, final LayerNorm)."""
    wl = W.decoder(layers=2, batch=2, seq=32, hidden=64, heads=4, ffn=128)
    s, got, ref = run_both(wl, flags, rewrite)
    (name,) = wl.graph.outputs
    close(got[name], ref[name], RTOL_BF16)
    if flags == FUSED:
        assert s.plan_stats.n_kernels <= 2 * 12 + 1


def test_encoder_full_size_one_layer_elementwise():
    wl = W.encoder(layers=1)
    for flags, rw, kernels in [(FUSED, B.REWRITE_CANON_MACRO, 9), (FUSED, B.REWRITE_DEFAULT, 11)]:
        s, got, ref = run_both(wl, flags, rw)
        (name,) = wl.graph.outputs
        close(got[name], ref[name], RTOL_BF16)
        assert s.plan_stats.n_kernels == kernels


def test_encoder_full_size_twelve_layers():
    # bf16 activations between blocks accumulate rounding over 12 layers: bound the relative L2 error end to end
    wl = W.encoder()
    assert len(wl.graph.ops) == 576
    s, got, ref = run_both(wl, FUSED, B.REWRITE_CANON_MACRO)
    (name,) = wl.graph.outputs
    rel = np.linalg.norm(got[name] - ref[name]) / np.linalg.norm(ref[name])
    assert rel < 2e-2, rel
    assert s.plan_stats.n_kernels == 108 and np.all(np.isfinite(got[name]))


@pytest.mark.parametrize("flags", [B.PLAN_FUSED, B.PLAN_UNFUSED])
@pytest.mark.parametrize("nhw,cin,cout,slices", [((2, 32, 32), 256, 64, 2), ((1, 40, 40), 384, 32, 2), ((1, 24, 24), 576, 48, 3),
                                                  ((1, 24, 24), 960, 24, 4), ((2, 16, 16), 248, 40, 2)])
@pytest.mark.parametrize("tail", ["bn_clip", "bn"])
def test_deep_pointwise_convolution_is_split_along_k(nhw, cin, cout, slices, flags, tail):
    """fp32 pointwise convolutions deeper than the split-TF32 kernel takes (K > 244) are planned as 2-4 tensor-core
    contractions over K slices (as few as fit the kernel's shared memory), the partial sums riding in a later slice's
    epilogue."""
    flags |= B.PLAN_SPLIT_ALWAYS                       # the sizes here are below the planner's break-even
    n, h, w = nhw
    g = graph("deep_pw")
    g.ext("X", (n, h, w, cin)); g.ext("Wt", (cin, cout), kind="weight"); g.ext("s", (cout,)); g.ext("t", (cout,))
    y = g.add("ScaleShift", [g.add("Conv1x1", ["X", "Wt"]), "s", "t"], axis=-1)
    if tail == "bn_clip":
        y = g.add("Clip", [y], lo=0.0, hi=6.0)
    g.mark_output(y)
    ins = {"X": rnd((n, h, w, cin), 90, 0.0, 1.0), "Wt": rnd((cin, cout), 91, -0.2, 0.2), "s": rnd((cout,), 92, 0.5, 1.5),
           "t": rnd((cout,), 93, -0.5, 0.5)}
    s = check(W.Workload(g, ins), 2e-5, flags)
    gemms = [b for b in s.g.blocks() if b["family"] == "gemm"]
    assert len(gemms) >= slices and all(b["variant"] in (4, 7) for b in gemms), s.g.blocks()
    assert not [b for b in s.g.blocks() if b["family"] == "conv1x1"], s.g.blocks()
    assert s.plan_stats.n_ops == (3 if tail == "bn_clip" else 2)          # the slices count as the one convolution they came from


@pytest.mark.parametrize("mnk", [(2048, 64, 512), (700, 100, 300), (4096, 16, 1024)])
def test_deep_fp32_matrix_product_is_split_along_k(mnk):
    m, n, k = mnk
    g = graph("deep_mm")
    g.ext("A", (m, k)); g.ext("Bm", (k, n), kind="weight"); g.ext("b", (n,))
    g.mark_output(g.add("Relu", [g.add("Add", [g.add("MatMul", ["A", "Bm"]), "b"])]))
    s = check(W.Workload(g, {"A": rnd((m, k), 94, -1.0, 1.0), "Bm": rnd((k, n), 95, -0.2, 0.2), "b": rnd((n,), 96)}), 2e-5,
              B.PLAN_FUSED | B.PLAN_SPLIT_ALWAYS)
    gemms = [b for b in s.g.blocks() if b["family"] == "gemm"]
    assert len(gemms) >= 2 and all(b["variant"] in (4, 7) for b in gemms), s.g.blocks()


@pytest.mark.parametrize("flags", [B.PLAN_FUSED, B.PLAN_UNFUSED])
@pytest.mark.parametrize("nhw,cin,cout,tail", [((2, 32, 32), 64, 384, "bn_clip_res_relu"), ((1, 40, 40), 96, 200, "bn_clip"),
                                               ((2, 24, 24), 32, 256, "none"), ((1, 32, 32), 24, 240, "bias_two_readers"),
                                               ((3, 16, 16), 48, 512, "prelu")])
def test_wide_pointwise_convolution_is_split_into_channel_blocks(nhw, cin, cout, tail, flags):
    """fp32 pointwise convolutions with more output channels than the split-TF32 kernel's accumulators hold (N > 192) are
    planned as tensor-core contractions over column blocks of W; the channel-wise operators behind the convolution move
    into each block's epilogue and the blocks store straight into the result (parts of a Concat)."""
    fused = flags == B.PLAN_FUSED
    flags |= B.PLAN_SPLIT_ALWAYS
    n, h, w = nhw
    g = graph("wide_pw")
    g.ext("X", (n, h, w, cin)); g.ext("Wt", (cin, cout), kind="weight"); g.ext("s", (cout,)); g.ext("t", (cout,)); g.ext("R", (n, h, w, cout))
    y = g.add("Conv1x1", ["X", "Wt"])
    if tail == "bn_clip_res_relu":
        y = g.add("Relu", [g.add("Add", [g.add("Clip", [g.add("ScaleShift", [y, "s", "t"], axis=-1)], lo=0.0, hi=6.0), "R"])])
    elif tail == "bn_clip":
        y = g.add("Clip", [g.add("ScaleShift", [y, "s", "t"], axis=-1)], lo=0.0, hi=6.0)
    elif tail == "bias_two_readers":
        y = g.add("Add", [y, "t"])
        g.mark_output(g.add("Tanh", [y]))            # a second reader ends the chain that moves into the blocks
        y = g.add("Sigmoid", [y])
    elif tail == "prelu":
        y = g.add("PRelu", [g.add("Sub", ["R", y]), "s"])
    g.mark_output(y)
    ins = {"X": rnd((n, h, w, cin), 97, 0.0, 1.0), "Wt": rnd((cin, cout), 98, -0.2, 0.2), "s": rnd((cout,), 99, 0.5, 1.5),
           "t": rnd((cout,), 100, -0.5, 0.5), "R": rnd((n, h, w, cout), 101, -1.0, 1.0)}
    s = check(W.Workload(g, ins), 2e-5, flags)
    gemms = [b for b in s.g.blocks() if b["family"] == "gemm"]
    assert len(gemms) >= 2 and all(b["variant"] in (4, 7) for b in gemms), s.g.blocks()
    assert not [b for b in s.g.blocks() if b["family"] == "conv1x1"], s.g.blocks()
    if fused and tail in ("bn_clip_res_relu", "bn_clip", "none", "prelu"):
        assert s.plan_stats.n_kernels == len(gemms), s.g.blocks()      # nothing but the column blocks runs


def test_split_decision_follows_the_cost_model():
    """At 25088 pixels a 160 -> 960 convolution is worth 18 tensor-core kernels; a 576 -> 160 one at 6272 pixels is not
    worth 12 (measured: 263 us against 675 us, and 123 us against 111 us).  At 6272 pixels the one-tile-per-CTA kernel is
    the unsplit alternative: a deep 576 -> 96 projection stays whole (41 us against 95 us in six K slices), a wide
    96 -> 576 expansion is cut into column blocks (36 us in three kernels against 61 us)."""
    for (n, hw, cin, cout), split in [((32, 28, 160, 960), True), ((32, 14, 576, 160), False), ((32, 14, 576, 96), False),
                                      ((32, 14, 96, 576), True)]:
        g = graph("split_cost")
        g.ext("X", (n, hw, hw, cin)); g.ext("Wt", (cin, cout), kind="weight")
        g.mark_output(g.add("Conv1x1", ["X", "Wt"]))
        from paper_2108_13342_b200.runtime import build_graph
        G, ids = build_graph(g)
        G.rewrite(B.REWRITE_NONE)
        G.plan(B.PLAN_FUSED)
        fams = {b["family"] for b in G.blocks()}
        assert ("gemm" in fams) == split, G.blocks()


def test_rebinding_any_epilogue_operand_reencodes_the_tensor_maps():
    """GEMM -> scale, shift -> + residual: the residual is the THIRD epilogue operand and is read through a TMA
    descriptor, which embeds its address.  Binding another buffer for it (and then for A and for the output) must
    be followed by the kernel; a stale descriptor would silently keep reading the old buffer."""
    import torch
    m, n, k = 512, 256, 128
    g = graph()
    g.ext("A", (m, k), "bf16"); g.ext("Bm", (k, n), "bf16"); g.ext("sc", (n,), "f32"); g.ext("sh", (n,), "f32"); g.ext("R", (m, n), "bf16")
    t = g.add("MatMul", ["A", "Bm"])
    t = g.add("ScaleShift", [t, "sc", "sh"], axis=-1)
    t = g.add("Add", [t, "R"], out="Y")
    g.mark_output(t)
    ins = {"A": _bf(rnd((m, k), 61, -1, 1)), "Bm": _bf(rnd((k, n), 62, -0.1, 0.1)), "sc": rnd((n,), 63, 0.5, 1.5),
           "sh": rnd((n,), 64, -0.5, 0.5), "R": _bf(rnd((m, n), 65, -1, 1))}
    wl = W.Workload(g, ins)
    s, got, ref = run_both(wl, FUSED)
    assert s.plan_stats.n_kernels == 1
    close(got["Y"], ref["Y"], RTOL_BF16)
    from oracle import interp as O
    for name, seed in [("R", 66), ("A", 67)]:
        old = s.buffers[name]                                   # keep the old buffer alive: a stale map reads valid memory
        ins[name] = _bf(rnd(ins[name].shape, seed, -1, 1))
        s.set_input(name, ins[name])
        assert s.buffers[name].data_ptr() != old.data_ptr()
        s.run()
        close(s.output("Y"), O.run_graph(wl.graph, ins)["Y"], RTOL_BF16)
    old = s.buffers["Y"]
    new = torch.full_like(old, float("nan"))
    s.buffers["Y"] = new
    s.g.bind(s.ids["Y"], new.data_ptr())
    s.run()
    close(s.output("Y"), O.run_graph(wl.graph, ins)["Y"], RTOL_BF16)
    assert s.g.status() == (0, -1)



# fp32 contractions with few rows: one 16 x 32 tile per CTA, K split over its four warps (mma.sync, split TF32)
@pytest.mark.parametrize("cfg", [(1, 14, 14, 384, 64), (1, 14, 14, 64, 384), (1, 7, 7, 576, 160), (1, 28, 28, 24, 144), (2, 9, 11, 40, 24),
                                 (1, 5, 3, 16, 8), (1, 20, 20, 144, 24), (1, 1, 1, 320, 104), (1, 30, 30, 72, 200),
                                 (1, 1, 1, 320, 100), (2, 3, 3, 64, 20), (4, 1, 1, 48, 2)])
@pytest.mark.parametrize("epi", ["clip", "residual", "affine", "chain", "none"])
def test_conv1x1_few_rows(cfg, epi):
    n, h, w, ci, co = cfg
    g = graph()
    g.ext("X", (n, h, w, ci)); g.ext("Wc", (ci, co), kind="weight"); g.ext("s", (co,), kind="weight"); g.ext("t", (co,), kind="weight")
    ins = {"X": rnd((n, h, w, ci), 11, -1, 1), "Wc": rnd((ci, co), 12, -0.5, 0.5), "s": rnd((co,), 13, 0.5, 1.5), "t": rnd((co,), 14, -0.5, 0.5)}
    e = g.add("Conv1x1", ["X", "Wc"])
    if epi == "none":
        g.mark_output(e)
    elif epi == "chain":                       # interpreted: a per-pixel operand, a gate, two outputs
        g.ext("P", (n, h, w, 1)); ins["P"] = rnd((n, h, w, 1), 16, 0.5, 1.5)
        z = g.add("Mul", [g.add("Add", [e, "t"]), "P"])
        g.mark_output(z)
        g.mark_output(g.add("Mul", [z, g.add("Sigmoid", [z])]))
    else:
        e = g.add("ScaleShift", [e, "s", "t"], axis=-1)
        if epi == "clip":
            g.mark_output(g.add("Clip", [e], lo=0.0, hi=6.0, out="Y"))
        elif epi == "affine":
            g.mark_output(e)
        else:
            g.ext("R", (n, h, w, co)); ins["R"] = rnd((n, h, w, co), 15, -1, 1)
            g.mark_output(g.add("Add", [e, "R"], out="Y"))
    s = check(W.Workload(g, ins), RTOL_F32, FUSED, expect_blocks=1)
    _expect_variant(s, 7)
    s = check(W.Workload(g, ins), RTOL_F32, FUSED | B.PLAN_NO_SMALL_CONV, expect_blocks=1)     # the kernels it replaces
    assert s.g.blocks()[0]["variant"] != 7
