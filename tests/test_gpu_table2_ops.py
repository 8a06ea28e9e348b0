"""Parity of the remaining Table 2 operators against the oracle: DepthToSpace / SpaceToDepth (Shuffle), Resize
(One-to-Many), Concat (One-to-One, as changed store indices of its inputs' producer blocks, Section 4.4.2),
MaxPool / AveragePool (Many-to-Many anchors with an epilogue), alone and fused with their neighbours, and a
CNN fragment that uses all of them."""
import numpy as np
import pytest

from paper_2108_13342_b200 import binding as B
from paper_2108_13342_b200 import workloads as W
from util import RTOL_F32, check, graph, rnd, run_both, close

pytestmark = pytest.mark.gpu

PLANS = [B.PLAN_FUSED, B.PLAN_UNFUSED]


def _exact(wl, flags):
    s, got, ref = run_both(wl, flags)
    for n in wl.graph.outputs:
        assert np.array_equal(got[n].astype(np.float64), ref[n]), (n, s.g.blocks())
    return s


@pytest.mark.parametrize("flags", PLANS)
@pytest.mark.parametrize("shape,b", [((2, 8, 8, 16), 2), ((1, 5, 7, 36), 3), ((3, 4, 6, 8), 2), ((2, 9, 3, 64), 4)])
def test_depthtospace_and_back_are_exact_moves(shape, b, flags):
    g = graph("d2s")
    g.ext("X", shape)
    y = g.add("DepthToSpace", ["X"], block=b)
    z = g.add("SpaceToDepth", [y], block=b)
    g.mark_output(y); g.mark_output(z)
    _exact(W.Workload(g, {"X": rnd(shape, 1)}), flags)


@pytest.mark.parametrize("flags", PLANS)
@pytest.mark.parametrize("shape,b", [((2, 8, 8, 16), 2), ((1, 6, 9, 18), 3)])
def test_shuffle_ops_inside_a_chain(shape, b, flags):
    n, h, w, c = shape
    g = graph("d2s_chain")
    g.ext("X", shape); g.ext("Y", (n, h * b, w * b, c // (b * b))); g.ext("v", (c // (b * b),))
    t = g.add("Relu", ["X"])
    t = g.add("DepthToSpace", [t], block=b)
    t = g.add("Add", [g.add("Mul", [t, "v"]), "Y"])
    u = g.add("Sigmoid", [g.add("SpaceToDepth", [t], block=b)])
    g.mark_output(t); g.mark_output(u)
    wl = W.Workload(g, {"X": rnd(shape, 2), "Y": rnd((n, h * b, w * b, c // (b * b)), 3), "v": rnd((c // (b * b),), 4, 0.5, 1.5)})
    check(wl, RTOL_F32, flags)


@pytest.mark.parametrize("flags", PLANS)
def test_spacetodepth_in_front_of_a_pointwise_convolution(flags):
    g = graph("s2d_conv")
    g.ext("X", (2, 12, 12, 8)); g.ext("Wt", (32, 24), kind="weight")
    t = g.add("Conv1x1", [g.add("SpaceToDepth", ["X"], block=2), "Wt"])
    g.mark_output(g.add("Relu", [t]))
    check(W.Workload(g, {"X": rnd((2, 12, 12, 8), 5), "Wt": rnd((32, 24), 6, -0.3, 0.3)}), RTOL_F32, flags)


@pytest.mark.parametrize("flags", PLANS)
@pytest.mark.parametrize("shape,s", [((2, 8, 8, 16), 2), ((1, 5, 7, 6), 3), ((2, 3, 4, 5), 2)])
def test_resize_nearest(shape, s, flags):
    n, h, w, c = shape
    g = graph("up")
    g.ext("X", shape); g.ext("Y", (n, h * s, w * s, c))
    r = g.add("Resize", ["X"], scale=s)
    t = g.add("Add", [g.add("Resize", [g.add("Tanh", ["X"])], scale=s), "Y"])
    g.mark_output(r); g.mark_output(t)
    sess, got, ref = run_both(W.Workload(g, {"X": rnd(shape, 7), "Y": rnd((n, h * s, w * s, c), 8)}), flags)
    names = list(g.outputs)
    assert np.array_equal(got[names[0]].astype(np.float64), ref[names[0]])
    close(got[names[1]], ref[names[1]], RTOL_F32)


@pytest.mark.parametrize("flags", PLANS)
@pytest.mark.parametrize("axis,shapes", [
    (3, [(2, 8, 8, 16), (2, 8, 8, 24), (2, 8, 8, 8)]),
    (3, [(1, 5, 3, 5), (1, 5, 3, 7)]),                       # ragged channel counts: unaligned bases
    (0, [(2, 4, 4, 8), (3, 4, 4, 8), (1, 4, 4, 8), (2, 4, 4, 8)]),
    (1, [(2, 3, 5, 4), (2, 6, 5, 4)]),
    (-1, [(7, 33), (7, 31)]),
])
def test_concat_of_external_and_produced_tensors(axis, shapes, flags):
    g = graph("cat")
    ins = {}
    parts = []
    for i, shp in enumerate(shapes):
        g.ext(f"X{i}", shp); ins[f"X{i}"] = rnd(shp, 10 + i)
        parts.append(f"X{i}" if i % 2 else g.add("Tanh", [f"X{i}"]))
    c = g.add("Concat", parts, axis=axis)
    g.mark_output(c)
    g.mark_output(g.add("Sigmoid", [c]))
    s = check(W.Workload(g, ins), RTOL_F32, flags)
    if flags == B.PLAN_FUSED and all(shp[-1] % 4 == 0 for shp in shapes):
        # each producer stores straight into the result: no kernel for the Concat itself (with ragged channel counts
        # the stores would be scalar and the cost model may prefer a separate copy)
        fams = [b["ops"] for b in s.g.blocks()]
        assert ["Tanh", "ConcatPart"] in fams, fams


@pytest.mark.parametrize("flags", PLANS)
def test_concat_is_exact_and_nests(flags):
    g = graph("cat_exact")
    g.ext("A", (3, 4, 8)); g.ext("Bt", (3, 2, 8)); g.ext("Ct", (3, 6, 5))
    ab = g.add("Concat", ["A", "Bt"], axis=1)                # [3, 6, 8]
    abc = g.add("Concat", [ab, "Ct", ab], axis=2)            # [3, 6, 21]: a Concat's result as a part, twice
    g.mark_output(abc)
    _exact(W.Workload(g, {"A": rnd((3, 4, 8), 20), "Bt": rnd((3, 2, 8), 21), "Ct": rnd((3, 6, 5), 22)}), flags)


def test_identical_concats_survive_common_subexpression_elimination():
    """Two Concats of the same inputs (and two that share a first input) under the rewriting pass: the parts fill their
    own results in place and are never merged."""
    g = graph("cat_cse")
    g.ext("X", (3, 12, 12, 4))
    a = g.add("DepthToSpace", ["X"], block=2)
    b = g.add("Sin", [a])
    c1 = g.add("Concat", [a, b], axis=3)
    c2 = g.add("Concat", [a, a], axis=3)
    c3 = g.add("Concat", [a, a], axis=3)
    g.mark_output(c1); g.mark_output(c2); g.mark_output(g.add("Relu", [c3]))
    check(W.Workload(g, {"X": rnd((3, 12, 12, 4), 25)}), RTOL_F32, B.PLAN_FUSED, B.REWRITE_DEFAULT)


@pytest.mark.parametrize("flags", PLANS)
def test_concat_fed_by_row_and_convolution_blocks(flags):
    g = graph("cat_blocks")
    g.ext("X", (2, 10, 10, 16)); g.ext("W1", (16, 24), kind="weight"); g.ext("s", (24,)); g.ext("t", (24,))
    g.ext("Kd", (3, 3, 16), kind="weight"); g.ext("ga", (16,)); g.ext("be", (16,))
    a = g.add("Clip", [g.add("ScaleShift", [g.add("Conv1x1", ["X", "W1"]), "s", "t"], axis=-1)], lo=0.0, hi=6.0)
    b = g.add("Relu", [g.add("DwConv3x3", ["X", "Kd"])])
    c = g.add("LayerNorm", ["X", "ga", "be"], axis=-1, eps=1e-5)
    d = g.add("MaxPool", ["X"], kernel=3, stride=1, pad=1)
    y = g.add("Concat", [a, b, c, d], axis=3)                 # [2, 10, 10, 72]
    g.mark_output(g.add("MulC", [y], c=0.5))
    ins = {"X": rnd((2, 10, 10, 16), 30), "W1": rnd((16, 24), 31, -0.3, 0.3), "s": rnd((24,), 32, 0.5, 1.5),
           "t": rnd((24,), 33, -0.5, 0.5), "Kd": rnd((3, 3, 16), 34, -0.5, 0.5), "ga": rnd((16,), 35, 0.8, 1.2),
           "be": rnd((16,), 36, -0.2, 0.2)}
    s = check(W.Workload(g, ins), 2e-4, flags)                # the convolution part runs as split TF32 when eligible
    if flags == B.PLAN_FUSED:
        assert s.plan_stats.n_kernels == 5, s.g.blocks()      # four producers (each ends in its part) + the consumer


@pytest.mark.parametrize("flags", PLANS)
def test_concat_bf16(flags):
    g = graph("cat_bf16")
    g.ext("X", (4, 64, 32), "bf16"); g.ext("Y", (4, 64, 16), "bf16")
    c = g.add("Concat", [g.add("Relu", ["X"]), "Y"], axis=2)
    g.mark_output(c)
    ins = {"X": W.round_to_bf16(rnd((4, 64, 32), 40)), "Y": W.round_to_bf16(rnd((4, 64, 16), 41))}
    _exact(W.Workload(g, ins), flags)


@pytest.mark.parametrize("flags", PLANS)
@pytest.mark.parametrize("kind", ["MaxPool", "AveragePool"])
@pytest.mark.parametrize("shape,k,s,p", [((2, 16, 16, 8), 2, 2, 0), ((1, 15, 13, 12), 3, 2, 1), ((3, 7, 9, 4), 3, 1, 1),
                                         ((2, 8, 8, 32), 8, 1, 0), ((1, 11, 11, 20), 5, 3, 2), ((2, 6, 10, 8), 2, 1, 0)])
def test_pooling_with_epilogue(kind, shape, k, s, p, flags):
    c = shape[3]
    g = graph("pool")
    g.ext("X", shape); g.ext("sc", (c,)); g.ext("sh", (c,))
    y = g.add(kind, ["X"], kernel=k, stride=s, pad=p)
    z = g.add("Relu", [g.add("ScaleShift", [y, "sc", "sh"], axis=-1)])
    g.mark_output(y); g.mark_output(z)
    sess = check(W.Workload(g, {"X": rnd(shape, 50), "sc": rnd((c,), 51, 0.5, 1.5), "sh": rnd((c,), 52, -0.5, 0.5)}),
                 RTOL_F32, flags)
    if flags == B.PLAN_FUSED:
        assert sess.plan_stats.n_kernels == 1, sess.g.blocks()


def test_maxpool_is_exact():
    g = graph("maxpool_exact")
    g.ext("X", (2, 17, 19, 8))
    g.mark_output(g.add("MaxPool", ["X"], kernel=3, stride=2, pad=1))
    _exact(W.Workload(g, {"X": rnd((2, 17, 19, 8), 53)}), B.PLAN_FUSED)


@pytest.mark.parametrize("flags,rewrite", [(B.PLAN_FUSED, B.REWRITE_DEFAULT), (B.PLAN_FUSED, B.REWRITE_NONE), (B.PLAN_UNFUSED, B.REWRITE_NONE)])
@pytest.mark.parametrize("dims", [(2, 16, 16, 8), (1, 24, 40, 16), (3, 64, 64, 32)])
def test_cnn_fragment(dims, flags, rewrite):
    wl = W.cnn_neck(*dims) if dims[1] == dims[2] else None
    if wl is None:      # the global pool of the fragment takes a square map: use the nearest square
        wl = W.cnn_neck(dims[0], dims[1], dims[1], dims[3])
    s = check(wl, 5e-4, flags, rewrite)          # several split-TF32 convolutions in sequence
    if flags == B.PLAN_FUSED:
        assert s.plan_stats.n_kernels < s.plan_stats.n_ops


# ---- further One-to-One operators of Table 2 -------------------------------------------------------------------

@pytest.mark.parametrize("flags", PLANS)
@pytest.mark.parametrize("shape", [(3, 37, 20), (2, 64, 256), (5, 7)])
def test_further_one_to_one_operators(shape, flags):
    """Sin / Cos / Asin in a chain; the discrete operators (Ceil, Floor, Round, Greater, Not) applied to inputs, where both
    sides see the same fp32-representable values, and their 0 / 1 or integer results used further down the chain."""
    g = graph("more_ops")
    g.ext("X", shape); g.ext("U", shape); g.ext("v", (shape[-1],)); g.ext("H", shape)
    t = g.add("Asin", [g.add("Mul", [g.add("Sin", ["X"]), g.add("Cos", ["X"])])])          # |sin cos| <= 1/2
    t = g.add("LeakyRelu", [g.add("Sub", [t, "U"])], alpha=0.125)
    t = g.add("PRelu", [g.add("Sub", [t, "v"]), "v"])                                      # slope broadcast along the rows
    g.mark_output(t)
    gt = g.add("Greater", ["X", "U"])
    sel = g.add("Add", [g.add("Mul", [gt, "X"]), g.add("Mul", [g.add("Not", [gt]), "U"])])  # max(X, U) spelled with a mask
    g.mark_output(sel)
    g.mark_output(g.add("Greater", ["X", "v"]))
    r = g.add("Add", [g.add("Ceil", ["H"]), g.add("Add", [g.add("Floor", ["H"]), g.add("Round", ["H"])])])
    g.mark_output(r)
    halves = np.round(rnd(shape, 63, -8.0, 8.0) * 2.0) / 2.0          # multiples of 1/2: ties included
    ins = {"X": rnd(shape, 60), "U": rnd(shape, 61), "v": rnd((shape[-1],), 62, 0.1, 0.9), "H": halves.astype(np.float32)}
    s, got, ref = run_both(W.Workload(g, ins), flags)
    names = list(g.outputs)
    close(got[names[0]], ref[names[0]], RTOL_F32)
    for n in names[1:]:
        assert np.array_equal(got[n].astype(np.float64), ref[n]), n
    assert np.array_equal(got[names[1]], np.maximum(ins["X"], ins["U"]))


@pytest.mark.parametrize("flags", PLANS)
def test_prelu_and_leakyrelu_in_a_convolution_epilogue(flags):
    g = graph("conv_prelu")
    g.ext("X", (2, 12, 12, 16)); g.ext("Wt", (16, 32), kind="weight"); g.ext("b", (32,)); g.ext("a", (32,))
    t = g.add("PRelu", [g.add("Add", [g.add("Conv1x1", ["X", "Wt"]), "b"]), "a"])
    t = g.add("LeakyRelu", [g.add("AddC", [t], c=-0.1)], alpha=0.2)
    g.mark_output(t)
    ins = {"X": rnd((2, 12, 12, 16), 64), "Wt": rnd((16, 32), 65, -0.3, 0.3), "b": rnd((32,), 66, -0.5, 0.5), "a": rnd((32,), 67, 0.05, 0.3)}
    s = check(W.Workload(g, ins), RTOL_F32, flags)
    if flags == B.PLAN_FUSED:
        assert s.plan_stats.n_kernels == 1, s.g.blocks()


# ---- ConvTranspose (stride = kernel) and Gather ------------------------------------------------------------------

@pytest.mark.parametrize("flags", PLANS)
@pytest.mark.parametrize("shape,k,cout", [((2, 8, 8, 16), 2, 8), ((1, 5, 7, 12), 3, 4), ((3, 16, 16, 32), 2, 32)])
def test_convtranspose_relu_concat(shape, k, cout, flags):
    """The paper's ConvTranspose + ReLU + Concat example: the transposed convolution's epilogue spreads each pixel's
    k x k cell over the result and stores it straight into the Concat."""
    n, h, w, c = shape
    g = graph("deconv")
    g.ext("X", shape); g.ext("Wt", (c, k, k, cout), kind="weight"); g.ext("S", (n, h * k, w * k, 8))
    t = g.add("Relu", [g.add("ConvTranspose", ["X", "Wt"], kernel=k)])
    y = g.add("Concat", [t, "S"], axis=3)
    g.mark_output(y)
    ins = {"X": rnd(shape, 70), "Wt": rnd((c, k, k, cout), 71, -0.3, 0.3), "S": rnd((n, h * k, w * k, 8), 72)}
    s = check(W.Workload(g, ins), 2e-4, flags)
    if flags == B.PLAN_FUSED and cout % 8 == 0:
        assert s.plan_stats.n_kernels == 2, s.g.blocks()      # the convolution block and the copy of the external part


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("v,d,idx_shape", [(50, 64, (7, 9)), (11, 5, (33,)), (1000, 768, (4, 128)), (3, 8, (2, 2, 2))])
def test_gather_rows(v, d, idx_shape, dtype):
    g = graph("gather")
    g.ext("T", (v, d), dtype); g.ext("I", idx_shape); g.ext("P", idx_shape[-1:] + (d,), dtype)
    e = g.add("Gather", ["T", "I"], axis=0)
    g.mark_output(e)
    g.mark_output(g.add("Add", [e, "P"]))                        # an embedding lookup plus a position table
    idx = np.floor(W.uniform(777, 80, idx_shape, 0.0, float(v))).clip(0, v - 1)
    tab = rnd((v, d), 81); pos = rnd(idx_shape[-1:] + (d,), 82)
    if dtype == "bf16":
        tab, pos = W.round_to_bf16(tab), W.round_to_bf16(pos)
    s, got, ref = run_both(W.Workload(g, {"T": tab, "I": idx, "P": pos}), B.PLAN_FUSED)
    names = list(g.outputs)
    assert np.array_equal(got[names[0]].astype(np.float64), ref[names[0]])
    close(got[names[1]], ref[names[1]], RTOL_F32 if dtype == "f32" else 1e-2)
    assert [b["family"] for b in s.g.blocks()][0] == "gather"


def test_gather_clamps_indices_outside_the_table():
    g = graph("gather_clamp")
    g.ext("T", (6, 12)); g.ext("I", (5,))
    g.mark_output(g.add("Gather", ["T", "I"], axis=0))
    tab = rnd((6, 12), 83)
    from paper_2108_13342_b200.runtime import Session
    s = Session(W.Workload(g, {"T": tab, "I": np.array([-3.0, 0.0, 5.0, 6.0, 1e9], dtype=np.float32)}))
    s.run()
    assert s.g.status()[0] == 0
    got = s.output(g.outputs[0])
    assert np.array_equal(got, tab[[0, 0, 5, 5, 5]].astype(np.float32))


@pytest.mark.parametrize("flags,always", [(B.PLAN_FUSED, False), (B.PLAN_FUSED, True), (B.PLAN_UNFUSED, True)])
def test_mobilenet_shaped_stack(flags, always):
    """Nine inverted-residual blocks, pooling between the stages, head and classifier: expansions wider than 192 channels
    and projections deeper than 244 go through the planner's column-block and K splits (forced at this small size in two
    of the three variants, decided by the cost model in the first)."""
    wl = W.mbconv_stack(n=4, hw=48)
    s = check(wl, 5e-4, flags | (B.PLAN_SPLIT_ALWAYS if always else 0), B.REWRITE_DEFAULT)
    fams = [b["family"] for b in s.g.blocks()]
    assert "dwconv" in fams and "pool" in fams
    if always:
        assert fams.count("gemm") >= 20, fams          # the split pieces
    if flags == B.PLAN_FUSED:
        assert s.plan_stats.n_kernels < s.plan_stats.n_ops


# ---- Section 4.4.2: layout selection ---------------------------------------------------------------------------------

@pytest.mark.parametrize("rewrite", [B.REWRITE_DEFAULT, B.REWRITE_KEEP_LAYOUT])
def test_channels_first_stack_with_and_without_layout_selection(rewrite):
    """The MobileNetV2-shaped stack written channels-first (a Transpose around every convolution and pool, batch
    normalisation on axis 1): same logits as the oracle's evaluation of that graph, whether the layout selection
    re-expresses the element-wise operators channels-last or every Transpose stays an index map."""
    wl = W.mbconv_stack(n=4, hw=48, layout="nchw")
    s = check(wl, 5e-4, B.PLAN_FUSED, rewrite)
    kinds = [k for b in s.g.blocks() for k in b["ops"]]
    assert kinds.count("Transpose") == (1 if rewrite == B.REWRITE_DEFAULT else 63)


def test_layout_selection_keeps_values_on_small_graphs():
    # composed (non-inverse) Transposes, a per-channel operand that follows its axis, a broadcast operand of full rank
    g = graph(); g.ext("X", (3, 5, 6, 7)); g.ext("s", (7,), kind="weight"); g.ext("t", (7,), kind="weight"); g.ext("b", (1, 7, 1, 1), kind="weight")
    y = g.add("Transpose", [g.add("Sigmoid", ["X"])], perm=(0, 3, 1, 2))                    # [3, 7, 5, 6]
    y = g.add("Add", [g.add("ScaleShift", [y, "s", "t"], axis=1), "b"])
    y = g.add("Transpose", [g.add("Tanh", [y])], perm=(0, 1, 3, 2))                          # [3, 7, 6, 5]
    g.mark_output(g.add("Softmax", [y], axis=-1))
    ins = {"X": rnd((3, 5, 6, 7), 1), "s": rnd((7,), 2, 0.5, 1.5), "t": rnd((7,), 3), "b": rnd((1, 7, 1, 1), 4)}
    s = check(W.Workload(g, ins), RTOL_F32, B.PLAN_FUSED, B.REWRITE_DEFAULT)
    assert s.rewrite_stats.layout_transposes_removed == 1
    # a residual Add whose operands both come back from the other layout, between two convolutions
    g = graph(); g.ext("X", (2, 9, 9, 16)); g.ext("W", (16, 16), kind="weight"); g.ext("s", (16,), kind="weight"); g.ext("t", (16,), kind="weight")
    a = g.add("Transpose", [g.add("Conv1x1", ["X", "W"])], perm=(0, 3, 1, 2))
    a = g.add("Clip", [g.add("ScaleShift", [a, "s", "t"], axis=1)], lo=0.0, hi=6.0)
    y = g.add("Transpose", [g.add("Add", [a, g.add("Transpose", ["X"], perm=(0, 3, 1, 2))])], perm=(0, 2, 3, 1))
    g.mark_output(g.add("Conv1x1", [y, "W"]))
    ins = {"X": rnd((2, 9, 9, 16), 5), "W": rnd((16, 16), 6, -0.3, 0.3), "s": rnd((16,), 7, 0.5, 1.5), "t": rnd((16,), 8)}
    s = check(W.Workload(g, ins), 5e-4, B.PLAN_FUSED, B.REWRITE_DEFAULT)
    assert s.rewrite_stats.layout_transposes_removed == 3


# ---- Where, Cast, CumSum, InstanceNormalization (Table 2) ------------------------------------------------------------

def test_where_is_a_selection_with_broadcasting():
    cond = (rnd((5, 1, 33), 1, 0.0, 1.0) > 0.5).astype(np.float32)
    a = rnd((1, 7, 33), 2); b = rnd((5, 7, 1), 3)
    b[0, 0, 0] = -np.inf; a[0, 1, 4] = np.inf                      # infinities pass through or stay out untouched
    g = graph(); g.ext("C", cond.shape); g.ext("A", a.shape); g.ext("Bv", b.shape)
    g.mark_output(g.add("Where", ["C", "A", "Bv"]))
    s, got, ref = run_both(W.Workload(g, {"C": cond, "A": a, "Bv": b}))
    assert s.plan_stats.n_kernels == 1
    np.testing.assert_array_equal(got[g.outputs[0]], ref[g.outputs[0]].astype(np.float32))          # bit-exact
    # inside a chain: Where(Greater(x, y), x * 2, Neg(y)) with every operand computed in the block
    g = graph(); g.ext("X", (64, 257)); g.ext("Y", (64, 257))
    c = g.add("Greater", ["X", "Y"])
    g.mark_output(g.add("Tanh", [g.add("Where", [c, g.add("MulC", ["X"], c=2.0), g.add("Neg", ["Y"])])]))
    s = check(W.Workload(g, {"X": rnd((64, 257), 4), "Y": rnd((64, 257), 5)}), RTOL_F32)
    assert s.plan_stats.n_kernels == 1


def test_where_masks_attention_scores_in_front_of_softmax():
    # the usual masking: scores where the mask is set, -1e9 elsewhere, then Softmax over the row
    S = 96
    mask = (np.tril(np.ones((S, S))) != 0).astype(np.float32)
    g = graph(); g.ext("Sc", (4, 3, S, S)); g.ext("M", (S, S), kind="weight"); g.ext("neg", (1,), kind="weight")
    w = g.add("Where", ["M", g.add("MulC", ["Sc"], c=0.125), "neg"])
    g.mark_output(g.add("Softmax", [w], axis=-1))
    s = check(W.Workload(g, {"Sc": rnd((4, 3, S, S), 6, -8, 8), "M": mask, "neg": np.full((1,), -1e9, np.float32)}), RTOL_F32)
    assert s.plan_stats.n_kernels == 1 and s.g.blocks()[0]["family"] == "row"
    y = s.output(g.outputs[0])
    assert np.all(y[..., np.triu_indices(S, 1)[0], np.triu_indices(S, 1)[1]] == 0.0)


@pytest.mark.parametrize("to", ["bf16", "i32", "bool", "f32"])
def test_cast_on_inputs_is_bit_exact(to):
    x = rnd((37, 130), 7, -300.0, 300.0)
    x[0, :6] = [0.0, -0.0, 0.5, -0.5, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8]          # zeros, halves and bfloat16 ties
    g = graph(); g.ext("X", x.shape)
    g.mark_output(g.add("Cast", ["X"], to=to))
    s, got, ref = run_both(W.Workload(g, {"X": x}))
    np.testing.assert_array_equal(got[g.outputs[0]].astype(np.float64), ref[g.outputs[0]])
    dt, _ = s.g.tensor_info(s.ids[g.outputs[0]])
    assert dt == (B.BF16 if to == "bf16" else B.F32)


def test_cast_inside_a_chain_rounds_the_value_its_consumers_see():
    # Sigmoid -> Cast(bf16) -> MulC -> Cast(i32): the second operator works on the rounded value
    x = rnd((64, 512), 8, -4.0, 4.0)
    g = graph(); g.ext("X", x.shape)
    k = g.add("Cast", [g.add("Sigmoid", ["X"])], to="bf16")
    g.mark_output(g.add("Cast", [g.add("MulC", [k], c=1024.0)], to="f32"))
    s, got, ref = run_both(W.Workload(g, {"X": x}))
    assert s.plan_stats.n_kernels == 1
    y, r = got[g.outputs[0]].astype(np.float64), ref[g.outputs[0]]
    # values are multiples of 1024 * 2^-9 at most apart by one bfloat16 step where fp32 and fp64 Sigmoid straddle a tie
    assert np.mean(y == r) > 0.99 and np.all(np.abs(y - r) <= 2.0 ** -7 * np.abs(r) + 1e-12)


@pytest.mark.parametrize("shape", [(5, 8), (33, 100), (16, 128), (7, 3, 1024), (6, 4096), (3, 8192), (64, 24), (9, 2052)])
@pytest.mark.parametrize("exclusive,reverse", [(0, 0), (1, 0), (0, 1), (1, 1)])
def test_cumsum_rows(shape, exclusive, reverse):
    g = graph(); g.ext("X", shape)
    g.mark_output(g.add("CumSum", ["X"], axis=-1, exclusive=exclusive, reverse=reverse))
    s = check(W.Workload(g, {"X": rnd(shape, 9)}), RTOL_F32)
    assert s.plan_stats.n_kernels == 1 and s.g.blocks()[0]["family"] == "row"


def test_cumsum_counts_exactly_and_fuses_with_its_neighbours():
    # running count of ones: integers, exact in fp32
    x = (rnd((11, 4096), 10, 0.0, 1.0) > 0.7).astype(np.float32)
    g = graph(); g.ext("X", x.shape)
    g.mark_output(g.add("CumSum", ["X"], axis=-1))
    s, got, ref = run_both(W.Workload(g, {"X": x}))
    np.testing.assert_array_equal(got[g.outputs[0]].astype(np.float64), ref[g.outputs[0]])
    # Exp in front, a normalisation by the row total behind: a cumulative distribution in one kernel
    g = graph(); g.ext("X", (40, 768))
    e = g.add("Exp", ["X"])
    g.mark_output(g.add("Div", [g.add("CumSum", [e], axis=-1), g.add("ReduceSum", [e], axis=-1, keepdims=1)]))
    s = check(W.Workload(g, {"X": rnd((40, 768), 11)}), RTOL_F32)
    assert s.plan_stats.n_kernels <= 2


@pytest.mark.parametrize("shape", [(2, 12, 12, 16), (3, 7, 9, 40), (4, 56, 56, 24)])
def test_instance_normalization(shape):
    c = shape[3]
    g = graph(); g.ext("X", shape); g.ext("s", (c,), kind="weight"); g.ext("t", (c,), kind="weight")
    g.mark_output(g.add("Relu", [g.add("InstanceNorm", ["X", "s", "t"], eps=1e-5)]))
    ins = {"X": rnd(shape, 12, -1.0, 3.0), "s": rnd((c,), 13, 0.5, 1.5), "t": rnd((c,), 14, -0.5, 0.5)}
    s = check(W.Workload(g, ins), RTOL_F32)
    assert s.plan_stats.n_ops == 2


# ---- Einsum (Table 2, Many-to-Many) ---------------------------------------------------------------------------------

@pytest.mark.parametrize("eq,sa,sb,dtype", [
    ("ik,kj->ij", (130, 72), (72, 40), "f32"),
    ("ik,jk->ij", (100, 64), (48, 64), "f32"),                              # K-major second operand
    ("bik,bkj->bij", (6, 70, 32), (6, 32, 24), "f32"),
    ("nhwc,co->nhwo", (2, 20, 20, 24), (24, 48), "f32"),                   # a pointwise convolution
    ("bhqd,bhkd->bhqk", (2, 4, 128, 64), (2, 4, 128, 64), "bf16"),         # attention scores
    ("bhqk,bhkd->bhqd", (2, 4, 128, 128), (2, 4, 128, 64), "bf16"),        # probabilities times V
    ("bqhd,bkhd->bhqk", (2, 128, 4, 64), (2, 128, 4, 64), "bf16"),         # heads inside: strided head views
    ("mck,knc->nm", (33, 8, 16), (16, 40, 8), "f32"),                      # two summed labels, permuted result
    ("ik,k->i", (257, 64), (64,), "f32"),
])
def test_einsum(eq, sa, sb, dtype):
    g = graph(); g.ext("A", sa, dtype); g.ext("Bm", sb, dtype)
    g.mark_output(g.add("Einsum", ["A", "Bm"], equation=eq))
    a, b = rnd(sa, 21, -1.0, 1.0), rnd(sb, 22, -1.0, 1.0)
    if dtype == "bf16":
        a, b = W.round_to_bf16(a), W.round_to_bf16(b)
    s = check(W.Workload(g, {"A": a, "Bm": b}), 2e-2 if dtype == "bf16" else RTOL_F32)
    assert s.plan_stats.n_ops == 1


def test_einsum_with_neighbours_fuses_like_a_matrix_product():
    # bias and activation behind the contraction go into its epilogue
    g = graph(); g.ext("A", (300, 48)); g.ext("Bm", (48, 64), kind="weight"); g.ext("b", (64,), kind="weight")
    g.mark_output(g.add("Relu", [g.add("Add", [g.add("Einsum", ["A", "Bm"], equation="ik,kj->ij"), "b"])]))
    s = check(W.Workload(g, {"A": rnd((300, 48), 23, -1, 1), "Bm": rnd((48, 64), 24, -0.3, 0.3), "b": rnd((64,), 25)}), RTOL_F32, expect_blocks=1)
    assert s.g.blocks()[0]["family"] == "gemm"


@pytest.mark.parametrize("shape,axis,idx_shape", [((6, 40, 32), 1, (7,)), ((5, 9, 64), 2, (3, 4)), ((12, 8, 4, 16), 0, (5,)), ((50,), 0, (4, 6)),
                                                  ((3, 20, 8), -2, (2, 2))])
def test_gather_along_any_axis(shape, axis, idx_shape):
    g = graph("gather_axis"); g.ext("T", shape); g.ext("I", idx_shape)
    g.mark_output(g.add("Relu", [g.add("Gather", ["T", "I"], axis=axis)]))
    v = shape[axis]
    idx = np.floor(W.uniform(777, 90, idx_shape, 0.0, float(v))).clip(0, v - 1)
    s, got, ref = run_both(W.Workload(g, {"T": rnd(shape, 91), "I": idx}))
    name = g.outputs[0]
    assert np.array_equal(got[name].astype(np.float64), ref[name])          # a selection followed by max(x, 0): bit-exact
    assert s.plan_stats.n_ops == 2


@pytest.mark.parametrize("flags", [B.PLAN_FUSED, B.PLAN_UNFUSED])
@pytest.mark.parametrize("shape,k,s,p,cout", [((2, 9, 11, 16), 4, 2, 1, 8), ((1, 16, 16, 32), 3, 2, 1, 16), ((3, 5, 7, 8), 3, 1, 1, 12),
                                               ((2, 6, 6, 24), 2, 1, 0, 4), ((1, 12, 10, 16), 4, 2, 0, 32), ((2, 8, 8, 8), 5, 3, 2, 8),
                                               ((4, 28, 28, 64), 4, 2, 1, 32)])
def test_convtranspose_with_overlapping_patches(shape, k, s, p, cout, flags):
    """Transposed convolutions whose patches overlap (stride < kernel) or are cropped (pad): the pointwise convolution onto
    all k x k x Cout patch values followed by the gather that adds, per output element, the values that land on it;
    ReLU and a residual ride in the gather's epilogue."""
    n, h, w, c = shape
    ho, wo = (h - 1) * s + k - 2 * p, (w - 1) * s + k - 2 * p
    g = graph("deconv2")
    g.ext("X", shape); g.ext("Wt", (c, k, k, cout), kind="weight"); g.ext("R", (n, ho, wo, cout))
    t = g.add("Relu", [g.add("ConvTranspose", ["X", "Wt"], kernel=k, stride=s, pad=p)])
    g.mark_output(g.add("Add", [t, "R"]))
    ins = {"X": rnd(shape, 73), "Wt": rnd((c, k, k, cout), 74, -0.3, 0.3), "R": rnd((n, ho, wo, cout), 75)}
    sess = check(W.Workload(g, ins), 2e-5, flags)
    assert sess.g.tensor_info(sess.ids[g.outputs[0]])[1] == (n, ho, wo, cout)
    if flags == B.PLAN_FUSED:
        assert sess.plan_stats.n_ops == 3 and [b["ops"] for b in sess.g.blocks()][-1] == ["Col2Im", "Relu", "Add"]


@pytest.mark.parametrize("shape", [(1, 64, 64, 128), (16, 20, 20, 8), (2, 33, 17, 36), (300, 4, 4, 64)])
def test_instance_normalization_channel_group_widths(shape):
    """One image with many channels, many images with few, a channel count that leaves a narrow last group, many small
    planes: the CTA's channel group goes from one to eight 128-bit lanes; a residual and an activation ride in the epilogue."""
    c = shape[3]
    g = graph(); g.ext("X", shape); g.ext("s", (c,), kind="weight"); g.ext("t", (c,), kind="weight"); g.ext("R", shape)
    g.mark_output(g.add("LeakyRelu", [g.add("Add", [g.add("InstanceNorm", ["X", "s", "t"], eps=1e-3), "R"])], alpha=0.2))
    ins = {"X": rnd(shape, 12, -1.0, 5.0), "s": rnd((c,), 13, 0.5, 1.5), "t": rnd((c,), 14, -0.5, 0.5), "R": rnd(shape, 15)}
    s = check(W.Workload(g, ins), RTOL_F32, expect_blocks=1)
    assert s.g.blocks()[0]["family"] == "instnorm"


@pytest.mark.parametrize("flags", [B.PLAN_FUSED, B.PLAN_UNFUSED])
def test_style_transfer_decoder(flags):
    """Residual block with instance normalisation, two overlapping transposed convolutions, Tanh head."""
    wl = W.style_decoder(n=2, hw=24, c=32)
    s = check(wl, 2e-4, flags)
    if flags == B.PLAN_FUSED:
        fams = [b["family"] for b in s.g.blocks() if b["family"] != "alias"]
        assert fams.count("instnorm") == 4 and fams.count("pool") == 2 and s.plan_stats.n_kernels == 11, s.g.blocks()
