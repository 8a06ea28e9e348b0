"""Parity of the CUDA path (through the C ABI) with the oracle, element by element.

Tolerances: bit-exact for pure Reorganize/Shuffle blocks; 1e-5 relative for fp32
element-wise and reduction chains; 2e-2 relative for bf16 GEMM-anchored blocks."""
import itertools

import numpy as np
import pytest

from paper_2108_13342_b200 import binding as B
from paper_2108_13342_b200 import workloads as W
from oracle import interp as O
from util import RTOL_BF16, RTOL_F32, check, close, graph, rnd, run_both

pytestmark = pytest.mark.gpu

FUSED, UNFUSED = B.PLAN_FUSED, B.PLAN_UNFUSED


# ---- workload 1: bias + scale + swish + NCHW->NHWC -------------------------------

@pytest.mark.parametrize("shape", [(1, 64, 56, 56), (2, 3, 5, 7), (3, 8, 4, 12), (1, 130, 9, 9), (2, 64, 1, 100)])
@pytest.mark.parametrize("flags", [FUSED, UNFUSED])
def test_swish_transpose(shape, flags):
    n, c, h, w = shape
    check(W.swish_transpose(n, c, h, w), RTOL_F32, flags, expect_blocks=1 if flags == FUSED else 5)


# ---- workload 2a / 2b ---------------------------------------------------------------

@pytest.mark.parametrize("cfg", [(8, 12, 128), (1, 2, 16), (2, 3, 17), (1, 1, 3), (2, 1, 257), (1, 2, 640), (1, 1, 1500)])
@pytest.mark.parametrize("flags", [FUSED, UNFUSED])
def test_masked_softmax(cfg, flags):
    b, h, s = cfg
    wl = W.masked_softmax(b, h, s)
    sess, got, ref = run_both(wl, flags)
    assert sess.plan_stats.n_kernels == (1 if flags == FUSED else 3)
    close(got["P"], ref["P"], RTOL_F32)
    p = got["P"]
    assert np.all(p[..., 0, 1:] == 0.0) and np.all(p[..., 0, 0] == 1.0)      # causal row 0 is one-hot
    assert np.max(np.abs(p.sum(-1) - 1.0)) < 1e-5


@pytest.mark.parametrize("cfg", [(1024, 768), (5, 48), (3, 770), (7, 1536), (2, 4096), (9, 1), (4, 33), (130, 256)])
@pytest.mark.parametrize("flags", [FUSED, UNFUSED])
def test_add_layernorm_gelu(cfg, flags):
    rows, hidden = cfg
    check(W.add_layernorm_gelu(rows, hidden), RTOL_F32, flags, expect_blocks=1 if flags == FUSED else 3)


# ---- pure Reorganize / Shuffle blocks: bit-exact --------------------------------------

def _special_values(shape, seed):
    x = rnd(shape, seed).astype(np.float32)
    flat = x.reshape(-1)
    specials = np.array([0.0, -0.0, np.inf, -np.inf, 1e-45, -1e-45, 1.17549435e-38, 3.4028235e38], dtype=np.float32)
    k = min(len(specials), flat.size)
    flat[:k] = specials[:k]
    return x


@pytest.mark.parametrize("shape", [(2, 3, 5, 7), (4, 64, 33), (65, 130), (1, 8, 128, 64), (3, 1, 5, 1)])
def test_transpose_all_perms_bit_exact_f32(shape):
    x = _special_values(shape, 3)
    for perm in itertools.permutations(range(len(shape))):
        g = graph()
        g.ext("X", shape)
        g.mark_output(g.add("Transpose", ["X"], perm=perm, out="Y"))
        s, got, ref = run_both(W.Workload(g, {"X": x}))
        y = s.buffers["Y"].cpu().numpy()
        assert np.array_equal(y.view(np.uint32), np.transpose(x, perm).copy().view(np.uint32)), perm
        assert np.array_equal(got["Y"], ref["Y"])


def test_transpose_bf16_bit_exact_with_nan_payloads():
    import torch
    shape = (2, 12, 40, 64)
    bits = (np.arange(int(np.prod(shape)), dtype=np.uint32) * 2654435761 >> 7).astype(np.uint16).reshape(shape)
    bits.reshape(-1)[:4] = [0x7FC1, 0xFFA5, 0x7F80, 0x8000]      # NaN payloads, inf, -0
    g = graph()
    g.ext("X", shape, "bf16")
    g.mark_output(g.add("Transpose", ["X"], perm=(0, 2, 1, 3), out="Y"))
    wl = W.Workload(g, {"X": W.bf16_bits_to_f32(bits)})
    from paper_2108_13342_b200.runtime import Session
    s = Session(wl, rewrite_flags=B.REWRITE_NONE, upload=False)
    xb = torch.from_numpy(bits.view(np.int16)).to("cuda").view(torch.bfloat16)
    s.buffers["X"] = xb
    s.g.bind(s.ids["X"], xb.data_ptr())
    s.run()
    torch.cuda.synchronize()
    y = s.buffers["Y"].view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(y, np.transpose(bits, (0, 2, 1, 3)))


def test_reshape_slice_split_are_exact():
    x = _special_values((6, 10, 8), 5)
    g = graph()
    g.ext("X", x.shape)
    a, b, c = g.add("Split", ["X"], n_out=3, axis=1, sizes=(2, 5, 3))
    r = g.add("Reshape", [b], shape=(6, 40), out="R")
    t = g.add("Transpose", [c], perm=(2, 0, 1), out="T")
    f = g.add("Flatten", [a], axis=1, out="F")
    for n in (r, t, f):
        g.mark_output(n)
    s, got, ref = run_both(W.Workload(g, {"X": x}))
    for n in ("R", "T", "F"):
        assert np.array_equal(got[n], ref[n]), n


# ---- every element-wise operator, alone and in chains ----------------------------------

UNARY = [("Sigmoid", {}, (-8, 8)), ("Tanh", {}, (-4, 4)), ("Erf", {}, (-3, 3)), ("Exp", {}, (-10, 10)),
         ("Log", {}, (0.1, 50)), ("Sqrt", {}, (0.0, 9)), ("Abs", {}, (-2, 2)), ("Neg", {}, (-2, 2)),
         ("Recip", {}, (0.5, 4)), ("Square", {}, (-3, 3)), ("Relu", {}, (-2, 2)), ("Clip", {"lo": 0.0, "hi": 6.0}, (-3, 9)),
         ("Pow", {"p": 3.0}, (0.2, 2)), ("Pow", {"p": 2.0}, (-2, 2)), ("Gelu", {"approx": "erf"}, (-5, 5)),
         ("Gelu", {"approx": "tanh"}, (-5, 5)), ("MulC", {"c": -1.75}, (-2, 2)), ("AddC", {"c": 0.375}, (-2, 2))]


@pytest.mark.parametrize("case", UNARY, ids=lambda c: c[0] + str(c[1].get("p", "")) + str(c[1].get("approx", "")))
def test_unary_ops(case):
    op, attrs, (lo, hi) = case
    for shape in [(1000, 36), (7, 13)]:
        g = graph()
        g.ext("X", shape)
        g.mark_output(g.add(op, ["X"], out="Y", **attrs))
        check(W.Workload(g, {"X": rnd(shape, 11, lo, hi)}), RTOL_F32)


@pytest.mark.parametrize("op", ["Add", "Sub", "Mul", "Div"])
@pytest.mark.parametrize("bshape", [(4, 6, 20), (20,), (6, 1), (4, 1, 1), (1,), (4, 1, 20)])
@pytest.mark.parametrize("swap", [False, True])
def test_binary_broadcast(op, bshape, swap):
    a = rnd((4, 6, 20), 12, 0.5, 2.0); b = rnd(bshape, 13, 0.5, 2.0)
    g = graph()
    g.ext("A", a.shape); g.ext("B", bshape)
    g.mark_output(g.add(op, ["B", "A"] if swap else ["A", "B"], out="Y"))
    check(W.Workload(g, {"A": a, "B": b}), RTOL_F32)


def test_long_chain_with_shared_subexpressions_and_two_outputs():
    # t1 = A*B ; out = Recip(t1*C) + t1*D   (the data-flow tree of the paper's code-generation example:
    # t1 feeds both products and is computed once); t1 itself is also an output (not removable).
    shape = (33, 100)
    ins = {k: rnd(shape, 20 + i, 0.5, 2.0) for i, k in enumerate("ABCD")}
    g = graph()
    for k in "ABCD":
        g.ext(k, shape)
    t1 = g.add("Mul", ["A", "B"], out="T1")
    t2 = g.add("Mul", [t1, "C"])
    t3 = g.add("Recip", [t2])
    t5 = g.add("Mul", [t1, "D"])
    o = g.add("Add", [t3, t5], out="Out")
    g.mark_output(o); g.mark_output(t1)
    s = check(W.Workload(g, ins), RTOL_F32, expect_blocks=1)
    assert s.g.blocks()[0]["n_microops"] <= 11      # 5 arithmetic ops, 2 stores, 2 saves, 2 moves


def test_chain_of_24_ops():
    shape = (64, 52)
    g = graph()
    g.ext("X", shape); g.ext("Y", shape)
    t = "X"
    for i in range(8):
        t = g.add("Add", [t, "Y"]); t = g.add("MulC", [t], c=0.9); t = g.add("Tanh", [t])
    g.mark_output(g.add("Abs", [t], out="Z"))
    check(W.Workload(g, {"X": rnd(shape, 30), "Y": rnd(shape, 31)}), RTOL_F32, expect_blocks=1)


def test_scaleshift_nchw_and_nhwc():
    x = rnd((2, 5, 6, 8), 40)
    for axis, c in ((1, 5), (-1, 8)):
        g = graph()
        g.ext("X", x.shape); g.ext("s", (c,)); g.ext("t", (c,))
        y = g.add("ScaleShift", ["X", "s", "t"], axis=axis)
        g.mark_output(g.add("Clip", [y], lo=0.0, hi=6.0, out="Y"))
        check(W.Workload(g, {"X": x, "s": rnd((c,), 41, 0.5, 1.5), "t": rnd((c,), 42)}), RTOL_F32, expect_blocks=1)


# ---- reductions ----------------------------------------------------------------------------

@pytest.mark.parametrize("op", ["ReduceSum", "ReduceMean", "ReduceMax", "ReduceProd"])
@pytest.mark.parametrize("keep", [0, 1])
@pytest.mark.parametrize("shape", [(6, 5, 128), (50, 37), (3, 2000)])
def test_reductions(op, keep, shape):
    g = graph()
    g.ext("X", shape)
    t = g.add("MulC", ["X"], c=1.01)
    g.mark_output(g.add(op, [t], axis=-1, keepdims=keep, out="Y"))
    lo, hi = (0.98, 1.02) if op == "ReduceProd" else (-2, 2)
    check(W.Workload(g, {"X": rnd(shape, 50, lo, hi)}), RTOL_F32, expect_blocks=1)


def test_layernorm_from_primitives_unfused_and_strict():
    # the 9-operator expansion runs as separate row / element-wise kernels and still matches
    g = graph()
    g.ext("x", (40, 96)); g.ext("g", (96,)); g.ext("b", (96,))
    g.mark_output(W._layernorm_primitives(g, "x", "g", "b", 1e-5))
    wl = W.Workload(g, {"x": rnd((40, 96), 60), "g": rnd((96,), 61, 0.9, 1.1), "b": rnd((96,), 62)})
    check(wl, RTOL_F32, UNFUSED)
    check(wl, RTOL_F32, FUSED)


def test_tensor_read_outside_its_block_is_written_in_full_when_a_slice_follows():
    """t = X + b is a graph output AND feeds Slice -> Relu.  A block {Add, Slice, Relu} would iterate over the slice
    only and leave two thirds of t unwritten: the planner has to keep the Slice out of the block that stores t."""
    g = graph()
    g.ext("X", (4, 8, 12)); g.ext("b", (12,))
    t = g.add("Add", ["X", "b"], out="T")
    g.mark_output(t)
    s = g.add("Slice", [t], axis=-1, start=4, end=8)
    g.mark_output(g.add("Relu", [s], out="Y"))
    wl = W.Workload(g, {"X": rnd((4, 8, 12), 1), "b": rnd((12,), 2)})
    sess = Session_poisoned(wl)
    ref = O.run_graph(wl.graph, wl.inputs)
    for n in ("T", "Y"):
        close(sess.output(n), ref[n], RTOL_F32)


def Session_poisoned(wl):
    """A session whose output buffers start as NaN: an element that no kernel writes is caught."""
    from paper_2108_13342_b200.runtime import Session
    s = Session(wl, plan_flags=B.PLAN_FUSED, rewrite_flags=B.REWRITE_NONE)
    for n in wl.graph.outputs:
        s.buffers[n].fill_(float("nan"))
    s.run()
    assert s.g.status()[0] == 0
    return s


def test_profiling_database_measured_on_the_device_drives_the_plan():
    """Section 4.3: candidate blocks of profile-dependent decisions are measured on the device, the plan is rebuilt
    from the measurements alone, and it still computes the oracle's result."""
    import torch
    from paper_2108_13342_b200 import profile_db
    B.profile_db_clear()
    wl = W.encoder(layers=1, batch=2, seq=32, hidden=64, heads=4, ffn=128)
    rounds = profile_db.fill(wl.graph, torch.device("cuda:0"), B.REWRITE_CANON_MACRO, scratch_bytes=64 << 20, iters=5)
    assert rounds[0]["misses"] > 0 and rounds[0]["measured"] == rounds[0]["misses"], rounds
    assert rounds[-1]["misses"] == 0 and rounds[-1]["hits"] > 0, rounds
    assert B.profile_db_size() >= rounds[0]["measured"]
    try:
        s, got, ref = run_both(wl, B.PLAN_FUSED, B.REWRITE_CANON_MACRO)
        (name,) = wl.graph.outputs
        close(got[name], ref[name], RTOL_BF16)
        assert s.plan_stats.n_profile_misses == 0
    finally:
        B.profile_db_clear()


def test_bounded_wait_expires_and_the_graph_runs_on():
    """The failure path of the tensor-core kernels without a failure: a wait on a barrier that nothing signals gives up
    after its limit (1 ms here), the status words report DNNF_ERR_TIMEOUT, nothing hangs or faults, and after the
    caller has cleared the status words the graph runs and is correct again."""
    import time
    import torch
    wl = W.ffn_block(m=256, hidden=128, ffn=256)
    s, got, ref = run_both(wl)
    close(got["Y"], ref["Y"], RTOL_BF16)
    stream = torch.cuda.current_stream().cuda_stream
    t0 = time.perf_counter()
    s.g.selftest_wait_expiry(1_000_000, stream)
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 0.5                      # it gave up after about a millisecond, not a second
    assert s.g.status() == (B.ERR_TIMEOUT, -2)
    s.workspace[: s.g.workspace_zero_bytes()].zero_()
    s.buffers["Y"].fill_(float("nan"))
    s.run()
    close(s.output("Y"), ref["Y"], RTOL_BF16)
    assert s.g.status() == (0, -1)
    with pytest.raises(B.DnnfError):
        s.g.selftest_wait_expiry(10**12, stream)               # limits beyond 100 ms are refused
