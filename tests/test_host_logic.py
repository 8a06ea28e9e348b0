"""Host-side logic through the C ABI (no GPU needed): exported symbols, mapping types
(Table 2), the Table 3 reconstruction, graph rewriting (Table 4 with its #FLOPS counts),
fusion-plan generation (Listing 1 and the worked examples in the text), IR_removable,
the data-flow-tree linearisation, and the error / state behaviour of the boundary."""
import ctypes
import os
import re

import pytest

from paper_2108_13342_b200 import binding as B
from paper_2108_13342_b200 import workloads as W
from paper_2108_13342_b200.runtime import build_graph

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
OO, RE, SH, OM, MM = B.ONE_TO_ONE, B.REORGANIZE, B.SHUFFLE, B.ONE_TO_MANY, B.MANY_TO_MANY


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "dnnf.h")).read()
    declared = set(re.findall(r"DNNF_API\s+[\w\s\*]+?\b(dnnf_\w+)\s*\(", hdr))
    assert len(declared) >= 25
    lib = ctypes.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(B.EXPORTS), declared ^ set(B.EXPORTS)


# ---- Table 2 and the most-complex-pair rule ------------------------------------------------

def _one_op_graph(op, in_shapes, **attrs):
    g = B.Graph()
    ids = [g.add_tensor(f"i{k}", B.F32, s) for k, s in enumerate(in_shapes)]
    g.add_op(op, ids, **attrs)
    return g


@pytest.mark.parametrize("op,shapes,attrs,expect", [
    ("Add", [(4, 8), (4, 8)], {}, OO), ("Relu", [(4, 8)], {}, OO), ("Clip", [(4, 8)], {"lo": 0, "hi": 6}, OO),
    ("Erf", [(4, 8)], {}, OO), ("Exp", [(4, 8)], {}, OO), ("Sigmoid", [(4, 8)], {}, OO), ("Sqrt", [(4, 8)], {}, OO),
    ("Tanh", [(4, 8)], {}, OO), ("Recip", [(4, 8)], {}, OO), ("Slice", [(4, 8)], {"axis": 1, "start": 0, "end": 4}, OO),
    ("ScaleShift", [(2, 4, 4, 8), (8,), (8,)], {"axis": -1}, OO),
    ("Add", [(4, 8), (8,)], {}, OM), ("Mul", [(4, 8), (4, 1)], {}, OM), ("Expand", [(1, 8)], {"shape": (4, 8)}, OM),
    ("MatMul", [(4, 8), (8, 16)], {}, MM), ("Conv1x1", [(1, 4, 4, 8), (8, 16)], {}, MM), ("Softmax", [(4, 8)], {"axis": -1}, MM),
    ("ReduceSum", [(4, 8)], {"axis": -1}, MM), ("ReduceMean", [(4, 8)], {"axis": -1}, MM), ("ReduceProd", [(4, 8)], {"axis": -1}, MM),
    ("LayerNorm", [(4, 8), (8,), (8,)], {"axis": -1}, MM), ("DwConv3x3", [(1, 4, 4, 8), (3, 3, 8)], {}, MM),
    ("Reshape", [(4, 8)], {"shape": (8, 4)}, RE), ("Flatten", [(2, 4, 8)], {"axis": 1}, RE), ("Squeeze", [(4, 1, 8)], {"axes": (1,)}, RE),
    ("Unsqueeze", [(4, 8)], {"axes": (0,)}, RE), ("Transpose", [(4, 8)], {"perm": (1, 0)}, SH)])
def test_operator_mapping_types(op, shapes, attrs, expect):
    assert _one_op_graph(op, shapes, **attrs).op_mapping(0) == expect


# ---- Table 3 ------------------------------------------------------------------------------------

def test_table3_has_23_fusable_cells_and_the_two_named_red_ones():
    cells = {(a, b): B.mapping_check(a, b) for a in range(5) for b in range(5)}
    red = [k for k, v in cells.items() if v[1] == B.RED]
    assert sorted(red) == [(OM, MM), (MM, MM)]          # Expand->Conv and Conv->Conv
    assert sum(1 for v in cells.values() if v[1] != B.RED) == 23     # one code-generation rule each
    for t in range(5):                                  # One-to-One takes the partner's type, green, either order
        assert cells[(OO, t)] == (t, B.GREEN) and cells[(t, OO)] == (t, B.GREEN)
    for rs in (RE, SH):                                 # Reorganize/Shuffle with One-to-Many / Many-to-Many: profile
        for strong in (OM, MM):
            assert cells[(rs, strong)] == (strong, B.YELLOW) and cells[(strong, rs)] == (strong, B.YELLOW)
    assert cells[(MM, OM)][1] == B.YELLOW               # Conv -> Expand / Resize
    assert cells[(RE, SH)][1] == B.GREEN and cells[(SH, SH)] == (SH, B.GREEN)


# ---- Table 4 -----------------------------------------------------------------------------------

M_, N_ = 6, 10
MN = M_ * N_


def _g(names=("A", "B", "C")):
    g = W.GraphDesc()
    for n in names:
        g.ext(n, (M_, N_))
    return g


def _rewrite(desc, flags=B.REWRITE_DEFAULT):
    g, ids = build_graph(desc)
    st = g.rewrite(flags)
    kinds = sorted(B.OP_NAMES[k] for k, alive in (g.op_kind(i) for i in range(g.op_count())) if alive)
    return g, st, kinds


def test_rewrite_associative_rows():
    g = _g(("A", "B"))
    g.mark_output(g.add("Mul", [g.add("Recip", ["A"]), g.add("Recip", [g.add("Mul", ["A", "B"])])]))
    _, st, kinds = _rewrite(g)
    assert (st.flops_before, st.flops_after) == (4 * MN, 4 * MN) and kinds == ["Mul", "Recip", "Recip", "Square"]

    g = _g()
    g.mark_output(g.add("Mul", [g.add("Mul", ["A", g.add("Sqrt", ["B"])]), g.add("Mul", [g.add("Sqrt", ["B"]), "C"])]))
    _, st, kinds = _rewrite(g)
    assert (st.flops_before, st.flops_after) == (5 * MN, 2 * MN) and kinds == ["Mul", "Mul"]

    g = _g()
    g.mark_output(g.add("Mul", [g.add("Mul", [g.add("Abs", ["A"]), "B"]), g.add("Abs", ["C"])]))
    _, st, kinds = _rewrite(g)
    assert (st.flops_before, st.flops_after) == (4 * MN, 3 * MN) and kinds == ["Abs", "Mul", "Mul"]

    g = _g()
    r1 = g.add("ReduceSum", ["B"], axis=-1, keepdims=1); r2 = g.add("ReduceSum", ["B"], axis=-1, keepdims=1)
    g.mark_output(g.add("Mul", [g.add("Mul", ["A", r1]), g.add("Mul", [r2, "C"])]))
    _, st, kinds = _rewrite(g)
    assert (st.flops_before, st.flops_after) == (5 * MN, 3 * MN + M_) and kinds == ["Mul", "Mul", "ReduceSum", "Square"]


def test_rewrite_distributive_rows():
    g = _g()
    g.mark_output(g.add("Add", [g.add("Mul", ["A", "C"]), g.add("Mul", ["B", "C"])]))
    _, st, kinds = _rewrite(g)
    assert (st.flops_before, st.flops_after) == (3 * MN, 2 * MN) and kinds == ["Add", "Mul"]

    g = _g(("A", "B"))
    g.mark_output(g.add("Add", ["A", g.add("Mul", ["A", "B"])]))
    _, st, kinds = _rewrite(g)
    assert (st.flops_before, st.flops_after) == (2 * MN, 2 * MN) and kinds == ["AddC", "Mul"]

    g = _g()
    s1 = g.add("Add", ["A", "B"]); s2 = g.add("Add", ["A", "B"])
    g.mark_output(g.add("Sub", [g.add("Square", [s1]), g.add("Mul", [s2, "C"])]))
    _, st, kinds = _rewrite(g)
    assert (st.flops_before, st.flops_after) == (5 * MN, 3 * MN) and kinds == ["Add", "Mul", "Sub"]


def test_rewrite_commutative_rows():
    g = _g(("A",))
    g.mark_output(g.add("ReduceSum", [g.add("BitShift", ["A"], bits=3)], axis=-1, keepdims=1))
    gg, st, kinds = _rewrite(g)
    assert (st.flops_before, st.flops_after) == (2 * MN, MN + M_) and kinds == ["BitShift", "ReduceSum"]
    order = [B.OP_NAMES[gg.op_kind(i)[0]] for i in range(gg.op_count()) if gg.op_kind(i)[1]]
    assert order == ["ReduceSum", "BitShift"]

    g = _g(("A",))
    g.mark_output(g.add("ReduceProd", [g.add("Exp", ["A"])], axis=-1, keepdims=1))
    _, st, kinds = _rewrite(g)
    assert (st.flops_before, st.flops_after) == (2 * MN, MN + M_) and kinds == ["Exp", "ReduceSum"]


def test_rewrite_is_greedy_largest_gain_first_and_reaches_a_fixed_point():
    # two independent sites: the sqrt pair saves 3mn, the common factor 1mn; both must be gone at the end
    g = _g(("A", "B", "C", "D"))
    p = g.add("Mul", [g.add("Mul", ["A", g.add("Sqrt", ["B"])]), g.add("Mul", [g.add("Sqrt", ["B"]), "C"])])
    q = g.add("Add", [g.add("Mul", ["A", "D"]), g.add("Mul", ["C", "D"])])
    g.mark_output(g.add("Sub", [p, q]))
    gg, st, kinds = _rewrite(g)
    assert st.flops_before == 9 * MN and st.flops_after == 5 * MN and st.rules_applied >= 2
    st2 = gg.rewrite(B.REWRITE_DEFAULT)
    assert st2.rules_applied == 0 and st2.flops_after == 5 * MN
    _, st3, _ = _rewrite(g, B.REWRITE_NONE)
    assert st3.flops_after == 9 * MN and st3.rules_applied == 0


def test_canonicalise_layernorm_flag():
    wl = W.encoder(layers=1, batch=2, seq=8, hidden=16, heads=2, ffn=32)
    g, st, kinds = _rewrite(wl.graph, B.REWRITE_CANON_MACRO)
    assert kinds.count("LayerNorm") == 2 and "ReduceMean" not in kinds and st.ops_after == st.ops_before - 16
    g2, st2, kinds2 = _rewrite(wl.graph)
    assert "LayerNorm" not in kinds2 and kinds2.count("Square") == 2 and "Pow" not in kinds2     # Pow(x,2) -> Square only


# ---- Listing 1 -----------------------------------------------------------------------------------

def _block_sets(g):
    return [tuple(b["ops"]) for b in g.blocks()]


def test_plan_example_of_section_4_3():
    # GEMM -> Add -> Conv -> Relu -> Mul -> Sub with equal result sizes: Add is the first seed, the successor pass
    # gives {Add, Conv, Relu, Mul, Sub} (Many-to-Many), and the predecessor GEMM is refused (Many-to-Many with
    # Many-to-Many is red).  Add sits in FRONT of Conv, so the plan is made with the literal Listing 1 (planning only).
    g = W.GraphDesc()
    g.ext("X", (1, 4, 4, 8)); g.ext("Wg", (8, 8)); g.ext("b", (1, 4, 4, 8)); g.ext("Wc", (8, 8)); g.ext("s", (1, 4, 4, 8)); g.ext("t", (1, 4, 4, 8))
    y = g.add("MatMul", ["X", "Wg"])
    y = g.add("Add", [y, "b"]); y = g.add("Conv1x1", [y, "Wc"]); y = g.add("Relu", [y]); y = g.add("Mul", [y, "s"])
    g.mark_output(g.add("Sub", [y, "t"]))
    gg, _ = build_graph(g)
    st = gg.plan(B.PLAN_ALLOW_PROLOGUE)
    assert st.n_blocks == 2
    assert sorted(_block_sets(gg), key=len) == [("MatMul",), ("Add", "Conv1x1", "Relu", "Mul", "Sub")]
    assert [b["mapping"] for b in gg.blocks() if len(b["ops"]) == 5] == ["Many-to-Many"]
    with pytest.raises(B.DnnfError) as e:          # such a plan is not executable here
        gg.workspace_size()
    assert e.value.code == B.ERR_STATE
    # the executable profile keeps One-to-One operators out of the front of a contraction anchor
    gg, _ = build_graph(g)
    gg.plan(B.PLAN_FUSED)
    assert sorted(_block_sets(gg)) == [("Conv1x1", "Relu", "Mul", "Sub"), ("MatMul", "Add")]


def test_chains_the_paper_names_fuse_into_one_block():
    # MatMul + Reshape + Transpose + Add (GPT-2)
    g = W.GraphDesc()
    g.ext("X", (16, 32), "bf16"); g.ext("Wt", (32, 64), "bf16"); g.ext("b", (64,))
    y = g.add("MatMul", ["X", "Wt"]); y = g.add("Add", [y, "b"]); y = g.add("Reshape", [y], shape=(16, 4, 16))
    g.mark_output(g.add("Transpose", [y], perm=(1, 0, 2)))
    gg, _ = build_graph(g)
    assert gg.plan().n_blocks == 1 and gg.blocks()[0]["family"] == "gemm"
    # Sub + Pow + ReduceMean + Add + Sqrt (TinyBERT)
    g = W.GraphDesc()
    g.ext("X", (8, 64)); g.ext("mu", (8, 1))
    y = g.add("Sub", ["X", "mu"]); y = g.add("Pow", [y], p=2.0); y = g.add("ReduceMean", [y], axis=-1, keepdims=1)
    y = g.add("AddC", [y], c=1e-5); g.mark_output(g.add("Sqrt", [y]))
    gg, _ = build_graph(g)
    assert gg.plan().n_blocks == 1 and gg.blocks()[0]["family"] == "row"
    # GEMM + Div + Transpose: Transpose and Div fuse first (Shuffle), GEMM stores through the resulting index map
    g = W.GraphDesc()
    g.ext("X", (16, 32), "bf16"); g.ext("Wt", (32, 64), "bf16"); g.ext("d", (16, 64))
    y = g.add("MatMul", ["X", "Wt"]); y = g.add("Div", [y, "d"]); g.mark_output(g.add("Transpose", [y], perm=(1, 0)))
    gg, _ = build_graph(g)
    assert gg.plan().n_blocks == 1 and gg.block_program(0) == "MOV anchor; DIV in0; STORE out0"


def test_config_plans_and_strict_table3():
    cases = [(W.swish_transpose(), 1, 1), (W.masked_softmax(), 1, 2), (W.add_layernorm_gelu(), 1, 1),
             (W.ffn_block(m=256, hidden=64, ffn=128), 2, 2), (W.mbconv_block(n=1, h=8, w=8), 3, 3)]
    for wl, fused, strict in cases:
        g, _ = build_graph(wl.graph)
        assert g.plan(B.PLAN_FUSED).n_kernels == fused, wl.graph.name
        g, _ = build_graph(wl.graph)
        assert g.plan(B.PLAN_STRICT_TABLE3).n_kernels == strict, wl.graph.name
        g, _ = build_graph(wl.graph)
        st = g.plan(B.PLAN_UNFUSED)
        assert st.n_kernels == len(wl.graph.ops) and abs(st.fusion_rate - 1.0) < 1e-9


def test_encoder_plan_kernel_counts_and_fusion_rate():
    wl = W.encoder(layers=2, batch=2, seq=16, hidden=32, heads=2, ffn=64)
    g, _ = build_graph(wl.graph)
    g.rewrite(B.REWRITE_CANON_MACRO)
    st = g.plan()
    assert st.n_kernels == 2 * 9 and st.n_ops == 2 * 32 and st.irs_bytes_fused < st.irs_bytes_unfused / 3
    g, _ = build_graph(wl.graph)
    g.rewrite(B.REWRITE_NONE)
    st = g.plan()
    assert st.n_kernels == 2 * 11 and abs(st.fusion_rate - 96 / 22) < 1e-9
    fams = [b["family"] for b in g.blocks()][:11]
    assert fams == ["gemm", "gemm", "row", "gemm", "gemm", "row", "row", "gemm", "gemm", "row", "row"]


def test_ir_removable_a_tensor_with_an_outside_consumer_is_stored():
    g = W.GraphDesc()
    g.ext("X", (8, 32)); g.ext("Y", (8, 32)); g.ext("Wm", (32, 16))
    t = g.add("Add", ["X", "Y"], out="T")
    g.mark_output(g.add("Relu", [t], out="R"))
    g.mark_output(g.add("MatMul", [t, "Wm"], out="S"))         # second consumer: a contraction takes no prologue, other block
    gg, ids = build_graph(g)
    st = gg.plan()
    progs = [gg.block_program(b) for b in range(gg.block_count())]
    assert st.irs_bytes_fused == 8 * 32 * 4 and any(p.count("STORE") == 2 for p in progs)


def test_data_flow_tree_shares_common_subtrees():
    # Out = Recip(A*B*C) + (A*B)*D : A*B feeds both products and is evaluated once (Section 4.4)
    g = W.GraphDesc()
    for n in "ABCD":
        g.ext(n, (8, 16))
    t1 = g.add("Mul", ["A", "B"]); t3 = g.add("Recip", [g.add("Mul", [t1, "C"])]); t5 = g.add("Mul", [t1, "D"])
    g.mark_output(g.add("Add", [t3, t5]))
    gg, _ = build_graph(g)
    assert gg.plan().n_blocks == 1
    prog = gg.block_program(0)
    assert prog.count("MUL") == 3 and prog.count("in0") == 1 and prog.count("in1") == 1 and "SAVE t0" in prog
    assert gg.blocks()[0]["mapping"] == "One-to-One"


# ---- errors and the state machine ------------------------------------------------------------

def test_errors_leave_the_graph_usable():
    g = B.Graph()
    a = g.add_tensor("a", B.F32, (4, 8)); b = g.add_tensor("b", B.F32, (5, 8))
    with pytest.raises(B.DnnfError) as e:
        g.add_op("Add", [a, b])
    assert e.value.code == B.ERR_SHAPE
    with pytest.raises(B.DnnfError) as e:
        g.add_op("Transpose", [a], perm=(0, 0))
    assert e.value.code == B.ERR_SHAPE
    with pytest.raises(B.DnnfError) as e:
        g.add_op(999, [a])
    assert e.value.code == B.ERR_UNSUPPORTED_OP
    with pytest.raises(B.DnnfError) as e:
        g.add_op("Relu", [77])
    assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(B.DnnfError) as e:
        g.plan()
    assert e.value.code == B.ERR_STATE                      # nothing added yet
    (y,) = g.add_op("Relu", [a])
    with pytest.raises(B.DnnfError) as e:
        g.plan()
    assert e.value.code == B.ERR_STATE                      # no output marked
    with pytest.raises(B.DnnfError) as e:
        g.mark_output(a)
    assert e.value.code == B.ERR_INVALID_ARG
    g.mark_output(y)
    with pytest.raises(B.DnnfError) as e:
        g.run(0)
    assert e.value.code == B.ERR_STATE                      # run before plan
    assert g.plan().n_blocks == 1
    with pytest.raises(B.DnnfError) as e:
        g.add_op("Relu", [y])
    assert e.value.code == B.ERR_STATE                      # graph is frozen after plan
    with pytest.raises(B.DnnfError) as e:
        g.rewrite()
    assert e.value.code == B.ERR_STATE
    with pytest.raises(B.DnnfError) as e:
        g.bind(a, 0)
    assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(B.DnnfError) as e:
        g.bind(a, 0x1008)                                   # not 16-byte aligned
    assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(B.DnnfError) as e:
        g.run(0)
    assert e.value.code == B.ERR_UNBOUND and "not bound" in str(e.value)
    with pytest.raises(B.DnnfError) as e:
        g.bind_workspace(0x1000, 0)
    assert e.value.code == B.ERR_WORKSPACE


def test_unsupported_block_fails_the_plan_instead_of_falling_back():
    g = W.GraphDesc()
    g.ext("A", (4, 8))
    g.mark_output(g.add("BitShift", ["A"], bits=2))
    gg, _ = build_graph(g)
    with pytest.raises(B.DnnfError) as e:
        gg.plan()
    assert e.value.code == B.ERR_UNSUPPORTED_OP


def test_product_of_three_equal_computed_factors_is_handled():
    """x*x*x with x computed inside the graph: the associative Square rule is tried (Square(x) * x has the same #FLOPS,
    so it need not be kept); the placeholder for the not-yet-created Square must not be looked up as a tensor by the
    next simplification step (that was an out-of-bounds read)."""
    g = W.GraphDesc("cube")
    g.ext("A", (8, 16)); g.ext("Bv", (16,))
    x = g.add("Add", ["A", "Bv"])
    x2 = g.add("Mul", [x, x])
    g.mark_output(g.add("Mul", [x2, x], out="Y"))
    G = build_graph(g)[0]
    st = G.rewrite(B.REWRITE_DEFAULT)
    kinds = sorted(B.OP_NAMES[G.op_kind(i)[0]] for i in range(G.op_count()) if G.op_kind(i)[1])
    assert kinds in (["Add", "Mul", "Mul"], ["Add", "Mul", "Square"]), kinds
    assert st.ops_after == 3 and st.flops_after <= st.flops_before


# ---- profiling database (Section 4.3, Step 2.3) ----------------------------------------------------

def _matmul_then_transpose():
    g = W.GraphDesc("mm_t")
    g.ext("A", (512, 64), "bf16"); g.ext("Bm", (64, 256), "bf16")
    t = g.add("MatMul", ["A", "Bm"])
    t = g.add("Relu", [t])                      # the One-to-One seed of Listing 1
    g.mark_output(g.add("Transpose", [t], perm=(1, 0), out="Y"))
    return g


def test_profile_database_round_trip(tmp_path):
    B.profile_db_clear()
    assert B.profile_db_size() == 0 and B.profile_db_get("x|y") is None
    B.profile_db_set("gemm|MatMul|bf16,bf16,->bf16,|M1N2K3B1v0|bytes10", 12.5)
    B.profile_db_set("row|Softmax|f32,->f32,|rows8L16|bytes1024", 3.25)
    assert B.profile_db_size() == 2
    assert B.profile_db_get("row|Softmax|f32,->f32,|rows8L16|bytes1024") == 3.25
    path = str(tmp_path / "db.tsv")
    B.profile_db_save(path)
    B.profile_db_clear()
    assert B.profile_db_load(path) == 2
    assert B.profile_db_get("gemm|MatMul|bf16,bf16,->bf16,|M1N2K3B1v0|bytes10") == 12.5
    with pytest.raises(ValueError):
        B.profile_db_set("bad", -1.0)
    B.profile_db_clear()


def test_yellow_decision_follows_the_profiling_database():
    """Many-to-Many followed by Shuffle is a profile-dependent (yellow) cell of Table 3: with measured latencies in
    the database the planner fuses exactly when the fused block is not slower than the two separate ones."""
    B.profile_db_clear()
    g = build_graph(_matmul_then_transpose())[0]
    g.rewrite(B.REWRITE_NONE)
    st = g.plan(B.PLAN_FUSED)
    assert st.n_yellow_decisions >= 1 and st.n_profile_hits == 0 and st.n_profile_misses >= 3
    misses = g.profile_misses()
    fused = [m for m in misses if m.startswith("gemm|") and "Transpose" in m]
    alone_mm = [m for m in misses if m.startswith("gemm|MatMul|")]
    alone_t = [m for m in misses if m.startswith("transpose|")]
    assert len(fused) == 1 and len(alone_mm) == 1 and len(alone_t) == 1, misses

    # measured: fusing is a loss -> two kernels
    B.profile_db_set(fused[0], 50.0); B.profile_db_set(alone_mm[0], 5.0); B.profile_db_set(alone_t[0], 4.0)
    g2 = build_graph(_matmul_then_transpose())[0]
    g2.rewrite(B.REWRITE_NONE)
    st2 = g2.plan(B.PLAN_FUSED)
    assert st2.n_kernels == 2 and st2.n_profile_hits >= 3 and st2.n_profile_misses == 0
    assert g2.block_signature(0) == alone_mm[0]

    # measured: fusing wins -> one kernel
    B.profile_db_set(fused[0], 6.0)
    g3 = build_graph(_matmul_then_transpose())[0]
    g3.rewrite(B.REWRITE_NONE)
    st3 = g3.plan(B.PLAN_FUSED)
    assert st3.n_kernels == 1 and st3.n_yellow_fused >= 1
    assert g3.block_signature(0) == fused[0]
    B.profile_db_clear()


# ---- the rest of Table 2: index operators recorded as their parts, Concat as in-place parts, pooling -------------

def _desc():
    from paper_2108_13342_b200.workloads import GraphDesc
    return GraphDesc("t")


def _plan_desc(desc, flags=B.PLAN_FUSED):
    from paper_2108_13342_b200.runtime import build_graph
    G, ids = build_graph(desc)
    G.rewrite(B.REWRITE_NONE)
    st = G.plan(flags)
    return G, ids, st


def test_shuffle_and_resize_operators_are_recorded_as_index_operators():
    g = _desc(); g.ext("X", (2, 8, 8, 16))
    g.mark_output(g.add("Sigmoid", [g.add("DepthToSpace", [g.add("Relu", ["X"])], block=2)]))
    G, ids, st = _plan_desc(g)
    assert st.n_ops == 3 and st.n_kernels == 1
    assert G.blocks()[0]["ops"] == ["Relu", "Reshape", "Transpose", "Reshape", "Sigmoid"]
    assert G.tensor_info(ids[g.outputs[0]])[1] == (2, 16, 16, 4)
    g = _desc(); g.ext("X", (2, 8, 8, 16))
    g.mark_output(g.add("Resize", ["X"], scale=3))
    G, ids, st = _plan_desc(g)
    assert G.blocks()[0]["ops"] == ["Reshape", "Expand", "Reshape"] and G.blocks()[0]["mapping"] == "One-to-Many"
    assert G.tensor_info(ids[g.outputs[0]])[1] == (2, 24, 24, 16)
    g = _desc(); g.ext("X", (2, 8, 6, 4))
    g.mark_output(g.add("SpaceToDepth", ["X"], block=2))
    G, ids, st = _plan_desc(g)
    assert G.tensor_info(ids[g.outputs[0]])[1] == (2, 4, 3, 16)
    for bad in [dict(op="DepthToSpace", block=3), dict(op="SpaceToDepth", block=4), dict(op="Resize", scale=0)]:
        g = _desc(); g.ext("X", (2, 8, 6, 4))
        op = bad.pop("op")
        g.add(op, ["X"], **bad)
        with pytest.raises(B.DnnfError):
            _plan_desc(g)


def test_concat_parts_fuse_into_their_producers_and_share_the_result():
    g = _desc(); g.ext("X", (2, 8, 8, 16)); g.ext("Y", (2, 8, 8, 24)); g.ext("Z", (2, 8, 8, 8))
    c = g.add("Concat", [g.add("Relu", ["X"]), g.add("Sigmoid", ["Y"]), "Z"], axis=3)
    g.mark_output(g.add("Tanh", [c]))
    G, ids, st = _plan_desc(g)
    ops = [b["ops"] for b in G.blocks()]
    assert ops == [["Relu", "ConcatPart"], ["Sigmoid", "ConcatPart"], ["ConcatPart"], ["Tanh"]]
    assert st.n_ops == 4                                   # the three parts count as the one Concat they came from
    assert all(b["mapping"] == "One-to-One" for b in G.blocks())
    full = 2 * 8 * 8 * 48 * 4
    assert st.workspace_bytes - G.workspace_zero_bytes() == full          # one buffer for the result, none per part
    assert st.irs_bytes_fused == full
    assert [b["bytes"] for b in G.blocks()[:3]] == [2 * 2 * 8 * 8 * n * 4 for n in (16, 24, 8)]   # a part writes its range only
    # unfused: one copy kernel per part, still one shared result
    G, ids, st = _plan_desc(g, B.PLAN_UNFUSED)
    assert [b["ops"] for b in G.blocks()].count(["ConcatPart"]) == 3
    for bad_axis, shapes in [(3, [(2, 8, 8, 16), (2, 8, 7, 16)]), (5, [(2, 8), (2, 8)]), (0, [(2, 8), (2, 8, 1)])]:
        g = _desc()
        for i, shp in enumerate(shapes):
            g.ext(f"X{i}", shp)
        g.add("Concat", [f"X{i}" for i in range(len(shapes))], axis=bad_axis)
        with pytest.raises(B.DnnfError):
            _plan_desc(g)
    g = _desc(); g.ext("X", (2, 8))
    g.add("ConcatPart", ["X"], axis=0, start=0, shape=(4, 8))
    with pytest.raises(B.DnnfError):
        _plan_desc(g)


def test_pooling_shapes_types_and_epilogue_fusion():
    g = _desc(); g.ext("X", (2, 15, 13, 12)); g.ext("s", (12,)); g.ext("t", (12,))
    y = g.add("MaxPool", ["X"], kernel=3, stride=2, pad=1)
    g.mark_output(g.add("Relu", [g.add("ScaleShift", [y, "s", "t"], axis=-1)]))
    G, ids, st = _plan_desc(g)
    assert G.tensor_info(ids[g.outputs[0]])[1] == (2, 8, 7, 12)
    assert st.n_kernels == 1 and G.blocks()[0]["family"] == "pool" and G.blocks()[0]["mapping"] == "Many-to-Many"
    # Many-to-Many followed by Many-to-Many is a red cell: two pools never share a block
    g = _desc(); g.ext("X", (2, 16, 16, 8))
    g.mark_output(g.add("AveragePool", [g.add("MaxPool", ["X"], kernel=2, stride=2, pad=0)], kernel=8, stride=1, pad=0))
    G, ids, st = _plan_desc(g)
    assert st.n_kernels == 2 and G.tensor_info(ids[g.outputs[0]])[1] == (2, 1, 1, 8)
    for at in [dict(kernel=0), dict(kernel=3, pad=3), dict(kernel=3, stride=0), dict(kernel=40)]:
        g = _desc(); g.ext("X", (2, 16, 16, 8))
        g.add("MaxPool", ["X"], **at)
        with pytest.raises(B.DnnfError):
            _plan_desc(g)


def test_further_one_to_one_operators_type_and_fuse():
    g = _desc(); g.ext("X", (4, 8)); g.ext("v", (8,))
    t = g.add("PRelu", [g.add("Sin", ["X"]), "v"])
    t = g.add("Greater", [g.add("LeakyRelu", [t], alpha=0.1), g.add("Round", ["X"])])
    g.mark_output(g.add("Not", [t]))
    G, ids, st = _plan_desc(g)
    assert st.n_ops == 6 and st.n_kernels == 1
    kinds = G.blocks()[0]["ops"]
    assert kinds == ["Sin", "PRelu", "LeakyRelu", "Round", "Greater", "Not"], kinds
    prog = G.block_program(0)
    for name in ("SIN", "PRELU", "LEAKY", "ROUND", "NOT"):
        assert name in prog, prog
    assert "GT" in prog or "LT" in prog
    # the two pools differ only in attributes the common-subexpression pass must tell apart
    g = _desc(); g.ext("X", (1, 8, 8, 4))
    a = g.add("MaxPool", ["X"], kernel=2, stride=2, pad=0)
    b = g.add("MaxPool", ["X"], kernel=2, stride=1, pad=0)
    ra = g.add("Relu", [a]); rb = g.add("Relu", [b])
    g.mark_output(ra); g.mark_output(rb)
    from paper_2108_13342_b200.runtime import build_graph
    G, ids = build_graph(g)
    G.rewrite(B.REWRITE_DEFAULT)
    G.plan(B.PLAN_FUSED)
    assert G.tensor_info(ids[ra])[1] == (1, 4, 4, 4) and G.tensor_info(ids[rb])[1] == (1, 7, 7, 4)
    assert len([x for x in G.blocks() if x["family"] == "pool"]) == 2


def test_convtranspose_and_gather_recording_and_errors():
    g = _desc(); g.ext("X", (2, 8, 8, 16)); g.ext("Wt", (16, 2, 2, 8), kind="weight"); g.ext("S", (2, 16, 16, 8))
    t = g.add("Relu", [g.add("ConvTranspose", ["X", "Wt"], kernel=2)])
    g.mark_output(g.add("Concat", [t, "S"], axis=3))
    G, ids, st = _plan_desc(g)
    assert st.n_ops == 3 and st.n_kernels == 2
    assert ["Conv1x1", "Reshape", "Transpose", "Reshape", "Relu", "ConcatPart"] in [b["ops"] for b in G.blocks()]
    assert G.tensor_info(ids[g.outputs[0]])[1] == (2, 16, 16, 16)
    for wshape, at in [((16, 2, 3, 8), dict(kernel=2)), ((8, 2, 2, 8), dict(kernel=2)), ((16, 2, 2, 8), dict(kernel=2, stride=3))]:
        g = _desc(); g.ext("X", (2, 8, 8, 16)); g.ext("Wt", wshape, kind="weight")
        g.add("ConvTranspose", ["X", "Wt"], **at)
        with pytest.raises(B.DnnfError):
            _plan_desc(g)
    g = _desc(); g.ext("T", (50, 64)); g.ext("I", (7, 9))
    g.mark_output(g.add("Relu", [g.add("Gather", ["T", "I"], axis=0)]))
    G, ids, st = _plan_desc(g)
    assert [b["family"] for b in G.blocks()] == ["gather", "elementwise"]
    assert G.blocks()[0]["mapping"] == "One-to-Many"
    assert G.tensor_info(ids[g.outputs[0]])[1] == (7, 9, 64)
    g = _desc(); g.ext("T", (50, 64)); g.ext("I", (7, 9))
    g.add("Gather", ["T", "I"], axis=1)
    with pytest.raises(B.DnnfError):
        _plan_desc(g)


def test_deep_pointwise_convolution_is_planned_as_k_slices():
    always = B.PLAN_FUSED | B.PLAN_SPLIT_ALWAYS        # below the planner's break-even size
    g = _desc(); g.ext("X", (2, 32, 32, 256)); g.ext("Wt", (256, 64), kind="weight"); g.ext("s", (64,)); g.ext("t", (64,))
    g.mark_output(g.add("Clip", [g.add("ScaleShift", [g.add("Conv1x1", ["X", "Wt"]), "s", "t"], axis=-1)], lo=0.0, hi=6.0))
    G, ids, st = _plan_desc(g, always)
    fams = [(b["family"], b["variant"]) for b in G.blocks() if b["family"] != "alias"]
    assert [f for f, _ in fams] == ["gemm", "gemm"] and all(v in (4, 7) for _, v in fams), G.blocks()
    assert st.n_ops == 3 and st.n_kernels == 2                    # the slices count as the convolution they came from
    assert G.blocks()[-1]["ops"][-3:] == ["ScaleShift", "Clip"][-3:] or "Clip" in G.blocks()[-1]["ops"]
    assert "ADD anchor" in G.block_program(G.block_count() - 1)   # the partial sum rides in the last slice's epilogue
    # shallow enough, too few rows for the tensor-core kernel, or bf16: left alone
    for shape, wshape, dt in [((2, 32, 32, 144), (144, 24), "f32"), ((1, 8, 8, 256), (256, 64), "f32"), ((2, 32, 32, 256), (256, 64), "bf16")]:
        g = _desc(); g.ext("X", shape, dt); g.ext("Wt", wshape, dt, kind="weight")
        g.mark_output(g.add("Conv1x1", ["X", "Wt"]))
        G, ids, st = _plan_desc(g, always)
        assert st.n_kernels == 1, G.blocks()


def test_blocks_that_would_need_each_other_are_not_formed():
    """a1 -> b1 and b2 -> a2, with b1 and b2 joined only through their common consumer b3: {a1, a2} and {b1, b2, b3}
    are each convex, together they would be a cycle of two blocks.  Whatever the planner merges, the blocks it
    returns must admit a launch order (plan_graph reports an internal error otherwise)."""
    for perm in range(4):
        g = _desc(); g.ext("X", (64, 32)); g.ext("Y", (64, 32)); g.ext("ga", (32,)); g.ext("be", (32,))
        a1 = g.add("Tanh", ["X"])
        b2 = g.add("Sigmoid", ["Y"])
        a2 = g.add("Mul", [a1, b2]) if perm & 1 else g.add("Add", [b2, a1])
        b1 = g.add("Relu", [a1])
        b3 = g.add("Sub", [b1, b2]) if perm & 2 else g.add("Mul", [b2, b1])
        g.mark_output(g.add("LayerNorm", [a2, "ga", "be"], axis=-1, eps=1e-5))
        g.mark_output(g.add("Softmax", [b3], axis=-1))
        G, ids, st = _plan_desc(g)
        order = {}
        for i, b in enumerate(G.blocks()):
            for o in b["ops"]:
                order.setdefault(o, i)
        assert st.n_kernels >= 2


# ---- Section 4.4.2: layout selection ---------------------------------------------------------------------------------

def _rewritten_kinds(desc, flags=B.REWRITE_DEFAULT):
    G, ids = build_graph(desc)
    st = G.rewrite(flags)
    G.plan(B.PLAN_FUSED)
    kinds = [k for b in G.blocks() for k in b["ops"]]
    return G, st, kinds


def test_layout_selection_gives_elementwise_operators_the_layout_of_the_dominant_one():
    """A channels-first network reaches the channels-last convolutions and pools through Transposes.  Batch normalisation,
    ReLU6 and the residual Adds take the convolutions' layout, every Transpose pair between them cancels, and what is left
    is the NHWC network behind one Transpose of the input image."""
    nhwc = W.mbconv_stack(n=2, hw=16)
    nchw = W.mbconv_stack(n=2, hw=16, layout="nchw")
    Ga, sa, ka = _rewritten_kinds(nhwc.graph)
    Gb, sb, kb = _rewritten_kinds(nchw.graph)
    assert sa.layout_transposes_removed == 0
    assert sb.ops_before == 147 and sb.ops_after == sa.ops_after + 1
    assert sb.layout_transposes_removed == 62 and kb.count("Transpose") == 1
    assert sb.flops_after == sa.flops_after
    fam = lambda G: sorted(b["family"] for b in G.blocks())
    assert fam(Gb) == sorted(fam(Ga) + ["transpose"])
    assert all(b["n_outputs"] == 1 for b in Gb.blocks())
    # without the pass the residual sources are stored twice, once per layout
    Gc, sc, kc = _rewritten_kinds(nchw.graph, B.REWRITE_KEEP_LAYOUT)
    assert sc.layout_transposes_removed == 0 and sc.ops_after == 147
    assert sum(b["n_outputs"] for b in Gc.blocks()) > len(Gc.blocks())


def test_layout_selection_small_cases():
    # inverse Transposes around a layout-indifferent chain cancel; the per-channel operand follows its axis
    g = _desc(); g.ext("X", (2, 5, 6, 7)); g.ext("s", (7,), kind="weight"); g.ext("t", (7,), kind="weight")
    y = g.add("Transpose", [g.add("Relu", ["X"])], perm=(0, 3, 1, 2))
    y = g.add("Clip", [g.add("ScaleShift", [y, "s", "t"], axis=1)], lo=0.0, hi=6.0)
    g.mark_output(g.add("Sigmoid", [g.add("Transpose", [y], perm=(0, 2, 3, 1))]))
    G, st, kinds = _rewritten_kinds(g)
    assert st.layout_transposes_removed == 2 and kinds == ["Relu", "ScaleShift", "Clip", "Sigmoid"]
    # Transposes that are not inverses compose into one
    g = _desc(); g.ext("X", (2, 5, 6, 7))
    y = g.add("Tanh", [g.add("Transpose", [g.add("Relu", ["X"])], perm=(0, 3, 1, 2))])
    g.mark_output(g.add("Transpose", [y], perm=(0, 1, 3, 2)))
    G, st, kinds = _rewritten_kinds(g)
    assert st.layout_transposes_removed == 1 and kinds.count("Transpose") == 1
    # an operator that fixes a layout (Softmax on the last axis) is not crossed
    g = _desc(); g.ext("X", (2, 5, 6, 7))
    y = g.add("Softmax", [g.add("Transpose", ["X"], perm=(0, 3, 1, 2))], axis=-1)
    g.mark_output(g.add("Transpose", [y], perm=(0, 2, 3, 1)))
    G, st, kinds = _rewritten_kinds(g)
    assert st.layout_transposes_removed == 0 and kinds.count("Transpose") == 2
    # a lone Transpose behind element-wise operators stays where the graph has it (nothing to meet)
    G, st, kinds = _rewritten_kinds(W.swish_transpose(n=1, c=8, h=4, w=4).graph)
    assert st.layout_transposes_removed == 0 and kinds[-1] == "Transpose"
    # both operands of a residual Add come back from the other layout
    g = _desc(); g.ext("X", (2, 4, 4, 8)); g.ext("W", (8, 8), kind="weight")
    a = g.add("Transpose", [g.add("Conv1x1", ["X", "W"])], perm=(0, 3, 1, 2))
    b = g.add("Transpose", ["X"], perm=(0, 3, 1, 2))
    y = g.add("Transpose", [g.add("Add", [g.add("Relu", [a]), b])], perm=(0, 2, 3, 1))
    g.mark_output(g.add("Conv1x1", [y, "W"]))
    G, st, kinds = _rewritten_kinds(g)
    assert st.layout_transposes_removed == 3 and "Transpose" not in kinds


# ---- Where, Cast, CumSum, InstanceNormalization (Table 2) ------------------------------------------------------------

def test_where_cast_cumsum_instancenorm_recording_types_and_plans():
    # Table 2: Where and Cast are One-to-One (Where with a broadcast operand takes the operand's One-to-Many), CumSum and
    # InstanceNormalization Many-to-Many
    g = _desc(); g.ext("C", (4, 1, 8)); g.ext("A", (4, 6, 8)); g.ext("Bv", (8,))
    w = g.add("Where", ["C", "A", "Bv"])
    k = g.add("Cast", [w], to="bf16")
    g.mark_output(g.add("CumSum", [g.add("Cast", [k], to="f32")], axis=-1, exclusive=1))
    G, ids, st = _plan_desc(g)
    assert [G.op_mapping(i) for i in range(4)] == [OM, OO, OO, MM]
    assert G.tensor_info(ids[w]) == (B.F32, (4, 6, 8)) and G.tensor_info(ids[k])[0] == B.BF16
    assert st.n_kernels == 1 and G.blocks()[0]["family"] == "row"
    prog = G.block_program(0)
    assert "SELECT" in prog and "BF16R" in prog and "ROWSCAN_X" in prog, prog
    g = _desc(); g.ext("C", (4, 8)); g.ext("A", (4, 8)); g.ext("Bv", (4, 8))
    g.mark_output(g.add("Where", ["C", "A", "Bv"]))
    G, ids, st = _plan_desc(g)
    assert G.op_mapping(0) == OO and G.block_program(0) == "MOV in0; SAVE t0; MOV in1; SELECT in2; STORE out0"
    # InstanceNormalization is a Many-to-Many anchor of its own: One-to-One successors ride in its epilogue, nothing in front
    g = _desc(); g.ext("X", (2, 6, 6, 8)); g.ext("s", (8,), kind="weight"); g.ext("t", (8,), kind="weight"); g.ext("R", (2, 6, 6, 8))
    g.mark_output(g.add("Add", [g.add("Relu", [g.add("InstanceNorm", [g.add("Tanh", ["X"]), "s", "t"], eps=1e-5)]), "R"]))
    G, ids, st = _plan_desc(g)
    assert [(b["family"], b["ops"]) for b in G.blocks()] == [("elementwise", ["Tanh"]), ("instnorm", ["InstanceNorm", "Relu", "Add"])]
    assert G.op_mapping(1) == MM and st.n_ops == 4 and st.n_kernels == 2
    # errors
    for op, ins, at in [("Where", ["X", "s"], {}), ("Cast", ["X"], dict(to=7)), ("CumSum", ["X"], dict(axis=1)),
                        ("InstanceNorm", ["X", "s"], {}), ("InstanceNorm", ["s", "s", "t"], {})]:
        g2 = _desc(); g2.ext("X", (2, 6, 6, 8)); g2.ext("s", (8,), kind="weight"); g2.ext("t", (8,), kind="weight")
        g2.add(op, ins, **at)
        with pytest.raises(B.DnnfError):
            _plan_desc(g2)


def test_beyond_table3_forms_the_single_kernel_inverted_residual_block_only_while_it_pays():
    def fams(wl, flags):
        G, ids = build_graph(wl.graph)
        G.rewrite(B.REWRITE_NONE)
        st = G.plan(flags)
        return [b["family"] for b in G.blocks()], st
    beyond = B.PLAN_FUSED | B.PLAN_BEYOND_TABLE3
    small, full = W.mbconv_block(n=1, h=56, w=56), W.mbconv_block()
    assert fams(small, B.PLAN_FUSED)[0] == ["conv1x1", "dwconv", "conv1x1"]          # Table 3: Many-to-Many + Many-to-Many is red
    f, st = fams(small, beyond)
    assert f == ["mbconv"] and st.n_kernels == 1 and st.n_ops == 9
    assert fams(full, beyond)[0] == ["conv1x1", "dwconv", "conv1x1"]                 # 896 tiles: more than one wave
    assert fams(full, beyond | B.PLAN_MBCONV_ALWAYS)[0] == ["mbconv"]
    # the intermediate tensors of the single kernel never reach memory
    assert fams(small, beyond)[1].irs_bytes_fused == 0 and fams(small, B.PLAN_FUSED)[1].irs_bytes_fused > 0


def test_einsum_is_recorded_as_a_batched_matrix_product_between_index_operators():
    def kinds_of(eq, sa, sb):
        g = _desc(); g.ext("A", sa); g.ext("Bm", sb)
        y = g.add("Einsum", ["A", "Bm"], equation=eq)
        g.mark_output(y)
        G, ids = build_graph(g)
        kinds = [B.OP_NAMES[k] for k, alive in (G.op_kind(i) for i in range(G.op_count())) if alive]
        return G, ids[y], kinds
    G, y, kinds = kinds_of("ik,kj->ij", (4, 7), (7, 3))
    assert kinds == ["MatMul"] and G.tensor_info(y)[1] == (4, 3) and G.op_mapping(0) == MM
    G, y, kinds = kinds_of("bhqd,bhkd->bhqk", (2, 3, 4, 5), (2, 3, 6, 5))
    assert kinds == ["Reshape", "Transpose", "Reshape", "MatMul", "Reshape"] and G.tensor_info(y)[1] == (2, 3, 4, 6)
    G, y, kinds = kinds_of("mck,knc->nm", (3, 2, 4), (4, 5, 2))
    assert kinds.count("MatMul") == 1 and kinds[-1] == "Transpose" and G.tensor_info(y)[1] == (5, 3)
    G.rewrite(B.REWRITE_NONE)
    assert G.plan().n_ops == 1                                        # the pieces count as the one operator they came from
    for eq, sa, sb in [("ii,ij->j", (3, 3), (3, 4)), ("ik,kj->ijz", (2, 3), (3, 4)), ("ik,lj->ij", (2, 3), (3, 4)), ("ij,ij->ij", (2, 3), (2, 3)),
                       ("ik,kj->ij", (2, 3), (4, 5)), ("ikl,kj->ij", (2, 3), (3, 4))]:
        g = _desc(); g.ext("A", sa); g.ext("Bm", sb)
        with pytest.raises(B.DnnfError):
            build_graph_with(g, eq)
    g = _desc(); g.ext("A", (2, 3)); g.ext("Bm", (3, 4))
    assert g.add("Relu", ["A"])                                       # the graph stays usable after the refusals above


def build_graph_with(g, eq):
    g.add("Einsum", ["A", "Bm"], equation=eq)
    return build_graph(g)


def test_convtranspose_with_overlap_is_recorded_as_patches_plus_gather():
    g = _desc(); g.ext("X", (2, 8, 8, 16)); g.ext("Wt", (16, 4, 4, 8), kind="weight")
    y = g.add("ConvTranspose", ["X", "Wt"], kernel=4, stride=2, pad=1)
    g.mark_output(g.add("Relu", [y]))
    G, ids, st = _plan_desc(g)
    assert G.tensor_info(ids[y])[1] == (2, 16, 16, 8)
    assert [b["ops"] for b in G.blocks() if b["family"] != "alias"] == [["Conv1x1"], ["Col2Im", "Relu"]]
    assert st.n_ops == 2 and G.blocks()[-1]["family"] == "pool" and G.blocks()[-1]["mapping"] == "Many-to-Many"
    # stride = kernel without padding stays the index-only form; bad strides and pads are refused
    g = _desc(); g.ext("X", (2, 8, 8, 16)); g.ext("Wt", (16, 2, 2, 8), kind="weight")
    g.mark_output(g.add("ConvTranspose", ["X", "Wt"], kernel=2, stride=2))
    G, ids, st = _plan_desc(g)
    assert "Col2Im" not in [k for b in G.blocks() for k in b["ops"]]
    for at in (dict(kernel=2, stride=3), dict(kernel=2, stride=0), dict(kernel=3, stride=1, pad=3), dict(kernel=3, stride=1, pad=-1)):
        g = _desc(); g.ext("X", (2, 8, 8, 16)); g.ext("Wt", (16, at["kernel"], at["kernel"], 8), kind="weight")
        g.add("ConvTranspose", ["X", "Wt"], **at)
        with pytest.raises(B.DnnfError):
            _plan_desc(g)
