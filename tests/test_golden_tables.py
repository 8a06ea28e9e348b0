"""The tables the paper prints (tests/golden/), read as data and compared with what the library records: the mapping type
of every operator of Table 2, and the #FLOPS before and after each rewriting rule of Table 4."""
import os

import pytest

from paper_2108_13342_b200 import binding as B
from paper_2108_13342_b200 import workloads as W
from paper_2108_13342_b200.runtime import build_graph

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
TYPE = {"One-to-One": B.ONE_TO_ONE, "One-to-Many": B.ONE_TO_MANY, "Many-to-Many": B.MANY_TO_MANY, "Reorganize": B.REORGANIZE, "Shuffle": B.SHUFFLE}


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [line.rstrip("\n").split("\t") for line in f if line.strip() and not line.startswith("#")]


# how each operator of Table 2 is spelled at this library's boundary: (operator, input shapes, attributes)
X4 = (2, 8, 8, 16)
SPELLING = {
    "Add": ("Add", [(4, 8), (4, 8)], {}), "Asin": ("Asin", [(4, 8)], {}), "BatchNormalization": ("ScaleShift", [X4, (16,), (16,)], {"axis": -1}),
    "Cast": ("Cast", [(4, 8)], {"to": "bf16"}), "Ceil": ("Ceil", [(4, 8)], {}), "Clip": ("Clip", [(4, 8)], {"lo": 0.0, "hi": 6.0}),
    "Concat": ("Concat", [(4, 8), (4, 8)], {"axis": 1}), "Cos": ("Cos", [(4, 8)], {}), "Erf": ("Erf", [(4, 8)], {}), "Exp": ("Exp", [(4, 8)], {}),
    "Greater": ("Greater", [(4, 8), (4, 8)], {}), "LeakyRelu": ("LeakyRelu", [(4, 8)], {"alpha": 0.1}), "Log": ("Log", [(4, 8)], {}),
    "Not": ("Not", [(4, 8)], {}), "PRelu": ("PRelu", [(4, 8), (4, 8)], {}), "Reciprocal": ("Recip", [(4, 8)], {}), "Relu": ("Relu", [(4, 8)], {}),
    "Round": ("Round", [(4, 8)], {}), "Sigmoid": ("Sigmoid", [(4, 8)], {}), "Sin": ("Sin", [(4, 8)], {}),
    "Slice": ("Slice", [(4, 8)], {"axis": 1, "start": 0, "end": 4}), "Split": ("Split", [(4, 8)], {"axis": 1, "sizes": (4, 4)}),
    "Sqrt": ("Sqrt", [(4, 8)], {}), "Tanh": ("Tanh", [(4, 8)], {}), "Where": ("Where", [(4, 8), (4, 8), (4, 8)], {}),
    "Elementwise w/ broadcast": ("Mul", [(4, 8), (8,)], {}), "Expand": ("Expand", [(1, 8)], {"shape": (4, 8)}),
    "Gather": ("Gather", [(10, 8), (5,)], {"axis": 0}), "Resize": ("Resize", [X4], {"scale": 2}), "Upsample": ("Resize", [X4], {"scale": 2}),
    "AveragePool": ("AveragePool", [X4], {"kernel": 2, "stride": 2}), "CONV": ("Conv1x1", [X4, (16, 8)], {}),
    "ConvTranspose": ("ConvTranspose", [X4, (16, 4, 4, 8)], {"kernel": 4, "stride": 2, "pad": 1}), "CumSum": ("CumSum", [(4, 8)], {"axis": -1}),
    "Einsum": ("Einsum", [(4, 8), (8, 6)], {"equation": "ik,kj->ij"}), "GEMM": ("MatMul", [(4, 8), (8, 6)], {}),
    "InstanceNormalization": ("InstanceNorm", [X4, (16,), (16,)], {}), "MaxPool": ("MaxPool", [X4], {"kernel": 2, "stride": 2}),
    "ReduceProd": ("ReduceProd", [(4, 8)], {"axis": -1}), "ReduceMean": ("ReduceMean", [(4, 8)], {"axis": -1}), "Softmax": ("Softmax", [(4, 8)], {"axis": -1}),
    "Flatten": ("Flatten", [(2, 4, 8)], {"axis": 1}), "Reshape": ("Reshape", [(4, 8)], {"shape": (8, 4)}), "Squeeze": ("Squeeze", [(4, 1, 8)], {"axes": (1,)}),
    "Unsqueeze": ("Unsqueeze", [(4, 8)], {"axes": (0,)}), "DepthToSpace": ("DepthToSpace", [X4], {"block": 2}),
    "SpaceToDepth": ("SpaceToDepth", [X4], {"block": 2}), "Transpose": ("Transpose", [(4, 8)], {"perm": (1, 0)}),
}


@pytest.mark.parametrize("name,mapping", _rows("table2_mapping_types.tsv"))
def test_table2_operator_has_the_printed_mapping_type(name, mapping):
    """Every operator the table names exists at the boundary, and the operator that carries its arithmetic is recorded with
    the printed type.  (Operators recorded as several - a transposed convolution is a pointwise convolution plus a
    gather, DepthToSpace a Reshape / Transpose / Reshape - are represented by the most complex of their pieces, the
    rule of Section 3.1 for mixed mappings.)"""
    op, shapes, attrs = SPELLING[name]
    g = W.GraphDesc("t")
    ins = [g.ext("x%d" % i, s) for i, s in enumerate(shapes)]
    out = g.add(op, ins, n_out=2 if name == "Split" else 1, **attrs)
    g.mark_output(out[0] if isinstance(out, list) else out)
    G, _ = build_graph(g)
    order = {B.ONE_TO_ONE: 0, B.REORGANIZE: 1, B.SHUFFLE: 2, B.ONE_TO_MANY: 3, B.MANY_TO_MANY: 4}      # increasing complexity (Section 3.1)
    kinds = [G.op_mapping(i) for i in range(G.op_count())]
    if name in ("Concat", "Split", "Slice"):
        assert all(k == B.ONE_TO_ONE for k in kinds)
    else:
        assert max(kinds, key=lambda k: order[k]) == TYPE[mapping], (name, kinds)


M_, N_ = 6, 10


def _rule_graph(rule):
    g = W.GraphDesc("r")
    for n in "ABC":
        g.ext(n, (M_, N_))
    a = g.add
    if rule.startswith("associative: Recip"):
        y = a("Mul", [a("Recip", ["A"]), a("Recip", [a("Mul", ["A", "B"])])])
    elif rule.startswith("associative: (A * sqrt"):
        y = a("Mul", [a("Mul", ["A", a("Sqrt", ["B"])]), a("Mul", [a("Sqrt", ["B"]), "C"])])
    elif rule.startswith("associative: Abs"):
        y = a("Mul", [a("Mul", [a("Abs", ["A"]), "B"]), a("Abs", ["C"])])
    elif rule.startswith("associative: (A * ReduceSum"):
        y = a("Mul", [a("Mul", ["A", a("ReduceSum", ["B"], axis=-1, keepdims=1)]), a("Mul", [a("ReduceSum", ["B"], axis=-1, keepdims=1), "C"])])
    elif rule.startswith("distributive: A * C"):
        y = a("Add", [a("Mul", ["A", "C"]), a("Mul", ["A", "B"])])
    elif rule.startswith("distributive: A + A"):
        y = a("Add", ["A", a("Mul", ["A", "B"])])
    elif rule.startswith("distributive: Square"):
        y = a("Sub", [a("Square", [a("Add", ["A", "B"])]), a("Mul", [a("Add", ["A", "B"]), "C"])])
    elif rule.startswith("commutative: A * B"):
        y = a("Mul", ["A", "B"])
    elif rule.startswith("commutative: ReduceSum"):
        y = a("ReduceSum", [a("BitShift", ["A"], bits=3)], axis=-1, keepdims=1)
    elif rule.startswith("commutative: ReduceProd"):
        y = a("ReduceProd", [a("Exp", ["A"])], axis=-1, keepdims=1)
    else:
        raise KeyError(rule)
    g.mark_output(y)
    return g


@pytest.mark.parametrize("rule,ba,bb,aa,ab", _rows("table4_flops.tsv"))
def test_table4_flops_before_and_after(rule, ba, bb, aa, ab):
    G, _ = build_graph(_rule_graph(rule))
    st = G.rewrite(B.REWRITE_DEFAULT)
    mn, m = M_ * N_, M_
    assert st.flops_before == int(ba) * mn + int(bb) * m, (rule, st.flops_before)
    assert st.flops_after == int(aa) * mn + int(ab) * m, (rule, st.flops_after)
