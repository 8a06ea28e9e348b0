"""Differential test over fusion plans: the profiling database is filled with pseudo-random latencies, which makes the
planner take fusion decisions it would not take otherwise; every resulting plan must still compute the oracle's result.
Workspace and outputs start as NaN, so a tensor that some plan leaves partly unwritten (or reads before it is written)
shows up."""
import numpy as np
import pytest

from paper_2108_13342_b200 import binding as B
from paper_2108_13342_b200 import workloads as W
from paper_2108_13342_b200.runtime import Session, build_graph
from oracle import interp as O
from util import RTOL_BF16, RTOL_F32, close, graph, rnd

pytestmark = pytest.mark.gpu


def _random_costs(desc, rewrite, seed, rounds=4):
    """Give every candidate block the planner asks about a pseudo-random latency: 1 .. 20 us for even seeds; for odd
    seeds the latency also grows with the number of operators in the block, which talks the planner out of fusing."""
    for r in range(rounds):
        g = build_graph(desc)[0]
        g.rewrite(rewrite)
        st = g.plan(B.PLAN_FUSED)
        misses = g.profile_misses()
        if not misses:
            return st
        for i, sig in enumerate(misses):
            u = float(W.uniform(9000 + seed, 100 * r + i, (1,), 1.0, 20.0)[0])
            if seed % 2:
                u *= 1 + 3 * sig.split("|")[1].count("+")
            B.profile_db_set(sig, u)
    return st


def _run_poisoned(wl, rewrite):
    s = Session(wl, plan_flags=B.PLAN_FUSED, rewrite_flags=rewrite)
    zero = s.g.workspace_zero_bytes()
    s.workspace[zero:].fill_(0xFF)                 # NaN in fp32 and bf16
    for n in wl.graph.outputs:
        s.buffers[n].fill_(float("nan"))
    s.run()
    assert s.g.status()[0] == 0
    return s


def _mixed_graph():
    # element-wise ops around a Slice, a Transpose and a reduction, with tensors read both inside and outside blocks
    g = graph()
    g.ext("X", (6, 16, 24)); g.ext("b", (24,)); g.ext("Wm", (24, 32))
    t = g.add("Add", ["X", "b"], out="T")
    g.mark_output(t)
    a, c = g.add("Split", [t], n_out=2, axis=-1, sizes=(8, 16))
    r = g.add("Relu", [a])
    g.mark_output(g.add("Transpose", [r], perm=(0, 2, 1), out="RT"))
    e = g.add("Exp", [g.add("MulC", [c], c=0.1)])
    g.mark_output(g.add("Softmax", [e], axis=-1, out="S"))
    m = g.add("MatMul", [t, "Wm"])
    g.mark_output(g.add("Transpose", [g.add("Tanh", [m])], perm=(0, 2, 1), out="MT"))
    ins = {"X": rnd((6, 16, 24), 1), "b": rnd((24,), 2), "Wm": rnd((24, 32), 3, -0.3, 0.3)}
    return W.Workload(g, ins)


CASES = [("mixed", _mixed_graph, B.REWRITE_NONE, RTOL_F32),
         ("encoder", lambda: W.encoder(layers=2, batch=2, seq=32, hidden=64, heads=4, ffn=128), B.REWRITE_CANON_MACRO, RTOL_BF16),
         ("encoder-primitive", lambda: W.encoder(layers=1, batch=2, seq=32, hidden=64, heads=4, ffn=128), B.REWRITE_DEFAULT, RTOL_BF16),
         ("decoder", lambda: W.decoder(layers=1, batch=2, seq=32, hidden=64, heads=4, ffn=128), B.REWRITE_CANON_MACRO, RTOL_BF16),
         ("mbconv", lambda: W.mbconv_block(2, 14, 14, 24, 144), B.REWRITE_NONE, RTOL_F32),
         ("ffn", lambda: W.ffn_block(256, 64, 128), B.REWRITE_NONE, RTOL_BF16)]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
@pytest.mark.parametrize("seed", range(6))
def test_every_plan_the_planner_can_be_talked_into_is_correct(case, seed):
    _, make, rewrite, rtol = case
    wl = make()
    ref = O.run_graph(wl.graph, wl.inputs)
    B.profile_db_clear()
    try:
        _random_costs(wl.graph, rewrite, seed)
        s = _run_poisoned(wl, rewrite)
        for n in wl.graph.outputs:
            got = s.output(n)
            assert np.isfinite(got).all(), f"{n}: unwritten or poisoned elements"
            # un-fusing adds bf16 roundings of intermediates: the bf16 workloads get the tolerance of the unfused plan
            close(got, ref[n], rtol)
    finally:
        B.profile_db_clear()
