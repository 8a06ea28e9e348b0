"""Shared helpers for the parity tests (CUDA path vs. oracle)."""
import numpy as np

from oracle import interp as O
from paper_2108_13342_b200 import binding as B
from paper_2108_13342_b200 import workloads as W
from paper_2108_13342_b200.runtime import Session

RTOL_F32 = 1e-5      # fp32 element-wise / reduction chains
RTOL_BF16 = 2e-2     # bf16 GEMM-anchored blocks, fp32 accumulate


def close(got, ref, rtol):
    """Per-element |g-o| <= rtol*|o| + rtol*rms(o): a relative bound that stays
    meaningful where outputs cross or equal zero (masked softmax entries, GELU)."""
    got = np.asarray(got, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    rms = float(np.sqrt(np.mean(ref * ref))) if ref.size else 0.0
    err = np.abs(got - ref)
    bound = rtol * np.abs(ref) + rtol * rms
    bad = err > bound
    if bad.any():
        i = np.unravel_index(np.argmax(err - bound), err.shape)
        raise AssertionError(f"{bad.sum()} of {bad.size} elements off; worst at {i}: got {got[i]!r} ref {ref[i]!r} "
                             f"err {err[i]:.3e} bound {bound[i]:.3e}")
    return float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300))


def run_both(wl, plan_flags=B.PLAN_FUSED, rewrite_flags=B.REWRITE_NONE):
    s = Session(wl, plan_flags=plan_flags, rewrite_flags=rewrite_flags)
    s.run()
    got = {n: s.output(n) for n in wl.graph.outputs}
    st, blk = s.g.status()
    assert st == 0, f"device status {st} from block {blk}"
    ref = O.run_graph(wl.graph, wl.inputs)
    return s, got, ref


def check(wl, rtol, plan_flags=B.PLAN_FUSED, rewrite_flags=B.REWRITE_NONE, expect_blocks=None):
    s, got, ref = run_both(wl, plan_flags, rewrite_flags)
    if expect_blocks is not None:
        assert s.plan_stats.n_kernels == expect_blocks, (s.plan_stats.n_kernels, s.g.blocks())
    for n in wl.graph.outputs:
        close(got[n], ref[n], rtol)
    return s


def graph(name="t"):
    return W.GraphDesc(name)


def rnd(shape, seed, lo=-2.0, hi=2.0):
    return W.uniform(777, seed, shape, lo, hi)
