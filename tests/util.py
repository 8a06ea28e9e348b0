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


RTOL_BF16_ROUNDING = 8e-3    # a block without a contraction whose result is stored as bf16: one rounding (2^-9) plus fp32 math


def check_blocks(wl, plan_flags=B.PLAN_FUSED, rewrite_flags=B.REWRITE_NONE, min_checked=1):
    """Per-block parity: every block of the plan is run ALONE on inputs taken from the oracle (its external inputs are
    overwritten with the oracle's tensors in the tensor's storage type) and its outputs are compared with the oracle's
    operators applied to exactly those inputs, element by element at the single-block tolerance: 1e-5 for fp32 blocks, 2e-2 for bf16 blocks around a
    contraction, one bf16 rounding for other bf16 blocks.  Errors cannot build up from block to block, so deep
    graphs are held to the same bar as single blocks.  Blocks that touch a tensor the graph description does not
    name (intermediates made by rewriting or by splitting an operator) are skipped; returns (checked, skipped)."""
    import torch
    s = Session(wl, plan_flags=plan_flags, rewrite_flags=rewrite_flags)
    name_of = {v: k for k, v in s.ids.items()}
    # The oracle, operator by operator, with ONE change: a bf16 tensor that the plan keeps in memory between blocks is
    # rounded to bf16 before an operator of ANOTHER block reads it, because that is the value that block is given
    # (readers inside the producing block get the unrounded value, as the kernel keeps it in registers).  `ref` holds
    # every operator's unrounded result (what a block's output is compared with), `env` what is fed to the blocks.
    stored_bf16 = set()
    for name, tid in s.ids.items():
        dt, _ = s.g.tensor_info(tid)
        if dt == B.BF16 and s.g.tensor_location(tid)[0] != 2:
            stored_bf16.add(name)
    # which block an operator of the description runs in: the block that stores its result, else the block of a reader
    made_in = {}
    for b in range(s.g.block_count()):
        for t in s.g.block_tensors(b)[1]:
            if t in name_of:
                made_in[name_of[t]] = b
    readers = {}
    for i, o in enumerate(wl.graph.ops):
        for n in o.inputs:
            readers.setdefault(n, []).append(i)
    op_block = [None] * len(wl.graph.ops)
    for i in reversed(range(len(wl.graph.ops))):
        o = wl.graph.ops[i]
        for n in o.outputs:
            if op_block[i] is None and n in made_in:
                op_block[i] = made_in[n]
        for n in o.outputs:
            for r in readers.get(n, []):
                if op_block[i] is None and op_block[r] is not None and n not in made_in:
                    op_block[i] = op_block[r]
    producer = {n: i for i, o in enumerate(wl.graph.ops) for n in o.outputs}
    ref = {k: np.asarray(v, dtype=np.float64) for k, v in wl.inputs.items()}
    rounded = {}

    def seen_by(i, n):
        """The value of tensor n as operator i reads it: through memory (bf16) unless both sit in one block."""
        if n in stored_bf16 and n in producer and op_block[producer[n]] != op_block[i]:
            if n not in rounded:
                rounded[n] = W.round_to_bf16(ref[n].astype(np.float32)).astype(np.float64)
            return rounded[n]
        return ref[n]

    for i, o in enumerate(wl.graph.ops):
        outs = O._apply(o.op, [seen_by(i, n) for n in o.inputs], o.attrs)
        for n, v in zip(o.outputs, outs):
            ref[n] = np.asarray(v, dtype=np.float64)
    env = {n: (W.round_to_bf16(v.astype(np.float32)).astype(np.float64) if n in stored_bf16 else v) for n, v in ref.items()}
    stream = torch.cuda.current_stream().cuda_stream

    def storage(tid):
        dt, dims = s.g.tensor_info(tid)
        tdt = torch.float32 if dt == B.F32 else torch.bfloat16
        where, off = s.g.tensor_location(tid)
        if where == 3:
            where, tid2 = 0, off
            return s.buffers[name_of[tid2]].view(-1)[: int(np.prod(dims))].view(dims), tdt
        if where == 0:
            return s.buffers[name_of[tid]], tdt
        assert where == 1, (name_of.get(tid), where)
        n = int(np.prod(dims))
        nbytes = n * (4 if dt == B.F32 else 2)
        return s.workspace[off: off + nbytes].view(tdt).view(dims), tdt

    checked = skipped = 0
    blocks = s.g.blocks()
    for b in range(s.g.block_count()):
        if blocks[b]["family"] == "alias":
            continue
        ins, outs = s.g.block_tensors(b)
        if any(t not in name_of for t in ins + outs) or "ConcatPart" in blocks[b]["ops"]:
            skipped += 1
            continue
        for t in ins:
            buf, tdt = storage(t)
            buf.copy_(torch.from_numpy(np.ascontiguousarray(env[name_of[t]], dtype=np.float32)).to(buf.device).to(tdt).view(buf.shape))
        for t in outs:
            storage(t)[0].fill_(float("nan"))
        s.g.run_block(b, stream)
        torch.cuda.synchronize()
        assert s.g.status()[0] == 0
        contraction = blocks[b]["family"] in ("gemm", "conv1x1", "attention")
        for t in outs:
            buf, tdt = storage(t)
            got = buf.float().cpu().numpy().astype(np.float64)
            rtol = RTOL_F32 if tdt == torch.float32 else (RTOL_BF16 if contraction else RTOL_BF16_ROUNDING)
            try:
                close(got, ref[name_of[t]].reshape(got.shape), rtol)
            except AssertionError as e:
                raise AssertionError(f"block {b} {blocks[b]['family']} {'+'.join(blocks[b]['ops'][:8])} -> {name_of[t]}: {e}") from None
        checked += 1
    assert checked >= min_checked, (checked, skipped)
    return checked, skipped
