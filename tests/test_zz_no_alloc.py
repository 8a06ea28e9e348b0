"""dnnf_run_static_ws: the entry point for callers that are not allowed to allocate
device memory (an allocator's out-of-memory hook, a host application that freezes
allocation after start-up).  It must give the same results as dnnf_run with a
caller-provided workspace, call after call, although every call reuses one array
that still holds the previous call's data.

Collected last on purpose: a run that stops at the first failure has then already
run every other test."""
import numpy as np
import pytest

from paper_2108_13342_b200 import binding as B
from paper_2108_13342_b200 import workloads as W
from paper_2108_13342_b200.runtime import Session
from util import RTOL_BF16, RTOL_F32, close

pytestmark = pytest.mark.gpu


def _outputs(sess):
    return {n: sess.output(n) for n in sess.desc.outputs}


@pytest.mark.parametrize("make,rtol", [(lambda: W.add_layernorm_gelu(rows=64, hidden=768), RTOL_F32),
                                       (lambda: W.swish_transpose(n=2, c=64, h=12, w=20), RTOL_F32),
                                       # tensor-core blocks: their TMA descriptors must follow the intermediates into the
                                       # built-in array, and the split-K arrival counters live in its cleared header
                                       (lambda: W.ffn_block(m=1024, hidden=768, ffn=3072), RTOL_BF16)],
                         ids=["add_layernorm_gelu", "swish_transpose", "ffn_block_gemm"])
def test_static_workspace_matches_caller_workspace_twice(make, rtol):
    import torch
    wl = make()
    # one kernel per operator: every intermediate goes through the workspace
    ref = Session(wl, plan_flags=B.PLAN_UNFUSED, rewrite_flags=B.REWRITE_NONE)
    assert ref.plan_stats.workspace_bytes > 256
    ref.run()
    want = _outputs(ref)

    s = Session(wl, plan_flags=B.PLAN_UNFUSED, rewrite_flags=B.REWRITE_NONE)
    stream = torch.cuda.current_stream().cuda_stream
    for call in range(2):
        for n in s.desc.outputs:
            s.buffers[n].fill_(float("nan"))          # a stale result cannot pass
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        s.g.run_static_ws(stream)
        torch.cuda.synchronize()
        if call == 1:                                 # the first call on a device may load the kernels' code
            assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the amount of free device memory"
        assert s.g.status() == (0, -1)                # read from the built-in array, where this run kept its status words
        got = _outputs(s)
        for n in want:
            close(got[n], want[n], rtol)
            if rtol == RTOL_F32:
                assert np.array_equal(got[n], want[n]), f"call {call}: {n} differs from dnnf_run"
    # the caller's own workspace is still bound and still works
    s.run()
    assert s.g.status() == (0, -1)
    for n in want:
        close(s.output(n), want[n], rtol)


def test_static_workspace_rejects_plans_that_do_not_fit():
    wl = W.add_layernorm_gelu(rows=8192, hidden=768)        # 25 MB per intermediate, two alive at once
    s = Session(wl, plan_flags=B.PLAN_UNFUSED, rewrite_flags=B.REWRITE_NONE)
    assert s.plan_stats.workspace_bytes > B.STATIC_WS_BYTES
    with pytest.raises(B.DnnfError) as e:
        s.g.run_static_ws(0)
    assert e.value.code == B.ERR_WORKSPACE and "built-in array" in str(e.value)
