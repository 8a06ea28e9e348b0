"""Fills the planner's profiling database (Section 4.3: yellow Table 3 cells are decided by measured latencies).

    python -m paper_2108_13342_b200.profile_db --workload encoder --kw layers=1 --out encoder.tsv

plans the workload, lets the library run every candidate block the planner asked about and did not find
(`dnnf_profile_measure`: CUDA-event timing of the lowered candidate on scratch memory), plans again with the
measurements, and repeats until a plan needs no unmeasured candidate.  The database is a text file of
"signature<TAB>microseconds" lines; `binding.profile_db_load` brings it back in a later process.
"""
import argparse
import json

from . import binding as B
from . import workloads as W
from .runtime import build_graph


def fill(graph_desc, device, rewrite_flags=B.REWRITE_DEFAULT, plan_flags=B.PLAN_FUSED, scratch_bytes=1 << 30, iters=20,
         max_rounds=6):
    """Measure until the plan of `graph_desc` is decided by measurements only.  Returns a list with one record per
    planning round: kernels, yellow decisions, database hits and misses, candidates measured."""
    import torch
    scratch = torch.empty(scratch_bytes, dtype=torch.uint8, device=device)
    stream = torch.cuda.current_stream(device).cuda_stream
    rounds = []
    for _ in range(max_rounds):
        g = build_graph(graph_desc)[0]
        g.rewrite(rewrite_flags)
        st = g.plan(plan_flags)
        rec = {"kernels": st.n_kernels, "yellow": st.n_yellow_decisions, "yellow_fused": st.n_yellow_fused,
               "hits": st.n_profile_hits, "misses": st.n_profile_misses, "measured": 0}
        if st.n_profile_misses:
            rec["measured"] = g.profile_measure(scratch.data_ptr(), scratch_bytes, stream, iters)
        rounds.append(rec)
        if st.n_profile_misses == 0 or rec["measured"] == 0:
            break
    return rounds


def main():
    import torch
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", required=True)
    ap.add_argument("--kw", nargs="*", default=[])
    ap.add_argument("--canon", action="store_true", help="canonicalise LayerNorm / GELU macro operators before planning")
    ap.add_argument("--out", default=None)
    ap.add_argument("--load", default=None, help="start from an existing database file")
    a = ap.parse_args()
    kw = {k: int(v) for k, v in (x.split("=") for x in a.kw)}
    wl = W.by_name(a.workload, **kw)
    if a.load:
        B.profile_db_load(a.load)
    rounds = fill(wl.graph, torch.device("cuda:0"), B.REWRITE_CANON_MACRO if a.canon else B.REWRITE_DEFAULT)
    print(json.dumps({"workload": a.workload, "rounds": rounds, "entries": B.profile_db_size()}))
    if a.out:
        B.profile_db_save(a.out)


if __name__ == "__main__":
    main()
