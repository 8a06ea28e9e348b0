"""Per-configuration measurements printed beside the headline benchmark number:
each fused block's time, GB/s (or TFLOP/s) and roofline fraction; the same graph
unfused, one kernel per operator; plain launches and CUDA-graph replay."""
from __future__ import annotations

import numpy as np

from . import binding as B
from . import workloads as W
from .runtime import Session

L2_BYTES = 126 * 1024 * 1024


def _time_region(torch, dev, fn, iters):
    st = torch.cuda.current_stream(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(dev)
    e0.record(st)
    for _ in range(iters):
        fn()
    e1.record(st)
    torch.cuda.synchronize(dev)
    return e0.elapsed_time(e1) * 1e3 / iters          # us per call


def _graph_of(torch, dev, fn):
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream(dev)
    s.wait_stream(torch.cuda.current_stream(dev))
    with torch.cuda.stream(s):
        fn_s = lambda: fn(s.cuda_stream)
        fn_s()                                         # warm-up on the side stream
        torch.cuda.synchronize(dev)
        with torch.cuda.graph(g, stream=s):
            fn_s()
    torch.cuda.current_stream(dev).wait_stream(s)
    return g


def measure_workload(torch, dev, wl, pk, flags, copies, iters=20, rewrite=B.REWRITE_NONE, per_block_limit=40):
    """`copies` sessions with distinct buffers, run round-robin so that every launch
    sees cold data when copies * footprint exceeds L2."""
    sess = [Session(wl, plan_flags=flags, rewrite_flags=rewrite, device=dev) for _ in range(copies)]
    s0 = sess[0]
    nb = s0.g.block_count()
    blocks = s0.g.blocks()

    def all_plain():
        sp = torch.cuda.current_stream(dev).cuda_stream
        for s in sess:
            s.g.run(sp)

    def all_on(sp):
        for s in sess:
            s.g.run(sp)

    for _ in range(3):
        all_plain()
    t_plain = _time_region(torch, dev, all_plain, iters) / copies
    cg = _graph_of(torch, dev, all_on)
    t_graph = _time_region(torch, dev, cg.replay, iters) / copies
    per_block = []
    if nb <= per_block_limit:
        for b in range(nb):
            if blocks[b]["family"] == "alias":
                continue

            def one(sp, b=b):
                for s in sess:
                    s.g.run_block(b, sp)

            cgb = _graph_of(torch, dev, one)
            cgb.replay()
            t = _time_region(torch, dev, cgb.replay, iters) / copies
            by, fl = blocks[b]["bytes"], blocks[b]["flops"]
            roof_us = max(by / (pk["hbm_gbs"] * 1e3), fl / (pk["bf16_tflops"] * 1e6))
            per_block.append({"ops": "+".join(blocks[b]["ops"][:8]), "family": blocks[b]["family"], "us": round(t, 3),
                              "bytes": by, "GBps": round(by / t / 1e3, 1), "flops": fl,
                              "TFLOPs": round(fl / t / 1e6, 1) if fl else 0, "roofline_us": round(roof_us, 3),
                              "frac_of_roofline": round(roof_us / t, 3)})
    return {"kernels": s0.plan_stats.n_kernels, "ops": s0.plan_stats.n_ops, "fusion_rate": round(s0.plan_stats.fusion_rate, 2),
            "us_plain_launches": round(t_plain, 3), "us_cuda_graph": round(t_graph, 3), "copies": copies,
            "irs_bytes": int(s0.plan_stats.irs_bytes_fused), "blocks": per_block}


def per_config(dev, pk, only=None):
    import torch
    out = {}
    cases = [
        ("cfg1 swish+transpose [1,64,56,56]", W.swish_transpose(), 96),
        ("cfg1 batch-512 variant", W.swish_transpose(n=512), 1),
        ("cfg2a scale+mask+softmax [8,12,128,128]", W.masked_softmax(), 24),
        ("cfg2a batch-512 variant", W.masked_softmax(batch=512), 1),
        ("cfg2b add+LayerNorm+GELU [1024,768]", W.add_layernorm_gelu(), 24),
        ("cfg2b 131072-row variant", W.add_layernorm_gelu(rows=131072), 1),
        ("cfg3 GEMM+bias+GELU ; GEMM+bias+residual bf16 [4096,768,3072]", W.ffn_block(), 8),
        ("cfg4 MBConv fp32 NHWC [32,56,56,24->144->24]", W.mbconv_block(), 2),
        ("next: CNN fragment with pooling, SpaceToDepth/DepthToSpace, Resize, Concat fp32 NHWC [32,64,64,32]", W.cnn_neck(n=32), 2),
        ("next: MobileNetV2-shaped stack of 9 inverted-residual blocks + head, fp32 NHWC [32,56,56,16] (84 operators)", W.mbconv_stack(), 1),
        ("next: the same stack on ONE image [1,56,56,16] (the paper's operating point)", W.mbconv_stack(n=1), 4),
        ("next: style-transfer decoder with InstanceNormalization and overlapping ConvTranspose, fp32 NHWC [8,64,64,64] -> [8,256,256,4]", W.style_decoder(), 1),
    ]
    for name, wl, copies in cases:
        if only and only not in name:
            continue
        try:
            fused = measure_workload(torch, dev, wl, pk, B.PLAN_FUSED, copies)
            unfused = measure_workload(torch, dev, wl, pk, B.PLAN_UNFUSED, copies)
            out[name] = {"fused": fused, "unfused": unfused,
                         "speedup_fused_vs_unfused_graph": round(unfused["us_cuda_graph"] / fused["us_cuda_graph"], 2)}
        except Exception as e:      # report, never hide
            out[name] = {"error": repr(e)}
        torch.cuda.empty_cache()
    return out


def encoder_report(dev, pk, layers=12):
    """Whole-graph workload: the 12-layer encoder as primitive operators, through rewriting,
    planning and fused execution; compared with one kernel per operator."""
    import torch
    wl = W.encoder(layers=layers)
    out = {}
    for name, flags, rw in [("fused", B.PLAN_FUSED, B.REWRITE_DEFAULT), ("fused+layernorm-canon", B.PLAN_FUSED, B.REWRITE_CANON_MACRO),
                            ("unfused", B.PLAN_UNFUSED, B.REWRITE_NONE)]:
        r = measure_workload(torch, dev, wl, pk, flags, 1, iters=10, rewrite=rw, per_block_limit=0)
        out[name] = r
        torch.cuda.empty_cache()
    # per-block table for one layer of the canonicalised plan
    s = Session(wl, rewrite_flags=B.REWRITE_CANON_MACRO, device=dev)
    blocks = s.g.blocks()
    per = []
    nb_layer = max(1, s.g.block_count() // layers)
    for b in range(nb_layer, 2 * nb_layer if layers > 1 else nb_layer):
        if blocks[b]["family"] == "alias":
            continue
        reps = 20        # several launches per replay: a one-node graph is bound by the replay overhead itself
        cg = _graph_of(torch, dev, lambda sp, b=b: [s.g.run_block(b, sp) for _ in range(reps)])
        cg.replay()
        t = _time_region(torch, dev, cg.replay, 10) / reps
        by, fl = blocks[b]["bytes"], blocks[b]["flops"]
        roof = max(by / (pk["hbm_gbs"] * 1e3), fl / (pk["bf16_tflops"] * 1e6))
        per.append({"ops": "+".join(blocks[b]["ops"][:10]), "family": blocks[b]["family"], "us_warm_l2": round(t, 3), "bytes": by,
                    "flops": fl, "roofline_us": round(roof, 3), "frac_of_roofline": round(roof / t, 3)})
    out["layer_blocks_canon_plan"] = per
    # Same graph planned from measured latencies (profiling database, Section 4.3) instead of the analytic model.
    from . import profile_db
    del s
    torch.cuda.empty_cache()
    B.profile_db_clear()
    try:
        rounds = profile_db.fill(wl.graph, dev, B.REWRITE_CANON_MACRO, scratch_bytes=1 << 30, iters=20)
        r = measure_workload(torch, dev, wl, pk, B.PLAN_FUSED, 1, iters=10, rewrite=B.REWRITE_CANON_MACRO, per_block_limit=0)
        r["profiling_rounds"] = rounds
        r["database_entries"] = B.profile_db_size()
        out["fused+layernorm-canon+profiled-plan"] = r
    finally:
        B.profile_db_clear()
    torch.cuda.empty_cache()
    out["speedup_fused_vs_unfused_graph"] = round(out["unfused"]["us_cuda_graph"] / out["fused+layernorm-canon"]["us_cuda_graph"], 2)
    out["speedup_fused_vs_unfused_plain"] = round(out["unfused"]["us_plain_launches"] / out["fused+layernorm-canon"]["us_plain_launches"], 2)
    return out


def decoder_report(dev, pk, layers=12):
    """Second whole-graph workload: a GPT-2 style decoder as primitive operators.  The analogue of the paper's
    optimisation breakdown: one kernel per operator / fusion without rewriting / fusion after the printed rewriting
    rules / fusion after LayerNorm canonicalisation."""
    import torch
    wl = W.decoder(layers=layers)
    out = {}
    for name, flags, rw in [("unfused", B.PLAN_UNFUSED, B.REWRITE_NONE), ("fused, no rewriting", B.PLAN_FUSED, B.REWRITE_NONE),
                            ("fused + printed rules", B.PLAN_FUSED, B.REWRITE_DEFAULT),
                            ("fused + layernorm-canon", B.PLAN_FUSED, B.REWRITE_CANON_MACRO)]:
        out[name] = measure_workload(torch, dev, wl, pk, flags, 1, iters=10, rewrite=rw, per_block_limit=0)
        torch.cuda.empty_cache()
    out["speedup_fused_vs_unfused_graph"] = round(out["unfused"]["us_cuda_graph"] / out["fused + layernorm-canon"]["us_cuda_graph"], 2)
    return out


def encoder_latency_pair(dev, pk, layers=12):
    """Whole-graph latency of the encoder workload, fused (LayerNorm canonicalised) against one kernel per
    operator, both as CUDA-graph replays and as plain launches."""
    import torch
    wl = W.encoder(layers=layers)
    f = measure_workload(torch, dev, wl, pk, B.PLAN_FUSED, 1, iters=20, rewrite=B.REWRITE_CANON_MACRO, per_block_limit=0)
    torch.cuda.empty_cache()
    u = measure_workload(torch, dev, wl, pk, B.PLAN_UNFUSED, 1, iters=10, rewrite=B.REWRITE_NONE, per_block_limit=0)
    torch.cuda.empty_cache()
    # reported apart: the plan that also fuses what Table 3 forbids (each attention head's three blocks as one kernel)
    x = measure_workload(torch, dev, wl, pk, B.PLAN_FUSED | B.PLAN_BEYOND_TABLE3, 1, iters=20, rewrite=B.REWRITE_CANON_MACRO, per_block_limit=0)
    torch.cuda.empty_cache()
    return {"workload": "configs[4]: 12-layer encoder, 576 operators, bf16; CUDA-graph replays", "cfg5_fused_us": f["us_cuda_graph"],
            "cfg5_beyond_table3_us": x["us_cuda_graph"], "cfg5_beyond_table3_kernels": x["kernels"],
            "cfg5_unfused_us": u["us_cuda_graph"], "cfg5_fused_plain_us": f["us_plain_launches"],
            "cfg5_unfused_plain_us": u["us_plain_launches"], "cfg5_fused_kernels": f["kernels"], "cfg5_unfused_kernels": u["kernels"],
            "cfg5_sum_of_block_rooflines_us": 160.0}


def layout_report(dev, pk):
    """Layout selection (Section 4.4.2) on the MobileNetV2-shaped stack: the network written channels-first with a
    Transpose around every convolution and pool, planned with and without the pass, beside the channels-last network."""
    import torch
    out = {}
    for name, wl, rw in [("channels-last graph", W.mbconv_stack(), B.REWRITE_DEFAULT),
                         ("channels-first graph, layout selection", W.mbconv_stack(layout="nchw"), B.REWRITE_DEFAULT),
                         ("channels-first graph, Transposes kept", W.mbconv_stack(layout="nchw"), B.REWRITE_KEEP_LAYOUT)]:
        r = measure_workload(torch, dev, wl, pk, B.PLAN_FUSED, 1, iters=20, rewrite=rw, per_block_limit=0)
        out[name] = {k: r[k] for k in ("ops", "kernels", "us_cuda_graph", "us_plain_launches", "irs_bytes")}
        torch.cuda.empty_cache()
    return out


def mbconv_single_kernel_report(dev, pk):
    """The inverted-residual block of configs[3] as three kernels (the paper's rules) and as one (beyond Table 3), from one
    image to the full batch; the planner forms the single kernel only while its tiles fit one wave."""
    import torch
    out = {}
    for n, hw in [(1, 14), (1, 56), (4, 28), (8, 56), (32, 56)]:
        wl = W.mbconv_block(n, hw, hw)
        a = measure_workload(torch, dev, wl, pk, B.PLAN_FUSED, 3, iters=20, per_block_limit=0)
        b = measure_workload(torch, dev, wl, pk, B.PLAN_FUSED | B.PLAN_BEYOND_TABLE3 | B.PLAN_MBCONV_ALWAYS, 3, iters=20, per_block_limit=0)
        c = measure_workload(torch, dev, wl, pk, B.PLAN_FUSED | B.PLAN_BEYOND_TABLE3, 3, iters=20, per_block_limit=0)
        out["[%d,%d,%d,24->144->24]" % (n, hw, hw)] = {"three_kernels_us": a["us_cuda_graph"], "one_kernel_us": b["us_cuda_graph"],
                                                        "planner_forms_it": c["kernels"] == 1}
        torch.cuda.empty_cache()
    return out
