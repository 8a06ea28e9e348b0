#!/usr/bin/env python
"""Benchmark of the fused-block executor on one B200.

Default arm: `python bench.py --gpus N --steps K --warmup W` prints ONE short JSON line
(the last line of stdout).

A step is one pass of the hot path -- dnnf_run of the fused MobileNetV2-style
inverted-residual block (fp32 NHWC [32,56,56,24 -> 144 -> 24]: pointwise expansion +
BN + ReLU6, depthwise 3x3 + BN + ReLU6, pointwise projection + BN + residual; three
kernels) -- over one batch of 32 synthetic images.  It is the largest memory-bound
configuration: 260.1 MB of algorithmic traffic per step.  Consecutive steps rotate
over SETS complete, independent buffer sets (inputs, intermediates, outputs) so that
no step finds its data in L2.

  value     algorithmic GB/s over the whole step (every block's external inputs and
            outputs once), inputs resident in HBM, plain stream launches of dnnf_run
  roofline  the longest kernel of the step by its own CUDA-event time (a second pass
            over the same steps with an event between the blocks)
  e2e       the same step with the images copied from pinned host memory and the
            result copied back inside the timed region
  graph_latency  the metric's second half: the 12-layer encoder (576 primitive
            operators) fused against one kernel per operator, CUDA-graph replays

`--detail` writes the per-configuration / per-block tables to
bench_detail.json in the output folder (OUT_DIR below).  `--impl reference` times the CPU oracle on the same
workload (bounded sample).
"""
from __future__ import annotations

OUT_DIR = "gpurun_out"      # where files that a run produces go

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "fused-block GB/s as % of HBM peak; graph latency fused vs unfused per-op"
UNIT = "GB/s"
SETS = 3
WORKLOAD = "configs[3]: MobileNetV2-style inverted-residual block, fp32 NHWC [32,56,56,24->144->24], 3 fused kernels"


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"], "bf16_tflops_sustained": d["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    def __init__(self, index=0):
        self.samples = []
        self.reasons = set()
        self.stop = threading.Event()
        self.index = index
        self.th = None

    def _run(self):
        q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        while not self.stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits", "-i", str(self.index)],
                                     capture_output=True, text=True, timeout=5).stdout.strip().split(",")
                self.samples.append((float(out[0]), float(out[1])))
                for n, v in zip(names, out[2:]):
                    if v.strip().lower().startswith("active"):
                        self.reasons.add(n)
            except Exception:
                pass
            self.stop.wait(0.1)

    def __enter__(self):
        self.th = threading.Thread(target=self._run, daemon=True)
        self.th.start()
        return self

    def __exit__(self, *a):
        self.stop.set()
        self.th.join(timeout=6)

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": sorted(self.reasons)}
        sm = sorted(s[0] for s in self.samples)
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(s[1] for s in self.samples), "reasons": sorted(self.reasons),
                "samples": len(sm)}


def max_over_ranks(value, device=None):
    """Slowest rank's time (all ranks get it).  Works with any initialised backend (nccl on GPUs, gloo on CPU)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(bytes_per_rank_step, ms_step_max, world):
    """Whole-job GB/s when every rank processes its own replica of the step (weak scaling, no exchange step)."""
    return world * bytes_per_rank_step / (ms_step_max * 1e-3) / 1e9


def rank_seed(base_seed, rank):
    """Each replica draws its own inputs."""
    return base_seed + 100 * rank


def block_bytes(sess):
    return [sess.g.block_info(b).bytes_in + sess.g.block_info(b).bytes_out for b in range(sess.g.block_count())]


def mbconv_algorithmic_bytes(n=32, h=56, w=56, cin=24, cexp=144):
    """External inputs and outputs of the three fused blocks, each once (fp32)."""
    x, e = n * h * w * cin, n * h * w * cexp
    blocks = [x + cin * cexp + 2 * cexp + e,            # expansion: X, W1, scale, shift -> E
              e + 9 * cexp + 2 * cexp + e,              # depthwise: E, Kd, scale, shift -> E2
              e + cexp * cin + 2 * cin + x + x]         # projection: E2, W3, scale, shift, X -> Y
    return [4 * b for b in blocks]


def oracle_pass_timer(wl):
    """Times the oracle on the workload; returns (seconds per pass, passes, threads it kept busy)."""
    from oracle import interp as O
    O.run_graph(wl.graph, wl.inputs)
    n, t0, c0 = 0, time.perf_counter(), time.process_time()
    while time.perf_counter() - t0 < 10.0 or n < 2:
        O.run_graph(wl.graph, wl.inputs)
        n += 1
    wall, cpu = time.perf_counter() - t0, time.process_time() - c0
    return wall / n, n, max(1, int(round(cpu / wall)))


# --------------------------------------------------------------------------------------
def run_reference(args):
    """CPU oracle arm: the unfused fp64 interpreter on the host cores, same workload and metric."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import interp as O
    from paper_2108_13342_b200 import workloads as W
    n_img = 4                                         # bounded sample: 4 of the step's 32 images per reference step
    wl = W.mbconv_block(n=n_img)
    bytes_step = sum(mbconv_algorithmic_bytes(n=n_img))      # the step's algorithmic bytes, scaled to the sample
    for _ in range(max(1, min(args.warmup, 1))):
        O.run_graph(wl.graph, wl.inputs)
    t0, c0 = time.perf_counter(), time.process_time()
    for _ in range(args.steps):
        O.run_graph(wl.graph, wl.inputs)
    wall, cpu = time.perf_counter() - t0, time.process_time() - c0
    dt = wall / args.steps
    cores = max(1, int(round(cpu / wall)))
    val = bytes_step / dt / 1e9
    sample = f"{n_img} of the step's 32 images per reference step, numpy fp64 unfused interpreter"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": {"workload": WORKLOAD + "; " + sample},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# --------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="dnnf")
    ap.add_argument("--detail", action="store_true", help="also write per-configuration / per-block tables to bench_detail.json in the output folder")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-graph-latency", action="store_true", help="skip the encoder fused / unfused latency pair")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import torch.distributed as dist
    from paper_2108_13342_b200 import binding as B
    from paper_2108_13342_b200 import workloads as W
    from paper_2108_13342_b200.runtime import Session

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    pk = peaks()
    steps, warm = args.steps, max(args.warmup, 3)

    # ---- the step: dnnf_run of the fused block on one of SETS independent buffer sets ------------
    wl = W.mbconv_block(seed=rank_seed(W.BASE_SEED, rank))
    S = [Session(wl, rewrite_flags=B.REWRITE_NONE, device=dev) for _ in range(SETS)]
    nb = S[0].g.block_count()
    bbytes = block_bytes(S[0])
    assert bbytes == mbconv_algorithmic_bytes(), (bbytes, mbconv_algorithmic_bytes())
    bytes_step = sum(bbytes)
    stream = torch.cuda.current_stream(dev)
    sptr = stream.cuda_stream

    for i in range(warm):
        S[i % SETS].g.run(sptr)
    torch.cuda.synchronize(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize(dev)
    with ClockSampler(local) as clk:
        e0.record(stream)
        for i in range(steps):
            S[i % SETS].g.run(sptr)
        e1.record(stream)
        torch.cuda.synchronize(dev)
        ms_step = e0.elapsed_time(e1) / steps
        # second pass, one kernel at a time: the same `steps` launches of block b over the rotating buffer sets, back
        # to back on the same stream and with the same launch attributes as inside dnnf_run, between two events.
        # (An event between the blocks of a step would add the gap it creates to every kernel: those figures summed
        # to a quarter more than the step itself; these sum to the step.)
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(nb)]
        for b in range(nb):
            ev[b][0].record(stream)
            for i in range(steps):
                S[i % SETS].g.run_block(b, sptr)
            ev[b][1].record(stream)
        torch.cuda.synchronize(dev)
        # keep the GPU busy a little longer so that the sampler sees clocks under load
        t_end = time.time() + 1.0
        i = 0
        while time.time() < t_end:
            S[i % SETS].g.run(sptr)
            i += 1
            if i % 64 == 0:
                torch.cuda.synchronize(dev)
        torch.cuda.synchronize(dev)
    if world > 1:
        dist.barrier()
    for s in S:
        st, blk = s.g.status()
        if st != 0:
            raise SystemExit(f"device status {st} from block {blk}")
    ms_step = max_over_ranks(ms_step, dev)
    value = aggregate_throughput(bytes_step, ms_step, world)

    blocks = S[0].g.blocks()
    k_us = [ev[b][0].elapsed_time(ev[b][1]) / steps * 1e3 for b in range(nb)]
    kernels = [{"ops": "+".join(blocks[b]["ops"]), "us": round(k_us[b], 2),
                "frac": round(bbytes[b] / (k_us[b] * 1e-6) / 1e9 / pk["hbm_gbs"], 3)} for b in range(nb)]
    top = max(range(nb), key=lambda b: k_us[b])
    ach = bbytes[top] / (k_us[top] * 1e-6) / 1e9
    roof = {"bound": "hbm", "kernel": "%s kernel of block %d (%s)" % (blocks[top]["family"], top, "+".join(blocks[top]["ops"])),
            "achieved": round(ach, 1), "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": round(ach / pk["hbm_gbs"], 4),
            "peak_source": pk["source"], "traffic": None, "bytes_per_launch": bbytes[top], "us_per_launch": round(k_us[top], 3)}
    tp = os.path.join(ROOT, "profiles", "traffic.json")
    if os.path.exists(tp):                       # DRAM bytes per launch of that kernel from the committed ncu capture
        with open(tp) as f:
            tj = json.load(f)
        ent = tj.get("mbconv_block", {}).get(str(top))
        if ent:
            roof["traffic"] = ent["dram_bytes_per_launch"]
            roof["traffic_source"] = "committed ncu capture, profiles/mbconv_fp32_kernels.md"

    # ---- end to end: images from pinned host memory, result back to the host, same C-ABI calls --------
    hin = [torch.from_numpy(wl.inputs["X"]).pin_memory() for _ in range(SETS)]
    hout = [torch.empty_like(hin[0]).pin_memory() for _ in range(SETS)]
    h2d = hin[0].numel() * 4
    d2h = hout[0].numel() * 4
    # Three streams: host->device copies, the blocks, device->host copies (two DMA directions beside the kernels).
    # Events order copy-in -> run -> copy-out per buffer set, and a set's next copy-in after its previous copy-out.
    s_in, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    ev_in = [torch.cuda.Event() for _ in range(SETS)]
    ev_run = [torch.cuda.Event() for _ in range(SETS)]
    ev_out = [torch.cuda.Event() for _ in range(SETS)]
    for e in ev_out + ev_run:
        e.record(stream)

    def e2e_step(i):
        k = i % SETS
        sess = S[k]
        s_in.wait_event(ev_out[k])
        s_in.wait_event(ev_run[k])                 # the residual reads X until the set's last kernel ends
        with torch.cuda.stream(s_in):
            sess.buffers["X"].copy_(hin[k], non_blocking=True)
            ev_in[k].record(s_in)
        stream.wait_event(ev_in[k])
        stream.wait_event(ev_out[k])
        sess.g.run(sptr)
        ev_run[k].record(stream)
        s_out.wait_event(ev_run[k])
        with torch.cuda.stream(s_out):
            hout[k].copy_(sess.buffers["Y"], non_blocking=True)
            ev_out[k].record(s_out)

    e2e_steps = max(3, min(steps, 60))
    for i in range(SETS):
        e2e_step(i)
    stream.wait_stream(s_in); stream.wait_stream(s_out)
    torch.cuda.synchronize(dev)
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record(stream)
    for i in range(e2e_steps):
        e2e_step(i)
    stream.wait_stream(s_in); stream.wait_stream(s_out)     # the region ends when the last result has reached the host
    f1.record(stream)
    torch.cuda.synchronize(dev)
    e2e_ms = max_over_ranks(f0.elapsed_time(f1) / e2e_steps, dev)
    e2e = {"value": round(aggregate_throughput(bytes_step, e2e_ms, world), 1), "unit": UNIT, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "ms_per_step": round(e2e_ms, 4)}

    line = {"metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warm,
            "ms_per_step": round(ms_step, 5), "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": WORKLOAD, "bytes_per_step": bytes_step, "launches_per_step": nb,
                       "l2": f"steps rotate over {SETS} buffer sets of {bytes_step // 2 // 1000000} MB each (> L2)",
                       "launch_mode": "plain stream launches, PDL between kernels"},
            "frac_of_hbm_peak": round(value / world / pk["hbm_gbs"], 4),
            "clocks": clk.summary(), "e2e": e2e, "gpu_launches": steps * nb, "roofline": roof, "kernels": kernels}

    del S
    torch.cuda.empty_cache()
    if rank == 0 and not args.no_graph_latency:
        from paper_2108_13342_b200 import report
        try:
            line["graph_latency"] = report.encoder_latency_pair(dev, pk)
        except Exception as e:      # report, never hide
            line["graph_latency"] = {"error": repr(e)[:200]}
    if rank == 0 and not args.no_cpu:
        sec, n, cores = oracle_pass_timer(W.mbconv_block(n=4))
        line["cpu_baseline"] = {"value": round(sum(mbconv_algorithmic_bytes(n=4)) / sec / 1e9, 4), "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"{n} passes over 4 of the step's 32 images (about {sec * n:.0f} s of CPU work)"}
    if rank == 0 and args.detail:
        from paper_2108_13342_b200 import report
        detail = report.per_config(dev, pk)
        for name, fn in [("cfg5 12-layer encoder (576 primitive operators)", report.encoder_report),
                         ("next: 12-layer GPT-2 style decoder (633 primitive operators)", report.decoder_report),
                         ("next: layout selection on the MobileNetV2-shaped stack written channels-first", report.layout_report),
                         ("beyond Table 3: the inverted-residual block as one kernel", report.mbconv_single_kernel_report)]:
            try:
                detail[name] = fn(dev, pk)
            except Exception as e:  # noqa: BLE001
                detail[name] = {"error": repr(e)}
        detail["paper_context"] = {"note": "mobile-device figures from the paper, not comparable hardware",
                                   "fusion_rate_vs_other_frameworks": "up to 8.8x", "speedup_vs_other_frameworks": "up to 9.3x",
                                   "speedup_vs_own_unfused_backend": "1.5-5.8x"}
        os.makedirs(os.path.join(ROOT, OUT_DIR), exist_ok=True)
        with open(os.path.join(ROOT, OUT_DIR, "bench_detail.json"), "w") as f:
            json.dump(detail, f, indent=1)
    if rank == 0:
        sys.stdout.flush()
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
