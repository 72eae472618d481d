#!/usr/bin/env python
"""Benchmark of the WTConv hot path (forward + backward) on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME] [--no-table]

Headline workload (default): the full WTConvNeXt-T stage set in bf16 storage / fp32 arithmetic at B = 128
per GPU, k = 5: (C=96, 56x56, L=3), (C=192, 28x28, L=2), (C=384, 14x14, L=1), (C=768, 7x7, L=1).  One
"step" = wtconv_forward + wtconv_backward on each of the four stage tensors.  Prints ONE JSON line.

  value          elements/s: sum of the stages' B*C*H*W per step (times the ranks) / step time, inputs in HBM
  ms_per_step    median over repeated regions of exactly K steps (regions repeat until >= 0.5 s is timed)
  e2e            the same metric through wtconv_step_host: pinned HOST buffers, H2D and D2H copies inside
  roofline       the dominant kernel of the stage that sits furthest below its roof, against the FP32 ALU roof
  per_workload   every benchmark configuration (level sweep fp32/fp16, stage-1 fp32, the stage set, the
                 network's depth schedule, k = 3 / 7, the large planes) with forward / backward time,
                 elements/s, ALU and HBM fractions and the kernel family that served it (N = 1 only)
  comparator     per level count L of the sweep: this library's own reference-style chain (separate operators,
                 every intermediate in HBM, Sec. 3.1) timed beside the fused kernels, the cumulative ablation of
                 Table 8 on the forward pass, and ncu DRAM bytes per element against Eq. 2 / Eq. 10 where captured
  cpu_baseline   the fp64 oracle on this machine's host cores on a bounded sample (rank 0, N = 1 only)

`--workload NAME` times that single workload instead of the stage set (used for profiler captures).
Under torchrun (N > 1) every rank runs the same per-rank batch (weak scaling); the parameter gradients of
a stage live in one flat buffer that is summed across ranks with one NCCL all-reduce per stage and step.
`--impl reference` times the CPU oracle instead (rank 0 only).
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

FP32_ALU_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12  # SMs x FP32 lanes x 2 FLOP x max SM clock = 74.4
PEAK_SOURCE = "derived: 148 SMs x 128 FP32 lanes x 2 FLOP x 1.965 GHz (a packed-FMA loop measured 74.1 on this pool)"
L2_BYTES = 126 << 20

STAGE_SET = ["stage1_bf16", "stage2_bf16", "stage3_bf16", "stage4_bf16"]
TABLE = (["stage1_f32"] + ["sweep_L%d_f32" % l for l in range(1, 6)] + ["sweep_L%d_f16" % l for l in range(1, 6)] +
         STAGE_SET + ["convnext_s%d_bf16" % s for s in range(1, 5)] + ["stage1_k3_f32", "stage1_k7_f32"] +
         ["large_f16", "large_odd_f16"])

# dram__bytes_read.sum + dram__bytes_write.sum per library call from the ncu captures summarised under profiles/
# (bytes; keyed by workload and path).  Absent = no capture of that call exists.
NCU_DRAM_TRAFFIC = {
    # profiles/io_model_traffic_f32.md
    ("traffic_L1_f32", "reference_fwd"): 4271524242, ("traffic_L1_f32", "tiled_fwd"): 1333854757,
    ("traffic_L3_f32", "reference_fwd"): 5002461952, ("traffic_L3_f32", "tiled_fwd"): 1597085367,
    ("traffic_L5_f32", "reference_fwd"): 5039999049, ("traffic_L5_f32", "tiled_fwd"): 1607475639,
    # profiles/plane_kernels_stage_set_bf16_sections.md (kernel + epilogue of one call)
    ("stage1_bf16", "plane_fwd"): 104200000, ("stage1_bf16", "plane_bwd"): 201700000,
    # profiles/large_planes_traffic.md
    ("large_f16", "window_fwd"): 1797000000, ("large_f16", "window_bwd"): 3089000000,
    ("large_f16", "tiled_fwd"): 4988000000, ("large_f16", "tiled_bwd"): 7101000000,
    ("large_odd_f16", "window_fwd"): 1387000000, ("large_odd_f16", "window_bwd"): 2383000000,
    ("sweep_L3_f32", "reference_fwd"): 948305810, ("sweep_L3_f32", "tiled_fwd"): 320324425, ("sweep_L3_f32", "plane_fwd"): 89365248,
}


def load_measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return json.load(open(p)), "measured"
        except Exception:
            pass
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "sm_max_mhz": 1965.0}, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.samples, self.proc, self.gpu = [], None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            f = [s.strip() for s in line.split(",")]
            if len(f) >= 7:
                self.samples.append((time.time(), f))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        inside = [f for (t, f) in self.samples if t0 - 0.05 <= t <= t1 + 0.05] or [f for (_, f) in self.samples[-3:]]
        mhz, reasons, smax, pw = [], set(), None, []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for f in inside:
            try:
                mhz.append(float(f[0])); smax = float(f[1]); pw.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        mhz.sort()
        return {"sm_mhz": mhz[len(mhz) // 2] if mhz else None, "sm_max_mhz": smax, "reasons": sorted(reasons),
                "samples": len(mhz), "power_w_max": max(pw) if pw else None}


def oracle_step_seconds(wls, reps):
    """Seconds per fwd+bwd of the fp64 oracle over the given (batch-reduced) workloads; returns (s, elements)."""
    from oracle import wtconv_oracle as O
    from paper_2608_10805_b200 import inputs
    Is = [inputs.make_inputs(w) for w in wls]
    def step():
        for w, I in zip(wls, Is):
            O.forward(I["x"], I["w0"], I["s0"], None, I["wl"], I["sl"], w.L)
            O.backward(I["x"], I["g"], I["w0"], I["s0"], None, I["wl"], I["sl"], w.L)
    step()
    t0 = time.time()
    for _ in range(reps):
        step()
    return (time.time() - t0) / reps, sum(w.N for w in wls)


def run_reference(args, wls, name):
    """The CPU oracle, as it stands, on this machine's host cores (bounded sample of the workload)."""
    from oracle import wtconv_oracle as O
    if int(os.environ.get("RANK", "0")) != 0:
        return
    Bs = min(min(w.B for w in wls), args.ref_batch)
    sample_wls = [w.with_(B=Bs) for w in wls]
    steps = max(1, min(args.steps, 5))
    dt, n = oracle_step_seconds(sample_wls, steps)
    val = n / dt
    sample = "fwd+bwd of B=%d of %d images of %s (per-plane cost is batch-independent)" % (Bs, wls[0].B, name)
    print(json.dumps({
        "impl": "reference", "metric": "wtconv_fwd_bwd_elements_per_s", "value": val, "unit": "elements/s",
        "n_gpus": args.gpus, "steps": steps, "warmup": 1, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": name, "stages": [w.name for w in wls], "sample_B": Bs},
        "cpu_baseline": {"value": val, "unit": "elements/s", "cores": O.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": val, "unit": "elements/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


class Runner:
    """Device buffers of one workload and the two library calls of a step."""

    def __init__(self, wl, dev, rank, tune, torch, wt, inputs, dp):
        self.wl, self.torch, self.wt = wl, torch, wt
        tdt = wt.DTYPE_NAMES[wl.dtype]
        self.esz = 4 if wl.dtype == "f32" else 2
        self.desc = wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, tdt, tune)
        # rotating input sets: together with the outputs a pass over all sets touches more than the L2 holds
        step_bytes = 4 * wl.N * self.esz
        self.nbuf = 1 if step_bytes > 2 * L2_BYTES else min(8, -(-2 * L2_BYTES // step_bytes) + 1)
        gen = torch.Generator(device=dev)
        gen.manual_seed(1000 * wl.seed + 17 * rank + 1)
        shape = (wl.B, wl.C, wl.H, wl.W)
        self.xs = [torch.randn(shape, generator=gen, device=dev, dtype=torch.float32).to(tdt) for _ in range(self.nbuf)]
        self.gs = [torch.randn(shape, generator=gen, device=dev, dtype=torch.float32).to(tdt) for _ in range(self.nbuf)]
        P = inputs.make_inputs(wl.with_(B=1))  # parameters do not depend on B (own Philox stream per tensor)
        up = lambda a: torch.from_numpy(a).to(dev).contiguous()
        self.w0, self.s0, self.wl_, self.sl = up(P["w0"]), up(P["s0"]), up(P["wl"]), up(P["sl"])
        self.out, self.gx = torch.empty_like(self.xs[0]), torch.empty_like(self.xs[0])
        self.grads = dp.FlatGrads(wl.C, wl.k, wl.L, bias=False, device=dev)
        self.ws = wt.alloc_workspace(self.desc, dev)
        self.ws_fwd, self.ws_bwd = wt.wtconv_workspace_bytes(self.desc)
        self.nf, self.nb = wt.wtconv_launch_count(self.desc)
        self.plan = wt.wtconv_plan_name(self.desc)

    def fwd(self, i, stream):
        self.wt.wtconv_forward(self.desc, self.xs[i % self.nbuf], self.w0, self.s0, None, self.wl_, self.sl, self.out,
                               self.ws, stream)

    def bwd(self, i, stream):
        g = self.grads
        self.wt.wtconv_backward(self.desc, self.xs[i % self.nbuf], self.gs[i % self.nbuf], self.w0, self.s0, None,
                                self.wl_, self.sl, self.gx, g["dw0"], g["ds0"], None, g["dwl"], g["dsl"], self.ws, stream)

    def device_bytes(self):
        act = self.wl.N * self.esz
        par = 4 * sum(t.numel() for t in (self.w0, self.s0, self.wl_, self.sl))
        return {"x": act, "out": act, "params": par, "workspace_fwd": self.ws_fwd, "workspace_bwd": self.ws_bwd,
                "forward_peak": 2 * act + par + self.ws_fwd,
                "training_step_peak": 4 * act + 2 * par + max(self.ws_fwd, self.ws_bwd)}


def time_regions(runners, K, warmup, stream, torch, sync_all, all_reduce, min_seconds, max_regions, direction="both"):
    """Milliseconds of regions of exactly K steps (nothing but the library calls and the gradient exchange on the
    stream), repeated until `min_seconds` have been timed."""
    def step(i):
        for r in runners:
            if direction != "bwd":
                r.fwd(i, stream)
            if direction != "fwd":
                r.bwd(i, stream)
            all_reduce(r)
    for i in range(warmup):
        step(i)
    sync_all()
    regions, total = [], 0.0
    while len(regions) < max_regions and (total < min_seconds or not regions):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sync_all()
        e0.record(stream)
        for i in range(K):
            step(i)
        e1.record(stream)
        sync_all()
        regions.append(e0.elapsed_time(e1))
        total += regions[-1] * 1e-3
    return regions


def time_calls(fn, K, reps, stream, torch, sync_all):
    """Milliseconds per call: median over `reps` regions of K consecutive calls of one kind with nothing between them
    on the stream (as in a training loop, a call may start its set-up behind the tail of the call before it)."""
    for i in range(2):
        fn(i)
    sync_all()
    ts = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(K):
            fn(i)
        e1.record(stream)
        sync_all()
        ts.append(e0.elapsed_time(e1) / K)
    return statistics.median(ts)


def row_for(r, fwd_ms, bwd_ms, peaks, io_model):
    wl = r.wl
    fl_f = io_model.algorithmic_flops(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, "fwd")
    by_f = io_model.compulsory_bytes(wl.N, r.esz, "fwd")
    by_s = io_model.compulsory_bytes(wl.N, r.esz, "fwd+bwd")
    peak_f, peak_b = FP32_ALU_PEAK_TFLOPS * 1e12, peaks["hbm_gbs"] * 1e9
    t_f, t_b = fwd_ms * 1e-3, bwd_ms * 1e-3
    t_s = t_f + t_b
    alu_floor, hbm_floor = 3 * fl_f / peak_f, by_s / peak_b
    return {
        "workload": wl.name, "shape": [wl.B, wl.C, wl.H, wl.W], "k": wl.k, "L": wl.L, "storage": wl.dtype,
        "plan": r.plan, "launches": [r.nf, r.nb],
        "fwd_us": round(fwd_ms * 1e3, 2), "bwd_us": round(bwd_ms * 1e3, 2),
        "fwd_gelem_s": round(wl.N / t_f / 1e9, 2), "gelem_s": round(wl.N / t_s / 1e9, 2),
        "fwd_alu_frac": round(fl_f / t_f / peak_f, 4), "bwd_alu_frac": round(2 * fl_f / t_b / peak_f, 4),
        "alu_frac": round(3 * fl_f / t_s / peak_f, 4),
        "fwd_hbm_frac_of_measured": round(by_f / t_f / peak_b, 4), "hbm_frac_of_measured": round(by_s / t_s / peak_b, 4),
        "bound": "alu" if alu_floor >= hbm_floor else "hbm",
        "roof_frac": round(max(alu_floor, hbm_floor) / t_s, 4),
        "workspace_bytes": [r.ws_fwd, r.ws_bwd],
        "ncu_dram_bytes": {k_[1]: v_ for k_, v_ in NCU_DRAM_TRAFFIC.items() if k_[0] == wl.name} or None,
        "compulsory_bytes": [by_f, by_s - by_f],
        "paper_q_fused_fwd_N": round(io_model.q_fused(wl.L), 3) if wl.L else None,
        "paper_q_ref_fwd_N": round(io_model.q_ref(wl.L), 3) if wl.L else None,
    }


# Paper's own ratios on its hardware (RTX A6000, k = 5, geometric mean over its layer sweep), context only:
# Table 2 (training step, reference / fused) and Table 3 (forward), fp32, L = 1..5.
PAPER_TRAIN_RATIO_F32 = [3.71, 4.23, 4.34, 4.35, 4.33]
PAPER_FWD_RATIO_F32 = [3.67, 4.20, 4.32, 4.35, 4.37]


def comparator_rows(names, mk, wt, io_model, stream, torch, sync_all, have):
    """Reference-style chain and ablation steps next to the fused kernels, one row per workload."""
    REF, FA, CS = wt.FLAG_REFERENCE_CHAIN, wt.FLAG_ABLATE_FUSED_ANALYSIS, wt.FLAG_ABLATE_COLLAPSED_SYNTHESIS
    def timed(fn, reps):  # the protocol of the fused rows: consecutive calls, nothing between them
        return time_calls(fn, 3, reps, stream, torch, sync_all) * 1e3

    out = []
    for name in names:
        ours = have[name]
        row = {"workload": name, "L": ours["L"], "storage": ours["storage"],
               "fused_fwd_us": ours["fwd_us"], "fused_train_step_us": round(ours["fwd_us"] + ours["bwd_us"], 2)}
        from paper_2608_10805_b200 import inputs
        wl = inputs.WORKLOADS[name]
        r = mk(wl, REF)
        row["reference_fwd_us"] = round(timed(lambda i: r.fwd(i, stream), 5), 1)
        row["reference_train_step_us"] = round(timed(lambda i: r.bwd(i, stream), 3), 1)  # this call = forward chain + backward chain
        row["reference_launches"] = [r.nf, r.nb]
        row["reference_workspace_bytes"] = [r.ws_fwd, r.ws_bwd]
        del r
        torch.cuda.empty_cache()
        abl = {"reference": row["reference_fwd_us"]}
        for label, fl in (("+fused_analysis", REF | FA), ("+collapsed_synthesis", REF | FA | CS), ("+scale_folding", wt.FLAG_TILED_ONLY)):
            r = mk(wl, fl)
            abl[label] = round(timed(lambda i: r.fwd(i, stream), 5), 1)
            del r
            torch.cuda.empty_cache()
        abl["whole_plane_kernels"] = ours["fwd_us"]
        row["ablation_fwd_us"] = abl
        row["fwd_ratio_reference_over_fused"] = round(row["reference_fwd_us"] / ours["fwd_us"], 2)
        row["train_ratio_reference_over_fused"] = round(row["reference_train_step_us"] / row["fused_train_step_us"], 2)
        if ours["storage"] == "f32" and 1 <= ours["L"] <= 5:
            row["paper_a6000_ratio"] = {"fwd": PAPER_FWD_RATIO_F32[ours["L"] - 1], "train": PAPER_TRAIN_RATIO_F32[ours["L"] - 1]}
        n = wl.N
        row["io_model_N"] = {"q_ref_fwd": round(io_model.q_ref(wl.L), 3), "q_fused_fwd": round(io_model.q_fused(wl.L), 3),
                             "ours_fwd_compulsory": 2.0}
        meas = {}
        for kind in ("reference_fwd", "tiled_fwd", "plane_fwd", "plane_bwd"):
            v = NCU_DRAM_TRAFFIC.get((name, kind))
            if v is not None:
                meas[kind] = round(v / (n * (4 if wl.dtype == "f32" else 2)), 3)
        if meas:
            row["ncu_dram_bytes_per_element_over_elem_size"] = meas
        out.append(row)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="stage_set_bf16", help="stage_set_bf16 (default) or one workload name")
    ap.add_argument("--ref-batch", type=int, default=16, help="images per oracle step in --impl reference")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--min-seconds", type=float, default=0.5, help="repeat the K-step region until this much is timed")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-table", action="store_true", help="skip the per_workload table")
    ap.add_argument("--no-comparator", action="store_true", help="skip the reference-chain / ablation rows")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--tune", type=lambda s: int(s, 0), default=0, help="desc.flags: path selection and launch-plan override bits (see wtconv.h)")
    ap.add_argument("--direction", default="both", choices=["both", "fwd", "bwd"],
                    help="profiler captures: enqueue only the forward or only the backward call of every step")
    args = ap.parse_args()

    from paper_2608_10805_b200 import inputs, io_model
    names = STAGE_SET if args.workload == "stage_set_bf16" else [args.workload]
    wls = [inputs.WORKLOADS[n] for n in names]
    head_name = "wtconvnext_t_stage_set_bf16_B128" if args.workload == "stage_set_bf16" else args.workload
    if args.impl == "reference":
        return run_reference(args, wls, head_name)

    import torch
    import torch.distributed as dist
    from paper_2608_10805_b200 import dp
    from paper_2608_10805_b200 import wtconv as wt

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the WTConv library has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)
    wt.lib()  # fail loudly here if the CUDA library is missing
    stream = torch.cuda.current_stream()

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def all_reduce(r):
        if world > 1:
            r.grads.all_reduce()  # one collective per stage and step: the flat parameter-gradient buffer

    mk = lambda w, tune=0: Runner(w, dev, rank, tune, torch, wt, inputs, dp)
    runners = [mk(w, args.tune) for w in wls]
    K, W = max(args.steps, 1), max(args.warmup, 3)
    for i in range(3):  # first calls: plan search, function attributes, module load
        for r in runners:
            if args.direction != "bwd":
                r.fwd(i, stream)
            if args.direction != "fwd":
                r.bwd(i, stream)
    sync_all()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.2)
    t0 = time.time()
    # the headline: plain sequences of calls, nothing between them on the stream
    regions = time_regions(runners, K, W, stream, torch, sync_all, all_reduce, args.min_seconds, 400, args.direction)
    # the per-call split behind the roofline entries: each call of the step on its own, K in a row
    if args.direction == "both":
        fwd_ms = [time_calls(lambda i, r=r: r.fwd(i, stream), K, 5, stream, torch, sync_all) for r in runners]
        bwd_ms = [time_calls(lambda i, r=r: r.bwd(i, stream), K, 5, stream, torch, sync_all) for r in runners]
    else:  # a profiling run of one direction: no split
        fwd_ms = bwd_ms = [1e-6 for _ in runners]
    t1 = time.time()
    med = statistics.median(regions)
    ms = torch.tensor([med], device=dev)
    if world > 1:
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    ms_region = float(ms.item())
    clocks = sampler.stop(t0, t1) if rank == 0 else None

    # ---- end to end through the host entry point: pinned host buffers, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        host = []
        for r in runners:
            hb = lambda t: torch.empty(t.shape, dtype=t.dtype).pin_memory()
            g = r.grads
            host.append(dict(
                hx=r.xs[0].cpu().pin_memory(), hg=r.gs[0].cpu().pin_memory(),
                hp=[t.cpu().pin_memory() for t in (r.w0, r.s0, r.wl_, r.sl)],
                ho=[hb(r.out), hb(r.gx), hb(g["dw0"]), hb(g["ds0"]), hb(g["dwl"]), hb(g["dsl"])],
                ws=torch.empty(wt.wtconv_step_host_workspace_bytes(r.desc), dtype=torch.uint8, device=dev)))

        def host_step():
            for r, h in zip(runners, host):
                wt.wtconv_step_host(r.desc, h["hx"], h["hg"], h["hp"][0], h["hp"][1], None, h["hp"][2], h["hp"][3],
                                    h["ho"][0], h["ho"][1], h["ho"][2], h["ho"][3], None, h["ho"][4], h["ho"][5],
                                    h["ws"], stream)
        host_step()
        sync_all()
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record(stream)
        for _ in range(args.e2e_steps):
            host_step()
        h1.record(stream)
        sync_all()
        hms = torch.tensor([h0.elapsed_time(h1)], device=dev)
        if world > 1:
            dist.all_reduce(hms, op=dist.ReduceOp.MAX)
        n_step = sum(r.wl.N for r in runners)
        psz = sum(4 * sum(t.numel() for t in (r.w0, r.s0, r.wl_, r.sl)) for r in runners)
        act = sum(2 * r.wl.N * r.esz for r in runners)
        e2e = {"value": n_step * world * args.e2e_steps / (float(hms.item()) * 1e-3), "unit": "elements/s",
               "h2d_bytes_per_step": act + psz, "d2h_bytes_per_step": act + psz, "steps": args.e2e_steps,
               "api": "wtconv_step_host (host pointers; uploads, kernels and downloads pipelined by batch chunk)"}
        del host

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks, peak_kind = load_measured_peaks()
    ms_step = ms_region / K
    n_step = sum(r.wl.N for r in runners)
    value = n_step * world / (ms_step * 1e-3)
    rows = [row_for(r, f, b, peaks, io_model) for r, f, b in zip(runners, fwd_ms, bwd_ms)]
    fl_step = sum(io_model.algorithmic_flops(r.wl.B, r.wl.C, r.wl.H, r.wl.W, r.wl.k, r.wl.L, "fwd+bwd") for r in runners)
    by_step = sum(io_model.compulsory_bytes(r.wl.N, r.esz, "fwd+bwd") for r in runners)
    alu_floor_ms = fl_step / (FP32_ALU_PEAK_TFLOPS * 1e12) * 1e3
    hbm_floor_ms = by_step / (peaks["hbm_gbs"] * 1e9) * 1e3
    # roofline: the dominant kernel = the library call with the largest share of the step time; the call furthest below
    # its roof is reported beside it (roofline_worst_call)
    def call_entry(j, kind):
        r_, row_ = runners[j], rows[j]
        f_ = io_model.algorithmic_flops(r_.wl.B, r_.wl.C, r_.wl.H, r_.wl.W, r_.wl.k, r_.wl.L, "fwd")
        ms_, fl_ = (bwd_ms[j], 2 * f_) if kind == "backward" else (fwd_ms[j], f_)
        ach_ = fl_ / (ms_ * 1e-3) / 1e12
        return {"bound": row_["bound"], "kernel": "%s call of %s (%s kernels)" % (kind, r_.wl.name, r_.plan),
                "achieved": ach_, "peak": FP32_ALU_PEAK_TFLOPS, "unit": "TFLOP/s", "frac": ach_ / FP32_ALU_PEAK_TFLOPS,
                "traffic": NCU_DRAM_TRAFFIC.get((r_.wl.name, "plane_bwd" if kind == "backward" else "plane_fwd")),
                "peak_source": PEAK_SOURCE, "launch_ms": ms_, "flops_per_launch": fl_,
                "share_of_step": ms_ / (sum(fwd_ms) + sum(bwd_ms))}
    calls = [call_entry(j, kind) for j in range(len(rows)) for kind in ("forward", "backward")]
    dominant = max(calls, key=lambda c_: c_["launch_ms"])
    worst_call = min(calls, key=lambda c_: c_["frac"])
    result = {
        "metric": "wtconv_fwd_bwd_elements_per_s", "value": value, "unit": "elements/s", "n_gpus": world,
        "steps": K, "warmup": W, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": wt.ARITHMETIC_DTYPE, "data": "synthetic",
        "config": {"workload": head_name,
                   "stages": [{"name": r.wl.name, "B_per_gpu": r.wl.B, "C": r.wl.C, "H": r.wl.H, "W": r.wl.W, "k": r.wl.k,
                               "L": r.wl.L, "storage_dtype": r.wl.dtype, "plan": r.plan} for r in runners],
                   "l2": "a step touches %d MB (> 126 MB L2) over rotating input sets" %
                         (sum(4 * r.wl.N * r.esz * (r.nbuf if len(runners) == 1 else 1) for r in runners) >> 20),
                   "timing": "median of %d regions of %d steps (%.2f s timed), CUDA events on the launch stream around each "
                             "region, nothing between the calls; per-call times: median of 5 regions of %d consecutive "
                             "calls of that kind (their sum: %.4f ms per step)"
                             % (len(regions), K, sum(regions) * 1e-3, K, sum(fwd_ms) + sum(bwd_ms)),
                   "parallelism": "dp%d (batch-sharded; one all-reduce of the flat parameter-gradient buffer per stage)" % world},
        "clocks": clocks,
        "ms_per_step_x_sm_mhz": ms_step * clocks["sm_mhz"] if clocks and clocks.get("sm_mhz") else None,
        "region_ms": {"min": min(regions), "median": med, "max": max(regions), "n": len(regions)},
        "e2e": e2e,
        "gpu_launches": sum(r.nf + r.nb for r in runners) * K,
        "roofline": dominant,
        "roofline_worst_call": worst_call,
        "roofline_calls": [{"kernel": c_["kernel"], "launch_ms": round(c_["launch_ms"], 4), "frac": round(c_["frac"], 4),
                            "share_of_step": round(c_["share_of_step"], 4)} for c_ in calls],
        "step_rooflines": {
            "alu_frac": alu_floor_ms / ms_step,
            "hbm_compulsory_gbs": by_step / (ms_step * 1e-3) / 1e9,
            "hbm_frac_of_%s" % peak_kind: hbm_floor_ms / ms_step,
            "hbm_frac_of_8TBs": by_step / (ms_step * 1e-3) / 1e9 / 8000.0,
            "alu_floor_ms": alu_floor_ms, "hbm_floor_ms": hbm_floor_ms,
            "roof_frac": max(alu_floor_ms, hbm_floor_ms) / ms_step},
        "device_bytes": {r.wl.name: r.device_bytes() for r in runners},
        "stages": rows,
    }
    if world == 1 and not args.no_cpu_baseline:
        from oracle import wtconv_oracle as O
        Bs = min(min(w.B for w in wls), 32)
        cdt, cn = oracle_step_seconds([w.with_(B=Bs) for w in wls], 3)
        result["cpu_baseline"] = {"value": cn / cdt, "unit": "elements/s", "cores": O.num_threads(),
                                  "kind": "oracle", "seconds_per_step": cdt,
                                  "sample": "3 x fwd+bwd of B=%d images of %s, fp64 (%.0f core-seconds)"
                                            % (Bs, head_name, 3 * cdt * O.num_threads())}
    if world == 1 and not args.no_table:
        table = []
        have = {r.wl.name: row for r, row in zip(runners, rows)}
        del runners
        torch.cuda.empty_cache()
        for name in TABLE:
            if name in have:
                table.append(have[name])
                continue
            r = mk(inputs.WORKLOADS[name])
            k = 3 if r.wl.N > (1 << 27) else 10
            f = time_calls(lambda i: r.fwd(i, stream), k, 5, stream, torch, sync_all)
            b = time_calls(lambda i: r.bwd(i, stream), k, 5, stream, torch, sync_all)
            table.append(row_for(r, f, b, peaks, io_model))
            del r
            torch.cuda.empty_cache()
        result["per_workload"] = table
        if not args.no_comparator:
            byname = {r_["workload"]: r_ for r_ in table}
            result["io_model_validation"] = [
                {"workload": w_, "N": inputs.WORKLOADS[w_].N, "L": inputs.WORKLOADS[w_].L,
                 "ncu_dram_over_4N": {k_: round(NCU_DRAM_TRAFFIC[(w_, k_)] / (4.0 * inputs.WORKLOADS[w_].N), 3)
                                      for k_ in ("reference_fwd", "tiled_fwd") if (w_, k_) in NCU_DRAM_TRAFFIC},
                 "model": {"q_ref": round(io_model.q_ref(inputs.WORKLOADS[w_].L), 3),
                           "q_fused_minus_base_pass": round(io_model.q_fused(inputs.WORKLOADS[w_].L) - 2.0, 3)},
                 "source": "profiles/io_model_traffic_f32.md"}
                for w_ in ("traffic_L1_f32", "traffic_L3_f32", "traffic_L5_f32")]
            result["comparator"] = comparator_rows(["sweep_L%d_f32" % l for l in range(1, 6)] + ["sweep_L3_f16", "stage1_f32"],
                                                   mk, wt, io_model, stream, torch, sync_all, byname)
    print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
