#!/usr/bin/env python
"""Benchmark of the WTConv hot path (forward + backward) on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One "step" = wtconv_forward + wtconv_backward over one batch of the workload (default: the
WTConvNeXt-T stage-1 block shape in fp32, B=64 C=96 56x56 k=5 L=3).  Prints ONE JSON line.

  value        elements/s (N = B*C*H*W per step and rank, summed over ranks), inputs resident in HBM
  e2e          the same metric through wtconv_step_host: pinned HOST buffers, H2D and D2H copies inside
  roofline     the dominant kernel (the whole-plane forward / input-gradient kernel) against the FP32
               ALU roof, from CUDA events around the forward call inside the timed steps
  cpu_baseline the fp64 oracle on this machine's host cores (rank 0, N=1 only)

Under torchrun (N > 1) every rank runs the same per-rank batch (weak scaling); the parameter
gradients are summed across ranks with one NCCL all-reduce per step (the only exchange the
batch-sharded operator has).  `--impl reference` times the CPU oracle instead (rank 0 only).
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

FP32_ALU_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12  # SMs x FP32 lanes x 2 FLOP x max SM clock = 74.4

# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under profiles/
# (bytes; keyed by workload and kernel).  None where no capture exists.
NCU_DRAM_TRAFFIC = {
    ("stage1_f32", "plane_bwd_kernel"): 154664704 + 48539904,
    ("stage1_f32", "plane_fwd_kernel"): 77319680 + 32544768,
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


def run_reference(args, wl):
    """The CPU oracle, as it stands, on this machine's host cores (bounded sample of the workload)."""
    import numpy as np
    from oracle import wtconv_oracle as O
    from paper_2608_10805_b200 import inputs
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    Bs = min(wl.B, args.ref_batch)
    wls = wl.with_(B=Bs)
    I = inputs.make_inputs(wls)
    step = lambda: (O.forward(I["x"], I["w0"], I["s0"], None, I["wl"], I["sl"], wls.L),
                    O.backward(I["x"], I["g"], I["w0"], I["s0"], None, I["wl"], I["sl"], wls.L))
    for _ in range(args.warmup):
        step()
    t0 = time.time()
    for _ in range(args.steps):
        step()
    dt = time.time() - t0
    val = wls.N * args.steps / dt
    sample = "fwd+bwd of B=%d of %d images of %s (per-plane cost is batch-independent)" % (Bs, wl.B, wl.name)
    print(json.dumps({
        "impl": "reference", "metric": "wtconv_fwd_bwd_elements_per_s", "value": val, "unit": "elements/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "B": wl.B, "C": wl.C, "H": wl.H, "W": wl.W, "k": wl.k, "L": wl.L,
                   "sample_B": Bs},
        "cpu_baseline": {"value": val, "unit": "elements/s", "cores": O.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": val, "unit": "elements/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="stage1_f32")
    ap.add_argument("--ref-batch", type=int, default=16, help="images per oracle step in --impl reference")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tune", type=lambda s: int(s, 0), default=0, help="launch-plan override bits (see wtconv.h)")
    args = ap.parse_args()

    from paper_2608_10805_b200 import inputs, io_model
    wl = inputs.WORKLOADS[args.workload]
    if args.impl == "reference":
        args.steps = min(args.steps, 5)
        args.warmup = min(args.warmup, 1)
        return run_reference(args, wl)

    import numpy as np
    import torch
    import torch.distributed as dist
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

    tdt = wt.DTYPE_NAMES[wl.dtype]
    esz = 4 if wl.dtype == "f32" else 2
    desc = wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, tdt, args.tune)
    # seeded synthetic inputs (per-rank stream), two rotating input sets so no step re-reads a warm L2
    nbuf = 2
    sets = []
    for i in range(nbuf):
        I = inputs.make_inputs(wl.with_(seed=wl.seed + 100 * rank + 7 * i))
        sets.append(I)
    up = lambda a, dt=torch.float32: torch.from_numpy(a).to(dev).to(dt).contiguous()
    xs = [up(I["x"], tdt) for I in sets]
    gs = [up(I["g"], tdt) for I in sets]
    P = sets[0]
    w0, s0, wl_, sl = up(P["w0"]), up(P["s0"]), up(P["wl"]), up(P["sl"])
    out, gx = torch.empty_like(xs[0]), torch.empty_like(xs[0])
    gw0, gs0, gwl, gsl = torch.empty_like(w0), torch.empty_like(s0), torch.empty_like(wl_), torch.empty_like(sl)
    flat_grads = [gw0, gs0, gwl, gsl]
    ws = wt.alloc_workspace(desc, dev)
    stream = torch.cuda.current_stream()

    def step(i, ev=None):
        x, g = xs[i % nbuf], gs[i % nbuf]
        if ev:
            ev[0].record(stream)
        wt.wtconv_forward(desc, x, w0, s0, None, wl_, sl, out, ws, stream)
        if ev:
            ev[1].record(stream)
        wt.wtconv_backward(desc, x, g, w0, s0, None, wl_, sl, gx, gw0, gs0, None, gwl, gsl, ws, stream)
        if ev:
            ev[2].record(stream)
        if world > 1:
            for t in flat_grads:
                dist.all_reduce(t)

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(args.warmup, 3)):
        step(i)
    # keep the GPU busy for a moment so the sampled clocks are the clocks under load
    sync_all()
    sync_all()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    K = args.steps
    fev = [tuple(torch.cuda.Event(enable_timing=True) for _ in range(3)) for _ in range(K)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    t0 = time.time()
    e0.record(stream)
    for i in range(K):
        step(i, fev[i])
    e1.record(stream)
    sync_all()
    t1 = time.time()
    ms = torch.tensor([e0.elapsed_time(e1)], device=dev)
    if world > 1:
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    ms_total = float(ms.item())
    clocks = sampler.stop(t0, t1) if rank == 0 else None
    fwd_kernel_ms = sum(a.elapsed_time(b) for a, b, _ in fev) / len(fev)
    bwd_call_ms = sum(b.elapsed_time(c) for _, b, c in fev) / len(fev)

    # ---- end to end through the host entry point: pinned host buffers, copies inside the timed region
    hb = lambda t: torch.empty(t.shape, dtype=t.dtype).pin_memory()
    hx, hg = xs[0].cpu().pin_memory(), gs[0].cpu().pin_memory()
    hw0, hs0, hwl, hsl = (t.cpu().pin_memory() for t in (w0, s0, wl_, sl))
    hout, hgx, hgw0, hgs0, hgwl, hgsl = hb(out), hb(gx), hb(gw0), hb(gs0), hb(gwl), hb(gsl)
    hws = torch.empty(wt.wtconv_step_host_workspace_bytes(desc), dtype=torch.uint8, device=dev)

    def host_step():
        wt.wtconv_step_host(desc, hx, hg, hw0, hs0, None, hwl, hsl, hout, hgx, hgw0, hgs0, None, hgwl, hgsl, hws, stream)
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
    e2e_val = wl.N * world * args.e2e_steps / (float(hms.item()) * 1e-3)
    psz = sum(t.numel() * 4 for t in (w0, s0, wl_, sl))
    h2d = 2 * wl.N * esz + psz
    d2h = 2 * wl.N * esz + psz

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks, peak_kind = load_measured_peaks()
    ms_step = ms_total / K
    value = wl.N * world * K / (ms_total * 1e-3)
    fl_fwd = io_model.algorithmic_flops(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, "fwd")
    fl_bwd = io_model.algorithmic_flops(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, "bwd")
    fl_step = io_model.algorithmic_flops(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, "fwd+bwd")
    nf, nb = wt.wtconv_launch_count(desc)
    plane = wt.wtconv_plan_name(desc) == "plane"
    fused_bwd = plane and nb == 2
    # dominant kernel: the fused backward kernel (about two thirds of a step) where the plan has one, timed by the
    # events around wtconv_backward (which also cover its small epilogue launch and memset: a conservative rate);
    # otherwise the forward kernel, timed by the events around wtconv_forward
    if fused_bwd:
        dom_name, dom_ms, dom_fl = "plane_bwd_kernel (+ epilogue)", bwd_call_ms, fl_bwd
    else:
        dom_name, dom_ms, dom_fl = ("plane_fwd_kernel" if plane else "tiled forward launches"), fwd_kernel_ms, fl_fwd
    achieved = dom_fl / (dom_ms * 1e-3) / 1e12
    hbm_step = io_model.compulsory_bytes(wl.N, esz, "fwd+bwd")
    result = {
        "metric": "wtconv_fwd_bwd_elements_per_s", "value": value, "unit": "elements/s", "n_gpus": world,
        "steps": K, "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": wl.name, "B_per_gpu": wl.B, "C": wl.C, "H": wl.H, "W": wl.W, "k": wl.k, "L": wl.L,
                   "storage_dtype": wl.dtype, "plan": wt.wtconv_plan_name(desc),
                   "l2": "two rotating input sets; a step touches %d MB > 126 MB L2" % (4 * wl.N * esz // 2 ** 20),
                   "parallelism": "dp%d (batch-sharded, NCCL all-reduce of parameter gradients)" % world},
        "clocks": clocks,
        "e2e": {"value": e2e_val, "unit": "elements/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": args.e2e_steps},
        "gpu_launches": (nf + nb) * K,
        "roofline": {"bound": "alu", "kernel": dom_name,
                     "achieved": achieved, "peak": FP32_ALU_PEAK_TFLOPS, "unit": "TFLOP/s",
                     "frac": achieved / FP32_ALU_PEAK_TFLOPS, "traffic": NCU_DRAM_TRAFFIC.get((wl.name, dom_name.split()[0])),
                     "peak_source": "derived: 148 SMs x 128 FP32 lanes x 2 FLOP x 1.965 GHz (measured 74.1 with a packed-FMA loop)",
                     "launch_ms": dom_ms, "flops_per_launch": dom_fl,
                     "forward_kernel": {"launch_ms": fwd_kernel_ms, "achieved": fl_fwd / (fwd_kernel_ms * 1e-3) / 1e12,
                                        "frac": fl_fwd / (fwd_kernel_ms * 1e-3) / 1e12 / FP32_ALU_PEAK_TFLOPS,
                                        "traffic": NCU_DRAM_TRAFFIC.get((wl.name, "plane_fwd_kernel"))}},
        "step_rooflines": {
            "alu_frac": fl_step / (ms_step * 1e-3) / 1e12 / FP32_ALU_PEAK_TFLOPS,
            "hbm_compulsory_gbs": hbm_step / (ms_step * 1e-3) / 1e9,
            "hbm_frac_of_%s" % peak_kind: hbm_step / (ms_step * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "hbm_frac_of_8TBs": hbm_step / (ms_step * 1e-3) / 1e9 / 8000.0,
            "alu_floor_ms": fl_step / (FP32_ALU_PEAK_TFLOPS * 1e12) * 1e3,
            "hbm_floor_ms": hbm_step / (peaks["hbm_gbs"] * 1e9) * 1e3},
        "paper_io_model": {"q_fused_fwd_N": io_model.q_fused(wl.L), "q_ref_fwd_N": io_model.q_ref(wl.L),
                           "ours_fwd_N": 2.0, "ours_bwd_N": 3.0 if nb == 2 else 4.0},
    }
    if world == 1 and not args.no_cpu_baseline:
        from oracle import wtconv_oracle as O
        Bs = min(wl.B, 64)
        Ic = inputs.make_inputs(wl.with_(B=Bs))
        reps = 3
        c0 = time.time()
        for _ in range(reps):
            O.forward(Ic["x"], Ic["w0"], Ic["s0"], None, Ic["wl"], Ic["sl"], wl.L)
            O.backward(Ic["x"], Ic["g"], Ic["w0"], Ic["s0"], None, Ic["wl"], Ic["sl"], wl.L)
        cdt = (time.time() - c0) / reps
        result["cpu_baseline"] = {"value": wl.with_(B=Bs).N / cdt, "unit": "elements/s", "cores": O.num_threads(),
                                  "kind": "oracle", "seconds_per_step": cdt,
                                  "sample": "%d x fwd+bwd of B=%d images of %s, fp64 (%.0f core-seconds)"
                                            % (reps, Bs, wl.name, reps * cdt * O.num_threads())}
    print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
