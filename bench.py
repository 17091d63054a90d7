#!/usr/bin/env python
"""Throughput of one fdg_step (all modules: forward, loss, backward, update) on synthetic data.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 0..4] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` = samples/s with inputs resident in HBM, timed with nothing but
the step's own work on the device; `e2e` = the same through fdg_step_host with pinned host buffers
(host->device copies and the loss read-back inside the timed region); `roofline` describes the kernel
class with the largest share of device time, timed launch by launch in a separate pass with every module
on one stream (so that a launch's events bracket that kernel alone), and carries the whole step's
fraction of the tensor roofline under `step`; `cpu_baseline` is the CPU oracle timed on a bounded sample.  With N > 1 every rank runs an
independent replica (the method has no exchange between GPUs here) and the time is the maximum
over ranks.  `--impl reference` times the CPU oracle only.
"""
from __future__ import annotations

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

from paper_2509_05679_b200 import synth as sy  # noqa: E402

METRIC = "training samples/sec per B200 per fdg_step; % of bf16 tensor roofline"
UNIT = "samples/s"
FMA_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12      # 148 SMs x 128 fp32 FMA lanes x 2 flop x 1.965 GHz


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel classes of the default
# workload: ncu counters of a few launches of one kernel at a reduced per-worker batch, scaled to the full batch by
# the samples a launch processes (traffic of these kernels grows in proportion to the batch).  Valid only for the kernel
# source it was taken from: a changed source gives null.
NCU_SHA1 = "66b137a0c097fa99f51cdadd53689aab7acafe4a"   # sha1 of csrc/tc_gemm.cu when the counters were taken
NCU_TRAFFIC = {          # two steps' launches at per-worker batch 64 (M = 512, grids for 50 SMs), x 2: average per launch of the class
    "tc_gemm_fwd": {"bytes_per_launch": 92.4e6, "sha1": NCU_SHA1},       # km_kernel, 76 forward + input-gradient launches
    "tc_gemm_dgrad": {"bytes_per_launch": 92.4e6, "sha1": NCU_SHA1},
    "tc_gemm_wgrad": {"bytes_per_launch": 121.7e6, "sha1": NCU_SHA1},    # wg_kernel + wg2_kernel, 38 launches (partials stay in L2)
}


def _kernel_source_sha1():
    import hashlib
    h = hashlib.sha1()
    h.update(open(os.path.join(ROOT, "paper_2509_05679_b200", "csrc", "tc_gemm.cu"), "rb").read())
    return h.hexdigest()


def traffic_per_launch(kernel_class):
    rec = NCU_TRAFFIC.get(kernel_class)
    if not rec or rec.get("sha1") != _kernel_source_sha1():
        return None            # never captured, or the kernel has changed since the counters were taken
    return rec["bytes_per_launch"]


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm": p["hbm_gbs"], "tensor_burst": p["bf16_tflops"], "tensor": p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                "source": "measured"}
    return {"hbm": 6650.0, "tensor_burst": 1590.0, "tensor": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device: int):
        self.device, self.rows, self.proc = device, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                                          "-i", str(self.device)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm = [float(r[1]) for r in self.rows if len(r) >= 9 and r[1].replace(".", "").isdigit()]
        mx = [float(r[2]) for r in self.rows if len(r) >= 9 and r[2].replace(".", "").isdigit()]
        reasons = set()
        for r in self.rows:
            if len(r) >= 9:
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of floats over all ranks (the job is as slow as its slowest replica)."""
    if dist is None:
        return [float(v) for v in values]
    import torch
    t = torch.tensor([float(v) for v in values], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_throughput(samples_per_rank_step: int, steps: int, world: int, seconds: float) -> float:
    """samples/s of the whole job: every rank is an independent replica processing its own batches."""
    return samples_per_rank_step * steps * world / seconds


def oracle_sample(net: sy.Net, timed_steps: int, warm_steps: int):
    """The CPU oracle, as it stands, on a bounded sample of the workload: same network, same K, same
    number of workers, ONE sample per worker; the pipeline is filled first, then `timed_steps`
    steady-state steps are timed.  Returns (samples/s, cores, description)."""
    from oracle import oracle as orc
    small = sy.Net(net.name, net.layers, net.splits, net.in_h, net.in_w, net.in_c, net.classes, net.n_workers, 1, net.lr, net.dtype)
    o = orc.Oracle(small.layers, small.splits, small.n_workers, 1, (net.in_h, net.in_w, net.in_c), net.classes)
    o.storage_bf16(net.dtype == "bf16")
    o.set_params(sy.init_params(small.layers, 0, bf16=net.dtype == "bf16"))
    fill = 2 * small.K - 2
    for t in range(fill + warm_steps):
        o.step(sy.batch_inputs(small, t), sy.batch_labels(small, t), small.lr)
    t0 = time.perf_counter()
    for t in range(fill + warm_steps, fill + warm_steps + timed_steps):
        o.step(sy.batch_inputs(small, t), sy.batch_labels(small, t), small.lr)
    dt = (time.perf_counter() - t0) / timed_steps
    desc = (f"same network and K={small.K}, {small.n_workers} workers x 1 sample (M={small.M}) instead of x{net.batch}; "
            f"{timed_steps} steady-state step(s) after {fill + warm_steps} fill/warm-up steps; fp64, std::thread over samples")
    return small.M / dt, orc.threads(), desc, dt


def run_reference(args, net):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    timed, warm = max(1, min(args.steps, 3)), min(args.warmup, 1)      # bounded: a step of the oracle takes seconds
    v, cores, desc, dt = oracle_sample(net, timed, warm)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": timed, "warmup": warm,
        "steps_requested": args.steps, "warmup_requested": args.warmup,
        "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": net.name, "K": net.K, "n_workers": net.n_workers, "per_worker_batch": net.batch, "note": desc},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=3, help="0..4 = the five configurations; 3 = ResNet-18-shaped K=4, 8 workers x 128; 5 / 6 = the paper's ResNet-20 experiment shape with K = 1 / K = 2")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--worker-groups", type=int, default=0, help="0: chosen by the library; n: every module but the last runs its layers once per n-th of the workers")
    ap.add_argument("--kernel-path", type=int, default=0, help="0: tensor-core kernels where shapes allow (CTA pairs for the 256-column tile), 1: plain FMA kernels only, 2: tensor-core kernels without CTA pairs")
    ap.add_argument("--batch", type=int, default=None, help="per-worker batch override (testing only; changes the workload name)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-kernel-pass", action="store_true", help="skip the extra one-stream pass that times every kernel class (roofline becomes null)")
    ap.add_argument("--grid-sms", type=int, default=0, help="SMs the persistent kernels size their grids for (0: the library's choice, a third of the device with concurrent module streams)")
    ap.add_argument("--kernel-pass-grid-sms", type=int, default=0, help="grid size of the one-stream kernel pass (0: all SMs, a kernel alone; diagnosis: the timed steps' grid_sms shows what each kernel does on its share)")
    ap.add_argument("--serial", action="store_true", help="diagnosis: all modules on one stream (uncontended per-kernel times)")
    args = ap.parse_args()

    net = sy.config(args.config, batch=args.batch)
    if args.impl == "reference":
        return run_reference(args, net)

    import torch
    from paper_2509_05679_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    warmup = max(args.warmup, 3)
    fill = 2 * net.K - 2                      # iterations until every module has a backward batch
    timing_stream = torch.cuda.Stream()       # carries only the two timing events; the library runs on its own streams
    ctx = binding.Context(net.layers, net.splits, net.n_workers, net.batch, net.lr, dtype=net.dtype,
                          in_shape=(net.in_h, net.in_w, net.in_c), num_classes=net.classes, device=local,
                          kernel_path=args.kernel_path, serial=args.serial, worker_groups=args.worker_groups, grid_sms=args.grid_sms)
    ctx.set_params(sy.init_params(net.layers, 0, bf16=net.dtype == "bf16"))
    grid_sms = ctx.grid_sms

    # a pool of distinct batches, resident in HBM (device arm) and in pinned host memory (e2e arm)
    pool = 4
    tdt = torch.bfloat16 if net.dtype == "bf16" else torch.float32
    host_x = [torch.from_numpy(sy.batch_inputs(net, t, stream=rank)).to(tdt).pin_memory() for t in range(pool)]
    host_y = [torch.from_numpy(sy.batch_labels(net, t, stream=rank)).pin_memory() for t in range(pool)]
    dev_x = [x.cuda() for x in host_x]
    dev_y = [y.cuda() for y in host_y]
    torch.cuda.synchronize()

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        torch.cuda.synchronize()

    def join_event():
        """An event that fires when all module streams are done (fdg_join makes the timing stream wait for them)."""
        ctx.join(timing_stream.cuda_stream)
        e = torch.cuda.Event(enable_timing=True)
        e.record(timing_stream)
        return e

    step_no = 0

    def dev_steps(n):
        nonlocal step_no
        for _ in range(n):
            ctx.step(dev_x[step_no % pool], dev_y[step_no % pool])
            step_no += 1

    # ---- device-resident arm (no per-launch instrumentation: only the step's own work is on the device)
    dev_steps(fill + warmup)
    barrier()
    _, launches0 = ctx.stats()
    sampler = ClockSampler(local)
    sampler.start()
    start = torch.cuda.Event(enable_timing=True)
    start.record(timing_stream)              # the device is idle here: this is the start of the timed region
    dev_steps(args.steps)
    end = join_event()
    barrier()
    ms = start.elapsed_time(end)
    clocks = sampler.stop()
    dev_bytes, launches1 = ctx.stats()
    mod_ms = [float(v) for v in ctx.module_times()]

    # ---- end-to-end arm: host buffers in, loss out, every step
    for _ in range(2):
        ctx.step_host(host_x[step_no % pool], host_y[step_no % pool], want_loss=True); step_no += 1
    barrier()
    t0 = time.perf_counter()
    loss = float("nan")
    for _ in range(args.steps):
        loss = ctx.step_host(host_x[step_no % pool], host_y[step_no % pool], want_loss=True); step_no += 1
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0

    # ---- kernel passes: the same workload with every module on ONE stream and CUDA events around every launch, so that
    # an event pair brackets one kernel running alone (with the module streams running side by side a pair would also
    # contain whatever the other modules had on the GPU).  First with the grids of the timed steps (`grid_sms` SMs per
    # persistent kernel: the launch configuration that was timed, and the one an ncu launch list of this command shows),
    # then with grids for the whole device (what the same kernels do when nothing is meant to run beside them).
    # Not part of `value`.
    kernel_steps = 3
    device_sms = torch.cuda.get_device_properties(local).multi_processor_count

    def kernel_pass(sms):
        c = binding.Context(net.layers, net.splits, net.n_workers, net.batch, net.lr, dtype=net.dtype,
                            in_shape=(net.in_h, net.in_w, net.in_c), num_classes=net.classes, device=local,
                            kernel_path=args.kernel_path, serial=True, worker_groups=args.worker_groups, grid_sms=sms)
        c.set_params(sy.init_params(net.layers, 0, bf16=net.dtype == "bf16"))
        for i in range(fill + 3):
            c.step(dev_x[i % pool], dev_y[i % pool])
        torch.cuda.synchronize()
        c.profile(True)
        for i in range(kernel_steps):
            c.step(dev_x[i % pool], dev_y[i % pool])
        c.profile(False)
        kall = c.profile_read()
        sms = c.grid_sms
        c.close()
        return {k: v for k, v in kall.items() if "[" not in k}, {k: v for k, v in kall.items() if "[" in k}, sms

    kstats, kshapes, kernel_grid_sms, kstats_all = None, None, None, None
    if not args.no_kernel_pass:
        ctx.close()
        ctx = None
        kstats, kshapes, kernel_grid_sms = kernel_pass(args.kernel_pass_grid_sms or grid_sms)
        if kernel_grid_sms != device_sms:
            kstats_all, _, _ = kernel_pass(device_sms)

    ms, e2e_s = max_over_ranks([ms, e2e_s], dist, "cuda")

    if rank == 0:
        pk = peaks()
        total_samples = net.M * args.steps * world
        value = whole_job_throughput(net.M, args.steps, world, ms * 1e-3)
        flops_step = sy.flops_per_sample(net) * net.M
        ms_step = ms / args.steps
        # which measured peak: the sustained figure for a whole step under load; for a kernel timed alone the burst figure
        step_tflops = flops_step / (ms_step * 1e-3) / 1e12
        step_entry = {"flop_per_step": flops_step, "ms_per_step": ms_step, "achieved": step_tflops, "unit": "TFLOP/s",
                      "peak": pk["tensor_burst"], "frac": step_tflops / pk["tensor_burst"],
                      "peak_sustained": pk["tensor"], "frac_of_sustained": step_tflops / pk["tensor"],
                      "peak_source": pk["source"] + ": bf16 GEMM, burst (frac) and sustained (frac_of_sustained)"}

        def roofline_of(stats):
            """Roofline entry of the kernel class with the largest summed time in the one-stream kernel pass."""
            if not stats:
                return None
            name, st = max(stats.items(), key=lambda kv: kv[1]["ms"])
            total_ms = sum(v["ms"] for v in stats.values())
            per_step = st["launches"] / kernel_steps
            base = {"kernel": name, "grid_sms": kernel_grid_sms, "device_sms": device_sms,
                    "launches_per_step": per_step, "avg_launch_ms": st["ms"] / st["launches"],
                    "class_ms_per_step": st["ms"] / kernel_steps, "share_of_kernel_time": st["ms"] / total_ms,
                    "kernel_ms_per_step_all_classes": total_ms / kernel_steps, "traffic": traffic_per_launch(name),
                    "timing": f"CUDA events around every launch, separate pass of {kernel_steps} steps with all modules on one stream "
                              "(each event pair brackets one kernel running alone); not part of the timed region of `value`"}
            if name.startswith("tc_gemm") or name.startswith("igemm_fma"):
                tensor = name.startswith("tc_gemm")
                ach = st["flops"] / (st["ms"] * 1e-3) / 1e12
                peak = pk["tensor_burst"] if tensor else FMA_PEAK_TFLOPS
                base.update({"bound": "tensor" if tensor else "alu", "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": ach / peak,
                             # the launch is sized for grid_sms of the device's SMs (others run kernels of other modules
                             # meanwhile): its fraction of what those SMs can do
                             "frac_of_sm_share": ach / (peak * kernel_grid_sms / device_sms),
                             "peak_source": (pk["source"] + ", burst bf16 GEMM (a kernel timed alone)") if tensor
                             else "derived: 148 SMs x 128 FMA x 2 x 1.965 GHz"})
            else:
                ach = st["bytes"] / (st["ms"] * 1e-3) / 1e9
                base.update({"bound": "hbm", "achieved": ach, "peak": pk["hbm"], "unit": "GB/s", "frac": ach / pk["hbm"], "peak_source": pk["source"]})
            return base

        roof = roofline_of(kstats)
        if roof:
            if kstats_all and roof["kernel"] in kstats_all:
                # the same kernel class with every grid sized for the whole device, each launch alone
                sa = kstats_all[roof["kernel"]]
                work, peak = (sa["bytes"] / 1e9, roof["peak"]) if roof["bound"] == "hbm" else (sa["flops"] / 1e12, roof["peak"])
                ach = work / (sa["ms"] * 1e-3)
                roof["all_sms"] = {"grid_sms": device_sms, "avg_launch_ms": sa["ms"] / sa["launches"], "class_ms_per_step": sa["ms"] / kernel_steps,
                                   "achieved": ach, "frac": ach / peak,
                                   "kernel_ms_per_step_all_classes": sum(v["ms"] for v in kstats_all.values()) / kernel_steps}
            roof["step"] = step_entry
        else:
            roof = {"kernel": None, "step": step_entry}
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if net.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": net.name + ("" if args.batch is None else f"-B{args.batch}"), "K": net.K, "n_workers": net.n_workers,
                       "per_worker_batch": net.batch, "M": net.M, "lr": net.lr, "pipeline_fill_steps": fill,
                       "l2": "inputs rotate over 4 batches; each step streams the multi-GB activation stash, far larger than L2",
                       "multi_gpu": "independent replicas (no exchange between GPUs)", "kernel_path": args.kernel_path, "serial": bool(args.serial), "worker_groups": args.worker_groups,
                       "grid_sms": grid_sms, "kernel_pass_grid_sms": kernel_grid_sms},
            "clocks": clocks,
            "roofline": roof,
            "kernels": {k: {"launches_per_step": v["launches"] / kernel_steps, "ms_per_step": round(v["ms"] / kernel_steps, 4),
                            "tflops": round(v["flops"] / (v["ms"] * 1e-3) / 1e12, 2) if v["ms"] > 0 else None,
                            "gbs": round(v["bytes"] / (v["ms"] * 1e-3) / 1e9, 1) if v["ms"] > 0 else None}
                        for k, v in sorted((kstats or {}).items(), key=lambda kv: -kv[1]["ms"])},
            "kernels_all_sms": {k: {"ms_per_step": round(v["ms"] / kernel_steps, 4),
                                    "tflops": round(v["flops"] / (v["ms"] * 1e-3) / 1e12, 2) if v["ms"] > 0 else None,
                                    "gbs": round(v["bytes"] / (v["ms"] * 1e-3) / 1e9, 1) if v["ms"] > 0 else None}
                                for k, v in sorted((kstats_all or {}).items(), key=lambda kv: -kv[1]["ms"])},
            "kernel_shapes": {k: {"launches_per_step": v["launches"] / kernel_steps, "ms_per_step": round(v["ms"] / kernel_steps, 4),
                                  "tflops": round(v["flops"] / (v["ms"] * 1e-3) / 1e12, 1) if v["ms"] > 0 else None,
                                  "gbs": round(v["bytes"] / (v["ms"] * 1e-3) / 1e9, 1) if v["ms"] > 0 else None}
                              for k, v in sorted((kshapes or {}).items(), key=lambda kv: -kv[1]["ms"])},
            "module_ms_last_step": mod_ms, "device_bytes": int(dev_bytes),
            "gpu_launches": int(launches1 - launches0),
            "e2e": {"value": total_samples / e2e_s, "unit": UNIT,
                    "h2d_bytes_per_step": int(host_x[0].numel() * host_x[0].element_size() + host_y[0].numel() * 4),
                    "d2h_bytes_per_step": 4, "last_loss": loss},
        }
        if world == 1 and not args.no_cpu_baseline:
            v, cores, desc, _ = oracle_sample(net, 3, 0)
            out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}
        print(json.dumps(out))
    if ctx is not None:
        ctx.close()
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
