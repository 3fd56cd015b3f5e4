#!/usr/bin/env python
"""Benchmark: RevNet train-step images/sec on B200 (one replica per GPU, no collectives).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config revnet104] [--impl ours|reference]

A step is one whole train step of the stack (forward, reconstructing backward through every
stage, SGD update) on one synthetic batch.  The headline workload is the largest configuration
that fits one GPU (the large-image bottleneck network, batch 64 of 224x224); the three CIFAR-sized
configurations are timed in the same run and reported under "other_workloads".
Prints ONE JSON line (rank 0).
"""
import argparse
import json
import os
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "revnet_train_step_images_per_sec"
UNIT = "images/s"


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=d["hbm_gbs"], tc_burst=d["bf16_tflops"], tc_sustained=d["bf16_tflops_sustained"], source="measured")
    return dict(hbm=6650.0, tc_burst=1590.0, tc_sustained=1400.0, source="fallback")


# fp32 FMA peak of the CUDA cores: 148 SMs x 128 lanes x 2 flop x 1.965 GHz (max SM clock)
ALU_FP32_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12

ALU_KERNELS = ("gemm_simt_kernel",)   # fp32 CUDA-core GEMMs

# profile record name (one per call site class) -> the CUDA kernel that runs it, and the source files it is built from
DEVICE_KERNEL = {
    "conv_fprop_fused": "conv_fused_kernel", "conv_dgrad_fused": "conv_fused_kernel",
    "conv_fprop_tc": "conv_tc_kernel", "conv_dgrad_tc": "conv_tc_kernel", "conv_wgrad_tc": "wgrad_tc_kernel",
    "conv_fprop_tc2": "conv_tc2_kernel", "conv_dgrad_tc2": "conv_tc2_kernel", "conv_wgrad_tc2": "wgrad_tc2_kernel",
    "conv_fprop_simt": "gemm_simt_kernel", "conv_dgrad_simt": "gemm_simt_kernel", "conv_wgrad_simt": "gemm_simt_kernel",
    "bn_stats_partial": "col_reduce_kernel", "bn_bwd_partial": "col_reduce_kernel",
}
KERNEL_SOURCES = {
    "conv_fused_kernel": ("conv_fused.cu", "conv_epilogue.cuh", "tc_ptx.cuh"),
    "conv_tc_kernel": ("conv_tc.cu", "conv_epilogue.cuh", "tc_ptx.cuh"),
    "wgrad_tc_kernel": ("conv_tc.cu", "tc_ptx.cuh"),
    "conv_tc2_kernel": ("conv_tc.cu", "conv_epilogue.cuh", "tc_ptx.cuh"),
    "wgrad_tc2_kernel": ("conv_tc.cu", "tc_ptx.cuh"),
}


def by_device_kernel(prof, peaks=None):
    """Per-launch-shape profile records ("name|bytes|flops" per launch) -> per device kernel.  With peaks, a
    convolution kernel is split by what binds each of its launch shapes: the same kernel runs the memory-bound 1x1
    layers (a few flops per byte) and the tensor-bound 3x3 layers and transitions, and one roofline cannot
    describe both.  The two halves are reported as "kernel [tensor-bound layers]" and "kernel [hbm-bound layers]"."""
    out = {}
    for key, v in prof.items():
        name = key.split("|")[0]
        k = DEVICE_KERNEL.get(name, name)
        if peaks and k in KERNEL_SOURCES and v["launches"]:
            t_mem = v["bytes"] / (peaks["hbm"] * 1e9)
            t_tc = v["flops"] / (peaks["tc_sustained"] * 1e12)
            k = f"{k} [{'tensor' if t_tc > t_mem else 'hbm'}-bound layers]"
        a = out.setdefault(k, dict(launches=0, ms=0.0, bytes=0.0, flops=0.0))
        for f in a:
            a[f] += v[f]
    return out


def source_digest(kernel):
    import hashlib
    h = hashlib.sha256()
    for f in KERNEL_SOURCES.get(kernel, ()):
        with open(os.path.join(ROOT, "paper_1707_04585_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def measured_traffic(kernel, workload):
    """DRAM bytes per launch of `kernel` on `workload` from the ncu capture summarised under profiles/,
    or None if there is none or the kernel's sources have changed since it was taken."""
    p = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(p):
        return None
    rec = json.load(open(p)).get(workload, {}).get(kernel)
    if not rec or rec.get("source_digest") != source_digest(kernel):
        return None
    return rec["dram_bytes_per_launch"]


def binding_roofline(name, rec, peaks):
    """Which roofline bounds a kernel class on this workload: the one that needs more time for the
    kernel's algorithmic bytes and flops (summed over its launches).  Convolutions of narrow layers
    are bound by memory, wide ones by the tensor cores."""
    if name in ALU_KERNELS:
        return "alu"
    t_mem = rec["bytes"] / (peaks["hbm"] * 1e9)
    t_tc = rec["flops"] / (peaks["tc_sustained"] * 1e12)
    return "tensor" if t_tc > t_mem else "hbm"


class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.idx, self.proc = gpu_index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                                          "-i", str(self.idx)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if not self.proc:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def cpu_baseline(cfg, sample_n, steps=1):
    """The oracle, as it stands, on a bounded sample of the workload (reduced batch)."""
    from oracle import revnet as orc
    from paper_1707_04585_b200 import synthetic as syn
    from tests import helpers as hp
    sc = syn.shrink(cfg, N=sample_n)
    inp = syn.make_stack_inputs(sc)
    net = hp.oracle_net(sc, inp["params"])
    vel = {k: np.zeros_like(v, dtype=np.float64) for k, v in inp["params"].items()}
    times = []
    for _ in range(steps):
        t0 = time.perf_counter()
        r = orc.stack_train_grads(net, inp["images"], inp["labels"], "reconstruct")
        orc.sgd_step(inp["params"], r["grads"], vel, sc.lr, sc.momentum, sc.weight_decay, hp.decayed_names(sc))
        times.append(time.perf_counter() - t0)
    try:
        cores = len(os.sched_getaffinity(0))
    except Exception:
        cores = os.cpu_count()
    omp = os.environ.get("OMP_NUM_THREADS")
    if omp:
        cores = min(cores, int(omp))
    return dict(value=sample_n / float(np.mean(times)), unit=UNIT, cores=cores, kind="oracle",
                sample=f"{steps} train step(s) (forward + reconstructing backward + SGD) on batch {sample_n} of {cfg.N}, fp64",
                seconds_per_step=float(np.mean(times)))


def ref_batch(args, cfg):
    """Batch of the bounded oracle sample: about 10-30 s of CPU work per step."""
    if args.ref_batch:
        return max(2, min(cfg.N, args.ref_batch))
    return 2 if cfg.img > 64 else min(cfg.N, 32)


def time_steps(run, steps, warmup, flush, stream):
    """Device time (ms, summed) of `steps` train steps from the initial weights, L2 flushed in between."""
    import torch
    p0 = run.params.clone()
    for _ in range(warmup):
        run.params.copy_(p0); run.momentum.zero_()
        st = run.step(want_logits=False)
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in ev:
        run.params.copy_(p0); run.momentum.zero_()
        flush.zero_()
        a.record(stream)
        st = run.step(want_logits=False)
        b.record(stream)
    torch.cuda.synchronize()
    return sum(a.elapsed_time(b) for a, b in ev), st


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sample = ref_batch(args, cfg)
    t0 = time.perf_counter()
    cb = cpu_baseline(cfg, sample, steps=1)            # untimed warm-up of caches is not separated: the oracle is timed as it stands
    k = max(1, min(args.steps, int(60.0 / max(cb["seconds_per_step"], 1e-3))))
    cb = cpu_baseline(cfg, sample, steps=k)
    line = dict(metric=METRIC, value=cb["value"], unit=UNIT, n_gpus=args.gpus, steps=k, warmup=1,
                ms_per_step=cb["seconds_per_step"] * 1e3, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic", impl="reference",
                config=dict(workload=cfg.name, global_batch=cfg.N, sample_batch=sample),
                cpu_baseline=dict(value=cb["value"], unit=UNIT, cores=cb["cores"], kind="oracle", sample=cb["sample"]),
                e2e=dict(value=cb["value"], unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                wall_s=time.perf_counter() - t0)
    print(json.dumps(line), flush=True)


def depth_sweep(ctx, cfg):
    """Stored activation MB of the same network with 1..36 units per stage (plans only, nothing runs):
    Section 3.2, storage independent of depth."""
    from paper_1707_04585_b200 import binding as B, synthetic as syn
    out = {}
    for units in (1, 3, 9, 18, 36):
        c = syn.shrink(cfg, units=units)
        plan = B.revnet_stack_plan(ctx, B.stack_desc(c, 0, False, 16, False))
        out[str(units)] = round(plan.activation_bytes / 1e6, 3)
        plan.close()
    return out


def max_over_ranks(values, world, device):
    """Element-wise maximum of `values` (floats) over the ranks of the default process group: a job is as slow
    as its slowest replica.  With one rank the values come back unchanged."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def replica_seed(seed, rank):
    """Every rank trains its own replica on its own synthetic batch."""
    return seed + 1000 * rank


def whole_job_rate(units_per_rank_step, world, steps, total_ms):
    """Units all ranks processed in `steps` steps divided by the (max over ranks) time they took."""
    return units_per_rank_step * world * steps / (total_ms * 1e-3)


def run_ours(args, cfg):
    import torch
    import torch.distributed as dist
    from paper_1707_04585_b200 import binding as B, runner as R, synthetic as syn

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    ctx = B.Context(local)
    # every rank trains its own replica on its own batch (weak scaling, no exchange step)
    import dataclasses
    rcfg = dataclasses.replace(cfg, seed=replica_seed(cfg.seed, rank))
    inp = syn.make_stack_inputs(rcfg)
    run = R.StackRunner(ctx, rcfg, mode=0)
    run.load(inp["images"], inp["labels"], inp["params"])
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")     # > 126 MB of L2
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    params0 = run.params.clone()

    def reset():
        # every timed step starts from the initial weights and zero momentum: repeated SGD steps at the
        # paper's learning rate on random labels would drive the activations out of range
        run.params.copy_(params0)
        run.momentum.zero_()

    # the clock sampler runs from the warm-up to the end of the end-to-end loop: nvidia-smi needs about a second
    # to deliver its first line, longer than the timed steps of the small workloads take
    sampler = ClockSampler(local)
    t_sampling = time.perf_counter()
    if rank == 0:
        sampler.start()
    for _ in range(args.warmup):
        reset()
        st = run.step(want_logits=False)
    barrier()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for a, b in ev:
        reset()
        flush.zero_()                      # evict L2 between timed iterations (outside the timed span)
        a.record(stream)
        st = run.step(want_logits=False)
        b.record(stream)
    barrier()
    dev_ms = sum(a.elapsed_time(b) for a, b in ev)
    launches = int(st.kernel_launches) * args.steps

    # ---- end to end through the host-buffer entry point: pinned H2D of the batch, D2H of loss + predictions
    h_img = torch.from_numpy(B.to_nhwc(inp["images"])).pin_memory()
    h_lab = torch.from_numpy(inp["labels"]).pin_memory()
    h_loss = torch.zeros(1, dtype=torch.float32).pin_memory()
    h_pred = torch.zeros(rcfg.N, dtype=torch.int32).pin_memory()
    for _ in range(2):
        B.revnet_train_step_host(ctx, run.plan, h_img, h_lab, run.images, run.labels, run.params, run.grads, run.momentum,
                                 run.act, run.ws, run.loss, run.pred, h_loss, h_pred)
    barrier()
    e2e_ms = 0.0
    for _ in range(args.steps):
        reset()
        flush.zero_()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        B.revnet_train_step_host(ctx, run.plan, h_img, h_lab, run.images, run.labels, run.params, run.grads, run.momentum,
                                 run.act, run.ws, run.loss, run.pred, h_loss, h_pred)   # returns after its own stream sync
        e2e_ms += (time.perf_counter() - t0) * 1e3
    barrier()
    # a short workload is over before nvidia-smi has delivered ten lines: the same step goes on running, untimed, until
    # the sampler has had 2.5 s of it (clock record = warm-up, timed steps, end-to-end steps and these)
    extra_steps = 0
    while time.perf_counter() - t_sampling < 2.5:
        reset()
        run.step(want_logits=False)
        extra_steps += 1
        if extra_steps % 8 == 0:
            torch.cuda.synchronize()
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    if clocks is not None:
        clocks["untimed_steps_while_sampling"] = extra_steps

    # ---- the same network trained with ordinary backprop on stored activations (Section 3.2: the cost the
    # reversible step trades storage for), graph replay, same timing rules; rank 0 only
    stored = None
    if rank == 0 and not args.no_stored:
        srun = R.StackRunner(ctx, rcfg, mode=0, store_activations=True)
        srun.load(inp["images"], inp["labels"], inp["params"])
        sp0 = srun.params.clone()
        for _ in range(args.warmup):
            srun.params.copy_(sp0); srun.momentum.zero_()
            sst = srun.step(want_logits=False)
        torch.cuda.synchronize()
        n_s = max(3, args.steps // 2)
        sev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_s)]
        for a, b in sev:
            srun.params.copy_(sp0); srun.momentum.zero_()
            flush.zero_()
            a.record(stream)
            sst = srun.step(want_logits=False)
            b.record(stream)
        torch.cuda.synchronize()
        s_ms = sum(a.elapsed_time(b) for a, b in sev) / n_s
        stored = dict(ms_per_step=s_ms, images_per_sec=rcfg.N / (s_ms * 1e-3), stored_activation_bytes=int(sst.stored_activation_bytes),
                      workspace_bytes=int(sst.workspace_peak_bytes), flops_per_step=int(sst.flops_fwd + sst.flops_bwd), steps=n_s)
        del srun
        torch.cuda.empty_cache()

    # ---- per-kernel timing with CUDA events on the launching stream (same process, after the timed steps)
    B.revnet_profile_enable(ctx, 2)          # one record per kernel and launch shape
    psteps = 2
    for _ in range(psteps):
        reset()
        run.step(want_logits=False)
    prof = B.revnet_profile_summary(ctx)
    B.revnet_profile_enable(ctx, False)
    # ---- the same step as it runs inside the replayed graph: start / end stamps written by the kernels themselves
    B.revnet_profile_enable(ctx, 3)
    for _ in range(3):                       # the first of them captures the stamped graph, the others replay it
        reset()
        run.step(want_logits=False)
    torch.cuda.synchronize()
    timeline = B.revnet_profile_summary(ctx)
    B.revnet_profile_enable(ctx, False)
    final_loss = float(run.loss.item())
    # per-block forward / reconstructing-backward time at each stage shape of the workload
    block_ms = {}
    if rank == 0:
        for s_cfg, H in zip(rcfg.stages, syn.stage_resolutions(rcfg)):
            bc = syn.BlockCfg(rcfg.N, H, H, s_cfg.c, s_cfg.w, s_cfg.kind, seed=9)
            block_ms[f"{s_cfg.kind}_c{s_cfg.c}_{H}x{H}"] = R.time_block(ctx, bc, 0, reps=5, warmup=3)

    # ---- the other configurations, same timing rules, fewer steps (rank 0, single-GPU runs only)
    others = {}
    if rank == 0 and world == 1 and not args.no_others:
        del run
        torch.cuda.empty_cache()
        for oname in syn.STACK_NAMES:
            if oname == cfg.name:
                continue
            ocfg = syn.stack_config(oname)
            oin = syn.make_stack_inputs(ocfg)
            orun = R.StackRunner(ctx, ocfg, mode=0)
            orun.load(oin["images"], oin["labels"], oin["params"])
            n_o = max(5, min(args.steps, 30))
            oms, ost = time_steps(orun, n_o, args.warmup, flush, stream)
            others[oname] = dict(ms_per_step=oms / n_o, images_per_sec=ocfg.N * n_o / (oms * 1e-3), steps=n_o, batch=ocfg.N,
                                 activation_bytes=int(ost.stored_activation_bytes), flops_per_step=int(ost.flops_fwd + ost.flops_bwd),
                                 gpu_launches_per_step=int(ost.kernel_launches))
            del orun
            torch.cuda.empty_cache()

    dev_ms, e2e_ms = max_over_ranks([dev_ms, e2e_ms], world, "cuda")
    if rank == 0:
        peaks = load_peaks()
        total_images = rcfg.N * world * args.steps
        assert abs(whole_job_rate(rcfg.N, world, args.steps, dev_ms) - total_images / (dev_ms * 1e-3)) < 1e-6 * total_images
        shapes = {k: v for k, v in prof.items() if not k.startswith("step_begin")}    # not a kernel: the host-ahead hold of a profiled step
        classes = {k: v for k, v in by_device_kernel(shapes, peaks).items() if " [" in k}
        prof = by_device_kernel(shapes)
        tot = sum(v["ms"] for v in prof.values()) or 1.0
        top = max(prof.items(), key=lambda kv: kv[1]["ms"])
        name, rec = top
        bound = binding_roofline(name, rec, peaks)
        avg_s = rec["ms"] / rec["launches"] * 1e-3
        if bound == "hbm":
            ach, peak, runit = rec["bytes"] / rec["launches"] / avg_s / 1e9, peaks["hbm"], "GB/s"
        elif bound == "tensor":
            ach, peak, runit = rec["flops"] / rec["launches"] / avg_s / 1e12, peaks["tc_sustained"], "TFLOP/s"
        else:
            ach, peak, runit = rec["flops"] / rec["launches"] / avg_s / 1e12, ALU_FP32_TFLOPS, "TFLOP/s"
        # the step as a whole against both rooflines: algorithmic bytes and flops of all its kernels over the
        # graph-replayed step time (the per-kernel spans above come from a step enqueued kernel by kernel on ONE
        # stream, events in between: they add up to more than the replayed step, which overlaps weight gradients
        # and the recomputation of F with the main chain and has no events between launches)
        step_s = dev_ms / args.steps * 1e-3
        step_bytes = sum(v["bytes"] for v in prof.values()) / psteps
        step_flops = sum(v["flops"] for v in prof.values()) / psteps
        whole = dict(algorithmic_gb=step_bytes / 1e9, tflop=step_flops / 1e12,
                     gbs=step_bytes / step_s / 1e9, frac_hbm=step_bytes / step_s / 1e9 / peaks["hbm"],
                     tflops=step_flops / step_s / 1e12, frac_tensor=step_flops / step_s / 1e12 / peaks["tc_sustained"],
                     roofline_ms=sum(max(v["bytes"] / (peaks["hbm"] * 1e9), v["flops"] / (peaks["tc_sustained"] * 1e12)) for v in shapes.values()) / psteps * 1e3,
                     profiled_serial_ms=tot / psteps)
        if timeline.get("stamped_span"):
            tl = by_device_kernel({k: v for k, v in timeline.items() if not k.startswith("stamped_")}, peaks)
            whole["graph_timeline"] = dict(
                note="one replayed step; start of first CTA to end of last CTA per launch, summed per kernel (overlapping kernels each count)",
                span_ms=timeline["stamped_span"]["ms"], busy_ms=timeline["stamped_busy"]["ms"],
                stamped_launches=timeline["stamped_busy"]["launches"],
                kernels={k: dict(launches=v["launches"], ms=v["ms"],
                                 gbs=(v["bytes"] / (v["ms"] * 1e-3) / 1e9) if v["ms"] > 0 else None,
                                 tflops=(v["flops"] / (v["ms"] * 1e-3) / 1e12) if v["ms"] > 0 else None)
                         for k, v in sorted(tl.items(), key=lambda kv: -kv[1]["ms"])})
        roof = dict(bound=bound, achieved=ach, peak=peak, unit=runit, frac=ach / peak, traffic=measured_traffic(name, cfg.name), kernel=name, whole_step=whole,
                    kernel_share=rec["ms"] / tot, avg_launch_us=avg_s * 1e6, peak_source=peaks["source"],
                    kernels={k: dict(launches=v["launches"] // psteps, ms_per_step=v["ms"] / psteps, share=v["ms"] / tot,
                                     gbs=(v["bytes"] / (v["ms"] * 1e-3) / 1e9) if v["ms"] > 0 else None,
                                     tflops=(v["flops"] / (v["ms"] * 1e-3) / 1e12) if v["ms"] > 0 else None)
                             for k, v in sorted(prof.items(), key=lambda kv: -kv[1]["ms"])},
                    # the convolution kernels once more, their launches split by what binds each launch shape
                    layer_classes={k: dict(launches=v["launches"] // psteps, ms_per_step=v["ms"] / psteps,
                                           gbs=v["bytes"] / (v["ms"] * 1e-3) / 1e9, frac_hbm=v["bytes"] / (v["ms"] * 1e-3) / 1e9 / peaks["hbm"],
                                           tflops=v["flops"] / (v["ms"] * 1e-3) / 1e12, frac_tensor=v["flops"] / (v["ms"] * 1e-3) / 1e12 / peaks["tc_sustained"])
                                   for k, v in sorted(classes.items(), key=lambda kv: -kv[1]["ms"]) if v["ms"] > 0})
        img_bytes = h_img.numel() * 4 + h_lab.numel() * 4
        line = dict(metric=METRIC, value=total_images / (dev_ms * 1e-3), unit=UNIT, n_gpus=world, steps=args.steps,
                    warmup=args.warmup, ms_per_step=dev_ms / args.steps, higher_is_better=True, scaling="weak",
                    vs_baseline=None, dtype="bf16", data="synthetic",
                    config=dict(workload=cfg.name, global_batch=rcfg.N * world, per_gpu_batch=rcfg.N, image=cfg.img,
                                parallelism=f"replicas x{world}", l2="flushed between timed steps (256 MB write)",
                                mode="bf16 conv operands, fp32 accumulate and coupling state"),
                    e2e=dict(value=total_images / (e2e_ms * 1e-3), unit=UNIT, h2d_bytes_per_step=img_bytes,
                             d2h_bytes_per_step=4 + 4 * rcfg.N, ms_per_step=e2e_ms / args.steps),
                    gpu_launches=launches, clocks=clocks, roofline=roof,
                    activation_bytes=int(st.stored_activation_bytes), workspace_bytes=int(st.workspace_peak_bytes),
                    activation_mb_vs_units_per_stage=depth_sweep(ctx, rcfg),
                    flops_per_step=int(st.flops_fwd + st.flops_bwd), final_loss=final_loss, block_ms=block_ms)
        if stored:
            stored["reversible_over_stored_time"] = (dev_ms / args.steps) / stored["ms_per_step"]
            stored["reversible_over_stored_bytes"] = int(st.stored_activation_bytes) / stored["stored_activation_bytes"]
            line["stored_activation_step"] = stored
        if others:
            line["other_workloads"] = others
        if not args.no_cpu and world == 1:
            line["cpu_baseline"] = {k: v for k, v in cpu_baseline(cfg, ref_batch(args, cfg)).items() if k != "seconds_per_step"}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="revnet104")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--ref-batch", type=int, default=0, help="batch of the bounded CPU-oracle sample (0: 2 for 224x224 images, else 32)")
    ap.add_argument("--no-others", action="store_true", help="skip timing the other configurations")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle leg")
    ap.add_argument("--no-stored", action="store_true", help="skip the stored-activation comparison step")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    from paper_1707_04585_b200 import synthetic as syn
    cfg = syn.stack_config(args.config)
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
