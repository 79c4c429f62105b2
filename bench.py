#!/usr/bin/env python
"""Benchmark of the fused visual-token reduction (covspec_prune) on synthetic inputs.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config c5] [--impl ours|reference]

One step = one pass of the whole hot path (Eq. 10 through the compacted buffer) over one batch.
The default workload is c5, the largest configuration that runs on one GPU.  `value` is whole-job
visual tokens pruned per second with inputs resident in HBM; `e2e` repeats the measurement with host
(pinned) inputs copied in and the results copied out inside the timed region (two sets of device
input buffers, so that the copy of the next step overlaps the kernels of this one).  `roofline` is
about the fused call: the algorithmic flops (or bytes) of all stages over the measured step time,
against the measured peak; the stage that takes the largest share of the step and the relevance
kernel are reported beside it.  `other_configs` holds the step time and the same fraction of every
other named configuration, measured in the same process.
N > 1 (launched with torch.distributed.run): requests are independent, so every rank prunes its own
batch of the same shape (different seed) with no collective on the data path (weak scaling); the
time is the maximum over ranks.

--impl reference times the CPU oracle (oracle/) on the host cores on a bounded sample of the same
workload; it is a deliberately plain program, reported for context.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2605_02218_b200 import workloads

# dram__bytes_read.sum + dram__bytes_write.sum of the visual-side relevance kernel from one ncu
# capture on c5 cut to one request (16384 tokens: 148.6 MB, of which the 25.7 MB of projection
# weights are read once per launch and the rest grows with the tokens), scaled to the tokens one
# launch of the full workload processes; see the summary named here.
NCU_RELEVANCE_TRAFFIC = {"bytes_per_token": (148.589e6 - 25.69e6) / 16384, "fixed_bytes": 25.69e6, "config": "c5",
                         "source": "profiles/relevance_tc_kernel_c5_one_request.md"}
NCU_CORRECT_BYTES_PER_ROW = 366.5e6 / 512          # profiles/correct_kernel_vocab152k.md

METRIC = "visual_tokens_pruned_per_s"
UNIT = "tokens/s"
L2_BYTES = 126e6


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm=p["hbm_gbs"], tf_burst=p["bf16_tflops"], tf_sust=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm=6650.0, tf_burst=1590.0, tf_sust=1400.0, source="fallback")


def _describe(name, n_vis, n_txt, keep):
    c = workloads.CONFIGS[name]
    return dict(batch=len(keep), n_vis=[int(min(n_vis)), int(max(n_vis))],
                n_txt=[int(min(n_txt)), int(max(n_txt))], d=c["d"], n_heads=c["n_heads"],
                head_dim=128, act_layers=4, keep=[int(min(keep)), int(max(keep))],
                dtype=str(c["dtype"]).replace("torch.", ""))


def config_sizes(name):
    """Request sizes of a named configuration without building its tensors (uniform sizes only);
    None for the ragged one, whose sizes are drawn with the tensors."""
    c = workloads.CONFIGS[name]
    if isinstance(c["n_vis"], (tuple, list)) or isinstance(c["n_txt"], (tuple, list)):
        return None
    n = [c["n_vis"]] * c["batch"]
    t = [c["n_txt"]] * c["batch"]
    keep = [c["keep"] if "keep" in c else workloads.keep_from_ratio(v, c["keep_ratio"]) for v in n]
    return n, t, keep


def config_dict(name, n_vis, n_txt, keep, world):
    """The `config` object of the JSON line; both arms build it here so that they agree key by key."""
    e = 2 if workloads.CONFIGS[name]["dtype"] == torch.bfloat16 else 4
    d = workloads.CONFIGS[name]["d"]
    in_bytes = (sum(n_vis) * 6 + sum(n_txt)) * d * e
    return dict(workload=f"{name}: " + json.dumps(_describe(name, n_vis, n_txt, keep)),
                l2=("inputs of one step (%.0f MB) exceed the 126 MB L2" % (in_bytes / 1e6)
                    if in_bytes > 2 * L2_BYTES else
                    "consecutive steps rotate through independent input sets larger than twice the L2"),
                parallelism=f"dp{world} (requests sharded, no collective)")


def algorithmic_work(name, n_vis, n_txt, keep, budgets):
    """Algorithmic flops and bytes of one fused call: every input read once, the preselected and the
    kept rows gathered, the outputs written; projection, logits, Gram and eight subspace
    multiplications with r + 32 vectors.  budgets(n, keep) -> (B_vis, M, r)."""
    c = workloads.CONFIGS[name]
    d, H = c["d"], c["n_heads"]
    P = H * 128 if H else d
    e = 2 if c["dtype"] == torch.bfloat16 else 4
    A = 4
    n = np.asarray(n_vis, dtype=np.float64)
    t = np.asarray(n_txt, dtype=np.float64)
    bm = [budgets(int(a), int(k)) for a, k in zip(n_vis, keep)]
    B = np.array([x[0] for x in bm], dtype=np.float64)
    M = np.array([x[1] for x in bm], dtype=np.float64)
    r = np.array([x[2] for x in bm], dtype=np.float64)
    stage2 = B < M
    proj = 2.0 * n.sum() * d * P if H else 0.0
    qproj = 2.0 * t.sum() * d * P if H else 0.0
    logits = 2.0 * (n * t).sum() * P
    gram = float((2.0 * M * M * d * stage2).sum())
    eig = float((8 * 2.0 * M * M * (r + 32) * stage2).sum())
    inputs = n.sum() * d * e * (A + 2) + t.sum() * d * e + (2 * P * d * e if H else 0)
    gathers = float((M * stage2 + B).sum()) * d * e
    outputs = float(B.sum()) * d * e + 4 * float(B.sum())
    return dict(flops=proj + qproj + logits + gram + eig, bytes=inputs + gathers + outputs,
                relevance_flops=proj + logits, qembed_flops=qproj, gram_flops=gram, eig_flops=eig,
                activity_bytes=n.sum() * d * e * (A + 1), input_bytes=inputs)


# stage (as the library's event timing names it) -> its own roofline: ("tensor", flops key) or
# ("hbm", bytes key); stages with neither are small latency-bound kernels
STAGE_BOUND = {"query_embed": ("tensor", "qembed_flops"), "relevance": ("tensor", "relevance_flops"),
               "activity": ("hbm", "activity_bytes"), "gram": ("tensor", "gram_flops"),
               "subspace": ("tensor", "eig_flops")}


def fused_roofline(work, ms_step, peaks, f32):
    """max(t_HBM, t_tensor) / t_measured of one fused call, with the figures it comes from."""
    tf = peaks["tf_sust"] * (0.5 if f32 else 1.0)     # tf32 / float32 path: nominal ratio to bf16
    t_hbm = work["bytes"] / (peaks["hbm"] * 1e9) * 1e3
    t_tensor = work["flops"] / (tf * 1e12) * 1e3
    if t_tensor >= t_hbm:
        achieved = work["flops"] / (ms_step * 1e-3) / 1e12
        return dict(bound="tensor", achieved=achieved, peak=tf, unit="TFLOP/s", frac=achieved / tf,
                    t_hbm_ms=t_hbm, t_tensor_ms=t_tensor)
    achieved = work["bytes"] / (ms_step * 1e-3) / 1e9
    return dict(bound="hbm", achieved=achieved, peak=peaks["hbm"], unit="GB/s",
                frac=achieved / peaks["hbm"], t_hbm_ms=t_hbm, t_tensor_ms=t_tensor)


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz, self.mask = [], set(), None, 0
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
            "applications_clocks_setting": getattr(nv, "nvmlClocksThrottleReasonApplicationsClocksSetting", 0x2),
            "sync_boost": getattr(nv, "nvmlClocksThrottleReasonSyncBoost", 0x10),
            "display_clock_setting": getattr(nv, "nvmlClocksThrottleReasonDisplayClockSetting", 0x100),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.mask |= int(mask)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(0.01)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return dict(sm_mhz=None, sm_max_mhz=self.max_mhz, reasons=sorted(self.reasons), samples=0)
        return dict(sm_mhz=float(np.median(self.samples)), sm_min_mhz=float(min(self.samples)),
                    sm_max_mhz=self.max_mhz, reasons=sorted(self.reasons), reason_mask=hex(self.mask),
                    samples=len(self.samples))


def oracle_sample(name, wl_cpu=None):
    """The bounded sample of a configuration that the CPU legs time: whole requests of the workload;
    for requests of more than 4096 tokens, one request cut to its first 2048 tokens with the keep
    budget scaled by the same factor.  Returns (workload on the CPU, description)."""
    c = workloads.CONFIGS[name]
    if not isinstance(c["n_vis"], (tuple, list)) and c["n_vis"] > 4096:
        frac = 2048 / c["n_vis"]
        keep = max(1, int(round(c["keep"] * frac))) if "keep" in c else None
        kw = dict(batch=1, n_vis=2048)
        if keep is not None:
            kw["keep"] = keep
        return (workloads.make_config(name, **kw),
                f"one request cut to its first 2048 of {c['n_vis']} tokens, keep budget scaled to {keep}")
    if wl_cpu is None:
        wl_cpu = workloads.make_config(name, batch=min(16, c["batch"]))
    return wl_cpu, "whole requests of the workload"


def cpu_baseline(wl_cpu, what, budget_s=20.0, min_s=10.0):
    """Times the oracle as it stands on a bounded sample: the sample's requests one after the other,
    repeated until about `min_s` seconds of CPU work are done, stopping at `budget_s`."""
    from oracle import covspec_oracle as oracle
    n = np.diff(wl_cpu.vis_offsets)
    done_tokens, reqs, passes = 0, 0, 0
    t0 = time.perf_counter()
    stop = False
    while not stop:
        for b in range(wl_cpu.batch):
            oracle.prune_batch(wl_cpu, requests=[b])
            done_tokens += int(n[b])
            reqs += 1
            if time.perf_counter() - t0 > budget_s:
                stop = True
                break
        passes += 1
        if time.perf_counter() - t0 >= min_s:
            stop = True
    dt = time.perf_counter() - t0
    cores = len(os.sched_getaffinity(0))
    return dict(value=done_tokens / dt, unit=UNIT, cores=cores, kind="oracle",
                sample=f"{what}: {reqs} request run(s), {done_tokens} tokens, {dt:.2f} s",
                seconds=dt)


def rank_seed(config, rank):
    """Requests are independent, so every rank prunes its own batch: same shapes, its own seed."""
    return workloads.CONFIGS[config]["seed"] + 1000 * rank


def reduce_max(values, dist, device):
    """Maximum over ranks of a list of per-rank timings (the job is as slow as its slowest rank)."""
    if dist is None:
        return list(values)
    t = torch.tensor(values, device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def run_reference(args, rank):
    if rank != 0:
        return
    sizes = config_sizes(args.config)
    full = None
    if sizes is None:                                  # ragged: the sizes come with the tensors
        full = workloads.make_config(args.config)
        sizes = (np.diff(full.vis_offsets).tolist(), np.diff(full.txt_offsets).tolist(), full.keep.tolist())
    wl, what = oracle_sample(args.config, full)
    for _ in range(args.warmup):
        cpu_baseline(wl.request(0), what, budget_s=0, min_s=0)
    t_total, tok_total, samples = 0.0, 0, []
    per_step = max(0.5, min(10.0, args.ref_budget, 150.0 / max(args.steps + args.warmup, 1)))
    for _ in range(args.steps):
        # every step is a bounded sample; the whole run stays within a few minutes
        r = cpu_baseline(wl, what, budget_s=1.5 * per_step, min_s=per_step)
        t_total += r["seconds"]
        tok_total += r["value"] * r["seconds"]
        samples.append(r["sample"])
    value = tok_total / t_total
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=1e3 * t_total / args.steps, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="f64", data="synthetic", impl="reference",
                config=config_dict(args.config, *sizes, args.gpus),
                cpu_baseline=dict(value=value, unit=UNIT, cores=len(os.sched_getaffinity(0)),
                                  kind="oracle", sample=samples[-1]),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line))


def run_correction(args):
    """Secondary measurement (not the headline metric): covspec_correct, the device-side gating and
    residual-correction kernel (Eq. 5, 6, 16, 17), on float16 logit rows of a 151,674-token
    vocabulary.  HBM-bound: both logit rows are read once from HBM."""
    from paper_2605_02218_b200 import api, build
    from oracle import correction_oracle
    build.build()
    torch.cuda.set_device(0)
    rows, vocab = args.corr_rows, 151674
    data = workloads.make_logits(seed=11, rows=rows, vocab=vocab, dtype=torch.float16, device="cuda:0")
    call = lambda: api.correct(data["z_draft"], data["z_target"], data["uniforms"], 0.02, data["drafted"], vocab=vocab)
    for _ in range(max(args.warmup, 3)):
        call()
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(0) as clk:
        ev0.record()
        for _ in range(args.steps):
            call()
        ev1.record()
        torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / args.steps
    bytes_alg = 2.0 * rows * vocab * 2                       # both logit rows, once
    peaks = _peaks()
    gbs = bytes_alg / (ms * 1e-3) / 1e9
    zd = data["z_draft"][:8, :vocab].cpu().double().numpy(); zt = data["z_target"][:8, :vocab].cpu().double().numpy()
    xs = data["uniforms"][:8].cpu().numpy()
    t0 = time.perf_counter(); n = 0
    while time.perf_counter() - t0 < 10.0:
        correction_oracle.correct_position(zd[n % 8], zt[n % 8], float(xs[n % 8]), 0.02, y=3)
        n += 1
    dt = time.perf_counter() - t0
    print(json.dumps(dict(
        metric="positions_corrected_per_s", value=rows / (ms * 1e-3), unit="positions/s", n_gpus=1,
        steps=args.steps, warmup=max(args.warmup, 3), ms_per_step=ms, higher_is_better=True,
        dtype="f32", data="synthetic",
        config=dict(workload=f"covspec_correct: {rows} positions x {vocab} logits, float16, draft + target rows",
                    l2="inputs (%.0f MB) larger than L2" % (bytes_alg / 1e6)),
        gpu_launches=args.steps, clocks=clk.summary(),
        roofline=dict(bound="hbm", achieved=gbs, peak=peaks["hbm"], unit="GB/s", frac=gbs / peaks["hbm"],
                      traffic=NCU_CORRECT_BYTES_PER_ROW * rows, kernel="correct_kernel<__half>",
                      peak_source="copy bandwidth, " + peaks["source"], bytes_per_launch=bytes_alg),
        cpu_baseline=dict(value=n / dt, unit="positions/s", cores=1, kind="oracle",
                          sample=f"{n} positions of the same rows, {dt:.1f} s"))))


class Runner:
    """One configuration on one device: input sets, context, output buffers."""

    def __init__(self, api, name, dev, seed, copies=0, batch=0):
        self.name, self.dev = name, dev
        over = dict(batch=batch) if batch else {}
        wl0 = workloads.make_config(name, device=dev, seed=seed, **over)
        self.wl0 = wl0
        self.n_vis = np.diff(wl0.vis_offsets).tolist()
        self.n_txt = np.diff(wl0.txt_offsets).tolist()
        self.keep = wl0.keep.tolist()
        in_bytes = (wl0.X.nbytes + wl0.Q.nbytes + sum(h.nbytes for h in wl0.Hs))
        # rotate through enough independent input sets that consecutive steps cannot hit in L2
        copies = copies or max(2, int(math.ceil(4 * L2_BYTES / in_bytes)))
        self.copies = min(copies, 8)
        sizes = (self.n_vis, self.n_txt)
        self.sets = [wl0] + [workloads.make_config(name, device=dev, seed=seed + 17 * (i + 1), sizes=sizes, **over)
                             for i in range(self.copies - 1)]
        self.pr = api.Pruner.for_workload(wl0)
        self.ms = [self.pr.marshal(w) for w in self.sets]
        ko, _ = self.pr.plan_sizes(self.ms[0])
        self.n_keep = int(ko[-1])
        self.outs = [torch.empty((self.n_keep, wl0.d), dtype=wl0.dtype, device=dev) for _ in self.sets]
        self.keeps = [torch.empty(self.n_keep, dtype=torch.int32, device=dev) for _ in self.sets]
        self.tokens = wl0.total_vis
        self.work = algorithmic_work(name, self.n_vis, self.n_txt, self.keep,
                                     lambda n, k: api.budgets(self.pr.cfg, n, k))

    def step(self, i, rotate=True):
        j = i % self.copies if rotate else 0
        self.pr.prune(self.ms[j], self.outs[j], self.keeps[j])

    def timed(self, steps, warmup, rotate=True, barrier=None, profile=False, clocks=None):
        """`steps` timed steps after `warmup`: total ms between the first and the last event (the
        contract's figure), the per-step times (for the median) and the per-stage times."""
        for i in range(max(warmup, 3)):
            self.step(i, rotate)
        self.pr.check_device_status()
        launches = self.pr.last_launch_count
        (barrier or torch.cuda.synchronize)()
        if profile:
            self.pr.profile_begin(steps)
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        ctx = clocks if clocks is not None else _Null()
        with ctx:
            evs[0].record()
            for i in range(steps):
                self.step(i, rotate)
                evs[i + 1].record()
            (barrier or torch.cuda.synchronize)()
        total = evs[0].elapsed_time(evs[steps])
        per = [evs[i].elapsed_time(evs[i + 1]) for i in range(steps)]
        stages, calls = (self.pr.profile_end() if profile else ({}, 0))
        self.pr.check_device_status()
        return dict(total_ms=total, per_step_ms=per, launches=launches,
                    stages={k: v / max(calls, 1) for k, v in stages.items()})

    def close(self):
        self.pr.close()
        self.sets = self.ms = self.outs = self.keeps = None
        torch.cuda.empty_cache()


class _Null:
    def __enter__(self):
        return self

    def __exit__(self, *a):
        return False


def measure_other(api, name, dev, peaks, steps):
    """Step time and fused-call roofline fraction of another configuration (cold: rotating input
    sets; warm: the same set every step, reported for the two that nearly fit in L2)."""
    r = Runner(api, name, dev, workloads.CONFIGS[name]["seed"])
    cold = r.timed(steps, 5, profile=True)
    ms_mean = cold["total_ms"] / steps
    ms_med = float(np.median(cold["per_step_ms"]))
    f32 = r.wl0.dtype != torch.bfloat16
    roof = fused_roofline(r.work, ms_med, peaks, f32)
    out = dict(ms_per_step=ms_mean, ms_median=ms_med, tokens_per_s=r.tokens / (ms_med * 1e-3),
               us_per_request=1e3 * ms_med / r.wl0.batch, launches_per_step=cold["launches"],
               roofline=dict(bound=roof["bound"], frac=roof["frac"], t_hbm_ms=roof["t_hbm_ms"],
                             t_tensor_ms=roof["t_tensor_ms"]),
               stages_ms=cold["stages"], input_sets=r.copies)
    if r.work["input_bytes"] < 4 * L2_BYTES:
        warm = r.timed(steps, 5, rotate=False)
        out["warm_l2_ms_median"] = float(np.median(warm["per_step_ms"]))
    r.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", default="c5", choices=sorted(workloads.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--copies", type=int, default=0, help="independent input sets to rotate through")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-others", action="store_true", help="skip the other named configurations")
    ap.add_argument("--no-e2e", action="store_true", help="skip the end-to-end leg (profiling runs)")
    ap.add_argument("--batch", type=int, default=0,
                    help="cut the configuration to this many requests (small cases for profiler captures; "
                         "the line then says so in config.workload)")
    ap.add_argument("--ref-budget", type=float, default=20.0)
    ap.add_argument("--kernel", default="prune", choices=["prune", "correct"],
                    help="prune: the headline path (default); correct: the gating / correction kernel")
    ap.add_argument("--corr-rows", type=int, default=1024)
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", 0))
    local_rank = int(os.environ.get("LOCAL_RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.kernel == "correct":
        if rank == 0:
            run_correction(args)
        return

    from paper_2605_02218_b200 import api, build
    build.build()
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    run = Runner(api, args.config, dev, rank_seed(args.config, rank), args.copies, args.batch)
    wl0, pr, work = run.wl0, run.pr, run.work
    tokens = run.tokens

    # ---- device-resident timing ---------------------------------------------------------------
    clk = ClockSampler(local_rank)
    res = run.timed(args.steps, args.warmup, barrier=barrier, profile=True, clocks=clk)
    ms_total, stage_ms = res["total_ms"], res["stages"]
    launches_per_step = res["launches"]
    ms_median = float(np.median(res["per_step_ms"]))

    # ---- end to end: pinned host inputs in, results out, every step -----------------------------
    host = wl0.to("cpu")
    ms_e2e, h2d, d2h = float("nan"), 0, 0
    if not args.no_e2e:
        pin = lambda t: t.pin_memory()
        hX, hQ, hHs = pin(host.X), pin(host.Q), [pin(h) for h in host.Hs]
        # Two sets of device input buffers: the copy of step i+1 (on a copy stream) overlaps the
        # kernels of step i.  Every step still copies all of its inputs in and its results out.
        n_buf = 2
        dXs = [run.sets[i % run.copies].X for i in range(n_buf)]
        dQs = [run.sets[i % run.copies].Q for i in range(n_buf)]
        dHss = [run.sets[i % run.copies].Hs for i in range(n_buf)]
        m_e2e = [pr.marshal(X=dXs[i], Q=dQs[i], vis_offsets=wl0.vis_offsets, txt_offsets=wl0.txt_offsets,
                            Wq=wl0.Wq, Wk=wl0.Wk, Hs=dHss[i], keep=wl0.keep) for i in range(n_buf)]
        n_keep = run.n_keep
        h_out = torch.empty((n_keep, wl0.d), dtype=wl0.dtype).pin_memory()
        h_keep = torch.empty(n_keep, dtype=torch.int32).pin_memory()
        h2d = hX.nbytes + hQ.nbytes + sum(h.nbytes for h in hHs)
        d2h = h_out.nbytes + h_keep.nbytes
        copy_stream = torch.cuda.Stream(device=dev)
        main_stream = torch.cuda.current_stream(dev)
        copied = [torch.cuda.Event() for _ in range(n_buf)]      # inputs of the set are on the device
        consumed = [torch.cuda.Event() for _ in range(n_buf)]    # the kernels that read the set are done
        for ev in consumed:
            ev.record(main_stream)

        def upload(i):
            j = i % n_buf
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(consumed[j])
                dXs[j].copy_(hX, non_blocking=True)
                dQs[j].copy_(hQ, non_blocking=True)
                for a_, b_ in zip(dHss[j], hHs):
                    a_.copy_(b_, non_blocking=True)
                copied[j].record(copy_stream)

        def run_e2e(n_steps):
            upload(0)
            for i in range(n_steps):
                j = i % n_buf
                if i + 1 < n_steps:
                    upload(i + 1)
                main_stream.wait_event(copied[j])
                pr.prune(m_e2e[j], run.outs[0], run.keeps[0])
                consumed[j].record(main_stream)
                h_out.copy_(run.outs[0], non_blocking=True)
                h_keep.copy_(run.keeps[0], non_blocking=True)

        e2e_steps = max(3, min(args.steps, 20))
        run_e2e(3)
        barrier()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        run_e2e(e2e_steps)
        ev1.record()
        barrier()
        ms_e2e = ev0.elapsed_time(ev1) / e2e_steps
        pr.check_device_status()
        del hX, hQ, hHs

    # ---- reduce over ranks ------------------------------------------------------------------
    ms_step = ms_total / args.steps
    ms_step, ms_e2e, ms_median = reduce_max([ms_step, ms_e2e, ms_median], dist, dev)
    run.close()
    if rank == 0:
        peaks = _peaks()
        f32 = wl0.dtype != torch.bfloat16
        roof = fused_roofline(work, ms_step, peaks, f32)
        # the stage that takes the largest share of the step, against its own bound
        dom = max(stage_ms, key=lambda k: stage_ms[k]) if stage_ms else None
        dom_info = None
        if dom is not None:
            dom_info = dict(stage=dom, ms=stage_ms[dom], share_of_step=stage_ms[dom] / ms_step)
            kind, key = STAGE_BOUND.get(dom, (None, None))
            burst = peaks["tf_burst"] * (0.5 if f32 else 1.0)
            if kind == "tensor":
                a = work[key] / (stage_ms[dom] * 1e-3) / 1e12
                dom_info.update(bound="tensor", achieved=a, peak=burst, unit="TFLOP/s", frac=a / burst)
            elif kind == "hbm":
                a = work[key] / (stage_ms[dom] * 1e-3) / 1e9
                dom_info.update(bound="hbm", achieved=a, peak=peaks["hbm"], unit="GB/s", frac=a / peaks["hbm"])
        rel_ms = stage_ms.get("relevance", 0.0)
        burst = peaks["tf_burst"] * (0.5 if f32 else 1.0)
        rel_tf = work["relevance_flops"] / (rel_ms * 1e-3) / 1e12 if rel_ms > 0 else 0.0
        traffic = None
        if NCU_RELEVANCE_TRAFFIC["bytes_per_token"] and NCU_RELEVANCE_TRAFFIC["config"] == args.config:
            traffic = NCU_RELEVANCE_TRAFFIC["bytes_per_token"] * tokens + NCU_RELEVANCE_TRAFFIC["fixed_bytes"]
        roofline = dict(bound=roof["bound"], achieved=roof["achieved"], peak=roof["peak"], unit=roof["unit"],
                        frac=roof["frac"], traffic=traffic,
                        kernel="covspec_prune (fused call, all stages); dominant stage: %s" % dom,
                        what="max(t_HBM, t_tensor) of the algorithmic work of all stages over the measured step",
                        peak_source="sustained bf16 / copy bandwidth, " + peaks["source"],
                        t_hbm_ms=roof["t_hbm_ms"], t_tensor_ms=roof["t_tensor_ms"],
                        flops_per_step=work["flops"], bytes_per_step=work["bytes"],
                        dominant_stage=dom_info,
                        relevance_kernel=dict(bound="tensor", achieved=rel_tf, peak=burst, unit="TFLOP/s",
                                              frac=rel_tf / burst if burst else None, ms_per_launch=rel_ms,
                                              flops_per_launch=work["relevance_flops"], traffic=traffic,
                                              traffic_source=NCU_RELEVANCE_TRAFFIC["source"],
                                              note="stage time by events; the activity stream (Eq. 11) runs "
                                                   "beside this kernel on a second stream and slows it",
                                              peak_source="burst bf16, " + peaks["source"]))
        line = dict(
            metric=METRIC, value=world * tokens / (ms_step * 1e-3), unit=UNIT, n_gpus=world,
            steps=args.steps, warmup=max(args.warmup, 3), ms_per_step=ms_step, higher_is_better=True,
            scaling="weak", vs_baseline=None,
            dtype="bf16" if not f32 else "f32", data="synthetic",
            config=config_dict(args.config, run.n_vis, run.n_txt, run.keep, world),
            us_per_request=1e3 * ms_step / wl0.batch, ms_median=ms_median, input_sets=run.copies,
            e2e=dict(value=world * tokens / (ms_e2e * 1e-3), unit=UNIT, h2d_bytes_per_step=int(h2d),
                     d2h_bytes_per_step=int(d2h), ms_per_step=ms_e2e) if not args.no_e2e else None,
            gpu_launches=launches_per_step * args.steps,
            clocks=clk.summary(),
            roofline=roofline,
            stages_ms=stage_ms,
        )
        if world == 1 and not args.no_others:
            others = {}
            for name in sorted(workloads.CONFIGS):
                if name != args.config:
                    others[name] = measure_other(api, name, dev, peaks, max(10, min(args.steps, 30)))
            line["other_configs"] = others
        if not args.no_cpu_baseline and world == 1:
            sample, what = oracle_sample(args.config, host)
            cb = cpu_baseline(sample, what)
            cb.pop("seconds")
            line["cpu_baseline"] = cb
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
