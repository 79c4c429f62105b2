#!/usr/bin/env python
"""Benchmark of the fused visual-token reduction (covspec_prune) on synthetic inputs.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config c2] [--impl ours|reference]

One step = one pass of the whole hot path (Eq. 10 through the compacted buffer) over one batch.
`value` is whole-job visual tokens pruned per second with inputs resident in HBM; `e2e` repeats the
measurement with host (pinned) inputs copied in and the results copied out inside the timed region
(two sets of device input buffers, so that the copy of the next step overlaps the kernels of this one).
N > 1 (launched with torch.distributed.run): requests are independent, so every rank prunes its own
batch of the same shape (different seed) with no collective on the data path (weak scaling); the
time is the maximum over ranks.

--impl reference times the CPU oracle (oracle/) on the host cores on a bounded sample of the same
workload; it is a deliberately plain program, reported for context.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2605_02218_b200 import workloads

# dram__bytes_read.sum + dram__bytes_write.sum of one visual-side relevance_tc_kernel launch (ncu,
# profiles/relevance_tc_kernel_c2.md); None where no capture of the current kernel exists.
NCU_TRAFFIC_BYTES = {"c2": 55.62e6, "correct_per_row": 343.9e6 / 512}   # profiles/correct_kernel_vocab152k.md

METRIC = "visual_tokens_pruned_per_s"
UNIT = "tokens/s"


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm=p["hbm_gbs"], tf_burst=p["bf16_tflops"], tf_sust=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm=6650.0, tf_burst=1590.0, tf_sust=1400.0, source="fallback")


def _describe(wl):
    n = np.diff(wl.vis_offsets)
    t = np.diff(wl.txt_offsets)
    return dict(batch=wl.batch, n_vis=[int(n.min()), int(n.max())], n_txt=[int(t.min()), int(t.max())],
                d=wl.d, n_heads=wl.n_heads, head_dim=wl.head_dim, act_layers=wl.act_layers,
                keep=[int(wl.keep.min()), int(wl.keep.max())],
                dtype=str(wl.dtype).replace("torch.", ""))


def algorithmic_work(wl):
    """Algorithmic flops of the relevance stage and bytes of the whole path (per step)."""
    n = np.diff(wl.vis_offsets).astype(np.float64)
    t = np.diff(wl.txt_offsets).astype(np.float64)
    P = wl.n_heads * wl.head_dim if wl.n_heads else wl.d
    e = 2 if wl.dtype == torch.bfloat16 else 4
    proj = 2.0 * n.sum() * wl.d * P if wl.n_heads else 0.0
    qproj = 2.0 * t.sum() * wl.d * P if wl.n_heads else 0.0
    logits = 2.0 * (n * t).sum() * P
    in_bytes = (n.sum() * wl.d * e * (1 + (wl.act_layers + 1 if wl.act_layers else 0))
                + t.sum() * wl.d * e + (2 * P * wl.d * e if wl.n_heads else 0))
    return dict(relevance_flops=proj + logits, qembed_flops=qproj, input_bytes=in_bytes,
                activity_bytes=n.sum() * wl.d * e * (wl.act_layers + 1 if wl.act_layers else 0))


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
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
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(0.02)

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
        return dict(sm_mhz=float(np.median(self.samples)), sm_max_mhz=self.max_mhz,
                    reasons=sorted(self.reasons), samples=len(self.samples))


def cpu_baseline(wl_cpu, budget_s=20.0, min_s=10.0):
    """Times the oracle as it stands on a bounded sample of the workload: whole requests, the batch
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
                sample=f"{reqs} requests ({done_tokens} tokens; the batch of {wl_cpu.batch} visited "
                       f"{passes} time(s)), {dt:.2f} s",
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
    wl = workloads.make_config(args.config, batch=min(args.ref_batch, workloads.CONFIGS[args.config]["batch"]))
    for _ in range(args.warmup):
        cpu_baseline(wl.request(0), budget_s=0, min_s=0)
    t_total, tok_total, samples = 0.0, 0, []
    for _ in range(args.steps):
        # every step is a bounded sample; the whole run stays within a few minutes
        per_step = max(0.5, min(10.0, args.ref_budget, 150.0 / max(args.steps, 1)))
        r = cpu_baseline(wl, budget_s=max(per_step, 1.5 * per_step), min_s=per_step)
        t_total += r["seconds"]
        tok_total += r["value"] * r["seconds"]
        samples.append(r["sample"])
    value = tok_total / t_total
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=1e3 * t_total / args.steps, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="f64", data="synthetic", impl="reference",
                config=dict(workload=f"{args.config}: " + json.dumps(_describe(wl)),
                            note="CPU oracle on a bounded sample of the workload"),
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
    # The kernel evaluates 4.25 exponentials per vocabulary entry (softmax denominators with one
    # rescale per 8-element vector, then both probabilities again for the residual); the special
    # function units deliver 16 per clock per SM.
    exps = 4.25 * rows * vocab
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    xu_peak = 16.0 * sms * 1.965                             # G exp/s at the 1965 MHz maximum clock
    gexp = exps / (ms * 1e-3) / 1e9
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
        roofline=dict(bound="alu", achieved=gexp, peak=xu_peak, unit="Gexp/s", frac=gexp / xu_peak,
                      traffic=NCU_TRAFFIC_BYTES.get("correct_per_row", 0) * rows or None,
                      kernel="correct_kernel<__half>",
                      peak_source="16 exp/clk/SM x %d SMs x 1.965 GHz" % sms,
                      hbm=dict(achieved=gbs, peak=peaks["hbm"], unit="GB/s", frac=gbs / peaks["hbm"],
                               bytes_per_launch=bytes_alg)),
        cpu_baseline=dict(value=n / dt, unit="positions/s", cores=1, kind="oracle",
                          sample=f"{n} positions of the same rows, {dt:.1f} s"))))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", default="c2", choices=sorted(workloads.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--copies", type=int, default=0, help="independent input sets to rotate through")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--ref-batch", type=int, default=16)
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

    # Input sets: rotate through enough independent copies that the working set of consecutive
    # steps exceeds twice the 126 MB L2.
    base_seed = rank_seed(args.config, rank)
    wl0 = workloads.make_config(args.config, device=dev, seed=base_seed)
    work = algorithmic_work(wl0)
    copies = args.copies or max(2, int(np.ceil(2 * 126e6 * 2 / work["input_bytes"])))
    copies = min(copies, 8)
    sizes = (np.diff(wl0.vis_offsets).tolist(), np.diff(wl0.txt_offsets).tolist())
    sets = [wl0] + [workloads.make_config(args.config, device=dev, seed=base_seed + 17 * (i + 1),
                                          sizes=sizes) for i in range(copies - 1)]
    pr = api.Pruner.for_workload(wl0)
    ms = [pr.marshal(w) for w in sets]
    ko, _ = pr.plan_sizes(ms[0])
    n_keep = int(ko[-1])
    outs = [torch.empty((n_keep, wl0.d), dtype=wl0.dtype, device=dev) for _ in sets]
    keeps = [torch.empty(n_keep, dtype=torch.int32, device=dev) for _ in sets]
    tokens = wl0.total_vis

    def step(i):
        j = i % copies
        pr.prune(ms[j], outs[j], keeps[j])

    # ---- device-resident timing ---------------------------------------------------------------
    for i in range(max(args.warmup, 3)):
        step(i)
    pr.check_device_status()
    launches_per_step = pr.last_launch_count
    barrier()
    pr.profile_begin(args.steps)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local_rank) as clk:
        ev0.record()
        for i in range(args.steps):
            step(i)
        ev1.record()
        barrier()
    ms_total = ev0.elapsed_time(ev1)
    stage_ms, prof_calls = pr.profile_end()
    pr.check_device_status()

    # ---- end to end: pinned host inputs in, results out, every step -----------------------------
    host = wl0.to("cpu")
    pin = lambda t: t.pin_memory()
    hX, hQ, hHs = pin(host.X), pin(host.Q), [pin(h) for h in host.Hs]
    # Two sets of device input buffers: the copy of step i+1 (on a copy stream) overlaps the kernels
    # of step i.  Every step still copies all of its inputs in and its results out.
    n_buf = 2
    dXs = [torch.empty_like(wl0.X) for _ in range(n_buf)]
    dQs = [torch.empty_like(wl0.Q) for _ in range(n_buf)]
    dHss = [[torch.empty_like(h) for h in wl0.Hs] for _ in range(n_buf)]
    m_e2e = [pr.marshal(X=dXs[i], Q=dQs[i], vis_offsets=wl0.vis_offsets, txt_offsets=wl0.txt_offsets,
                        Wq=wl0.Wq, Wk=wl0.Wk, Hs=dHss[i], keep=wl0.keep) for i in range(n_buf)]
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
            pr.prune(m_e2e[j], outs[0], keeps[0])
            consumed[j].record(main_stream)
            h_out.copy_(outs[0], non_blocking=True)
            h_keep.copy_(keeps[0], non_blocking=True)

    e2e_steps = max(3, min(args.steps, 20))
    run_e2e(3)
    barrier()
    ev0.record()
    run_e2e(e2e_steps)
    ev1.record()
    barrier()
    ms_e2e = ev0.elapsed_time(ev1) / e2e_steps

    # ---- reduce over ranks ------------------------------------------------------------------
    ms_step = ms_total / args.steps
    ms_step, ms_e2e = reduce_max([ms_step, ms_e2e], dist, dev)
    if rank == 0:
        peaks = _peaks()
        rel_ms = stage_ms["relevance"] / max(prof_calls, 1)
        long_region = ms_total > 1000.0
        peak_tf = peaks["tf_sust"] if long_region else peaks["tf_burst"]
        if wl0.dtype != torch.bfloat16:
            peak_tf *= 0.5            # tf32 / fp32 path: nominal ratio to the bf16 peak
        achieved = work["relevance_flops"] / (rel_ms * 1e-3) / 1e12 if rel_ms > 0 else 0.0
        traffic = NCU_TRAFFIC_BYTES.get(args.config)
        line = dict(
            metric=METRIC, value=world * tokens / (ms_step * 1e-3), unit=UNIT, n_gpus=world,
            steps=args.steps, warmup=max(args.warmup, 3), ms_per_step=ms_step, higher_is_better=True,
            scaling="weak", vs_baseline=None,
            dtype="bf16" if wl0.dtype == torch.bfloat16 else "f32", data="synthetic",
            config=dict(workload=f"{args.config}: " + json.dumps(_describe(wl0)),
                        l2="rotating %d independent input sets (%.0f MB) between steps" %
                           (copies, copies * work["input_bytes"] / 1e6),
                        us_per_request=1e3 * ms_step / wl0.batch, parallelism=f"dp{world} (requests sharded)"),
            e2e=dict(value=world * tokens / (ms_e2e * 1e-3), unit=UNIT, h2d_bytes_per_step=int(h2d),
                     d2h_bytes_per_step=int(d2h), ms_per_step=ms_e2e),
            gpu_launches=launches_per_step * args.steps,
            clocks=clk.summary(),
            roofline=dict(bound="tensor", achieved=achieved, peak=peak_tf, unit="TFLOP/s",
                          frac=achieved / peak_tf, traffic=traffic,
                          kernel="relevance stage (projection + cosine max, Eq. 10)",
                          peak_source=("sustained" if long_region else "burst") + " bf16, " + peaks["source"],
                          flops_per_step=work["relevance_flops"], ms_per_launch=rel_ms),
            stages_ms={k: v / max(prof_calls, 1) for k, v in stage_ms.items()},
        )
        if not args.no_cpu_baseline and world == 1:
            cb = cpu_baseline(host)
            cb.pop("seconds")
            line["cpu_baseline"] = cb
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
