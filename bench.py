#!/usr/bin/env python
"""Benchmark of the scoring-and-selection path on B200.

One step = one pass of the whole path over one batch of synthetic input: sp_score (SneakPeek head,
softmax, accuracy contraction, variance) followed by sp_schedule_round until every instance is drained.
Default workload: the batched configuration, 16,384 independent scheduling instances x 512 requests
(3 applications x 6 models, 20 labels, 128 fp32 features), 8.39 M requests and 4.3 GB of features per step.

  python bench.py --gpus 1 --steps 300 --warmup 5           # this library
  python bench.py --impl reference --steps 3 --warmup 1      # the CPU oracle, as it stands, on host cores
Under torchrun every rank runs its own shard of instances (weak scaling, no collective on the data path).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "requests scored+scheduled/sec"
UNIT = "requests/s"
FULL = {"C1": {}, "C2": {}, "C3": {}, "C4": {}, "C5": {}}
ROUND_CAP = 16              # round records kept per instance in the batched workload


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C4", choices=sorted(FULL))
    ap.add_argument("--instances", type=int, default=None, help="override the number of instances (C4)")
    ap.add_argument("--requests", type=int, default=None, help="override requests per instance")
    ap.add_argument("--cpu-sample-instances", type=int, default=4096)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-side-workloads", action="store_true", help="skip the short C3 and C5 passes of the default run")
    return ap.parse_args()


def make(args, rank, n_instances=None):
    from paper_2505_06641_b200 import synth
    kw = {}
    if args.requests is not None:
        kw["n_requests"] = args.requests
    ni = n_instances if n_instances is not None else args.instances
    if args.workload == "C4":
        from paper_2505_06641_b200 import shard
        full = synth._SPECS["C4"][2]
        ni = ni if ni is not None else full
        first, _ = shard.instance_shard(rank, max(rank + 1, int(os.environ.get("WORLD_SIZE", "1"))), full)
        return synth.make_workload("C4", n_instances=ni, first_instance=first, **kw)
    return synth.make_workload(args.workload, **kw)


def algorithmic_bytes_per_request(w):
    """Bytes the scoring kernel must move per request: the feature row in, acc[Mmax] and v out."""
    esz = 2 if int(w.feat_dtype) == 1 else 4
    return int(w.feat_dim) * esz + 4 * (int(np.max(w.models_per_app)) + 1)


def cpu_oracle_workload(args):
    """The bounded sample of the workload that the oracle is timed on."""
    from paper_2505_06641_b200 import synth
    if args.workload == "C4":
        ni = args.cpu_sample_instances if args.instances is None else min(args.instances, args.cpu_sample_instances)
        w = make(args, 0, n_instances=ni)
        return w, "first %d of the instances (%d requests)" % (ni, w.n_requests)
    n = {"C1": None, "C2": None, "C3": 16384, "C5": 100000}[args.workload]
    if args.requests is not None:
        n = args.requests if n is None else min(n, args.requests)
    w = synth.make_workload(args.workload, **({} if n is None else {"n_requests": n}))
    return w, "%d requests of the workload" % w.n_requests


def cpu_oracle_time(w):
    """One oracle pass (score + drain) over ``w``: (seconds, rounds)."""
    from oracle import oracle
    t = time.perf_counter()
    s = oracle.score(w)
    d = oracle.drain(w, s.acc, s.v)
    return time.perf_counter() - t, int(d.n_rounds.sum())


def cpu_oracle_sample(args):
    """Times the oracle, as it stands, on a bounded sample; returns (requests/s, cores, description)."""
    from oracle import oracle
    w, what = cpu_oracle_workload(args)
    cpu_oracle_time(w)                                          # load the library, touch the pages
    dt, _ = cpu_oracle_time(w)
    return w.n_requests / dt, oracle.num_threads(), what + ", score+drain %.2f s" % dt


KERNEL_NAMES = ("k_score_tiled", "k_score_small", "k_score_mma", "k_score_gemm<bf16>", "k_score_gemm<f32>")


def roofline_entry(w, n, kernel, score_ms, peaks, traffic):
    """Roofline object of the scoring kernel of workload ``w`` (n requests per launch, score_ms per launch)."""
    if kernel.startswith("k_score_gemm"):
        # the head is a dense contraction far above the HBM ridge: bound by the tensor pipe.  The kernel is short and
        # timed by its own events, so the burst figure of the measured bf16 peak applies; the fp32 flavour runs on the
        # tf32 unit (nominal ratio to bf16: 0.5) and needs three MMA passes for fp32 accuracy, but the algorithmic
        # flops (2 n D C) are what is counted.
        f32 = kernel.endswith("<f32>")
        flops = 2.0 * n * int(w.feat_dim) * int(w.n_classes)
        peak, peak_src = (float(peaks["bf16_tflops"]), "measured") if peaks else (1590.0, "fallback")
        if f32:
            peak, peak_src = peak * 0.5, peak_src + " bf16 x 0.5 (tf32)"
        achieved = flops / (score_ms * 1e-3) / 1e12 if score_ms > 0 else None
        return {"bound": "tensor", "kernel": kernel, "achieved": achieved, "peak": peak, "peak_source": peak_src,
                "unit": "TFLOP/s", "frac": achieved / peak if achieved else None, "traffic": traffic,
                "algorithmic_flops": flops, "mma_passes": 3 if f32 else 1,
                "algorithmic_bytes": algorithmic_bytes_per_request(w) * n, "kernel_ms": score_ms}
    bytes_per_launch = algorithmic_bytes_per_request(w) * n
    peak, peak_src = (float(peaks["hbm_gbs"]), "measured") if peaks else (6650.0, "fallback")
    achieved = bytes_per_launch / (score_ms * 1e-3) / 1e9 if score_ms > 0 else None
    return {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peak, "peak_source": peak_src,
            "unit": "GB/s", "frac": achieved / peak if achieved else None, "traffic": traffic,
            "algorithmic_bytes": bytes_per_launch, "kernel_ms": score_ms}


def side_workload(name, steps, peaks, device):
    """A short pass over another full-size configuration (score + drain, inputs resident), for the record beside the
    headline workload: step time, scoring-kernel roofline, scheduling time per round."""
    import torch
    from paper_2505_06641_b200 import api, runner, synth
    w = synth.make_workload(name)
    n = w.n_requests
    ses = runner.Session(w, device=device)
    api.sp_set_options(ses.ctx, trace_mode=bool(w.trace_mode), timing=True)
    ses.upload()
    ses.alloc_outputs(max(1, min(n, 1 << 16)))
    for _ in range(3):
        ses.score(); ses.schedule(n + 1)
    api.sp_check(ses.ctx)
    api.sp_get_stats(ses.ctx)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        ses.score(); ses.schedule(n + 1)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    api.sp_check(ses.ctx)
    st = api.sp_get_stats(ses.ctx)
    rounds = int(ses.n_done.sum().item())
    score_ms = st["score_kernel_ms"] / max(1, st["score_calls"])
    sched_ms = st["sched_kernel_ms"] / max(1, st["sched_calls"])
    kernel = KERNEL_NAMES[int(st["score_kernel"])]
    ses.close()
    return {"workload": name, "requests": n, "steps": steps, "ms_per_step": ms, "requests_per_s": n / (ms * 1e-3),
            "roofline": roofline_entry(w, n, kernel, score_ms, peaks, None), "sched_kernel_ms": sched_ms,
            "rounds_per_step": rounds, "us_per_round": sched_ms * 1e3 / max(1, rounds),
            "l2": "features %.2f GB per step" % (w.feats.nbytes / 1e9)}


class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "50"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.p.terminate()
        self.p.wait()
        self.f.flush(); self.f.seek(0)
        sm, smax, reasons = [], [], set()
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1])); smax.append(float(c[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.f.close(); os.unlink(self.f.name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def run_reference(args, rank):
    if rank != 0:
        return
    from oracle import oracle
    # the sample shrinks with the number of passes asked for, so that the whole run stays within a few minutes
    args.cpu_sample_instances = max(64, min(args.cpu_sample_instances, 40960 // max(1, args.steps + args.warmup)))
    w, what = cpu_oracle_workload(args)
    for _ in range(args.warmup):
        cpu_oracle_time(w)
    times = [cpu_oracle_time(w)[0] for _ in range(args.steps)]
    dt = float(np.mean(times))
    value = w.n_requests / dt
    cb = {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": what}
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(args), "sample": what}, "cpu_baseline": cb,
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def workload_name(args):
    names = {"C1": "tiny single instance (C1)", "C2": "medium instance (C2)", "C3": "large-class instance (C3)",
             "C4": "batched independent instances (C4)", "C5": "trace replay (C5)"}
    return names[args.workload]


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:     # before the first GPU call
        v, cores, what = cpu_oracle_sample(args)
        cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": what}

    import torch
    import torch.distributed as dist
    from paper_2505_06641_b200 import api, runner
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    w = make(args, rank)
    n = w.n_requests
    per_inst = int(np.max(np.bincount(np.asarray(w.instance), minlength=int(w.n_instances))))
    max_rounds = per_inst + 1
    cap = ROUND_CAP if int(w.n_instances) > 1 else max(1, min(per_inst, 1 << 16))
    ses = runner.Session(w, device=local)
    api.sp_set_options(ses.ctx, trace_mode=bool(w.trace_mode), timing=True)
    ses.upload()
    ses.alloc_outputs(cap)

    def step():
        ses.score()
        ses.schedule(max_rounds)

    for _ in range(max(args.warmup, 0)):
        step()
    api.sp_check(ses.ctx)
    api.sp_get_stats(ses.ctx)                                   # drop the warm-up timings
    launches0 = api.sp_get_stats(ses.ctx)["kernel_launches"]
    sampler = ClockSampler(local) if rank == 0 else None
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if sampler else None
    api.sp_check(ses.ctx)
    st = api.sp_get_stats(ses.ctx)
    launches = st["kernel_launches"] - launches0
    n_rounds = int(ses.n_done.sum().item())
    from paper_2505_06641_b200 import shard
    ms, (n_total, launches, n_rounds_total) = shard.reduce_step_stats(ms, [n, launches, n_rounds], "cuda")
    ms_per_step = ms / args.steps
    value = n_total / (ms_per_step * 1e-3)

    # ---- roofline of the dominant kernel (the scoring kernel), from CUDA events recorded around it
    score_ms = st["score_kernel_ms"] / max(1, st["score_calls"])
    sched_ms = st["sched_kernel_ms"] / max(1, st["sched_calls"])
    kernel = KERNEL_NAMES[int(st.get("score_kernel", 0))]
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peaks = json.load(open(peaks_path)) if os.path.exists(peaks_path) else None
    traffic = None
    tpath = os.path.join(ROOT, "profiles", "traffic.json")      # DRAM bytes per launch from the committed ncu capture
    if os.path.exists(tpath):
        tj = json.load(open(tpath)).get(args.workload)
        if tj and tj.get("kernel_version") == KERNEL_VERSION:
            traffic = tj["dram_bytes_per_request"] * n
    roofline = roofline_entry(w, n, kernel, score_ms, peaks, traffic)

    # ---- one scheduling round per call (launch, the round, synchronise): the latency a caller sees per decision
    ses.score()
    torch.cuda.synchronize()
    single = []
    for _ in range(min(21, max_rounds)):
        t0 = time.perf_counter()
        ses.schedule(1)
        torch.cuda.synchronize()
        single.append(time.perf_counter() - t0)
    us_single_round_call = float(np.median(single[1:] or single)) * 1e6
    api.sp_check(ses.ctx)

    # ---- end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    e2e = None
    if not args.no_e2e:
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory().numpy()
        hf = pin(w.feats.view(np.int16) if int(w.feat_dtype) == 1 else w.feats)
        ha, harr, hdl = pin(w.app.astype(np.int32)), pin(w.arrival_ns), pin(w.deadline_ns)
        hinst = pin(w.instance.astype(np.int32)) if int(w.n_instances) > 1 else None
        ht0, hl0 = pin(w.t0_ns), pin(np.full(int(w.n_instances), -1, dtype=np.int32))
        reqs = pin(np.zeros(n, dtype=api.REQ_DTYPE).view(np.uint8)).view(api.REQ_DTYPE)
        rounds = pin(np.zeros((int(w.n_instances), cap), dtype=api.ROUND_DTYPE).view(np.uint8)).view(api.ROUND_DTYPE)
        nd = pin(np.zeros(int(w.n_instances), dtype=np.int32))
        call = lambda: api.sp_run_host(ses.ctx, n, hf, ha, harr, hdl, hinst, ht0, hl0, max_rounds, reqs, rounds, cap, nd)
        call()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        e2e_steps = max(1, min(args.steps, 50))          # each step moves GBs over PCIe: a bounded number is enough
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            call()
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        dt, _ = shard.reduce_step_stats(dt, [], "cuda")
        h2d = hf.nbytes + ha.nbytes + harr.nbytes + hdl.nbytes + (hinst.nbytes if hinst is not None else 0) + ht0.nbytes + hl0.nbytes
        d2h = reqs.nbytes + rounds.nbytes + nd.nbytes
        e2e = {"value": n_total / (dt / e2e_steps), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(d2h), "ms_per_step": dt / e2e_steps * 1e3, "steps": e2e_steps}
    ses.close()
    del ses
    torch.cuda.empty_cache()

    # ---- the other two large configurations, a few steps each, for the record (single-GPU run of the default only)
    others = None
    if rank == 0 and world == 1 and args.workload == "C4" and args.instances is None and not args.no_side_workloads:
        others = [side_workload("C3", 3, peaks, local), side_workload("C5", 2, peaks, local)]

    if rank == 0:
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16 in / f32" if int(w.feat_dtype) == 1 else "f32", "data": "synthetic",
            "config": {"workload": workload_name(args), "instances_per_gpu": int(w.n_instances),
                       "requests_per_gpu": n, "apps": int(w.n_apps), "models_per_app": int(w.max_models),
                       "classes": int(w.n_classes), "feat_dim": int(w.feat_dim), "sharding": "instances over ranks",
                       "l2": "inputs larger than L2 (%.2f GB of features per step)" % (w.feats.nbytes / 1e9)},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu,
            "extra": {"score_kernel_ms": score_ms, "sched_kernel_ms": sched_ms, "rounds_per_step": n_rounds_total,
                      "us_per_round_amortised": sched_ms * 1e3 / max(1, n_rounds_total),
                      "us_single_round_call": us_single_round_call,
                      "exact_utility_rounds": st["exact_utility"], "exact_priority_rounds": st["exact_priority"],
                      "exact_rows": st["exact_rows"], "other_workloads": others},
        }
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


KERNEL_VERSION = 5     # bump when the scoring kernel changes: stale ncu traffic figures are then ignored


if __name__ == "__main__":
    main()
