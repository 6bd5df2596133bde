#!/usr/bin/env python
"""Benchmark of the DBA step on the serving-scale workload (B=256, k=20, V=64000, bf16, 120-step stream).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A step is one dba_step call: both kernels (row scan; candidates + allocation) over one batch of logits.  The logit stream is generated
once, untimed, by running the step in closed loop (every row depends on the hypothesis' last token), and
kept resident in HBM; the timed loop then replays it, resetting the beam whenever the stream wraps.
One JSON line is printed by rank 0.  With N > 1 every rank runs an independent replica (sentences do not
interact, the path has no collective); the value is the sum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "dba_steps_per_sec"
L2_BYTES = 126 * 2**20


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1200)
    ap.add_argument("--warmup", type=int, default=120)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="serving")
    ap.add_argument("--C", type=int, default=None, help="constraint count of the 'scaling' workload")
    ap.add_argument("--B", type=int, default=None, help="fewer sentences than the workload has (for profiling a small case)")
    ap.add_argument("--gbs-base", type=int, default=None,
                    help="grid-beam-search simulation of the paper's Section 5 on the 'scaling' workload: beam "
                         "b*(C+1) for this base beam b, bank adjustment off")
    ap.add_argument("--stream-steps", type=int, default=None, help="keep only the first steps of the stream resident")
    ap.add_argument("--e2e-steps", type=int, default=16)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--fused", action="store_true",
                    help="the step fused into the output projection (dba_step_fused): hidden states and embedding in, "
                         "logits never materialised; reports a tensor-core roofline")
    ap.add_argument("--D", type=int, default=1024, help="hidden size of the fused step")
    return ap.parse_args()


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def measured_tensor_peak():
    """Dense bf16 TFLOP/s of a cuBLAS GEMM loop under the power cap (the kernel is timed inside a long step)."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return float(json.load(open(p))["bf16_tflops_sustained"]), "measured, sustained"
    return 1400.0, "fallback, sustained"


def ncu_traffic(workload, open_rows_per_launch):
    """DRAM bytes (read + write) per row-scan launch, scaled from the committed ncu capture of a smaller case
    by the rows a launch processes (traffic grows in proportion: one pass per open row).  None when the
    kernel source has changed since the counters were taken."""
    import hashlib
    p = os.path.join(ROOT, "profiles", "row_scan_traffic.txt")
    src = os.path.join(ROOT, "paper_1804_06609_b200", "csrc", "row_scan_tma.cu")
    if not (os.path.exists(p) and os.path.exists(src)):
        return None
    digest = hashlib.sha256(open(src, "rb").read()).hexdigest()[:16]
    for line in open(p):
        f = line.split()
        if len(f) == 3 and f[0] == workload and f[1] == digest:
            return float(f[2]) * open_rows_per_launch
    return None


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.stop_flag, self.sm, self.reasons, self.max_mhz = index, False, [], set(), None

    def run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            names = {nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
                     nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
                     nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
                     nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap"}
            while not self.stop_flag:
                self.sm.append(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
                time.sleep(0.01)
        except Exception as e:  # NVML missing: report that no clocks were seen
            self.reasons.add(f"nvml_unavailable:{type(e).__name__}")

    def result(self):
        import statistics
        return {"sm_mhz": statistics.median(self.sm) if self.sm else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.sm)}


def workload_of(args):
    from synth_inputs import make_workload
    kw = {"B": args.B} if args.B else {}
    if args.gbs_base:                       # Section 5: every bank has its own b slots, so the beam grows with C
        kw["k"] = args.gbs_base * ((args.C if args.C is not None else 10) + 1)
    return make_workload(args.workload, C=args.C, **kw)


# ---------------------------------------------------------------------------------------------- oracle
def unit_of(wl):
    return f"steps/s (one step = {wl.R} hypotheses x {wl.V} {wl.dtype} logits per GPU)"


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def oracle_rate(wl, n_sent, steps, warmup=0, budget_s=None, threads=1):
    """Times the CPU oracle, as it stands, on the first n_sent sentences of the workload in closed loop: one
    thread, or (threads > 1) sentences stepped concurrently, one oracle instance per sentence, the arithmetic
    per sentence unchanged.  Returns (whole-batch steps/s equivalent, seconds timed, steps timed)."""
    from oracle import dba_oracle as O
    from synth_inputs import LogitStream
    sub = wl.subset(range(n_sent))
    gen = LogitStream(sub)
    orc = O.Batch(sub.k, sub.V, wl.steps, sub.constraints, threads=threads)
    t_spent, done, t_in = 0.0, 0, 0
    for i in range(warmup + steps):
        if t_in == wl.steps:
            orc = O.Batch(sub.k, sub.V, wl.steps, sub.constraints, threads=threads); t_in = 0
        b = orc.beam()
        x = gen.step_logits(t_in, b["token"], b["met_mask"])       # input generation is not timed
        t0 = time.perf_counter()
        orc.step(x)
        dt = time.perf_counter() - t0
        t_in += 1
        if i >= warmup:
            t_spent += dt; done += 1
            if budget_s is not None and t_spent > budget_s:
                break
    per_sentence_step = t_spent / (done * n_sent)
    return 1.0 / (per_sentence_step * wl.B), t_spent, done


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = workload_of(args)
    total = args.steps + args.warmup
    per_sentence = 0.003 * wl.k * wl.V / 64000 * (wl.k / 20) + 0.002     # rough seconds per sentence-step
    n_sent = max(1, min(wl.B, 16, int(150.0 / (total * per_sentence))))
    value, secs, done = oracle_rate(wl, n_sent, args.steps, args.warmup)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": unit_of(wl), "n_gpus": args.gpus,
            "extrapolated": n_sent < wl.B,      # a step of the oracle was timed on n_sent sentences and scaled to wl.B
            "steps": done, "warmup": args.warmup, "ms_per_step": 1e3 / value, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "B": wl.B, "k": wl.k, "V": wl.V, "logits": wl.dtype},
            "cpu_baseline": {"value": value, "unit": "steps/s", "cores": 1, "host_cores": host_cores(), "kind": "oracle",
                             "sample": f"{n_sent} of {wl.B} sentences per step, {done} steps of the stream after "
                                       f"{args.warmup} untimed ones, scaled by {wl.B}/{n_sent}"},
            "e2e": {"value": value, "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------- replicas
def replica_workload(wl, rank):
    """Rank `rank`'s replica of the workload: the same shapes and constraints recipe, its own sentence ids (and
    hence its own logit streams).  Sentences never interact, so ranks exchange nothing on the data path."""
    import numpy as np
    wl.sent_ids = wl.sent_ids + np.int64(rank * wl.B)
    return wl


def job_rate(units_per_rank, seconds_local, world, device):
    """Whole-job rate: the units all ranks processed over the slowest rank's time (max over ranks)."""
    if world > 1:
        import torch
        import torch.distributed as dist
        t = torch.tensor([seconds_local], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        seconds_local = float(t)
    return world * units_per_rank / seconds_local, seconds_local


# ---------------------------------------------------------------------------------------------- ours
def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_1804_06609_b200 as pkg
    from synth_inputs.gpu import GpuLogitStream

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    pkg.lib()

    wl = workload_of(args)
    if world > 1:                                   # replicas: every rank gets its own sentences
        wl = replica_workload(wl, rank)
    esize = 2 if wl.dtype == "bf16" else 4
    step_bytes = wl.R * wl.V * esize
    free, _ = torch.cuda.mem_get_info(dev)
    T = int(max(1, min(wl.steps, (free * 0.6) // step_bytes, args.stream_steps or wl.steps)))
    # rotate enough distinct step buffers that consecutive steps never find their input in L2
    gen = GpuLogitStream(wl, dev)
    cfg_flags = pkg.FLAG_ADJUST_OFF if args.gbs_base else 0
    st = pkg.DbaStepper(wl.B, wl.k, wl.V, wl.steps, constraints=wl.constraints,
                        dtype=pkg.BF16 if wl.dtype == "bf16" else pkg.F32, device=dev, flags=cfg_flags)
    logits = torch.empty(T, wl.R, wl.V, dtype=gen.tdtype, device=dev)

    # --- untimed: generate the stream in closed loop, count the rows that are open at each step -------
    tok = torch.zeros(wl.R, dtype=torch.int32, device=dev); tok[::wl.k] = 1
    mask = torch.zeros(wl.R, dtype=torch.int64, device=dev)
    open_rows = []
    for t in range(T):
        open_rows.append(wl.B if t == 0 else int(((out["score"] > float("-inf")) & (out["token"] != 2)).sum()))
        gen.step_logits(t, tok, mask, out=logits[t])
        out = st.step(logits[t])
        tok, mask = out["token"], out["met_mask"]
    tokens, length, score, flags = st.finalize()
    completed = int((flags & 1).sum())

    def replay(n, start=0):
        for i in range(start, start + n):
            t = i % T
            if t == 0:
                st.reset()
            st.step(logits[t])

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    # --- timed: K steps, device clock, max over ranks ---------------------------------------------------
    replay(args.warmup)
    launches0 = st.launch_count()
    sampler = ClockSampler(local); sampler.start()
    time.sleep(0.05)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    replay(args.steps, start=args.warmup)
    e1.record()
    barrier()
    sampler.stop_flag = True; sampler.join()
    ms = e0.elapsed_time(e1)
    launches = st.launch_count() - launches0
    value, secs = job_rate(args.steps, ms / 1e3, world, dev)
    ms = secs * 1e3

    # --- per-kernel time of the same replay (events inside the library, on its stream) -----------------
    st.timing_enable(True)
    kt, ksteps, kbytes = [0.0, 0.0, 0.0], 0, 0
    pos = args.warmup + args.steps
    remaining = args.steps
    while remaining > 0:
        n = min(remaining, 2048)
        replay(n, start=pos)
        part, cnt = st.timing_read()
        kt = [a + b for a, b in zip(kt, part)]; ksteps += cnt
        kbytes += sum(open_rows[i % T] for i in range(pos, pos + n)) * wl.V * esize
        pos += n; remaining -= n
    st.timing_enable(False)
    peak, peak_kind = measured_peak()
    scan_ms = kt[0] / ksteps
    achieved = kbytes / ksteps / (scan_ms / 1e3) / 1e9
    traffic = ncu_traffic(wl.name, kbytes / ksteps / (wl.V * esize))

    # --- end to end: host logits in pinned memory, outputs read back, through dba_step_host ------------
    Th = min(T, 8)
    ste = pkg.DbaStepper(wl.B, wl.k, wl.V, wl.steps, constraints=wl.constraints,
                         dtype=pkg.BF16 if wl.dtype == "bf16" else pkg.F32, device=dev,
                         flags=pkg.FLAG_HOST_STAGING | cfg_flags)
    host = torch.empty(Th, wl.R, wl.V, dtype=gen.tdtype, pin_memory=True)
    host.copy_(logits[:Th])
    host_out = ste.new_outputs(host=True)
    d2h = sum(v.numel() * v.element_size() for v in host_out.values())

    def replay_host(n):
        for i in range(n):
            if i % Th == 0:
                ste.reset()
            ste.step_host(host[i % Th], host_out)

    replay_host(3)
    barrier()
    t0 = time.perf_counter()
    replay_host(args.e2e_steps)
    torch.cuda.synchronize(dev)
    e2e_s = time.perf_counter() - t0
    e2e_value, e2e_s = job_rate(args.e2e_steps, e2e_s, world, dev)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    cpu = None
    if not args.no_cpu_baseline and world == 1:
        n_sent = min(8, wl.B)
        v, secs, done = oracle_rate(wl, n_sent, 24, warmup=2, budget_s=15.0)
        cores = host_cores()
        n_par = min(wl.B, 2 * cores)
        va, secs_a, done_a = oracle_rate(wl, n_par, 12, warmup=2, budget_s=10.0, threads=cores)
        cpu = {"value": v, "unit": "steps/s", "cores": 1, "host_cores": cores, "kind": "oracle",
               "sample": f"first {n_sent} of {wl.B} sentences, steps 2-{done + 1} of the stream in closed loop (every beam "
                         f"slot is live from step 1 on), {secs:.1f} s of oracle time, scaled by {wl.B}/{n_sent}",
               "all_cores": {"value": va, "unit": "steps/s", "cores": cores,
                             "sample": f"first {n_par} of {wl.B} sentences stepped concurrently by {cores} threads (one "
                                       f"single-threaded oracle instance per sentence), steps 2-{done_a + 1}, "
                                       f"{secs_a:.1f} s wall, scaled by {wl.B}/{n_par}"}}
    unit = unit_of(wl)
    line = {
        "metric": METRIC, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": wl.name, "B": wl.B, "k": wl.k, "V": wl.V, "logits": wl.dtype,
                   "constraint_tokens_per_sentence": sorted({sum(len(p) for p in c) for c in wl.constraints}),
                   "stream_steps": T, "open_rows_mean": sum(open_rows) / T, "rows": wl.R,
                   "completed_sentences": completed,
                   "l2": f"inputs larger than L2: {step_bytes >> 20} MiB of logits per step, {T} step buffers"
                         if step_bytes > L2_BYTES else f"{T} rotating step buffers, {T * step_bytes >> 20} MiB in all",
                   "parallelism": "replicas" if world > 1 else "single GPU",
                   **({"gbs_simulation": {"base_beam": args.gbs_base, "beam": wl.k, "bank_adjustment": "off"}} if args.gbs_base else {})},
        "hyp_steps_per_sec": value * wl.R,
        "kernel_ms": {"row_scan": scan_ms, "candidates_and_allocation": kt[1] / ksteps},
        "roofline": {"bound": "hbm", "kernel": "row_scan", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "frac_of_8TBs_nominal": achieved / 8000.0,
                     "algorithmic_bytes_per_launch": kbytes / ksteps, "traffic": traffic},
        "e2e": {"value": e2e_value, "unit": "steps/s", "h2d_bytes_per_step": step_bytes, "d2h_bytes_per_step": d2h,
                "steps": args.e2e_steps},
        "gpu_launches": launches,
        "clocks": sampler.result(),
        "cpu_baseline": cpu,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_fused(args):
    """dba_step_fused on the workload's shape: synthetic hidden states [R, D] and output embedding [V, D] (bf16,
    Zipf-shaped word offsets in one embedding column, an end-token column that rises along the stream), one GPU."""
    import torch
    import paper_1804_06609_b200 as pkg
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    wl = workload_of(args)
    D, R, V = args.D, wl.R, wl.V
    g = torch.Generator(device=dev); g.manual_seed(wl.seed)
    e = torch.randn(V, D, device=dev, generator=g) / D ** 0.5
    e[:, 0] = -1.1 * torch.log(torch.randperm(V, device=dev, generator=g).float() + 1.0)
    e[:, 1] = 0.0; e[2, 1] = 1.0
    for c in wl.constraints:
        for ph in c:
            e[ph, 0] = 1.0                     # constraint tokens are likely words: the constraints get met
    embed = e.to(torch.bfloat16)
    T = min(wl.steps, 32)
    hidden = torch.randn(T, R, D, device=dev, generator=g)
    hidden[:, :, 0] = 1.0
    hidden[:, :, 1] = torch.linspace(-8.0, 10.0, T, device=dev)[:, None]
    hidden = hidden.to(torch.bfloat16)
    st = pkg.DbaStepper(wl.B, wl.k, V, wl.steps, constraints=wl.constraints, dtype=pkg.F32, device=dev,
                        flags=pkg.FLAG_FUSED_PROJECTION)

    def replay(n, start=0):
        for i in range(start, start + n):
            if i % T == 0:
                st.reset()
            st.step_fused(hidden[i % T], embed)

    replay(args.warmup)
    launches0 = st.launch_count()
    sampler = ClockSampler(0); sampler.start()
    time.sleep(0.05)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(dev)
    e0.record()
    replay(args.steps, start=args.warmup)
    e1.record()
    torch.cuda.synchronize(dev)
    sampler.stop_flag = True; sampler.join()
    ms = e0.elapsed_time(e1)
    launches = st.launch_count() - launches0
    st.timing_enable(True)
    replay(args.steps, start=args.warmup + args.steps)
    kt, ksteps = st.timing_read()
    st.timing_enable(False)
    tokens, length, score, flags = st.finalize()
    # for comparison, the same work unfused: a library GEMM that writes the logits (bf16), then the step on them
    st2 = pkg.DbaStepper(wl.B, wl.k, V, wl.steps, constraints=wl.constraints, dtype=pkg.BF16, device=dev)
    logits = torch.empty(R, V, dtype=torch.bfloat16, device=dev)
    embed_t = embed.t()

    def replay_unfused(n, start=0):
        for i in range(start, start + n):
            if i % T == 0:
                st2.reset()
            torch.matmul(hidden[i % T], embed_t, out=logits)
            st2.step(logits)

    replay_unfused(args.warmup)
    torch.cuda.synchronize(dev)
    u0, u1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    u0.record()
    replay_unfused(args.steps, start=args.warmup)
    u1.record()
    torch.cuda.synchronize(dev)
    unfused_ms = u0.elapsed_time(u1) / args.steps
    proj_ms = kt[0] / ksteps
    flops = 2.0 * R * V * D
    peak, peak_kind = measured_tensor_peak()
    achieved = flops / (proj_ms / 1e3) / 1e12
    line = {
        "metric": METRIC, "value": args.steps / (ms / 1e3),
        "unit": f"steps/s (one step = {R} hypotheses x {V} words, hidden size {D}, projection fused into the step)",
        "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16 x bf16 -> f32", "data": "synthetic",
        "config": {"workload": wl.name + "-fused", "B": wl.B, "k": wl.k, "V": V, "D": D, "rows": R, "stream_steps": T,
                   "l2": f"operands per step: {R * D * 2 >> 20} MiB of hidden states ({T} rotating buffers) and "
                         f"{V * D * 2 >> 20} MiB of embedding, which is larger than L2",
                   "parallelism": "single GPU", "completed_sentences": int((flags & 1).sum())},
        "kernel_ms": {"projection_scan_and_merge": proj_ms, "constraint_logits_and_candidates": kt[1] / ksteps},
        "unfused_for_comparison": {"ms_per_step": unfused_ms,
                                   "what": "torch.matmul (library GEMM, bf16 logits written to HBM) followed by dba_step on them"},
        "roofline": {"bound": "tensor", "kernel": "project_scan", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                     "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "flops_per_launch": flops, "traffic": None},
        "gpu_launches": launches, "clocks": sampler.result(), "cpu_baseline": None,
        "e2e": None,
    }
    print(json.dumps(line), flush=True)


def main():
    args = parse()
    if args.impl == "reference":
        run_reference(args)
    elif args.fused:
        run_fused(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
