#!/usr/bin/env python
"""Benchmark of the delta-rule linear-attention prefill library on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One "step" = one pass of the whole hot path (plan + every compute kernel of ha_la_prefill)
over one batch of the synthetic workload.  Prints ONE JSON line (rank 0).

* value        : tokens/s, inputs resident in HBM, device-timed (CUDA events, max over ranks).
                 Each step uses a different one of R resident input/output sets whose total
                 size exceeds 2x the L2 cache, so no step finds its inputs in L2.
* e2e          : the same metric through the public API with HOST buffers: pinned host -> device
                 copies of every input and device -> host copies of o and hT inside the timed region.
* roofline     : for the dominant kernel, timed live with CUDA events between kernels
                 (ha_la_prefill_timed): the path's algorithmic bytes over that kernel's time over the
                 measured HBM rate; `path` gives the whole-call figure (slower of FLOPs at the measured
                 bf16 peak and bytes at the measured HBM rate, over the time of the whole call).
* parity       : o and hT of the last timed step against the fp64 oracle (all heads), same run; a result
                 outside the stated tolerance makes the run fail.
* cpu_baseline : the fp64 oracle, as it stands, on this machine's host cores, on a bounded sample.
* --impl reference : times only the oracle (rank 0) and prints its line with "impl": "reference".

With N > 1 (torchrun) every rank runs its own independent batch (the path shards over
sequences and heads with no exchange): weak scaling, no collective on the data path.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2609_32114_b200 import synth  # noqa: E402

L2_BYTES = 126 * 1024 * 1024
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
METRIC = "LA-layer prefill tokens/s"


def load_traffic():
    """DRAM bytes per launch of each profiled kernel (profiles/traffic.json, written from the ncu summaries by
    `python -m paper_2609_32114_b200.ncu_summary traffic`)."""
    p = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(p):
        return {}
    with open(p) as f:
        return json.load(f)


def ncu_traffic(workload: str, kernel: str):
    e = load_traffic().get(workload, {}).get(kernel)
    return None if e is None else e["dram_read"] + e["dram_write"]


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
    return dict(FALLBACK_PEAKS, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx = float(r[1])
            except (ValueError, IndexError):
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def oracle_time(inp, budget_heads=None):
    """Times the oracle on (a sample of) the workload.  Returns (seconds, tokens processed per V-head set,
    threads, description)."""
    import oracle

    w = inp["workload"]
    N = inp["N"]
    pairs = None
    desc = f"all {N} sequences x {w.hv} V-heads, every token"
    if budget_heads is not None and budget_heads < N * w.hv:
        allp = [(n, j) for n in range(N) for j in range(w.hv)]
        step = max(1, len(allp) // budget_heads)
        pairs = allp[::step][:budget_heads]
        desc = f"{len(pairs)} of {N * w.hv} (sequence, V-head) pairs, every token of each"
    t0 = time.perf_counter()
    _, _, threads = oracle.recurrent(inp["q"], inp["k"], inp["v"], inp["g"], inp["beta"], variant=w.variant,
                                     h0=inp["h0"], cu_seqlens=inp["cu_seqlens"], pairs=pairs)
    dt = time.perf_counter() - t0
    if pairs is None:
        tok_heads = inp["T"] * w.hv
    else:
        cu = inp["cu_seqlens"]
        tok_heads = sum(int(cu[n + 1] - cu[n]) for n, _ in pairs)
    # tokens/s of the LAYER: token-heads per second divided by heads per token
    return dt, tok_heads / w.hv, threads, desc


def cpu_baseline(inp):
    w = inp["workload"]
    # aim at 10-30 s: the recurrence costs about 6 dk dv flops per token-head in fp64
    work = inp["T"] * w.hv * 6.0 * w.dk * w.dv
    cores = os.cpu_count() or 1
    est = work / (cores * 1.0e9)
    heads = None
    if est > 25:
        heads = max(cores, int(inp["N"] * w.hv * 20 / est))
    # repeat until the sample amounts to roughly 10-30 s of CPU work (cores x wall)
    total, reps, tokens, threads, desc = 0.0, 0, 0.0, 1, ""
    while reps < 50:
        dt, tokens, threads, desc = oracle_time(inp, heads)
        total += dt
        reps += 1
        if total * threads >= 12.0:
            break
    return {"value": tokens * reps / total, "unit": "tokens/s", "cores": threads, "kind": "oracle",
            "sample": f"{desc}; {reps} repetition(s), {total:.2f} s wall in total"}


def run_reference(args, inp, rank):
    """The reference arm of this tier is the oracle itself, timed on the host cores."""
    if rank != 0:
        return
    w = inp["workload"]
    times = []
    tokens = threads = None
    desc = ""
    work = inp["T"] * w.hv * 6.0 * w.dk * w.dv
    cores = os.cpu_count() or 1
    est = work / (cores * 1.0e9)
    budget = 60.0 / max(1, args.steps + args.warmup)          # keep the whole run within a few minutes
    heads = None if est <= budget else max(cores, int(inp["N"] * w.hv * budget / est))
    for i in range(args.warmup + args.steps):
        dt, tokens, threads, desc = oracle_time(inp, heads)
        if i >= args.warmup:
            times.append(dt)
    ms = 1e3 * float(np.mean(times))
    val = tokens / (ms / 1e3)
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "tokens_per_step": tokens, "sample": desc},
            "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def rank_seed(rank: int) -> int:
    """Every rank draws its own batch of the same workload (weak scaling over independent batches)."""
    return synth.BASE_SEED + 1000 * rank


def max_over_ranks(dist, ms: float, device) -> float:
    """Device-timed milliseconds, maximum over all ranks (the job is as slow as its slowest rank)."""
    if dist is None:
        return ms
    import torch

    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(world: int, tokens_per_rank: int, ms_per_step: float) -> float:
    """Whole-job tokens/s: all ranks' tokens over the slowest rank's step time."""
    return world * tokens_per_rank / (ms_per_step / 1e3)


# ---- the decoding step (one new token per sequence on the prefill's state layout): an extra measured row, not
# the headline metric.  Batch of sequences x heads of the headline layer; the fp32 states (268 MB) exceed L2.
DECODE_WORKLOADS = {"gdn_decode_b256": ("gdn", 256, 16, 16, 128), "kda_decode_b256": ("kda", 256, 16, 16, 128)}


def decode_bench(args, rank, local_rank, world):
    variant, N, hk, hv, d = DECODE_WORKLOADS[args.workload]
    base = synth.WORKLOADS["gdn_varlen" if variant == "gdn" else "kda_8k"]
    w = synth.shrink(base, seq_lens=[1] * N, hk=hk, hv=hv, dk=d, dv=d, dtype="bf16", h0_std=0.5, varlen=True)
    inp = synth.make_inputs(w, seed=rank_seed(rank))
    # bytes one step must move: state in and out, q k v g beta in, o out
    state_bytes = N * hv * d * d * 4
    io_bytes = N * (2 * hk * d * 2 + 2 * hv * d * 2 + hv * 4 * (1 + (d if variant == "kda" else 1)))
    alg_bytes = 2 * state_bytes + io_bytes
    alg_flops = N * hv * 6.0 * d * d
    metric = "LA-layer decode tokens/s"

    def oracle_run():
        import oracle
        t0 = time.perf_counter()
        _, _, threads = oracle.recurrent(inp["q"], inp["k"], inp["v"], inp["g"], inp["beta"], variant=variant,
                                         h0=inp["h0"], cu_seqlens=inp["cu_seqlens"])
        return time.perf_counter() - t0, threads

    if args.impl == "reference":
        if rank != 0:
            return
        for _ in range(max(args.warmup, 1)):
            oracle_run()
        ts = [oracle_run() for _ in range(args.steps)]
        sec = float(np.mean([t for t, _ in ts]))
        val = N / sec
        cpu = {"value": val, "unit": "tokens/s", "cores": ts[0][1], "kind": "oracle",
               "sample": f"all {N} sequences x {hv} V-heads, one token each"}
        print(json.dumps({"impl": "reference", "metric": metric, "value": val, "unit": "tokens/s", "n_gpus": world,
                          "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
                          "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
                          "data": "synthetic", "config": {"workload": args.workload}, "cpu_baseline": cpu,
                          "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0,
                                  "d2h_bytes_per_step": 0}}), flush=True)
        return

    import torch
    import paper_2609_32114_b200 as ha

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path (use --impl reference for the oracle)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)
    t = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dev).to(dt).contiguous()
    bf, f32 = torch.bfloat16, torch.float32
    q, k, v = t(inp["q"], bf), t(inp["k"], bf), t(inp["v"], bf)
    g, beta, state = t(inp["g"], f32), t(inp["beta"], f32), t(inp["h0"], f32)
    dargs, keep = ha.prepare_decode_args(q, k, v, g, beta, state, variant=variant)
    stream = torch.cuda.current_stream(dev)
    sptr = stream.cuda_stream

    def step():
        rc = ha.ha_la_decode_raw(dargs, sptr)
        if rc != 0:
            raise ha.HaLaError(rc, "ha_la_decode")

    def barrier():
        torch.cuda.synchronize(dev)
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize(dev)

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    t_wall = time.perf_counter()
    for i in range(args.steps):
        evs[i][0].record(stream)
        step()
        evs[i][1].record(stream)
    barrier()
    t_wall = time.perf_counter() - t_wall
    total_ms = max_over_ranks(dist, float(np.sum([a.elapsed_time(b) for a, b in evs])), dev)
    ms_per_step = total_ms / args.steps
    t_load = time.perf_counter()
    while len(sampler.rows) < 4 and time.perf_counter() - t_load < 2.0:
        for _ in range(64):
            step()
        barrier()
    clocks = sampler.stop()
    clocks["window"] = f"timed region and {time.perf_counter() - t_load:.2f} s of the same steps"

    # end to end: the state stays on the device (that is the point of a decoder), the token's inputs come from
    # pinned host memory and its outputs go back, every step
    names = ("q", "k", "v", "g", "beta")
    host = {n_: keep[n_].cpu().pin_memory() for n_ in names}
    o_host = torch.empty_like(keep["o"], device="cpu").pin_memory()
    h2d = sum(host[n_].numel() * host[n_].element_size() for n_ in names)
    d2h = o_host.numel() * o_host.element_size()

    def e2e_step():
        for n_ in names:
            keep[n_].copy_(host[n_], non_blocking=True)
        step()
        o_host.copy_(keep["o"], non_blocking=True)

    for _ in range(2):
        e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        e2e_step()
    e1.record(stream)
    barrier()
    e2e_ms = max_over_ranks(dist, e0.elapsed_time(e1), dev)
    peaks = load_peaks()
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        oracle_run()
        reps, tot, thr = 0, 0.0, 0
        while tot * max(thr, 1) < 12.0 and reps < 200:
            sec, thr = oracle_run()
            tot += sec
            reps += 1
        cpu = {"value": N * reps / tot, "unit": "tokens/s", "cores": thr, "kind": "oracle",
               "sample": f"all {N} sequences x {hv} V-heads, one token each; {reps} repetition(s), {tot:.2f} s wall"}
    if rank == 0:
        sec = ms_per_step / 1e3
        achieved = alg_bytes / sec / 1e9
        roofline = {"bound": "hbm", "kernel": "decode_kernel", "achieved": achieved, "peak": peaks["hbm_gbs"],
                    "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                    "traffic": ncu_traffic(args.workload, "decode"), "kernel_alg_bytes": alg_bytes,
                    "peak_source": peaks["source"], "kernel_ms": {"decode_kernel": ms_per_step},
                    "path": {"bound": "hbm", "roofline_us": 1e6 * alg_bytes / (peaks["hbm_gbs"] * 1e9),
                             "measured_us": 1e3 * ms_per_step, "frac": achieved / peaks["hbm_gbs"],
                             "achieved_gbs": achieved, "achieved_tflops": alg_flops / sec / 1e12,
                             "alg_bytes": alg_bytes, "alg_flops": alg_flops}}
        print(json.dumps({
            "metric": metric, "value": job_throughput(world, N, ms_per_step), "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload, "variant": variant, "sequences": N, "qk_heads": hk, "v_heads": hv,
                       "d_k": d, "d_v": d, "state_bytes": state_bytes,
                       "l2": "the states (read and rewritten in place every step) exceed L2",
                       "parallelism": "replicas (independent batch per GPU, no collective)" if world > 1 else "1 GPU"},
            "clocks": clocks,
            "e2e": {"value": job_throughput(world, N, e2e_ms / args.steps), "unit": "tokens/s",
                    "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                    "mode": "states resident on the device; the token's inputs in and outputs out every step"},
            "gpu_launches": args.steps, "roofline": roofline, "cpu_baseline": cpu,
            "wall_s_timed_region": t_wall}), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def measure(ha, helpers, w, inp, steps, warmup, dev, local_rank, dist, peaks, world, sample_clocks=True):
    """Device-timed steps of ha_la_prefill on workload `w`: `steps` timed calls after max(warmup, 3) untimed ones,
    between CUDA events on the launching stream, every step on a different resident input/output set."""
    import torch

    T, N = inp["T"], inp["N"]
    alg_bytes = synth.algorithmic_bytes(w, T, N)
    alg_flops = synth.algorithmic_flops(w, T)
    # R resident buffer sets, total > 2 x L2, visited round-robin
    base = helpers.to_device(inp, dev)
    R = max(2, int(np.ceil(2.2 * L2_BYTES / alg_bytes)) + 1)
    R = min(R, 8)
    sets = []
    shared_ws = None                                     # the workspace is the caller's scratch: one for all sets
    for r in range(R):
        d = base if r == 0 else {k: (v.clone() if hasattr(v, "clone") else v) for k, v in base.items()}
        a, keep = ha.prepare_args(d["q"], d["k"], d["v"], d["g"], d["beta"], variant=w.variant, h0=d["h0"],
                                  cu_seqlens=d["cu_seqlens"], max_seqlen=d["max_seqlen"], workspace=shared_ws)
        shared_ws = keep["workspace"]
        sets.append((a, keep))
    flush = None
    if R * alg_bytes < 2 * L2_BYTES:
        flush = torch.empty(3 * L2_BYTES, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream(dev)
    sptr = stream.cuda_stream

    def step(i):
        rc = ha.ha_la_prefill_raw(sets[i % R][0], sptr)
        if rc != 0:
            raise ha.HaLaError(rc, "ha_la_prefill")

    def barrier():
        torch.cuda.synchronize(dev)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def check_status(when):
        for a, keep in sets:
            st = int(keep["status_word"].item())
            if st != 0:
                raise SystemExit(f"device status word = {st} ({ha.status_string(st)}) {when}")

    for i in range(max(warmup, 3)):
        step(i)
    barrier()
    check_status("during warm-up")

    # ---- timed region: exactly `steps` steps back to back on the launching stream between one pair of CUDA events
    # (every step works on another resident set, together larger than twice the L2).  Workloads so small that L2 has
    # to be flushed between steps are timed step by step instead, the flush outside the events.
    sampler = ClockSampler(local_rank) if sample_clocks else None
    if sampler:
        sampler.start()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    e_all = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
    barrier()
    t_wall = time.perf_counter()
    if flush is None:
        e_all[0].record(stream)
        for i in range(steps):
            step(i)
        e_all[1].record(stream)
    else:
        for i in range(steps):
            flush.fill_(i & 0xff)
            evs[i][0].record(stream)
            step(i)
            evs[i][1].record(stream)
    barrier()
    t_wall = time.perf_counter() - t_wall
    check_status("during the timed steps")
    last = sets[(steps - 1) % R][1]
    last_out = {"o": last["o"].clone(), "hT": last["hT"].clone()}     # what the last timed step wrote
    if flush is None:
        total_local = e_all[0].elapsed_time(e_all[1])
        # the spread of single steps: the same steps once more, one event pair each (an event between two calls costs
        # a couple of microseconds and keeps the next call's set-up from running under this call's tail, so these
        # are a little longer than the steps of the timed region)
        for i in range(steps):
            evs[i][0].record(stream)
            step(i)
            evs[i][1].record(stream)
        barrier()
        check_status("during the single-step timing")
        step_ms = [a.elapsed_time(b) for a, b in evs]
    else:
        step_ms = [a.elapsed_time(b) for a, b in evs]
        total_local = float(np.sum(step_ms))
    total_ms = max_over_ranks(dist, float(total_local), dev)
    ms_per_step = total_ms / steps
    value = job_throughput(world, T, ms_per_step)

    # ---- per-kernel device time (events between kernels), averaged over a few cold-L2 steps
    kt = {}
    for i in range(min(steps, 8)):
        if flush is not None:
            flush.fill_(i)
        for name, ms in ha.ha_la_prefill_timed(sets[(i + 1) % R][0], sptr):
            kt.setdefault(name, []).append(ms)
    clocks = None
    if sampler:
        # nvidia-smi samples every ~100 ms: if the timed region was shorter than a few samples, keep the same
        # steps running (untimed) until some have been taken under this load
        t_load = time.perf_counter()
        i = 0
        while len(sampler.rows) < 4 and time.perf_counter() - t_load < 2.0:
            for _ in range(16):
                step(i)
                i += 1
            barrier()
        clocks = sampler.stop()
        clocks["window"] = (f"timed region ({t_wall * 1e3:.0f} ms), per-kernel timing and "
                            f"{time.perf_counter() - t_load:.2f} s of the same steps")
    kernel_ms = {k: float(np.mean(v)) for k, v in kt.items()}
    dom = max(kernel_ms, key=kernel_ms.get)
    # per-kernel attribution: the algorithmic bytes each kernel is the one to touch (the prep kernel reads q, k, v,
    # g, beta; the chain kernel reads h0 and writes o and hT; the operand images between them are not algorithmic)
    e = 2 if w.dtype == "bf16" else 4
    in_bytes = T * (2 * w.hk * w.dk * e + w.hv * w.dv * e + w.hv * 4 * (1 + (w.dk if w.variant == "kda" else 1)))
    kernel_alg_bytes = {"simt_prefill": alg_bytes, "tc_prep": in_bytes, "tc_chain": alg_bytes - in_bytes, "plan": 0.0}
    dom_s = kernel_ms[dom] / 1e3
    achieved = alg_bytes / dom_s / 1e9                   # the path's bytes over the dominant kernel's time
    t_hbm = alg_bytes / (peaks["hbm_gbs"] * 1e9)
    t_flop = alg_flops / (peaks["bf16_tflops"] * 1e12)
    path_s = ms_per_step / 1e3
    nv_plan, conc_plan = ha.ha_la_prefill_launch_plan(sets[0][0])
    launch_mode = ("fp32 CUDA-core kernel" if nv_plan == 0 else
                   f"{nv_plan}-channel slices, prep and chain kernels " + ("side by side" if conc_plan else "back to back"))
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "traffic": ncu_traffic(w.name, dom),
                "alg_bytes": alg_bytes, "peak_source": peaks["source"],
                "kernel_ms": kernel_ms,      # each kernel alone (sequential launches with events in between)
                "per_kernel": {k: {"alg_bytes_it_touches": kernel_alg_bytes.get(k, 0.0),
                                   "achieved_gbs": kernel_alg_bytes.get(k, 0.0) / (v / 1e3) / 1e9 if v > 0 else None,
                                   "traffic": ncu_traffic(w.name, k)} for k, v in kernel_ms.items()},
                # what the timed steps used (kernel_ms is always back to back, and then with the planner's
                # back-to-back slice width, which may differ)
                "launch_mode": launch_mode,
                "path": {"bound": "hbm" if t_hbm >= t_flop else "tensor", "roofline_us": 1e6 * max(t_hbm, t_flop),
                         "measured_us": 1e6 * path_s, "frac": max(t_hbm, t_flop) / path_s,
                         "achieved_gbs": alg_bytes / path_s / 1e9, "achieved_tflops": alg_flops / path_s / 1e12,
                         "alg_bytes": alg_bytes, "alg_flops": alg_flops}}
    return dict(sets=sets, R=R, base=base, stream=stream, sptr=sptr, ms_per_step=ms_per_step, value=value,
                ms_median=float(np.median(step_ms)), ms_min=float(np.min(step_ms)), ms_max=float(np.max(step_ms)),
                roofline=roofline, clocks=clocks, alg_bytes=alg_bytes, wall_s=t_wall, check_status=check_status,
                last_out=last_out, flushed=flush is not None,
                launches_per_step=ha.ha_la_prefill_num_launches(sets[0][0]), path=ha.ha_la_prefill_path(sets[0][0]))


def profile_range(ha, helpers, w, inp, warmup, dev):
    """One call of ha_la_prefill between cudaProfilerStart and cudaProfilerStop, after `warmup` untimed calls."""
    import torch

    d = helpers.to_device(inp, dev)
    a, keep = ha.prepare_args(d["q"], d["k"], d["v"], d["g"], d["beta"], variant=w.variant, h0=d["h0"],
                              cu_seqlens=d["cu_seqlens"], max_seqlen=d["max_seqlen"])
    sptr = torch.cuda.current_stream(dev).cuda_stream
    for _ in range(warmup):
        ha.ha_la_prefill_raw(a, sptr)
    flush = torch.empty(3 * L2_BYTES, dtype=torch.uint8, device=dev)
    flush.fill_(1)                                       # the profiled call starts from a cold L2
    torch.cuda.synchronize(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.profiler.start()
    e0.record()
    rc = ha.ha_la_prefill_raw(a, sptr)
    e1.record()
    torch.cuda.synchronize(dev)
    torch.cuda.profiler.stop()
    nv, conc = ha.ha_la_prefill_launch_plan(a)
    print(json.dumps({"profile_range": w.name, "tokens": inp["T"], "rc": rc, "status": int(keep["status_word"].item()),
                      "ms": e0.elapsed_time(e1), "slice_width": nv, "side_by_side": bool(conc),
                      "alg_bytes": synth.algorithmic_bytes(w, inp["T"], inp["N"])}), flush=True)


def parity_of(helpers, inp, out):
    """o and hT in `out` (device tensors a step wrote) against the oracle on every (sequence, V-head) pair."""
    w = inp["workload"]
    o = out["o"].float().cpu().numpy().reshape(inp["T"], w.hv, w.dv)
    hT = out["hT"].cpu().numpy().astype(np.float64)
    o_ref, hT_ref = helpers.run_oracle(inp)
    tol = helpers.TOL[w.dtype]
    res = {"o_err": helpers.rel_max_err(o, o_ref), "hT_err": helpers.rel_max_err(hT, hT_ref),
           "o_nmse": helpers.nmse(o, o_ref), "hT_nmse": helpers.nmse(hT, hT_ref), "tolerance": tol,
           "metric": "max|err| / max|ref| per tensor, all heads, outputs of the last timed step"}
    res["ok"] = bool(np.isfinite(o).all() and np.isfinite(hT).all() and res["o_err"] <= tol and res["hT_err"] <= tol)
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="gdn_layer_4k", choices=sorted(synth.WORKLOADS) + sorted(DECODE_WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-parity", action="store_true", help="skip the oracle comparison of the timed outputs")
    ap.add_argument("--no-other-workloads", action="store_true", help="skip the short timings of the other workloads")
    ap.add_argument("--seq-len", type=int, default=0,
                    help="profiling captures: the same workload with sequences of this length (equal-length workloads)")
    ap.add_argument("--profile-range", action="store_true",
                    help="profiling captures: warm up, bracket ONE call with cudaProfilerStart/Stop, print its device "
                         "time and exit (for `ncu --replay-mode range`, which measures the call's kernels together)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.workload in DECODE_WORKLOADS:
        return decode_bench(args, rank, local_rank, world)
    w = synth.WORKLOADS[args.workload]
    if args.seq_len > 0:
        if w.seq_lens is None:
            raise SystemExit("--seq-len applies to the equal-length workloads")
        w = synth.shrink(w, seq_lens=[args.seq_len] * len(w.seq_lens), hk=w.hk, hv=w.hv)
    if args.impl == "reference":
        if rank == 0:
            run_reference(args, synth.make_inputs(w), rank)
        return

    import torch
    import paper_2609_32114_b200 as ha
    from tests import helpers

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path (use --impl reference for the oracle)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)

    # every rank draws its own batch of the same workload (weak scaling over independent batches)
    inp = synth.make_inputs(w, seed=rank_seed(rank))
    T, N = inp["T"], inp["N"]
    if args.profile_range:
        return profile_range(ha, helpers, w, inp, max(args.warmup, 3), dev)
    peaks = load_peaks()
    m = measure(ha, helpers, w, inp, args.steps, args.warmup, dev, local_rank, dist, peaks, world)
    sets, R, base, stream, sptr = m["sets"], m["R"], m["base"], m["stream"], m["sptr"]
    ms_per_step, value, roofline, clocks = m["ms_per_step"], m["value"], m["roofline"], m["clocks"]
    alg_bytes = m["alg_bytes"]

    def barrier():
        torch.cuda.synchronize(dev)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    # ---- parity of the timed configuration, same run: what the LAST timed step wrote, against the oracle
    parity = None
    if rank == 0 and not args.no_parity:
        parity = parity_of(helpers, inp, m["last_out"])

    # ---- end to end: pinned host buffers in, o and hT back out, through the public API
    host = {k: (v.cpu().pin_memory() if hasattr(v, "cpu") else v) for k, v in base.items()}
    a0, keep0 = sets[0]
    o_host = torch.empty_like(keep0["o"], device="cpu").pin_memory()
    hT_host = torch.empty_like(keep0["hT"], device="cpu").pin_memory()
    names = [k for k in ("q", "k", "v", "g", "beta", "h0", "cu_seqlens") if hasattr(base.get(k), "copy_")]
    h2d = sum(host[k].numel() * host[k].element_size() for k in names)
    d2h = o_host.numel() * o_host.element_size() + hT_host.numel() * hT_host.element_size()

    # Steady-state serving loop: two device buffer sets and three streams, so that the host->device copy of step
    # k+1 and the device->host copy of step k-1 run under the compute of step k (the link is full duplex).  Every
    # step still moves all of its inputs in and its outputs out inside the timed region.
    s_in, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    bufs = [sets[0], sets[1 % R]]
    o_hosts = [o_host, torch.empty_like(o_host).pin_memory()]
    hT_hosts = [hT_host, torch.empty_like(hT_host).pin_memory()]
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_comp = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]

    def e2e_step(k):
        b = k % 2
        a_b, keep_b = bufs[b]
        with torch.cuda.stream(s_in):
            if k >= 2:
                s_in.wait_event(ev_comp[b])              # the previous user of these input buffers has finished
            for name in names:
                keep_b[name].copy_(host[name].view_as(keep_b[name]), non_blocking=True)
            ev_in[b].record(s_in)
        stream.wait_event(ev_in[b])
        if k >= 2:
            stream.wait_event(ev_out[b])                 # its outputs have been copied out
        rc = ha.ha_la_prefill_raw(a_b, sptr)
        if rc != 0:
            raise ha.HaLaError(rc, "ha_la_prefill")
        ev_comp[b].record(stream)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_comp[b])
            o_hosts[b].copy_(keep_b["o"], non_blocking=True)
            hT_hosts[b].copy_(keep_b["hT"], non_blocking=True)
            ev_out[b].record(s_out)

    for k in range(2):
        e2e_step(k)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    s_in.wait_event(e0)
    for k in range(args.steps):
        e2e_step(k + 2)
    s_out.wait_stream(stream)
    e1.record(s_out)
    barrier()
    e2e_ms = max_over_ranks(dist, e0.elapsed_time(e1), dev)
    m["check_status"]("during the end-to-end steps")
    e2e = {"value": job_throughput(world, T, e2e_ms / args.steps), "unit": "tokens/s", "h2d_bytes_per_step": int(h2d),
           "d2h_bytes_per_step": int(d2h),
           "mode": "two buffer sets, copies of neighbouring steps overlap the compute (3 streams)"}

    # ---- the other full-size workloads, device time only (a few seconds in total): extra rows, not the metric
    others = None
    if rank == 0 and world == 1 and not args.no_other_workloads and w.name == "gdn_layer_4k":
        others = {}
        del sets, base, m["sets"], m["base"]
        torch.cuda.empty_cache()
        for name in ("gdn_gva_16k", "kda_8k", "gdn_varlen"):
            wo = synth.WORKLOADS[name]
            io = synth.make_inputs(wo)
            mo = measure(ha, helpers, wo, io, 30, 5, dev, local_rank, None, peaks, 1)
            po = parity_of(helpers, io, mo["last_out"]) if not args.no_parity else None
            others[name] = {"ms_per_step": mo["ms_per_step"], "ms_median": mo["ms_median"], "ms_min": mo["ms_min"],
                            "tokens_per_s": mo["value"], "steps": 30, "path_frac": mo["roofline"]["path"]["frac"],
                            "roofline_us": mo["roofline"]["path"]["roofline_us"],
                            "kernel_ms": mo["roofline"]["kernel_ms"], "launch_mode": mo["roofline"]["launch_mode"],
                            "clocks": mo["clocks"], "parity": po, "tokens": io["T"]}
            del mo, io
            torch.cuda.empty_cache()

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(inp)

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "ms_per_step_median": m["ms_median"],
                "ms_per_step_min": m["ms_min"], "ms_per_step_max": m["ms_max"], "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32",
                "data": "synthetic",
                "config": {"workload": w.name, "variant": w.variant, "tokens_per_step_per_gpu": T, "sequences": N,
                           "seq_lens": inp["seq_lens"] if N <= 16 else None, "qk_heads": w.hk, "v_heads": w.hv,
                           "d_k": w.dk, "d_v": w.dv, "chunk": 64, "path": m["path"],
                           "l2": f"{R} resident input/output sets visited round-robin ({R * alg_bytes / 1e6:.0f} MB), one scratch workspace"
                                 + (" + L2 flush write between steps" if m["flushed"] else ""),
                           "parallelism": "replicas (independent batch per GPU, no collective)" if world > 1 else "1 GPU"},
                "clocks": clocks, "e2e": e2e, "gpu_launches": m["launches_per_step"] * args.steps,
                "roofline": roofline, "parity": parity, "cpu_baseline": cpu, "other_workloads": others,
                "wall_s_timed_region": m["wall_s"],
                "timing": ("ms_per_step: the timed steps back to back between one pair of CUDA events on the launching stream; "
                           "median/min/max: the same steps again with one event pair each" if not m["flushed"] else
                           "one CUDA-event pair per step, the L2 flush outside the events")}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()
    if parity is not None and not parity["ok"]:
        raise SystemExit(f"parity of the timed configuration failed: {parity}")
    if others and any(v["parity"] is not None and not v["parity"]["ok"] for v in others.values()):
        raise SystemExit("parity of another workload failed (see other_workloads in the line above)")


if __name__ == "__main__":
    main()
