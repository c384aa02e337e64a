#!/usr/bin/env python
"""Benchmark of the HORA rollout-allocation hot path on B200.

One step = one pass of the whole path over one synthetic batch:
    hora_gains -> hora_allocate -> hora_group_advantage      on workload cfg4 (N = 2^20 prompts, G0 = 8,
                                                              ld = 256, B = 24 N, per-prompt real priors, GRPO)
    hora_token_broadcast                                      of the first 262144 rollout advantages of that
                                                              batch over response lengths ~ U{32..2048}
                                                              (the cfg3 token layout, ~2.7e8 tokens)
`value` is prompts per second over the whole step with every input resident in HBM; `e2e` is the same
metric with the step's inputs copied from pinned host memory and its results copied back inside the
timed region.  With --gpus N every rank runs its own independent batch (the paper allocates in
independent shards), no data-path collective, weak scaling.

`--impl reference` times the CPU oracle (a deliberately plain program) on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "hora_alloc_advantage_prompts_per_s"
UNIT = "prompts/s"
WORKLOAD = "cfg4"
BCAST_ROLLOUTS = 262144
FALLBACK_HBM_GBS = 6650.0

NOMINAL_HBM_GBS = 8000.0                  # datasheet figure, context beside the measured peak
PIPELINE_TARGET_FRAC = 0.60               # the stated bar for the allocation + advantage pipeline at cfg4
# fp64 operations per candidate gain as the method states them (recurrence after Eq. marginal:
# M(l+1) = M(l) (b + l) / (a + b + l + 1): two additions, one multiplication, one division)
FP64_OPS_PER_CANDIDATE = 4

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures summarised
# under profiles/ (taken at N = 131072 and scaled by the row count: the traffic is proportional to it);
# None = no usable capture (for gains_kernel the small case leaves a large share of its output in L2).
TRAFFIC_BYTES = {"select_level0": 2185488128, "gains_kernel": None}


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.005):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self.period = period_s
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
            nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
            nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def time_events(torch, fn, reps: int, warm: int = 3) -> float:
    """Mean milliseconds per call of fn, CUDA events on the current stream, after `warm` untimed calls."""
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def shard_seed(rank: int) -> int:
    """Every rank draws its own independent batch; rank 0 uses the workload's published seed."""
    return 3 + rank


def max_over_ranks(x: float, world: int, device=None) -> float:
    """Slowest rank's time: the job is done when the last shard is."""
    if world == 1:
        return x
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(prompts_per_rank: int, world: int, ms_per_step: float) -> float:
    """Whole-job prompts per second: every rank processes its own shard of prompts_per_rank prompts."""
    return prompts_per_rank * world / (ms_per_step * 1e-3)


# --------------------------------------------------------------------------------------- our arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2605_07114_b200 import hora, workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    hora.load()

    if args.only is not None:
        # one of the secondary measurements alone (a small process to profile): its object, as one JSON line
        peak = measured_peak()[0]
        fp64 = measure_fp64_peak(torch, hora, dev)
        if args.only == "batched":
            res = bench_batched(torch, hora, wl, dev, peak, fp64["value"], shards=args.shards)
        else:
            res = bench_configs(torch, hora, wl, dev, peak)
        print(json.dumps({args.only: res}))
        return

    w = wl.make(WORKLOAD, args.prompts, seed=shard_seed(rank))
    N, ld, G0, B = w.N, w.ld, w.G0, w.B
    h_alpha = torch.from_numpy(w.alpha).pin_memory()
    h_beta = torch.from_numpy(w.beta).pin_memory()
    h_c = torch.from_numpy(w.c).pin_memory()
    alpha, beta, c = h_alpha.to(dev), h_beta.to(dev), h_c.to(dev)
    cap_scalar = ld
    al = hora.Allocator(N, ld, G0, exact_int=False, device=dev)

    # one untimed pass fixes the group layout, from which the synthetic rewards are drawn
    al.run(alpha, beta, 1.0, 1.0, c, None, cap_scalar, B)
    info = al.read_info()
    if info.status != 0:
        raise RuntimeError(f"allocation failed: {hora.status_string(info.status)}")
    off_h = al.group_offsets.cpu().numpy()
    total = int(off_h[-1])
    h_rewards = torch.from_numpy(w.rewards(off_h)).pin_memory()
    rewards = h_rewards.to(dev)
    adv = torch.empty(total, dtype=torch.float32, device=dev)
    R = min(BCAST_ROLLOUTS, total)
    tok_h = w.token_offsets(R)
    T = int(tok_h[-1])
    tok = torch.from_numpy(tok_h).to(dev)
    token_adv = torch.empty(T, dtype=torch.float32, device=dev)
    h_delta = torch.empty(N, dtype=torch.int32).pin_memory()
    h_G = torch.empty(N, dtype=torch.int32).pin_memory()
    h_adv = torch.empty(total, dtype=torch.float32).pin_memory()
    eps = float(w.eps)

    def step(events=None):
        if events is not None:
            events[0].record()
        hora.hora_gains(alpha, beta, 1.0, 1.0, c, G0, None, cap_scalar, N, ld, al.gains)
        if events is not None:
            events[1].record()
        hora.hora_allocate(alpha, beta, 1.0, 1.0, c, G0, None, cap_scalar, N, ld, al.gains, B, al.flags, al.delta,
                           al.G, al.group_offsets, al.info, al.workspace)
        if events is not None:
            events[2].record()
        hora.hora_group_advantage(rewards, al.group_offsets, N, w.adv_mode, eps, w.ddof, adv)
        if events is not None:
            events[3].record()
        hora.hora_token_broadcast(adv, tok, R, T, token_adv)
        if events is not None:
            events[4].record()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- before any timing counts: the oracle's pass over (a prefix of) this batch, and the four calls held
    # against it, output by output.  The same pass is the CPU baseline reported beside the result. ----
    ref = parity = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        ref = oracle_pass(w, min(args.cpu_sample, N))
        parity = check_against_oracle(torch, hora, dev, ref)

    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        step()
    barrier()

    # ---- timed region: device-resident inputs ----
    stage_ev = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(args.steps)]
    # events the library records around its full-read selection kernel (the dominant launch of the step)
    l0_ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
    for pair in l0_ev:
        for ev in pair:
            ev.record()                                  # creates the underlying cudaEvent_t
    launches0 = hora.hora_launch_count()
    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()
    barrier()
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    for k in range(args.steps):
        hora.hora_allocate_profile_events(l0_ev[k][0].cuda_event, l0_ev[k][1].cuda_event)
        step(stage_ev[k])
    t1.record()
    hora.hora_allocate_profile_events(None, None)
    barrier()
    launches = hora.hora_launch_count() - launches0
    ms_total = max_over_ranks(t0.elapsed_time(t1), world, dev)
    ms_step = ms_total / args.steps
    # a short timed region gives the clock sampler only a few samples: the same step loop goes on, untimed, until
    # the sampler has seen about 0.3 s of this load
    extra_steps = max(0, int(0.3 / (ms_step * 1e-3)) - args.steps)
    for _ in range(extra_steps):
        step()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    clocks["covers"] = f"the {args.steps} timed steps and {extra_steps} further identical steps"
    stages = np.array([[ev[i].elapsed_time(ev[i + 1]) for i in range(4)] for ev in stage_ev])
    st_mean = stages.mean(axis=0)
    st_min = stages.min(axis=0)
    l0_ms = float(np.mean([a.elapsed_time(b) for a, b in l0_ev]))

    info = al.read_info()
    if info.status != 0 or info.sum_G != total:
        raise RuntimeError("allocation changed during the timed loop")

    # ---- where hora_allocate spends its time: events the library records at its stage boundaries ----
    n_prof = max(3, min(args.steps, 20))
    st_ev = [[torch.cuda.Event(enable_timing=True) for _ in range(7)] for _ in range(n_prof)]
    for evs in st_ev:
        for ev in evs:
            ev.record()
    for k in range(n_prof):
        hora.hora_allocate_profile_stages([ev.cuda_event for ev in st_ev[k]])
        step()
    hora.hora_allocate_profile_stages(None)
    torch.cuda.synchronize()
    st = np.array([[evs[i].elapsed_time(evs[i + 1]) for i in range(6)] for evs in st_ev]).mean(axis=0)
    alloc_stages = dict(zip(("estimate", "full_read_level0", "rows_level1", "tail_threshold_and_scan",
                             "exact_ranking", "outputs"), (round(float(x), 4) for x in st)))

    # ---- the same four-call step replayed from a CUDA graph (launch gaps between the nine kernels removed) ----
    graph_ms = None
    if world == 1:
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                step()                                   # the capture stream has run every kernel once
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                step()
            for _ in range(3):
                g.replay()
            torch.cuda.synchronize()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ng = max(3, min(args.steps, 100))
            g0.record()
            for _ in range(ng):
                g.replay()
            g1.record()
            torch.cuda.synchronize()
            if al.read_info().status == 0 and al.read_info().sum_G == total:
                graph_ms = g0.elapsed_time(g1) / ng
            del g
        except Exception as exc:                         # a capture that fails must not cost the line
            print(f"graph replay skipped: {exc}", file=sys.stderr)
            torch.cuda.synchronize()

    # ---- the same step with the fused call: hora_allocate builds the matrix itself and counts on the way ----
    fused_ms = None
    if world == 1:
        al.gains = None                                  # release the stand-alone matrix before taking the fused one
        torch.cuda.empty_cache()
        alf = hora.Allocator(N, ld, G0, exact_int=False, materialise=False, device=dev)

        def fused_allocate():
            hora.hora_allocate(alpha, beta, 1.0, 1.0, c, G0, None, cap_scalar, N, ld, None, B, alf.flags, alf.delta,
                               alf.G, alf.group_offsets, alf.info, alf.workspace)

        def step_fused():
            fused_allocate()
            hora.hora_group_advantage(rewards, alf.group_offsets, N, w.adv_mode, eps, w.ddof, adv)
            hora.hora_token_broadcast(adv, tok, R, T, token_adv)
        for _ in range(3):
            step_fused()
        torch.cuda.synchronize()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        nf = max(3, min(args.steps, 50))
        f0.record()
        for _ in range(nf):
            step_fused()
        f1.record()
        torch.cuda.synchronize()
        fused_ms = f0.elapsed_time(f1) / nf
        fused_alloc_ms = time_events(torch, fused_allocate, nf)
        if not torch.equal(alf.delta, al.delta):
            raise RuntimeError("fused and two-call allocations differ")
        del alf
        torch.cuda.empty_cache()
        al.gains = torch.empty((N, ld), dtype=torch.float64, device=dev)

    # ---- token-level advantages of the broadcast rollouts: two calls against the one fused call ----
    tok_cmp = None
    if world == 1:
        n_bc = int(np.searchsorted(off_h, R, side="left"))          # groups that cover the first R rollouts
        check = torch.empty_like(token_adv)

        def two_calls():
            hora.hora_group_advantage(rewards, al.group_offsets, n_bc, w.adv_mode, eps, w.ddof, adv)
            hora.hora_token_broadcast(adv, tok, R, T, token_adv)

        def one_call():
            hora.hora_group_advantage_tokens(rewards, al.group_offsets, N, tok, R, T, w.adv_mode, eps, w.ddof, check)
        ms = []
        for fn in (two_calls, one_call):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            nt = max(3, min(args.steps, 50))
            a0.record()
            for _ in range(nt):
                fn()
            a1.record()
            torch.cuda.synchronize()
            ms.append(a0.elapsed_time(a1) / nt)
        if float((check - token_adv).abs().max()) > 1e-5:
            raise RuntimeError("fused and two-call token advantages differ")
        tok_cmp = {"rollouts": R, "tokens": T, "ms_two_calls": round(ms[0], 4), "ms_fused": round(ms[1], 4),
                   "fused_gbs": round(4.0 * T / ms[1] / 1e6, 1)}

    # ---- end to end: pinned host inputs in, results out, every step ----
    # Three streams (copy in, compute, copy out) over two sets of device and host buffers: step k's results leave
    # while step k+1's inputs arrive (PCIe is full duplex) and its kernels run.  Every step still copies all of its
    # inputs from pinned host memory and all of its results back inside the timed region.
    cur = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    sets = []
    for k in range(2):
        sets.append({
            "alpha": torch.empty_like(alpha), "beta": torch.empty_like(beta), "c": torch.empty_like(c),
            "rewards": torch.empty_like(rewards), "adv": torch.empty_like(adv), "delta": torch.empty_like(al.delta),
            "G": torch.empty_like(al.G), "off": torch.empty_like(al.group_offsets), "info": torch.zeros_like(al.info),
            "h_delta": h_delta if k == 0 else torch.empty_like(h_delta).pin_memory(),
            "h_G": h_G if k == 0 else torch.empty_like(h_G).pin_memory(),
            "h_adv": h_adv if k == 0 else torch.empty_like(h_adv).pin_memory(),
            "in_ready": torch.cuda.Event(), "computed": torch.cuda.Event(), "out_done": torch.cuda.Event()})
    torch.cuda.synchronize()

    def step_e2e(k):
        b = sets[k % 2]
        s_in.wait_event(b["computed"])                   # the step that last read these inputs is over
        with torch.cuda.stream(s_in):
            b["alpha"].copy_(h_alpha, non_blocking=True)
            b["beta"].copy_(h_beta, non_blocking=True)
            b["c"].copy_(h_c, non_blocking=True)
            b["rewards"].copy_(h_rewards, non_blocking=True)
            b["in_ready"].record(s_in)
        cur.wait_event(b["in_ready"])
        cur.wait_event(b["out_done"])                    # the results that lived here have left
        hora.hora_gains(b["alpha"], b["beta"], 1.0, 1.0, b["c"], G0, None, cap_scalar, N, ld, al.gains)
        hora.hora_allocate(b["alpha"], b["beta"], 1.0, 1.0, b["c"], G0, None, cap_scalar, N, ld, al.gains, B, al.flags,
                           b["delta"], b["G"], b["off"], b["info"], al.workspace)
        hora.hora_group_advantage(b["rewards"], b["off"], N, w.adv_mode, eps, w.ddof, b["adv"])
        hora.hora_token_broadcast(b["adv"], tok, R, T, token_adv)
        b["computed"].record(cur)
        s_out.wait_event(b["computed"])
        with torch.cuda.stream(s_out):
            b["h_delta"].copy_(b["delta"], non_blocking=True)
            b["h_G"].copy_(b["G"], non_blocking=True)
            b["h_adv"].copy_(b["adv"], non_blocking=True)
            b["out_done"].record(s_out)

    def drain():
        cur.wait_stream(s_in)
        cur.wait_stream(s_out)

    e2e_steps = max(4, min(args.steps, 20))
    for k in range(2):
        step_e2e(k)
    drain()
    barrier()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for k in range(e2e_steps):
        step_e2e(k)
    drain()
    e1.record()
    barrier()
    for b in sets:
        if not (torch.equal(b["h_delta"], al.delta.cpu()) and torch.equal(b["h_adv"], adv.cpu())):
            raise RuntimeError("end-to-end results differ from the device-resident step")
    ms_e2e = max_over_ranks(e0.elapsed_time(e1), world, dev) / e2e_steps
    h2d = h_alpha.numel() * 8 + h_beta.numel() * 8 + h_c.numel() * 4 + h_rewards.numel() * 4
    d2h = h_delta.numel() * 4 + h_G.numel() * 4 + h_adv.numel() * 4

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    cand = N * ld
    bytes_gains = cand * 8 + N * 20
    bytes_alloc = cand * 8 + N * (20 + 4 + 4 + 8)
    bytes_adv = total * 8 + (N + 1) * 8
    bytes_bc = T * 4 + R * 12
    algo = [bytes_gains, bytes_alloc, bytes_adv, bytes_bc]
    names = ["hora_gains", "hora_allocate", "hora_group_advantage", "hora_token_broadcast"]
    stage_report = {}
    for nm, by, ms, mn in zip(names, algo, st_mean, st_min):
        gbs = by / (ms * 1e-3) / 1e9
        stage_report[nm] = {"ms": round(float(ms), 4), "ms_min": round(float(mn), 4), "algorithmic_bytes": int(by),
                            "gbs": round(gbs, 1), "frac_of_hbm_peak": round(gbs / peak, 4)}
    pipe_bytes = sum(algo[:3])
    pipe_ms = float(st_mean[:3].sum())
    g_ms = float(st_mean[0])                           # hora_gains is exactly one launch (gains_kernel)
    bytes_l0 = cand * 8                                # the full-read pass: every candidate key once
    achieved = bytes_l0 / (l0_ms * 1e-3) / 1e9
    achieved_gains = bytes_gains / (g_ms * 1e-3) / 1e9
    out = {
        "metric": METRIC, "value": job_throughput(N, world, ms_step), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{WORKLOAD}: N={N} prompts per GPU, G0={G0}, ld={ld}, B={B}, per-prompt real priors, "
                               f"GRPO; then token broadcast of {R} rollouts to {T} tokens (lengths U{{32..2048}})",
                   "l2": "inputs larger than L2 (the gains matrix alone is %.2f GB)" % (cand * 8 / 1e9),
                   "shard": "one independent batch per GPU, no collective"},
        "clocks": clocks,
        "e2e": {"value": job_throughput(N, world, ms_e2e), "unit": UNIT, "ms_per_step": ms_e2e,
                "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                "overlap": "copy-in, kernels and copy-out on three streams over two buffer sets"},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "select_level0 (the full-read pass of hora_allocate, timed by events the "
                                               "library records around its launch)",
                     "achieved": round(achieved, 1), "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                     "frac": round(achieved / peak, 4), "traffic": TRAFFIC_BYTES.get("select_level0"),
                     "algorithmic_bytes_per_launch": int(bytes_l0), "ms_per_launch": round(l0_ms, 4)},
        "roofline_gains": {"bound": "hbm", "kernel": "gains_kernel (the one launch of hora_gains)",
                           "achieved": round(achieved_gains, 1), "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                           "frac": round(achieved_gains / peak, 4), "traffic": TRAFFIC_BYTES.get("gains_kernel"),
                           "algorithmic_bytes_per_launch": int(bytes_gains), "ms_per_launch": round(g_ms, 4)},
        "pipeline": {"calls": "hora_gains+hora_allocate+hora_group_advantage", "ms": round(pipe_ms, 4),
                     "algorithmic_bytes": int(pipe_bytes), "gbs": round(pipe_bytes / (pipe_ms * 1e-3) / 1e9, 1),
                     "frac_of_hbm_peak": round(pipe_bytes / (pipe_ms * 1e-3) / 1e9 / peak, 4),
                     "prompts_per_s": N / (pipe_ms * 1e-3), "candidate_gains_per_s": cand / (pipe_ms * 1e-3)},
        "tokens_per_s": T / (float(st_mean[3]) * 1e-3),
        "stages": stage_report,
        "allocate_stages_ms": alloc_stages,
        "allocation": {"lambda": info.lambda_, "n_above": info.n_above, "n_tied": info.n_tied,
                       "objective": info.objective},
    }
    out["pipeline"].update({"target_frac": PIPELINE_TARGET_FRAC,
                            "frac_of_nominal_hbm": round(pipe_bytes / (pipe_ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS, 4),
                            "nominal_hbm_gbs": NOMINAL_HBM_GBS})
    fp64 = None
    if world == 1:
        fp64 = measure_fp64_peak(torch, hora, dev)
        out["peak_fp64_tflops"] = fp64
    if fused_ms is not None:
        out["token_advantages"] = tok_cmp
        flops = FP64_OPS_PER_CANDIDATE * cand
        ach = flops / (fused_alloc_ms * 1e-3) / 1e12
        out["fused_step"] = {"calls": "hora_allocate(gains=NULL)+hora_group_advantage+hora_token_broadcast",
                             "ms_per_step": round(fused_ms, 4), "prompts_per_s": N / (fused_ms * 1e-3),
                             "hora_allocate_ms": round(fused_alloc_ms, 4),
                             "roofline": {"bound": "alu", "kernel": "hora_allocate(gains=NULL): rows computed and counted "
                                          "in one pass (gains_level0_fused and the passes behind it)",
                                          "achieved": round(ach, 3), "peak": fp64["value"], "unit": "TFLOP/s",
                                          "frac": round(ach / fp64["value"], 4), "traffic": None,
                                          "algorithmic_flops_per_launch": int(flops),
                                          "flops_per_candidate": FP64_OPS_PER_CANDIDATE,
                                          "peak_kind": "measured fp64 FMA rate (hora_fp64_probe), 2 flop per FMA"},
                             "hbm_view": {"bytes_written_once": int(cand * 8), "gbs": round(cand * 8 / (fused_alloc_ms * 1e-3) / 1e9, 1),
                                          "frac_of_hbm_peak": round(cand * 8 / (fused_alloc_ms * 1e-3) / 1e9 / peak, 4),
                                          "note": "the call still writes the matrix once into its workspace; against "
                                                  "that one write it runs at this fraction of the measured copy peak"},
                             "note": "same outputs; the matrix is written once inside the workspace and not read back in "
                                     "full, so this step moves 2.15 GB less than the four-call step timed above"}
    if graph_ms is not None:
        out["graph_step"] = {"ms_per_step": round(graph_ms, 4), "prompts_per_s": N / (graph_ms * 1e-3),
                             "note": "the same four calls captured once in a CUDA graph and replayed"}
    if world == 1:
        out["batched"] = bench_batched(torch, hora, wl, dev, peak, fp64["value"])
        out["configs"] = bench_configs(torch, hora, wl, dev, peak)
    if ref is not None:
        out["cpu_baseline"] = cpu_baseline(w, args.cpu_sample, ref)
        out["parity"] = parity
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def measure_fp64_peak(torch, hora, dev, iters=4096, reps=5):
    """fp64 rate of this GPU from the library's FMA probe: best of `reps` launches, 2 flop per FMA."""
    sink = torch.zeros(1, dtype=torch.float64, device=dev)
    hora.hora_fp64_probe(256, sink)
    torch.cuda.synchronize()
    best = 0.0
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fmas = hora.hora_fp64_probe(iters, sink)
        e1.record()
        torch.cuda.synchronize()
        best = max(best, 2.0 * fmas / (e0.elapsed_time(e1) * 1e-3) / 1e12)
    return {"value": round(best, 2), "unit": "TFLOP/s", "how": f"hora_fp64_probe: 8 independent FMA chains per thread, "
            f"{iters} steps, 8 CTAs of 256 threads per SM, best of {reps}; flop = 2 per FMA"}


def bench_batched(torch, hora, wl, dev, hbm_peak, fp64_peak, shards=65536, shard_prompts=15, per_prompt=24, reps=20):
    """Secondary measurement: hora_allocate_batched on the shape the paper trains with (shards of 15 prompts,
    G0 = 8, 24 extra rollouts per prompt, exact ties), many shards in one call: with the paper's uniform prior
    (solved on exact ranks, a warp per shard) and with per-prompt real priors (a CTA per shard, rows in shared memory)."""
    rng = np.random.default_rng(15)
    G0, ld = 8, shard_prompts * per_prompt
    N = shards * shard_prompts
    c_h = rng.choice(G0 + 1, size=N, p=[0.15] + [0.34 / 7] * 7 + [0.51]).astype(np.int32)
    c = torch.from_numpy(c_h).to(dev)
    seg = np.arange(0, N + 1, shard_prompts, dtype=np.int64)
    budgets = np.full(shards, ld, np.int64)
    delta = torch.empty(N, dtype=torch.int32, device=dev)
    G = torch.empty(N, dtype=torch.int32, device=dev)
    off = torch.empty(N + 1, dtype=torch.int64, device=dev)
    info = torch.zeros(shards * hora.INFO_BYTES, dtype=torch.uint8, device=dev)
    ws = torch.empty(hora.hora_allocate_batched_workspace_bytes(N, shards), dtype=torch.uint8, device=dev)

    def uniform():
        hora.hora_allocate_batched(None, None, 1.0, 1.0, c, G0, None, ld, N, ld, seg, budgets, hora.FLAG_EXACT_INT,
                                   delta, G, off, info, ws)
    ms = time_events(torch, uniform, reps)
    if int(delta.sum().item()) != shards * ld:
        raise RuntimeError("batched allocation did not hand out the whole budget")
    # algorithmic traffic of the uniform-prior form: 4 B of c in, Delta, G (8 B) and an offset (8 B) out per
    # prompt, a 16-byte segment entry in and a 64-byte summary out per shard
    by = N * 20 + shards * 80
    out = {"call": "hora_allocate_batched", "shards": shards, "prompts_per_shard": shard_prompts, "G0": G0, "ld": ld,
           "budget_per_shard": ld, "prior": "uniform Beta(1,1), exact ties (rank-based route)", "ms": round(ms, 4),
           "shards_per_s": shards / (ms * 1e-3), "prompts_per_s": N / (ms * 1e-3), "candidates_per_s": N * ld / (ms * 1e-3),
           "roofline": {"bound": "hbm", "kernel": "whole call (rank tables, one warp per shard, offsets scan; the segment "
                        "table is copied from host memory inside the call)", "achieved": round(by / (ms * 1e-3) / 1e9, 1),
                        "peak": hbm_peak, "unit": "GB/s", "frac": round(by / (ms * 1e-3) / 1e9 / hbm_peak, 4), "traffic": None,
                        "algorithmic_bytes_per_launch": int(by),
                        "note": "a few tens of MB per call: launch latency and the host-to-device copy of the segment "
                                "table set the time, not bandwidth"}}
    # per-prompt real priors on a quarter of the shards (the general path)
    s2 = shards // 4
    n2 = s2 * shard_prompts
    al = torch.from_numpy(np.exp(rng.uniform(np.log(0.05), np.log(20), n2))).to(dev)
    be = torch.from_numpy(np.exp(rng.uniform(np.log(0.05), np.log(20), n2))).to(dev)

    def real():
        hora.hora_allocate_batched(al, be, 1.0, 1.0, c[:n2], G0, None, ld, n2, ld, seg[:s2 + 1], budgets[:s2], 0,
                                   delta[:n2], G[:n2], off[:n2 + 1], info[:s2 * hora.INFO_BYTES], ws)
    ms2 = time_events(torch, real, max(3, reps // 4))
    flops = FP64_OPS_PER_CANDIDATE * n2 * ld
    ach = flops / (ms2 * 1e-3) / 1e12
    out["real_priors"] = {"shards": s2, "ms": round(ms2, 4), "shards_per_s": s2 / (ms2 * 1e-3),
                          "prompts_per_s": n2 / (ms2 * 1e-3),
                          "roofline": {"bound": "alu", "kernel": "allocate_batched_kernel (a CTA of 128 threads per shard: rows built in "
                                       "shared memory, the threshold built two bits a step by one warp)", "achieved": round(ach, 3), "peak": fp64_peak,
                                       "unit": "TFLOP/s", "frac": round(ach / fp64_peak, 4), "traffic": None,
                                       "algorithmic_flops_per_launch": int(flops),
                                       "flops_per_candidate": FP64_OPS_PER_CANDIDATE}}
    return out


def bench_configs(torch, hora, wl, dev, peak):
    """The other named workloads (parity cases of the test-suite), event-timed here so that their numbers come from
    the same run: hora_gains + hora_allocate with the matrix, the rank-based route where the prior is the shared
    integer one, the advantages over the resulting groups, and for cfg3 the broadcast to its 2.7e8 tokens."""
    res = {}
    for name in ("cfg1", "cfg2", "cfg3", "cfg5"):
        w = wl.make(name)
        N, ld, G0, B = w.N, w.ld, w.G0, w.B
        t = lambda x: None if x is None else torch.from_numpy(x).to(dev)
        alpha, beta, c, cap = t(w.alpha), t(w.beta), t(w.c), t(w.cap)
        al = hora.Allocator(N, ld, G0, exact_int=w.exact_int, device=dev)
        reps = 50 if N <= (1 << 16) else 10

        def gains():
            hora.hora_gains(alpha, beta, w.alpha0, w.beta0, c, G0, cap, 0, N, ld, al.gains)

        def allocate():
            hora.hora_allocate(alpha, beta, w.alpha0, w.beta0, c, G0, cap, 0, N, ld, al.gains, B, al.flags, al.delta, al.G,
                               al.group_offsets, al.info, al.workspace)
        g_ms = time_events(torch, gains, reps)
        a_ms = time_events(torch, allocate, reps)
        if al.read_info().status != 0:
            raise RuntimeError(f"{name}: allocation failed")
        cand = N * ld
        entry = {"N": N, "ld": ld, "G0": G0, "B": B, "prior": "shared Beta(1,1), exact ties" if w.exact_int else "per-prompt real",
                 "hora_gains_us": round(g_ms * 1e3, 1), "hora_allocate_us": round(a_ms * 1e3, 1)}
        if w.exact_int:
            ar = hora.Allocator(N, ld, G0, exact_int=True, materialise=False, shared_int_prior=True, device=dev)

            def on_ranks():
                hora.hora_allocate(None, None, w.alpha0, w.beta0, c, G0, cap, 0, N, ld, None, B, ar.flags, ar.delta, ar.G,
                                   ar.group_offsets, ar.info, ar.workspace)
            r_ms = time_events(torch, on_ranks, reps)
            if not torch.equal(ar.delta, al.delta):
                raise RuntimeError(f"{name}: the rank-based route and the matrix route disagree")
            entry["hora_allocate_on_ranks_us"] = round(r_ms * 1e3, 1)
            entry["on_ranks_bytes"] = int(N * 24 + N * 16)           # three reads of (c, cap), Delta, G, offset out
            entry["on_ranks_gbs"] = round(entry["on_ranks_bytes"] / (r_ms * 1e-3) / 1e9, 1)
            del ar
        off_h = al.group_offsets.cpu().numpy()
        rewards_h = w.rewards(off_h)
        rewards = torch.from_numpy(rewards_h).to(dev)
        adv = torch.empty_like(rewards)

        def advantage():
            hora.hora_group_advantage(rewards, al.group_offsets, N, w.adv_mode, float(w.eps), w.ddof, adv)
        v_ms = time_events(torch, advantage, reps)
        entry["hora_group_advantage_us"] = round(v_ms * 1e3, 1)
        entry["rollouts"] = int(off_h[-1])
        if N >= (1 << 20):                                           # large enough for bandwidth to mean something
            bg, ba = cand * 8 + N * 20, cand * 8 + N * 36
            bv = int(off_h[-1]) * 8 + (N + 1) * 8
            entry["gbs"] = {"hora_gains": round(bg / (g_ms * 1e-3) / 1e9, 1), "hora_allocate": round(ba / (a_ms * 1e-3) / 1e9, 1),
                            "hora_group_advantage": round(bv / (v_ms * 1e-3) / 1e9, 1)}
            entry["frac_of_hbm_peak"] = {k: round(v / peak, 4) for k, v in entry["gbs"].items()}
        else:
            entry["note"] = "launch- and latency-bound at this size: microseconds per call, bandwidth figures would mean nothing"
        if w.with_tokens:
            Rn = int(off_h[-1])
            tok_h = w.token_offsets(Rn)
            T = int(tok_h[-1])
            tok = torch.from_numpy(tok_h).to(dev)
            token_adv = torch.empty(T, dtype=torch.float32, device=dev)

            def broadcast():
                hora.hora_token_broadcast(adv, tok, Rn, T, token_adv)
            b_ms = time_events(torch, broadcast, 20)
            bb = T * 4 + Rn * 12
            entry["hora_token_broadcast"] = {"tokens": T, "ms": round(b_ms, 4), "tokens_per_s": T / (b_ms * 1e-3),
                                             "gbs": round(bb / (b_ms * 1e-3) / 1e9, 1),
                                             "frac_of_hbm_peak": round(bb / (b_ms * 1e-3) / 1e9 / peak, 4)}
            del tok, token_adv
        res[name] = entry
        del al, rewards, adv
        torch.cuda.empty_cache()
    res["parity"] = "each of these workloads is compared with the oracle, at full size, by the test-suite (tests/test_gpu_parity.py, tests/test_gpu_fullsize.py, tests/test_gpu_rank_route.py)"
    return res


# ------------------------------------------------------------------------------- oracle timing
def oracle_pass(w, n):
    """The oracle, as it stands, on the first n prompts of the workload (budget scaled with n).
    Returns the seconds spent inside oracle calls (input generation excluded) and what it computed."""
    from oracle import hora_oracle as orc
    sl = slice(0, n)
    alpha, beta, c, cap = w.alpha[sl], w.beta[sl], w.c[sl], w.cap[sl]
    B = (w.B // w.N) * n
    t0 = time.perf_counter()
    orc.gains(alpha, beta, w.alpha0, w.beta0, c, w.G0, cap, w.ld)
    d, G, lam, obj = orc.greedy_real(alpha, beta, w.alpha0, w.beta0, c, w.G0, cap, B)
    t1 = time.perf_counter()
    off = np.zeros(n + 1, np.int64)
    np.cumsum(G.astype(np.int64), out=off[1:])
    sub = type(w)(**{**w.__dict__, "N": n, "p": w.p[sl], "c": c, "cap": cap, "alpha": alpha, "beta": beta, "B": B})
    rewards = sub.rewards(off)
    R = max(1, min(len(rewards), BCAST_ROLLOUTS * n // w.N))
    tok = sub.token_offsets(R)
    t2 = time.perf_counter()
    adv = orc.group_advantage(rewards, off, w.adv_mode, float(np.float32(w.eps)), w.ddof)
    token_adv = orc.token_broadcast(adv[:R], tok)
    t3 = time.perf_counter()
    return {"seconds": (t1 - t0) + (t3 - t2), "n": n, "B": B, "delta": d, "G": G, "lambda": lam, "objective": obj,
            "offsets": off, "rewards": rewards, "adv": adv, "R": R, "token_offsets": tok, "token_adv": token_adv,
            "workload": sub}


def oracle_step(w, n):
    return oracle_pass(w, n)["seconds"]


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def oracle_all_cores(ref, n_gain_rows=1 << 17):
    """The parts of the oracle that split over prompts with no interaction — gain rows, group advantages, token
    repeat — run as they stand on every host core (one thread per core, each on its own contiguous slice; the C
    routines release the interpreter lock).  The heap greedy is one sequential loop and stays on one core."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import hora_oracle as orc
    w = ref["workload"]
    cores = host_cores()
    n = min(n_gain_rows, ref["n"])

    def split(total):
        edges = np.linspace(0, total, cores + 1).astype(np.int64)
        return [(int(edges[k]), int(edges[k + 1])) for k in range(cores) if edges[k + 1] > edges[k]]

    def run(jobs):
        t0 = time.perf_counter()
        with ThreadPoolExecutor(max_workers=cores) as ex:
            list(ex.map(lambda f: f(), jobs))
        return time.perf_counter() - t0
    t_gains = run([lambda a=a, b=b: orc.gains(w.alpha[a:b], w.beta[a:b], w.alpha0, w.beta0, w.c[a:b], w.G0, w.cap[a:b], w.ld)
                   for a, b in split(n)])
    off, rewards = ref["offsets"], ref["rewards"]
    eps = float(np.float32(w.eps))
    t_adv = run([lambda a=a, b=b: orc.group_advantage(rewards[off[a]:off[b]], off[a:b + 1] - off[a], w.adv_mode, eps, w.ddof)
                 for a, b in split(ref["n"])])
    tok, R = ref["token_offsets"], ref["R"]
    t_bc = run([lambda a=a, b=b: orc.token_broadcast(ref["adv"][a:b], tok[a:b + 1] - tok[a]) for a, b in split(R)])
    return {"cores": cores, "gain_rows_per_s": n / t_gains, "candidate_gains_per_s": n * w.ld / t_gains,
            "advantage_rollouts_per_s": len(rewards) / t_adv, "broadcast_tokens_per_s": int(tok[-1]) / t_bc,
            "seconds": {"gains": round(t_gains, 3), "advantage": round(t_adv, 3), "broadcast": round(t_bc, 3)},
            "sample": f"gain rows of the first {n} prompts; advantages of all {len(rewards)} rollouts of the oracle pass; "
                      f"broadcast of {R} rollouts to {int(tok[-1])} tokens",
            "note": "the heap greedy (Algorithm 1's loop) is sequential: it is timed on one core in `value`"}


def cpu_baseline(w, n, ref=None):
    n = min(n, w.N)
    ref = ref if ref is not None else oracle_pass(w, n)
    secs = ref["seconds"]
    out = {"value": n / secs, "unit": UNIT, "cores": 1, "kind": "oracle", "seconds": round(secs, 2),
           "sample": f"first {n} of {w.N} prompts of {WORKLOAD} (budget and token count scaled by the same factor), "
                     "one pass: long-double gain rows, heap greedy, group advantages, token repeat"}
    out["all_cores"] = oracle_all_cores(ref)
    return out


def check_against_oracle(torch, hora, dev, ref, band=1e-12):
    """Runs the four calls on the prompts the oracle pass covered and compares every output with the oracle's:
    Delta may differ only on candidates whose oracle gain is within `band` (relative) of the oracle threshold,
    G and the offsets must follow from Delta, lambda and the objective agree to 1e-12 relative, advantages to
    1e-5 absolute (on the oracle's group layout), the token broadcast bitwise.  Raises on any violation."""
    from oracle import hora_oracle as orc
    w = ref["workload"]
    n, ld, G0, B = ref["n"], w.ld, w.G0, ref["B"]
    alpha, beta = torch.from_numpy(w.alpha).to(dev), torch.from_numpy(w.beta).to(dev)
    c = torch.from_numpy(w.c).to(dev)
    al = hora.Allocator(n, ld, G0, exact_int=False, device=dev)
    al.run(alpha, beta, w.alpha0, w.beta0, c, None, ld, B)
    info = al.read_info()
    if info.status != 0:
        raise RuntimeError(f"parity check: allocation failed: {hora.status_string(info.status)}")
    d = al.delta.cpu().numpy()
    if int(d.astype(np.int64).sum()) != B or (d < 0).any() or (d > w.cap).any():
        raise RuntimeError("parity check: Delta is not a feasible allocation")
    if not np.array_equal(al.G.cpu().numpy(), G0 + d):
        raise RuntimeError("parity check: G != G0 + Delta")
    off = np.zeros(n + 1, np.int64)
    np.cumsum((G0 + d).astype(np.int64), out=off[1:])
    if not np.array_equal(al.group_offsets.cpu().numpy(), off):
        raise RuntimeError("parity check: group offsets are not the prefix sums of G")
    lam = ref["lambda"]
    differ = np.nonzero(d != ref["delta"])[0]
    in_band = 0
    for i in differ:
        lo, hi = sorted((int(d[i]), int(ref["delta"][i])))
        a_i, b_i = float(w.alpha[i]) + int(w.c[i]), float(w.beta[i]) + (G0 - int(w.c[i]))
        for D in range(lo + 1, hi + 1):
            g = orc.gain_one(a_i, b_i, D)
            if abs(g - lam) > band * lam:
                raise RuntimeError(f"parity check: Delta differs outside the band at prompt {i}, candidate {D}")
            in_band += 1
    if abs(info.lambda_ - lam) > 1e-12 * lam or abs(info.objective - ref["objective"]) > 1e-12 * ref["objective"]:
        raise RuntimeError("parity check: threshold or objective differ from the oracle's")
    rewards = torch.from_numpy(ref["rewards"]).to(dev)
    off_o = torch.from_numpy(ref["offsets"]).to(dev)
    adv = torch.empty_like(rewards)
    hora.hora_group_advantage(rewards, off_o, n, w.adv_mode, float(w.eps), w.ddof, adv)
    adv_err = float(np.abs(adv.cpu().numpy().astype(np.float64) - ref["adv"].astype(np.float64)).max())
    if not adv_err <= 1e-5:
        raise RuntimeError(f"parity check: advantages differ by {adv_err}")
    R, tok_h = ref["R"], ref["token_offsets"]
    T = int(tok_h[-1])
    token_adv = torch.empty(T, dtype=torch.float32, device=dev)
    hora.hora_token_broadcast(torch.from_numpy(ref["adv"][:R].copy()).to(dev), torch.from_numpy(tok_h).to(dev), R, T,
                              token_adv)
    if not np.array_equal(token_adv.cpu().numpy().view(np.uint32), ref["token_adv"].view(np.uint32)):
        raise RuntimeError("parity check: token broadcast differs")
    return {"parity_checked": True, "prompts": n, "delta_differences": int(len(differ)),
            "band_differences": in_band, "adv_max_abs_err": adv_err, "tokens_compared": T}


REFERENCE_CPU_SECONDS = 150.0             # what the whole --impl reference run may cost
ORACLE_US_PER_PROMPT = 15.0               # measured on this machine's hosts at cfg4 (14.9 s for 2^20 prompts)


def reference_sample_size(steps: int, warmup: int, N: int):
    """Prompts per oracle step: the whole workload when steps + warm-up of it fit the time allowed for this arm,
    else the largest power of two that does.  Returns (n, reason)."""
    per_step = REFERENCE_CPU_SECONDS / max(1, steps + warmup)
    if N * ORACLE_US_PER_PROMPT * 1e-6 <= per_step:
        return N, "the whole workload per step"
    n = int(per_step / (ORACLE_US_PER_PROMPT * 1e-6))
    n = 1 << (max(n, 1).bit_length() - 1)
    n = max(1024, min(n, N))
    return n, (f"one oracle pass over all {N} prompts takes about {N * ORACLE_US_PER_PROMPT * 1e-6:.0f} s on one host core; "
               f"{steps} + {warmup} of them would take {(steps + warmup) * N * ORACLE_US_PER_PROMPT * 1e-6 / 60:.0f} min, so each "
               f"step covers the first {n} prompts (budget and tokens scaled); run with fewer steps (steps + warmup <= "
               f"{int(REFERENCE_CPU_SECONDS / (N * ORACLE_US_PER_PROMPT * 1e-6))}) for the whole workload per step")


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2605_07114_b200 import workloads as wl
    world = int(os.environ.get("WORLD_SIZE", "1"))
    w = wl.make(WORKLOAD, args.prompts, seed=shard_seed(0))
    steps, warm = args.steps, args.warmup
    n, why = reference_sample_size(steps, warm, w.N)
    for _ in range(warm):
        oracle_step(w, n)
    secs = [oracle_step(w, n) for _ in range(steps)]
    ms = 1e3 * sum(secs) / steps
    val = n / (ms * 1e-3)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": world, "steps": steps,
        "warmup": warm, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f80", "data": "synthetic",
        "config": {"workload": f"{WORKLOAD}: each step is the first {n} of {w.N} prompts (budget and tokens scaled), "
                               "CPU oracle, one host thread", "same_workload_as_repo_arm": n == w.N, "sample_reason": why},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": f"first {n} prompts of {WORKLOAD} per step"},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--prompts", type=int, default=None, help="override N (default: the workload's 2^20)")
    ap.add_argument("--cpu-sample", type=int, default=1 << 20)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--only", default=None, choices=["batched", "configs"],
                    help="run one secondary measurement alone and print its object (not the benchmark line)")
    ap.add_argument("--shards", type=int, default=65536, help="shards of the batched measurement")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
