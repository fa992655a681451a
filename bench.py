#!/usr/bin/env python
"""Benchmark of one cross-layer MoE step (route -> schedule -> permute -> grouped expert FFN ->
combine) on seeded synthetic inputs shaped like the benchmark configurations.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4] [--impl ours|reference]

Prints ONE JSON line.  The default workload is the large-expert shape (the largest single-GPU configuration);
the decode, fine-grained and layer-0 shapes are reported compactly under detail.other_workloads.  `value` is tokens of the chosen micro-batches per second with all inputs
resident in HBM; `e2e` is the same with pinned host buffers, every step copying its inputs in and its result
out inside the timed region, two steps in flight (eb_step_host_submit / eb_step_host_wait;
`e2e.one_step_at_a_time` is the blocking eb_step_host).  With N > 1 (torchrun) every rank runs an independent replica
on its own seeded batch (no collective on the data path); rank 0 reports the aggregate.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2608_07964_b200 import synth  # noqa: E402

METRIC = "cross-layer MoE step tokens/s"
UNIT = "tokens/s"
# Kernels per step: route, schedule, permute (one fused kernel or four, plus the gather), expert pass 4 (plan, fill,
# gate/up, down), combine 1.  bench counts them from the library's own launch counter.

# DRAM traffic of the dominant kernel (ffn gate/up) from an ncu capture: (dram__bytes_read.sum +
# dram__bytes_write.sum) over the algorithmic bytes of the captured launch.  The captures ran on cut-down cases
# of the same shapes (a full-size capture would hold tens of GB); traffic grows in proportion to the weight
# bytes streamed, so a full launch is that ratio times its own algorithmic bytes.
NCU_TRAFFIC_RATIO = {"c4": 4.093019 / 3.909091, "c4small": 4.093019 / 3.909091,          # captured on c4small
                     "c2": 1.495264 / 1.487012, "c2small": 1.495264 / 1.487012,          # captured on c2small
                     "c3init": 1.170937 / 1.101005, "c3initsmall": 1.170937 / 1.101005}  # captured on c3initsmall


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=d["hbm_gbs"], tensor=d["bf16_tflops"], tensor_sustained=d["bf16_tflops_sustained"], src="measured")
    return dict(hbm=6650.0, tensor=1590.0, tensor_sustained=1400.0, src="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        sm, pw, mx, reasons = [], [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.lines:
            f = [v.strip() for v in line.split(",")]
            if len(f) < 7:
                continue
            try:
                clk, mxc = float(f[0]), float(f[1])
            except ValueError:
                continue
            mx = mxc
            if t0 - 0.05 <= ts <= t1 + 0.15:
                sm.append(clk)
                try:
                    pw.append(float(f[2]))
                except ValueError:
                    pass
                for n, v in zip(names, f[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
        if not sm:
            sm = [float(l.split(",")[0]) for _, l in self.lines[-3:] if l and l.split(",")[0].strip().replace(".", "").isdigit()]
        out = dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=mx, reasons=sorted(reasons), samples=len(sm))
        if pw:
            out["power_w"] = statistics.median(pw)
        return out


def timed(fn, reps: int):
    """CUDA-event time of `reps` back-to-back calls on the current stream, in ms."""
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record()
    for _ in range(reps):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b)


def make_inputs(wl, device):
    logits = synth.packed_logits(wl, device=device)
    x = synth.packed_hidden(wl, device=device)
    return logits, x


def algorithmic_bytes(wl, group_off, group_w, n_groups):
    """Bytes and flops one expert pass needs at least: every weight matrix that has rows is read once (the
    replicas of a shared expert on the virtual devices are one matrix in memory), every row once in and out."""
    sizes = np.diff(group_off[:n_groups + 1])
    active = int((sizes > 0).sum())
    distinct = int(len(set(group_w[:n_groups][sizes > 0].tolist())))
    R = int(sizes.sum())
    w = wl.H * wl.I * 2
    return dict(active_groups=active, distinct_matrices=distinct, rows=R,
                gateup=distinct * 2 * w + R * wl.H * 2 + R * wl.I * 2,
                down=distinct * w + R * wl.I * 2 + R * wl.H * 2,
                gateup_flops=4.0 * wl.H * wl.I * R, down_flops=2.0 * wl.H * wl.I * R)


# ----------------------------------------------------------------------------------------------
def oracle_step_sample(wl, logits, x, weights_bf16_cpu, budget_s: float):
    """The oracle's whole step on the CPU; the expert pass covers the first groups that fit the
    time budget and the other stages are scaled to the same share of rows."""
    from oracle import eb_oracle as O
    dev = wl.expert_to_device()
    t = {}
    t0 = time.perf_counter()
    idx, w, mb_load, mb_cnt = O.route(logits, wl.K, dev, wl.D, wl.tok_off, bool(wl.renorm_topk))
    t["route"] = time.perf_counter() - t0
    t0 = time.perf_counter()
    sched = O.schedule(mb_load, (1 << wl.N) - 1, wl.m, O.POLICY_MAXUTIL)
    t["schedule"] = time.perf_counter() - t0
    t0 = time.perf_counter()
    goff, gw, row_src, pos, xp, groups = O.permute(x, idx, sched["run_mask"], wl.layers, wl.tok_off, dev,
                                                   wl.E, wl.K, wl.S, wl.D)
    t["permute"] = time.perf_counter() - t0
    R = int(goff[-1])
    get = lambda wi: tuple(a.float().numpy() for a in weights_bf16_cpu(wi))
    y = np.zeros((R, wl.H), dtype=np.float32)
    t0 = time.perf_counter()
    rows_done = 0
    groups_done = 0
    for g in range(len(gw)):
        r0, r1 = int(goff[g]), int(goff[g + 1])
        if r1 > r0:
            wg, wu, wd = get(int(gw[g]))
            y[r0:r1] = O.swiglu_mlp(xp[r0:r1], wg, wu, wd)
            rows_done = r1
            groups_done += 1
        if time.perf_counter() - t0 > budget_s:
            break
    t["ffn"] = time.perf_counter() - t0
    t0 = time.perf_counter()
    O.combine(y, pos, w, wl.K, wl.S)
    t["combine"] = time.perf_counter() - t0
    share = rows_done / max(R, 1)
    tokens_run = sum(wl.T for j in range(wl.N) if (sched["run_mask"] >> j) & 1)
    total = t["ffn"] + share * (t["route"] + t["schedule"] + t["permute"] + t["combine"])
    return dict(tokens=tokens_run * share, seconds=total, share=share, groups=groups_done, rows=rows_done,
                rows_total=R, stages=t)


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info()]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def lazy_cpu_weights(wl, device):
    """Callable giving one expert's (gate, up, down) as CPU bf16 tensors, generated on demand."""
    cache = {}

    def get(wi):
        if wi not in cache:
            l, e = divmod(wi, wl.E + wl.S)
            cache[wi] = tuple(synth.expert_weight(wl, k, l, e, device).cpu() for k in ("gate", "up", "down"))
        return cache[wi]
    return get


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    gen_dev = "cuda" if torch.cuda.is_available() else "cpu"
    logits, x = make_inputs(wl, gen_dev)
    logits = logits.cpu().numpy()
    x = x.float().cpu().numpy()
    get = lazy_cpu_weights(wl, gen_dev)
    budget = max(1.0, min(10.0, 150.0 / max(1, args.steps + args.warmup)))
    # stage the weights of the groups the sample will touch outside the timed region
    r = oracle_step_sample(wl, logits, x, get, budget)
    for _ in range(max(0, args.warmup - 1)):
        r = oracle_step_sample(wl, logits, x, get, budget)
    tok = sec = 0.0
    for _ in range(args.steps):
        r = oracle_step_sample(wl, logits, x, get, budget)
        tok += r["tokens"]
        sec += r["seconds"]
    value = tok / sec if sec > 0 else 0.0
    sample = (f"oracle whole step on {wl.name}; expert pass over the first {r['groups']} non-empty groups "
              f"({r['rows']} of {r['rows_total']} rows) within {budget:.0f} s, other stages scaled to that share")
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps, warmup=args.warmup,
                ms_per_step=1000.0 * sec / max(1, args.steps), higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f32", data="synthetic", impl="reference",
                config=workload_config(wl),
                cpu_baseline=dict(value=value, unit=UNIT, cores=cpu_threads(), kind="oracle", sample=sample),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


def replica_workload(wl, rank: int):
    """Independent replicas: every rank draws its own batch, routing and weights."""
    return synth.Workload(**{**wl.__dict__, "seed": wl.seed + rank}) if rank else wl


def reduce_over_ranks(dist, device, ms: float, ms_e2e: float, tokens: float):
    """Max over ranks of the two device times, sum over ranks of the tokens processed."""
    if dist is None:
        return ms, ms_e2e, tokens
    v = torch.tensor([ms, ms_e2e], device=device, dtype=torch.float64)
    dist.all_reduce(v, op=dist.ReduceOp.MAX)
    tk = torch.tensor([tokens], device=device, dtype=torch.float64)
    dist.all_reduce(tk, op=dist.ReduceOp.SUM)
    return v[0].item(), v[1].item(), tk.item()


def workload_config(wl):
    return dict(workload=f"{wl.name}: L={wl.L} E={wl.E} K={wl.K} S={wl.S} H={wl.H} I={wl.I} D={wl.D} "
                         f"map={wl.mapping} N={wl.N}x{wl.T} tokens at layers {wl.layers} m={wl.m} zipf_s={wl.zipf_s}",
                policy="MaxUtil", seed=wl.seed,
                l2=("inputs larger than L2: each step streams the touched expert weights (GBs) from HBM"
                    if wl.weight_bytes() > (1 << 30) else
                    "small workload: all weights fit in L2 and no flush is done, figures are L2-warm"))


# ----------------------------------------------------------------------------------------------
def roof_of(nbytes, flops, ms, peaks):
    """Roofline entry of one launch: the bound is whichever of bytes / HBM bandwidth and flops / tensor peak
    takes longer with the measured peaks; achieved and frac are in that bound's unit."""
    t = ms / 1e3
    if nbytes / (peaks["hbm"] * 1e9) >= flops / (peaks["tensor"] * 1e12):
        ach = nbytes / t / 1e9
        d = dict(bound="hbm", achieved=ach, peak=peaks["hbm"], unit="GB/s", frac=ach / peaks["hbm"])
    else:
        ach = flops / t / 1e12
        d = dict(bound="tensor", achieved=ach, peak=peaks["tensor"], unit="TFLOP/s", frac=ach / peaks["tensor"])
    d.update(ms=ms, algorithmic_bytes=nbytes, algorithmic_flops=flops, peak_source=peaks["src"])
    return d


def measure(args, wl, device, local, dist, full):
    """One workload on this rank: device-resident step time, per-kernel times, rooflines, idle block; with
    `full` also the clock samples, the end-to-end figure and the CPU baseline.  Frees its device memory."""
    from paper_2608_07964_b200 import binding as B
    peaks = measured_peaks()
    step = B.from_workload(wl, device=device)
    wg, wu, wd = (synth.all_weights(wl, k, device) for k in ("gate", "up", "down"))
    step.bind_weights(wg, wu, wd)
    logits, x = make_inputs(wl, device)
    T = wl.T_tot
    step.logits[:T].copy_(logits)
    step.x[:T].copy_(x)
    batch = B.Batch(wl.tok_off, wl.layers)
    m = wl.m
    run = lambda: step.eb_step(batch, m)
    captured = None
    if args.graph:
        run()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        captured0 = B.launch_count()
        with torch.cuda.graph(graph):
            step.eb_step(batch, m)
        captured = B.launch_count() - captured0     # kernel nodes of one step
        run = graph.replay

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing
    for _ in range(args.warmup):
        run()
    barrier()
    sampler = ClockSampler(local)
    if full:
        sampler.start()
        time.sleep(0.25)
    t0 = time.time()
    launches0 = B.launch_count()
    ms = timed(run, args.steps)
    launches = B.launch_count() - launches0
    if captured is not None:
        launches = captured * args.steps
    t1 = time.time()
    clocks = sampler.stop(t0, t1) if full else None
    barrier()
    status = step.device_status()
    sched = step.sched_result()
    tokens_run = sum(wl.T for j in range(wl.N) if (sched["run_mask"] >> j) & 1)

    # ---- per-kernel durations (events inside the library around every launch), same steps again
    step.set_timing(True)
    per = {}
    for _ in range(args.steps):
        run()
        for k, v in step.kernel_ms().items():
            per.setdefault(k, []).append(v)
    step.set_timing(False)
    kern_ms = {k: sum(v) / len(v) for k, v in per.items()}

    res = dict(wl=wl, ms=ms, launches=launches, clocks=clocks, status=status, sched=sched, tokens_run=tokens_run,
               kern_ms=kern_ms, ms_e2e=float("nan"), ms_e2e_blocking=float("nan"))

    # ---- the same step in a loop of about 1.5 s: on a 1 kW part the K timed steps above finish before the power
    # controller has settled, so the sustained figure is reported beside them (not the headline: the contract times K steps)
    res["sustained"] = None
    if full and args.sustain_s > 0:
        n_batch = max(10, int(0.1 / max(ms / args.steps / 1e3, 1e-6)))       # about 0.1 s per batch
        sampler2 = ClockSampler(local)
        sampler2.start()
        time.sleep(0.25)
        s0 = time.time()
        batches = []
        while time.time() - s0 < args.sustain_s:
            batches.append(timed(run, n_batch) / n_batch)
        s1 = time.time()
        tail = batches[len(batches) // 2:]                                   # the settled half
        res["sustained"] = dict(ms_per_step=sum(tail) / len(tail), first_batch_ms_per_step=batches[0], seconds=s1 - s0,
                                steps=n_batch * len(batches), clocks=sampler2.stop(s0 + (s1 - s0) / 2, s1))

    # ---- end to end with host buffers
    if full:
        h_logits = logits.cpu().pin_memory()
        h_x = x.cpu().pin_memory()
        h_out = torch.empty((T, wl.H), dtype=torch.bfloat16).pin_memory()
        run_host = lambda: step.eb_step_host(batch, m, h_logits, h_x, h_out)
        side = torch.cuda.Stream()      # a stream of its own: the legacy default stream adds implicit synchronisation
        side.wait_stream(torch.cuda.current_stream())
        # the same with two steps in flight (eb_step_host_submit / eb_step_host_wait): the copies of one step overlap
        # the kernels of the other; every step still copies its inputs in and its result out inside the timed region
        depth = 2
        h_outs = [torch.empty((T, wl.H), dtype=torch.bfloat16).pin_memory() for _ in range(depth)]

        def run_pipelined(n):
            for i in range(n):
                s = i % depth
                if i >= depth:
                    step.step_host_wait(s)
                step.step_host_submit(s, batch, m, h_logits, h_x, h_outs[s])
            for s in range(min(depth, n)):
                step.step_host_wait(s)

        with torch.cuda.stream(side):
            for _ in range(max(args.warmup, 3)):
                run_host()
            barrier()
            res["ms_e2e_blocking"] = timed(run_host, args.steps)
            run_pipelined(max(args.warmup, 3))
            barrier()
            res["ms_e2e"] = timed(lambda: run_pipelined(args.steps), 1)
        barrier()
        for h in h_outs:      # rows of deferred micro-batches are not written by a step
            for j in range(wl.N):
                if (sched["run_mask"] >> j) & 1:
                    a, b = wl.tok_off[j], wl.tok_off[j + 1]
                    assert torch.equal(h[a:b], h_out[a:b]), "pipelined host path disagrees with the blocking one"

    # ---- algorithmic work and rooflines of the two expert launches
    meta = step.meta()
    alg = algorithmic_bytes(wl, step.group_off.cpu().numpy(), step.group_w.cpu().numpy(), meta["groups"])
    t_gu, t_dn = kern_ms.get("ffn_gateup", float("nan")), kern_ms.get("ffn_down", float("nan"))
    roofs = dict(ffn_gateup=roof_of(alg["gateup"], alg["gateup_flops"], t_gu, peaks),
                 ffn_down=roof_of(alg["down"], alg["down_flops"], t_dn, peaks))
    ffn_flops = alg["gateup_flops"] + alg["down_flops"]
    ffn_bytes = alg["gateup"] + alg["down"]
    t_ffn = (t_gu + t_dn) / 1e3
    move = 2 * (tokens_run * wl.H + alg["rows"] * wl.H)      # gather: read T_run rows, write R rows; combine the reverse
    t_g, t_c = kern_ms.get("permute_gather", float("nan")) / 1e3, kern_ms.get("combine", float("nan")) / 1e3
    res.update(alg=alg, roofs=roofs, extra=dict(
        kernel_ms=kern_ms, launches=roofs,
        ffn=dict(tflops=ffn_flops / t_ffn / 1e12, frac_tensor_peak=ffn_flops / t_ffn / 1e12 / peaks["tensor"],
                 frac_tensor_sustained=ffn_flops / t_ffn / 1e12 / peaks["tensor_sustained"],
                 gbs=ffn_bytes / t_ffn / 1e9, frac_hbm=ffn_bytes / t_ffn / 1e9 / peaks["hbm"],
                 active_groups=alg["active_groups"], distinct_matrices=alg["distinct_matrices"], rows=alg["rows"]),
        front_end_ms=sum(v for k, v in kern_ms.items() if not k.startswith("ffn_gate") and not k.startswith("ffn_down")),
        permute_gather=dict(bytes=move, gbs=move / t_g / 1e9, frac_hbm=move / t_g / 1e9 / peaks["hbm"],
                            frac_hbm_nominal_8tbs=move / t_g / 1e9 / 8000.0),
        combine=dict(bytes=move, gbs=move / t_c / 1e9, frac_hbm=move / t_c / 1e9 / peaks["hbm"],
                     frac_hbm_nominal_8tbs=move / t_c / 1e9 / 8000.0)))
    res["idle"] = idle_report(step, batch, wl, sched, B) if dist is None and not args.no_idle else None

    res["cpu"] = None
    if not full and dist is None and not args.no_cpu_baseline and wl.name in ("c1", "c2"):
        # small shapes: the oracle's whole step with all host threads and with one (a few seconds each)
        from threadpoolctl import threadpool_limits
        get = lazy_cpu_weights(wl, device)
        lg, xx = logits.cpu().numpy(), x.float().cpu().numpy()
        oracle_step_sample(wl, lg, xx, get, 1.0)          # stages the sampled weights on the host
        r = oracle_step_sample(wl, lg, xx, get, 4.0)
        with threadpool_limits(limits=1):
            r1 = oracle_step_sample(wl, lg, xx, get, 4.0)
        res["cpu"] = dict(value=r["tokens"] / r["seconds"], unit=UNIT, cores=cpu_threads(), kind="oracle",
                          rows=f"{r['rows']} of {r['rows_total']}", single_thread_value=r1["tokens"] / r1["seconds"],
                          single_thread_rows=f"{r1['rows']} of {r1['rows_total']}")
    if full and dist is None and not args.no_cpu_baseline:
        get = lazy_cpu_weights(wl, device)
        lg, xx = logits.cpu().numpy(), x.float().cpu().numpy()
        oracle_step_sample(wl, lg, xx, get, 4.0)          # stages the sampled weights on the host
        r = oracle_step_sample(wl, lg, xx, get, 12.0)
        res["cpu"] = dict(value=r["tokens"] / r["seconds"], unit=UNIT, cores=cpu_threads(), kind="oracle",
                          sample=(f"oracle whole step; expert pass over the first {r['groups']} non-empty groups "
                                  f"({r['rows']} of {r['rows_total']} rows), other stages scaled to that share; "
                                  f"{r['seconds']:.1f} s of CPU work"),
                          stage_seconds={k: round(v, 4) for k, v in r["stages"].items()})
    step.close()
    del wg, wu, wd, step
    torch.cuda.empty_cache()
    return res


def compact(res, peaks):
    """Sub-line of a secondary workload."""
    wl, ex = res["wl"], res["extra"]
    ms_step = res["ms"] / res["steps"]
    g = ex["launches"]["ffn_gateup"]
    return dict(workload=workload_config(wl)["workload"], ms_per_step=ms_step,
                tokens_per_s=res["tokens_run"] / (ms_step / 1e3), device_status=res["status"],
                gateup=dict(bound=g["bound"], frac=g["frac"], ms=g["ms"]),
                down=dict(bound=ex["launches"]["ffn_down"]["bound"], frac=ex["launches"]["ffn_down"]["frac"],
                          ms=ex["launches"]["ffn_down"]["ms"]),
                expert_pass_tflops=ex["ffn"]["tflops"], expert_pass_frac_burst=ex["ffn"]["frac_tensor_peak"],
                expert_pass_frac_sustained=ex["ffn"]["frac_tensor_sustained"], expert_pass_frac_hbm=ex["ffn"]["frac_hbm"],
                front_end_ms=ex["front_end_ms"], gather_gbs=ex["permute_gather"]["gbs"], combine_gbs=ex["combine"]["gbs"],
                idle=res["idle"], cpu_baseline=res["cpu"])


def run_ours(args, wl):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    local = local % max(1, torch.cuda.device_count())
    if world > 1:
        import torch.distributed as dist
        if args.dist_backend == "nccl":
            dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
        else:
            dist.init_process_group(args.dist_backend)
    torch.cuda.set_device(local)
    device = f"cuda:{local}"
    red_device = device if args.dist_backend == "nccl" else "cpu"   # where the timing reductions live
    wl = replica_workload(wl, rank)
    peaks = measured_peaks()

    res = measure(args, wl, device, local, dist, full=True)
    res["steps"] = args.steps

    # ---- reductions over ranks
    ms_max, ms_e2e_max, tok_total = reduce_over_ranks(dist, red_device, res["ms"], res["ms_e2e"], float(res["tokens_run"]))
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    T = wl.T_tot
    ms_step = ms_max / args.steps
    value = tok_total / (ms_step / 1e3)
    # dominant kernel: the gate/up launch of the grouped expert FFN
    roof = dict(res["roofs"]["ffn_gateup"])
    roof.update(kernel="ffn_gateup",
                traffic=(NCU_TRAFFIC_RATIO[wl.name] * roof["algorithmic_bytes"] if wl.name in NCU_TRAFFIC_RATIO else None))
    extra = res["extra"]
    if res["sustained"]:
        su = res["sustained"]
        flops = res["alg"]["gateup_flops"] + res["alg"]["down_flops"]
        # share of the step the two expert launches take in the K-step run (their event times over the step time)
        share = min(1.0, (res["kern_ms"].get("ffn_gateup", 0.0) + res["kern_ms"].get("ffn_down", 0.0)) / ms_step)
        su["tokens_per_s"] = res["tokens_run"] / (su["ms_per_step"] / 1e3)
        # expert pass of the settled loop (same share of the step) against the sustained GEMM peak
        su["expert_pass_tflops"] = flops / (su["ms_per_step"] * share / 1e3) / 1e12
        su["expert_pass_frac_of_sustained_peak"] = su["expert_pass_tflops"] / peaks["tensor_sustained"]
        extra["sustained"] = su
    if world == 1 and args.others:
        extra["other_workloads"] = {}
        for name in args.others.split(","):
            sub = measure(args, named_workload(name), device, local, None, full=False)
            sub["steps"] = args.steps
            extra["other_workloads"][name] = compact(sub, peaks)

    h2d = T * wl.E * 4 + T * wl.H * 2
    d2h = T * wl.H * 2 + 96
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                ms_per_step=ms_step, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16",
                data="synthetic", config=workload_config(wl), clocks=res["clocks"],
                e2e=dict(value=tok_total / (ms_e2e_max / args.steps / 1e3), unit=UNIT, h2d_bytes_per_step=h2d,
                         d2h_bytes_per_step=d2h, mode="host buffers, 2 steps in flight (eb_step_host_submit/_wait)",
                         one_step_at_a_time=res["tokens_run"] / (res["ms_e2e_blocking"] / args.steps / 1e3)),
                gpu_launches=res["launches"], roofline=roof, cpu_baseline=res["cpu"],
                tokens_per_step=tok_total, run_mask=res["sched"]["run_mask"], device_status=res["status"],
                idle=res["idle"], detail=extra)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def idle_report(step, batch, wl, sched, B):
    """Virtual-device idle fraction of the step, cross-layer versus each chosen micro-batch alone.

    Token based: 1 - sum(W) / (D max(W)) from the routed loads.  Time based: the expert pass is run
    on each virtual device's contiguous group range by itself (median of 5) and the same formula is
    applied to the times (expert-pass kernels only, from the library's per-kernel events); 'per layer' runs
    every chosen micro-batch's workload alone."""
    D = wl.D
    run = [j for j in range(wl.N) if (sched["run_mask"] >> j) & 1]
    loads = step.mb_load[:wl.N].cpu().numpy().astype(np.int64)
    joint = loads[run].sum(axis=0)
    tok_cross = 1.0 - joint.sum() / (D * joint.max()) if joint.max() else 0.0
    alone_cap = D * sum(int(loads[j].max()) for j in run)
    tok_alone = 1.0 - joint.sum() / alone_cap if alone_cap else 0.0

    from paper_2608_07964_b200 import driver
    device_times = lambda: driver.device_times(step, D, reps=5)

    step.eb_step(batch, wl.m)
    t_cross = device_times()
    busy = cap = 0.0
    for j in run:
        one = B.Batch(wl.tok_off, wl.layers, 1 << j)
        step.eb_schedule(one, 1, B.POLICY_ALL)
        step.eb_permute(one)
        tj = device_times()
        busy += sum(tj)
        cap += D * max(tj)
    step.eb_step(batch, wl.m)
    torch.cuda.synchronize()
    # what the emulated expert-parallel step costs is the slowest device's time: lead with that.  On shapes whose
    # groups stream their weights (few rows per expert) a device's time follows the experts it touches, not its
    # tokens, so the time-based idle fraction need not fall even though the slowest device gets faster.
    return dict(step_max_ms_cross_layer=max(t_cross), sum_max_ms_per_layer=cap / D,
                max_device_time_ratio=max(t_cross) / (cap / D) if cap else None,
                token_cross_layer=tok_cross, token_per_layer=tok_alone,
                time_cross_layer=1.0 - sum(t_cross) / (D * max(t_cross)),
                time_per_layer=1.0 - busy / cap if cap else 0.0,
                device_ms_cross_layer=t_cross)


def named_workload(name):
    if name == "c3init":
        # Algorithm 1's first step on the fine-grained shape: every micro-batch at layer 0 (tensor-bound groups)
        wl = synth.workload("c3", layers_override=tuple([0] * 16))
    elif name == "c3initsmall":
        # c3init with the model cut to 2 layers (2.3 GB of weights): same kernels and tile shapes, small enough for ncu
        wl = synth.workload("c3", L=2, layers_override=tuple([0] * 16))
    elif name == "c4small":
        # the large-expert shape cut to 2 layers and 2 micro-batches (5.6 GB of weights): small enough for ncu
        wl = synth.workload("c4", L=2, N=2, m_override=2)
    elif name == "c2small":
        # the decode shape cut to 6 layers and 6 micro-batches (6.6 GB of weights): the case ncu captures run on
        wl = synth.workload("c2", L=6, N=6)
    else:
        return synth.workload(name)
    return synth.Workload(**{**wl.__dict__, "name": name})


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4", choices=["c1", "c2", "c2small", "c3", "c3init", "c3initsmall", "c4", "c4small"],
                    help="the workload of the JSON line; c4 (large experts, 90 GB of weights) is the largest single-GPU one")
    ap.add_argument("--others", default=None,
                    help="comma-separated workloads reported compactly under detail.other_workloads "
                         "(default: c2,c3,c3init when the main workload is c4; 'none' for none)")
    ap.add_argument("--graph", action="store_true", help="replay the step from a captured CUDA graph")
    ap.add_argument("--dist-backend", default="nccl", choices=["nccl", "gloo"],
                    help="process-group backend for the barrier and the timing reductions (replicas share no data)")
    ap.add_argument("--sustain-s", type=float, default=1.5,
                    help="seconds of the same step in a loop after the timed region, reported under detail.sustained (0: off)")
    ap.add_argument("--no-idle", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.others is None:
        args.others = "c2,c3,c3init" if args.workload == "c4" else ""
    if args.others == "none":
        args.others = ""
    wl = named_workload(args.workload)
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
