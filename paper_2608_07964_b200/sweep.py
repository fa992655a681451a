"""Skew / micro-batch sweep on the 64-expert, top-6, hidden-2048 shape (8 layers, 8 virtual devices).

    python -m paper_2608_07964_b200.sweep [--out results.md] [--policy 0] [--ep | --msweep | --latency | --sched | --whole | --front]

For every point (Zipf s, micro-batch count N, tokens per micro-batch T) it reports
  * whole-run under-utilisation 1 - u of Algorithm 1 driven on the GPU (route + schedule every
    step): cross-layer with m = ceil(0.75 N) and m = ceil(0.5 N), against every workload executed
    alone and against lock-step execution (all micro-batches jointly, layer by layer);
  * time and tokens/s of one full cross-layer step at the staggered state l_j = floor(j L / N).
All arithmetic of the method runs in the library's kernels; this module only loops and prints.
"""
from __future__ import annotations

import argparse
import sys

import torch

from . import binding as B
from . import driver, synth


def timed_ms(fn, reps=5, warm=2):
    for _ in range(warm):
        fn()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record()
    for _ in range(reps):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / reps


def ep_size_sweep(args, dev, weights):
    """Expert-parallel size sweep at constant per-device tokens (the paper's Table 4 set-up: batch grows
    with the number of devices), N = 4 micro-batches and m = 3 as in the paper's default; plus how often a
    micro-batch's workload peaks on the same device in N consecutive layers (the paper's Table 2 statistic).
    Peak devices are read off the load vectors eb_route produced."""
    lines = ["| s | D | tokens per micro-batch | idle EB (MaxUtil) | idle EB (CumUtil) | idle EB (DiffPeak) | idle alone | idle lock-step | same peak, 2 layers | same peak, 3 layers |",
             "|---|---|---|---|---|---|---|---|---|---|"]
    for s in (0.5, 1.0):
        for D in (2, 4, 8):
            wl = synth.workload_c5(4, 64 * D, s, D=D, m_override=3)
            bias = synth.zipf_bias(wl)
            step = B.from_workload(wl, device=dev)
            step.bind_weights(*weights)
            logits_of = lambda j, l: synth.logits_for(wl, j, l, dev, bias)
            res = {}
            for name, pol in (("max", B.POLICY_MAXUTIL), ("cum", B.POLICY_CUMUTIL), ("diff", B.POLICY_DIFFPEAK)):
                res[name] = driver.idle_fractions(driver.run_load_trace(step, wl.tok_off, wl.L, wl.m, pol, logits_of), D)
            lock = driver.idle_fractions(driver.run_load_trace(step, wl.tok_off, wl.L, wl.N, B.POLICY_ALL, logits_of), D)
            # how often a micro-batch's workload keeps its peak device over 2 and 3 consecutive layers
            loads = driver.routed_loads(step, wl.tok_off, wl.L, logits_of)
            same2 = sum(driver.same_peak_windows(loads[j], 2)[0] for j in range(wl.N))
            same3 = sum(driver.same_peak_windows(loads[j], 3)[0] for j in range(wl.N))
            lines.append(f"| {s} | {D} | {wl.T} | {res['max']['idle_cross_layer']:.3f} | {res['cum']['idle_cross_layer']:.3f} | "
                         f"{res['diff']['idle_cross_layer']:.3f} | {res['max']['idle_each_alone']:.3f} | {lock['idle_cross_layer']:.3f} | "
                         f"{same2}/{wl.N * (wl.L - 1)} | {same3}/{wl.N * (wl.L - 2)} |")
            step.close()
            print(lines[-1], flush=True)
    return lines


def latency_report(args, dev):
    """Emulated expert-parallel MoE latency of a whole Algorithm-1 run: cross-layer scheduling (the three
    policies) against lock-step execution and against every workload alone; per step the cost is the
    slowest virtual device's expert pass."""
    lines = ["| shape | N x T | policy | steps | MoE latency ms (sum of slowest device) | time idle | vs alone | vs lock-step |",
             "|---|---|---|---|---|---|---|---|"]
    shapes = [("c5 s=1.0 (64 experts, top-6, 8 layers)", synth.workload_c5(4, 1024, 1.0, m_override=3)),
              ("c5 s=1.0", synth.workload_c5(8, 512, 1.0)),
              ("c4 cut to 8 layers (8 experts, top-2, H 4096, I 14336)", synth.workload("c4", L=8, N=4, T=2048, m_override=3))]
    for label, wl in shapes:
        bias = synth.zipf_bias(wl)
        step = B.from_workload(wl, device=dev)
        weights = tuple(synth.all_weights(wl, k, dev) for k in ("gate", "up", "down"))
        step.bind_weights(*weights)
        logits_of = lambda j, l: synth.logits_for(wl, j, l, dev, bias)
        x0 = torch.cat([synth.hidden_for(wl, j, 0, dev) for j in range(wl.N)], 0)
        res = {}
        res["alone"] = driver.run_emulated_latency(step, wl.tok_off, wl.L, wl.D, 1, B.POLICY_ALL, logits_of, x0, alone=True)
        res["lock-step"] = driver.run_emulated_latency(step, wl.tok_off, wl.L, wl.D, wl.N, B.POLICY_ALL, logits_of, x0)
        for name, pol in (("MaxUtil", B.POLICY_MAXUTIL), ("CumUtil", B.POLICY_CUMUTIL), ("DiffPeak", B.POLICY_DIFFPEAK)):
            res[name] = driver.run_emulated_latency(step, wl.tok_off, wl.L, wl.D, wl.m, pol, logits_of, x0)
        for name, r in res.items():
            lines.append(f"| {label} | {wl.N} x {wl.T} | {name} | {r['steps']} | {r['latency_ms']:.2f} | {r['idle_time']:.3f} | "
                         f"{r['latency_ms'] / res['alone']['latency_ms']:.2f} | {r['latency_ms'] / res['lock-step']['latency_ms']:.2f} |")
            print(lines[-1], flush=True)
        assert step.device_status() == 0
        step.close()
        del weights
        torch.cuda.empty_cache()
    return lines


def schedule_latency_report(args, dev):
    """Time of one Schedule(S, m) call per policy (CUDA events, mean of 200 back-to-back calls) on routed
    loads of the 64-expert shape; the paper's Table 3 reports 0.13-0.28 ms per step on its host."""
    lines = ["| micro-batches N | m | MaxUtil us | CumUtil us | DiffPeak us |", "|---|---|---|---|---|"]
    for N in (4, 8, 16):
        wl = synth.workload_c5(N, 128, 1.0)
        step = B.from_workload(wl, device=dev)
        step.logits[:wl.T_tot].copy_(synth.packed_logits(wl, device=dev))
        batch = B.Batch(wl.tok_off, wl.layers)
        step.eb_route(batch)
        row = []
        for pol in (B.POLICY_MAXUTIL, B.POLICY_CUMUTIL, B.POLICY_DIFFPEAK):
            row.append(1000.0 * timed_ms(lambda: step.eb_schedule(batch, wl.m, pol), reps=200, warm=5))
        lines.append(f"| {N} | {wl.m} | {row[0]:.1f} | {row[1]:.1f} | {row[2]:.1f} |")
        print(lines[-1], flush=True)
        step.close()
    return lines


def whole_run_report(args, dev):
    """Whole Algorithm-1 runs executed in full on the benchmark shapes (every step one eb_step with the residual
    added in place): device time and token-layers per second for cross-layer scheduling (MaxUtil, m = ceil(0.75 N)),
    for lock-step execution (all micro-batches jointly, layer by layer) and with each step replayed from a CUDA
    graph; plus the emulated expert-parallel latency (per step the slowest virtual device's expert pass) and the
    time-based idle fraction of cross-layer scheduling, lock-step execution and every workload alone."""
    lines = ["| shape | policy | steps | whole-run ms | token-layers/s | same, steps replayed from CUDA graphs | emulated EP latency ms | time idle |",
             "|---|---|---|---|---|---|---|---|"]
    for name in ("c3", "c4"):
        wl = synth.workload(name)
        bias = synth.zipf_bias(wl)
        step = B.from_workload(wl, device=dev)
        weights = tuple(synth.all_weights(wl, k, dev) for k in ("gate", "up", "down"))
        step.bind_weights(*weights)
        logits_of = lambda j, l: synth.logits_for(wl, j, l, dev, bias)
        # random-weight blocks without the normalisation layers of a real model grow the hidden state layer by
        # layer; a twentieth of the unit scale keeps 26 to 32 of them finite (timing does not depend on the values)
        x0 = (torch.cat([synth.hidden_for(wl, j, 0, dev) for j in range(wl.N)], 0).float() * 0.05).to(torch.bfloat16)
        for label, m, pol in (("cross-layer MaxUtil", wl.m, B.POLICY_MAXUTIL), ("lock-step", wl.N, B.POLICY_ALL)):
            driver.run_full(step, wl.tok_off, wl.L, m, pol, logits_of, x0)                       # warm
            r = driver.run_full(step, wl.tok_off, wl.L, m, pol, logits_of, x0)
            graphs = driver.StepGraphs(step, wl.tok_off, capacity=4096)
            driver.run_full(step, wl.tok_off, wl.L, m, pol, logits_of, x0, graphs=graphs)       # captures
            rg = driver.run_full(step, wl.tok_off, wl.L, m, pol, logits_of, x0, graphs=graphs)  # replays
            same = torch.equal(r["x"].view(torch.int16), rg["x"].view(torch.int16))
            finite = bool(torch.isfinite(r["x"].float()).all())
            assert same and finite, (label, same, finite)
            lat = driver.run_emulated_latency(step, wl.tok_off, wl.L, wl.D, m, pol, logits_of, x0)
            lines.append(f"| {name} | {label} (m = {m}) | {len(r['steps'])} | {r['ms']:.1f} | {r['token_layers'] / r['ms'] * 1e3:.3e} | "
                         f"{rg['ms']:.1f} ms, {rg['token_layers'] / rg['ms'] * 1e3:.3e} | {lat['latency_ms']:.2f} | {lat['idle_time']:.3f} |")
            print(lines[-1], flush=True)
        lat = driver.run_emulated_latency(step, wl.tok_off, wl.L, wl.D, 1, B.POLICY_ALL, logits_of, x0, alone=True)
        lines.append(f"| {name} | every workload alone | {lat['steps']} | - | - | - | {lat['latency_ms']:.2f} | {lat['idle_time']:.3f} |")
        print(lines[-1], flush=True)
        assert step.device_status() == 0
        step.close()
        del weights
        torch.cuda.empty_cache()
    return lines


def front_end_steps(args, dev, weights):
    """A few whole steps at N = 4, 8, 16 micro-batches of 16 tokens (the fused permutation path), for a launch
    list: the scheduling and permutation kernels' durations are read off a profiler's per-launch times."""
    for N in (4, 8, 16):
        wl = synth.workload_c5(N, 16, 1.0)
        step = B.from_workload(wl, device=dev)
        step.bind_weights(*weights)
        step.logits[:wl.T_tot].copy_(synth.packed_logits(wl, device=dev))
        step.x[:wl.T_tot].copy_(synth.packed_hidden(wl, device=dev))
        batch = B.Batch(wl.tok_off, wl.layers)
        ms = timed_ms(lambda: step.eb_step(batch, wl.m), reps=5, warm=3)
        assert step.device_status() == 0
        print(f"N={N} m={wl.m} step {ms:.3f} ms", flush=True)
        step.close()
    return []


def m_sweep(args, dev, weights):
    """Minimum combination size sweep (the paper's micro-batching ablation): for every micro-batch count N and
    every m from 1 to N, whole-run under-utilisation of Algorithm 1 under the three policies, the number of steps,
    and the ratio of effective to maximum workload summed over steps (max_d sum_j w_j against sum_j max_d w_j,
    the two curves of the paper's per-step plot)."""
    lines = ["| s | N | m | steps (MaxUtil) | idle MaxUtil | idle CumUtil | idle DiffPeak | idle alone | effective / maximum workload (MaxUtil) |",
             "|---|---|---|---|---|---|---|---|---|"]
    for s in (0.5, 1.0):
        for N in (2, 4, 8, 16):
            wl = synth.workload_c5(N, 128, s)
            bias = synth.zipf_bias(wl)
            step = B.from_workload(wl, device=dev)
            step.bind_weights(*weights)
            logits_of = lambda j, l: synth.logits_for(wl, j, l, dev, bias)
            for m in range(1, N + 1):
                res = {}
                for name, pol in (("max", B.POLICY_MAXUTIL), ("cum", B.POLICY_CUMUTIL), ("diff", B.POLICY_DIFFPEAK)):
                    tr = driver.run_load_trace(step, wl.tok_off, wl.L, m, pol, logits_of)
                    res[name] = (driver.idle_fractions(tr, wl.D), tr)
                tr = res["max"][1]
                eff = sum(max(st["joint_load"][:wl.D]) for st in tr)
                mx = sum(max(w) for st in tr for w in st["member_loads"].values())
                f = res["max"][0]
                lines.append(f"| {s} | {N} | {m} | {f['steps']} | {f['idle_cross_layer']:.3f} | {res['cum'][0]['idle_cross_layer']:.3f} | "
                             f"{res['diff'][0]['idle_cross_layer']:.3f} | {f['idle_each_alone']:.3f} | {eff / mx:.3f} |")
                print(lines[-1], flush=True)
            step.close()
    return lines


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default=None)
    ap.add_argument("--policy", type=int, default=B.POLICY_MAXUTIL)
    ap.add_argument("--quick", action="store_true", help="s in {0, 1.0}, N in {4, 16} only")
    ap.add_argument("--ep", action="store_true", help="expert-parallel size sweep instead of the skew sweep")
    ap.add_argument("--latency", action="store_true", help="emulated expert-parallel latency of whole runs")
    ap.add_argument("--sched", action="store_true", help="time of one scheduling call per policy")
    ap.add_argument("--msweep", action="store_true", help="minimum combination size sweep")
    ap.add_argument("--whole", action="store_true", help="whole Algorithm-1 runs executed in full on the benchmark shapes")
    ap.add_argument("--front", action="store_true", help="a few steps at N = 4, 8, 16 for a launch list of the small kernels")
    args = ap.parse_args(argv)
    dev = "cuda:0"
    if args.sched:
        text = "\n".join(schedule_latency_report(args, dev)) + "\n"
        if args.out:
            with open(args.out, "w") as f:
                f.write(text)
        return 0
    if args.whole:
        text = "\n".join(whole_run_report(args, dev)) + "\n"
        if args.out:
            with open(args.out, "w") as f:
                f.write(text)
        return 0
    if args.latency:
        text = "\n".join(latency_report(args, dev)) + "\n"
        if args.out:
            with open(args.out, "w") as f:
                f.write(text)
        return 0
    base = synth.workload_c5(2, 16, 0.0)
    weights = tuple(synth.all_weights(base, k, dev) for k in ("gate", "up", "down"))
    if args.front:
        front_end_steps(args, dev, weights)
        return 0
    if args.msweep:
        text = "\n".join(m_sweep(args, dev, weights)) + "\n"
        if args.out:
            with open(args.out, "w") as f:
                f.write(text)
        return 0
    if args.ep:
        text = "\n".join(ep_size_sweep(args, dev, weights)) + "\n"
        if args.out:
            with open(args.out, "w") as f:
                f.write(text)
        return 0
    svals = [0.0, 1.0] if args.quick else [0.0, 0.5, 1.0, 1.5]
    nvals = [4, 16] if args.quick else [2, 4, 8, 16]
    lines = ["| s | N | T | steps EB(.75) | idle EB m=.75N | idle EB m=.5N | idle alone | idle lock-step | step ms | step tokens/s | step run/N |",
             "|---|---|---|---|---|---|---|---|---|---|---|"]
    for s in svals:
        for N in nvals:
            for T in (16, 128, 1024):
                wl = synth.workload_c5(N, T, s)
                bias = synth.zipf_bias(wl)
                step = B.from_workload(wl, device=dev)
                step.bind_weights(*weights)
                logits_of = lambda j, l: synth.logits_for(wl, j, l, dev, bias)
                m75, m50 = wl.m, -(-N // 2)
                tr75 = driver.run_load_trace(step, wl.tok_off, wl.L, m75, args.policy, logits_of)
                tr50 = driver.run_load_trace(step, wl.tok_off, wl.L, m50, args.policy, logits_of)
                lock = driver.run_load_trace(step, wl.tok_off, wl.L, N, B.POLICY_ALL, logits_of)
                f75, f50, fl = (driver.idle_fractions(t, wl.D) for t in (tr75, tr50, lock))
                # one full step at the staggered state
                step.logits[:wl.T_tot].copy_(synth.packed_logits(wl, device=dev))
                step.x[:wl.T_tot].copy_(synth.packed_hidden(wl, device=dev))
                batch = B.Batch(wl.tok_off, wl.layers)
                ms = timed_ms(lambda: step.eb_step(batch, m75, args.policy))
                run = step.sched_result()["n_run"]
                assert step.device_status() == 0
                lines.append(f"| {s} | {N} | {T} | {f75['steps']} | {f75['idle_cross_layer']:.3f} | {f50['idle_cross_layer']:.3f} | "
                             f"{f75['idle_each_alone']:.3f} | {fl['idle_cross_layer']:.3f} | {ms:.3f} | {run * T / ms * 1e3:.0f} | {run}/{N} |")
                step.close()
                print(lines[-1], flush=True)
    text = "\n".join(lines) + "\n"
    if args.out:
        with open(args.out, "w") as f:
            f.write(text)
    return 0


if __name__ == "__main__":
    sys.exit(main())
