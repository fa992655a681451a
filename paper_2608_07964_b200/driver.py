"""Algorithm 1 around the library's calls.

`run_load_trace` drives the scheduling loop of Algorithm 1 on the GPU in load-trace mode: each
step routes the micro-batches that just advanced (eb_route with a route mask, so deferred ones
keep their routing), schedules (eb_schedule, result copied to the host to advance the layer
counters) and records the run set and the joint per-device load; the expert pass is skipped.
`run_full` does the same but executes every step completely (eb_step: the five calls, the last one adding
the residual h <- h + MLP(h) in place), optionally replaying each step from a CUDA graph.

Logits of (micro-batch j, layer l) come from a caller-supplied function, so the loop itself holds
no routing or scheduling arithmetic: those run in the CUDA kernels.
"""
from __future__ import annotations

from typing import Callable, Dict, List, Optional

import torch

from . import binding as B


def run_load_trace(step: "B.MoEStep", tok_off: List[int], L: int, m: int, policy: int,
                   logits_of: Callable[[int, int], torch.Tensor]) -> List[Dict]:
    """Runs Algorithm 1 with route + schedule only.  Returns one record per step:
    pool, run_mask, layers of the run set, joint_load, util_num, util_den, member_loads."""
    N = len(tok_off) - 1
    layer = [0] * N
    pool = (1 << N) - 1 if L > 0 else 0
    route_mask = pool
    steps: List[Dict] = []
    while pool:
        for j in range(N):
            if (route_mask >> j) & 1:
                step.logits[tok_off[j]:tok_off[j + 1]].copy_(logits_of(j, layer[j]))
        batch = B.Batch(tok_off, [min(l, L - 1) for l in layer], pool)
        if route_mask:
            step.eb_route(batch, route_mask)
        res = step.eb_schedule(batch, m, policy, to_host=True)
        run = res["run_mask"]
        loads = step.mb_load[:N].cpu().tolist()
        steps.append(dict(pool=pool, run_mask=run, layers={j: layer[j] for j in range(N) if (run >> j) & 1},
                          joint_load=res["joint_load"], util_num=res["util_num"], util_den=res["util_den"],
                          member_loads={j: loads[j] for j in range(N) if (run >> j) & 1}))
        route_mask = 0
        for j in range(N):
            if (run >> j) & 1:
                layer[j] += 1
                if layer[j] >= L:
                    pool &= ~(1 << j)
                else:
                    route_mask |= 1 << j
    return steps


class StepGraphs:
    """CUDA graphs of whole steps, one per distinct (pool, layers, route mask, m, policy): a step's launches are
    fixed by those host-side values (which micro-batches run is read from device memory by the kernels), so a
    state that comes up again - the same schedule trajectory on the next batch - is replayed as one graph
    launch instead of about a dozen kernel launches."""

    def __init__(self, step: "B.MoEStep", tok_off: List[int], capacity: int = 256):
        self.step, self.tok_off, self.capacity = step, list(tok_off), capacity
        self.graphs: Dict = {}
        self.hits = self.captures = 0

    def run(self, layers: List[int], pool: int, route_mask: int, m: int, policy: int):
        key = (pool, tuple(layers), route_mask, m, policy)
        g = self.graphs.get(key)
        if g is None:
            if len(self.graphs) >= self.capacity:
                self.graphs.pop(next(iter(self.graphs)))
            batch = B.Batch(self.tok_off, layers, pool)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                self.step.eb_step(batch, m, policy, route_mask, in_place=True)
            g = self.graphs[key] = (graph, batch)
            self.captures += 1
        else:
            self.hits += 1
        g[0].replay()


def run_full(step: "B.MoEStep", tok_off: List[int], L: int, m: int, policy: int,
             logits_of: Callable[[int, int], torch.Tensor], x0: torch.Tensor,
             on_step: Optional[Callable[[int, Dict], None]] = None, graphs: Optional[StepGraphs] = None) -> Dict:
    """Runs Algorithm 1 executing every step in full.  `x0` bf16 [T_tot, H] are the hidden states
    entering layer 0.  A step is one eb_step call whose aggregation adds the residual in place: the chosen
    micro-batches take h <- h + MLP(h) (Section 2.1; attention is outside the method), so no arithmetic
    happens outside the library.  With `graphs` every step is replayed from (or first captured into) a CUDA
    graph.  Returns the final hidden states, the step records and the device time of the whole run."""
    N = len(tok_off) - 1
    T = tok_off[-1]
    layer = [0] * N
    pool = (1 << N) - 1 if L > 0 else 0
    route_mask = pool
    step.x[:T].copy_(x0)
    steps: List[Dict] = []
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    while pool:
        for j in range(N):
            if (route_mask >> j) & 1:
                step.logits[tok_off[j]:tok_off[j + 1]].copy_(logits_of(j, layer[j]))
        lay = [min(l, L - 1) for l in layer]
        if graphs is not None:
            graphs.run(lay, pool, route_mask, m, policy)
        else:
            step.eb_step(B.Batch(tok_off, lay, pool), m, policy, route_mask, in_place=True)
        res = step.sched_result()          # the host needs the run set to advance the layer counters
        run = res["run_mask"]
        rec = dict(pool=pool, run_mask=run, layers={j: layer[j] for j in range(N) if (run >> j) & 1},
                   joint_load=res["joint_load"], util_num=res["util_num"], util_den=res["util_den"])
        steps.append(rec)
        if on_step is not None:
            on_step(len(steps) - 1, rec)
        route_mask = 0
        for j in range(N):
            if (run >> j) & 1:
                layer[j] += 1
                if layer[j] >= L:
                    pool &= ~(1 << j)
                else:
                    route_mask |= 1 << j
    t1.record()
    torch.cuda.synchronize()
    return dict(x=step.x[:T].clone(), steps=steps, ms=t0.elapsed_time(t1), token_layers=T * L)


def peak_device(load: List[int]) -> int:
    """Device with the largest load; the lowest index among equal maxima (an all-zero workload peaks on device 0)."""
    best = 0
    for d in range(1, len(load)):
        if load[d] > load[best]:
            best = d
    return best


def same_peak_windows(loads_by_layer: List[List[int]], n: int):
    """(count, windows): in how many of the L - n + 1 windows of n consecutive layers the workload peaks on one
    and the same device - the worst case of cross-layer combination (Section 4.1), the statistic of the paper's
    table on consecutive layers with identical skew."""
    peaks = [peak_device(w) for w in loads_by_layer]
    windows = max(len(peaks) - n + 1, 0)
    return sum(1 for l in range(windows) if len(set(peaks[l:l + n])) == 1), windows


def routed_loads(step: "B.MoEStep", tok_off: List[int], L: int,
                 logits_of: Callable[[int, int], torch.Tensor]) -> List[List[List[int]]]:
    """loads[j][l] = per-device load vector of micro-batch j at layer l, routed by eb_route."""
    N = len(tok_off) - 1
    out = [[None] * L for _ in range(N)]
    for l in range(L):
        for j in range(N):
            step.logits[tok_off[j]:tok_off[j + 1]].copy_(logits_of(j, l))
        step.eb_route(B.Batch(tok_off, [l] * N))
        loads = step.mb_load[:N].cpu().tolist()
        for j in range(N):
            out[j][l] = loads[j]
    return out


def idle_fractions(steps: List[Dict], D: int) -> Dict[str, float]:
    """Under-utilisation 1 - u of a recorded run: cross-layer (one term per step) and the same
    workloads each executed alone."""
    work = sum(s["util_num"] for s in steps)
    cap = sum(s["util_den"] for s in steps)
    out = dict(steps=len(steps), idle_cross_layer=(1.0 - work / cap) if cap else 0.0)
    if steps and "member_loads" in steps[0]:
        alone = D * sum(max(w) for s in steps for w in s["member_loads"].values())
        out["idle_each_alone"] = (1.0 - work / alone) if alone else 0.0
    return out


def device_times(step: "B.MoEStep", D: int, reps: int = 3) -> List[float]:
    """Median time (ms) of the expert-pass kernels (gate/up and down)
    restricted to each virtual device's groups, from the library's per-kernel CUDA events; the tile-list
    construction that precedes them is not counted."""
    out = []
    step.set_timing(True)
    try:
        for d in range(D):
            step.eb_expert_ffn_grouped(device=d)                   # warm the path
            ts = []
            for _ in range(reps):
                step.eb_expert_ffn_grouped(device=d)
                k = step.kernel_ms()
                ts.append(sum(v for name, v in k.items() if name.startswith(("ffn_gateup", "ffn_down"))))
            out.append(sorted(ts)[len(ts) // 2])
    finally:
        step.set_timing(False)
    return out


def run_emulated_latency(step: "B.MoEStep", tok_off: List[int], L: int, D: int, m: int, policy: int,
                         logits_of: Callable[[int, int], torch.Tensor], x0: torch.Tensor,
                         alone: bool = False) -> Dict:
    """Expert-parallel latency of a whole run as the virtual devices would see it.

    Every step is routed, scheduled and permuted by the library; the expert pass is then timed on each
    virtual device's groups by itself, and a step costs the slowest device (the others idle until the
    gather, Section 2.3).  Returns the summed step latency, the summed busy time and the resulting
    time-based under-utilisation 1 - sum(busy) / (D * sum(max)).  With `alone` every (micro-batch,
    layer) workload is executed by itself (no combination at all)."""
    N = len(tok_off) - 1
    T = tok_off[-1]
    layer = [0] * N
    pool = (1 << N) - 1 if L > 0 else 0
    route_mask = pool
    step.x[:T].copy_(x0)
    lat = busy = 0.0
    n_steps = 0
    while pool:
        for j in range(N):
            if (route_mask >> j) & 1:
                step.logits[tok_off[j]:tok_off[j + 1]].copy_(logits_of(j, layer[j]))
        lay = [min(l, L - 1) for l in layer]
        if route_mask:
            step.eb_route(B.Batch(tok_off, lay, pool), route_mask)
        if alone:
            j0 = min(j for j in range(N) if (pool >> j) & 1 and layer[j] == min(layer[i] for i in range(N) if (pool >> i) & 1))
            batch = B.Batch(tok_off, lay, 1 << j0)
            run = step.eb_schedule(batch, 1, B.POLICY_ALL, to_host=True)["run_mask"]
        else:
            batch = B.Batch(tok_off, lay, pool)
            run = step.eb_schedule(batch, m, policy, to_host=True)["run_mask"]
        step.eb_permute(batch)
        t = device_times(step, D)
        lat += max(t)
        busy += sum(t)
        n_steps += 1
        route_mask = 0
        for j in range(N):
            if (run >> j) & 1:
                layer[j] += 1
                if layer[j] >= L:
                    pool &= ~(1 << j)
                else:
                    route_mask |= 1 << j
    return dict(steps=n_steps, latency_ms=lat, busy_ms=busy, idle_time=1.0 - busy / (D * lat) if lat else 0.0)
