"""Algorithm 1 around the library's calls.

`run_load_trace` drives the scheduling loop of Algorithm 1 on the GPU in load-trace mode: each
step routes the micro-batches that just advanced (eb_route with a route mask, so deferred ones
keep their routing), schedules (eb_schedule, result copied to the host to advance the layer
counters) and records the run set and the joint per-device load; the expert pass is skipped.
`run_full` does the same but executes every step completely (eb_permute, eb_expert_ffn_grouped,
eb_combine) and carries the hidden state with the residual h <- h + MLP(h) between layers.

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


def run_full(step: "B.MoEStep", tok_off: List[int], L: int, m: int, policy: int,
             logits_of: Callable[[int, int], torch.Tensor], x0: torch.Tensor,
             on_step: Optional[Callable[[int, Dict], None]] = None) -> Dict:
    """Runs Algorithm 1 executing every step in full.  `x0` bf16 [T_tot, H] are the hidden states
    entering layer 0.  After a step the chosen micro-batches take h <- h + MLP(h) (the residual
    of the transformer block; attention is outside the method).  Returns the final hidden
    states and the step records."""
    N = len(tok_off) - 1
    T = tok_off[-1]
    layer = [0] * N
    pool = (1 << N) - 1 if L > 0 else 0
    route_mask = pool
    step.x[:T].copy_(x0)
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
        step.eb_permute(batch)
        step.eb_expert_ffn_grouped()
        step.eb_combine(batch)
        rec = dict(pool=pool, run_mask=run, layers={j: layer[j] for j in range(N) if (run >> j) & 1},
                   joint_load=res["joint_load"], util_num=res["util_num"], util_den=res["util_den"])
        steps.append(rec)
        if on_step is not None:
            on_step(len(steps) - 1, rec)
        route_mask = 0
        for j in range(N):
            if (run >> j) & 1:
                a, b = tok_off[j], tok_off[j + 1]
                step.x[a:b].add_(step.out[a:b])          # residual; plain elementwise plumbing between steps
                layer[j] += 1
                if layer[j] >= L:
                    pool &= ~(1 << j)
                else:
                    route_mask |= 1 << j
    torch.cuda.synchronize()
    return dict(x=step.x[:T].clone(), steps=steps)


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
    """Median time (ms) of the expert-pass kernels (gate/up and down, single-CTA and CTA-pair launches)
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
