"""Shared helpers of the GPU parity tests: build a seeded case, run the oracle and the CUDA
library on the same bytes, compare stage by stage."""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from oracle import eb_oracle as O
from paper_2608_07964_b200 import synth

# elementwise bar for expert outputs: |gpu - ref| <= 2e-2 * max|ref| + 1e-3
REL, ABS = 2e-2, 1e-3


def within_bar(gpu: np.ndarray, ref: np.ndarray) -> bool:
    if ref.size == 0:
        return True
    return bool((np.abs(gpu.astype(np.float64) - ref.astype(np.float64)) <= REL * np.abs(ref).max() + ABS).all())


def worst(gpu: np.ndarray, ref: np.ndarray) -> float:
    if ref.size == 0:
        return 0.0
    return float(np.abs(gpu.astype(np.float64) - ref).max() / (REL * np.abs(ref).max() + ABS))


@dataclass
class Case:
    wl: synth.Workload
    tok_off: List[int]
    layers: List[int]
    logits: torch.Tensor      # cpu f32 [T_tot, E]
    x: torch.Tensor           # cpu bf16 [T_tot, H]

    @property
    def T_tot(self):
        return self.tok_off[-1]


def make_case(wl: synth.Workload, tokens: Optional[Sequence[int]] = None, layers: Optional[Sequence[int]] = None,
              device="cpu") -> Case:
    tokens = [wl.T] * wl.N if tokens is None else list(tokens)
    layers = wl.layers if layers is None else list(layers)
    tok_off = [0]
    for t in tokens:
        tok_off.append(tok_off[-1] + t)
    bias = synth.zipf_bias(wl)
    lg = [synth.logits_for(wl, j, layers[j], device, bias, T=tokens[j]) for j in range(len(tokens))]
    xs = [synth.hidden_for(wl, j, layers[j], device, T=tokens[j]) for j in range(len(tokens))]
    logits = torch.cat(lg, 0) if lg else torch.zeros((0, wl.E))
    x = torch.cat(xs, 0) if xs else torch.zeros((0, wl.H), dtype=torch.bfloat16)
    return Case(wl, tok_off, layers, logits.cpu(), x.cpu())


class WeightStore:
    """Expert weights on the GPU (bound to the library) with per-expert CPU copies for the oracle."""

    def __init__(self, wl: synth.Workload, device="cuda"):
        self.wl = wl
        self.gate = synth.all_weights(wl, "gate", device)
        self.up = synth.all_weights(wl, "up", device)
        self.down = synth.all_weights(wl, "down", device)

    def get(self, w: int):
        n = self.wl.E + self.wl.S
        l, e = divmod(w, n)
        f = lambda t: t[l, e].float().cpu().numpy()
        return f(self.gate), f(self.up), f(self.down)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy()


def oracle_front(case: Case, pool_mask: int, m: int, policy: int):
    """Oracle route + schedule + permute."""
    wl = case.wl
    dev = wl.expert_to_device()
    idx, w, mb_load, mb_cnt = O.route(case.logits.numpy(), wl.K, dev, wl.D, case.tok_off, bool(wl.renorm_topk))
    sched = O.schedule(mb_load, pool_mask, m, policy)
    goff, gw, row_src, pos, xp_bits, groups = O.permute(bf16_bits(case.x), idx, sched["run_mask"], case.layers,
                                                        case.tok_off, dev, wl.E, wl.K, wl.S, wl.D)
    return dict(idx=idx, w=w, mb_load=mb_load, mb_cnt=mb_cnt, sched=sched, group_off=goff, group_w=gw,
                row_src=row_src, pos=pos, xp_bits=xp_bits, groups=groups)


def check_front(step, case: Case, ref: Dict, n_mb: int):
    """Bit-exact comparison of routing, schedule and permutation outputs already on the GPU."""
    wl = case.wl
    T = case.T_tot
    assert np.array_equal(step.topk_idx[:T].cpu().numpy(), ref["idx"]), "top-k indices"
    assert np.allclose(step.topk_w[:T].cpu().numpy(), ref["w"], rtol=0, atol=1e-6), "gate weights"
    assert np.array_equal(step.mb_load[:n_mb].cpu().numpy(), ref["mb_load"]), "per-device loads"
    assert np.array_equal(step.mb_cnt[:n_mb].cpu().numpy(), ref["mb_cnt"]), "per-expert counts"
    got = step.sched_result()
    for k in ("run_mask", "defer_mask", "n_run", "joint_load", "util_num", "util_den"):
        assert got[k] == ref["sched"][k], (k, got[k], ref["sched"][k])
    meta = step.meta()
    G, R = len(ref["group_w"]), int(ref["group_off"][-1])
    assert meta["groups"] == G and meta["rows"] == R
    assert np.array_equal(step.group_off[:G + 1].cpu().numpy(), ref["group_off"]), "group offsets"
    assert np.array_equal(step.group_w[:G].cpu().numpy(), ref["group_w"]), "group weight ids"
    assert np.array_equal(step.row_src[:R].cpu().numpy(), ref["row_src"]), "row sources"
    assert np.array_equal(step.pos[:T].cpu().numpy(), ref["pos"]), "positions"
    assert np.array_equal(bf16_bits(step.xp[:R]), ref["xp_bits"]), "gathered rows"
    # first group of every virtual device
    firsts = [next((g for g, (d, _, _) in enumerate(ref["groups"]) if d >= dd), G) for dd in range(wl.D)] + [G]
    assert meta["dev_group_off"] == firsts
