"""Seeded synthetic inputs for the cross-layer MoE step.

This module only *draws numbers*: it contains none of the method's arithmetic
(no gating, scheduling, permutation or expert math).  It is the one module the
tests hand to both the CPU oracle and the CUDA library, so that both see the
same bytes.

Every value is a pure function ``f(seed, tensor_id, element_index)`` built from
64-bit integer mixing, so any slice of any tensor can be produced on its own,
on the CPU or on a CUDA device, with identical bits:

* ``h = mix64(key + (index + 1) * GOLDEN)`` with the splitmix64 finaliser;
* an approximately normal integer ``s = lane0 + lane1 + lane2 + lane3 - 131070``
  from the four 16-bit lanes of ``h`` (Irwin-Hall, exact integer arithmetic,
  support about +-3.46 sigma);
* one fp32 multiply ``s * (sigma / 37837.2249...)`` (a single rounding), then a
  round-to-nearest-even cast where bf16 is asked for.

The workloads below are the shapes named by the benchmark configurations: they
stand in for routing traces of trained MoE models on long-context tasks (the
paper's Section 5 set-up), which are not available offline.  Router logits are
N(0,1) noise plus a per-layer expert bias ``-s * ln(rank)`` over a seeded
per-layer permutation of the experts, i.e. a Zipf(s)-shaped popularity whose
hot set is resampled for every layer.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Sequence

import numpy as np
import torch

BASE_SEED = 20260807

_MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB

KIND_X = 1
KIND_LOGIT = 2
KIND_W_GATE = 3
KIND_W_UP = 4
KIND_W_DOWN = 5
KIND_PERM = 6

# standard deviation of the sum of four independent uniform 16-bit integers
_LANE_VAR = (65536.0 ** 2 - 1.0) / 12.0
_IH4_STD = math.sqrt(4.0 * _LANE_VAR)
_IH4_MEAN = 4 * 65535 // 2  # 131070


def _s64(v: int) -> int:
    """Two's-complement view of an unsigned 64-bit value as a Python int."""
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def mix64_int(z: int) -> int:
    """splitmix64 finaliser on a Python integer (unsigned 64-bit)."""
    z &= _MASK64
    z = ((z ^ (z >> 30)) * _M1) & _MASK64
    z = ((z ^ (z >> 27)) * _M2) & _MASK64
    return z ^ (z >> 31)


def stream_key(seed: int, tensor_id: int) -> int:
    """Key of the number stream of one tensor."""
    return mix64_int((seed * _GOLDEN + tensor_id * _M1 + 0x1234567) & _MASK64)


def tensor_id(kind: int, layer: int = 0, mb: int = 0) -> int:
    return kind | (layer << 8) | (mb << 24)


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of int64 values holding unsigned 64-bit patterns."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def _mix64_t(z: torch.Tensor) -> torch.Tensor:
    z = (z ^ _lsr(z, 30)) * _s64(_M1)
    z = (z ^ _lsr(z, 27)) * _s64(_M2)
    return z ^ _lsr(z, 31)


def _ih4(key: int, start: int, count: int, device) -> torch.Tensor:
    """Centred Irwin-Hall(4) integers for elements [start, start+count)."""
    idx = torch.arange(start + 1, start + 1 + count, dtype=torch.int64, device=device)
    h = _mix64_t(idx * _s64(_GOLDEN) + _s64(key))
    s = (h & 0xFFFF) + (_lsr(h, 16) & 0xFFFF) + (_lsr(h, 32) & 0xFFFF) + _lsr(h, 48)
    return s - _IH4_MEAN


def normal_f32(seed: int, tid: int, start: int, count: int, sigma: float = 1.0,
               device="cpu", chunk: int = 1 << 24) -> torch.Tensor:
    """fp32 values ~ N(0, sigma^2) (Irwin-Hall(4) shape) for a slice of a stream."""
    key = stream_key(seed, tid)
    scale = float(np.float32(sigma / _IH4_STD))
    out = torch.empty(count, dtype=torch.float32, device=device)
    for c0 in range(0, count, chunk):
        n = min(chunk, count - c0)
        s = _ih4(key, start + c0, n, device)
        out[c0:c0 + n] = s.to(torch.float32) * scale
    return out


def normal_bf16(seed: int, tid: int, start: int, count: int, sigma: float = 1.0,
                device="cpu", chunk: int = 1 << 24, out: torch.Tensor | None = None) -> torch.Tensor:
    """bf16 (round-to-nearest-even of the fp32 draw) slice of a stream."""
    key = stream_key(seed, tid)
    scale = float(np.float32(sigma / _IH4_STD))
    if out is None:
        out = torch.empty(count, dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    for c0 in range(0, count, chunk):
        n = min(chunk, count - c0)
        s = _ih4(key, start + c0, n, device)
        flat[c0:c0 + n] = (s.to(torch.float32) * scale).to(torch.bfloat16)
    return out


def seeded_permutation(seed: int, tid: int, n: int) -> List[int]:
    """Fisher-Yates shuffle of range(n) driven by the integer hash."""
    key = stream_key(seed, tid)
    p = list(range(n))
    for i in range(n - 1, 0, -1):
        r = mix64_int((key + (i + 1) * _GOLDEN) & _MASK64) % (i + 1)
        p[i], p[r] = p[r], p[i]
    return p


@dataclass(frozen=True)
class Workload:
    """One benchmark configuration: model shape, virtual devices, micro-batches."""
    name: str
    L: int           # MoE layers
    E: int           # routed experts per layer
    K: int           # experts per token
    S: int           # always-on shared experts per layer
    H: int           # hidden size
    I: int           # expert intermediate size
    D: int           # virtual expert-parallel devices
    mapping: str     # "contiguous" or "mod"
    N: int           # micro-batches
    T: int           # tokens per micro-batch
    zipf_s: float    # routing skew
    renorm_topk: int = 1
    seed: int = BASE_SEED
    layers_override: tuple | None = None
    m_override: int | None = None

    @property
    def n_weight_mats(self) -> int:
        return self.L * (self.E + self.S)

    @property
    def m(self) -> int:
        """Minimum combination size: ceil(0.75 N), the upper end of the suggested range."""
        if self.m_override is not None:
            return self.m_override
        return -(-3 * self.N // 4)

    @property
    def layers(self) -> List[int]:
        """Staggered current layer of each micro-batch: floor(j L / N)."""
        if self.layers_override is not None:
            return list(self.layers_override)
        return [(j * self.L) // self.N for j in range(self.N)]

    @property
    def tok_off(self) -> List[int]:
        return [j * self.T for j in range(self.N + 1)]

    @property
    def T_tot(self) -> int:
        return self.N * self.T

    def expert_to_device(self) -> List[int]:
        if self.mapping == "mod":
            return [e % self.D for e in range(self.E)]
        if self.mapping == "contiguous":
            return [(e * self.D) // self.E for e in range(self.E)]
        raise ValueError(self.mapping)

    def weight_bytes(self) -> int:
        return 3 * self.n_weight_mats * self.H * self.I * 2


def workload(name: str, **over) -> Workload:
    base = {
        # 4 layers x 8 experts, top-2, 4 devices x 2 experts, 4 x 64 tokens at layers 0..3
        "c1": dict(L=4, E=8, K=2, S=0, H=256, I=512, D=4, mapping="contiguous", N=4, T=64, zipf_s=1.0),
        # decode-like: 60 routed + 4 shared experts, top-4, e mod 8, 8 x 32 tokens
        "c2": dict(L=24, E=60, K=4, S=4, H=2048, I=1408, D=8, mapping="mod", N=8, T=32, zipf_s=1.2),
        # fine-grained: 64 routed + 2 shared, top-6, contiguous, 16 x 512 tokens
        "c3": dict(L=26, E=64, K=6, S=2, H=2048, I=1408, D=8, mapping="contiguous", N=16, T=512, zipf_s=0.8),
        # large experts: 8 experts, top-2, 1 expert per device, 8 x 1024 tokens (~90 GB of weights)
        "c4": dict(L=32, E=8, K=2, S=0, H=4096, I=14336, D=8, mapping="contiguous", N=8, T=1024, zipf_s=1.0),
    }[name]
    base.update(over)
    return Workload(name=name, **base)


def workload_c5(N: int, T: int, s: float, **over) -> Workload:
    """One point of the skew / micro-batch-count sweep."""
    base = dict(L=8, E=64, K=6, S=0, H=2048, I=1408, D=8, mapping="contiguous", N=N, T=T, zipf_s=s)
    base.update(over)
    return Workload(name=f"c5_N{N}_T{T}_s{s}", **base)


def zipf_bias(wl: Workload) -> np.ndarray:
    """fp32 table [L, E]: -s * ln(rank_l(e)), rank from a seeded per-layer shuffle."""
    tab = np.zeros((wl.L, wl.E), dtype=np.float64)
    for l in range(wl.L):
        perm = seeded_permutation(wl.seed, tensor_id(KIND_PERM, l), wl.E)
        for pos, e in enumerate(perm):
            tab[l, e] = -wl.zipf_s * math.log(pos + 1.0)
    return tab.astype(np.float32)


def logits_for(wl: Workload, mb: int, layer: int, device="cpu", bias: np.ndarray | None = None,
               T: int | None = None) -> torch.Tensor:
    """Router logits fp32 [T, E] of micro-batch `mb` when it sits at `layer`."""
    if bias is None:
        bias = zipf_bias(wl)
    T = wl.T if T is None else T
    n = normal_f32(wl.seed, tensor_id(KIND_LOGIT, layer, mb), 0, T * wl.E, 1.0, device)
    b = torch.from_numpy(bias[layer]).to(device)
    return n.view(T, wl.E) + b


def packed_logits(wl: Workload, layers: Sequence[int] | None = None, device="cpu") -> torch.Tensor:
    """fp32 [T_tot, E]: logits of every micro-batch at its current layer, packed."""
    layers = wl.layers if layers is None else layers
    bias = zipf_bias(wl)
    return torch.cat([logits_for(wl, j, layers[j], device, bias) for j in range(wl.N)], dim=0)


def hidden_for(wl: Workload, mb: int, layer: int, device="cpu", T: int | None = None) -> torch.Tensor:
    """Hidden states bf16 [T, H] ~ N(0,1) of micro-batch `mb` entering `layer`."""
    T = wl.T if T is None else T
    return normal_bf16(wl.seed, tensor_id(KIND_X, layer, mb), 0, T * wl.H, 1.0, device).view(T, wl.H)


def packed_hidden(wl: Workload, layers: Sequence[int] | None = None, device="cpu") -> torch.Tensor:
    layers = wl.layers if layers is None else layers
    return torch.cat([hidden_for(wl, j, layers[j], device) for j in range(wl.N)], dim=0)


_W_KIND = {"gate": KIND_W_GATE, "up": KIND_W_UP, "down": KIND_W_DOWN}


def expert_weight(wl: Workload, which: str, layer: int, e: int, device="cpu") -> torch.Tensor:
    """One expert matrix, bf16 ~ N(0, 0.02^2): [I, H] for gate/up, [H, I] for down.

    `e` indexes routed experts 0..E-1 then shared experts E..E+S-1.  The slice is
    bit-identical to the same rows of `all_weights`.
    """
    per = wl.H * wl.I
    start = (layer * (wl.E + wl.S) + e) * per
    t = normal_bf16(wl.seed, tensor_id(_W_KIND[which]), start, per, 0.02, device)
    return t.view(wl.I, wl.H) if which != "down" else t.view(wl.H, wl.I)


def all_weights(wl: Workload, which: str, device="cpu") -> torch.Tensor:
    """Full weight tensor bf16: [L, E+S, I, H] (gate, up) or [L, E+S, H, I] (down)."""
    n = wl.n_weight_mats * wl.H * wl.I
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    chunk = 1 << 26 if str(device).startswith("cuda") else 1 << 24
    normal_bf16(wl.seed, tensor_id(_W_KIND[which]), 0, n, 0.02, device, chunk=chunk, out=out)
    if which == "down":
        return out.view(wl.L, wl.E + wl.S, wl.H, wl.I)
    return out.view(wl.L, wl.E + wl.S, wl.I, wl.H)
