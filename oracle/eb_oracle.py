"""CPU oracle for one cross-layer MoE step of EasyBalance.  TEST INFRASTRUCTURE ONLY.

Plain, slow, written from the paper's definitions with numpy; it shares no code
with the CUDA library and imports nothing from it.  Only the test-suite, the
smoke check and the benchmark's CPU-baseline leg may call it.

What each function follows:

* ``route``        - Section 2.1, top-k gating ``W_l, I_l = topk(G(h'_l))`` with G = softmax,
                     and the per-device workload vector ``w in Z^D`` of Section 2.3.
* ``utilisation``  - Eq. 3 restricted to one step; ``effective_workload`` is Eq. 2.
* ``schedule``     - Section 4.2 (subset with ``|RunSet| >= m`` maximising utilisation, MaxUtil)
                     and Section 5.2 (CumUtil, DiffPeak), taken step by step.
* ``group_table`` / ``permute`` - the dispatch of Section 2.2 written as a stable grouping of
                     (token, expert) assignments by (virtual device, layer, expert).
* ``expert_ffn``   - ``expert_i(.)`` of Eq. 1 as a bias-free SwiGLU MLP.
* ``combine``      - Eq. 1, the weighted aggregation; optionally h_{l+1} = h'_l + MLP(h'_l) of Section 2.1.
* ``dense_masked_moe`` - Eq. 1 evaluated with every expert on every token and a 0/weight mask:
                     a brute-force cross-check that uses no permutation at all.
* ``run_algorithm1`` - Algorithm 1 on load vectors (which workloads run at which step).
* ``same_peak_windows`` - the count of N-consecutive layers with the same skew device (the paper's
                     table of worst-case occurrences, Section 4.1).
* ``idle_*``       - under-utilisation ``1 - u`` (Section 5, Metrics) for the cross-layer run,
                     for each workload executed alone, and for lock-step execution.

Readings taken where the paper is silent are listed in the repository's design notes.  Three of
them are choices the paper cannot confirm ("parity unpinned" in that sense): the placement of
shared experts (replicated on every virtual device, serving that device's home tokens, not
counted in scheduling loads), the MaxUtil tie rule (higher U, then larger set, then smaller
bitmask), and how CumUtil / DiffPeak are topped up to ``m`` members (best utilisation of the
union, ties to the lower index).  What each reading *is* is fixed by hand-worked examples in the
test-suite, so a slip in their code fails a test; that the paper means them is not checkable.

Floating point is fp32 by default (the precision the parity bar is stated in); every float
function takes ``dtype`` so the tests can repeat it in fp64 to bound the oracle's own error.
"""
from __future__ import annotations

from fractions import Fraction
from typing import Callable, Dict, List, Sequence, Tuple

import numpy as np

POLICY_MAXUTIL = 0
POLICY_CUMUTIL = 1
POLICY_DIFFPEAK = 2
POLICY_ALL = 3


# --------------------------------------------------------------------------- routing
def route(logits: np.ndarray, K: int, expert_to_device: Sequence[int], D: int,
          tok_off: Sequence[int], renorm_topk: bool = True, dtype=np.float32):
    """Top-k softmax gating (Section 2.1) and per-micro-batch loads (Section 2.3).

    Experts are ranked by (logit descending, index ascending); the K best are kept in that
    order.  Weights are softmax probabilities, renormalised over the K kept experts when
    `renorm_topk`, otherwise left as the full-softmax values.  The workload unit is one
    (token, expert) assignment: ``mb_load[j, d]`` counts the assignments of micro-batch j that
    land on device d, ``mb_cnt[j, e]`` those that land on expert e.
    """
    T, E = logits.shape
    n_mb = len(tok_off) - 1
    order = np.argsort(-logits, axis=1, kind="stable")       # ties -> lower index first
    idx = order[:, :K].astype(np.int32)
    z = logits.astype(dtype)
    zsel = np.take_along_axis(z, idx.astype(np.int64), axis=1)
    ztop = zsel[:, :1]
    p = np.exp(zsel - ztop)
    if renorm_topk:
        w = p / p.sum(axis=1, keepdims=True)
    else:
        w = p / np.exp(z - ztop).sum(axis=1, keepdims=True)
    mb_load = np.zeros((n_mb, D), dtype=np.int32)
    mb_cnt = np.zeros((n_mb, E), dtype=np.int32)
    dev = np.asarray(expert_to_device)
    for j in range(n_mb):
        sel = idx[tok_off[j]:tok_off[j + 1]].reshape(-1)
        np.add.at(mb_cnt[j], sel, 1)
        np.add.at(mb_load[j], dev[sel], 1)
    return idx, w.astype(dtype), mb_load, mb_cnt


# --------------------------------------------------------------------------- utilisation
def effective_workload(w: Sequence[int]) -> int:
    """Eq. 2: the bottleneck device's load."""
    return int(max(w)) if len(w) else 0


def utilisation(w: Sequence[int]) -> Tuple[int, int]:
    """Eq. 3 for a single step, as an exact fraction (num, den) = (sum_d w_d, D * max_d w_d)."""
    w = [int(v) for v in w]
    return sum(w), len(w) * effective_workload(w)


def _u_greater(a: Tuple[int, int], b: Tuple[int, int]) -> bool:
    """U_a > U_b by cross-multiplication; a zero denominator (no work) counts as U = 1."""
    an, ad = a if a[1] != 0 else (1, 1)
    bn, bd = b if b[1] != 0 else (1, 1)
    return an * bd > bn * ad


def _members(mask: int) -> List[int]:
    return [j for j in range(32) if (mask >> j) & 1]


def _joint(mb_load: np.ndarray, mask: int) -> List[int]:
    D = mb_load.shape[1]
    tot = [0] * D
    for j in _members(mask):
        for d in range(D):
            tot[d] += int(mb_load[j, d])
    return tot


def _peak_device(w: Sequence[int]) -> int:
    """argmax_d with the lowest device index among equal maxima."""
    best = 0
    for d in range(1, len(w)):
        if w[d] > w[best]:
            best = d
    return best


def _fill_to_m(mb_load, chosen: int, pool: int, m: int) -> int:
    """Top-up rule for the O(n) policies: while fewer than m members are chosen, add the pool
    member whose inclusion gives the highest utilisation (lowest index on ties)."""
    while bin(chosen).count("1") < m:
        best_j, best_u = -1, None
        for j in _members(pool & ~chosen):
            u = utilisation(_joint(mb_load, chosen | (1 << j)))
            if best_u is None or _u_greater(u, best_u):
                best_j, best_u = j, u
        if best_j < 0:
            break
        chosen |= 1 << best_j
    return chosen


def schedule(mb_load: np.ndarray, pool_mask: int, m: int, policy: int = POLICY_MAXUTIL) -> Dict:
    """One call of Schedule(S, m) in Algorithm 1.

    MaxUtil (Section 4.2): every subset A of the pool with |A| >= m is scored by the
    utilisation of the summed load vector; the best wins, ties going to the larger subset and
    then to the numerically smaller bitmask.  If the pool has at most m members all of them run.
    CumUtil / DiffPeak (Section 5.2): pool members are visited in ascending index, the first is
    always taken, the next is taken iff it strictly raises utilisation / iff its peak device is
    not yet among the peak devices of the members taken so far.
    """
    mb_load = np.asarray(mb_load)
    pool = _members(pool_mask)
    if len(pool) <= m or policy == POLICY_ALL:
        run = pool_mask
    elif policy == POLICY_MAXUTIL:
        cands = []
        for sub in range(1, 1 << len(pool)):
            mask = sum(1 << j for b, j in enumerate(pool) if (sub >> b) & 1)
            if bin(mask).count("1") >= m:
                cands.append(mask)
        member = np.array([[(mask >> j) & 1 for j in range(mb_load.shape[0])] for mask in cands], dtype=np.int64)
        joint_all = member @ mb_load.astype(np.int64)            # summed load vector of every candidate
        D = mb_load.shape[1]

        def rank(i):
            num, peak = int(joint_all[i].sum()), int(joint_all[i].max())
            u = Fraction(num, D * peak) if peak > 0 else Fraction(1)
            return (u, bin(cands[i]).count("1"), -cands[i])

        run = cands[max(range(len(cands)), key=rank)]
    elif policy == POLICY_CUMUTIL:
        run = 1 << pool[0]
        for j in pool[1:]:
            if _u_greater(utilisation(_joint(mb_load, run | (1 << j))), utilisation(_joint(mb_load, run))):
                run |= 1 << j
        run = _fill_to_m(mb_load, run, pool_mask, m)
    elif policy == POLICY_DIFFPEAK:
        run = 1 << pool[0]
        peaks = {_peak_device(mb_load[pool[0]])}
        for j in pool[1:]:
            pk = _peak_device(mb_load[j])
            if pk not in peaks:
                run |= 1 << j
                peaks.add(pk)
        run = _fill_to_m(mb_load, run, pool_mask, m)
    else:
        raise ValueError(policy)
    joint = _joint(mb_load, run)
    num, den = utilisation(joint)
    return dict(run_mask=run, defer_mask=pool_mask & ~run, n_run=bin(run).count("1"),
                joint_load=joint, util_num=num, util_den=den)


# --------------------------------------------------------------------------- grouping
def group_table(run_mask: int, layers: Sequence[int], expert_to_device: Sequence[int],
                E: int, S: int, D: int) -> List[Tuple[int, int, int]]:
    """Groups (device, layer, expert slot) of one step, device-major.

    Active layers are the distinct current layers of the selected micro-batches, ascending.
    For each device, for each active layer: the routed experts hosted by the device (ascending),
    then shared experts, whose slot index is E + s.
    """
    active = sorted({layers[j] for j in _members(run_mask)})
    groups = []
    for d in range(D):
        for l in active:
            for e in range(E):
                if expert_to_device[e] == d:
                    groups.append((d, l, e))
            for s in range(S):
                groups.append((d, l, E + s))
    return groups


def home_device(t_local: int, T_j: int, D: int) -> int:
    """Data-parallel home of a token: contiguous split of a micro-batch over the devices."""
    return (t_local * D) // T_j


def permute(x_bits: np.ndarray, topk_idx: np.ndarray, run_mask: int, layers: Sequence[int],
            tok_off: Sequence[int], expert_to_device: Sequence[int], E: int, K: int, S: int, D: int):
    """Dispatch as a stable grouping (stands in for the first all-to-all of Section 2.2).

    Rows of a group are ordered by (micro-batch, token).  A shared expert's group on device d
    holds the tokens whose home device is d.  Returns group offsets, the weight-matrix index
    of every group (layer * (E + S) + slot), the source token of every row, the row of every
    (token, slot) and the gathered rows.  `x_bits` may be any dtype: rows are copied verbatim.
    """
    groups = group_table(run_mask, layers, expert_to_device, E, S, D)
    gid = {(l, e, d): g for g, (d, l, e) in enumerate(groups)}
    T_tot = topk_idx.shape[0]
    rows: List[List[Tuple[int, int]]] = [[] for _ in groups]     # (token, slot)
    for j in _members(run_mask):
        l = layers[j]
        T_j = tok_off[j + 1] - tok_off[j]
        for t in range(tok_off[j], tok_off[j + 1]):
            for k in range(K):
                e = int(topk_idx[t, k])
                rows[gid[(l, e, expert_to_device[e])]].append((t, k))
            for s in range(S):
                d = home_device(t - tok_off[j], T_j, D)
                rows[gid[(l, E + s, d)]].append((t, K + s))
    group_off = np.zeros(len(groups) + 1, dtype=np.int32)
    for g, r in enumerate(rows):
        group_off[g + 1] = group_off[g] + len(r)
    R = int(group_off[-1])
    row_src = np.zeros(R, dtype=np.int32)
    pos = np.full((T_tot, K + S), -1, dtype=np.int32)
    r = 0
    for g in range(len(groups)):
        for (t, slot) in rows[g]:
            row_src[r] = t
            pos[t, slot] = r
            r += 1
    group_w = np.array([l * (E + S) + e for (_, l, e) in groups], dtype=np.int32)
    xp = x_bits[row_src] if R else x_bits[:0]
    return group_off, group_w, row_src, pos, xp, groups


# --------------------------------------------------------------------------- experts
def silu(g: np.ndarray) -> np.ndarray:
    return g / (1.0 + np.exp(-g))


def swiglu_mlp(x: np.ndarray, w_gate: np.ndarray, w_up: np.ndarray, w_down: np.ndarray, dtype=np.float32):
    """expert(x) = W_down (silu(W_gate x) * (W_up x)); x [r, H], W_gate/W_up [I, H], W_down [H, I]."""
    x = x.astype(dtype)
    g = x @ w_gate.astype(dtype).T
    u = x @ w_up.astype(dtype).T
    a = silu(g) * u
    return a @ w_down.astype(dtype).T


def expert_ffn(xp: np.ndarray, group_off: np.ndarray, group_w: np.ndarray,
               get_weights: Callable[[int], Tuple[np.ndarray, np.ndarray, np.ndarray]],
               dtype=np.float32) -> np.ndarray:
    """Every group's rows through that group's expert; the intermediate stays unrounded.

    `get_weights(w)` returns (W_gate, W_up, W_down) of weight matrix index w.
    """
    R = int(group_off[-1])
    H = xp.shape[1]
    y = np.zeros((R, H), dtype=dtype)
    for g in range(len(group_w)):
        r0, r1 = int(group_off[g]), int(group_off[g + 1])
        if r1 == r0:
            continue
        wg, wu, wd = get_weights(int(group_w[g]))
        y[r0:r1] = swiglu_mlp(xp[r0:r1], wg, wu, wd, dtype)
    return y


def combine(y: np.ndarray, pos: np.ndarray, topk_w: np.ndarray, K: int, S: int, dtype=np.float32,
            residual: np.ndarray = None) -> np.ndarray:
    """Eq. 1: out[t] = sum_k W[t,k] * y[pos[t,k]] + sum_s y[pos[t,K+s]] (k ascending, then s).

    With `residual` (the MoE block's input h'_l, one row per token) the result is the next hidden
    state of Section 2.1, h_{l+1} = h'_l + MLP(h'_l): the row of `residual` is added last.
    Rows of tokens with pos < 0 (micro-batch not selected) are returned as zeros and flagged in
    the boolean vector that comes with the result.
    """
    T = pos.shape[0]
    H = y.shape[1]
    out = np.zeros((T, H), dtype=dtype)
    done = np.zeros(T, dtype=bool)
    for t in range(T):
        if pos[t, 0] < 0:
            continue
        acc = np.zeros(H, dtype=dtype)
        for k in range(K):
            acc = acc + dtype(topk_w[t, k]) * y[pos[t, k]].astype(dtype)
        for s in range(S):
            acc = acc + y[pos[t, K + s]].astype(dtype)
        if residual is not None:
            out[t] = acc + residual[t].astype(dtype)
        else:
            out[t] = acc
        done[t] = True
    return out, done


def dense_masked_moe(x: np.ndarray, topk_idx: np.ndarray, topk_w: np.ndarray, token_layer: np.ndarray,
                     E: int, S: int,
                     get_weights: Callable[[int], Tuple[np.ndarray, np.ndarray, np.ndarray]],
                     dtype=np.float64) -> np.ndarray:
    """Eq. 1 by brute force: every expert of the token's layer on every token, masked.

    out[t] = sum_e [e in I_t] * W_{t,e} * expert_{l,e}(x_t) + sum_s shared_{l,s}(x_t), with no
    permutation, grouping or scheduling involved.  token_layer[t] < 0 marks tokens that do not run.
    """
    T, H = x.shape
    out = np.zeros((T, H), dtype=dtype)
    for l in sorted({int(v) for v in token_layer if v >= 0}):
        toks = np.nonzero(token_layer == l)[0]
        xs = x[toks].astype(dtype)
        for e in range(E + S):
            wg, wu, wd = get_weights(l * (E + S) + e)
            ye = swiglu_mlp(xs, wg, wu, wd, dtype)
            if e < E:
                gate = np.zeros(len(toks), dtype=dtype)
                for i, t in enumerate(toks):
                    for k in range(topk_idx.shape[1]):
                        if topk_idx[t, k] == e:
                            gate[i] += dtype(topk_w[t, k])
                out[toks] += gate[:, None] * ye
            else:
                out[toks] += ye
    return out


# --------------------------------------------------------------------------- Algorithm 1
def run_algorithm1(load_of: Callable[[int, int], Sequence[int]], N: int, L: int, D: int, m: int,
                   policy: int = POLICY_MAXUTIL) -> List[Dict]:
    """Algorithm 1 on load vectors.  `load_of(j, l)` is the routed load vector w_j^{(l)}.

    Every micro-batch starts at layer 0 in the pool.  A step schedules a subset of the pool,
    "executes" it, advances the members' layers and drops those that passed the last layer.
    A deferred micro-batch keeps the routing it obtained when it reached its layer.  Returns,
    per step, the pool, the run set, the layers executed and the joint load.
    """
    l = [0] * N
    pool = (1 << N) - 1 if L > 0 else 0
    steps = []
    while pool:
        loads = np.array([list(load_of(j, l[j])) if (pool >> j) & 1 else [0] * D
                          for j in range(N)], dtype=np.int64)
        res = schedule(loads, pool, m, policy)
        run = res["run_mask"]
        steps.append(dict(pool=pool, run_mask=run, layers={j: l[j] for j in _members(run)},
                          joint_load=res["joint_load"],
                          member_loads={j: [int(v) for v in loads[j]] for j in _members(run)}))
        for j in _members(run):
            l[j] += 1
            if l[j] >= L:
                pool &= ~(1 << j)
    return steps


def same_peak_windows(loads_by_layer: Sequence[Sequence[int]], n: int) -> Tuple[int, int]:
    """How many windows of n consecutive layers have their workload skewed to the same device
    (the statistic of the paper's table on consecutive layers: the worst case of Section 4.1,
    where combining gains nothing).  `loads_by_layer[l]` is the load vector of layer l; the skew
    device is the peak device, lowest index among equal maxima.  Returns (count, windows) with
    windows = L - n + 1."""
    peaks = [_peak_device(w) for w in loads_by_layer]
    windows = max(len(peaks) - n + 1, 0)
    count = 0
    for l in range(windows):
        if all(peaks[l + i] == peaks[l] for i in range(1, n)):
            count += 1
    return count, windows


def idle_cross_layer(steps: List[Dict], D: int) -> Tuple[int, int]:
    """1 - u of the run as (idle_num, den): Eq. 3 with one term per executed step."""
    work = sum(sum(s["joint_load"]) for s in steps)
    cap = D * sum(effective_workload(s["joint_load"]) for s in steps)
    return cap - work, cap


def idle_each_alone(steps: List[Dict], D: int) -> Tuple[int, int]:
    """Same work with every (micro-batch, layer) workload executed by itself: the denominator
    is D * sum_j max(w_j) - the 'maximum workload' of the per-step plots, i.e. no combination."""
    work = sum(sum(w) for s in steps for w in s["member_loads"].values())
    cap = D * sum(effective_workload(w) for s in steps for w in s["member_loads"].values())
    return cap - work, cap


def idle_lock_step(load_of: Callable[[int, int], Sequence[int]], N: int, L: int, D: int) -> Tuple[int, int]:
    """All micro-batches executed jointly layer by layer (no deferral, same layer every step)."""
    work = cap = 0
    for l in range(L):
        tot = [0] * D
        for j in range(N):
            w = load_of(j, l)
            for d in range(D):
                tot[d] += int(w[d])
        work += sum(tot)
        cap += D * effective_workload(tot)
    return cap - work, cap
