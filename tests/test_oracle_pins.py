"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle.

The paper prints no numeric scheduling example (its overview figure is a drawing), so the
scheduling fixtures under tests/golden are worked by hand from Eq. 2, Eq. 3, Section 4.2,
Section 5.2 and Algorithm 1 and are labelled as derived.
"""
import itertools
import json
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import eb_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden", "schedule_examples.json")


def _mask(members):
    return sum(1 << j for j in members)


def _members(mask):
    return [j for j in range(32) if (mask >> j) & 1]


with open(GOLD) as f:
    EXAMPLES = json.load(f)


# ------------------------------------------------------------------ scheduling: worked examples
@pytest.mark.parametrize("ex", EXAMPLES["single_step"], ids=lambda e: e["name"])
def test_single_step_examples(ex):
    loads = np.array(ex["loads"])
    pool = _mask(ex["pool"])
    for key, (n, d) in ex["subset_util"].items():
        sub = [int(v) for v in key.split(",")]
        num, den = O.utilisation(loads[sub].sum(axis=0))
        assert Fraction(num, den) == Fraction(n, d), key
    for name, pol in (("maxutil", O.POLICY_MAXUTIL), ("cumutil", O.POLICY_CUMUTIL), ("diffpeak", O.POLICY_DIFFPEAK)):
        if name in ex:
            res = O.schedule(loads, pool, ex["m"], pol)
            assert _members(res["run_mask"]) == ex[name], name
            assert res["defer_mask"] == pool & ~res["run_mask"]
            assert res["joint_load"] == list(loads[ex[name]].sum(axis=0))
    if "idle_cross" in ex:
        res = O.schedule(loads, pool, ex["m"], O.POLICY_MAXUTIL)
        step = dict(joint_load=res["joint_load"],
                    member_loads={j: list(loads[j]) for j in _members(res["run_mask"])})
        n, d = O.idle_cross_layer([step], ex["D"])
        assert Fraction(n, d) == Fraction(*ex["idle_cross"])
        n, d = O.idle_each_alone([step], ex["D"])
        assert Fraction(n, d) == Fraction(*ex["idle_each_alone"])


def test_home_device_examples():
    for case in EXAMPLES["home_device"]["cases"]:
        got = [O.home_device(t, case["T"], case["D"]) for t in range(case["T"])]
        assert got == case["home"]


@pytest.mark.parametrize("ex", EXAMPLES["driver"], ids=lambda e: e["name"])
def test_driver_examples(ex):
    table = {tuple(int(v) for v in k.split(",")): v for k, v in ex["loads"].items()}
    load_of = lambda j, l: table[(j, l)]
    steps = O.run_algorithm1(load_of, ex["N"], ex["L"], ex["D"], ex["m"], O.POLICY_MAXUTIL)
    assert [_members(s["run_mask"]) for s in steps] == ex["run_sets"]
    assert [{str(j): l for j, l in s["layers"].items()} for s in steps] == ex["run_layers"]
    assert sum(O.effective_workload(s["joint_load"]) for s in steps) == ex["effective_sum"]
    assert sum(sum(s["joint_load"]) for s in steps) == ex["work"]
    n, d = O.idle_cross_layer(steps, ex["D"])
    assert 1 - Fraction(n, d) == Fraction(*ex["util_cross"])
    n, d = O.idle_each_alone(steps, ex["D"])
    assert 1 - Fraction(n, d) == Fraction(*ex["util_each_alone"])
    n, d = O.idle_lock_step(load_of, ex["N"], ex["L"], ex["D"])
    assert 1 - Fraction(n, d) == Fraction(*ex["util_lock_step"])


# ------------------------------------------------------------------ scheduling: invariants + brute force
def _recursive_best(loads, members, m, D):
    """Independent enumerator: recursion over include/exclude, float-free comparison."""
    best = [None]

    def rec(i, chosen, tot):
        if i == len(members):
            if len(chosen) < m:
                return
            peak = max(tot)
            u = Fraction(sum(tot), D * peak) if peak else Fraction(1)
            key = (u, len(chosen), -_mask(chosen))
            if best[0] is None or key > best[0][0]:
                best[0] = (key, list(chosen))
            return
        j = members[i]
        rec(i + 1, chosen + [j], [a + int(b) for a, b in zip(tot, loads[j])])
        rec(i + 1, chosen, tot)

    rec(0, [], [0] * D)
    return best[0]


def test_maxutil_matches_independent_enumeration_and_bounds():
    rng = np.random.default_rng(7)
    for trial in range(300):
        N = int(rng.integers(1, 7))
        D = int(rng.integers(1, 6))
        m = int(rng.integers(1, N + 1))
        loads = rng.integers(0, 12, size=(N, D))
        if trial % 5 == 0:
            loads[rng.integers(0, N)] = 0
        pool = int(rng.integers(1, 1 << N))
        members = _members(pool)
        res = O.schedule(loads, pool, m, O.POLICY_MAXUTIL)
        run = _members(res["run_mask"])
        assert res["run_mask"] & ~pool == 0
        assert len(run) >= min(m, len(members))
        if len(members) <= m:
            assert run == members
        else:
            key, chosen = _recursive_best(loads, members, m, D)
            assert run == sorted(chosen)
        num, den = res["util_num"], res["util_den"]
        if den:
            assert Fraction(1, D) <= Fraction(num, den) <= 1
        # worst-case-safe inequality of Section 4.1 on the chosen set
        assert max(res["joint_load"]) <= sum(int(loads[j].max()) for j in run)


def test_combination_inequality_and_equality_case():
    rng = np.random.default_rng(11)
    for _ in range(500):
        n, D = int(rng.integers(1, 6)), int(rng.integers(1, 9))
        w = rng.integers(0, 100, size=(n, D))
        assert O.effective_workload(w.sum(axis=0)) <= sum(O.effective_workload(r) for r in w)
        # equality when every workload peaks on the same device (Section 4.1, "mostly effective")
        w2 = w.copy()
        w2[:, 0] = w2.max(axis=1) + 1
        assert O.effective_workload(w2.sum(axis=0)) == sum(O.effective_workload(r) for r in w2)
        # strict when two unique peaks sit on different devices
        if n >= 2 and D >= 2:
            w3 = w.copy()
            w3[:, 0] = 0
            w3[:, 1] = 0
            w3[0, 0] = 1000
            w3[1, 1] = 1000
            assert O.effective_workload(w3.sum(axis=0)) < sum(O.effective_workload(r) for r in w3)


def test_maxutil_invariant_under_device_relabelling_and_scaling():
    rng = np.random.default_rng(3)
    checked = 0
    for _ in range(200):
        N, D, m = 5, 4, 3
        loads = rng.integers(1, 50, size=(N, D))
        pool = (1 << N) - 1
        res = O.schedule(loads, pool, m)
        # only tie-free cases: the winning utilisation must be unique
        vals = []
        for r in range(m, N + 1):
            for sub in itertools.combinations(range(N), r):
                tot = loads[list(sub)].sum(axis=0)
                vals.append(Fraction(int(tot.sum()), int(D * tot.max())))
        if sorted(vals)[-1] == sorted(vals)[-2]:
            continue
        checked += 1
        perm = rng.permutation(D)
        assert O.schedule(loads[:, perm], pool, m)["run_mask"] == res["run_mask"]
        assert O.schedule(loads * 7, pool, m)["run_mask"] == res["run_mask"]
    assert checked > 50


def test_policy_all_and_small_pool_run_everything():
    loads = np.array([[5, 1], [1, 5], [9, 0]])
    assert O.schedule(loads, 0b111, 1, O.POLICY_ALL)["run_mask"] == 0b111
    assert O.schedule(loads, 0b101, 2, O.POLICY_MAXUTIL)["run_mask"] == 0b101
    assert O.schedule(loads, 0b100, 3, O.POLICY_CUMUTIL)["run_mask"] == 0b100
    assert O.schedule(loads, 0, 2)["run_mask"] == 0
    z = O.schedule(np.zeros((3, 2), dtype=int), 0b111, 2)          # no work at all: U := 1, everything runs
    assert z["run_mask"] == 0b111 and z["util_den"] == 0


def test_linear_policies_respect_m_and_first_member():
    rng = np.random.default_rng(5)
    for _ in range(200):
        N, D = int(rng.integers(2, 8)), int(rng.integers(2, 6))
        m = int(rng.integers(1, N + 1))
        loads = rng.integers(0, 30, size=(N, D))
        pool = int(rng.integers(1, 1 << N))
        members = _members(pool)
        for pol in (O.POLICY_CUMUTIL, O.POLICY_DIFFPEAK):
            res = O.schedule(loads, pool, m, pol)
            run = _members(res["run_mask"])
            assert set(run) <= set(members) and members[0] in run
            assert len(run) >= min(m, len(members))


# ------------------------------------------------------------------ Algorithm 1 invariants
def test_algorithm1_invariants_random():
    rng = np.random.default_rng(19)
    for trial in range(40):
        N, L, D = int(rng.integers(1, 7)), int(rng.integers(1, 7)), int(rng.integers(2, 6))
        m = int(rng.integers(1, N + 1))
        tab = rng.integers(0, 40, size=(N, L, D))
        load_of = lambda j, l: tab[j, l]
        for pol in (O.POLICY_MAXUTIL, O.POLICY_CUMUTIL, O.POLICY_DIFFPEAK, O.POLICY_ALL):
            steps = O.run_algorithm1(load_of, N, L, D, m, pol)
            assert L <= len(steps) <= N * L
            seen = {j: [] for j in range(N)}
            for s in steps:
                run = _members(s["run_mask"])
                assert s["run_mask"] & ~s["pool"] == 0
                assert len(run) >= min(m, bin(s["pool"]).count("1"))
                for j in run:
                    seen[j].append(s["layers"][j])
                assert s["joint_load"] == [int(v) for v in sum(tab[j, s["layers"][j]] for j in run)]
            # every (micro-batch, layer) workload runs exactly once and in layer order
            for j in range(N):
                assert seen[j] == list(range(L))
            assert sum(sum(s["joint_load"]) for s in steps) == int(tab.sum())
            n1, d1 = O.idle_cross_layer(steps, D)
            n2, d2 = O.idle_each_alone(steps, D)
            assert d1 <= d2                                   # combining never hurts (Section 4.1)
            if pol == O.POLICY_ALL:
                n3, d3 = O.idle_lock_step(load_of, N, L, D)
                assert (n1, d1) == (n3, d3)


def test_uniform_routing_gives_zero_idle_and_full_run_set():
    # token t of every micro-batch picks experts (t*K + i) mod E: every expert, hence every
    # device, receives exactly T*K/E assignments
    E, K, D, N, T = 8, 2, 4, 4, 16
    dev = [(e * D) // E for e in range(E)]
    logits = np.full((N * T, E), -5.0, dtype=np.float32)
    for t in range(N * T):
        for i in range(K):
            logits[t, ((t % T) * K + i) % E] = 3.0 - i
    tok_off = [j * T for j in range(N + 1)]
    idx, w, mb_load, mb_cnt = O.route(logits, K, dev, D, tok_off)
    assert (mb_load == T * K // D).all() and (mb_cnt == T * K // E).all()
    res = O.schedule(mb_load, (1 << N) - 1, 3)
    assert res["run_mask"] == (1 << N) - 1
    assert res["util_num"] == res["util_den"]
    steps = O.run_algorithm1(lambda j, l: mb_load[j], N, 3, D, 3)
    assert len(steps) == 3 and O.idle_cross_layer(steps, D)[0] == 0


def test_combine_with_residual_by_hand():
    # two expert rows, one token with weights 1/4 and 3/4: 0.25*(4, 8) + 0.75*(8, -4) = (7, -1); plus h' = (1, 10)
    y = np.array([[4.0, 8.0], [8.0, -4.0]])
    pos = np.array([[0, 1], [-1, -1]], dtype=np.int32)
    w = np.array([[0.25, 0.75], [0.5, 0.5]])
    h = np.array([[1.0, 10.0], [5.0, 5.0]])
    out, done = O.combine(y, pos, w, 2, 0, dtype=np.float64)
    assert out.tolist() == [[7.0, -1.0], [0.0, 0.0]] and done.tolist() == [True, False]
    nxt, done = O.combine(y, pos, w, 2, 0, dtype=np.float64, residual=h)
    assert nxt.tolist() == [[8.0, 9.0], [0.0, 0.0]] and done.tolist() == [True, False]


def test_same_peak_windows_by_hand():
    # peaks 0, 0, 1, 0 (tied maxima -> lower device), 0: pairs (0,0) (0,1) (1,0) (0,0) -> 2 of 4; no triple of 3
    loads = [(3, 1), (2, 0), (0, 5), (1, 1), (4, 2)]
    assert O.same_peak_windows(loads, 2) == (2, 4)
    assert O.same_peak_windows(loads, 3) == (0, 3)
    # peaks 1, 1, 1, 0: pairs -> 2 of 3, triples -> 1 of 2; a window longer than the sequence -> 0 of 0
    loads = [(0, 2), (1, 9), (3, 4), (5, 0)]
    assert O.same_peak_windows(loads, 2) == (2, 3)
    assert O.same_peak_windows(loads, 3) == (1, 2)
    assert O.same_peak_windows(loads, 5) == (0, 0)
    # 48 layers give 47 pairs and 46 triples, the denominators the paper's table prints
    assert O.same_peak_windows([(1, 0)] * 48, 2) == (47, 47) and O.same_peak_windows([(1, 0)] * 48, 3) == (46, 46)


# ------------------------------------------------------------------ routing
def test_route_full_k_is_softmax_and_k1_is_argmax():
    from scipy.special import softmax
    rng = np.random.default_rng(2)
    T, E, D = 37, 12, 4
    logits = rng.normal(size=(T, E)).astype(np.float32)
    dev = [e % D for e in range(E)]
    idx, w, load, cnt = O.route(logits, E, dev, D, [0, 20, 37], dtype=np.float64)
    ref = softmax(logits.astype(np.float64), axis=1)
    assert np.allclose(np.take_along_axis(ref, idx.astype(np.int64), 1), w, rtol=0, atol=1e-14)
    assert (np.sort(idx, axis=1) == np.arange(E)).all()
    assert (np.diff(np.take_along_axis(logits, idx.astype(np.int64), 1), axis=1) <= 0).all()
    idx1, w1, load1, _ = O.route(logits, 1, dev, D, [0, 20, 37])
    assert (idx1[:, 0] == logits.argmax(axis=1)).all() and np.allclose(w1, 1.0)
    # without renormalisation the weights are the full-softmax entries of the chosen experts
    idx3, w3, _, _ = O.route(logits, 3, dev, D, [0, 37], renorm_topk=False, dtype=np.float64)
    assert np.allclose(np.take_along_axis(ref, idx3.astype(np.int64), 1), w3, atol=1e-14)
    idx3r, w3r, load3, cnt3 = O.route(logits, 3, dev, D, [0, 20, 37], dtype=np.float64)
    assert np.allclose(w3r.sum(axis=1), 1.0) and np.allclose(w3r, w3 / w3.sum(axis=1, keepdims=True))
    # token conservation: every micro-batch places T_j * K assignments
    assert load3.sum(axis=1).tolist() == [20 * 3, 17 * 3] and cnt3.sum(axis=1).tolist() == [60, 51]
    for j, (a, b) in enumerate([(0, 20), (20, 37)]):
        brute = np.zeros(D, dtype=int)
        for t in range(a, b):
            for k in range(3):
                brute[dev[idx3r[t, k]]] += 1
        assert (brute == load3[j]).all()


def test_route_tie_break_prefers_lower_index():
    logits = np.array([[1.0, 2.0, 2.0, 0.5, 2.0], [0.0, -0.0, 0.0, 0.0, 0.0]], dtype=np.float32)
    idx, w, _, _ = O.route(logits, 2, [0, 0, 1, 1, 1], 2, [0, 2])
    assert idx.tolist() == [[1, 2], [0, 1]]
    assert np.allclose(w, 0.5)


# ------------------------------------------------------------------ permutation
def _random_case(rng, N=3, T=(5, 9, 4), L=4, E=6, K=2, S=1, D=3, H=8):
    tok_off = np.concatenate([[0], np.cumsum(T)]).tolist()
    T_tot = tok_off[-1]
    layers = [int(v) for v in rng.integers(0, L, size=N)]
    dev = [int(v) for v in rng.integers(0, D, size=E)]
    logits = rng.normal(size=(T_tot, E)).astype(np.float32)
    idx, w, _, _ = O.route(logits, K, dev, D, tok_off)
    x = rng.normal(size=(T_tot, H)).astype(np.float32)
    return tok_off, layers, dev, idx, w, x


def test_permute_invariants():
    rng = np.random.default_rng(23)
    for trial in range(30):
        N, L, E, K, S, D, H = 3, 4, 6, 2, trial % 3, 3, 8
        tok_off, layers, dev, idx, w, x = _random_case(rng, N=N, L=L, E=E, K=K, S=S, D=D, H=H)
        run = int(rng.integers(0, 1 << N))
        goff, gw, row_src, pos, xp, groups = O.permute(x, idx, run, layers, tok_off, dev, E, K, S, D)
        sel_tokens = [t for j in _members(run) for t in range(tok_off[j], tok_off[j + 1])]
        R = len(sel_tokens) * (K + S)
        assert goff[-1] == R == len(row_src)
        assert len(groups) == len({layers[j] for j in _members(run)}) * (E + D * S)
        # pos and row_src are mutually inverse; each selected (token, slot) appears exactly once
        assert sorted(pos[pos >= 0].tolist()) == list(range(R))
        for t in range(tok_off[-1]):
            for slot in range(K + S):
                if t in sel_tokens:
                    assert row_src[pos[t, slot]] == t
                else:
                    assert pos[t, slot] == -1
        assert (xp == x[row_src]).all()
        # group membership, histogram and stable (micro-batch, token) order
        tok_mb = np.searchsorted(tok_off, np.arange(tok_off[-1]), side="right") - 1
        for g, (d, l, e) in enumerate(groups):
            rows = row_src[goff[g]:goff[g + 1]]
            assert (np.diff(rows) > 0).all()
            assert gw[g] == l * (E + S) + e
            for t in rows:
                j = tok_mb[t]
                assert layers[j] == l
                if e < E:
                    assert dev[e] == d and e in idx[t]
                else:
                    assert O.home_device(t - tok_off[j], tok_off[j + 1] - tok_off[j], D) == d
            if e < E:
                expect = sum(1 for t in sel_tokens if layers[tok_mb[t]] == l and e in idx[t])
                assert len(rows) == expect
        # device-major enumeration
        assert [g[0] for g in groups] == sorted(g[0] for g in groups)


# ------------------------------------------------------------------ expert MLP and aggregation
def test_swiglu_matches_library_mlp():
    import torch.nn.functional as F
    rng = np.random.default_rng(4)
    r, H, I = 7, 24, 40                       # non-square so a transposed operand cannot pass
    x, wg, wu, wd = (rng.normal(size=s) for s in ((r, H), (I, H), (I, H), (H, I)))
    got = O.swiglu_mlp(x, wg, wu, wd, dtype=np.float64)
    tx, tg, tu, td = (torch.from_numpy(a) for a in (x, wg, wu, wd))
    ref = F.linear(F.silu(F.linear(tx, tg)) * F.linear(tx, tu), td).numpy()
    assert np.allclose(got, ref, rtol=1e-12, atol=1e-12)
    assert (O.swiglu_mlp(x, np.zeros_like(wg), wu, wd) == 0).all()          # silu(0) = 0
    got32 = O.swiglu_mlp(x, wg, wu, wd, dtype=np.float32)
    assert np.abs(got32 - ref).max() <= 1e-4 * np.abs(ref).max()


def _weights(rng, n, H, I, scale=0.3):
    ws = [(rng.normal(size=(I, H)) * scale, rng.normal(size=(I, H)) * scale, rng.normal(size=(H, I)) * scale)
          for _ in range(n)]
    return ws


def test_pipeline_equals_dense_masked_bruteforce():
    rng = np.random.default_rng(31)
    for trial in range(6):
        N, L, E, K, S, D, H, I = 3, 3, 5, 2, trial % 3, 2, 10, 14
        tok_off, layers, dev, idx, w, x = _random_case(rng, N=N, L=L, E=E, K=K, S=S, D=D, H=H)
        ws = _weights(rng, L * (E + S), H, I)
        get = lambda i: ws[i]
        run = [0b111, 0b101, 0b010, 0b110, 0b011, 0b111][trial]
        goff, gw, row_src, pos, xp, _ = O.permute(x, idx, run, layers, tok_off, dev, E, K, S, D)
        y = O.expert_ffn(xp, goff, gw, get, dtype=np.float64)
        out, done = O.combine(y, pos, w, K, S, dtype=np.float64)
        tok_layer = np.full(tok_off[-1], -1)
        for j in _members(run):
            tok_layer[tok_off[j]:tok_off[j + 1]] = layers[j]
        ref = O.dense_masked_moe(x, idx, w, tok_layer, E, S, get, dtype=np.float64)
        assert (done == (tok_layer >= 0)).all()
        assert np.allclose(out, ref, rtol=1e-11, atol=1e-11)
        # Section 2.1: h_{l+1} = h' + MLP(h'); the brute-force MoE output plus the input, no shared code path
        nxt, _ = O.combine(y, pos, w, K, S, dtype=np.float64, residual=x)
        sel = tok_layer >= 0
        assert np.allclose(nxt[sel], (ref + x.astype(np.float64))[sel], rtol=1e-11, atol=1e-11)
        assert (nxt[~sel] == 0).all()
        # fp32 oracle against the fp64 one: bounds the oracle's own rounding error
        y32 = O.expert_ffn(xp, goff, gw, get, dtype=np.float32)
        out32, _ = O.combine(y32, pos, w, K, S, dtype=np.float32)
        assert np.abs(out32 - ref).max() <= 1e-5 * max(1.0, np.abs(ref).max())


def test_identical_experts_make_routing_irrelevant():
    rng = np.random.default_rng(41)
    N, L, E, K, S, D, H, I = 2, 2, 6, 3, 0, 3, 8, 12
    tok_off, layers, dev, idx, w, x = _random_case(rng, N=N, T=(6, 7), L=L, E=E, K=K, S=S, D=D, H=H)
    one = _weights(rng, 1, H, I)[0]
    get = lambda i: one
    goff, gw, row_src, pos, xp, _ = O.permute(x, idx, 0b11, layers, tok_off, dev, E, K, S, D)
    y = O.expert_ffn(xp, goff, gw, get, dtype=np.float64)
    out, _ = O.combine(y, pos, w.astype(np.float64), K, S, dtype=np.float64)
    ref = O.swiglu_mlp(x, *one, dtype=np.float64)      # renormalised weights sum to one
    assert np.allclose(out, ref, rtol=1e-6, atol=1e-6)


def test_single_expert_k1_is_a_dense_mlp():
    rng = np.random.default_rng(43)
    H, I, T = 8, 12, 9
    x = rng.normal(size=(T, H))
    one = _weights(rng, 1, H, I)[0]
    idx, w, _, _ = O.route(np.zeros((T, 1), dtype=np.float32), 1, [0], 1, [0, T])
    goff, gw, row_src, pos, xp, _ = O.permute(x, idx, 1, [0], [0, T], [0], 1, 1, 0, 1)
    assert row_src.tolist() == list(range(T))
    y = O.expert_ffn(xp, goff, gw, lambda i: one, dtype=np.float64)
    out, _ = O.combine(y, pos, w, 1, 0, dtype=np.float64)
    assert np.allclose(out, O.swiglu_mlp(x, *one, dtype=np.float64))
