"""GPU parity: every stage of the cross-layer MoE step, called through the C ABI, against the CPU
oracle on the same seeded inputs.  Integers (routing, schedule, loads, permutation) bit-exact;
expert outputs within |gpu - ref| <= 2e-2 * max|ref| + 1e-3 elementwise (oracle in fp32 from the
same bf16 weights)."""
import numpy as np
import pytest
import torch

from oracle import eb_oracle as O
from paper_2608_07964_b200 import synth
from tests import harness as Hn

pytestmark = pytest.mark.gpu


def _binding():
    from paper_2608_07964_b200 import binding
    return binding


def _sample_rows(r0, r1):
    """Rows of a group worth comparing at full size: its first and last rows, and the rows around every
    place where the expert kernels change tile or CTA.  Groups of at most 128 rows are one tile of a single
    CTA; larger groups are cut into ceil(rows / 256) nearly equal tiles, each shared by two CTAs that split
    its rows (rounded up to 16) in halves."""
    n = r1 - r0
    if n <= 64:
        return np.arange(r0, r1)
    pick = set(range(0, 24)) | set(range(n - 24, n))
    if n <= 128:
        pick |= set(range(n // 2 - 8, n // 2 + 8)) | set(range(28, 36))
    else:
        t = -(-n // 256)
        each, more = divmod(n, t)
        start = 0
        for i in range(t):
            rows = each + (1 if i < more else 0)
            half = ((rows + 15) // 16 * 16) // 2
            for c in (start, start + half, start + rows):
                pick |= set(range(max(0, c - 8), min(n, c + 8)))
            start += rows
    return np.array(sorted(pick)) + r0


def _full_step(case, store, m, policy=O.POLICY_MAXUTIL, pool_mask=None, check_ffn=True, groups_to_check=None,
               rows_per_group=None):
    B = _binding()
    wl = case.wl
    n_mb = len(case.layers)
    pool = ((1 << n_mb) - 1) if pool_mask is None else pool_mask
    step = B.from_workload(wl, max_tokens=max(case.T_tot, 1))
    step.bind_weights(store.gate, store.up, store.down)
    T = case.T_tot
    step.logits[:T].copy_(case.logits)
    step.x[:T].copy_(case.x)
    step.out.fill_(-7.0)
    batch = B.Batch(case.tok_off, case.layers, pool)
    step.eb_route(batch)
    step.eb_schedule(batch, m, policy)
    step.eb_permute(batch)
    step.eb_expert_ffn_grouped()
    step.eb_combine(batch)
    torch.cuda.synchronize()
    assert step.device_status() == 0
    assert step.check_permutation(batch) == 0
    assert step.check_workspace_guards() == 0, "a kernel wrote past the end of its workspace region"

    ref = Hn.oracle_front(case, pool, m, policy)
    Hn.check_front(step, case, ref, n_mb)
    if not check_ffn:
        return step, ref
    R = int(ref["group_off"][-1])
    xp = step.xp[:R].float().cpu().numpy()
    yp_gpu = step.yp[:R].float().cpu().numpy()
    G = len(ref["group_w"])
    if groups_to_check is None:
        y_ref = O.expert_ffn(xp, ref["group_off"], ref["group_w"], store.get)
        assert Hn.within_bar(yp_gpu, y_ref), f"expert outputs off by {Hn.worst(yp_gpu, y_ref):.2f} x bar"
        out_ref, done = O.combine(y_ref, ref["pos"], ref["w"], wl.K, wl.S)
        out_gpu = step.out[:T].float().cpu().numpy()
        assert Hn.within_bar(out_gpu[done], out_ref[done]), f"aggregated output off by {Hn.worst(out_gpu[done], out_ref[done]):.2f} x bar"
        assert (out_gpu[~done] == -7.0).all(), "rows of micro-batches that did not run must stay untouched"
    else:
        # sampled groups: the oracle computes chosen rows of each group over all output columns
        scale = 0.0
        checked = []
        for g in groups_to_check:
            r0, r1 = int(ref["group_off"][g]), int(ref["group_off"][g + 1])
            if r1 == r0:
                continue
            rows = np.arange(r0, min(r1, r0 + rows_per_group)) if rows_per_group else _sample_rows(r0, r1)
            wg, wu, wd = store.get(int(ref["group_w"][g]))
            y = O.swiglu_mlp(xp[rows], wg, wu, wd)
            checked.append((rows, y))
            scale = max(scale, float(np.abs(y).max()))
        assert checked
        for rows, y in checked:
            err = np.abs(yp_gpu[rows].astype(np.float64) - y)
            assert (err <= Hn.REL * scale + Hn.ABS).all(), f"group rows {rows[0]}..{rows[-1]} off by {err.max() / (Hn.REL * scale + Hn.ABS):.2f} x bar"
        # aggregation against the oracle's own expert outputs: a few tokens of one chosen micro-batch (one
        # layer, so only that layer's experts are fetched), every row of theirs through the oracle's MLP
        j = [jj for jj in range(n_mb) if (ref["sched"]["run_mask"] >> jj) & 1 and case.tok_off[jj + 1] > case.tok_off[jj]][-1]
        rng = np.random.default_rng(0)
        toks = np.sort(rng.choice(np.arange(case.tok_off[j], case.tok_off[j + 1]),
                                  size=min(12, case.tok_off[j + 1] - case.tok_off[j]), replace=False))
        need = np.unique(ref["pos"][toks].reshape(-1))
        y_rows = np.zeros((R, wl.H), dtype=np.float32)
        grp = np.searchsorted(ref["group_off"], need, side="right") - 1
        for g in np.unique(grp):
            rows = need[grp == g]
            wg, wu, wd = store.get(int(ref["group_w"][g]))
            y_rows[rows] = O.swiglu_mlp(xp[rows], wg, wu, wd)
        out_ref, done = O.combine(y_rows, ref["pos"][toks], ref["w"][toks], wl.K, wl.S)
        assert done.all()
        out_gpu = step.out[:T].float().cpu().numpy()[toks]
        assert Hn.within_bar(out_gpu, out_ref), f"aggregated output off by {Hn.worst(out_gpu, out_ref):.2f} x bar"
    return step, ref


# ----------------------------------------------------------------------------------- full configs
def test_c1_full_step_all_policies():
    wl = synth.workload("c1")
    store = Hn.WeightStore(wl)
    case = Hn.make_case(wl)
    for pol in (O.POLICY_MAXUTIL, O.POLICY_CUMUTIL, O.POLICY_DIFFPEAK, O.POLICY_ALL):
        _full_step(case, store, wl.m, pol)


def test_c1_not_renormalised_weights():
    wl = synth.workload("c1", renorm_topk=0)
    _full_step(Hn.make_case(wl), Hn.WeightStore(wl), wl.m)


def test_c2_decode_shape_full_step():
    wl = synth.workload("c2")
    store = Hn.WeightStore(wl)
    _full_step(Hn.make_case(wl), store, wl.m)


def test_c3_fine_grained_sampled():
    wl = synth.workload("c3")
    store = Hn.WeightStore(wl)
    case = Hn.make_case(wl)
    ref = Hn.oracle_front(case, (1 << wl.N) - 1, wl.m, O.POLICY_MAXUTIL)
    sizes = np.diff(ref["group_off"])
    G = len(sizes)
    order = np.argsort(sizes)
    pick = sorted({0, G - 1, int(order[-1]), int(order[-2]), int(order[len(order) // 2]),
                   *[int(g) for g in np.random.default_rng(1).choice(G, 12, replace=False)],
                   *[g for g, (_, _, e) in enumerate(ref["groups"]) if e >= wl.E][:3]})
    _full_step(case, store, wl.m, groups_to_check=pick)


def test_c3_initial_state_sampled():
    # Algorithm 1's first step: every micro-batch at layer 0 (large groups, many row tiles per group)
    wl = synth.workload("c3", layers_override=tuple([0] * 16))
    store = Hn.WeightStore(wl)
    case = Hn.make_case(wl)
    ref = Hn.oracle_front(case, (1 << wl.N) - 1, wl.m, O.POLICY_MAXUTIL)
    sizes = np.diff(ref["group_off"])
    routed = [g for g, (_, _, e) in enumerate(ref["groups"]) if e < wl.E and sizes[g] > 0]
    by_size = sorted(routed, key=lambda g: sizes[g])
    over = [g for g in by_size if sizes[g] > 128]
    under = [g for g in by_size if sizes[g] <= 128]
    shared = [g for g, (_, _, e) in enumerate(ref["groups"]) if e >= wl.E and sizes[g] > 0]
    pick = sorted({by_size[-1], over[0], over[len(over) // 2], *(under[-1:]), *(under[:1]), shared[0], shared[-1]})
    _full_step(case, store, wl.m, groups_to_check=pick)


def test_c4_large_experts_sampled():
    wl = synth.workload("c4")
    store = Hn.WeightStore(wl)
    case = Hn.make_case(wl)
    ref = Hn.oracle_front(case, (1 << wl.N) - 1, wl.m, O.POLICY_MAXUTIL)
    sizes = np.diff(ref["group_off"])
    nz = [int(g) for g in np.nonzero(sizes)[0]]
    over = sorted((g for g in nz if sizes[g] > 128), key=lambda g: sizes[g])
    under = sorted((g for g in nz if sizes[g] <= 128), key=lambda g: sizes[g])
    # the largest group (three pair tiles), the smallest and a middle one of those over 128 rows, the largest
    # and the smallest of the single-CTA groups; rows at every tile and CTA boundary, all output columns
    pick = sorted({int(np.argmax(sizes)), over[0], over[len(over) // 2], under[-1], under[0]})
    _full_step(case, store, wl.m, groups_to_check=pick)


# ----------------------------------------------------------------------------------- edge cases
def _small(**kw):
    base = dict(L=3, E=6, K=2, S=1, H=72, I=200, D=3, mapping="mod", N=4, T=8, zipf_s=1.0)
    base.update(kw)
    return synth.Workload(name="edge", **base)


@pytest.mark.parametrize("tokens,layers,pool,m", [
    ([5, 33, 0, 64], [0, 2, 1, 2], 0b1111, 3),       # ragged, an empty micro-batch, two sharing a layer
    ([1, 2, 3, 4], [1, 1, 1, 1], 0b1111, 2),         # fewer tokens than devices, one layer only
    ([40, 40, 40, 40], [0, 1, 2, 0], 0b0110, 1),     # pool is a strict subset
    ([130, 7, 129, 31], [2, 2, 0, 1], 0b1011, 4),    # pool smaller than m: everything in the pool runs
    ([16, 16, 16, 16], [0, 0, 0, 0], 0b0000, 2),     # empty pool: nothing runs
])
def test_edge_shapes(tokens, layers, pool, m):
    wl = _small()
    store = Hn.WeightStore(wl)
    case = Hn.make_case(wl, tokens, layers)
    _full_step(case, store, m, pool_mask=pool)


def test_edge_k_equals_e_single_device_no_shared():
    wl = _small(E=4, K=4, S=0, D=1, H=64, I=64)
    _full_step(Hn.make_case(wl, [9, 70, 3, 20], [0, 1, 2, 1]), Hn.WeightStore(wl), 3)


def test_edge_max_micro_batches_and_wide_router():
    wl = _small(L=5, E=200, K=8, S=2, D=16, N=16, T=12, H=128, I=136, mapping="mod")
    case = Hn.make_case(wl, [12 + (j % 5) for j in range(16)], [(j * 5) // 16 for j in range(16)])
    _full_step(case, Hn.WeightStore(wl), 12)


def test_multi_tile_groups_and_tails():
    # groups of several hundred rows: more than one 128-row tile per group, ragged last tiles,
    # output widths that are not multiples of the tile widths
    wl = _small(L=2, E=4, K=2, S=1, D=2, N=2, T=700, H=264, I=328, mapping="contiguous", zipf_s=0.5)
    _full_step(Hn.make_case(wl, [700, 519], [0, 0]), Hn.WeightStore(wl), 2)


# ----------------------------------------------------------------------------------- schedule alone
def test_schedule_random_load_matrices_bit_exact():
    B = _binding()
    rng = np.random.default_rng(12345)
    wl = _small(D=5)
    step = B.from_workload(wl, max_tokens=64)
    n_checked = 0
    for trial in range(2500):
        n_mb = int(rng.integers(1, 9)) if trial % 50 else 16
        D = 5
        hi = [3, 30, 5000][trial % 3]
        loads = rng.integers(0, hi, size=(n_mb, D)).astype(np.int32)
        if trial % 7 == 0:
            loads[rng.integers(0, n_mb)] = 0
        pool = int(rng.integers(0, 1 << n_mb))
        m = int(rng.integers(1, n_mb + 1))
        dev_loads = torch.zeros((16, D), dtype=torch.int32, device="cuda")
        dev_loads[:n_mb] = torch.from_numpy(loads).cuda()
        batch = B.Batch([0] * (n_mb + 1), [0] * n_mb, pool)
        for pol in (O.POLICY_MAXUTIL, O.POLICY_CUMUTIL, O.POLICY_DIFFPEAK, O.POLICY_ALL):
            if n_mb == 16 and pol == O.POLICY_MAXUTIL and trial % 200:
                continue
            got = step.eb_schedule(batch, m, pol, to_host=True, mb_load=dev_loads)
            ref = O.schedule(loads, pool, m, pol)
            for k in ("run_mask", "defer_mask", "n_run", "joint_load", "util_num", "util_den"):
                assert got[k] == ref[k], (trial, pol, k, got[k], ref[k], loads.tolist(), pool, m)
            n_checked += 1
    assert n_checked > 9000


# ----------------------------------------------------------------------------------- combine alone
def test_combine_alone_with_oracle_expert_outputs():
    B = _binding()
    wl = synth.workload("c1")
    case = Hn.make_case(wl)
    store = Hn.WeightStore(wl)
    step, ref = _full_step(case, store, wl.m, check_ffn=False)
    R = int(ref["group_off"][-1])
    xp = step.xp[:R].float().cpu().numpy()
    y = O.expert_ffn(xp, ref["group_off"], ref["group_w"], store.get)
    y_bf = torch.from_numpy(y).to(torch.bfloat16)
    step.yp[:R].copy_(y_bf)
    batch = B.Batch(case.tok_off, case.layers)
    step.eb_combine(batch)
    out_ref, done = O.combine(y_bf.float().numpy(), ref["pos"], ref["w"], wl.K, wl.S)
    out = step.out[:case.T_tot].float().cpu().numpy()
    # only the final bf16 rounding and fp32 summation order separate the two
    assert np.allclose(out[done], out_ref[done], rtol=2 ** -7, atol=1e-6)


# ----------------------------------------------------------------------------------- per-device pass
def test_per_device_pass_covers_exactly_its_rows():
    B = _binding()
    wl = synth.workload("c1")
    case = Hn.make_case(wl)
    store = Hn.WeightStore(wl)
    step, ref = _full_step(case, store, wl.m)
    R = int(ref["group_off"][-1])
    full = step.yp[:R].clone()
    firsts = step.meta()["dev_group_off"]
    for d in range(wl.D):
        step.yp.fill_(3.0)
        step.eb_expert_ffn_grouped(device=d)
        torch.cuda.synchronize()
        r0, r1 = int(ref["group_off"][firsts[d]]), int(ref["group_off"][firsts[d + 1]])
        assert torch.equal(step.yp[r0:r1], full[r0:r1])
        assert (step.yp[:r0] == 3.0).all() and (step.yp[r1:R] == 3.0).all()
    assert step.device_status() == 0


# ----------------------------------------------------------------------------------- whole-step entry points
def test_step_and_step_host_match_the_five_calls():
    B = _binding()
    wl = synth.workload("c1")
    case = Hn.make_case(wl)
    store = Hn.WeightStore(wl)
    step, ref = _full_step(case, store, wl.m)
    T = case.T_tot
    want = step.out[:T].clone()
    batch = B.Batch(case.tok_off, case.layers)
    step.out.fill_(-7.0)      # rows of deferred micro-batches keep whatever the buffer held
    step.eb_step(batch, wl.m)
    torch.cuda.synchronize()
    assert torch.equal(step.out[:T], want)
    h_logits = case.logits.clone().pin_memory()
    h_x = case.x.clone().pin_memory()
    h_out = torch.full((T, wl.H), -7.0, dtype=torch.bfloat16).pin_memory()
    res = step.eb_step_host(batch, wl.m, h_logits, h_x, h_out)
    assert res["run_mask"] == ref["sched"]["run_mask"]
    assert torch.equal(h_out, want.cpu())
    # repeated identical calls on a side stream: same results, and new contents of the same host buffers
    # are picked up
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for rep in range(4):
            if rep == 2:
                h_x.copy_(torch.flip(case.x, dims=[0]))
            h_out.fill_(-7.0)
            res = step.eb_step_host(batch, wl.m, h_logits, h_x, h_out)
            assert res["run_mask"] == ref["sched"]["run_mask"]
            if rep < 2:
                assert torch.equal(h_out, want.cpu())
            else:
                assert not torch.equal(h_out, want.cpu())
        flipped = h_out.clone()
    step.x[:T].copy_(torch.flip(case.x, dims=[0]))
    step.out.fill_(-7.0)
    step.eb_step(batch, wl.m)
    torch.cuda.synchronize()
    assert torch.equal(step.out[:T].cpu(), flipped)


def test_pipelined_host_steps_match_the_blocking_call():
    """Several host-to-host steps in flight on different slots, each with its own inputs: every slot's
    result equals what the blocking call gives for the same inputs; slot misuse is refused."""
    B = _binding()
    wl = synth.workload("c1")
    case = Hn.make_case(wl)
    store = Hn.WeightStore(wl)
    step, ref = _full_step(case, store, wl.m)
    T = case.T_tot
    batch = B.Batch(case.tok_off, case.layers)
    n_slots = 4
    xs = [case.x.clone() if s == 0 else torch.roll(case.x, shifts=s, dims=0) for s in range(n_slots)]
    h_logits = case.logits.clone().pin_memory()
    h_xs = [x.clone().pin_memory() for x in xs]
    want = []
    for s in range(n_slots):
        h_out = torch.full((T, wl.H), -7.0, dtype=torch.bfloat16).pin_memory()
        step.eb_step_host(batch, wl.m, h_logits, h_xs[s], h_out)
        want.append(h_out.clone())
    run0 = [j for j in range(len(case.tok_off) - 1) if (ref["sched"]["run_mask"] >> j) & 1][0]
    a0, b0 = case.tok_off[run0], case.tok_off[run0 + 1]
    assert not torch.equal(want[0][a0:b0], want[1][a0:b0])
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for rounds in range(3):
            h_outs = [torch.full((T, wl.H), -7.0, dtype=torch.bfloat16).pin_memory() for _ in range(n_slots)]
            for s in range(n_slots):
                step.step_host_submit(s, batch, wl.m, h_logits, h_xs[s], h_outs[s])
            with pytest.raises(B.EbError):
                step.step_host_submit(1, batch, wl.m, h_logits, h_xs[1], h_outs[1])   # slot 1 is still in flight
            for s in reversed(range(n_slots)):
                res = step.step_host_wait(s)
                assert res["run_mask"] == ref["sched"]["run_mask"]
                for j in range(len(case.tok_off) - 1):      # rows of deferred micro-batches are not written
                    if (res["run_mask"] >> j) & 1:
                        a, b = case.tok_off[j], case.tok_off[j + 1]
                        assert torch.equal(h_outs[s][a:b], want[s][a:b]), (rounds, s, j)
        assert step.step_host_wait(2)["run_mask"] == ref["sched"]["run_mask"]   # waiting on an idle slot is a no-op
        with pytest.raises(B.EbError):
            step.step_host_submit(B.EB_HOST_SLOTS, batch, wl.m, h_logits, h_xs[0], h_outs[0])
    assert step.device_status() == 0


def test_two_contexts_on_two_streams_do_not_disturb_each_other():
    """Two contexts of different shapes stepping at the same time on two streams, no synchronisation in between:
    each ends with exactly what it computes alone (contexts share no mutable state)."""
    B = _binding()
    wl_a = synth.workload("c1")
    wl_b = synth.workload("c1", E=12, K=3, S=1, H=384, I=640, D=3, N=3, T=50, L=5, seed=77)
    cases, stores, steps, wants = [], [], [], []
    for wl in (wl_a, wl_b):
        case = Hn.make_case(wl)
        store = Hn.WeightStore(wl)
        step, _ = _full_step(case, store, wl.m)           # checked against the oracle inside
        cases.append(case); stores.append(store); steps.append(step)
        wants.append(step.out[:case.T_tot].clone())
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    batches = [B.Batch(c.tok_off, c.layers) for c in cases]
    for st in steps:
        st.out.fill_(-7.0)
    torch.cuda.synchronize()
    for rep in range(20):
        for i in (0, 1):
            with torch.cuda.stream(streams[i]):
                steps[i].eb_step(batches[i], (wl_a, wl_b)[i].m)
    torch.cuda.synchronize()
    for i in (0, 1):
        T = cases[i].T_tot
        got = steps[i].out[:T]
        # rows of deferred micro-batches were refilled with -7 and stay so; the others must match bit for bit
        run = steps[i].sched_result()["run_mask"]
        for j in range(len(cases[i].tok_off) - 1):
            a, b = cases[i].tok_off[j], cases[i].tok_off[j + 1]
            if (run >> j) & 1:
                assert torch.equal(got[a:b], wants[i][a:b]), (i, j)
        assert steps[i].device_status() == 0


def test_deferred_micro_batch_keeps_its_routing():
    B = _binding()
    wl = synth.workload("c1")
    case = Hn.make_case(wl)
    step = B.from_workload(wl)
    T = case.T_tot
    step.logits[:T].copy_(case.logits)
    batch = B.Batch(case.tok_off, case.layers)
    step.eb_route(batch)
    idx0, load0 = step.topk_idx.clone(), step.mb_load.clone()
    step.logits[:T].copy_(torch.flip(case.logits, dims=[1]))       # new logits, but only micro-batch 1 is re-routed
    step.eb_route(batch, route_mask=0b0010)
    a, b = case.tok_off[1], case.tok_off[2]
    assert torch.equal(step.topk_idx[:a], idx0[:a]) and torch.equal(step.topk_idx[b:T], idx0[b:T])
    assert not torch.equal(step.topk_idx[a:b], idx0[a:b])
    assert torch.equal(step.mb_load[[0, 2, 3]], load0[[0, 2, 3]])
    assert int(step.mb_load[1].sum()) == (b - a) * wl.K


def test_argument_errors_return_codes():
    B = _binding()
    wl = synth.workload("c1")
    step = B.from_workload(wl)
    batch = B.Batch([0, 10, 20], [0, 9])             # layer out of range
    with pytest.raises(B.EbError) as e:
        step.eb_route(batch)
    assert e.value.code == 1
    with pytest.raises(B.EbError):
        step.eb_schedule(B.Batch([0, 10], [0]), 0)   # m < 1
    with pytest.raises(B.EbError):
        step.eb_route(B.Batch([0, 10000], [0]))      # more tokens than the context was sized for
    with pytest.raises(B.EbError) as e:
        step.eb_expert_ffn_grouped()                 # weights not bound
    assert e.value.code == 1
    assert step.device_status() == 0


# ----------------------------------------------------------------------------------- CTA-pair tiles
@pytest.mark.parametrize("H,I", [(192, 328), (520, 264)])
def test_group_sizes_around_the_tile_boundaries(H, I):
    """Exact group sizes on both sides of every place where the expert kernel's tiling changes: the 16-row
    steps of a tile's column count, the 128 rows one CTA of a pair loads, and the 256-row limit at which a group
    is cut into two, three, four nearly equal tiles; output widths that end inside the first CTA's half of an
    output tile, inside the second, and just past a whole tile.  Every row of every group is compared."""
    sizes = [1, 8, 15, 16, 17, 31, 32, 33, 48, 63, 64, 65, 96, 97, 112, 128, 129, 144, 160, 255, 256, 257, 288, 511, 512,
             513, 767, 768, 769, 1000, 0]
    E = len(sizes)
    wl = synth.Workload(name="tiles", L=1, E=E, K=1, S=0, H=H, I=I, D=2, mapping="mod", N=1, T=sum(sizes),
                        zipf_s=0.0)
    store = Hn.WeightStore(wl)
    case = Hn.make_case(wl)
    logits = torch.full((wl.T, E), -4.0)
    t = 0
    for e, n in enumerate(sizes):
        logits[t:t + n, e] = 6.0
        t += n
    perm = torch.from_numpy(np.random.default_rng(5).permutation(wl.T))
    case.logits = logits[perm].contiguous()
    step, ref = _full_step(case, store, 1)
    assert sorted(np.diff(ref["group_off"]).tolist()) == sorted(sizes)


# ----------------------------------------------------------------------------------- failure reporting
def test_bounded_wait_gives_up_and_reports_without_harming_the_context():
    B = _binding()
    wl = synth.workload("c1")
    case = Hn.make_case(wl)
    store = Hn.WeightStore(wl)
    step, ref = _full_step(case, store, wl.m)
    want = step.out[:case.T_tot].clone()
    assert step.selftest_bounded_wait(2_000_000) == 1          # the wait ran out (about a millisecond)
    assert step.device_status() == 5                            # EB_ERR_TIMEOUT was recorded ...
    assert step.device_status() == 0                            # ... and reading it clears it
    batch = B.Batch(case.tok_off, case.layers)
    step.eb_step(batch, wl.m)                                   # the context is still usable
    torch.cuda.synchronize()
    assert torch.equal(step.out[:case.T_tot], want)
    assert step.device_status() == 0


# ----------------------------------------------------------------------------------- extreme shapes
def test_minimal_hidden_sizes_and_maximum_slots():
    # H = I = 8 (one 16-byte vector per row) and K + S = 16 slots per token
    wl = _small(L=2, E=16, K=8, S=8, D=4, N=3, T=20, H=8, I=8, mapping="mod")
    _full_step(Hn.make_case(wl, [20, 1, 45], [0, 1, 1]), Hn.WeightStore(wl), 2)


def test_sixteen_micro_batches_on_one_layer():
    wl = _small(L=1, E=8, K=2, S=1, D=4, N=16, T=40, H=128, I=192, mapping="contiguous", zipf_s=0.3)
    _full_step(Hn.make_case(wl, [40 + 3 * (j % 4) for j in range(16)], [0] * 16), Hn.WeightStore(wl), 12)


# ----------------------------------------------------------------------------------- CUDA graph
def test_step_replayed_from_a_cuda_graph_matches_eager():
    """The five calls only enqueue work on the stream, so a whole step can be captured once and replayed;
    new inputs are written into the same device buffers between replays."""
    B = _binding()
    wl = synth.workload("c1")
    store = Hn.WeightStore(wl)
    step = B.from_workload(wl)
    step.bind_weights(store.gate, store.up, store.down)
    batch = B.Batch(wl.tok_off, wl.layers)
    T = wl.T_tot
    case_a = Hn.make_case(wl)
    case_b = Hn.make_case(synth.workload("c1", seed=77))
    step.logits[:T].copy_(case_a.logits)
    step.x[:T].copy_(case_a.x)
    step.eb_step(batch, wl.m)                     # warm-up outside capture (first-use set-up)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step.eb_step(batch, wl.m)
    for case in (case_b, case_a, case_b):
        step.logits[:T].copy_(case.logits)
        step.x[:T].copy_(case.x)
        step.out.fill_(-7.0)
        graph.replay()
        torch.cuda.synchronize()
        replayed = step.out[:T].clone()
        mask_replayed = step.sched_result()["run_mask"]
        step.out.fill_(-7.0)
        step.eb_step(batch, wl.m)
        torch.cuda.synchronize()
        assert step.sched_result()["run_mask"] == mask_replayed
        assert torch.equal(step.out[:T], replayed)
    assert step.device_status() == 0


def test_workspace_guards_detect_a_write_past_a_region():
    B = _binding()
    wl = synth.workload("c1")
    step = B.from_workload(wl)
    assert step.check_workspace_guards() == 0
    # the first guard follows the first region (per-chunk histograms): overwrite three of its bytes from the host side
    first_region = 4 * ((wl.T_tot + 31) // 32 + B.EB_MAX_MB) * wl.E
    off = (first_region + 255) // 256 * 256
    step.workspace[off + 5:off + 8] = 0
    assert step.check_workspace_guards() == 3
    step.workspace[off + 5:off + 8] = 0xA5
    assert step.check_workspace_guards() == 0


def test_device_side_checker_flags_corrupted_tables():
    B = _binding()
    wl = synth.workload("c1")
    case = Hn.make_case(wl)
    step, ref = _full_step(case, Hn.WeightStore(wl), wl.m, check_ffn=False)
    batch = B.Batch(case.tok_off, case.layers)
    assert step.check_permutation(batch) == 0
    t_run = int(np.nonzero(ref["pos"][:, 0] >= 0)[0][0])
    saved = step.pos.clone()
    step.pos[t_run, 0] = 10 ** 6                      # out of range: reported, never dereferenced
    assert step.check_permutation(batch) > 0
    step.pos.copy_(saved)
    step.pos[t_run, 0], step.pos[t_run, 1] = int(saved[t_run, 1]), int(saved[t_run, 0])   # swapped slots
    assert step.check_permutation(batch) > 0
    step.pos.copy_(saved)
    step.row_src[0] = -3
    assert step.check_permutation(batch) > 0
    assert step.device_status() == 0


def test_c5_sweep_point_full_step():
    # the most skewed point of the sweep with the largest micro-batch count
    wl = synth.workload_c5(16, 128, 1.5)
    _full_step(Hn.make_case(wl), Hn.WeightStore(wl), wl.m)


def test_schedule_large_pools_split_over_blocks():
    """Pools of 12 to 16 members: the MaxUtil enumeration runs on several blocks; ties are frequent with
    these small loads, so the total order is exercised across block boundaries."""
    B = _binding()
    rng = np.random.default_rng(777)
    wl = _small(D=4)
    step = B.from_workload(wl, max_tokens=64)
    for trial in range(10):
        n_mb = 16
        np_pool = [12, 13, 14, 15, 16][trial % 5]
        members = sorted(rng.choice(n_mb, size=np_pool, replace=False).tolist())
        pool = sum(1 << j for j in members)
        m = int(rng.integers(max(1, np_pool - 5), np_pool))
        loads = rng.integers(0, 4 if trial % 2 else 40, size=(n_mb, 4)).astype(np.int32)
        dev_loads = torch.from_numpy(loads).cuda()
        batch = B.Batch([0] * (n_mb + 1), [0] * n_mb, pool)
        got = step.eb_schedule(batch, m, O.POLICY_MAXUTIL, to_host=True, mb_load=dev_loads)
        ref = O.schedule(loads, pool, m, O.POLICY_MAXUTIL)
        for k in ("run_mask", "defer_mask", "n_run", "joint_load", "util_num", "util_den"):
            assert got[k] == ref[k], (trial, k, got[k], ref[k])


# ----------------------------------------------------------------------------------- randomised shapes
def test_random_shapes_front_end_bit_exact():
    """Routing, scheduling and permutation on 120 random shapes (experts, top-k, shared experts, devices,
    micro-batch sizes, layers, pool, m, policy, mapping) against the oracle, bit for bit."""
    rng = np.random.default_rng(2026)
    for trial in range(120):
        E = int(rng.integers(1, 40))
        K = int(rng.integers(1, min(E, 8) + 1))
        S = int(rng.integers(0, 4))
        D = int(rng.integers(1, 9))
        N = int(rng.integers(1, 9))
        L = int(rng.integers(1, 6))
        tokens = [int(v) for v in rng.integers(0, 70, size=N)]
        if sum(tokens) == 0:
            tokens[0] = 3
        layers = [int(v) for v in rng.integers(0, L, size=N)]
        pool = int(rng.integers(0, 1 << N))
        m = int(rng.integers(1, N + 1))
        policy = int(rng.integers(0, 4))
        wl = synth.Workload(name=f"rnd{trial}", L=L, E=E, K=K, S=S, H=64, I=64, D=D,
                            mapping=["mod", "contiguous"][trial % 2], N=N, T=8, zipf_s=float(rng.uniform(0, 1.5)),
                            renorm_topk=trial % 3 != 0, seed=1000 + trial)
        case = Hn.make_case(wl, tokens, layers)
        _full_step(case, Hn.WeightStore(wl), m, policy, pool_mask=pool, check_ffn=(trial % 6 == 0))


def test_other_policies_on_the_decode_and_fine_grained_shapes():
    for name in ("c2", "c3"):
        wl = synth.workload(name)
        store = Hn.WeightStore(wl)
        case = Hn.make_case(wl)
        for pol in (O.POLICY_CUMUTIL, O.POLICY_DIFFPEAK, O.POLICY_ALL):
            _full_step(case, store, wl.m, pol, check_ffn=False)


def test_random_expert_shapes_full_compare():
    """Hidden and intermediate sizes that are multiples of 8 but of nothing larger, group sizes on both
    sides of the 32-, 128- and 256-row tile boundaries, with and without shared experts: every expert output
    and every aggregated output is compared."""
    rng = np.random.default_rng(4242)
    for trial in range(16):
        H = 8 * int(rng.integers(1, 70))
        I = 8 * int(rng.integers(1, 70))
        E = int(rng.integers(2, 7))
        K = int(rng.integers(1, min(E, 3) + 1))
        S = int(rng.integers(0, 3))
        D = int(rng.integers(1, 5))
        N = int(rng.integers(1, 4))
        tokens = [int(v) for v in rng.choice([1, 7, 33, 120, 129, 260, 400, 700], size=N)]
        layers = [int(v) for v in rng.integers(0, 2, size=N)]
        wl = synth.Workload(name=f"ffn{trial}", L=2, E=E, K=K, S=S, H=H, I=I, D=D, mapping="mod", N=N, T=8,
                            zipf_s=float(rng.uniform(0, 2.0)), seed=500 + trial)
        _full_step(Hn.make_case(wl, tokens, layers), Hn.WeightStore(wl), max(1, N - 1))
