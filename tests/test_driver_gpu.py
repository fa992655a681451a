"""Algorithm 1 driven through the library (route + schedule on the GPU every step) against the
oracle's Algorithm 1 on loads routed by the oracle from the same seeded logits."""
import numpy as np
import pytest
import torch

from oracle import eb_oracle as O
from paper_2608_07964_b200 import synth
from tests import harness as Hn

pytestmark = pytest.mark.gpu


def _oracle_loads(wl, bias):
    dev = wl.expert_to_device()
    cache = {}

    def load_of(j, l):
        if (j, l) not in cache:
            lg = synth.logits_for(wl, j, l, "cpu", bias).numpy()
            cache[(j, l)] = O.route(lg, wl.K, dev, wl.D, [0, wl.T])[2][0]
        return cache[(j, l)]
    return load_of


@pytest.mark.parametrize("name,kw", [("c1", {}), ("c5", dict(N=8, T=128, s=1.0)), ("c5", dict(N=4, T=16, s=1.5))])
def test_load_trace_matches_oracle_algorithm1(name, kw):
    from paper_2608_07964_b200 import binding as B, driver
    wl = synth.workload(name) if name != "c5" else synth.workload_c5(**kw)
    bias = synth.zipf_bias(wl)
    load_of = _oracle_loads(wl, bias)
    step = B.from_workload(wl)
    logits_of = lambda j, l: synth.logits_for(wl, j, l, "cuda", bias)
    for pol in (O.POLICY_MAXUTIL, O.POLICY_CUMUTIL, O.POLICY_DIFFPEAK, O.POLICY_ALL):
        got = driver.run_load_trace(step, wl.tok_off, wl.L, wl.m, pol, logits_of)
        ref = O.run_algorithm1(load_of, wl.N, wl.L, wl.D, wl.m, pol)
        assert len(got) == len(ref)
        for g, r in zip(got, ref):
            assert g["pool"] == r["pool"] and g["run_mask"] == r["run_mask"]
            assert g["layers"] == r["layers"] and g["joint_load"] == r["joint_load"]
            assert g["member_loads"] == r["member_loads"]
        n, d = O.idle_cross_layer(ref, wl.D)
        fr = driver.idle_fractions(got, wl.D)
        assert abs(fr["idle_cross_layer"] - n / d) < 1e-12
        n2, d2 = O.idle_each_alone(ref, wl.D)
        assert abs(fr["idle_each_alone"] - n2 / d2) < 1e-12
        assert fr["idle_cross_layer"] <= fr["idle_each_alone"] + 1e-12     # combining never hurts (Section 4.1)


def _oracle_chain(wl, bias, store, x0, policy=O.POLICY_MAXUTIL):
    """Algorithm 1 with every step executed by the oracle in fp32 (no intermediate rounding), the residual
    h <- h + MLP(h) of Section 2.1 carried between layers.  Returns the final hidden states and the run sets."""
    dev = wl.expert_to_device()
    cache = {}

    def get(wi):
        if wi not in cache:
            cache[wi] = store.get(wi)
        return cache[wi]

    x = x0.float().cpu().numpy()
    layer = [0] * wl.N
    idx = np.zeros((wl.T_tot, wl.K), dtype=np.int32)
    w = np.zeros((wl.T_tot, wl.K), dtype=np.float32)
    loads = np.zeros((wl.N, wl.D), dtype=np.int64)
    pool = (1 << wl.N) - 1
    route_mask = pool
    runs = []
    while pool:
        for j in range(wl.N):
            if (route_mask >> j) & 1:
                a, b = wl.tok_off[j], wl.tok_off[j + 1]
                lg = synth.logits_for(wl, j, layer[j], "cpu", bias).numpy()
                idx[a:b], w[a:b], ld, _ = O.route(lg, wl.K, dev, wl.D, [0, wl.T])
                loads[j] = ld[0]
        run = O.schedule(loads, pool, wl.m, policy)["run_mask"]
        runs.append(run)
        goff, gw, row_src, pos, xp, _ = O.permute(x, idx, run, [min(l, wl.L - 1) for l in layer], wl.tok_off, dev,
                                                  wl.E, wl.K, wl.S, wl.D)
        y = O.expert_ffn(xp, goff, gw, get)
        nxt, done = O.combine(y, pos, w, wl.K, wl.S, residual=x)
        x[done] = nxt[done]
        route_mask = 0
        for j in range(wl.N):
            if (run >> j) & 1:
                layer[j] += 1
                if layer[j] >= wl.L:
                    pool &= ~(1 << j)
                else:
                    route_mask |= 1 << j
    return x, runs


@pytest.mark.parametrize("name", ["c1", "c5_cut", "shared_small"])
def test_full_chain_matches_oracle_chain(name):
    """Every step executed in full (one eb_step per step, the aggregation adding the residual in place) against
    the oracle running the same schedule in fp32: the tiny shape, a point of the sweep shape (64 experts, top-6,
    no shared experts, cut to 3 layers so that the oracle finishes in seconds) and a small shape with shared
    experts.  The same run replayed from CUDA graphs must give the same bits."""
    from paper_2608_07964_b200 import binding as B, driver
    if name == "c1":
        wl = synth.workload("c1")
    elif name == "c5_cut":
        wl = synth.workload_c5(4, 16, 1.0, L=3)
    else:
        wl = synth.Workload(name="chain_shared", L=3, E=6, K=2, S=2, H=72, I=200, D=3, mapping="mod", N=4, T=24, zipf_s=1.0)
    bias = synth.zipf_bias(wl)
    store = Hn.WeightStore(wl)
    step = B.from_workload(wl)
    step.bind_weights(store.gate, store.up, store.down)
    x0 = torch.cat([synth.hidden_for(wl, j, 0, "cuda") for j in range(wl.N)], 0)
    logits_of = lambda j, l: synth.logits_for(wl, j, l, "cuda", bias)
    got = driver.run_full(step, wl.tok_off, wl.L, wl.m, O.POLICY_MAXUTIL, logits_of, x0)
    assert step.device_status() == 0
    x_ref, runs = _oracle_chain(wl, bias, store, x0)
    assert [s["run_mask"] for s in got["steps"]] == runs
    xg = got["x"].float().cpu().numpy()
    assert Hn.within_bar(xg, x_ref), f"final hidden states off by {Hn.worst(xg, x_ref):.2f} x bar"
    assert got["ms"] > 0 and got["token_layers"] == wl.T_tot * wl.L

    graphs = driver.StepGraphs(step, wl.tok_off)
    first = driver.run_full(step, wl.tok_off, wl.L, wl.m, O.POLICY_MAXUTIL, logits_of, x0, graphs=graphs)
    again = driver.run_full(step, wl.tok_off, wl.L, wl.m, O.POLICY_MAXUTIL, logits_of, x0, graphs=graphs)
    assert graphs.captures == len(runs) and graphs.hits == len(runs)      # the second run replays every step
    assert torch.equal(first["x"], got["x"]) and torch.equal(again["x"], got["x"])
    assert step.device_status() == 0


def test_combine_with_residual_alone():
    """eb_combine_residual fed with the oracle's expert outputs (rounded to bf16) against the oracle's aggregation
    with the residual, including the in-place form (residual and out the same buffer)."""
    from paper_2608_07964_b200 import binding as B
    wl = synth.Workload(name="res", L=2, E=6, K=3, S=1, H=264, I=64, D=3, mapping="mod", N=3, T=40, zipf_s=0.5)
    case = Hn.make_case(wl, [40, 17, 33], [0, 1, 1])
    step = B.from_workload(wl, max_tokens=case.T_tot)
    T = case.T_tot
    step.logits[:T].copy_(case.logits)
    step.x[:T].copy_(case.x)
    batch = B.Batch(case.tok_off, case.layers, 0b111)
    step.eb_route(batch)
    step.eb_schedule(batch, 2)
    step.eb_permute(batch)
    ref = Hn.oracle_front(case, 0b111, 2, O.POLICY_MAXUTIL)
    R = int(ref["group_off"][-1])
    rng = np.random.default_rng(5)
    y = torch.from_numpy(rng.normal(size=(R, wl.H)).astype(np.float32)).to(torch.bfloat16)
    step.yp[:R].copy_(y)
    x32 = case.x.float().numpy()
    want, done = O.combine(y.float().numpy(), ref["pos"], ref["w"], wl.K, wl.S, residual=x32)
    step.out.fill_(-7.0)
    step.eb_combine(batch, residual=step.x)
    out = step.out[:T].float().cpu().numpy()
    assert Hn.within_bar(out[done], want[done]) and (out[~done] == -7.0).all()
    assert np.abs(out[done] - want[done]).max() <= 2 ** -7 * np.abs(want[done]).max()      # one bf16 rounding
    before = step.x[:T].clone()
    step.eb_combine(batch, out=step.x, residual=step.x)                                  # in place
    assert torch.equal(step.x[:T][torch.from_numpy(done).cuda()], step.out[:T][torch.from_numpy(done).cuda()])
    assert torch.equal(step.x[:T][torch.from_numpy(~done).cuda()], before[torch.from_numpy(~done).cuda()])


@pytest.mark.parametrize("D", [2, 4, 8])
def test_ep_size_sweep_points_match_oracle(D):
    """The expert-parallel size sweep (the paper's table of under-utilisation against EP size: the batch grows with
    the number of devices, 4 micro-batches, m = 3) on a small token count: every step of Algorithm 1 against the
    oracle for the three policies, and the count of consecutive layers with the same skew device against the
    oracle's statistic on the oracle's own loads."""
    from paper_2608_07964_b200 import binding as B, driver
    wl = synth.workload_c5(4, 8 * D, 1.0, D=D, m_override=3)
    bias = synth.zipf_bias(wl)
    load_of = _oracle_loads(wl, bias)
    step = B.from_workload(wl)
    logits_of = lambda j, l: synth.logits_for(wl, j, l, "cuda", bias)
    for pol in (O.POLICY_MAXUTIL, O.POLICY_CUMUTIL, O.POLICY_DIFFPEAK, O.POLICY_ALL):
        got = driver.run_load_trace(step, wl.tok_off, wl.L, wl.m if pol != O.POLICY_ALL else wl.N, pol, logits_of)
        ref = O.run_algorithm1(load_of, wl.N, wl.L, wl.D, wl.m if pol != O.POLICY_ALL else wl.N, pol)
        assert [(g["pool"], g["run_mask"], g["joint_load"]) for g in got] == [(r["pool"], r["run_mask"], r["joint_load"]) for r in ref]
        n, d = O.idle_cross_layer(ref, wl.D)
        assert abs(driver.idle_fractions(got, wl.D)["idle_cross_layer"] - n / d) < 1e-12
    loads = driver.routed_loads(step, wl.tok_off, wl.L, logits_of)
    for j in range(wl.N):
        ref_loads = [[int(v) for v in load_of(j, l)] for l in range(wl.L)]
        assert loads[j] == ref_loads
        for n in (2, 3):
            assert driver.same_peak_windows(loads[j], n) == O.same_peak_windows(ref_loads, n)


def test_emulated_latency_accounts_every_step_and_device():
    """The emulated expert-parallel latency loop takes the same steps as the load trace, costs each step its
    slowest virtual device, and with `alone` executes every (micro-batch, layer) workload by itself."""
    from paper_2608_07964_b200 import binding as B, driver
    wl = synth.workload("c1")
    bias = synth.zipf_bias(wl)
    store = Hn.WeightStore(wl)
    step = B.from_workload(wl)
    step.bind_weights(store.gate, store.up, store.down)
    x0 = torch.cat([synth.hidden_for(wl, j, 0, "cuda") for j in range(wl.N)], 0)
    logits_of = lambda j, l: synth.logits_for(wl, j, l, "cuda", bias)
    trace = driver.run_load_trace(step, wl.tok_off, wl.L, wl.m, O.POLICY_MAXUTIL, logits_of)
    r = driver.run_emulated_latency(step, wl.tok_off, wl.L, wl.D, wl.m, O.POLICY_MAXUTIL, logits_of, x0)
    assert r["steps"] == len(trace)
    assert r["latency_ms"] > 0 and 0 < r["busy_ms"] <= wl.D * r["latency_ms"] * (1 + 1e-6)
    assert 0.0 <= r["idle_time"] < 1.0
    alone = driver.run_emulated_latency(step, wl.tok_off, wl.L, wl.D, 1, O.POLICY_ALL, logits_of, x0, alone=True)
    assert alone["steps"] == wl.N * wl.L
    lock = driver.run_emulated_latency(step, wl.tok_off, wl.L, wl.D, wl.N, O.POLICY_ALL, logits_of, x0)
    assert lock["steps"] == wl.L
    assert step.device_status() == 0
