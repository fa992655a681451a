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


def test_full_chain_matches_oracle_chain_on_c1():
    """Every step executed in full with the residual carried between layers; the oracle runs the
    same schedule in fp32 without intermediate rounding."""
    from paper_2608_07964_b200 import binding as B, driver
    wl = synth.workload("c1")
    bias = synth.zipf_bias(wl)
    store = Hn.WeightStore(wl)
    step = B.from_workload(wl)
    step.bind_weights(store.gate, store.up, store.down)
    x0 = torch.cat([synth.hidden_for(wl, j, 0, "cuda") for j in range(wl.N)], 0)
    logits_of = lambda j, l: synth.logits_for(wl, j, l, "cuda", bias)
    got = driver.run_full(step, wl.tok_off, wl.L, wl.m, O.POLICY_MAXUTIL, logits_of, x0)
    assert step.device_status() == 0

    dev = wl.expert_to_device()
    x = x0.float().cpu().numpy()
    layer = [0] * wl.N
    idx = np.zeros((wl.T_tot, wl.K), dtype=np.int32)
    w = np.zeros((wl.T_tot, wl.K), dtype=np.float32)
    loads = np.zeros((wl.N, wl.D), dtype=np.int64)
    pool = (1 << wl.N) - 1
    route_mask = pool
    n_steps = 0
    while pool:
        for j in range(wl.N):
            if (route_mask >> j) & 1:
                a, b = wl.tok_off[j], wl.tok_off[j + 1]
                lg = synth.logits_for(wl, j, layer[j], "cpu", bias).numpy()
                idx[a:b], w[a:b], ld, _ = O.route(lg, wl.K, dev, wl.D, [0, wl.T])
                loads[j] = ld[0]
        sched = O.schedule(loads, pool, wl.m)
        run = sched["run_mask"]
        assert got["steps"][n_steps]["run_mask"] == run
        goff, gw, row_src, pos, xp, _ = O.permute(x, idx, run, [min(l, wl.L - 1) for l in layer], wl.tok_off, dev,
                                                  wl.E, wl.K, wl.S, wl.D)
        y = O.expert_ffn(xp, goff, gw, store.get)
        out, done = O.combine(y, pos, w, wl.K, wl.S)
        x[done] += out[done]
        n_steps += 1
        route_mask = 0
        for j in range(wl.N):
            if (run >> j) & 1:
                layer[j] += 1
                if layer[j] >= wl.L:
                    pool &= ~(1 << j)
                else:
                    route_mask |= 1 << j
    assert n_steps == len(got["steps"])
    xg = got["x"].float().cpu().numpy()
    assert Hn.within_bar(xg, x), f"final hidden states off by {Hn.worst(xg, x):.2f} x bar"


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
