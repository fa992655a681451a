"""eb_permute_noalloc: the dispatch step for callers that cannot allocate device memory at the
point of call (a server whose HBM is fully committed, a plug-in inside another framework's
callback, a latency-critical loop).  It must give what the oracle's dispatch gives (and so what
eb_permute gives), call after call, although all its calls share one static scratch array that keeps
the previous call's contents; and it must not allocate.

Collected last on purpose (file name): a run that stops at the first failure has already run every
other test."""
import numpy as np
import pytest
import torch

from oracle import eb_oracle as O
from paper_2608_07964_b200 import synth

pytestmark = pytest.mark.gpu


def _front(B, wl, tokens, layers, pool, m, device="cuda:0"):
    """Routing and schedule on the GPU (inputs of the dispatch) and the oracle's dispatch of the same case."""
    from tests import harness as Hn
    case = Hn.make_case(wl, tokens, layers)
    T = case.T_tot
    step = B.from_workload(wl, max_tokens=max(T, 1), device=device)
    step.logits[:T].copy_(case.logits)
    step.x[:T].copy_(case.x)
    batch = B.Batch(case.tok_off, case.layers, pool)
    step.eb_route(batch)
    step.eb_schedule(batch, m)
    torch.cuda.synchronize(device)
    ref = Hn.oracle_front(case, pool, m, O.POLICY_MAXUTIL)
    return case, step, batch, ref


def _poisoned_outputs(B, step):
    # caller-owned outputs, poisoned so that anything left unwritten shows up
    return dict(group_off=torch.full_like(step.group_off, -9), group_w=torch.full_like(step.group_w, -9),
                row_src=torch.full_like(step.row_src, -9), pos=torch.full_like(step.pos, -9),
                xp=torch.full_like(step.xp, 5.0),
                meta=torch.full((B.EB_META_LEN,), -9, dtype=torch.int32, device=step.xp.device))


def _call(B, wl, step, batch, out, topk_idx=None):
    B.permute_noalloc(wl.L, wl.E, wl.K, wl.S, wl.H, wl.D, wl.expert_to_device(), batch, step.sched, step.x,
                      step.topk_idx if topk_idx is None else topk_idx, out["group_off"], out["group_w"],
                      out["row_src"], out["pos"], out["xp"], out["meta"])


def _check_against_oracle(case, wl, out, ref):
    from tests import harness as Hn
    T = case.T_tot
    G, R = len(ref["group_w"]), int(ref["group_off"][-1])
    meta = out["meta"].cpu().numpy()
    assert meta[0] == R and meta[1] == G and meta[-1] == 0
    assert np.array_equal(out["group_off"][:G + 1].cpu().numpy(), ref["group_off"])
    assert np.array_equal(out["group_w"][:G].cpu().numpy(), ref["group_w"])
    assert np.array_equal(out["row_src"][:R].cpu().numpy(), ref["row_src"])
    assert np.array_equal(out["pos"][:T].cpu().numpy(), ref["pos"])
    assert np.array_equal(Hn.bf16_bits(out["xp"][:R]), ref["xp_bits"])
    return R


def _oracle_and_noalloc(B, wl, tokens, layers, pool, m, stream=None, device="cuda:0"):
    case, step, batch, ref = _front(B, wl, tokens, layers, pool, m, device)
    out = _poisoned_outputs(B, step)
    # the existing entry point on the same inputs must agree too
    step.eb_permute(batch)
    free0 = torch.cuda.mem_get_info(step.xp.device)[0]
    launches0 = B.launch_count()
    if stream is None:
        _call(B, wl, step, batch, out)
    else:
        stream.wait_stream(torch.cuda.current_stream(step.xp.device))
        with torch.cuda.stream(stream):
            _call(B, wl, step, batch, out)
        stream.synchronize()
    torch.cuda.synchronize(step.xp.device)
    assert torch.cuda.mem_get_info(step.xp.device)[0] == free0, "the call changed the device's free memory"
    assert B.launch_count() == launches0, "launches of the allocation-free entry point are documented as not counted"
    R = _check_against_oracle(case, wl, out, ref)
    G = len(ref["group_w"])
    assert torch.equal(out["group_off"][:G + 1], step.group_off[:G + 1]) and torch.equal(out["pos"], step.pos)
    assert torch.equal(out["xp"][:R].view(torch.int16), step.xp[:R].view(torch.int16))
    return R


def test_noalloc_matches_the_oracle_on_calls_in_a_row():
    from paper_2608_07964_b200 import binding as B
    # warm-up call: resolves the scratch array's address on this device (and loads the kernels), so that
    # the free-memory comparison around the later calls sees the steady state
    case, step, batch, ref = _front(B, synth.workload("c1"), None, None, 0b1111, 3)
    _call(B, synth.workload("c1"), step, batch, _poisoned_outputs(B, step))
    torch.cuda.synchronize()
    # first call: the 4-layer / 8-expert configuration; second call: another shape, pool and routing,
    # so stale scratch from the first call would change the result if it were not re-initialised
    r1 = _oracle_and_noalloc(B, synth.workload("c1"), None, None, 0b1111, 3)
    wl2 = synth.Workload(name="na2", L=3, E=12, K=3, S=2, H=64, I=64, D=4, mapping="mod", N=5, T=8, zipf_s=0.7)
    r2 = _oracle_and_noalloc(B, wl2, [40, 7, 0, 33, 130], [2, 0, 1, 0, 2], 0b11011, 2)
    r3 = _oracle_and_noalloc(B, synth.workload("c1"), None, None, 0b0101, 1)
    # and on a stream of the caller's, not the default one
    r4 = _oracle_and_noalloc(B, wl2, [64, 64, 1, 200, 31], [0, 0, 1, 2, 2], 0b11111, 3, stream=torch.cuda.Stream())
    assert r1 > 0 and r2 > 0 and r3 > 0 and r4 > 0


def test_noalloc_rejects_sizes_beyond_its_static_scratch():
    from paper_2608_07964_b200 import binding as B
    wl = synth.Workload(name="big", L=2, E=8, K=2, S=0, H=64, I=64, D=2, mapping="mod", N=2, T=2049, zipf_s=0.0)
    batch = B.Batch([0, 2049, 4098], [0, 1])
    z = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(B.EbError) as e:
        B.permute_noalloc(wl.L, wl.E, wl.K, wl.S, wl.H, wl.D, wl.expert_to_device(), batch, z, z, z, z, z, z, z, z, z)
    assert e.value.code == 2 and "4096" in str(e.value)
    assert "context" not in str(e.value)


def test_noalloc_skips_and_counts_a_routing_index_out_of_range():
    # this entry point has no context, so its routing indices are arbitrary caller data: an index outside
    # [0, E) must never be used as an index; the slot gets no row and step_meta's last word counts it
    from paper_2608_07964_b200 import binding as B
    wl = synth.workload("c1")
    case, step, batch, ref = _front(B, wl, None, None, 0b1111, 4)
    bad = step.topk_idx.clone()
    run = [j for j in range(wl.N) if (ref["sched"]["run_mask"] >> j) & 1]
    t_bad = case.tok_off[run[0]] + 3
    bad[t_bad, 1] = wl.E + 1000
    bad[t_bad + 1, 0] = -5
    out = _poisoned_outputs(B, step)
    _call(B, wl, step, batch, out, topk_idx=bad)
    torch.cuda.synchronize()
    meta = out["meta"].cpu().numpy()
    assert meta[-1] == 2
    assert meta[0] == int(ref["group_off"][-1]) - 2
    pos = out["pos"].cpu().numpy()
    assert pos[t_bad, 1] == -1 and pos[t_bad + 1, 0] == -1
    assert pos[t_bad, 0] >= 0 and (pos[pos >= 0] < meta[0]).all()


@pytest.mark.skipif(torch.cuda.device_count() < 2, reason="needs a second GPU")
def test_noalloc_on_a_second_device():
    from paper_2608_07964_b200 import binding as B
    with torch.cuda.device(1):
        case, step, batch, ref = _front(B, synth.workload("c1"), None, None, 0b1111, 3, device="cuda:1")
        _call(B, synth.workload("c1"), step, batch, _poisoned_outputs(B, step))   # resolves the address on this device
        torch.cuda.synchronize()
        assert _oracle_and_noalloc(B, synth.workload("c1"), None, None, 0b1111, 3, device="cuda:1") > 0
