"""eb_permute_noalloc: the dispatch step for callers that cannot allocate device memory at the
point of call (a server whose HBM is fully committed, a plug-in inside another framework's
callback, a latency-critical loop).  It must give exactly what eb_permute gives, call after call,
although all its calls share one static scratch array that keeps the previous call's contents.

Collected last on purpose (file name): a run that stops at the first failure has already run every
other test."""
import pytest
import torch

from paper_2608_07964_b200 import synth

pytestmark = pytest.mark.gpu


def _reference_and_noalloc(B, wl, tokens, layers, pool, m):
    from tests import harness as Hn
    case = Hn.make_case(wl, tokens, layers)
    T = case.T_tot
    step = B.from_workload(wl, max_tokens=max(T, 1))
    step.logits[:T].copy_(case.logits)
    step.x[:T].copy_(case.x)
    batch = B.Batch(case.tok_off, case.layers, pool)
    step.eb_route(batch)
    step.eb_schedule(batch, m)
    step.eb_permute(batch)                                   # existing entry point: context + workspace
    torch.cuda.synchronize()
    meta = step.meta()
    G, R = meta["groups"], meta["rows"]
    want = dict(group_off=step.group_off[:G + 1].clone(), group_w=step.group_w[:G].clone(),
                row_src=step.row_src[:R].clone(), pos=step.pos[:T].clone(), xp=step.xp[:R].clone(),
                meta=step.step_meta.clone())

    # caller-owned outputs, poisoned so that anything left unwritten shows up
    i32 = torch.int32
    out = dict(group_off=torch.full_like(step.group_off, -9), group_w=torch.full_like(step.group_w, -9),
               row_src=torch.full_like(step.row_src, -9), pos=torch.full_like(step.pos, -9),
               xp=torch.full_like(step.xp, 5.0), meta=torch.full((B.EB_META_LEN,), -9, dtype=i32, device="cuda"))
    B.permute_noalloc(wl.L, wl.E, wl.K, wl.S, wl.H, wl.D, wl.expert_to_device(), batch, step.sched, step.x,
                      step.topk_idx, out["group_off"], out["group_w"], out["row_src"], out["pos"], out["xp"], out["meta"])
    torch.cuda.synchronize()
    assert torch.equal(out["meta"], want["meta"])
    assert torch.equal(out["group_off"][:G + 1], want["group_off"])
    assert torch.equal(out["group_w"][:G], want["group_w"])
    assert torch.equal(out["row_src"][:R], want["row_src"])
    assert torch.equal(out["pos"][:T], want["pos"])
    assert torch.equal(out["xp"][:R].view(torch.int16), want["xp"].view(torch.int16))
    return R


def test_noalloc_matches_eb_permute_on_two_calls_in_a_row():
    from paper_2608_07964_b200 import binding as B
    # first call: the 4-layer / 8-expert configuration; second call: another shape, pool and routing,
    # so stale scratch from the first call would change the result if it were not re-initialised
    r1 = _reference_and_noalloc(B, synth.workload("c1"), None, None, 0b1111, 3)
    wl2 = synth.Workload(name="na2", L=3, E=12, K=3, S=2, H=64, I=64, D=4, mapping="mod", N=5, T=8, zipf_s=0.7)
    r2 = _reference_and_noalloc(B, wl2, [40, 7, 0, 33, 130], [2, 0, 1, 0, 2], 0b11011, 2)
    r3 = _reference_and_noalloc(B, synth.workload("c1"), None, None, 0b0101, 1)
    assert r1 > 0 and r2 > 0 and r3 > 0


def test_noalloc_rejects_sizes_beyond_its_static_scratch():
    from paper_2608_07964_b200 import binding as B
    wl = synth.Workload(name="big", L=2, E=8, K=2, S=0, H=64, I=64, D=2, mapping="mod", N=2, T=2049, zipf_s=0.0)
    batch = B.Batch([0, 2049, 4098], [0, 1])
    z = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(B.EbError) as e:
        B.permute_noalloc(wl.L, wl.E, wl.K, wl.S, wl.H, wl.D, wl.expert_to_device(), batch, z, z, z, z, z, z, z, z, z)
    assert e.value.code == 2 and "4096" in str(e.value)
