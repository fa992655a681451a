"""The seeded input generator: slices agree with whole tensors, streams are reproducible and
have the stated moments, workload tables have the stated shapes."""
import numpy as np
import pytest
import torch

from paper_2608_07964_b200 import synth


def test_slices_are_consistent_and_reproducible():
    tid = synth.tensor_id(synth.KIND_W_GATE)
    whole = synth.normal_bf16(1234, tid, 0, 5000, 0.02, chunk=777)
    part = synth.normal_bf16(1234, tid, 1000, 321, 0.02)
    assert torch.equal(whole[1000:1321].view(torch.int16), part.view(torch.int16))
    again = synth.normal_bf16(1234, tid, 0, 5000, 0.02)
    assert torch.equal(whole.view(torch.int16), again.view(torch.int16))
    other = synth.normal_bf16(1235, tid, 0, 5000, 0.02)
    assert not torch.equal(whole.view(torch.int16), other.view(torch.int16))


def test_moments():
    v = synth.normal_f32(synth.BASE_SEED, synth.tensor_id(synth.KIND_X, 3, 2), 0, 400000, 1.0).double()
    assert abs(v.mean().item()) < 0.01 and abs(v.std().item() - 1.0) < 0.01
    assert v.abs().max().item() < 3.47
    w = synth.normal_bf16(synth.BASE_SEED, synth.tensor_id(synth.KIND_W_UP), 0, 400000, 0.02).double()
    assert abs(w.std().item() - 0.02) < 3e-4


def test_expert_weight_is_a_slice_of_the_full_tensor():
    wl = synth.workload("c1")
    full = synth.all_weights(wl, "down")
    assert full.shape == (wl.L, wl.E + wl.S, wl.H, wl.I)
    one = synth.expert_weight(wl, "down", 2, 5)
    assert torch.equal(full[2, 5].view(torch.int16), one.view(torch.int16))
    g = synth.all_weights(wl, "gate")
    assert g.shape == (wl.L, wl.E, wl.I, wl.H)
    assert torch.equal(g[1, 7].view(torch.int16), synth.expert_weight(wl, "gate", 1, 7).view(torch.int16))


def test_workload_tables():
    c1, c2, c3, c4 = (synth.workload(n) for n in ("c1", "c2", "c3", "c4"))
    assert c1.layers == [0, 1, 2, 3] and c1.m == 3 and c1.expert_to_device() == [0, 0, 1, 1, 2, 2, 3, 3]
    assert c2.layers == [3 * j for j in range(8)] and c2.m == 6
    assert c2.expert_to_device()[:10] == [0, 1, 2, 3, 4, 5, 6, 7, 0, 1]
    assert len(set(c3.layers)) == 16 and c3.m == 12
    assert c4.layers == [4 * j for j in range(8)] and c4.weight_bytes() == 3 * 32 * 8 * 4096 * 14336 * 2
    b = synth.zipf_bias(c1)
    assert b.shape == (4, 8) and b.dtype == np.float32
    for l in range(4):                       # a permutation of -s*ln(1..E) per layer
        assert np.allclose(np.sort(-b[l]), np.log(np.arange(1, 9)), atol=1e-6)
    assert not np.array_equal(np.argsort(b[0]), np.argsort(b[1])) or not np.array_equal(np.argsort(b[1]), np.argsort(b[2]))
    lg = synth.packed_logits(c1)
    assert lg.shape == (256, 8) and lg.dtype == torch.float32
    x = synth.packed_hidden(c1)
    assert x.shape == (256, 256) and x.dtype == torch.bfloat16


@pytest.mark.gpu
def test_cpu_and_cuda_streams_are_bit_identical():
    tid = synth.tensor_id(synth.KIND_W_DOWN)
    a = synth.normal_bf16(99, tid, 12345, 100000, 0.02, device="cpu")
    b = synth.normal_bf16(99, tid, 12345, 100000, 0.02, device="cuda").cpu()
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    wl = synth.workload("c1")
    assert torch.equal(synth.packed_logits(wl, device="cuda").cpu(), synth.packed_logits(wl))
