"""The seeded input generator: reproducible, per-unit addressable, shaped like the workloads."""
import torch

from paper_2404_01365_b200 import synth


def test_workloads_match_the_named_shapes():
    w = synth.WORKLOADS
    assert (w["tiny_swiglu_f32"].d, w["tiny_swiglu_f32"].d_ff, w["tiny_swiglu_f32"].S) == (256, 688, 64)
    assert (w["llama2_7b"].d, w["llama2_7b"].d_ff, w["llama2_7b"].L) == (4096, 11008, 32)
    assert (w["gemma_7b"].d, w["gemma_7b"].d_ff, w["gemma_7b"].act) == (3072, 24576, synth.GEGLU_TANH)
    assert (w["llama2_13b"].d, w["llama2_13b"].d_ff, w["llama2_13b"].B) == (5120, 13824, 8)
    assert w["mistral_7b"].keeps == (0.25, 0.5, 0.75, 1.0)
    assert (w["opt_6p7b"].d, w["opt_6p7b"].d_ff, w["opt_6p7b"].act) == (4096, 16384, synth.RELU)
    assert synth.make_weights(synth.scaled(w["opt_6p7b"], d=64, d_ff=96), 0)[0] is None   # no W_g without a gate


def test_generation_is_reproducible_and_unit_addressable():
    w = synth.scaled(synth.WORKLOADS["llama2_7b"], d=64, d_ff=96, S=8, T=3)
    a = synth.make_weights(w, 3)
    b = synth.make_weights(w, 3)
    c = synth.make_weights(w, 4)
    assert all(torch.equal(p, q) for p, q in zip(a, b))
    assert not torch.equal(a[0], c[0]) and not torch.equal(a[0], a[1])
    assert a[0].shape == (96, 64) and a[2].shape == (64, 96) and a[0].dtype == torch.bfloat16
    x0, x1 = synth.make_prompt(w, 0, 0), synth.make_prompt(w, 0, 1)
    assert x0.shape == (8, 64) and not torch.equal(x0, x1)
    assert torch.equal(x0, synth.make_prompt(w, 0, 0))
    assert synth.make_decode_inputs(w, 0, 0).shape == (3, 64)


def test_hidden_states_carry_the_shared_direction():
    w = synth.scaled(synth.WORKLOADS["tiny_swiglu_f32"], S=4096)
    x = synth.make_prompt(w, 0, 0).double()
    xd = synth.make_decode_inputs(w, 0, 0, T=4096).double()
    m, md = x.mean(0), xd.mean(0)
    assert abs(float(m.norm()) - 2.0) < 0.3            # mean direction of norm 2
    assert float(torch.dot(m, md) / (m.norm() * md.norm())) > 0.9   # decode shares it
    assert abs(float(x.var(0).mean()) - 1.0) < 0.05


def test_weight_scale():
    w = synth.WORKLOADS["tiny_swiglu_f32"]
    wg, wu, wd = synth.make_weights(w, 0)
    assert abs(float(wg.var()) * w.d - 1.0) < 0.05
    assert abs(float(wd.var()) * w.d_ff - 1.0) < 0.05


def test_shard_units_partition():
    for n in (1, 7, 32, 40):
        for world in (1, 2, 3, 8):
            got = [u for r in range(world) for u in synth.shard_units(n, r, world)]
            assert got == list(range(n))
            sizes = [len(synth.shard_units(n, r, world)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
