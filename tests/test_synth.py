"""The shared seeded input generators: the properties both sides rely on.  (The generators hold
none of the method's arithmetic; these checks are about the inputs only.)"""
import numpy as np
import pytest
import torch

import eesd_synth as synth


def test_normal_stream_moments_and_independence_of_chunking():
    z = synth.normal_f32(3, 7, 1 << 18).double()
    assert abs(z.mean().item()) < 4 / np.sqrt(z.numel())
    assert abs(z.var().item() - 1.0) < 0.02
    # a counter-based stream: any window equals the same window of a longer draw
    np.testing.assert_array_equal(synth.normal_f32(3, 7, 1000, start=5000).numpy(), z[5000:6000].float().numpy())
    assert not torch.equal(synth.normal_f32(3, 8, 1000), synth.normal_f32(3, 7, 1000))     # streams differ
    assert not torch.equal(synth.normal_f32(4, 7, 1000), synth.normal_f32(3, 7, 1000))     # seeds differ


def test_uniforms_are_multiples_of_2_pow_minus_24_in_the_unit_interval():
    u = synth.uniforms(1, synth.STREAM_ACCEPT, 1 << 16)
    assert u.dtype == torch.float32 and float(u.min()) >= 0.0 and float(u.max()) < 1.0
    m = u.double() * (1 << 24)
    assert torch.equal(m, m.round())
    assert abs(u.double().mean().item() - 0.5) < 4 / np.sqrt(12 * u.numel())


def test_prompt_tokens_are_in_range_and_weights_have_the_stated_scale():
    t = synth.prompt_tokens(2, 4096, 1000)
    assert t.dtype == torch.int32 and int(t.min()) >= 0 and int(t.max()) < 1000
    spec = synth.TINY
    w0, w2 = synth.layer_weights(spec, 0), synth.layer_weights(spec, 2)
    assert abs(w0["wqkv"].double().std().item() - 0.02) < 1e-3
    # Wo and W_down of the layers after the exit depth are damped, the other matrices are not
    assert abs(w2["wo"].double().std().item() - 0.02 * spec.damp) < 1e-3 * spec.damp + 1e-5
    assert abs(w2["wd"].double().std().item() - 0.02 * spec.damp) < 1e-3 * spec.damp + 1e-5
    assert abs(w2["wgu"].double().std().item() - 0.02) < 1e-3
    assert torch.all(w0["g_attn"] == 1.0)
    ex = synth.exit_layer_weights(spec)
    last = synth.layer_weights(spec, spec.n_layers - 1)
    assert all(torch.equal(ex[k], last[k]) for k in last)       # the exit layer starts as a copy of the last layer


@pytest.mark.gpu
def test_generators_give_the_same_bits_on_the_host_and_on_the_device():
    for n, start in ((100000, 0), (4097, 123456789)):
        assert torch.equal(synth.normal_f32(9, 2, n, "cuda", start=start).cpu(), synth.normal_f32(9, 2, n, "cpu", start=start))
        assert torch.equal(synth.uniforms(9, 3, n, "cuda", start=start).cpu(), synth.uniforms(9, 3, n, "cpu", start=start))
    assert torch.equal(synth.prompt_tokens(9, 5000, 32000, "cuda").cpu(), synth.prompt_tokens(9, 5000, 32000))
    spec = synth.TINY.with_(dtype="bf16")
    a, b = synth.layer_weights(spec, 1, device="cuda"), synth.layer_weights(spec, 1)
    assert all(torch.equal(a[k].cpu(), b[k]) for k in b)
    assert torch.equal(synth.embedding(spec, device="cuda").cpu(), synth.embedding(spec))
