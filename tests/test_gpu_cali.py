"""Thompson sampling with calibration on the GPU (Sec. 3.3, Eq. 5-8, Algorithm 3) against the
oracle: the predictor's output theta_M from the device's own hidden states, the host posterior
arithmetic, and whole generations (draft lengths, accepted counts, tokens) on the tiny fp32
model, where every decision can be followed bit for bit."""
import numpy as np
import pytest
import torch

import eesd_synth as synth
import oracle
from tests.helpers import engine_from_spec, oracle_from_spec

pytestmark = pytest.mark.gpu
SM, SS, TH0 = 0.2, 0.5, 0.5


def _cali_engine(spec, **kw):
    from paper_2406_03853_b200 import binding as b
    eng = engine_from_spec(spec, controller=b.CTRL_CALI_TS, cali_sigma_m=SM, cali_sigma_s=SS, cali_theta0=TH0, **kw)
    cw = synth.cali_weights(spec, device=eng.device)
    g = eng.global_views()
    g["cali_w"].copy_(cw["w"])
    g["cali_wp"].copy_(cw["wp"])
    cwo = synth.cali_weights(spec)
    return eng, dict(w=cwo["w"].float().numpy(), wp=cwo["wp"].numpy(), sigma_m=SM, sigma_s=SS, theta_hat0=TH0)


@pytest.mark.parametrize("variant", ["f32", "bf16_tensor_core"])
def test_predictor_output_matches_oracle_from_the_same_states(variant):
    spec = synth.TINY if variant == "f32" else synth.TINY.with_(dtype="bf16", ffn_dim=640)
    tol = 2e-5 if variant == "f32" else 5e-3
    eng, cali = _cali_engine(spec, max_ctx=96, k_cap=10)
    m = oracle_from_spec(spec, 96)
    prompt = synth.prompt_tokens(31, 23, spec.vocab).numpy()       # 22 rows: the wide prompt path on the bf16 variant
    eng.prefill(prompt)
    hid, _ = m.target_rows(prompt[:-1], 0, want_hidden=True, want_logits=False)
    hT = hid[spec.n_layers, -1]
    tok = int(prompt[-1])
    for step in range(1, 4):                                        # W^1, W^2, W^3
        nxt = int(eng.draft(1)[0])
        lg, hD = m.draft_row(tok, len(prompt) - 1 + step - 1, want_hidden=True)
        assert nxt == int(lg.argmax())
        want = oracle.cali_theta_m(cali["w"][step - 1], cali["wp"], hT, hD)
        assert abs(eng.cali_predict() - want) < tol
        tok = nxt
    # after a verification H^(T) is the row that produced the next token
    drafted = [int(prompt[-1])]
    m2 = oracle_from_spec(spec, 96)
    m2.target_rows(prompt[:-1], 0, want_logits=False)
    for i in range(3):
        drafted.append(int(m2.draft_row(drafted[-1], len(prompt) - 1 + i).argmax()))
    n_acc, y = eng.verify_accept(None, 0.0)
    hid, pl = m2.target_rows(np.array(drafted, np.int32), len(prompt) - 1, want_hidden=True)
    assert y == int(pl[n_acc].argmax())
    nxt = int(eng.draft(1)[0])
    _, hD = m2.draft_row(y, len(prompt) + n_acc, want_hidden=True)
    want = oracle.cali_theta_m(cali["w"][0], cali["wp"], hid[spec.n_layers, n_acc], hD)
    assert abs(eng.cali_predict() - want) < tol
    eng.close()


def test_host_posterior_equals_oracle():
    from paper_2406_03853_b200 import binding as b
    for th_m, th_hat, n in ((0.7, 0.4, 0), (0.31, 0.9, 3), (0.5, 0.5, 1000)):
        assert b.cali_posterior(th_m, th_hat, n, SM, SS) == pytest.approx(oracle.cali_posterior(th_m, th_hat, n, SM, SS), rel=1e-14)
    with pytest.raises(b.EesdError):
        b.cali_posterior(0.5, 0.5, 1, 0.0, 1.0)


@pytest.mark.parametrize("temperature", [0.0, 1.0])
def test_generation_with_calibration_follows_the_oracle_round_by_round(temperature):
    spec = synth.TINY
    eng, cali = _cali_engine(spec, max_ctx=160, k_cap=10, temperature=temperature)
    prompt = synth.prompt_tokens(synth.SEED, 20, spec.vocab).numpy()
    u = {k: v.numpy() for k, v in synth.generate_uniforms(160, 20000).items()}
    out, trace, st = eng.generate(prompt, 48, uniforms=u)
    ref, rtrace, _ = oracle_from_spec(spec, 160).generate(prompt, 48, controller=2, temperature=temperature, uniforms=u, cali=cali)
    np.testing.assert_array_equal(out, ref)
    assert trace == rtrace and len({k for k, _, _ in trace}) > 1
    th, n_verify, trials = eng.cali_state()
    assert n_verify == len(trace) and 0.0 <= th <= 1.0 and trials >= n_verify
    # a second prompt starts from the initial state again
    eng.prefill(prompt[:5])
    assert eng.cali_state() == (TH0, 0, 0)
    eng.close()
