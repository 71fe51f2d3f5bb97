"""Pins for the oracle's Thompson sampling with calibration (Sec. 3.3 "TS with Calibration",
Eq. 5-8, Algorithm 3): closed forms, limits, a brute-force Bayesian posterior on a grid, draw
statistics, and the generation loop rebuilt from the model primitives."""
import numpy as np
import pytest

import eesd_synth as synth
import oracle
from tests.helpers import oracle_from_spec, np_softmax


def test_posterior_limits_and_the_two_printed_forms_of_the_variance():
    sm, ss = 0.3, 0.7
    assert oracle.cali_posterior(0.8, 0.2, 0, sm, ss) == pytest.approx((0.8, sm * sm))        # nothing verified: the model's word
    mu, var = oracle.cali_posterior(0.8, 0.2, 10 ** 9, sm, ss)
    assert mu == pytest.approx(0.2, abs=1e-6) and var < 1e-9                                    # samples take over
    for n in (1, 3, 40):
        mu, var = oracle.cali_posterior(0.8, 0.2, n, sm, ss)
        assert 1.0 / var == pytest.approx(1.0 / sm ** 2 + n / ss ** 2)                          # Eq. 7 against Algorithm 3's product form
        assert mu == pytest.approx(var * (0.8 / sm ** 2 + n * 0.2 / ss ** 2))                   # precision-weighted mean
        assert min(0.2, 0.8) < mu < max(0.2, 0.8)


def test_posterior_equals_a_bayesian_update_done_by_brute_force_on_a_grid():
    # prior mu ~ N(theta_M, sigma_M^2); n observations ~ N(mu, sigma_S^2) whose mean is theta_hat
    rng = np.random.default_rng(3)
    th_m, sm, ss, n = 0.65, 0.25, 0.5, 7
    obs = rng.normal(0.3, ss, n)
    grid = np.linspace(-3, 4, 700001)
    logp = -0.5 * ((grid - th_m) / sm) ** 2 - 0.5 * (((obs[:, None] - grid[None, :]) / ss) ** 2).sum(0)
    w = np.exp(logp - logp.max())
    w /= w.sum()
    mean = (w * grid).sum()
    var = (w * (grid - mean) ** 2).sum()
    mu, v = oracle.cali_posterior(th_m, float(obs.mean()), n, sm, ss)
    assert mu == pytest.approx(mean, abs=1e-6) and v == pytest.approx(var, rel=1e-5)


def test_theta_m_is_the_class_one_probability_of_a_two_class_softmax():
    rng = np.random.default_rng(5)
    d = 12
    Wi, Wp = rng.normal(0, 0.3, (d, d)).astype(np.float32), rng.normal(0, 0.3, (2, 2 * d)).astype(np.float32)
    hT, hD = rng.normal(0, 1, d), rng.normal(0, 1, d)
    z = np.concatenate([Wi.astype(np.float64) @ hT, hD])
    want = np_softmax(Wp.astype(np.float64) @ z)[1]
    got = oracle.cali_theta_m(Wi, Wp, hT, hD)
    assert got == pytest.approx(want, abs=1e-12)
    assert oracle.cali_theta_m(Wi, Wp[::-1].copy(), hT, hD) == pytest.approx(1.0 - got, abs=1e-12)   # rows swapped: the other class
    assert oracle.cali_theta_m(Wi, np.zeros_like(Wp), hT, hD) == 0.5
    # hand example, d = 1: v = 2 * 3 = 6; l0 = 0, l1 = 0.5 * 6 - 1 * 2 = 1 -> sigmoid(1)
    assert oracle.cali_theta_m(np.array([[2.0]]), np.array([[0.0, 0.0], [0.5, -1.0]]), np.array([3.0]), np.array([2.0])) == \
        pytest.approx(1.0 / (1.0 + np.exp(-1.0)), abs=1e-15)
    # the transform acts on the target's state only: a transposed W^i changes the value
    assert abs(oracle.cali_theta_m(Wi.T.copy(), Wp, hT, hD) - got) > 1e-6


def test_theta_hat_is_the_sample_mean_with_the_initial_value_as_one_observation():
    th, trials, succ = 0.5, 0, 0
    for r, n in ((2, 3), (0, 2), (4, 4), (1, 3)):
        th = oracle.cali_theta_hat(th, trials, r, n)
        trials += n
        succ += r
        assert th == pytest.approx((0.5 + succ) / (1 + trials))
    assert 0.0 <= th <= 1.0
    assert oracle.cali_theta_hat(0.3, 0, 0, 0) == pytest.approx(0.3)        # nothing observed, nothing changes


def test_gaussian_draw_moments_and_stop_probability():
    u = synth.uniforms(11, synth.STREAM_CTRL, 300000).numpy()
    mu, var = 0.6, 0.09
    cur, thetas, chis = 0, [], []
    while cur + 3 <= len(u):
        chi, th, new = oracle.cali_continue(mu, var, u, cur)
        assert new == cur + 3
        cur = new
        thetas.append(th)
        chis.append(chi)
    thetas, chis = np.array(thetas), np.array(chis)
    n = len(thetas)
    assert abs(thetas.mean() - mu) < 4 * np.sqrt(var / n)
    assert abs(thetas.var() - var) < 0.02 * var + 4 * var * np.sqrt(2.0 / n)
    p_cont = np.clip(thetas, 0.0, 1.0).mean()                               # P(u < theta) given theta
    assert abs(chis.mean() - p_cont) < 4 * np.sqrt(0.25 / n)
    assert oracle.cali_continue(mu, var, u[:2], 0)[0] == -1                  # stream exhausted
    assert oracle.cali_continue(5.0, 1e-12, u, 0)[0] == 1 and oracle.cali_continue(-5.0, 1e-12, u, 0)[0] == 0


def test_generation_with_calibration_is_lossless_and_matches_the_loop_rebuilt_from_primitives():
    spec = synth.TINY
    prompt = synth.prompt_tokens(synth.SEED, 20, spec.vocab).numpy()
    u = {k: v.numpy() for k, v in synth.generate_uniforms(160, 20000).items()}
    cw = synth.cali_weights(spec)
    cali = dict(w=cw["w"].float().numpy(), wp=cw["wp"].numpy(), sigma_m=0.2, sigma_s=0.5, theta_hat0=0.5)
    out, trace, _ = oracle_from_spec(spec, 160).generate(prompt, 30, controller=2, uniforms=u, cali=cali)
    ref, _, _ = oracle_from_spec(spec, 160).generate(prompt, 30, fixed_k=1)
    np.testing.assert_array_equal(out, ref)                                  # the controller only moves draft lengths
    assert len({k for k, _, _ in trace}) > 1                                 # and it does move them
    # the same rounds by hand: hidden states from the primitives, decisions from the formulas
    m = oracle_from_spec(spec, 160)
    L, T = spec.n_layers, len(prompt)
    hid, _ = m.target_rows(prompt[:-1], 0, want_hidden=True, want_logits=False)
    hT, theta_hat, trials, cur, ctx = hid[L, -1], 0.5, 0, 0, list(prompt)
    for rnd, (k_ref, a_ref, y_ref) in enumerate(trace[:6]):
        xs, K = [ctx[-1]], 0
        while True:
            lg, hD = m.draft_row(xs[-1], len(ctx) - 1 + K, want_hidden=True)
            xs.append(int(lg.argmax()))
            K += 1
            if K >= 10:
                break
            th_m = oracle.cali_theta_m(cali["w"][min(K, 10) - 1], cali["wp"], hT, hD)
            mu, var = oracle.cali_posterior(th_m, theta_hat, rnd, 0.2, 0.5)
            chi, _, cur = oracle.cali_continue(mu, var, u["u_ctrl"], cur)
            if not chi:
                break
        hid, pl = m.target_rows(np.array(xs, np.int32), len(ctx) - 1, want_hidden=True)
        a = 0
        while a < K and xs[a + 1] == int(pl[a].argmax()):
            a += 1
        y = int(pl[a].argmax())
        assert (K, a, y) == (k_ref, a_ref, y_ref)
        hT = hid[L, a]
        q_v = a + 1
        r, n = q_v - 1, max(min(q_v + 1, K), q_v - 1)
        theta_hat = oracle.cali_theta_hat(theta_hat, trials, r, n)
        trials += n
        ctx += xs[1:1 + a] + [y]
