"""The library's own host-side controller (Eq. 3-4 / Algorithm 2; Eq. 6-7 / Algorithm 3), fed
hand-picked uniforms through the C ABI and checked against numbers worked out by hand from the
definitions.  No GPU and no oracle involved: the GPU parity tests compare whole generations with the
oracle, this file makes sure that agreement does not rest on two copies of one misreading."""
import math

import numpy as np
import pytest

from paper_2406_03853_b200 import binding as b


def f32(x):
    return float(np.float32(x))


def test_beta_draw_from_unit_exponentials_hand_values():
    # alpha = beta = 1: theta = X / (X + Y) with X = -ln u_0, Y = -ln u_1.  u_0 = 1/2, u_1 = 1/8 give
    # X = ln 2, Y = 3 ln 2, theta = 1/4 exactly; chi = [u_2 < 1/4].
    chi, theta, cur = b.ts_decide(1, 1, [0.5, 0.125, 0.2])
    assert (chi, cur) == (1, 3) and abs(theta - 0.25) < 1e-15
    chi, theta, cur = b.ts_decide(1, 1, [0.5, 0.125, 0.25])          # strict comparison
    assert chi == 0 and cur == 3
    # alpha = 2, beta = 3, cursor 1: X = -ln(1/2) - ln(1/4) = 3 ln 2, Y = -3 ln(1/2) = 3 ln 2: theta = 1/2
    u = [0.9, 0.5, 0.25, 0.5, 0.5, 0.5, 0.4999, 0.7]
    chi, theta, cur = b.ts_decide(2, 3, u, cursor=1)
    assert (chi, cur) == (1, 7) and abs(theta - 0.5) < 1e-15
    # the order matters: the first alpha uniforms feed X (successes), the next beta feed Y
    chi, theta, _ = b.ts_decide(2, 1, [0.5, 0.5, 0.0625, 0.5])
    assert abs(theta - 2 / 6) < 1e-15 and chi == 0
    chi, theta, _ = b.ts_decide(1, 2, [0.0625, 0.5, 0.5, 0.5])
    assert abs(theta - 4 / 6) < 1e-15 and chi == 1
    # a zero uniform stands for 2^-25
    _, theta, _ = b.ts_decide(1, 1, [0.0, 2.0 ** -25, 0.0])
    assert abs(theta - 0.5) < 1e-15
    # stream too short: refused, nothing consumed
    with pytest.raises(b.EesdError):
        b.ts_decide(2, 2, [0.5, 0.5, 0.5, 0.5])


def test_beta_draw_moments():
    # Beta(3, 2): mean 3/5, variance ab / ((a+b)^2 (a+b+1)) = 6 / 150 = 0.04
    rng = np.random.default_rng(1)
    n, a, bb = 40000, 3, 2
    u = (rng.integers(1, 1 << 24, size=n * (a + bb + 1)) * 2.0 ** -24).astype(np.float32)
    th, chis, cur = [], [], 0
    for _ in range(n):
        chi, t, cur = b.ts_decide(a, bb, u, cur)
        th.append(t)
        chis.append(chi)
    th = np.array(th)
    assert abs(th.mean() - 0.6) < 4 * 0.2 / math.sqrt(n)
    assert abs(th.var() - 0.04) < 0.002
    assert abs(np.mean(chis) - 0.6) < 4 * math.sqrt(0.24 / n)   # marginal stop law: Bernoulli(a / (a + b))


def test_posterior_update_hand_examples():
    # Algorithm 2 as printed: r = |Q_v| - 1, n = min(|Q_v| + 1, |Q_d|); alpha += r, beta += n - r.
    # K = 4 drafted, 1 accepted: |Q_v| = 2, r = 1, n = min(3, 4) = 3 -> alpha + 1, beta + 2
    assert b.ts_posterior_update(1, 1, 2, 4) == (2, 3)
    # K = 4, all accepted: |Q_v| = 5, r = 4, n = min(6, 4) = 4 -> alpha + 4, beta + 0
    assert b.ts_posterior_update(1, 1, 5, 4) == (5, 1)
    # K = 4, three accepted: |Q_v| = 4, r = 3, n = min(5, 4) = 4 -> beta + 1
    assert b.ts_posterior_update(2, 2, 4, 4) == (5, 3)
    # K = 1, none accepted: |Q_v| = 1, r = 0, n = min(2, 1) = 1 -> beta + 1
    assert b.ts_posterior_update(7, 3, 1, 1) == (7, 4)
    # K = 5, none accepted: r = 0, n = min(2, 5) = 2 -> beta + 2 (the printed rule counts two failures)
    assert b.ts_posterior_update(1, 1, 1, 5) == (1, 3)
    # one-failure rule: n = min(|Q_v|, |Q_d|)
    assert b.ts_posterior_update(1, 1, 1, 5, rule=1) == (1, 2)
    assert b.ts_posterior_update(1, 1, 2, 4, rule=1) == (2, 2)
    assert b.ts_posterior_update(1, 1, 5, 4, rule=1) == (5, 1)
    # for every reachable round n >= r, so beta never decreases
    for K in range(1, 16):
        for a in range(0, K + 1):
            for rule in (0, 1):
                al, be = b.ts_posterior_update(10, 10, a + 1, K, rule)
                assert al == 10 + a and be >= 10
    with pytest.raises(b.EesdError):
        b.ts_posterior_update(1, 1, 7, 4)      # more accepted than drafted


def test_calibrated_draw_hand_values():
    # Box-Muller with u_0 = e^-2 (radius sqrt(4) = 2) and u_1 = 0 (angle 0): z = 2 (up to the fp32
    # rounding of u_0), theta = mu + 2 sigma
    u0 = f32(math.exp(-2.0))
    z = math.sqrt(-2.0 * math.log(u0))
    chi, theta, cur = b.cali_decide(0.3, 0.01, [u0, 0.0, 0.49])
    assert cur == 3 and abs(theta - (0.3 + 0.1 * z)) < 1e-15 and abs(z - 2.0) < 1e-6 and chi == 1
    # angle pi (u_1 = 1/2): z = -2, theta = 0.3 - 0.2 = 0.1
    chi, theta, _ = b.cali_decide(0.3, 0.01, [u0, 0.5, 0.11])
    assert abs(theta - (0.3 - 0.1 * z)) < 1e-12 and chi == 0
    # theta outside [0, 1] acts as 0 / 1
    assert b.cali_decide(-5.0, 0.0, [0.3, 0.3, 0.0])[0] == 0
    assert b.cali_decide(5.0, 0.0, [0.3, 0.3, 0.999])[0] == 1


def test_calibrated_posterior_limits():
    # Eq. 6-7: n = 0 returns the model's prediction with its variance sigma_M^2; many verifications
    # tend to the observed mean with variance sigma_S^2 / n
    mu, var = b.cali_posterior(0.7, 0.2, 0, 0.3, 0.5)
    assert abs(mu - 0.7) < 1e-15 and abs(var - 0.09) < 1e-15
    mu, var = b.cali_posterior(0.7, 0.2, 10 ** 6, 0.3, 0.5)
    assert abs(mu - 0.2) < 1e-5 and abs(var - 0.25 / 10 ** 6) < 1e-10
    # sigma_M = sigma_S, n = 1: the two sources weigh the same
    mu, var = b.cali_posterior(0.8, 0.4, 1, 0.2, 0.2)
    assert abs(mu - 0.6) < 1e-15 and abs(var - 0.02) < 1e-15
