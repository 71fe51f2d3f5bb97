"""Pins for the oracle's lossless acceptance / resampling arithmetic.

The rule (accept with probability min(1, p/q); on rejection resample from
normalize(max(0, p - q)); on full acceptance sample a bonus token from p) is the standard
lossless speculative-sampling rule the paper relies on for its "identical distribution"
claim.  These tests check it against closed forms and exact integer brute force.
"""
import math
from fractions import Fraction

import numpy as np
import pytest
from scipy import stats

import eesd_synth as synth
import oracle
from tests.helpers import np_softmax


def test_exp_spec_tracks_exp_to_a_few_ulp_and_flushes():
    ts = -np.concatenate([np.linspace(0, 64, 20001), np.geomspace(1e-8, 64, 3000)])
    got = np.array([oracle.exp_spec(t) for t in ts], np.float64)
    ref = np.exp(ts.astype(np.float32).astype(np.float64))
    assert np.max(np.abs(got - ref) / ref) < 4 * 2.0 ** -24
    assert oracle.exp_spec(0.0) == 1.0
    assert oracle.exp_spec(-64.5) == 0.0 and oracle.exp_spec(-1e30) == 0.0
    assert oracle.exp_spec(-64.0) > 0.0


def test_softmax_spec_matches_fp64_softmax_and_sums_to_one():
    lg = synth.normal_f32(5, 9, 32000).numpy() * 3.0
    for T in (1.0, 0.7, 2.0):
        p = oracle.softmax_spec(lg, T).astype(np.float64)
        ref = np_softmax(lg.astype(np.float64) / T)
        assert abs(p.sum() - 1.0) < 1e-5
        big = ref > 1e-9
        assert np.max(np.abs(p[big] - ref[big]) / ref[big]) < 2e-6
    # shift invariance is exact when the shift itself is (logits on a 2^-10 grid): only logit - max enters
    lq = (np.round(lg * 1024) / 1024).astype(np.float32)
    np.testing.assert_array_equal(oracle.softmax_spec(lq, 1.0), oracle.softmax_spec(lq + np.float32(8.0), 1.0))


def _brute_sample(w, m_u):
    """Exact integer restatement: floors of w * 2^32, target floor(m_u * W / 2^24)."""
    fl = [int(Fraction(float(x)) * 2**32) for x in w]
    W = sum(fl)
    tau = (m_u * W) >> 24
    acc = 0
    for v, f in enumerate(fl):
        acc += f
        if acc > tau:
            return v
    raise AssertionError


def test_inverse_cdf_brute_force_and_exact_distribution():
    rng = np.random.default_rng(1)
    for V in (1, 2, 5, 16):
        w = rng.random(V).astype(np.float32)
        w[rng.integers(V)] = 0.0 if V > 1 else w[0]
        w /= max(w.sum(), 1e-9)
        for m_u in list(rng.integers(0, 2**24, 200)) + [0, 2**24 - 1]:
            assert oracle.sample_weights(w, m_u * 2.0 ** -24) == _brute_sample(w, int(m_u))
    # dyadic weights: the number of m_u values mapping to v is exactly w_v * 2^24
    w = np.array([0.5, 0.25, 0.0, 0.125, 0.125], np.float32)
    grid = np.arange(0, 2**24, 2**12)  # every 4096-th value: counts are exact multiples
    got = np.bincount([oracle.sample_weights(w, m * 2.0 ** -24) for m in grid], minlength=5)
    np.testing.assert_array_equal(got, (w * len(grid)).astype(int))
    assert oracle.sample_weights(np.zeros(4, np.float32), 0.3) == -1


def test_q_equal_p_accepts_every_draft_token():
    # with q == p, min(1, p/q) = 1: no uniform in [0,1) may reject
    for case in range(4):
        p, _, u_acc, u_res, u_dr = synth.accept_case(case, 1, 8, 4096, 3.0, 0.0)
        p, u_acc = p[0].numpy(), u_acc[0].numpy()
        q = p[:8].copy()
        x = [oracle.sample_logits(q[i], 1.0, float(u_dr[0, i])) for i in range(8)]
        for ua in (u_acc, np.full(8, 1 - 2.0 ** -24, np.float32), np.zeros(8, np.float32)):
            n, y = oracle.accept_resample(p, q, x, ua, float(u_res[0]), 1.0)
            assert n == 8
            assert y == oracle.sample_logits(p[8], 1.0, float(u_res[0]))  # bonus token from p_{K+1}


def test_acceptance_rate_equals_sum_min_p_q():
    # P(accept) for x ~ q is sum_v q_v min(1, p_v/q_v) = sum_v min(p_v, q_v)
    V, n = 64, 120000
    lp = (synth.normal_f32(21, 1, V).numpy() * 1.5).astype(np.float32)
    lq = (lp + synth.normal_f32(21, 2, V).numpy() * 1.0).astype(np.float32)
    P, Q = np_softmax(lp), np_softmax(lq)
    expect = np.minimum(P, Q).sum()
    ud = synth.uniforms(21, 3, n).numpy()
    ua = synth.uniforms(21, 4, n).numpy()
    ur = synth.uniforms(21, 5, n).numpy()
    p_l = np.broadcast_to(np.stack([lp, lp]), (n, 2, V)).copy()
    q_l = np.broadcast_to(lq[None, None], (n, 1, V)).copy()
    xs = np.array([oracle.sample_logits(lq, 1.0, float(u)) for u in ud], np.int32)  # x ~ q
    n_acc, y = oracle.accept_resample_batch(p_l, q_l, xs.reshape(n, 1), ua.reshape(n, 1), ur, 1.0)
    rate = n_acc.mean()
    sd = math.sqrt(expect * (1 - expect) / n)
    assert abs(rate - expect) < 4 * sd, (rate, expect)
    # lossless: the first emitted token (accepted draft or correction) is distributed as p
    first = np.where(n_acc == 1, xs, y)
    obs = np.bincount(first, minlength=V)
    assert (P * n >= 5).all()
    assert stats.chisquare(obs, P * n).pvalue > 1e-3


def test_chi_square_emitted_tokens_follow_target_on_16_token_vocab():
    # the distribution of every emitted position is p, whatever q is: K = 2, V = 16
    V, K, n = 16, 2, 200000
    lp = (synth.normal_f32(33, 1, (K + 1) * V).numpy() * 1.2).reshape(K + 1, V).astype(np.float32)
    lq = (lp[:K] + synth.normal_f32(33, 2, K * V).numpy().reshape(K, V) * 1.5).astype(np.float32)
    ud = synth.uniforms(33, 3, n * K).numpy().reshape(n, K)
    ua = synth.uniforms(33, 4, n * K).numpy().reshape(n, K)
    ur = synth.uniforms(33, 5, n).numpy()
    # tokens drawn from q by the oracle's sampler (rows are context-free here, so q_i is fixed)
    table = [np.array([oracle.sample_logits(lq[i], 1.0, m * 2.0 ** -24) for m in range(0, 2**24, 2**10)])
             for i in range(K)]
    xs = np.stack([table[i][(ud[:, i] * 2**14).astype(np.int64)] for i in range(K)], 1).astype(np.int32)
    p_l = np.broadcast_to(lp[None], (n, K + 1, V)).copy()
    q_l = np.broadcast_to(lq[None], (n, K, V)).copy()
    n_acc, y = oracle.accept_resample_batch(p_l, q_l, xs, ua, ur, 1.0)
    P = np_softmax(lp)
    # position 1: accepted x_1 or the correction
    first = np.where(n_acc >= 1, xs[:, 0], y)
    assert stats.chisquare(np.bincount(first, minlength=V), P[0] * n).pvalue > 1e-3
    # position 2, given x_1 accepted: accepted x_2 or the correction drawn for row 2
    sel = n_acc >= 1
    second = np.where(n_acc[sel] >= 2, xs[sel, 1], y[sel])
    assert stats.chisquare(np.bincount(second, minlength=V), P[1] * sel.sum()).pvalue > 1e-3
    # bonus token after full acceptance follows p_{K+1}
    sel = n_acc == K
    assert sel.sum() > 2000
    assert stats.chisquare(np.bincount(y[sel], minlength=V), P[2] * sel.sum()).pvalue > 1e-3


def test_residual_distribution_is_normalized_positive_part():
    # force a rejection (u_acc just below 1 and p(x) < q(x)); y must follow max(0,p-q)/sum
    V, n = 16, 100000
    lp = (synth.normal_f32(44, 1, 2 * V).numpy()).reshape(2, V).astype(np.float32)
    lq = (lp[:1] + synth.normal_f32(44, 2, V).numpy().reshape(1, V) * 2.0).astype(np.float32)
    P, Q = np_softmax(lp[0]), np_softmax(lq[0])
    x = int(np.argmax(Q - P))
    ur = synth.uniforms(44, 5, n).numpy()
    p_l = np.broadcast_to(lp[None], (n, 2, V)).copy()
    q_l = np.broadcast_to(lq[None], (n, 1, V)).copy()
    n_acc, y = oracle.accept_resample_batch(p_l, q_l, np.full((n, 1), x, np.int32),
                                            np.full((n, 1), 1 - 2.0 ** -24, np.float32), ur, 1.0)
    assert (n_acc == 0).all()
    res = np.maximum(P - Q, 0)
    res /= res.sum()
    obs = np.bincount(y, minlength=V)
    assert (obs[res == 0] == 0).all()
    keep = res > 0
    assert stats.chisquare(obs[keep], res[keep] * n).pvalue > 1e-3


def test_accept_threshold_is_p_over_q():
    # deterministic boundary: with u just below / above p(x)/q(x) the decision flips
    V = 8
    lp = np.array([[0, 1, 2, 0, 0, 0, 0, 0], [0] * 8], np.float32)
    lq = np.array([[2, 1, 0, 0, 0, 0, 0, 0]], np.float32)
    P, Q = oracle.softmax_spec(lp[0]).astype(np.float64), oracle.softmax_spec(lq[0]).astype(np.float64)
    ratio = P[0] / Q[0]  # token 0: p < q
    lo = math.floor(ratio * 2**24 - 2) * 2.0 ** -24
    hi = math.ceil(ratio * 2**24 + 2) * 2.0 ** -24
    assert oracle.accept_resample(lp, lq, [0], [lo], 0.5, 1.0)[0] == 1
    assert oracle.accept_resample(lp, lq, [0], [hi], 0.5, 1.0)[0] == 0
    # token 2: p > q, accepted for any u
    assert oracle.accept_resample(lp, lq, [2], [1 - 2.0 ** -24], 0.5, 1.0)[0] == 1


def test_greedy_rule_keeps_prefix_equal_to_target_top1():
    V, K = 32, 5
    lp = synth.normal_f32(55, 1, (K + 1) * V).numpy().reshape(K + 1, V)
    top = lp.argmax(1)
    lq = np.zeros((K, V), np.float32)
    x = top[:K].copy()
    assert oracle.accept_resample(lp, lq, x, np.zeros(K), 0.0, 0.0) == (K, int(top[K]))
    x[3] = (x[3] + 1) % V
    assert oracle.accept_resample(lp, lq, x, np.zeros(K), 0.0, 0.0) == (3, int(top[3]))
    x[0] = (x[0] + 1) % V
    assert oracle.accept_resample(lp, lq, x, np.zeros(K), 0.0, 0.0) == (0, int(top[0]))
    # ties go to the lowest index
    t = np.zeros(V, np.float32)
    t[[4, 9]] = 1.0
    assert oracle.sample_logits(t, 0.0, 0.0) == 4
