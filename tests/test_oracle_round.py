"""Pins for the oracle's generation loop (Algorithm 1) and Thompson-sampling controller
(Eq. 3-4, Algorithm 2)."""
import numpy as np
import pytest

import eesd_synth as synth
import oracle
from tests.helpers import oracle_from_spec


def _autoregressive_greedy(model, prompt, n_new):
    """Vanilla decoding by full-prefix recompute: no draft model, no acceptance, no reuse."""
    ctx = list(prompt)
    for _ in range(n_new):
        _, lg = model.target_rows(np.array(ctx, np.int32), 0)
        ctx.append(int(lg[-1].argmax()))
    return np.array(ctx[len(prompt):], np.int32)


def test_greedy_eesd_equals_vanilla_autoregressive_for_any_k_schedule():
    # The verification pass makes the output identical to the target model's own greedy
    # decoding (abstract; case study appendix), whatever the draft lengths are.
    spec = synth.TINY
    prompt = synth.prompt_tokens(synth.SEED, 32, spec.vocab).numpy()
    ref = _autoregressive_greedy(oracle_from_spec(spec, 160), prompt, 40)
    u = {k: v.numpy() for k, v in synth.generate_uniforms(160, 100000).items()}
    runs = [dict(fixed_k=4), dict(fixed_k=1), dict(fixed_k=10),
            dict(k_schedule=[1, 7, 2, 10, 3, 5, 4, 6, 8, 9] * 5),
            dict(controller=1, uniforms=u), dict(controller=1, uniforms=u, ts_rule=1, alpha0=3, beta0=1)]
    accepted = 0
    for kw in runs:
        out, trace, _ = oracle_from_spec(spec, 160).generate(prompt, 40, **kw)
        np.testing.assert_array_equal(out, ref)
        assert sum(a + 1 for _, a, _ in trace) >= 40 > sum(a + 1 for _, a, _ in trace[:-1])
        assert all(1 <= k <= 10 and 0 <= a <= k for k, a, _ in trace)
        accepted += sum(a for _, a, _ in trace)
    assert accepted > 50  # the damped synthetic model really does accept drafts


def test_round_trace_is_consistent_with_draft_and_verify_primitives():
    # rebuild the first round by hand from draft_row / target_rows / accept_resample
    spec = synth.TINY
    prompt = synth.prompt_tokens(synth.SEED, 32, spec.vocab).numpy()
    u = {k: v.numpy() for k, v in synth.generate_uniforms(160, 1000).items()}
    out, trace, _ = oracle_from_spec(spec, 160).generate(prompt, 12, fixed_k=4, temperature=1.0, uniforms=u)
    m = oracle_from_spec(spec, 160)
    T = len(prompt)
    m.target_rows(prompt[:-1], 0, want_logits=False)
    xs, ql = [int(prompt[-1])], []
    for i in range(4):
        lg = m.draft_row(xs[-1], T - 1 + i)
        ql.append(lg)
        xs.append(oracle.sample_logits(lg, 1.0, float(u["u_draft"][T + i])))
    _, pl = m.target_rows(np.array(xs, np.int32), T - 1)
    n_acc, y = oracle.accept_resample(pl, np.stack(ql), xs[1:], u["u_accept"][T:T + 4], float(u["u_resample"][T]), 1.0)
    assert trace[0] == (4, n_acc, y)
    np.testing.assert_array_equal(out[:n_acc + 1], xs[1:1 + n_acc] + [y])


def test_stochastic_generation_first_token_follows_target_distribution():
    # lossless in distribution: over many uniform streams the first generated token follows
    # softmax(target logits of the prompt), although it is produced by draft + accept/resample
    from scipy import stats
    from tests.helpers import np_softmax
    spec = synth.TINY.with_(vocab=16, n_layers=2)
    prompt = np.array([3, 7, 1, 12], np.int32)
    m = oracle_from_spec(spec, 32)
    _, lg = m.target_rows(prompt, 0)
    P = np_softmax(lg[-1].astype(np.float64) * 60.0)
    # logits of a 0.02-scaled random model are nearly flat; a low temperature (1/60) sharpens p
    n, counts = 4000, np.zeros(16)
    for i in range(n):
        u = {k: v.numpy() for k, v in synth.generate_uniforms(32, 64, seed=1000 + i).items()}
        out, _, _ = m.generate(prompt, 1, fixed_k=2, temperature=1.0 / 60.0, uniforms=u)
        counts[out[0]] += 1
    keep = P * n >= 5
    o, e = np.append(counts[keep], counts[~keep].sum()), np.append(P[keep], P[~keep].sum()) * n
    if e[-1] == 0:
        o, e = o[:-1], e[:-1]
    assert stats.chisquare(o, e * o.sum() / e.sum()).pvalue > 1e-3


# ---------------------------------------------------------------- controller
def test_posterior_update_hand_examples():
    # r = |Q_v| - 1, n = min(|Q_v| + 1, |Q_d|)  (Algorithm 2, update steps), with |Q_v| = accepted + 1
    # K = 4 drafted, 1 accepted: |Q_v| = 2, r = 1, n = min(3, 4) = 3 -> alpha += 1, beta += 2
    assert oracle.ts_update(1, 1, 2, 4, 0) == (2, 3)
    # K = 4, all accepted: |Q_v| = 5, r = 4, n = min(6, 4) = 4 -> alpha += 4, beta += 0
    assert oracle.ts_update(1, 1, 5, 4, 0) == (5, 1)
    # K = 4, 3 accepted: |Q_v| = 4, r = 3, n = min(5, 4) = 4 -> beta += 1
    assert oracle.ts_update(2, 2, 4, 4, 0) == (5, 3)
    # K = 1, rejected: |Q_v| = 1, r = 0, n = min(2, 1) = 1 -> beta += 1
    assert oracle.ts_update(1, 1, 1, 1, 0) == (1, 2)
    # alternative rule: n = min(|Q_v|, |Q_d|): one failure at most
    assert oracle.ts_update(1, 1, 2, 4, 1) == (2, 2)
    assert oracle.ts_update(1, 1, 5, 4, 1) == (5, 1)


def test_beta_draw_moments_and_stop_probability():
    # theta ~ Beta(a, b): mean a/(a+b), variance ab/((a+b)^2 (a+b+1)); chi ~ Bernoulli(theta)
    # so P(chi = 1) = a/(a+b)
    u = synth.uniforms(77, synth.STREAM_CTRL, 400000).numpy()
    for a, b in ((1, 1), (3, 2), (2, 7)):
        cur, th, chis = 0, [], []
        while cur + a + b + 1 <= len(u) and len(th) < 30000:
            chi, t, cur = oracle.ts_continue(a, b, u, cur)
            th.append(t)
            chis.append(chi)
        th, chis = np.array(th), np.array(chis)
        mean, var = a / (a + b), a * b / ((a + b) ** 2 * (a + b + 1))
        assert abs(th.mean() - mean) < 5 * np.sqrt(var / len(th))
        assert abs(th.var() - var) < 0.05 * var + 1e-4
        assert abs(chis.mean() - mean) < 5 * np.sqrt(mean * (1 - mean) / len(chis))
    assert oracle.ts_continue(5, 5, u[:10], 0)[0] == -1  # stream exhausted is reported, not read past


def test_controller_posterior_in_generation_matches_trace():
    spec = synth.TINY
    prompt = synth.prompt_tokens(synth.SEED, 32, spec.vocab).numpy()
    u = {k: v.numpy() for k, v in synth.generate_uniforms(160, 100000).items()}
    _, trace, (a, b) = oracle_from_spec(spec, 160).generate(prompt, 48, controller=1, uniforms=u)
    aa, bb = 1, 1
    for k, n_acc, _ in trace:
        aa, bb = oracle.ts_update(aa, bb, n_acc + 1, k, 0)
    assert (a, b) == (aa, bb)
    assert len({k for k, _, _ in trace}) > 1  # the controller really varies the draft length


# ---------------------------------------------------------------- several early-exit layers
def test_one_exit_layer_given_as_a_list_is_the_same_model_bit_for_bit():
    spec = synth.TINY
    prompt = synth.prompt_tokens(synth.SEED + 3, 20, spec.vocab).numpy()
    a, b = oracle_from_spec(spec, 96), oracle_from_spec(spec, 96, n_exit=1)
    out_a, tr_a, _ = a.generate(prompt, 24, fixed_k=4)
    out_b, tr_b, _ = b.generate(prompt, 24, fixed_k=4)
    np.testing.assert_array_equal(out_a, out_b)
    assert tr_a == tr_b
    np.testing.assert_array_equal(a.draft_row(5, 60), b.draft_row(5, 60))


@pytest.mark.parametrize("n_exit", [2, 3])
def test_draft_row_with_several_exit_layers_is_the_stack_of_layers_on_the_early_hidden_state(n_exit):
    # Eq. 1 with a stack of exit layers: p = softmax(W^T RMSNorm(T^e_E(...T^e_1(H^N)))).  The cached
    # draft row after a target pass over the prefix must equal the stack composed from the layer
    # primitive on the WHOLE prefix (which also checks that the target pass left every exit layer's
    # keys / values for the prefix: exit layer e sees the output of exit layer e - 1 there).
    spec = synth.TINY
    toks = synth.prompt_tokens(5, 9, spec.vocab).numpy()
    m = oracle_from_spec(spec, 64, n_exit=n_exit)
    m.target_rows(toks[:-1], 0, want_logits=False)
    lg, hid = m.draft_row(toks[-1], 8, want_hidden=True)
    m2 = oracle_from_spec(spec, 64, n_exit=n_exit)
    x = m2.embed(toks)
    for l in range(spec.n_early):
        x = m2.layer_fwd(l, l, x, 0)
    for e in range(n_exit):
        x = m2.layer_fwd(spec.n_layers + e, spec.n_layers + e, x, 0)
    np.testing.assert_allclose(hid, x[-1], atol=1e-12)
    np.testing.assert_allclose(lg, m2.head(x[-1:], exit_head=True)[0], atol=1e-6)
    # the exit layers are copies of the last target layers, in order; and a second exit layer changes the draft
    for e in range(n_exit):
        a, b = synth.exit_layer_weights(spec, index=e, count=n_exit), synth.layer_weights(spec, spec.n_layers - n_exit + e)
        assert all((a[k] == b[k]).all() for k in a)
    m1 = oracle_from_spec(spec, 64)
    m1.target_rows(toks[:-1], 0, want_logits=False)
    assert np.abs(m1.draft_row(toks[-1], 8) - lg).max() > 1e-4
    # the target's own output does not depend on how many exit layers hang off layer N
    _, t1 = m1.target_rows(toks, 0)
    _, t2 = oracle_from_spec(spec, 64, n_exit=n_exit).target_rows(toks, 0)
    np.testing.assert_array_equal(t1, t2)


def test_greedy_eesd_with_two_exit_layers_still_equals_vanilla_autoregressive():
    spec = synth.TINY
    prompt = synth.prompt_tokens(synth.SEED, 32, spec.vocab).numpy()
    ref = _autoregressive_greedy(oracle_from_spec(spec, 160), prompt, 32)
    for kw in (dict(fixed_k=4), dict(k_schedule=[1, 7, 2, 10, 3, 5] * 6)):
        out, trace, _ = oracle_from_spec(spec, 160, n_exit=2).generate(prompt, 32, **kw)
        np.testing.assert_array_equal(out, ref)
    assert sum(a for _, a, _ in trace) > 5
