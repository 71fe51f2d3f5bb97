"""Pins for the oracle's greedy round with tree verification (tree-attention appendix):
whatever candidates are offered, the output is the target model's own greedy sequence."""
import numpy as np
import pytest

import eesd_synth as synth
from tests.helpers import oracle_from_spec
from tests.test_oracle_round import _autoregressive_greedy

SPEC = synth.TINY


@pytest.mark.parametrize("width,k", [(2, 4), (3, 5), (2, 7), (4, 3)])
def test_tree_round_output_equals_vanilla_autoregressive(width, k):
    prompt = synth.prompt_tokens(synth.SEED + width, 24, SPEC.vocab).numpy()
    ref = _autoregressive_greedy(oracle_from_spec(SPEC, 160), prompt, 36)
    out, trace, leaves = oracle_from_spec(SPEC, 160).generate_tree(prompt, 36, width=width, fixed_k=k)
    np.testing.assert_array_equal(out, ref)
    assert all(kk == k and 0 <= a <= kk for kk, a, _ in trace)
    assert sum(a + 1 for _, a, _ in trace) >= 36 > sum(a + 1 for _, a, _ in trace[:-1])
    assert leaves > 0   # the branch that keeps a leaf was taken


def test_tree_of_width_one_is_the_chain_round():
    prompt = synth.prompt_tokens(synth.SEED, 32, SPEC.vocab).numpy()
    sched = [1, 7, 2, 10, 3, 5, 4, 6, 8, 9] * 4
    out_c, trace_c, _ = oracle_from_spec(SPEC, 160).generate(prompt, 30, k_schedule=sched)
    out_t, trace_t, leaves = oracle_from_spec(SPEC, 160).generate_tree(prompt, 30, width=1, k_schedule=sched)
    np.testing.assert_array_equal(out_t, out_c)
    assert trace_t == trace_c and leaves == 0


def test_a_kept_leaf_saves_a_round_against_the_chain():
    # From the same state, a round that keeps a leaf at depth i emits i + 1 tokens where the
    # chain round emits i: rebuild such a round from the primitives.
    prompt = synth.prompt_tokens(synth.SEED + 2, 24, SPEC.vocab).numpy()
    m = oracle_from_spec(SPEC, 160)
    _, trace, leaves = m.generate_tree(prompt, 36, width=2, fixed_k=4)
    ref = _autoregressive_greedy(oracle_from_spec(SPEC, 160), prompt, 40)
    chain = oracle_from_spec(SPEC, 160)
    ctx, found = list(prompt), False
    for (k, a, y) in trace:
        T = len(ctx)
        chain.target_rows(np.array(ctx[:-1], np.int32), 0, want_logits=False)
        xs = [ctx[-1]]
        second = []
        for i in range(k):
            lg = chain.draft_row(xs[i], T - 1 + i)
            order = np.argsort(-lg.astype(np.float64), kind="stable")
            xs.append(int(order[0]))
            second.append(int(order[1]))
        truth = list(ref[T - len(prompt):T - len(prompt) + k + 1])   # the target's own next tokens
        a_chain = 0
        while a_chain < k and xs[1 + a_chain] == truth[a_chain]:
            a_chain += 1
        assert a in (a_chain, a_chain + 1)
        if a == a_chain + 1:   # the leaf at depth a is the target's token there
            assert second[a - 1] == truth[a - 1] and y == truth[a]
            found = True
        else:
            assert y == truth[a]
        ctx += truth[:a] + [y]
    assert found and leaves > 0
