"""Full-size properties on the LLaMA-2-13B-shaped model (all 40 layers, the launch
configuration the benchmark times), where the CPU oracle cannot follow in seconds:

* losslessness: greedy EESD emits the target model's own greedy sequence, so the tokens must
  not depend on the draft lengths (K = 1, 4, 10 and a Thompson-sampling run);
* sampled outputs against the oracle: the embedding row and the first decoder layer of a
  verify pass, checked on the rows the oracle computes from the same weights.
"""
import numpy as np
import pytest
import torch

import eesd_synth as synth
import oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def engine13b():
    import bench
    from paper_2406_03853_b200 import binding as b
    eng, spec, _, _ = bench.build_engine("13b-eesd", 0.0, b.CTRL_FIXED_K, torch.device("cuda:0"))
    yield eng, spec
    eng.close()


def test_greedy_tokens_do_not_depend_on_draft_length(engine13b):
    eng, spec = engine13b
    prompt = synth.prompt_tokens(synth.SEED, 200, spec.vocab).numpy()
    outs, accepted = [], []
    for ks in ([1] * 64, [4] * 64, [10] * 64, [3, 7, 1, 10, 2, 5] * 12):
        out, trace, st = eng.generate(prompt, 40, k_schedule=ks)
        outs.append(out)
        accepted.append(st.accepted)
        assert st.emitted == 40 and all(0 <= a <= k for k, a, _ in trace)
    for o in outs[1:]:
        np.testing.assert_array_equal(o, outs[0])
    assert max(accepted) > 0   # drafts are really accepted somewhere, so the equality is not vacuous


def test_first_layer_of_a_full_size_pass_matches_oracle(engine13b):
    eng, spec = engine13b
    from tests.helpers import oracle_from_spec
    m = oracle_from_spec(spec, max_ctx=64, n_layers=1, device="cuda")
    prompt = synth.prompt_tokens(11, 9, spec.vocab).numpy()
    m.target_rows(prompt[:-1], 0, want_logits=False)
    eng.prefill(prompt)
    cap = eng.capture_hidden(True)
    rows = np.concatenate([prompt[-1:], synth.prompt_tokens(12, 5, spec.vocab).numpy()]).astype(np.int32)
    eng.verify_only(rows)
    torch.cuda.synchronize()
    hid, _ = m.target_rows(rows, len(prompt) - 1, want_hidden=True, want_logits=False)
    got = cap[:2, :len(rows)].cpu().numpy()
    assert np.abs(got[0] - hid[0]).max() == 0.0          # embedding rows: exact
    assert np.abs(got[1] - hid[1]).max() < 2e-2          # after layer 1, bf16 tolerance
    eng.capture_hidden(False)
    # the pass left finite logits of the right shape behind
    lg = eng.logits(0, len(rows))
    assert torch.isfinite(lg).all() and lg.shape == (len(rows), spec.vocab)


def test_stochastic_rounds_at_13b_layer_shapes_follow_the_rule_on_the_gpus_own_logits():
    """Temperature 1 on bf16 weights: token streams may leave the fp64 oracle's after a draw near
    a boundary, so the stochastic path is checked on what stays exact and on statistics.  Every
    round, the q logits the draft steps left and the p logits the verify pass left are read
    back; the oracle's sampler must choose the same draft tokens from those q logits, the
    oracle's accept / resample rule must take the same decision on those (p, q, uniforms),
    bit for bit; and over all rounds the first draft token is accepted as often as the closed
    form sum_v min(p(v), q(v)) says (4 sigma)."""
    import bench
    from paper_2406_03853_b200 import binding as b
    eng, spec, _, _ = bench.build_engine("13b-eesd", 1.0, b.CTRL_FIXED_K, torch.device("cuda:0"), n_layers=8)
    prompt = synth.prompt_tokens(21, 40, spec.vocab).numpy()
    eng.prefill(prompt)
    K, rounds = 3, 60
    expect, var, hits = 0.0, 0.0, 0
    for r in range(rounds):
        ud = synth.uniforms(500 + r, 1, K).numpy()
        ua = synth.uniforms(500 + r, 2, K).numpy()
        ur = float(synth.uniforms(500 + r, 3, 1).numpy()[0])
        toks = eng.draft(K, ud)
        torch.cuda.synchronize()
        ql = eng.logits(1, K).clone()
        for i in range(K):
            assert oracle.sample_logits(ql[i].cpu().numpy(), 1.0, float(ud[i])) == toks[i]
        n_acc, y = eng.verify_accept(ua, ur)
        pl = eng.logits(0, K + 1).clone()
        assert (n_acc, y) == oracle.accept_resample(pl.cpu().numpy(), ql.cpu().numpy(), toks, ua, ur, 1.0)
        a1 = torch.minimum(torch.softmax(pl[0].double(), 0), torch.softmax(ql[0].double(), 0)).sum().item()
        expect += a1
        var += a1 * (1.0 - a1)
        hits += int(n_acc >= 1)
    assert abs(hits - expect) < 4.0 * np.sqrt(var) + 1.0, (hits, expect, var)
    assert 0.05 * rounds < expect < 0.999 * rounds          # neither a degenerate draft nor a copy of the target
    eng.close()


def test_tree_verification_at_full_size_emits_the_same_greedy_tokens(engine13b):
    """Losslessness of tree verification at the benchmark's size: whatever candidates a pass
    holds, the output is the target's own greedy sequence, so a tree run (two and three
    candidates per position, 7 to 16 rows per pass) must emit the chain run's tokens; and it
    must keep leaves, or the equality would say nothing."""
    import bench
    from paper_2406_03853_b200 import binding as b
    eng, spec = engine13b
    prompt = synth.prompt_tokens(synth.SEED, 200, spec.vocab).numpy()
    ref, _, st_chain = eng.generate(prompt, 40, k_schedule=[3] * 64)
    for width, ks in ((2, [3] * 64), (3, [5, 1, 4, 2, 3] * 13)):
        eng_t, _, _, _ = bench.build_engine("13b-eesd", 0.0, b.CTRL_FIXED_K, torch.device("cuda:0"), tree_width=width)
        out, trace, st = eng_t.generate(prompt, 40, k_schedule=ks)
        eng_t.close()
        del eng_t
        torch.cuda.empty_cache()
        np.testing.assert_array_equal(out, ref)
        assert st.leaves_kept > 0 and all(0 <= a <= k for k, a, _ in trace)
        if width == 2:
            assert st.rounds <= st_chain.rounds   # same draft length, more candidates: never more rounds here
