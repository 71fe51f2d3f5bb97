"""GPU parity of tree verification (several draft candidates per position, tree-attention
appendix) against the oracle's round: tokens, traces and kept leaves on the fp32 tiny model;
on bf16 models every row of the tree pass against the target run on that row's own path, the
walk against the engine's own logits, and the cache after a kept leaf."""
import numpy as np
import pytest
import torch

import eesd_synth as synth
from tests.helpers import engine_from_spec, oracle_from_spec

pytestmark = pytest.mark.gpu
TOL = 2e-2


@pytest.mark.parametrize("width,k", [(2, 4), (3, 5), (2, 7), (4, 3), (2, 1)])
def test_tree_generation_matches_oracle_token_for_token(width, k):
    spec = synth.TINY
    prompt = synth.prompt_tokens(synth.SEED + width, 24, spec.vocab).numpy()
    ref, rtrace, rleaves = oracle_from_spec(spec, 160).generate_tree(prompt, 36, width=width, fixed_k=k)
    eng = engine_from_spec(spec, max_ctx=160, fixed_k=k, k_cap=k, tree_width=width)
    out, trace, st = eng.generate(prompt, 36)
    np.testing.assert_array_equal(out, ref)
    assert trace == rtrace
    assert st.leaves_kept == rleaves and (rleaves > 0 or k == 1)
    eng.close()


def test_tree_generation_with_a_draft_length_schedule_and_small_pages():
    spec = synth.TINY
    prompt = synth.prompt_tokens(synth.SEED + 9, 31, spec.vocab).numpy()
    sched = [1, 5, 2, 4, 3] * 8
    ref, rtrace, rleaves = oracle_from_spec(spec, 160).generate_tree(prompt, 40, width=3, k_schedule=sched)
    eng = engine_from_spec(spec, max_ctx=160, k_cap=5, tree_width=3, page_tokens=8)
    out, trace, st = eng.generate(prompt, 40, k_schedule=sched)
    np.testing.assert_array_equal(out, ref)
    assert trace == rtrace and st.leaves_kept == rleaves
    eng.close()


def test_tree_configurations_that_are_refused():
    from paper_2406_03853_b200 import EesdError
    spec = synth.TINY
    for kw in (dict(tree_width=2, k_cap=8), dict(tree_width=2, k_cap=4, temperature=1.0), dict(tree_width=5, k_cap=2)):
        with pytest.raises(EesdError):
            engine_from_spec(spec, max_ctx=64, **kw)


def _rounds_through_the_step_api(spec, n_layers, width, k, n_prompt, n_rounds, max_ctx=128, seed=3):
    """Every round: draft k steps, read the engine's own draft logits to know the leaves, verify,
    compare each row of the pass with the oracle's target run on that row's path, redo the walk on
    the engine's own top-1 tokens, and check the context the engine reports."""
    eng = engine_from_spec(spec, n_layers=n_layers, max_ctx=max_ctx, k_cap=k, tree_width=width)
    prompt = synth.prompt_tokens(seed, n_prompt, spec.vocab).numpy()
    eng.prefill(prompt)
    ctx = [int(t) for t in prompt]
    kept = 0
    worst = 0.0
    m = oracle_from_spec(spec, max_ctx=max_ctx, n_layers=n_layers, device="cuda")
    for _ in range(n_rounds):
        T = len(ctx)
        if T > 1:   # the oracle's cache is indexed by position: feeding the whole context again resets it
            m.target_rows(np.array(ctx[:-1], np.int32), 0, want_logits=False)
        chain = [ctx[-1]] + [int(t) for t in eng.draft(k)]
        ql = eng.logits(1, k).cpu().numpy()
        for i in range(k):   # the cache the draft model sees is intact: its logits match the oracle's draft model
            worst = max(worst, float(np.abs(ql[i] - m.draft_row(chain[i], T - 1 + i)).max()))
        order = [np.argsort(-ql[i].astype(np.float64), kind="stable")[:width] for i in range(k)]
        assert [int(o[0]) for o in order] == chain[1:]
        leaves = [[int(v) for v in o[1:]] for o in order]
        a, y = eng.verify_accept()
        M = 1 + k * width
        pl = eng.logits(0, M).cpu().numpy()
        _, ref_chain = m.target_rows(np.array(chain, np.int32), T - 1)
        worst = max(worst, float(np.abs(pl[:k + 1] - ref_chain).max()))
        for i in range(1, k + 1):
            for j, tok in enumerate(leaves[i - 1]):
                m.target_rows(np.array(chain[:i], np.int32), T - 1, want_logits=False)   # the path before the leaf
                _, ref_leaf = m.target_rows(np.array([tok], np.int32), T - 1 + i)
                row = k + 1 + (i - 1) * (width - 1) + j
                worst = max(worst, float(np.abs(pl[row] - ref_leaf[0]).max()))
        top = pl.argmax(axis=1)
        acc, nxt = chain[1:], int(top[k])
        for i in range(1, k + 1):
            want = int(top[i - 1])
            if want == chain[i]:
                continue
            if want in leaves[i - 1]:
                row = k + 1 + (i - 1) * (width - 1) + leaves[i - 1].index(want)
                acc, nxt = chain[1:i] + [want], int(top[row])
                kept += 1
            else:
                acc, nxt = chain[1:i], want
            break
        assert (a, y) == (len(acc), nxt)
        ctx += acc + [nxt]
        np.testing.assert_array_equal(eng.context_tokens(), np.array(ctx, np.int32))
        assert eng.context_len()[1] == (len(ctx) - 1 + spec_page(eng) - 1) // spec_page(eng)
    eng.close()
    return worst, kept


def spec_page(eng):
    return eng.cfg.page_tokens


def test_tree_pass_rows_and_cache_bf16_tensor_core_path():
    spec = synth.TINY.with_(dtype="bf16", ffn_dim=640)
    worst, kept = _rounds_through_the_step_api(spec, None, width=3, k=5, n_prompt=37, n_rounds=8)
    print(f"tree pass, bf16 tiny: worst logit distance {worst:.3e}, leaves kept {kept}")
    assert worst < TOL and kept > 0


def test_tree_pass_rows_gqa_wide_heads():
    spec = synth.TINY.with_(dtype="bf16", ffn_dim=640, n_heads=8, n_kv_heads=2, head_dim=128, d_model=256)
    worst, kept = _rounds_through_the_step_api(spec, None, width=2, k=7, n_prompt=20, n_rounds=5)
    print(f"tree pass, GQA 8/2 x 128: worst logit distance {worst:.3e}, leaves kept {kept}")
    assert worst < TOL


def test_tree_pass_rows_fp32_long_context():
    # context past several attention slices
    spec = synth.TINY
    eng_kw = dict(width=4, k=3, n_prompt=230, n_rounds=4, max_ctx=320)
    worst, kept = _rounds_through_the_step_api(spec, None, **eng_kw)
    assert worst < 1e-3


def test_tree_pass_13b_layer_shape():
    spec = synth.LLAMA2_13B
    worst, kept = _rounds_through_the_step_api(spec, 2, width=3, k=5, n_prompt=21, n_rounds=2, max_ctx=96)
    print(f"tree pass, 13B layer shape (2 layers): worst logit distance {worst:.3e}")
    assert worst < TOL


def test_tree_pass_13b_layer_shape_1024_token_cache():
    # the cache length the benchmark times: a 7-row tree pass (width 2, three draft steps) over every attention slice
    spec = synth.LLAMA2_13B
    worst, kept = _rounds_through_the_step_api(spec, 2, width=2, k=3, n_prompt=1024, n_rounds=1, max_ctx=1100)
    print(f"tree pass, 13B layer shape (2 layers), 1023 cached tokens: worst logit distance {worst:.3e}")
    assert worst < TOL


def test_tree_generation_under_the_beta_controller():
    # draft lengths chosen by Thompson sampling; the oracle's round is driven by the lengths the engine took
    from paper_2406_03853_b200 import binding as b
    spec = synth.TINY
    prompt = synth.prompt_tokens(synth.SEED + 21, 28, spec.vocab).numpy()
    u = {k: v.numpy() for k, v in synth.generate_uniforms(160, 100000).items()}
    eng = engine_from_spec(spec, max_ctx=160, k_cap=7, tree_width=2, controller=b.CTRL_BETA_TS)
    out, trace, st = eng.generate(prompt, 48, uniforms=u)
    ks = [k for k, _, _ in trace]
    assert len(set(ks)) > 1 and max(ks) <= 7
    ref, rtrace, rleaves = oracle_from_spec(spec, 160).generate_tree(prompt, 48, width=2, k_schedule=ks)
    np.testing.assert_array_equal(out, ref)
    assert trace == rtrace and st.leaves_kept == rleaves
    eng.close()


def test_tree_generation_up_to_the_context_limit():
    # the last rounds draft fewer tokens so that the tree rows still fit; one token more is refused up front
    from paper_2406_03853_b200 import EesdError
    spec = synth.TINY
    prompt = synth.prompt_tokens(synth.SEED + 5, 30, spec.vocab).numpy()
    ref, rtrace, rleaves = oracle_from_spec(spec, 64).generate_tree(prompt, 31, width=3, fixed_k=5)
    eng = engine_from_spec(spec, max_ctx=64, fixed_k=5, k_cap=5, tree_width=3)
    out, trace, st = eng.generate(prompt, 31)
    np.testing.assert_array_equal(out, ref)
    assert trace == rtrace and st.leaves_kept == rleaves
    assert trace[-1][0] < 5   # shortened at the end
    with pytest.raises(EesdError):
        eng.generate(prompt, 32)
    eng.close()
