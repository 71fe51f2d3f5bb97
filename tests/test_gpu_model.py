"""GPU parity of the model path against the CPU oracle: tiny fp32 configuration end to end
(identical tokens), per-layer hidden states and logits, paging / rollback behaviour."""
import numpy as np
import pytest
import torch

import eesd_synth as synth
import oracle
from tests.helpers import engine_from_spec, oracle_from_spec

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tiny_engine():
    eng = engine_from_spec(synth.TINY, max_ctx=160, k_cap=10, fixed_k=4, page_tokens=8)
    yield eng
    eng.close()


def test_tiny_hidden_states_and_logits_match_oracle(tiny_engine):
    eng, spec = tiny_engine, synth.TINY
    prompt = synth.prompt_tokens(synth.SEED, 32, spec.vocab).numpy()
    m = oracle_from_spec(spec, 160)
    m.target_rows(prompt[:-1], 0, want_logits=False)
    eng.prefill(prompt)
    cap = eng.capture_hidden(True)
    rows = np.concatenate([prompt[-1:], [5, 900, 17, 333, 64, 1, 1023]]).astype(np.int32)
    eng.verify_only(rows)
    torch.cuda.synchronize()
    hid, lg = m.target_rows(rows, 31, want_hidden=True)
    got = cap[:spec.n_layers + 1, :len(rows)].cpu().numpy()
    assert np.abs(got - hid).max() < 2e-5
    assert np.abs(eng.logits(0, len(rows)).cpu().numpy() - lg).max() < 2e-5
    eng.capture_hidden(False)


def test_tiny_draft_logits_match_oracle(tiny_engine):
    eng, spec = tiny_engine, synth.TINY
    prompt = synth.prompt_tokens(synth.SEED + 1, 20, spec.vocab).numpy()
    m = oracle_from_spec(spec, 160)
    m.target_rows(prompt[:-1], 0, want_logits=False)
    eng.prefill(prompt)
    toks = eng.draft(3)
    torch.cuda.synchronize()
    ql = eng.logits(1, 3).cpu().numpy()
    x = int(prompt[-1])
    for i in range(3):
        ref = m.draft_row(x, 19 + i)
        assert np.abs(ql[i] - ref).max() < 2e-5
        x = int(ref.argmax())
        assert toks[i] == x
    n_acc, y = eng.verify_accept()
    _, pl = m.target_rows(np.concatenate([prompt[-1:], toks]).astype(np.int32), 19)
    assert (n_acc, y) == oracle.accept_resample(pl, ql, toks, np.zeros(3), 0.0, 0.0)
    assert eng.context_len()[0] == 20 + n_acc + 1


@pytest.mark.parametrize("mode", ["greedy_fixed4", "greedy_schedule", "greedy_ts", "t1_fixed4", "t1_ts"])
def test_tiny_generate_tokens_identical_to_oracle(tiny_engine, mode):
    from paper_2406_03853_b200 import binding as b
    spec = synth.TINY
    prompt = synth.prompt_tokens(synth.SEED, 32, spec.vocab).numpy()
    u = {k: v.numpy() for k, v in synth.generate_uniforms(160, 200000).items()}
    T = 1.0 if mode.startswith("t1") else 0.0
    ctrl = 1 if mode.endswith("ts") else 0
    ks = [1, 7, 2, 10, 3, 5, 4, 6, 8, 9] * 7 if mode == "greedy_schedule" else None
    eng = engine_from_spec(spec, max_ctx=160, k_cap=10, fixed_k=4, page_tokens=8, temperature=T, controller=ctrl)
    out, trace, st = eng.generate(prompt, 64, k_schedule=ks, uniforms=u)
    ref, rtrace, (a, bb) = oracle_from_spec(spec, 160).generate(prompt, 64, temperature=T, controller=ctrl, fixed_k=4,
                                                               k_schedule=ks, uniforms=u)
    np.testing.assert_array_equal(out, ref)
    assert trace == rtrace
    assert (st.alpha, st.beta) == (a, bb)
    assert st.emitted == 64 and st.drafted == sum(k for k, _, _ in trace) and st.kernel_launches > 0
    eng.close()


def test_paging_rollback_and_errors(tiny_engine):
    eng, spec = tiny_engine, synth.TINY
    prompt = synth.prompt_tokens(3, 17, spec.vocab).numpy()
    eng.prefill(prompt)
    assert eng.context_len() == (17, 3)          # 17 tokens -> 3 pages of 8
    eng.draft(8)                                 # rows up to position 24 -> 4 pages
    assert eng.context_len()[1] == 4
    n_acc, _ = eng.verify_accept()
    n_tok, pages = eng.context_len()
    assert n_tok == 17 + n_acc + 1 and pages == (n_tok - 1 + 7) // 8   # pages past the end were freed
    from paper_2406_03853_b200 import EesdError
    with pytest.raises(EesdError):
        eng.verify_accept()                      # nothing drafted
    with pytest.raises(EesdError):
        eng.draft(11)                            # beyond k_cap
    with pytest.raises(EesdError):
        eng.prefill(np.array([5, 99999], np.int32))  # token id out of range
    with pytest.raises(EesdError):
        eng.prefill(np.arange(200) % 1000)       # longer than max_ctx
    eng.reset()
    assert eng.context_len() == (0, 0)
    with pytest.raises(EesdError):
        eng.draft(1)                             # no prefill


def test_reproducible_and_independent_of_page_size():
    spec = synth.TINY
    prompt = synth.prompt_tokens(9, 40, spec.vocab).numpy()
    outs = []
    for pt in (8, 16, 64):
        eng = engine_from_spec(spec, max_ctx=160, page_tokens=pt, fixed_k=5)
        outs.append(eng.generate(prompt, 48)[0])
        outs.append(eng.generate(prompt, 48)[0])
        eng.close()
    for o in outs[1:]:
        np.testing.assert_array_equal(o, outs[0])


@pytest.mark.parametrize("mode", ["beta", "cali", "tree"])
def test_time_buckets_add_up_to_the_wall_time_of_the_call(mode):
    # the paper's time-breakdown table: drafting + verification + sampling + others = inference time.
    # The library's buckets (plus the prompt pass) must add up to the wall time it reports, and that
    # wall time must be the one a caller measures around the call.
    import time
    from paper_2406_03853_b200 import binding as b
    from paper_2406_03853_b200 import report
    spec = synth.TINY
    kw = dict(max_ctx=256, k_cap=7)
    if mode == "beta":
        kw.update(controller=b.CTRL_BETA_TS, temperature=1.0)
    elif mode == "cali":
        kw.update(controller=b.CTRL_CALI_TS, cali_sigma_m=0.3, cali_sigma_s=0.5, cali_theta0=0.5)
    else:
        kw.update(tree_width=2, fixed_k=3)
    eng = engine_from_spec(spec, **kw)
    if mode == "cali":
        cw = synth.cali_weights(spec, synth.SEED, "cuda")
        g = eng.global_views()
        g["cali_w"].copy_(cw["w"])
        g["cali_wp"].copy_(cw["wp"])
    prompt = synth.prompt_tokens(synth.SEED + 2, 40, spec.vocab).numpy()
    u = {k: v.numpy() for k, v in synth.generate_uniforms(256, 200000).items()}
    eng.generate(prompt, 32, uniforms=u)       # warm-up
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    _, _, st = eng.generate(prompt, 160, uniforms=u)
    wall = (time.perf_counter() - t0) * 1e3
    s = st.as_dict()
    parts = report.time_breakdown(s)
    assert abs(parts["total"] * 1e3 - s["ms_total"]) < 1e-6 * s["ms_total"]
    assert s["ms_total"] <= wall and wall - s["ms_total"] < 0.01 * wall + 0.5     # the binding adds well under 1 % + 0.5 ms
    for k in ("ms_draft", "ms_verify", "ms_sampling", "ms_other", "ms_prefill"):
        assert s[k] > 0.0, k
    assert s["ms_sampling"] < s["ms_verify"] + s["ms_draft"]
    eng.close()


@pytest.mark.parametrize("variant", ["fp32", "bf16"])
def test_two_and_three_exit_layers_match_the_oracle(variant):
    # the paper's experiment on the number of early-exit layers: the draft model is the first N layers plus a
    # stack of exit layers, each with its own cache slot that prefill, verification and draft steps keep in step
    base = synth.TINY if variant == "fp32" else synth.TINY.with_(dtype="bf16", ffn_dim=640)
    for E in (2, 3):
        eng = engine_from_spec(base, max_ctx=160, fixed_k=4, n_exit_layers=E)
        m = oracle_from_spec(base, 160, n_exit=E)
        prompt = synth.prompt_tokens(synth.SEED + E, 37, base.vocab).numpy()
        if variant == "fp32":
            out, trace, _ = eng.generate(prompt, 40, k_schedule=[4, 1, 7, 2, 5] * 8)
            ref, rtrace, _ = m.generate(prompt, 40, k_schedule=[4, 1, 7, 2, 5] * 8)
            np.testing.assert_array_equal(out, ref)
            assert trace == rtrace and sum(a for _, a, _ in trace) > 5
        else:
            # prompt pass (wide kernels), a verify pass, then draft steps whose exit caches were filled by both
            eng.prefill(prompt)
            m.target_rows(prompt[:-1], 0, want_logits=False)
            rows = np.concatenate([prompt[-1:], synth.prompt_tokens(5, 5, base.vocab).numpy()]).astype(np.int32)
            eng.verify_only(rows)
            torch.cuda.synchronize()
            _, lg = m.target_rows(rows, 36)
            assert np.abs(eng.logits(0, 6).cpu().numpy() - lg).max() < 2e-2
            eng.prefill(prompt)
            toks = eng.draft(3)
            torch.cuda.synchronize()
            ql = eng.logits(1, 3).cpu().numpy()
            x = int(prompt[-1])
            for i in range(3):
                ref_q = m.draft_row(x, 36 + i)
                assert np.abs(ql[i] - ref_q).max() < 2e-2
                x = int(toks[i])
        eng.close()
