"""Batch mode: several sequences share the rows of every pass.

Drafting, verification and acceptance of a sequence never look at another sequence (Algorithm 1),
so per sequence the batch must give what the CPU oracle gives for that sequence alone: logits of
a batched verification pass row by row against the oracle, and whole generations (tokens and the
per-round trace) against single-sequence decoding with the draft lengths the batch used and the
same uniforms."""
import numpy as np
import pytest
import torch

import eesd_synth as synth
from tests.helpers import engine_from_spec, oracle_from_spec

pytestmark = pytest.mark.gpu
TOL = 2e-2
BASE = synth.TINY.with_(dtype="bf16", ffn_dim=640)          # every projection tile-aligned: the tensor-core kernels
SPECS = {"mha": BASE, "gqa8": BASE.with_(n_heads=8, n_kv_heads=1, head_dim=64, n_layers=2),
         "wide_head": BASE.with_(n_heads=2, n_kv_heads=1, head_dim=128, n_layers=2),
         "f32": synth.TINY, "f32_gqa": synth.TINY.with_(n_kv_heads=2)}                 # fp32 cache: the SIMT attention kernel


@pytest.mark.parametrize("variant,lens,m,pt,max_ctx", [
    ("mha", (37, 16, 5), 5, 16, 96),            # three sequences, one ending on a page boundary, 15 rows
    ("mha", (9, 3, 30, 17, 2, 8, 33, 1), 2, 8, 64),   # eight sequences of two rows (a one-token prompt among them)
    ("gqa8", (40, 23), 8, 16, 96),              # 64 (head, row) pairs per sequence: two column batches each
    ("wide_head", (300, 150, 2), 4, 16, 384),   # contexts of very different length: 1 to several slices per sequence
    ("mha", (200, 90), 3, 128, 384),            # one page holds the whole context
    ("f32", (37, 16, 5), 5, 16, 96),
    ("f32_gqa", (300, 9, 120, 1), 4, 8, 384),   # fp32 cache, 8-token pages: up to 13 slices for one sequence, one for another
])
def test_batched_verification_pass_matches_the_oracle_row_by_row(variant, lens, m, pt, max_ctx):
    spec = SPECS[variant]
    B = len(lens)
    eng = engine_from_spec(spec, max_ctx=max_ctx, k_cap=10, fixed_k=3, page_tokens=pt, kv_pages=B * (max_ctx // pt))   # one pool for all
    eng.batch_begin(B)
    prompts = [synth.prompt_tokens(40 + b, n, spec.vocab).numpy() for b, n in enumerate(lens)]
    for b, p in enumerate(prompts):
        eng.batch_prefill(b, p)
    rows = np.stack([np.concatenate([p[-1:], synth.prompt_tokens(70 + b, m - 1, spec.vocab).numpy()]) for b, p in enumerate(prompts)])
    eng.batch_verify_only(rows.astype(np.int32))
    torch.cuda.synchronize()
    got = eng.logits(0, B * m).cpu().numpy().reshape(B, m, spec.vocab)
    for b, p in enumerate(prompts):
        o = oracle_from_spec(spec, max_ctx)
        if len(p) > 1:
            o.target_rows(p[:-1], 0, want_logits=False)
        _, lg = o.target_rows(rows[b].astype(np.int32), len(p) - 1)
        err = np.abs(got[b] - lg).max()
        assert err < (TOL if spec.dtype == "bf16" else 2e-4), (b, err)
        n_tok, pages = eng.batch_context_len(b)
        assert n_tok == len(p) and pages == (len(p) - 1 + m + pt - 1) // pt
    eng.batch_begin(0)
    assert eng.context_len() == (0, 0)
    eng.close()


@pytest.mark.parametrize("temperature", [0.0, 1.0])
@pytest.mark.parametrize("lens,pt", [((21, 40, 7), 8), ((12, 33, 5, 18, 26, 1, 9, 64), 16)])
def test_batch_decode_fp32_model_equals_the_oracle(lens, pt, temperature):
    # the fp32 tiny model is the configuration whose tokens equal the oracle's exactly: every sequence of a batch
    # must reproduce the oracle's own generation for its prompt, uniforms and draft lengths, token by token
    spec = synth.TINY
    max_new, max_ctx, B = 32, 128, len(lens)
    eng = engine_from_spec(spec, max_ctx=max_ctx, k_cap=10, fixed_k=3, temperature=temperature, page_tokens=pt, kv_pages=B * (max_ctx // pt))
    prompts = [synth.prompt_tokens(190 + b, n, spec.vocab).numpy() for b, n in enumerate(lens)]
    unis = [{k: v.numpy() for k, v in synth.generate_uniforms(max_ctx, 64, seed=500 + b).items()} for b in range(B)]
    eng.batch_begin(B)
    for b, p in enumerate(prompts):
        eng.batch_prefill(b, p)
    out, traces, _ = eng.batch_decode(max_new, k_schedule=[2, 5, 1, 3, 7, 4] * 8, uniforms=unis if temperature else None)
    for b, p in enumerate(prompts):
        ks = [k for k, _, _ in traces[b]]
        ref, rtrace, _ = oracle_from_spec(spec, max_ctx).generate(p, max_new, temperature=temperature, k_schedule=ks + [3] * 8, fixed_k=3,
                                                                  uniforms=unis[b] if temperature else None)
        np.testing.assert_array_equal(out[b], ref)
        assert traces[b] == rtrace[:len(traces[b])]
    eng.close()


@pytest.mark.parametrize("temperature", [0.0, 1.0])
@pytest.mark.parametrize("variant,lens,n_exit", [("mha", (21, 40, 7), 1), ("gqa8", (12, 33, 5, 18, 26), 1), ("mha", (9, 30), 2)])
def test_batch_decode_equals_single_sequence_decoding(variant, lens, n_exit, temperature):
    spec = SPECS[variant]
    max_new, max_ctx = 40, 128
    B = len(lens)
    eng = engine_from_spec(spec, max_ctx=max_ctx, k_cap=10, fixed_k=3, temperature=temperature, page_tokens=16, kv_pages=B * 8,
                           n_exit_layers=n_exit)     # (two early-exit layers: their caches are synchronised per sequence as well)
    prompts = [synth.prompt_tokens(90 + b, n, spec.vocab).numpy() for b, n in enumerate(lens)]
    unis = [{k: v.numpy() for k, v in synth.generate_uniforms(max_ctx, 64, seed=300 + b).items()} for b in range(B)]
    eng.batch_begin(B)
    for b, p in enumerate(prompts):
        eng.batch_prefill(b, p)
    schedule = [3, 1, 7, 2, 4, 4, 1, 5] * 6
    out, traces, st = eng.batch_decode(max_new, k_schedule=schedule, uniforms=unis if temperature else None)
    for b in range(B):
        n_tok, pages = eng.batch_context_len(b)
        assert n_tok == lens[b] + sum(a + 1 for _, a, _ in traces[b]) and pages == (n_tok - 1 + 15) // 16
        assert all(k * len(lens) <= 16 for k, _, _ in traces[b][:1])     # the first round holds every sequence
    assert st.emitted == B * max_new and st.drafted == sum(k for t in traces for k, _, _ in t)
    eng.batch_begin(0)
    # the same sequences one at a time, with the draft lengths the batch used for each
    for b, p in enumerate(prompts):
        ks = [k for k, _, _ in traces[b]]
        ref, rtrace, _ = eng.generate(p, max_new, k_schedule=ks + [3] * 8, uniforms=unis[b] if temperature else None)
        np.testing.assert_array_equal(out[b], ref)
        assert traces[b] == rtrace[:len(traces[b])]
    eng.close()


def test_batch_mode_errors():
    from paper_2406_03853_b200 import EesdError
    tree = engine_from_spec(synth.TINY, max_ctx=64, tree_width=2, k_cap=5)
    with pytest.raises(EesdError) as e:
        tree.batch_begin(2)                                 # a tree's rows belong to one sequence
    assert e.value.status == -8
    tree.close()
    eng = engine_from_spec(BASE, max_ctx=64, page_tokens=16, kv_pages=8)
    with pytest.raises(EesdError):
        eng.batch_begin(9)
    eng.batch_begin(2)
    p = synth.prompt_tokens(1, 9, BASE.vocab).numpy()
    with pytest.raises(EesdError) as e:
        eng.prefill(p)                                      # single-sequence calls are closed while the batch is open
    assert e.value.status == -4
    eng.batch_prefill(0, p)
    with pytest.raises(EesdError) as e:
        eng.batch_decode(8)                                 # sequence 1 has no prompt
    assert e.value.status == -4
    with pytest.raises(EesdError):
        eng.batch_prefill(2, p)
    eng.batch_prefill(1, p[:4])
    out, traces, _ = eng.batch_decode(8)
    assert out.shape == (2, 8)
    eng.batch_begin(0)
    out1, _, _ = eng.generate(p, 8)                         # and open again afterwards
    np.testing.assert_array_equal(out1, out[0])
    eng.close()


def test_batch_decode_continues_and_page_pool_exhaustion_is_reported():
    from paper_2406_03853_b200 import EesdError
    spec = BASE
    prompts = [synth.prompt_tokens(140 + b, n, spec.vocab).numpy() for b, n in enumerate((11, 30, 19))]
    eng = engine_from_spec(spec, max_ctx=128, k_cap=10, fixed_k=2, page_tokens=16, kv_pages=24)
    eng.batch_begin(3)
    for b, p in enumerate(prompts):
        eng.batch_prefill(b, p)
    whole, _, _ = eng.batch_decode(30)
    eng.batch_begin(3)
    for b, p in enumerate(prompts):
        eng.batch_prefill(b, p)
    first, traces, _ = eng.batch_decode(12)
    # a second call goes on from where every sequence stands (the surplus tokens of its last round included)
    have = [sum(a + 1 for _, a, _ in t) for t in traces]
    rest, _, _ = eng.batch_decode(30 - min(have))
    for b in range(3):
        n_tok, _ = eng.batch_context_len(b)
        np.testing.assert_array_equal(first[b], whole[b][:12])
        extra = have[b] - 12                                  # tokens the first call produced beyond its 12
        np.testing.assert_array_equal(rest[b][:30 - have[b]], whole[b][have[b]:30])
        assert extra >= 0 and n_tok >= len(prompts[b]) + 30
    eng.close()
    # a pool too small for the three contexts: the call says so, and the engine is usable afterwards
    small = engine_from_spec(spec, max_ctx=128, k_cap=10, fixed_k=2, page_tokens=16, kv_pages=8)
    small.batch_begin(3)
    for b, p in enumerate(prompts):
        small.batch_prefill(b, p)                             # 1 + 2 + 2 pages
    with pytest.raises(EesdError) as e:
        small.batch_decode(60)                                # needs about 5 + 6 + 5 pages
    assert e.value.status == -5
    small.batch_begin(0)
    out, _, _ = small.generate(prompts[0], 20)
    np.testing.assert_array_equal(out, whole[0][:20])
    small.close()


def test_a_wait_that_runs_out_in_a_batch_round_is_reported_and_cleared():
    from paper_2406_03853_b200 import EesdError
    eng = engine_from_spec(BASE, max_ctx=96, k_cap=10, fixed_k=3, page_tokens=16, kv_pages=18)
    prompts = [synth.prompt_tokens(160 + b, n, BASE.vocab).numpy() for b, n in enumerate((14, 29, 6))]
    eng.batch_begin(3)
    for b, p in enumerate(prompts):
        eng.batch_prefill(b, p)
    ref, _, _ = eng.batch_decode(16)
    eng.batch_begin(3)
    for b, p in enumerate(prompts):
        eng.batch_prefill(b, p)
    eng.set_wait_limit(0)                                   # every bounded wait gives up at once: nothing is stalled
    with pytest.raises(EesdError) as e:
        eng.batch_decode(16)
    assert e.value.status == -7
    eng.set_wait_limit(None)
    eng.clear_device_error()                                # leaves batch mode, all pages free
    assert eng.context_len() == (0, 0)
    eng.batch_begin(3)
    for b, p in enumerate(prompts):
        eng.batch_prefill(b, p)
    out, _, _ = eng.batch_decode(16)
    np.testing.assert_array_equal(out, ref)
    eng.close()
