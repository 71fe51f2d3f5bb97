"""GPU edge cases against the oracle: shortest and longest rounds, page boundaries, context
limits, grouped-query and wide-head variants, bf16 models on both projection paths, the step
API with explicit uniforms, and launch without programmatic dependent launch."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import eesd_synth as synth
import oracle
from tests.helpers import engine_from_spec, oracle_from_spec

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_one_token_prompt_one_new_token_and_longest_round():
    spec = synth.TINY
    eng = engine_from_spec(spec, max_ctx=96, k_cap=15, fixed_k=15, page_tokens=8)
    m = oracle_from_spec(spec, 96)
    out, trace, st = eng.generate(np.array([7], np.int32), 1)
    ref, rtrace, _ = m.generate(np.array([7], np.int32), 1, k_cap=15, fixed_k=15)
    np.testing.assert_array_equal(out, ref)
    assert trace == rtrace and trace[0][0] == 15          # a 15-token draft, 16-row verify pass
    prompt = synth.prompt_tokens(2, 9, spec.vocab).numpy()
    out, trace, _ = eng.generate(prompt, 40)
    ref, rtrace, _ = oracle_from_spec(spec, 96).generate(prompt, 40, k_cap=15, fixed_k=15)
    np.testing.assert_array_equal(out, ref)
    assert trace == rtrace
    eng.close()


def test_context_limit_is_an_error_not_a_fault():
    from paper_2406_03853_b200 import EesdError
    spec = synth.TINY
    eng = engine_from_spec(spec, max_ctx=48, k_cap=10, fixed_k=4, page_tokens=8)
    prompt = synth.prompt_tokens(3, 30, spec.vocab).numpy()
    with pytest.raises(EesdError) as e:
        eng.generate(prompt, 30)                           # 30 + 30 + 1 > max_ctx
    assert e.value.status == -5
    out, _, _ = eng.generate(prompt, 17)                   # exactly fits: 30 + 17 + 1 = 48
    ref, _, _ = oracle_from_spec(spec, 48).generate(prompt, 17, fixed_k=4)
    np.testing.assert_array_equal(out, ref)
    eng.prefill(prompt)
    eng.draft(10)
    with pytest.raises(EesdError):
        eng.draft(1)                                       # beyond k_cap within one round
    eng.close()
    with pytest.raises(EesdError):
        engine_from_spec(spec, max_ctx=64, kv_pages=3)     # page pool smaller than max_ctx needs


@pytest.mark.parametrize("variant", ["gqa", "wide_head", "bf16_simt", "bf16_tensor_core"])
def test_model_variants_match_oracle(variant):
    base = synth.TINY
    spec = {
        "gqa": base.with_(n_kv_heads=2),
        "wide_head": base.with_(n_heads=2, n_kv_heads=1, head_dim=128),
        "bf16_simt": base.with_(dtype="bf16"),                       # 2F = 1376 is not a multiple of 128
        "bf16_tensor_core": base.with_(dtype="bf16", ffn_dim=640),   # every projection tile-aligned
    }[variant]
    eng = engine_from_spec(spec, max_ctx=96, k_cap=10, fixed_k=3, page_tokens=16)
    m = oracle_from_spec(spec, 96)
    prompt = synth.prompt_tokens(4, 37, spec.vocab).numpy()
    m.target_rows(prompt[:-1], 0, want_logits=False)
    eng.prefill(prompt)
    cap = eng.capture_hidden(True)
    rows = np.concatenate([prompt[-1:], synth.prompt_tokens(5, 6, spec.vocab).numpy()]).astype(np.int32)
    eng.verify_only(rows)
    torch.cuda.synchronize()
    hid, lg = m.target_rows(rows, 36, want_hidden=True)
    tol = 2e-5 if spec.dtype == "f32" else 2e-2
    assert np.abs(cap[:spec.n_layers + 1, :7].cpu().numpy() - hid).max() < tol
    assert np.abs(eng.logits(0, 7).cpu().numpy() - lg).max() < tol
    eng.capture_hidden(False)
    if spec.dtype == "f32":
        out, trace, _ = eng.generate(prompt, 24)
        ref, rtrace, _ = oracle_from_spec(spec, 96).generate(prompt, 24, fixed_k=3)
        np.testing.assert_array_equal(out, ref)
        assert trace == rtrace
    eng.close()


def test_step_api_with_explicit_uniforms_equals_oracle_rounds():
    spec = synth.TINY
    eng = engine_from_spec(spec, max_ctx=128, k_cap=10, temperature=1.0, page_tokens=8)
    m = oracle_from_spec(spec, 128)
    prompt = synth.prompt_tokens(6, 15, spec.vocab).numpy()   # ends one short of a page boundary
    eng.prefill(prompt)
    m.target_rows(prompt[:-1], 0, want_logits=False)
    ctx = list(prompt)
    for rnd, K in enumerate([3, 1, 10, 2, 6]):
        ud = synth.uniforms(100 + rnd, 1, K).numpy()
        ua = synth.uniforms(100 + rnd, 2, K).numpy()
        ur = float(synth.uniforms(100 + rnd, 3, 1).numpy()[0])
        toks = np.concatenate([eng.draft(K - K // 2, ud[:K - K // 2]), eng.draft(K // 2, ud[K - K // 2:])]) if K > 1 \
            else eng.draft(1, ud)                              # drafting may be interleaved call by call
        T = len(ctx)
        xs, ql = [ctx[-1]], []
        for i in range(K):
            lgq = m.draft_row(xs[-1], T - 1 + i)
            ql.append(lgq)
            xs.append(oracle.sample_logits(lgq, 1.0, float(ud[i])))
        np.testing.assert_array_equal(toks, xs[1:])
        n_acc, y = eng.verify_accept(ua, ur)
        _, pl = m.target_rows(np.array(xs, np.int32), T - 1)
        assert (n_acc, y) == oracle.accept_resample(pl, np.stack(ql), xs[1:], ua, ur, 1.0)
        ctx += xs[1:1 + n_acc] + [y]
        n_tok, pages = eng.context_len()
        assert n_tok == len(ctx) and pages == (n_tok - 1 + 7) // 8
    eng.close()


def test_same_tokens_without_programmatic_dependent_launch():
    code = ("import sys; sys.path.insert(0, %r); import numpy as np, eesd_synth as synth;"
            "from tests.helpers import engine_from_spec;"
            "spec = synth.TINY.with_(dtype='bf16', ffn_dim=640);"
            "eng = engine_from_spec(spec, max_ctx=96, fixed_k=4);"
            "out, _, _ = eng.generate(synth.prompt_tokens(8, 20, 1024).numpy(), 32);"
            "print(' '.join(map(str, out)))") % ROOT
    outs = []
    for env_extra in ({}, {"EESD_NO_PDL": "1"}):
        env = dict(os.environ, **env_extra)
        r = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, env=env, timeout=600)
        assert r.returncode == 0, r.stderr[-2000:]
        outs.append(r.stdout.strip().splitlines()[-1])
    assert outs[0] == outs[1] and len(outs[0].split()) == 32


@pytest.mark.parametrize("variant,n_prompt,max_ctx,pt", [("mha", 300, 384, 16), ("gqa8", 150, 256, 16), ("wide_head", 200, 256, 16),
                                                           ("two_passes", 700, 768, 16), ("mha", 131, 256, 8), ("mha", 258, 384, 128),
                                                           ("wide_head", 700, 768, 128), ("wide_head", 530, 640, 8),
                                                           ("gqa8", 66, 128, 32)])
def test_wide_prompt_pass_matches_row_chunks_and_oracle(variant, n_prompt, max_ctx, pt):
    """Prompts longer than 16 rows go through the wide projection kernel (128-row panels) and
    the causal prompt attention kernel (128 query rows per block, streaming over 128-position
    tiles); the cache they leave must equal, up to summation order, the one built 16 rows at a
    time, and the next pass must match the oracle.  Variants: ragged panels and row tiles (a last
    tile of 1, 2 or 17 rows), 8 query heads per KV head, 128-wide heads, every page size from 8
    to 128 tokens, and prompts of more than 512 rows (a second pass that starts at a non-zero
    position, whose first row tile already sees four full tiles)."""
    base = synth.TINY.with_(dtype="bf16", ffn_dim=640, n_layers=3)
    spec = {"mha": base, "two_passes": base.with_(n_layers=2),
            "gqa8": base.with_(n_heads=8, n_kv_heads=1, head_dim=64),
            "wide_head": base.with_(n_heads=2, n_kv_heads=1, head_dim=128)}[variant]
    prompt = synth.prompt_tokens(9, n_prompt, spec.vocab).numpy()
    wide = engine_from_spec(spec, max_ctx=max_ctx, k_cap=10, fixed_k=3, page_tokens=pt)
    rows = engine_from_spec(spec, max_ctx=max_ctx, k_cap=10, fixed_k=3, page_tokens=pt)
    rows.capture_hidden(True)                                 # capture keeps the 16-row path
    n0 = wide.launch_count()
    wide.prefill(prompt)
    n_wide = wide.launch_count() - n0
    n0 = rows.launch_count()
    rows.prefill(prompt)
    assert n_wide < (rows.launch_count() - n0) // 2
    torch.cuda.synchronize()
    a = wide.kv_pool.view(torch.bfloat16).float()
    b = rows.kv_pool.view(torch.bfloat16).float()
    assert (a != 0).sum() == (b != 0).sum() > 0
    assert (a - b).abs().max().item() < 2e-2
    assert ((a - b).abs() > 1e-3).float().mean().item() < 1e-3   # bf16 rounding flips only
    m = oracle_from_spec(spec, max_ctx)
    m.target_rows(prompt[:-1], 0, want_logits=False)
    new = np.concatenate([prompt[-1:], synth.prompt_tokens(10, 4, spec.vocab).numpy()]).astype(np.int32)
    _, lg = m.target_rows(new, n_prompt - 1)
    for eng in (wide, rows):
        eng.verify_only(new)
        torch.cuda.synchronize()
        assert np.abs(eng.logits(0, 5).cpu().numpy() - lg).max() < 2e-2
    wide.close(); rows.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_long_context_many_slices(dtype):
    """Contexts far beyond one block's slice: the fp32 model (8-token pages, prompt fed 16 rows at
    a time) reaches 63 slices per head in the verify pass (both halves of the 64-entry merge);
    the bf16 model feeds a 2000-token prompt through four wide passes whose attention chunks
    see 1 to 11 slices."""
    if dtype == "f32":
        spec, n_prompt, max_ctx, pt, tol = synth.TINY.with_(n_layers=2), 4000, 4096, 8, 2e-4
    else:
        spec, n_prompt, max_ctx, pt, tol = synth.TINY.with_(dtype="bf16", ffn_dim=640, n_layers=2), 2000, 2048, 16, 2e-2
    eng = engine_from_spec(spec, max_ctx=max_ctx, k_cap=10, fixed_k=3, page_tokens=pt)
    m = oracle_from_spec(spec, max_ctx)
    prompt = synth.prompt_tokens(13, n_prompt, spec.vocab).numpy()
    eng.prefill(prompt)
    m.target_rows(prompt[:-1], 0, want_logits=False)
    new = np.concatenate([prompt[-1:], synth.prompt_tokens(14, 8, spec.vocab).numpy()]).astype(np.int32)
    eng.verify_only(new)
    torch.cuda.synchronize()
    _, lg = m.target_rows(new, n_prompt - 1)
    assert np.abs(eng.logits(0, 9).cpu().numpy() - lg).max() < tol
    eng.close()


@pytest.mark.parametrize("dtype,n_prompt", [("f32", 12), ("bf16", 12), ("bf16", 150)])
def test_a_wait_that_runs_out_is_reported_and_the_context_recovers(dtype, n_prompt):
    # With the bound of the in-kernel waits at zero, the first wait of every thread block (attention:
    # its cache slice; projection: the first ring stage / accumulator) gives up before any tensor-core
    # operation is issued; the blocks let the copies they had requested land and return.  The call
    # must report a device error (not hang, not fault), and after clearing it the same context must
    # produce the oracle's tokens again.  Nothing is stalled on the GPU to get here.
    from paper_2406_03853_b200 import EesdError
    spec = synth.TINY if dtype == "f32" else synth.TINY.with_(dtype="bf16", ffn_dim=640)
    eng = engine_from_spec(spec, max_ctx=96 if n_prompt < 64 else 192, fixed_k=3)
    prompt = synth.prompt_tokens(21, n_prompt, spec.vocab).numpy()   # 150 tokens: the prompt pass's wide kernels give up too
    out0, trace0, _ = eng.generate(prompt, 16)
    eng.set_wait_limit(0)
    with pytest.raises(EesdError) as e:
        eng.generate(prompt, 16)
    assert e.value.status == -7                             # EESD_ERR_DEVICE
    eng.set_wait_limit(None)
    eng.clear_device_error()
    out1, trace1, _ = eng.generate(prompt, 16)
    np.testing.assert_array_equal(out1, out0)
    assert trace1 == trace0
    if dtype == "f32":
        ref, rtrace, _ = oracle_from_spec(spec, 96).generate(prompt, 16, fixed_k=3)
        np.testing.assert_array_equal(out1, ref)
    eng.close()
