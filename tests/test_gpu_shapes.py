"""GPU parity at the LLaMA-2-13B and 70B layer shapes (bf16 weights, the launch configuration
the benchmark times) against the fp32-weight/fp64-math oracle on the same bf16-rounded
weights: projections element by element, and hidden states / logits of a shallow slice of
the model within the 2e-2 max-abs tolerance stated for bf16 against the oracle."""
import numpy as np
import pytest
import torch

import eesd_synth as synth
from tests.helpers import engine_from_spec, oracle_from_spec

pytestmark = pytest.mark.gpu
TOL = 2e-2


@pytest.mark.parametrize("M", [1, 2, 5, 11, 16])
@pytest.mark.parametrize("R,K", [(5120, 5120), (15360, 5120), (5120, 13824), (1000, 264), (8192, 28672), (136, 8192),
                                 (128, 64), (256, 640), (32000, 5120), (57344, 8192)])
def test_projection_matches_fp64_matmul(M, R, K):
    import paper_2406_03853_b200 as eesd
    if (R, K) in ((8192, 28672), (15360, 5120), (32000, 5120), (57344, 8192)) and M not in (1, 11):
        pytest.skip("large shape: two row counts are enough")
    A = synth.normal_f32(5, 1, M * K, "cuda").view(M, K)
    W = (synth.normal_f32(5, 2, R * K, "cuda").view(R, K) * 0.02).to(torch.bfloat16)
    got = eesd.project_rows(A, W).double().cpu().numpy()
    ref = (A.double() @ W.double().T).cpu().numpy()
    scale = np.abs(ref).max()
    assert np.abs(got - ref).max() < 2e-5 * scale + 1e-6   # fp32 accumulation, rows as two bf16 terms


def test_projection_fp32_ragged():
    import paper_2406_03853_b200 as eesd
    for M, R, K in [(1, 1, 8), (3, 33, 688), (16, 1376, 256), (7, 1024, 256)]:
        A = synth.normal_f32(6, 1, M * K, "cuda").view(M, K)
        W = synth.normal_f32(6, 2, R * K, "cuda").view(R, K) * 0.02
        got = eesd.project_rows(A, W).double().cpu().numpy()
        ref = (A.double() @ W.double().T).cpu().numpy()
        assert np.abs(got - ref).max() < 1e-5 * np.abs(ref).max() + 1e-7


def _slice_parity(spec, n_layers, n_prompt, M, max_ctx=96):
    eng = engine_from_spec(spec, n_layers=n_layers, max_ctx=max_ctx, k_cap=15)
    m = oracle_from_spec(spec, max_ctx=max_ctx, n_layers=n_layers, device="cuda")
    prompt = synth.prompt_tokens(synth.SEED, n_prompt, spec.vocab).numpy()
    m.target_rows(prompt[:-1], 0, want_logits=False)
    eng.prefill(prompt)
    cap = eng.capture_hidden(True)
    rows = np.concatenate([prompt[-1:], synth.prompt_tokens(99, M - 1, spec.vocab).numpy()]).astype(np.int32)
    eng.verify_only(rows)
    torch.cuda.synchronize()
    hid, lg = m.target_rows(rows, n_prompt - 1, want_hidden=True)
    got = cap[:n_layers + 1, :M].cpu().numpy()
    err_h = np.abs(got - hid).max(axis=(1, 2))
    err_l = np.abs(eng.logits(0, M).cpu().numpy() - lg).max()
    print(f"{spec.name}: hidden max-abs err per layer {err_h}, logits {err_l:.3e}, |hidden| {np.abs(hid).max():.2f}, "
          f"|logits| {np.abs(lg).max():.2f}")
    assert err_h.max() < TOL and err_l < TOL
    # for the record: distance to the oracle with an unrounded (fp64) cache, i.e. what storing
    # keys and values as bf16 costs; bounded by bf16 rounding of values of this magnitude
    m64 = oracle_from_spec(spec, max_ctx=max_ctx, n_layers=n_layers, device="cuda", kv_bf16=False)
    m64.target_rows(prompt[:-1], 0, want_logits=False)
    hid64, lg64 = m64.target_rows(rows, n_prompt - 1, want_hidden=True)
    e64 = np.abs(got - hid64).max()
    storage_h, storage_l = np.abs(hid - hid64).max(), np.abs(lg - lg64).max()
    print(f"{spec.name}: vs fp64-cache oracle: hidden {e64:.3e}, logits {np.abs(eng.logits(0, M).cpu().numpy() - lg64).max():.3e}; "
          f"storage alone (bf16-cache oracle against fp64-cache oracle): hidden {storage_h:.3e}, logits {storage_l:.3e}")
    assert e64 < 2.0 ** -7 * np.abs(hid64).max()
    # the tolerance is stated against the oracle with the SAME storage format: against an unrounded cache
    # the engine may be as far as the storage rounding itself moves the oracle, plus that tolerance
    assert e64 <= storage_h + TOL
    # the draft model on the same slice: one draft step against the oracle's draft row
    eng.prefill(prompt)
    eng.draft(1)
    torch.cuda.synchronize()
    m2_logits = m.draft_row(int(prompt[-1]), n_prompt - 1)
    err_q = np.abs(eng.logits(1, 1).cpu().numpy()[0] - m2_logits).max()
    print(f"{spec.name}: draft logits err {err_q:.3e}")
    assert err_q < TOL
    eng.close()


def test_13b_shape_slice_hidden_and_logits():
    _slice_parity(synth.LLAMA2_13B, n_layers=2, n_prompt=21, M=11)


def test_70b_shape_slice_hidden_and_logits():
    _slice_parity(synth.LLAMA2_70B, n_layers=1, n_prompt=19, M=6)


def _long_cache_parity(spec, n_layers, n_prompt, Ms, seed=synth.SEED + 3):
    """A real prefill of n_prompt tokens in the engine (wide prompt passes) and in the oracle, then verify
    passes of M rows for every M in Ms against ONE oracle pass of max(Ms) rows (rows are causal, so
    its first M rows are the oracle's answer for a pass of M rows), hidden states per layer and
    logits; then one draft step.  This is the cache length and the launch configuration the
    benchmark's verify-pass leg times: every attention slice of the pass is in play."""
    max_ctx = n_prompt + 32
    eng = engine_from_spec(spec, n_layers=n_layers, max_ctx=max_ctx, k_cap=15)
    m = oracle_from_spec(spec, max_ctx=max_ctx, n_layers=n_layers, device="cuda")
    prompt = synth.prompt_tokens(seed, n_prompt, spec.vocab).numpy()
    m.target_rows(prompt[:-1], 0, want_logits=False)
    eng.prefill(prompt)
    cap = eng.capture_hidden(True)
    Mx = max(Ms)
    rows = np.concatenate([prompt[-1:], synth.prompt_tokens(seed + 1, Mx - 1, spec.vocab).numpy()]).astype(np.int32)
    hid, lg = m.target_rows(rows, n_prompt - 1, want_hidden=True)
    for M in Ms:
        eng.verify_only(rows[:M])
        torch.cuda.synchronize()
        got = cap[:n_layers + 1, :M].cpu().numpy()
        err_h = np.abs(got - hid[:, :M]).max(axis=(1, 2))
        err_l = np.abs(eng.logits(0, M).cpu().numpy() - lg[:M]).max()
        print(f"{spec.name}, cache {n_prompt - 1}, {M} rows: hidden max-abs err per layer {err_h}, logits {err_l:.3e}")
        assert err_h.max() < TOL and err_l < TOL
    eng.capture_hidden(False)
    eng.prefill(prompt)
    eng.draft(1)
    torch.cuda.synchronize()
    err_q = np.abs(eng.logits(1, 1).cpu().numpy()[0] - m.draft_row(int(prompt[-1]), n_prompt - 1)).max()
    print(f"{spec.name}, cache {n_prompt - 1}: draft logits err {err_q:.3e}")
    assert err_q < TOL
    eng.close()


def test_13b_shape_1024_token_cache_verify_passes():
    _long_cache_parity(synth.LLAMA2_13B, n_layers=2, n_prompt=1024, Ms=(1, 6, 16))


def test_70b_shape_1024_token_cache_verify_passes():
    # 8 query heads per KV head: 6 rows are 48 (head, row) pairs, two column batches per KV head
    _long_cache_parity(synth.LLAMA2_70B, n_layers=1, n_prompt=1024, Ms=(1, 6))


def test_13b_shape_error_growth_over_eight_layers():
    # A deeper slice (8 layers, the first five undamped, short cache): the per-layer distance to the
    # oracle on record.  Logits stay within the stated 2e-2.  Hidden states of magnitude 30 do not, and
    # cannot for any fp32 implementation: with keys and values STORED as bf16 the function itself jumps
    # where a value sits on a rounding boundary.  The size of those jumps is measured here on the
    # oracle alone (its own output when the embedding moves by about one fp32 unit in the last place),
    # and the engine is asked to stay within the stated tolerance plus three times that distance.
    import oracle
    spec, L, n_prompt, M = synth.LLAMA2_13B, 8, 21, 6
    eng = engine_from_spec(spec, n_layers=L, max_ctx=64, k_cap=15)
    layers = [{k: v.cpu() for k, v in synth.layer_weights(spec, l, synth.SEED, "cuda").items()} for l in range(L)]
    ex = {k: v.cpu() for k, v in synth.exit_layer_weights(spec, synth.SEED, "cuda").items()}
    emb, head = synth.embedding(spec, synth.SEED, "cuda").cpu().float(), synth.lm_head(spec, synth.SEED, "cuda").cpu()
    s = spec.with_(n_layers=L, n_early=min(spec.n_early, L))
    prompt = synth.prompt_tokens(synth.SEED + 9, n_prompt, spec.vocab).numpy()
    rows = np.concatenate([prompt[-1:], synth.prompt_tokens(77, M - 1, spec.vocab).numpy()]).astype(np.int32)
    noise = 1 + (torch.rand(emb.shape, generator=torch.Generator().manual_seed(1)) - 0.5) * 2.0 ** -22
    runs = []
    for e in (emb, emb * noise):
        m = oracle.model_from_weights(s, layers, ex, e, head, max_ctx=64, kv_bf16=True)
        m.target_rows(prompt[:-1], 0, want_logits=False)
        runs.append(m.target_rows(rows, n_prompt - 1, want_hidden=True))
    (hid, lg), (hid_n, lg_n) = runs
    jump_h, jump_l = np.abs(hid - hid_n).max(axis=(1, 2)), np.abs(lg - lg_n).max()
    eng.prefill(prompt)
    cap = eng.capture_hidden(True)
    eng.verify_only(rows)
    torch.cuda.synchronize()
    err_h = np.abs(cap[:L + 1, :M].cpu().numpy() - hid).max(axis=(1, 2))
    err_l = np.abs(eng.logits(0, M).cpu().numpy() - lg).max()
    np.set_printoptions(linewidth=250)
    print(f"13b, {L} layers: engine vs oracle, hidden max-abs after the embedding and after each layer {np.array2string(err_h, precision=4)}; "
          f"oracle vs oracle with the embedding moved by one fp32 ulp {np.array2string(jump_h, precision=4)}; "
          f"|hidden| {np.array2string(np.abs(hid).max(axis=(1, 2)), precision=1)}; logits: engine {err_l:.3e}, oracle jump {jump_l:.3e}")
    assert err_l < TOL
    assert (err_h < TOL + 3 * jump_h).all()
    assert err_h[:3].max() < TOL          # the shallow part holds the plain tolerance
    eng.close()
