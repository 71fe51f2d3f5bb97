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
    print(f"{spec.name}: vs fp64-cache oracle: hidden {e64:.3e}, logits {np.abs(eng.logits(0, M).cpu().numpy() - lg64).max():.3e}")
    assert e64 < 2.0 ** -7 * np.abs(hid64).max()
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
