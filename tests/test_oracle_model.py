"""Pins for the oracle's model forward (Eq. 1 draft model, target verification pass).

Each test checks the C oracle against something fixed outside it: hand-computed numbers,
textbook identities, structural facts the paper prints (parameter counts), or an
independent dense-matrix formulation evaluated with numpy's matmul.
"""
import math

import numpy as np
import pytest

import eesd_synth as synth
import oracle
from tests.helpers import oracle_from_spec


# ---------------------------------------------------------------- RMSNorm / RoPE on hand-sized inputs
def test_rmsnorm_hand_values():
    # x = (1,2,3,4): mean square 7.5; with eps = 0 the result is x / sqrt(7.5), times the gain
    out = oracle.rmsnorm([1.0, 2.0, 3.0, 4.0], [1.0, 1.0, 2.0, 0.5], 0.0)
    r = 1.0 / math.sqrt(7.5)
    np.testing.assert_allclose(out, [r, 2 * r, 6 * r, 2 * r], rtol=1e-15)
    # eps enters under the root: x = (3,4), eps = 0.5 -> mean square 12.5 + 0.5 = 13
    out = oracle.rmsnorm([3.0, 4.0], [1.0, 1.0], 0.5)
    np.testing.assert_allclose(out, [3 / math.sqrt(13), 4 / math.sqrt(13)], rtol=1e-15)


def test_rope_hand_values_and_relative_property():
    # D = 2: a single pair turning by pos radians (theta^0 = 1)
    v = oracle.rope([1.0, 0.0], 1, 10000.0)
    np.testing.assert_allclose(v, [math.cos(1), math.sin(1)], rtol=1e-15)
    v = oracle.rope([0.0, 2.0], 3, 10000.0)
    np.testing.assert_allclose(v, [-2 * math.sin(3), 2 * math.cos(3)], rtol=1e-15)
    # D = 4, second pair turns by pos * 10000^(-1/2) = pos / 100
    v = oracle.rope([0.0, 0.0, 1.0, 0.0], 50, 10000.0)
    np.testing.assert_allclose(v, [0, 0, math.cos(0.5), math.sin(0.5)], atol=1e-15)
    # position 0 is the identity; rotation keeps the norm; <rope(q,m), rope(k,n)> depends on m-n only
    rng = np.random.default_rng(0)
    q, k = rng.standard_normal(64), rng.standard_normal(64)
    np.testing.assert_array_equal(oracle.rope(q, 0, 10000.0), q)
    assert abs(np.linalg.norm(oracle.rope(q, 77, 10000.0)) - np.linalg.norm(q)) < 1e-12
    a = oracle.rope(q, 9, 10000.0) @ oracle.rope(k, 4, 10000.0)
    b = oracle.rope(q, 105, 10000.0) @ oracle.rope(k, 100, 10000.0)
    assert abs(a - b) < 1e-10


# ---------------------------------------------------------------- independent dense formulation
def _dense_layer(x, lw, spec, theta=10000.0, eps=1e-5):
    """One LLaMA decoder layer on a whole sequence x[T,d] with a causal mask, as matrix
    products (numpy fp64).  Independent of the oracle's row-by-row cached loops."""
    T, d = x.shape
    H, Hkv, D, F = spec.n_heads, spec.n_kv_heads, spec.head_dim, spec.ffn_dim
    w = {k: v.double().numpy() for k, v in lw.items()}

    def norm(a, g):
        return a / np.sqrt((a * a).mean(-1, keepdims=True) + eps) * g

    def rot(a):  # a [T, heads, D]
        i = np.arange(D // 2)
        ang = np.arange(T)[:, None] * theta ** (-2.0 * i / D)[None, :]
        c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
        out = np.empty_like(a)
        out[..., 0::2] = a[..., 0::2] * c - a[..., 1::2] * s
        out[..., 1::2] = a[..., 0::2] * s + a[..., 1::2] * c
        return out

    n = norm(x, w["g_attn"])
    qkv = n @ w["wqkv"].T
    q = rot(qkv[:, :H * D].reshape(T, H, D))
    k = rot(qkv[:, H * D:(H + Hkv) * D].reshape(T, Hkv, D))
    v = qkv[:, (H + Hkv) * D:].reshape(T, Hkv, D)
    k = np.repeat(k, H // Hkv, axis=1)
    v = np.repeat(v, H // Hkv, axis=1)
    sc = np.einsum("thd,shd->hts", q, k) / math.sqrt(D)
    sc = np.where(np.tril(np.ones((T, T), bool))[None], sc, -np.inf)
    p = np.exp(sc - sc.max(-1, keepdims=True))
    p /= p.sum(-1, keepdims=True)
    att = np.einsum("hts,shd->thd", p, v).reshape(T, H * D)
    x = x + att @ w["wo"].T
    n = norm(x, w["g_ffn"])
    gu = n @ w["wgu"].T
    g, u = gu[:, :F], gu[:, F:]
    return x + (g / (1 + np.exp(-g)) * u) @ w["wd"].T


def test_layer_matches_dense_causal_formulation(tiny_oracle):
    spec = synth.TINY
    toks = synth.prompt_tokens(7, 24, spec.vocab).numpy()
    x0 = tiny_oracle.embed(toks) * 30.0  # O(1) inputs so attention is not flat
    for lidx in (0, 3):
        ref = _dense_layer(x0, synth.layer_weights(spec, lidx), spec)
        got = tiny_oracle.layer_fwd(lidx, lidx, x0, 0)
        np.testing.assert_allclose(got, ref, rtol=0, atol=1e-10)


def test_gqa_equals_mha_with_repeated_kv_heads():
    # A grouped-query layer must equal a multi-head layer whose k/v head weights are the
    # group's weights repeated (textbook definition of GQA).
    spec = synth.TINY.with_(n_kv_heads=2, n_layers=1, n_early=1)
    lw = synth.layer_weights(spec, 0)
    D, H, Hkv, d = spec.head_dim, spec.n_heads, spec.n_kv_heads, spec.d_model
    wq, wk, wv = lw["wqkv"][:H * D], lw["wqkv"][H * D:(H + Hkv) * D], lw["wqkv"][(H + Hkv) * D:]
    rep = lambda w: w.view(Hkv, D, d).repeat_interleave(H // Hkv, dim=0).reshape(H * D, d)
    lw_mha = dict(lw, wqkv=np.concatenate([wq, rep(wk), rep(wv)], 0))
    emb, head = synth.embedding(spec), synth.lm_head(spec)
    m_gqa = oracle.model_from_weights(spec, [lw], lw, emb, head, max_ctx=32)
    m_mha = oracle.model_from_weights(spec.with_(n_kv_heads=H), [lw_mha], lw_mha, emb, head, max_ctx=32)
    x0 = m_gqa.embed(np.arange(10)) * 30.0
    np.testing.assert_allclose(m_gqa.layer_fwd(0, 0, x0, 0), m_mha.layer_fwd(0, 0, x0, 0), atol=1e-12)


def test_single_position_attention_returns_value_and_zero_weights_are_identity():
    spec = synth.TINY.with_(n_layers=1, n_early=1)
    lw = synth.layer_weights(spec, 0)
    emb, head = synth.embedding(spec), synth.lm_head(spec)
    # Wd = 0, Wo = I: with one position softmax is 1, so the layer adds exactly v = Wv.RMSNorm(x)
    eye = np.eye(spec.d_model, dtype=np.float32)
    lw1 = dict(lw, wo=eye, wd=np.zeros_like(lw["wd"].numpy()))
    m = oracle.model_from_weights(spec, [lw1], lw1, emb, head, max_ctx=8)
    x0 = m.embed([5]) * 30.0
    wv = lw["wqkv"][(spec.n_heads + spec.n_kv_heads) * spec.head_dim:].double().numpy()
    v = wv @ oracle.rmsnorm(x0[0], np.ones(spec.d_model), 1e-5)
    np.testing.assert_allclose(m.layer_fwd(0, 0, x0, 0)[0], x0[0] + v, atol=1e-12)
    # Wo = 0 and Wd = 0: the layer is the identity on the residual stream
    lw0 = dict(lw, wo=np.zeros_like(eye), wd=np.zeros_like(lw["wd"].numpy()))
    m0 = oracle.model_from_weights(spec, [lw0], lw0, emb, head, max_ctx=8)
    x = m0.embed([1, 2, 3])
    np.testing.assert_array_equal(m0.layer_fwd(0, 0, x, 0), x)


# ---------------------------------------------------------------- cache consistency
def test_cached_rows_equal_full_recompute_and_row_by_row(tiny_oracle):
    m = tiny_oracle
    toks = synth.prompt_tokens(11, 20, synth.TINY.vocab).numpy()
    hid_full, lg_full = m.target_rows(toks, 0, want_hidden=True)
    # the same sequence fed as 12 rows, then 5, then 3 single rows: the KV cache carries the prefix
    parts, pos = [], 0
    for chunk in (12, 5, 1, 1, 1):
        h, lg = m.target_rows(toks[pos:pos + chunk], pos, want_hidden=True)
        parts.append((h, lg))
        pos += chunk
    hid_inc = np.concatenate([h for h, _ in parts], axis=1)
    lg_inc = np.concatenate([lg for _, lg in parts], axis=0)
    np.testing.assert_allclose(hid_inc, hid_full, atol=1e-12)
    np.testing.assert_allclose(lg_inc, lg_full, atol=1e-6)


def test_causality_future_tokens_do_not_change_earlier_rows(tiny_oracle):
    a = synth.prompt_tokens(3, 10, 1024).numpy()
    b = a.copy()
    b[7:] = (b[7:] + 13) % 1024
    _, la = tiny_oracle.target_rows(a, 0)
    _, lb = tiny_oracle.target_rows(b, 0)
    np.testing.assert_array_equal(la[:7], lb[:7])
    assert np.abs(la[7:] - lb[7:]).max() > 1e-4


# ---------------------------------------------------------------- draft model structure (Eq. 1)
def test_draft_row_is_first_n_layers_then_exit_layer_then_own_head(tiny_oracle):
    m, spec = tiny_oracle, synth.TINY
    toks = synth.prompt_tokens(5, 9, spec.vocab).numpy()
    m.target_rows(toks[:-1], 0, want_logits=False)           # fills target + exit KV for 0..7
    lg, hid = m.draft_row(toks[-1], 8, want_hidden=True)
    # compose the same thing from the layer primitive: layers 0..N-1 on slots 0..N-1, then
    # the exit weights (index L) on the exit slot (index L); exit KV for 0..7 must already exist
    m2 = oracle_from_spec(spec, max_ctx=160)
    x = m2.embed(toks)
    for l in range(spec.n_early):
        x = m2.layer_fwd(l, l, x, 0)
    x = m2.layer_fwd(spec.n_layers, spec.n_layers, x, 0)
    np.testing.assert_allclose(hid, x[-1], atol=1e-12)
    np.testing.assert_allclose(lg, m2.head(x[-1:], exit_head=True)[0], atol=1e-6)
    # tiny config: exit layer is a copy of the last target layer and the head is tied
    lw_last, lw_exit = synth.layer_weights(spec, spec.n_layers - 1), synth.exit_layer_weights(spec)
    assert all((lw_last[k] == lw_exit[k]).all() for k in lw_last)


def test_parameter_counts_match_the_papers_tables():
    # Table 1 prints the trainable parameters of EESD as 481M (13B) and 1.12B (70B): one
    # decoder layer plus one vocabulary head.  Table 6 prints loaded parameters 1.6B / 5.6B for
    # N = 3 / N = 5 early layers + exit layer + head + embedding.
    s13, s70 = synth.LLAMA2_13B, synth.LLAMA2_70B
    head13, head70 = s13.vocab * s13.d_model, s70.vocab * s70.d_model
    assert round((s13.layer_params + head13) / 1e6) == 481
    assert round((s70.layer_params + head70) / 1e9, 2) == 1.12
    assert round((4 * s13.layer_params + 2 * head13) / 1e9, 1) == 1.6
    assert abs((6 * s70.layer_params + 2 * head70) / 1e9 - 5.6) < 0.06
    # the shapes the oracle is built with carry exactly these counts
    lw = synth.layer_weights(synth.TINY, 0)
    assert sum(v.numel() for k, v in lw.items() if k.startswith("w")) == synth.TINY.layer_params


def test_bf16_storage_rounding_matches_library_conversion_and_only_touches_the_cache():
    import torch
    xs = np.concatenate([synth.normal_f32(8, 1, 20000).numpy().astype(np.float64) * 3.0,
                         [0.0, 1.0, 1.00390625, 1.001953125, 1.005859375, -2.5e-7, 3.0e38, 65504.0]])
    got = np.array([oracle.bf16_round(x) for x in xs])
    ref = torch.tensor(xs, dtype=torch.float32).to(torch.bfloat16).double().numpy()  # round-to-nearest-even
    np.testing.assert_array_equal(got, ref)
    # the storage rounding moves a layer's output: not a no-op on these inputs
    spec = synth.TINY.with_(n_layers=1, n_early=1)
    lw = synth.layer_weights(spec, 0)
    emb, head = synth.embedding(spec), synth.lm_head(spec)
    a = oracle.model_from_weights(spec, [lw], lw, emb, head, max_ctx=16, kv_bf16=False)
    b = oracle.model_from_weights(spec, [lw], lw, emb, head, max_ctx=16, kv_bf16=True)
    x0 = a.embed([5, 6, 7, 8]) * 30.0
    ya, yb = a.layer_fwd(0, 0, x0, 0), b.layer_fwd(0, 0, x0, 0)
    d = np.abs(ya - yb).max()
    assert 0 < d < 2.0 ** -7 * np.abs(ya).max()


def _bf16(a):
    """bfloat16 storage of fp64 values through the library conversion (fp64 -> fp32 -> bf16, nearest even)."""
    import torch
    return torch.tensor(np.asarray(a, np.float64), dtype=torch.float32).to(torch.bfloat16).double().numpy()


def test_bf16_cache_one_position_moves_the_output_by_exactly_wo_times_the_value_rounding():
    # One cached position: the softmax weight is 1 whatever the key is, so attention returns the
    # cached value itself.  With W_down = 0 the layer is x + Wo v, hence
    #   layer(bf16 cache) - layer(fp64 cache) = Wo (bf16(v) - v),   v = Wv RMSNorm(x)
    # exactly (a rounding of the value only; rounding anything else, or not rounding, breaks it).
    spec = synth.TINY.with_(n_layers=1, n_early=1, n_kv_heads=2)
    lw = synth.layer_weights(spec, 0)
    lw = dict(lw, wd=np.zeros_like(lw["wd"].numpy()))
    emb, head = synth.embedding(spec), synth.lm_head(spec)
    a = oracle.model_from_weights(spec, [lw], lw, emb, head, max_ctx=8, kv_bf16=False)
    b = oracle.model_from_weights(spec, [lw], lw, emb, head, max_ctx=8, kv_bf16=True)
    x0 = a.embed([5]) * 30.0
    H, Hkv, D = spec.n_heads, spec.n_kv_heads, spec.head_dim
    n = x0[0] / np.sqrt((x0[0] ** 2).mean() + spec.rms_eps)
    v = lw["wqkv"][(H + Hkv) * D:].double().numpy() @ n                     # [Hkv * D]
    dv = np.repeat((_bf16(v) - v).reshape(Hkv, D), H // Hkv, axis=0).reshape(H * D)   # every query head reads its group's value
    assert np.abs(dv).max() > 1e-6
    want = lw["wo"].double().numpy() @ dv
    got = b.layer_fwd(0, 0, x0, 0)[0] - a.layer_fwd(0, 0, x0, 0)[0]
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)


def _dense_layer_bf16_cache(x, lw, spec, where="after", theta=10000.0, eps=1e-5):
    """The dense causal formulation of a decoder layer with keys and values stored as bfloat16:
    keys rounded AFTER the rotation (what sits in a cache of rotated keys), values as projected.
    `where` = "before" rounds the keys before the rotation, "values_only" leaves the keys alone:
    the two misplacements the pin below must tell apart from the right one."""
    T, d = x.shape
    H, Hkv, D, F = spec.n_heads, spec.n_kv_heads, spec.head_dim, spec.ffn_dim
    w = {k: (v.double().numpy() if hasattr(v, "double") else np.asarray(v, np.float64)) for k, v in lw.items()}

    def norm(a, g):
        return a / np.sqrt((a * a).mean(-1, keepdims=True) + eps) * g

    def rot(a):
        i = np.arange(D // 2)
        ang = np.arange(T)[:, None] * theta ** (-2.0 * i / D)[None, :]
        c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
        out = np.empty_like(a)
        out[..., 0::2] = a[..., 0::2] * c - a[..., 1::2] * s
        out[..., 1::2] = a[..., 0::2] * s + a[..., 1::2] * c
        return out

    n = norm(x, w["g_attn"])
    qkv = n @ w["wqkv"].T
    q = rot(qkv[:, :H * D].reshape(T, H, D))
    k = qkv[:, H * D:(H + Hkv) * D].reshape(T, Hkv, D)
    k = {"after": lambda: _bf16(rot(k)), "before": lambda: rot(_bf16(k)), "values_only": lambda: rot(k)}[where]()
    v = _bf16(qkv[:, (H + Hkv) * D:].reshape(T, Hkv, D))
    k, v = np.repeat(k, H // Hkv, axis=1), np.repeat(v, H // Hkv, axis=1)
    sc = np.einsum("thd,shd->hts", q, k) / math.sqrt(D)
    sc = np.where(np.tril(np.ones((T, T), bool))[None], sc, -np.inf)
    p = np.exp(sc - sc.max(-1, keepdims=True))
    p /= p.sum(-1, keepdims=True)
    att = np.einsum("hts,shd->thd", p, v).reshape(T, H * D)
    x = x + att @ w["wo"].T
    n = norm(x, w["g_ffn"])
    gu = n @ w["wgu"].T
    g, u = gu[:, :F], gu[:, F:]
    return x + (g / (1 + np.exp(-g)) * u) @ w["wd"].T


def test_bf16_cache_rounds_rotated_keys_and_values_where_they_enter_the_cache():
    # The whole layer with a bf16 cache against the dense formulation above, on 24 positions and a
    # grouped-query layer: keys are rounded after the rotation, values as projected, queries and all
    # arithmetic stay fp64.  The two plausible misplacements differ from the oracle by far more than
    # the agreement asked of the right one.
    spec = synth.TINY.with_(n_layers=1, n_early=1, n_kv_heads=2)
    lw = synth.layer_weights(spec, 0)
    emb, head = synth.embedding(spec), synth.lm_head(spec)
    m = oracle.model_from_weights(spec, [lw], lw, emb, head, max_ctx=32, kv_bf16=True)
    x0 = m.embed(synth.prompt_tokens(7, 24, spec.vocab).numpy()) * 30.0
    got = m.layer_fwd(0, 0, x0, 0)
    np.testing.assert_allclose(got, _dense_layer_bf16_cache(x0, lw, spec, "after"), rtol=0, atol=1e-10)
    for wrong in ("before", "values_only"):
        assert np.abs(got - _dense_layer_bf16_cache(x0, lw, spec, wrong)).max() > 1e-6
    # cached across calls the same values come back: 16 rows, then 8 single rows
    m2 = oracle.model_from_weights(spec, [lw], lw, emb, head, max_ctx=32, kv_bf16=True)
    parts = [m2.layer_fwd(0, 0, x0[:16], 0)] + [m2.layer_fwd(0, 0, x0[i:i + 1], i) for i in range(16, 24)]
    np.testing.assert_allclose(np.concatenate(parts), got, rtol=0, atol=1e-12)


def test_bf16_cache_two_position_hand_case_key_rounded_after_rotation():
    # D = 2, one head, two positions, hand numbers.  Raw key at position 1: (1 + 2^-8, 1).  bf16 keeps
    # 8 significant bits, so rounding BEFORE the rotation turns it into (1, 1) (tie to even); rotated
    # by 1 radian first it is (cos1 - sin1 - 2^-8 sin1 ..., ...) and rounds to other values.  The
    # score difference s_1 - s_0 of the row at position 1 is read off the layer output through
    # values (1, 0) and (0, 1): output - x = (w_0, w_1), w = softmax(s).
    import types
    D = 2
    c1, s1 = math.cos(1.0), math.sin(1.0)
    spec = types.SimpleNamespace(d_model=2, n_heads=1, n_kv_heads=1, head_dim=2, ffn_dim=2, vocab=2, n_early=1,
                                 rms_eps=0.0, rope_theta=10000.0, dtype="bf16")
    # rows of x are chosen so that RMSNorm (gain 1, eps 0) returns them: mean square 1
    x = np.array([[1.0, 1.0], [1.0, -1.0]])
    a, b = 1.0 + 2.0 ** -8, 1.0
    # n_0 = (1, 1), n_1 = (1, -1): solve Wk n_0 = (1, 0) (position 0 is not rotated), Wk n_1 = (a, b)
    wk = np.array([[(1 + a) / 2, (1 - a) / 2], [b / 2, -b / 2]])
    wv = np.array([[0.5, 0.5], [0.5, -0.5]])   # v_0 = (1, 0), v_1 = (0, 1): exact in bf16
    wq = np.array([[1.0, 0.0], [0.0, 1.0]])
    lw = dict(g_attn=np.ones(2, np.float32), g_ffn=np.ones(2, np.float32), wqkv=np.concatenate([wq, wk, wv]).astype(np.float32),
              wo=np.eye(2, dtype=np.float32), wgu=np.zeros((4, 2), np.float32), wd=np.zeros((2, 2), np.float32))
    assert (lw["wqkv"].astype(np.float64) == np.concatenate([wq, wk, wv])).all()   # the weights are exact in fp32
    emb = np.zeros((2, 2), np.float32)
    m = oracle.model_from_weights(spec, [lw], lw, emb, emb, max_ctx=4, kv_bf16=True)
    y = m.layer_fwd(0, 0, x, 0)
    w = y[1] - x[1]
    got = math.log(w[1] / w[0])                      # s_1 - s_0
    q1 = np.array([c1 + s1, s1 - c1])                # (1, -1) rotated by 1 radian
    k0 = np.array([1.0, 0.0])
    k1_after = _bf16(np.array([a * c1 - b * s1, a * s1 + b * c1]))
    k1_before = np.array([1.0 * c1 - 1.0 * s1, 1.0 * s1 + 1.0 * c1])   # bf16(a) = 1
    want = (q1 @ k1_after - q1 @ k0) / math.sqrt(D)
    wrong = (q1 @ k1_before - q1 @ k0) / math.sqrt(D)
    assert abs(want - wrong) > 1e-4                  # the case tells the two placements apart
    assert abs(got - want) < 1e-12
