"""Shared test helpers: build the CPU oracle's model from a synthetic-model spec."""
import numpy as np

import eesd_synth as synth
import oracle


def oracle_from_spec(spec, max_ctx=256, n_layers=None, device="cpu", seed=synth.SEED, kv_bf16=None, n_exit=1):
    """Oracle model with the synthetic weights of `spec` (optionally only the first n_layers;
    the exit layers are then still the copies of the spec's last layers)."""
    L = spec.n_layers if n_layers is None else n_layers
    layers = [{k: v.cpu() for k, v in synth.layer_weights(spec, l, seed, device).items()} for l in range(L)]
    ex = [{k: v.cpu() for k, v in synth.exit_layer_weights(spec, seed, device, e, n_exit).items()} for e in range(n_exit)]
    emb = synth.embedding(spec, seed, device).cpu()
    head = synth.lm_head(spec, seed, device).cpu()
    s = spec.with_(n_layers=L, n_early=min(spec.n_early, L))
    return oracle.model_from_weights(s, layers, ex, emb, head, max_ctx=max_ctx, kv_bf16=kv_bf16)


def np_softmax(x):
    x = np.asarray(x, np.float64)
    e = np.exp(x - x.max(-1, keepdims=True))
    return e / e.sum(-1, keepdims=True)


# ------------------------------------------------------------------ CUDA engine from a spec
def config_from_spec(spec, n_layers=None, **kw):
    from paper_2406_03853_b200 import binding as b
    L = spec.n_layers if n_layers is None else n_layers
    return b.make_config(d_model=spec.d_model, n_heads=spec.n_heads, n_kv_heads=spec.n_kv_heads,
                         head_dim=spec.head_dim, ffn_dim=spec.ffn_dim, vocab=spec.vocab, n_layers=L,
                         n_early=min(spec.n_early, L), dtype=spec.dtype, tie_exit_head=spec.tie_exit_head,
                         rms_eps=spec.rms_eps, rope_theta=spec.rope_theta, **kw)


def fill_engine(engine, spec, seed=synth.SEED):
    """Writes the synthetic weights of `spec` into the engine's weight buffer (generated on
    the engine's device by the shared generator, so the oracle sees the same bits)."""
    dev = engine.device
    L = engine.cfg.n_layers
    for l in range(L):
        views = engine.layer_views(l)
        for k, v in synth.layer_weights(spec, l, seed, dev).items():
            views[k].copy_(v)
    E = max(1, engine.cfg.n_exit_layers)
    for e in range(E):
        views = engine.layer_views(L + e)
        for k, v in synth.exit_layer_weights(spec, seed, dev, e, E).items():
            views[k].copy_(v)
    g = engine.global_views()
    g["embed"].copy_(synth.embedding(spec, seed, dev))
    head = synth.lm_head(spec, seed, dev)
    g["lm_head"].copy_(head)
    if not engine.cfg.tie_exit_head:
        g["exit_head"].copy_(head)
    g["g_final"].fill_(1.0)
    g["g_exit"].fill_(1.0)


def engine_from_spec(spec, n_layers=None, seed=synth.SEED, kv_pages=None, **kw):
    from paper_2406_03853_b200 import Engine
    eng = Engine(config_from_spec(spec, n_layers, **kw), kv_pages=kv_pages)
    fill_engine(eng, spec, seed)
    return eng
