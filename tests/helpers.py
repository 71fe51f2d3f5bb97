"""Shared test helpers: build the CPU oracle's model from a synthetic-model spec."""
import numpy as np

import eesd_synth as synth
import oracle


def oracle_from_spec(spec, max_ctx=256, n_layers=None, device="cpu", seed=synth.SEED):
    """Oracle model with the synthetic weights of `spec` (optionally only the first n_layers;
    the exit layer is then still the copy of the spec's last layer)."""
    L = spec.n_layers if n_layers is None else n_layers
    layers = [{k: v.cpu() for k, v in synth.layer_weights(spec, l, seed, device).items()} for l in range(L)]
    ex = {k: v.cpu() for k, v in synth.exit_layer_weights(spec, seed, device).items()}
    emb = synth.embedding(spec, seed, device).cpu()
    head = synth.lm_head(spec, seed, device).cpu()
    s = spec.with_(n_layers=L)
    return oracle.model_from_weights(s, layers, ex, emb, head, max_ctx=max_ctx)


def np_softmax(x):
    x = np.asarray(x, np.float64)
    e = np.exp(x - x.max(-1, keepdims=True))
    return e / e.sum(-1, keepdims=True)
