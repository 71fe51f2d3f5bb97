"""ctypes wrapper around the C oracle (oracle/eesd_oracle.c) -- TEST INFRASTRUCTURE.

Only tests/, the smoke check and the benchmark's CPU-baseline leg import this package; the
CUDA library and its Python binding never do.  `build()` compiles the C file with gcc.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "eesd_oracle.c")
_LIB = os.path.join(_HERE, "libeesd_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class _Cfg(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("d", "H", "Hkv", "D", "F", "V", "L", "N", "max_ctx")] + \
               [("eps", C.c_double), ("theta", C.c_double), ("kv_bf16", C.c_int), ("E", C.c_int)]


class _GenCfg(C.Structure):
    _fields_ = [("max_new", C.c_int), ("k_cap", C.c_int), ("temperature", C.c_float),
                ("controller", C.c_int), ("fixed_k", C.c_int), ("alpha0", C.c_long), ("beta0", C.c_long),
                ("ts_rule", C.c_int), ("k_schedule", C.POINTER(C.c_int)), ("n_schedule", C.c_int),
                ("u_draft", C.POINTER(C.c_float)), ("u_accept", C.POINTER(C.c_float)),
                ("u_resample", C.POINTER(C.c_float)), ("u_ctrl", C.POINTER(C.c_float)), ("n_ctrl", C.c_long),
                ("cali_w", C.POINTER(C.c_float)), ("cali_wp", C.POINTER(C.c_float)),
                ("sigma_m", C.c_double), ("sigma_s", C.c_double), ("theta_hat0", C.c_double)]


class _Round(C.Structure):
    _fields_ = [("k", C.c_int), ("n_acc", C.c_int), ("y", C.c_int)]


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        L = _lib
        L.orc_model_new.restype = C.c_void_p
        L.orc_model_new.argtypes = [C.POINTER(_Cfg)]
        L.orc_model_free.argtypes = [C.c_void_p]
        L.orc_set_layer.argtypes = [C.c_void_p, C.c_int] + [C.c_void_p] * 7
        L.orc_set_globals.argtypes = [C.c_void_p] + [C.c_void_p] * 5
        L.orc_rmsnorm.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_double, C.c_void_p]
        L.orc_rope.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_double]
        L.orc_bf16_round.restype = C.c_double
        L.orc_bf16_round.argtypes = [C.c_double]
        L.orc_layer_fwd.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_int]
        L.orc_embed.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]
        L.orc_head.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_target_rows.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_draft_row.argtypes = [C.c_void_p, C.c_int32, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_exp_spec.restype = C.c_float
        L.orc_exp_spec.argtypes = [C.c_float]
        L.orc_softmax_spec.argtypes = [C.c_void_p, C.c_int, C.c_float, C.c_void_p]
        L.orc_sample_weights.restype = C.c_int
        L.orc_sample_weights.argtypes = [C.c_void_p, C.c_int, C.c_float]
        L.orc_argmax.restype = C.c_int
        L.orc_argmax.argtypes = [C.c_void_p, C.c_int]
        L.orc_sample_logits.restype = C.c_int
        L.orc_sample_logits.argtypes = [C.c_void_p, C.c_int, C.c_float, C.c_float]
        L.orc_accept_resample.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_float,
                                          C.c_int, C.c_int, C.c_float, C.POINTER(C.c_int), C.POINTER(C.c_int)]
        L.orc_accept_resample_batch.argtypes = [C.c_void_p] * 5 + [C.c_int, C.c_int, C.c_int, C.c_float,
                                                                  C.c_void_p, C.c_void_p]
        L.orc_ts_continue.restype = C.c_int
        L.orc_ts_continue.argtypes = [C.c_long, C.c_long, C.c_void_p, C.c_long, C.POINTER(C.c_long),
                                      C.POINTER(C.c_double)]
        L.orc_ts_update.argtypes = [C.POINTER(C.c_long), C.POINTER(C.c_long), C.c_int, C.c_int, C.c_int]
        L.orc_generate.restype = C.c_int
        L.orc_generate.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.POINTER(_GenCfg), C.c_void_p,
                                   C.c_void_p, C.c_int, C.POINTER(C.c_long), C.POINTER(C.c_long)]
    return _lib


def _f32(a) -> np.ndarray:
    """contiguous float32 numpy array from a numpy array or a torch tensor (any float dtype)."""
    if hasattr(a, "detach"):
        a = a.detach().float().cpu().numpy()
    return np.ascontiguousarray(a, dtype=np.float32)


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


# ----------------------------------------------------------------------------- free functions
def rmsnorm(x, g, eps: float) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64)
    g = _f32(g)
    out = np.empty_like(x)
    lib().orc_rmsnorm(_p(x), _p(g), x.shape[-1], eps, _p(out))
    return out


def rope(v, pos: int, theta: float) -> np.ndarray:
    v = np.array(v, dtype=np.float64, copy=True)
    lib().orc_rope(_p(v), v.shape[-1], pos, theta)
    return v


def exp_spec(t: float) -> float:
    return float(lib().orc_exp_spec(np.float32(t)))


def softmax_spec(logits, T: float = 1.0) -> np.ndarray:
    l = _f32(logits)
    out = np.empty_like(l)
    lib().orc_softmax_spec(_p(l), l.shape[-1], T, _p(out))
    return out


def sample_weights(w, u: float) -> int:
    w = _f32(w)
    return lib().orc_sample_weights(_p(w), w.shape[-1], np.float32(u))


def sample_logits(logits, T: float, u: float) -> int:
    l = _f32(logits)
    return lib().orc_sample_logits(_p(l), l.shape[-1], T, np.float32(u))


def accept_resample(p_logits, q_logits, x, u_acc, u_res: float, T: float):
    p, q = _f32(p_logits), _f32(q_logits)
    K, V = q.shape
    assert p.shape == (K + 1, V)
    x = np.ascontiguousarray(x, dtype=np.int32)
    ua = _f32(u_acc)
    n, y = C.c_int(), C.c_int()
    lib().orc_accept_resample(_p(p), _p(q), _p(x), _p(ua), np.float32(u_res), K, V, T, C.byref(n), C.byref(y))
    return n.value, y.value


def accept_resample_batch(p_logits, q_logits, x, u_acc, u_res, T: float):
    p, q = _f32(p_logits), _f32(q_logits)
    B, K, V = q.shape
    assert p.shape == (B, K + 1, V)
    x = np.ascontiguousarray(x, dtype=np.int32).reshape(B, K)
    ua, ur = _f32(u_acc).reshape(B, K), _f32(u_res).reshape(B)
    n, y = np.empty(B, np.int32), np.empty(B, np.int32)
    lib().orc_accept_resample_batch(_p(p), _p(q), _p(x), _p(ua), _p(ur), B, K, V, T, _p(n), _p(y))
    return n, y


def ts_continue(alpha: int, beta: int, u, cursor: int):
    """Returns (chi, theta, new_cursor)."""
    u = _f32(u)
    cur, th = C.c_long(cursor), C.c_double()
    chi = lib().orc_ts_continue(alpha, beta, _p(u), u.shape[0], C.byref(cur), C.byref(th))
    return chi, th.value, cur.value


def ts_update(alpha: int, beta: int, q_v: int, n_draft: int, rule: int = 0):
    a, b = C.c_long(alpha), C.c_long(beta)
    lib().orc_ts_update(C.byref(a), C.byref(b), q_v, n_draft, rule)
    return a.value, b.value


# Thompson sampling with calibration (Sec. 3.3, Eq. 5-8, Algorithm 3)
def cali_theta_m(Wi, Wp, hT, hD) -> float:
    Wi, Wp = _f32(Wi), _f32(Wp)
    hT, hD = np.ascontiguousarray(hT, np.float64), np.ascontiguousarray(hD, np.float64)
    d = hT.shape[0]
    assert Wi.shape == (d, d) and Wp.shape == (2, 2 * d) and hD.shape == (d,)
    f = lib().orc_cali_theta_m
    f.restype, f.argtypes = C.c_double, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int]
    return f(_p(Wi), _p(Wp), _p(hT), _p(hD), d)


def cali_posterior(theta_m: float, theta_hat: float, n: int, sigma_m: float, sigma_s: float):
    """Eq. 6-7: returns (mu, variance)."""
    mu, var = C.c_double(), C.c_double()
    f = lib().orc_cali_posterior
    f.argtypes = [C.c_double, C.c_double, C.c_long, C.c_double, C.c_double, C.POINTER(C.c_double), C.POINTER(C.c_double)]
    f(theta_m, theta_hat, n, sigma_m, sigma_s, C.byref(mu), C.byref(var))
    return mu.value, var.value


def cali_theta_hat(prev: float, trials_prev: int, r: int, n: int) -> float:
    f = lib().orc_cali_theta_hat
    f.restype, f.argtypes = C.c_double, [C.c_double, C.c_long, C.c_int, C.c_int]
    return f(prev, trials_prev, r, n)


def cali_continue(mu: float, var: float, u, cursor: int):
    """Returns (chi, theta, new_cursor)."""
    u = _f32(u)
    cur, th = C.c_long(cursor), C.c_double()
    f = lib().orc_cali_continue
    f.restype, f.argtypes = C.c_int, [C.c_double, C.c_double, C.c_void_p, C.c_long, C.POINTER(C.c_long), C.POINTER(C.c_double)]
    chi = f(mu, var, _p(u), u.shape[0], C.byref(cur), C.byref(th))
    return chi, th.value, cur.value


# ----------------------------------------------------------------------------- model
class OracleModel:
    """The target + draft model over fp32 copies of the given weights.

    layers: list of L dicts with g_attn, wqkv, wo, g_ffn, wgu ([2F, d], gate rows first), wd;
    exit_layer: one such dict, or a list of them (a draft model with several early-exit layers,
    stacked in that order).  Weights may be torch tensors of any float dtype: their values are
    widened to fp32 unchanged.
    """

    def __init__(self, *, d, H, Hkv, D, F, V, N, max_ctx, layers: Sequence[Dict], exit_layer: Dict,
                 embed, g_final, lm_head, g_exit, exit_head, eps=1e-5, theta=10000.0, kv_bf16=False):
        self.L = len(layers)
        exit_layers = list(exit_layer) if isinstance(exit_layer, (list, tuple)) else [exit_layer]
        self.E = len(exit_layers)
        self.cfg = _Cfg(d, H, Hkv, D, F, V, self.L, N, max_ctx, eps, theta, int(kv_bf16), self.E)
        self.d, self.V, self.F, self.N, self.max_ctx = d, V, F, N, max_ctx
        self._keep = []
        self.h = C.c_void_p(lib().orc_model_new(C.byref(self.cfg)))
        for i, lw in enumerate(list(layers) + exit_layers):
            wgu = _f32(lw["wgu"])
            arrs = [_f32(lw["g_attn"]), _f32(lw["wqkv"]), _f32(lw["wo"]), _f32(lw["g_ffn"]),
                    np.ascontiguousarray(wgu[:F]), np.ascontiguousarray(wgu[F:]), _f32(lw["wd"])]
            self._keep.append(arrs)
            lib().orc_set_layer(self.h, i, *[_p(a) for a in arrs])
        g = [_f32(embed), _f32(g_final), _f32(lm_head), _f32(g_exit), _f32(exit_head)]
        self._keep.append(g)
        lib().orc_set_globals(self.h, *[_p(a) for a in g])

    def __del__(self):
        try:
            lib().orc_model_free(self.h)
        except Exception:
            pass

    def embed(self, tokens) -> np.ndarray:
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        x = np.empty((len(t), self.d), np.float64)
        lib().orc_embed(self.h, _p(t), len(t), _p(x))
        return x

    def layer_fwd(self, lidx: int, slot: int, x: np.ndarray, pos0: int) -> np.ndarray:
        x = np.array(x, dtype=np.float64, copy=True)
        lib().orc_layer_fwd(self.h, lidx, slot, _p(x), x.shape[0], pos0)
        return x

    def head(self, x, exit_head: bool = False) -> np.ndarray:
        x = np.ascontiguousarray(x, dtype=np.float64)
        out = np.empty((x.shape[0], self.V), np.float32)
        g, w = (self._keep[-1][3], self._keep[-1][4]) if exit_head else (self._keep[-1][1], self._keep[-1][2])
        lib().orc_head(self.h, _p(x), x.shape[0], _p(g), _p(w), _p(out))
        return out

    def target_rows(self, tokens, pos0: int, want_hidden=False, want_logits=True):
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        M = len(t)
        hid = np.empty((self.L + 1, M, self.d), np.float64) if want_hidden else None
        lg = np.empty((M, self.V), np.float32) if want_logits else None
        lib().orc_target_rows(self.h, _p(t), M, pos0, _p(hid), _p(lg))
        return hid, lg

    def draft_row(self, token: int, pos: int, want_hidden=False):
        lg = np.empty(self.V, np.float32)
        hid = np.empty(self.d, np.float64) if want_hidden else None
        lib().orc_draft_row(self.h, int(token), pos, _p(lg), _p(hid))
        return (lg, hid) if want_hidden else lg

    def generate(self, prompt, max_new: int, *, k_cap=10, temperature=0.0, controller=0, fixed_k=4,
                 alpha0=1, beta0=1, ts_rule=0, k_schedule=None, uniforms=None, cali=None):
        """Algorithm 1.  Returns (tokens[max_new], trace[(k, n_acc, y)], (alpha, beta)).
        controller 2 (TS with calibration) takes cali = dict(w [10, d, d], wp [2, 2d], sigma_m,
        sigma_s, theta_hat0)."""
        prompt = np.ascontiguousarray(prompt, dtype=np.int32)
        g = _GenCfg()
        g.max_new, g.k_cap, g.temperature, g.controller, g.fixed_k = max_new, k_cap, temperature, controller, fixed_k
        g.alpha0, g.beta0, g.ts_rule = alpha0, beta0, ts_rule
        keep = []
        if k_schedule is not None:
            ks = np.ascontiguousarray(k_schedule, dtype=np.int32)
            keep.append(ks)
            g.k_schedule, g.n_schedule = ks.ctypes.data_as(C.POINTER(C.c_int)), len(ks)
        if uniforms is not None:
            for name in ("u_draft", "u_accept", "u_resample", "u_ctrl"):
                a = _f32(uniforms[name])
                keep.append(a)
                setattr(g, name, a.ctypes.data_as(C.POINTER(C.c_float)))
            g.n_ctrl = len(keep[-1])
        if cali is not None:
            cw, cp = _f32(cali["w"]), _f32(cali["wp"])
            assert cw.shape == (10, self.d, self.d) and cp.shape == (2, 2 * self.d)
            keep += [cw, cp]
            g.cali_w, g.cali_wp = cw.ctypes.data_as(C.POINTER(C.c_float)), cp.ctypes.data_as(C.POINTER(C.c_float))
            g.sigma_m, g.sigma_s, g.theta_hat0 = cali["sigma_m"], cali["sigma_s"], cali["theta_hat0"]
        out = np.empty(max_new, np.int32)
        cap = max_new + 1
        trace = (_Round * cap)()
        a, b = C.c_long(), C.c_long()
        n = lib().orc_generate(self.h, _p(prompt), len(prompt), C.byref(g), _p(out), trace, cap,
                               C.byref(a), C.byref(b))
        return out, [(trace[i].k, trace[i].n_acc, trace[i].y) for i in range(n)], (a.value, b.value)


    def generate_tree(self, prompt, max_new: int, *, width: int, fixed_k=4, k_schedule=None):
        """Greedy EESD with tree verification (the tree-attention appendix: several draft
        candidates per position, only the one equal to the target's top-1 token is kept).

        The paper fixes no tree shape.  Reading taken here: the draft model's greedy chain
        x_1..x_K, plus at every depth i the next `width - 1` best tokens of the same draft
        distribution as leaves (ranked by logit, lower token id first among equals).  The target's
        top-1 token after the accepted path so far is compared with the children at the next
        depth: the chain token continues the walk, a leaf ends it (the target's top-1 after the
        path ending in that leaf is the round's last token), neither ends it with the target's
        own token.  Each "top-1 after a path" is taken by its definition: the target run on that
        path.  Returns (tokens[max_new], trace[(k, n_acc, y)], leaves accepted); n_acc counts
        accepted draft tokens, an accepted leaf included."""
        ctx = [int(t) for t in prompt]
        if len(ctx) > 1:
            self.target_rows(np.array(ctx[:-1], np.int32), 0, want_logits=False)
        n0, trace, leaves, rounds = len(ctx), [], 0, 0
        while len(ctx) - n0 < max_new:
            T = len(ctx)
            K = int(k_schedule[rounds]) if k_schedule is not None and rounds < len(k_schedule) else fixed_k
            K = max(1, min(K, (self.max_ctx - T) // width))
            xs, sib = [ctx[-1]], []
            for i in range(K):
                lg = self.draft_row(xs[i], T - 1 + i)
                order = np.argsort(-lg.astype(np.float64), kind="stable")[:width]   # equal logits: lower id first
                xs.append(int(order[0]))
                sib.append([int(v) for v in order[1:]])
            _, pl = self.target_rows(np.array(xs, np.int32), T - 1)
            top = [int(row.argmax()) for row in pl]   # target's token after the chain prefix x_0..x_i
            accepted, y = xs[1:K + 1], top[K]
            for i in range(1, K + 1):
                want = top[i - 1]
                if want == xs[i]:
                    continue
                if want in sib[i - 1]:
                    # the path x_0..x_{i-1}, leaf: run the target on the leaf at its position (this
                    # also leaves the leaf's keys / values there, in every layer and the exit layer)
                    _, ps = self.target_rows(np.array([want], np.int32), T - 1 + i)
                    accepted, y = xs[1:i] + [want], int(ps[0].argmax())
                    leaves += 1
                else:
                    accepted, y = xs[1:i], want
                break
            ctx += accepted + [y]
            trace.append((K, len(accepted), y))
            rounds += 1
        return np.array(ctx[n0:n0 + max_new], np.int32), trace, leaves


def bf16_round(x: float) -> float:
    return float(lib().orc_bf16_round(float(x)))


def model_from_weights(spec_like, layers, exit_layer, embed, lm_head, exit_head=None, max_ctx=256,
                       g_final=None, g_exit=None, kv_bf16=None) -> OracleModel:
    """Convenience: build an OracleModel from shape fields (d_model, n_heads, ...) and weights."""
    s = spec_like
    ones = np.ones(s.d_model, np.float32)
    return OracleModel(d=s.d_model, H=s.n_heads, Hkv=s.n_kv_heads, D=s.head_dim, F=s.ffn_dim, V=s.vocab,
                       N=s.n_early, max_ctx=max_ctx, layers=layers, exit_layer=exit_layer, embed=embed,
                       g_final=ones if g_final is None else g_final, lm_head=lm_head,
                       g_exit=ones if g_exit is None else g_exit,
                       exit_head=lm_head if exit_head is None else exit_head,
                       eps=s.rms_eps, theta=s.rope_theta,
                       kv_bf16=(getattr(s, 'dtype', 'f32') == 'bf16') if kv_bf16 is None else kv_bf16)
