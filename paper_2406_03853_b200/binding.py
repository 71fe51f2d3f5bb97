"""ctypes binding of libeesd.so.  Argument marshalling only: every step of the decode round
runs in the library's CUDA kernels.  PyTorch provides device memory and the stream.

There is no CPU path: importing works without a GPU (so the symbols can be inspected), but
creating an Engine or calling a kernel entry point without CUDA raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Dict, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libeesd.so")
_lib = None

F32, BF16 = 0, 1
CTRL_FIXED_K, CTRL_BETA_TS, CTRL_CALI_TS = 0, 1, 2
MAX_ROWS = 16


class EesdError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        msg = lib().eesd_strerror(status).decode()
        super().__init__(f"{where}: {msg} ({status})" + (f" [{detail}]" if detail else ""))


class Config(C.Structure):
    _fields_ = [("d_model", C.c_int32), ("n_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("ffn_dim", C.c_int32), ("vocab", C.c_int32), ("n_layers", C.c_int32), ("n_early", C.c_int32),
                ("dtype", C.c_int32), ("tie_exit_head", C.c_int32), ("rms_eps", C.c_float), ("rope_theta", C.c_float),
                ("page_tokens", C.c_int32), ("max_ctx", C.c_int32), ("k_cap", C.c_int32), ("temperature", C.c_float),
                ("controller", C.c_int32), ("fixed_k", C.c_int32), ("alpha0", C.c_int32), ("beta0", C.c_int32),
                ("ts_update_rule", C.c_int32), ("cali_sigma_m", C.c_float), ("cali_sigma_s", C.c_float),
                ("cali_theta0", C.c_float), ("tree_width", C.c_int32), ("n_exit_layers", C.c_int32)]


class Layout(C.Structure):
    _fields_ = [(n, C.c_size_t) for n in
                ("embed", "layer0", "layer_stride", "off_g_attn", "off_wqkv", "off_wo", "off_g_ffn", "off_wgu",
                 "off_wd", "final_norm", "lm_head", "exit_layer", "exit_norm", "exit_head", "cali_w", "cali_wp",
                 "total_bytes", "tiled")]


class Sizes(C.Structure):
    _fields_ = [("weights_bytes", C.c_size_t), ("kv_page_bytes", C.c_size_t), ("min_pages", C.c_int64),
                ("workspace_bytes", C.c_size_t)]


class Buffers(C.Structure):
    _fields_ = [("weights", C.c_void_p), ("weights_bytes", C.c_size_t), ("kv_pool", C.c_void_p),
                ("kv_bytes", C.c_size_t), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t)]


class Uniforms(C.Structure):
    _fields_ = [("u_draft", C.c_void_p), ("u_accept", C.c_void_p), ("u_resample", C.c_void_p),
                ("u_ctrl", C.c_void_p), ("n_ctrl", C.c_int64)]


class Round(C.Structure):
    _fields_ = [("k", C.c_int32), ("n_accept", C.c_int32), ("next_token", C.c_int32)]


class Stats(C.Structure):
    _fields_ = [("rounds", C.c_int64), ("drafted", C.c_int64), ("accepted", C.c_int64), ("emitted", C.c_int64),
                ("ms_prefill", C.c_double), ("ms_draft", C.c_double), ("ms_verify", C.c_double),
                ("ms_total", C.c_double), ("kernel_launches", C.c_int64), ("alpha", C.c_int64), ("beta", C.c_int64),
                ("leaves_kept", C.c_int64), ("ms_sampling", C.c_double), ("ms_other", C.c_double)]

    def as_dict(self) -> Dict:
        return {n: getattr(self, n) for n, _ in self._fields_}


def lib_path() -> str:
    return _LIB_PATH


def lib():
    """Loads the CUDA library; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2406_03853_b200.build`")
        L = C.CDLL(_LIB_PATH)
        vp, i32p = C.c_void_p, C.POINTER(C.c_int32)
        L.eesd_strerror.restype = C.c_char_p
        L.eesd_strerror.argtypes = [C.c_int]
        L.eesd_last_cuda_error.restype = C.c_char_p
        L.eesd_last_cuda_error.argtypes = [vp]
        L.eesd_weight_layout.argtypes = [C.POINTER(Config), C.POINTER(Layout)]
        L.eesd_required_bytes.argtypes = [C.POINTER(Config), C.POINTER(Sizes)]
        L.eesd_init.argtypes = [C.POINTER(Config), C.POINTER(Buffers), vp, C.POINTER(vp)]
        L.eesd_destroy.argtypes = [vp]
        L.eesd_reset.argtypes = [vp]
        L.eesd_prefill.argtypes = [vp, vp, C.c_int]
        L.eesd_draft.argtypes = [vp, C.c_int, vp, vp]
        L.eesd_verify_accept.argtypes = [vp, vp, C.c_float, C.POINTER(C.c_int), i32p]
        L.eesd_generate.argtypes = [vp, vp, C.c_int, C.c_int, vp, C.c_int, C.POINTER(Uniforms), vp,
                                    C.POINTER(Stats), vp, C.c_int, C.POINTER(C.c_int)]
        L.eesd_decode.argtypes = [vp, C.c_int, vp, C.c_int, C.POINTER(Uniforms), vp, C.POINTER(Stats), vp, C.c_int,
                                  C.POINTER(C.c_int)]
        L.eesd_context_len.argtypes = [vp, C.POINTER(C.c_int), C.POINTER(C.c_int)]
        L.eesd_context_tokens.argtypes = [vp, C.c_int, C.c_int, vp]
        L.eesd_posterior.argtypes = [vp, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        L.eesd_cali_predict.argtypes = [vp, C.POINTER(C.c_float)]
        L.eesd_cali_state.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        L.eesd_cali_posterior.argtypes = [C.c_double, C.c_double, C.c_int64, C.c_double, C.c_double,
                                          C.POINTER(C.c_double), C.POINTER(C.c_double)]
        i64p, f64p = C.POINTER(C.c_int64), C.POINTER(C.c_double)
        L.eesd_ts_decide.argtypes = [C.c_int64, C.c_int64, vp, C.c_int64, i64p, f64p]
        L.eesd_ts_posterior_update.argtypes = [i64p, i64p, C.c_int, C.c_int, C.c_int]
        L.eesd_cali_decide.argtypes = [C.c_double, C.c_double, vp, C.c_int64, i64p, f64p]
        L.eesd_assume_context.argtypes = [vp, C.c_int, C.c_int32]
        L.eesd_verify_only.argtypes = [vp, vp, C.c_int]
        L.eesd_logits.argtypes = [vp, C.c_int, C.POINTER(vp)]
        L.eesd_batch_begin.argtypes = [vp, C.c_int]
        L.eesd_batch_prefill.argtypes = [vp, C.c_int, vp, C.c_int]
        L.eesd_batch_decode.argtypes = [vp, C.c_int, vp, C.c_int, vp, vp, C.POINTER(Stats), vp, C.c_int, vp]
        L.eesd_batch_context_len.argtypes = [vp, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int)]
        L.eesd_batch_verify_only.argtypes = [vp, vp, C.c_int]
        L.eesd_batch_assume_context.argtypes = [vp, C.c_int, C.c_int, C.c_int32]
        L.eesd_capture_hidden.argtypes = [vp, vp, C.c_size_t]
        L.eesd_launch_count.argtypes = [vp, C.POINTER(C.c_int64)]
        L.eesd_set_wait_limit.argtypes = [vp, C.c_uint32]
        L.eesd_clear_device_error.argtypes = [vp]
        L.eesd_attention_plan.argtypes = [C.c_int] * 6 + [C.POINTER(C.c_int), C.POINTER(C.c_int)]
        L.eesd_accept_scratch_bytes.restype = C.c_size_t
        L.eesd_accept_scratch_bytes.argtypes = [C.c_int, C.c_int]
        L.eesd_accept_resample.argtypes = [vp, vp, vp, vp, vp, vp, C.c_int, C.c_int, C.c_int, C.c_float, vp,
                                           C.c_size_t, vp, vp]
        L.eesd_project_scratch_bytes.restype = C.c_size_t
        L.eesd_project_scratch_bytes.argtypes = [C.c_int, C.c_int]
        L.eesd_project_rows.argtypes = [vp, C.c_int, vp, vp, vp, C.c_int, C.c_int, C.c_int, vp, C.c_size_t]
        L.eesd_time_projection.argtypes = [vp, C.c_int, C.c_int, C.POINTER(C.c_float), C.POINTER(C.c_size_t)]
        L.eesd_accept_resample_static.argtypes = [vp, vp, vp, vp, vp, vp, C.c_int, C.c_int, C.c_int, C.c_float, vp, vp]
        L.eesd_sample_rows.argtypes = [vp, vp, vp, C.c_int, C.c_int, C.c_float, vp]
        _lib = L
    return _lib


def _need_cuda():
    if not torch.cuda.is_available():
        raise RuntimeError("the EESD library needs a CUDA device (B200); there is no CPU path")


def _stream_ptr() -> int:
    return torch.cuda.current_stream().cuda_stream


def _np_i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _np_f32(a) -> np.ndarray:
    if hasattr(a, "detach"):
        a = a.detach().cpu().numpy()
    return np.ascontiguousarray(a, dtype=np.float32)


def make_config(*, d_model, n_heads, n_kv_heads, head_dim, ffn_dim, vocab, n_layers, n_early, dtype,
                tie_exit_head=False, rms_eps=1e-5, rope_theta=10000.0, page_tokens=16, max_ctx=2048, k_cap=10,
                temperature=0.0, controller=CTRL_FIXED_K, fixed_k=4, alpha0=1, beta0=1, ts_update_rule=0,
                cali_sigma_m=0.2, cali_sigma_s=0.5, cali_theta0=0.5, tree_width=0, n_exit_layers=1) -> Config:
    dt = {"f32": F32, "bf16": BF16}.get(dtype, dtype)
    return Config(d_model, n_heads, n_kv_heads, head_dim, ffn_dim, vocab, n_layers, n_early, dt, int(tie_exit_head),
                  rms_eps, rope_theta, page_tokens, max_ctx, k_cap, temperature, controller, fixed_k, alpha0, beta0,
                  ts_update_rule, cali_sigma_m, cali_sigma_s, cali_theta0, tree_width, n_exit_layers)


class TiledMatrix:
    """A weight matrix [R, K] (or a stack [n, R, K]) stored tile-major in the weight buffer:
    [R/128][K/64] tiles of [128][64] elements (eesd_layout.tiled).  `copy_` takes the matrix in
    its usual [.., R, K] form and places every element in its tile; `dense()` reads it back."""

    def __init__(self, flat: torch.Tensor, shape: Sequence[int]):
        *lead, R, K = shape
        assert R % 128 == 0 and K % 64 == 0
        self.shape = tuple(shape)
        n = len(lead)
        # storage order [.., R/128, K/64, 128, 64]; seen as [.., R/128, 128, K/64, 64]
        self._v = flat.view(*lead, R // 128, K // 64, 128, 64).permute(*range(n), n, n + 2, n + 1, n + 3)

    def copy_(self, t: torch.Tensor):
        self._v.copy_(t.reshape(self._v.shape))
        return self

    def dense(self) -> torch.Tensor:
        return self._v.reshape(self.shape)


class Engine:
    """One EESD context over torch-allocated device buffers (eesd_init .. eesd_destroy)."""

    def __init__(self, cfg: Config, kv_pages: Optional[int] = None, device="cuda:0"):
        _need_cuda()
        self.cfg = cfg
        self.device = torch.device(device)
        L = lib()
        self.layout, self.sizes = Layout(), Sizes()
        self._check(L.eesd_weight_layout(C.byref(cfg), C.byref(self.layout)), "eesd_weight_layout")
        self._check(L.eesd_required_bytes(C.byref(cfg), C.byref(self.sizes)), "eesd_required_bytes")
        pages = int(self.sizes.min_pages + 2 if kv_pages is None else kv_pages)
        self.wdtype = torch.float32 if cfg.dtype == F32 else torch.bfloat16
        with torch.cuda.device(self.device):
            self.weights = torch.zeros(self.sizes.weights_bytes, dtype=torch.uint8, device=self.device)
            self.kv_pool = torch.zeros(pages * self.sizes.kv_page_bytes, dtype=torch.uint8, device=self.device)
            self.workspace = torch.zeros(self.sizes.workspace_bytes, dtype=torch.uint8, device=self.device)
            torch.cuda.synchronize(self.device)
            b = Buffers(self.weights.data_ptr(), self.weights.numel(), self.kv_pool.data_ptr(), self.kv_pool.numel(),
                        self.workspace.data_ptr(), self.workspace.numel())
            self.h = C.c_void_p()
            self._check(L.eesd_init(C.byref(cfg), C.byref(b), _stream_ptr(), C.byref(self.h)), "eesd_init")
        self._capture = None

    # ---- plumbing
    def _check(self, st: int, where: str):
        if st != 0:
            detail = ""
            if getattr(self, "h", None):
                detail = lib().eesd_last_cuda_error(self.h).decode()
            raise EesdError(st, where, detail)

    def close(self):
        if getattr(self, "h", None):
            lib().eesd_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- weights (views into the caller-owned weight buffer)
    def _view(self, off: int, shape: Sequence[int], dtype) -> torch.Tensor:
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        return self.weights[off:off + n].view(dtype).view(*shape)

    def _matrix(self, off: int, shape: Sequence[int]):
        """A projection matrix of the weight buffer: a plain tensor view when the layout is
        row-major, a TiledMatrix (same `copy_`) when it is tile-major."""
        if not self.layout.tiled:
            return self._view(off, shape, self.wdtype)
        n = int(np.prod(shape)) * torch.empty((), dtype=self.wdtype).element_size()
        return TiledMatrix(self.weights[off:off + n].view(self.wdtype), shape)

    def layer_views(self, l: int) -> Dict[str, torch.Tensor]:
        """Tensors aliasing target layer l (l >= n_layers: early-exit layer l - n_layers)."""
        c, lay = self.cfg, self.layout
        base = lay.exit_layer + (l - c.n_layers) * lay.layer_stride if l >= c.n_layers else lay.layer0 + l * lay.layer_stride
        qd, kvd = c.n_heads * c.head_dim, c.n_kv_heads * c.head_dim
        return {
            "g_attn": self._view(base + lay.off_g_attn, (c.d_model,), torch.float32),
            "wqkv": self._matrix(base + lay.off_wqkv, (qd + 2 * kvd, c.d_model)),
            "wo": self._matrix(base + lay.off_wo, (c.d_model, qd)),
            "g_ffn": self._view(base + lay.off_g_ffn, (c.d_model,), torch.float32),
            "wgu": self._matrix(base + lay.off_wgu, (2 * c.ffn_dim, c.d_model)),
            "wd": self._matrix(base + lay.off_wd, (c.d_model, c.ffn_dim)),
        }

    def global_views(self) -> Dict[str, torch.Tensor]:
        c, lay = self.cfg, self.layout
        v = {
            "embed": self._view(lay.embed, (c.vocab, c.d_model), self.wdtype),
            "g_final": self._view(lay.final_norm, (c.d_model,), torch.float32),
            "lm_head": self._matrix(lay.lm_head, (c.vocab, c.d_model)),
            "g_exit": self._view(lay.exit_norm, (c.d_model,), torch.float32),
            "exit_head": self._matrix(lay.exit_head, (c.vocab, c.d_model)),
        }
        if c.controller == CTRL_CALI_TS:   # predictor of the calibrated controller: W^1..W^10 and W_p
            v["cali_w"] = self._matrix(lay.cali_w, (10, c.d_model, c.d_model))
            v["cali_wp"] = self._view(lay.cali_wp, (2, 2 * c.d_model), torch.float32)
        return v

    # ---- Thompson sampling with calibration
    def cali_predict(self) -> float:
        th = C.c_float()
        self._check(lib().eesd_cali_predict(self.h, C.byref(th)), "eesd_cali_predict")
        return th.value

    def cali_state(self):
        th, n, tr = C.c_double(), C.c_int64(), C.c_int64()
        self._check(lib().eesd_cali_state(self.h, C.byref(th), C.byref(n), C.byref(tr)), "eesd_cali_state")
        return th.value, n.value, tr.value

    # ---- the five calls
    def reset(self):
        self._check(lib().eesd_reset(self.h), "eesd_reset")

    def prefill(self, prompt):
        p = _np_i32(prompt)
        self._check(lib().eesd_prefill(self.h, p.ctypes.data, len(p)), "eesd_prefill")

    def draft(self, k: int, u_draft=None) -> np.ndarray:
        out = np.empty(k, np.int32)
        u = None if u_draft is None else _np_f32(u_draft)
        self._check(lib().eesd_draft(self.h, k, None if u is None else u.ctypes.data, out.ctypes.data), "eesd_draft")
        return out

    def verify_accept(self, u_accept=None, u_resample: float = 0.0):
        u = None if u_accept is None else _np_f32(u_accept)
        n, y = C.c_int(), C.c_int32()
        self._check(lib().eesd_verify_accept(self.h, None if u is None else u.ctypes.data, float(u_resample),
                                             C.byref(n), C.byref(y)), "eesd_verify_accept")
        return n.value, y.value

    def _uniforms(self, uniforms: Optional[Dict]):
        if uniforms is None:
            return None, []
        U, keep = Uniforms(), []
        for name in ("u_draft", "u_accept", "u_resample", "u_ctrl"):
            a = _np_f32(uniforms[name])
            keep.append(a)
            setattr(U, name, a.ctypes.data)
        U.n_ctrl = len(keep[-1])
        for a in keep[:3]:
            if len(a) < self.cfg.max_ctx:
                raise ValueError("position-indexed uniform streams need max_ctx entries")
        return U, keep

    def generate(self, prompt, max_new: int, k_schedule=None, uniforms: Optional[Dict] = None):
        """eesd_generate.  Returns (tokens[max_new], trace[(k, n_accept, next_token)], Stats)."""
        p = _np_i32(prompt)
        out = np.empty(max_new, np.int32)
        ks = None if k_schedule is None else _np_i32(k_schedule)
        U, keep = self._uniforms(uniforms)
        cap = max_new + 1
        trace = (Round * cap)()
        st, nr = Stats(), C.c_int()
        self._check(lib().eesd_generate(self.h, p.ctypes.data, len(p), max_new,
                                        None if ks is None else ks.ctypes.data, 0 if ks is None else len(ks),
                                        None if U is None else C.byref(U), out.ctypes.data, C.byref(st),
                                        C.cast(trace, C.c_void_p), cap, C.byref(nr)), "eesd_generate")
        return out, [(trace[i].k, trace[i].n_accept, trace[i].next_token) for i in range(nr.value)], st

    def decode(self, max_new: int, k_schedule=None, uniforms: Optional[Dict] = None):
        """eesd_decode: the decode loop from the current context (no prefill)."""
        out = np.empty(max_new, np.int32)
        ks = None if k_schedule is None else _np_i32(k_schedule)
        U, keep = self._uniforms(uniforms)
        cap = max_new + 1
        trace = (Round * cap)()
        st, nr = Stats(), C.c_int()
        self._check(lib().eesd_decode(self.h, max_new, None if ks is None else ks.ctypes.data,
                                      0 if ks is None else len(ks), None if U is None else C.byref(U),
                                      out.ctypes.data, C.byref(st), C.cast(trace, C.c_void_p), cap, C.byref(nr)),
                    "eesd_decode")
        return out, [(trace[i].k, trace[i].n_accept, trace[i].next_token) for i in range(nr.value)], st

    # ---- additions
    def context_len(self):
        n, p = C.c_int(), C.c_int()
        self._check(lib().eesd_context_len(self.h, C.byref(n), C.byref(p)), "eesd_context_len")
        return n.value, p.value

    def context_tokens(self, first: int = 0, n: Optional[int] = None) -> np.ndarray:
        if n is None:
            n = self.context_len()[0] - first
        out = np.empty(n, np.int32)
        self._check(lib().eesd_context_tokens(self.h, first, n, out.ctypes.data), "eesd_context_tokens")
        return out

    def posterior(self):
        a, b = C.c_int64(), C.c_int64()
        self._check(lib().eesd_posterior(self.h, C.byref(a), C.byref(b)), "eesd_posterior")
        return a.value, b.value

    def assume_context(self, n_ctx: int, pending: int = 0):
        self._check(lib().eesd_assume_context(self.h, n_ctx, pending), "eesd_assume_context")

    def verify_only(self, tokens):
        t = _np_i32(tokens)
        self._check(lib().eesd_verify_only(self.h, t.ctypes.data, len(t)), "eesd_verify_only")

    # ---- batch mode: several sequences decoded together
    def batch_begin(self, n_seq: int):
        """eesd_batch_begin: n_seq empty sequences (0 leaves batch mode)."""
        self._check(lib().eesd_batch_begin(self.h, n_seq), "eesd_batch_begin")
        self._n_seq = n_seq

    def batch_prefill(self, seq: int, prompt):
        p = _np_i32(prompt)
        self._check(lib().eesd_batch_prefill(self.h, seq, p.ctypes.data, len(p)), "eesd_batch_prefill")

    def batch_context_len(self, seq: int):
        n, p = C.c_int(), C.c_int()
        self._check(lib().eesd_batch_context_len(self.h, seq, C.byref(n), C.byref(p)), "eesd_batch_context_len")
        return n.value, p.value

    def batch_assume_context(self, seq: int, n_ctx: int, pending: int = 0):
        self._check(lib().eesd_batch_assume_context(self.h, seq, n_ctx, pending), "eesd_batch_assume_context")

    def batch_verify_only(self, tokens):
        """tokens: [n_seq, m] rows per sequence; logits of row b * m + i are row b * m + i of logits(0, n_seq * m)."""
        t = np.ascontiguousarray(np.asarray(tokens, np.int32))
        self._check(lib().eesd_batch_verify_only(self.h, t.ctypes.data, t.shape[1]), "eesd_batch_verify_only")

    def batch_decode(self, max_new: int, k_schedule=None, uniforms=None):
        """eesd_batch_decode.  uniforms: one dict per sequence (or None when greedy).  Returns
        (tokens[n_seq, max_new], per-sequence traces [(k, n_accept, next_token)], Stats)."""
        B = self._n_seq
        out = np.empty((B, max_new), np.int32)
        ks = None if k_schedule is None else _np_i32(k_schedule)
        keep, U = [], None
        if uniforms is not None:
            U = (Uniforms * B)()
            for b in range(B):
                Ub, kb = self._uniforms(uniforms[b])
                keep.append(kb)
                U[b] = Ub
        cap = max_new + 1
        trace = (Round * (cap * B))()
        st, nr = Stats(), (C.c_int * B)()
        self._check(lib().eesd_batch_decode(self.h, max_new, None if ks is None else ks.ctypes.data, 0 if ks is None else len(ks),
                                            None if U is None else C.cast(U, C.c_void_p), out.ctypes.data, C.byref(st),
                                            C.cast(trace, C.c_void_p), cap, C.cast(nr, C.c_void_p)), "eesd_batch_decode")
        traces = [[(trace[b * cap + i].k, trace[b * cap + i].n_accept, trace[b * cap + i].next_token) for i in range(nr[b])]
                  for b in range(B)]
        return out, traces, st

    def logits(self, which: int, rows: int) -> torch.Tensor:
        """fp32 [rows, V] tensor aliasing the context's logits (0: verify pass, 1: draft steps)."""
        ptr = C.c_void_p()
        self._check(lib().eesd_logits(self.h, which, C.byref(ptr)), "eesd_logits")
        off = ptr.value - self.workspace.data_ptr()
        n = rows * self.cfg.vocab * 4
        return self.workspace[off:off + n].view(torch.float32).view(rows, self.cfg.vocab)

    def capture_hidden(self, on: bool = True) -> Optional[torch.Tensor]:
        """[(L+2), MAX_ROWS, d] fp32 tensor the passes write the residual stream into."""
        if on:
            self._capture = torch.zeros(self.cfg.n_layers + 2, MAX_ROWS, self.cfg.d_model, dtype=torch.float32,
                                        device=self.device)
            self._check(lib().eesd_capture_hidden(self.h, self._capture.data_ptr(), self._capture.numel() * 4),
                        "eesd_capture_hidden")
        else:
            self._check(lib().eesd_capture_hidden(self.h, None, 0), "eesd_capture_hidden")
            self._capture = None
        return self._capture

    def time_projection(self, which: int, M: int):
        """(ms per launch, weight bytes per launch) of projection kind `which` over all layers."""
        ms, nb = C.c_float(), C.c_size_t()
        self._check(lib().eesd_time_projection(self.h, which, M, C.byref(ms), C.byref(nb)), "eesd_time_projection")
        return ms.value, nb.value

    def set_wait_limit(self, polls: Optional[int]):
        """eesd_set_wait_limit; None restores the default bound."""
        self._check(lib().eesd_set_wait_limit(self.h, 0xffffffff if polls is None else polls), "eesd_set_wait_limit")

    def clear_device_error(self):
        self._check(lib().eesd_clear_device_error(self.h), "eesd_clear_device_error")

    def launch_count(self) -> int:
        n = C.c_int64()
        self._check(lib().eesd_launch_count(self.h, C.byref(n)), "eesd_launch_count")
        return n.value


def accept_resample(p_logits: torch.Tensor, q_logits: torch.Tensor, tokens: torch.Tensor, u_accept: torch.Tensor,
                    u_resample: torch.Tensor, temperature: float, scratch: Optional[torch.Tensor] = None):
    """eesd_accept_resample on device tensors; returns (n_accept [B], next_token [B]) int32 tensors."""
    _need_cuda()
    B, K, V = q_logits.shape
    assert p_logits.shape == (B, K + 1, V) and p_logits.is_cuda and p_logits.dtype == torch.float32
    assert p_logits.is_contiguous() and q_logits.is_contiguous() and tokens.is_contiguous()
    need = lib().eesd_accept_scratch_bytes(B, K)
    if scratch is None:
        scratch = torch.empty(need, dtype=torch.uint8, device=p_logits.device)
    n = torch.empty(B, dtype=torch.int32, device=p_logits.device)
    y = torch.empty(B, dtype=torch.int32, device=p_logits.device)
    st = lib().eesd_accept_resample(_stream_ptr(), p_logits.data_ptr(), q_logits.data_ptr(), tokens.data_ptr(),
                                    u_accept.data_ptr(), u_resample.data_ptr(), B, K, V, temperature,
                                    scratch.data_ptr(), scratch.numel(), n.data_ptr(), y.data_ptr())
    if st:
        raise EesdError(st, "eesd_accept_resample")
    return n, y


def cali_posterior(theta_m: float, theta_hat: float, n: int, sigma_m: float, sigma_s: float):
    """eesd_cali_posterior (Eq. 6-7, host arithmetic): returns (mu, variance)."""
    mu, var = C.c_double(), C.c_double()
    st = lib().eesd_cali_posterior(C.c_double(theta_m), C.c_double(theta_hat), C.c_int64(n), C.c_double(sigma_m),
                                   C.c_double(sigma_s), C.byref(mu), C.byref(var))
    if st:
        raise EesdError(st, "eesd_cali_posterior")
    return mu.value, var.value


def ts_decide(alpha: int, beta: int, u, cursor: int = 0):
    """eesd_ts_decide (host arithmetic): returns (chi, theta, new cursor)."""
    u = _np_f32(u)
    cur, th = C.c_int64(cursor), C.c_double()
    chi = lib().eesd_ts_decide(alpha, beta, u.ctypes.data_as(C.c_void_p), len(u), C.byref(cur), C.byref(th))
    if chi < 0:
        raise EesdError(chi, "eesd_ts_decide")
    return chi, th.value, cur.value


def ts_posterior_update(alpha: int, beta: int, q_v: int, n_draft: int, rule: int = 0):
    """eesd_ts_posterior_update (host arithmetic, Eq. 3-4): returns the new (alpha, beta)."""
    a, b = C.c_int64(alpha), C.c_int64(beta)
    st = lib().eesd_ts_posterior_update(C.byref(a), C.byref(b), q_v, n_draft, rule)
    if st:
        raise EesdError(st, "eesd_ts_posterior_update")
    return a.value, b.value


def cali_decide(mu: float, variance: float, u, cursor: int = 0):
    """eesd_cali_decide (host arithmetic): returns (chi, theta, new cursor)."""
    u = _np_f32(u)
    cur, th = C.c_int64(cursor), C.c_double()
    chi = lib().eesd_cali_decide(C.c_double(mu), C.c_double(variance), u.ctypes.data_as(C.c_void_p), len(u),
                                 C.byref(cur), C.byref(th))
    if chi < 0:
        raise EesdError(chi, "eesd_cali_decide")
    return chi, th.value, cur.value


def attention_plan(dtype: int, ctx_len: int, page_tokens: int, n_kv_heads: int, pairs: int, n_sm: int = 148):
    """eesd_attention_plan (host arithmetic): returns (pages per block, slices per KV head)."""
    pps, ns = C.c_int(), C.c_int()
    st = lib().eesd_attention_plan(dtype, ctx_len, page_tokens, n_kv_heads, pairs, n_sm, C.byref(pps), C.byref(ns))
    if st:
        raise EesdError(st, "eesd_attention_plan")
    return pps.value, ns.value


def sample_rows(logits: torch.Tensor, u: Optional[torch.Tensor], temperature: float) -> torch.Tensor:
    _need_cuda()
    B, V = logits.shape
    assert logits.is_cuda and logits.dtype == torch.float32 and logits.is_contiguous()
    out = torch.empty(B, dtype=torch.int32, device=logits.device)
    st = lib().eesd_sample_rows(_stream_ptr(), logits.data_ptr(), None if u is None else u.data_ptr(), B, V,
                                temperature, out.data_ptr())
    if st:
        raise EesdError(st, "eesd_sample_rows")
    return out


def project_rows(A: torch.Tensor, W: torch.Tensor, scratch: Optional[torch.Tensor] = None) -> torch.Tensor:
    """eesd_project_rows: A [M, K] fp32 times W [R, K]^T (fp32 or bf16) -> [M, R] fp32."""
    _need_cuda()
    M, K = A.shape
    R = W.shape[0]
    assert W.shape[1] == K and A.dtype == torch.float32 and A.is_contiguous() and W.is_contiguous() and A.is_cuda
    dt = F32 if W.dtype == torch.float32 else BF16
    need = lib().eesd_project_scratch_bytes(R, K)
    if scratch is None:
        scratch = torch.empty(need, dtype=torch.uint8, device=A.device)
    out = torch.empty(M, R, dtype=torch.float32, device=A.device)
    st = lib().eesd_project_rows(_stream_ptr(), dt, A.data_ptr(), W.data_ptr(), out.data_ptr(), M, R, K,
                                 scratch.data_ptr(), scratch.numel())
    if st:
        raise EesdError(st, "eesd_project_rows")
    return out
