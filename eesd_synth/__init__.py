"""Seeded synthetic inputs for EESD decode rounds (weights, prompts, uniforms, logits).

Everything here is a pure function of (seed, stream id, element index), built from a
counter-based 64-bit mixing hash evaluated with wrap-around int64 tensor arithmetic, so the
same call yields the same bits on a CPU tensor and on a CUDA tensor.  The module holds input
recipes only: model shapes, which tensors exist, how they are scaled.  None of the method's
arithmetic (norms, projections, attention, softmax, acceptance, controller) lives here; it
is the one module both the CPU oracle's tests and the CUDA path's tests/bench may import.

Recipes (stand-ins for LLaMA-2 checkpoints and the 1-shot benchmark prompts the paper
evaluates on, Sec. 4.1, which are not redistributable / not available offline):

* weights  w = s * 0.02 * z,  z ~ approx N(0,1): centred sum of four 16-bit hash fields
  (Irwin-Hall, n = 4) times 1/sigma; s = 1 except the residual-writing matrices (attention
  output projection and FFN down projection) of the "damped" upper layers, s = damp.
* the early-exit layer is a copy of the last target layer and the exit head a copy of the
  target LM head (the paper's initialisation, Sec. 3.1), the exit norm a copy of the final
  norm; norm gains are 1.
* prompts  tok = hash mod V; uniforms u = (hash >> 40) * 2^-24 in [0, 1).
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional

import torch

SEED = 20240603

# stream ids for the position-indexed uniform streams
STREAM_DRAFT = 1
STREAM_ACCEPT = 2
STREAM_RESAMPLE = 3
STREAM_CTRL = 4
STREAM_PROMPT = 5
STREAM_LOGITS = 6

# tensor kinds inside one decoder layer (tensor_id = layer * 16 + kind)
KIND_WQKV, KIND_WO, KIND_WG, KIND_WU, KIND_WD = 0, 1, 2, 3, 4
TID_EMBED = 1 << 20
TID_LM_HEAD = (1 << 20) + 1

_M1 = -7046029254386353131  # 0x9E3779B97F4A7C15 as int64
_M2 = -4658895280553007687  # 0xBF58476D1CE4E5B9
_M3 = -7723592293110705685  # 0x94D049BB133111EB
_IH_SIGMA_INV = 1.0 / (65536.0 * (1.0 / 3.0) ** 0.5)  # 1/std of a sum of four U{0..65535}


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of an int64 tensor holding uint64 bit patterns."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def mix64(x: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser (Steele, Lea, Flood 2014) on int64 bit patterns."""
    x = x + _M1
    x = (x ^ _lsr(x, 30)) * _M2
    x = (x ^ _lsr(x, 27)) * _M3
    return x ^ _lsr(x, 31)


def _key(seed: int, stream: int) -> int:
    k = (seed * 0x9E3779B97F4A7C15 + stream * 0xD1B54A32D192ED03 + 0x2545F4914F6CDD1D) & (2**64 - 1)
    # one scalar splitmix round in Python integers
    k = (k ^ (k >> 30)) * 0xBF58476D1CE4E5B9 & (2**64 - 1)
    k = (k ^ (k >> 27)) * 0x94D049BB133111EB & (2**64 - 1)
    k ^= k >> 31
    return k - 2**64 if k >= 2**63 else k


def hash_u64(seed: int, stream: int, start: int, n: int, device="cpu") -> torch.Tensor:
    """int64 tensor [n] of hash bits for counters start..start+n-1 of (seed, stream)."""
    idx = torch.arange(start, start + n, dtype=torch.int64, device=device)
    return mix64(idx ^ _key(seed, stream))


def normal_f32(seed: int, stream: int, n: int, device="cpu", start: int = 0,
               chunk: int = 1 << 24) -> torch.Tensor:
    """fp32 tensor [n], approximately N(0,1) (Irwin-Hall n=4, |z| <= 3.47)."""
    out = torch.empty(n, dtype=torch.float32, device=device)
    for lo in range(0, n, chunk):
        m = min(chunk, n - lo)
        h = hash_u64(seed, stream, start + lo, m, device)
        s = (h & 0xFFFF) + (_lsr(h, 16) & 0xFFFF) + (_lsr(h, 32) & 0xFFFF) + _lsr(h, 48)
        out[lo:lo + m] = (s - 131070).to(torch.float32) * _IH_SIGMA_INV
    return out


def uniforms(seed: int, stream: int, n: int, device="cpu", start: int = 0) -> torch.Tensor:
    """fp32 tensor [n] of u = m * 2^-24, m integer in [0, 2^24)."""
    h = hash_u64(seed, stream, start, n, device)
    return _lsr(h, 40).to(torch.float32) * (2.0 ** -24)


def prompt_tokens(seed: int, n: int, vocab: int, device="cpu") -> torch.Tensor:
    """int32 tensor [n] of uniform-random token ids in [0, vocab)."""
    h = hash_u64(seed, STREAM_PROMPT, 0, n, device)
    return (_lsr(h, 20) % vocab).to(torch.int32)


# ----------------------------------------------------------------------------------------
# model shapes
# ----------------------------------------------------------------------------------------
@dataclass(frozen=True)
class ModelSpec:
    name: str
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    ffn_dim: int
    vocab: int
    n_layers: int        # L: target decoder layers
    n_early: int         # N: layers shared by the draft model before the exit layer
    dtype: str           # "f32" or "bf16": weights, projection inputs, KV cache
    damp: float          # scale of Wo / W_down in layers n_early+1 .. L (and the exit copy)
    tie_exit_head: bool  # exit head shares storage with the target LM head
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0

    @property
    def q_dim(self) -> int:
        return self.n_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def qkv_rows(self) -> int:
        return self.q_dim + 2 * self.kv_dim

    @property
    def layer_params(self) -> int:
        d, F = self.d_model, self.ffn_dim
        return self.qkv_rows * d + d * self.q_dim + 3 * d * F

    def with_(self, **kw) -> "ModelSpec":
        return replace(self, **kw)


TINY = ModelSpec("tiny", 256, 4, 4, 64, 688, 1024, 4, 1, "f32", 0.1, True)
LLAMA2_13B = ModelSpec("13b", 5120, 40, 40, 128, 13824, 32000, 40, 5, "bf16", 0.2, False)
LLAMA2_70B = ModelSpec("70b", 8192, 64, 8, 128, 28672, 32000, 80, 10, "bf16", 0.2, False)
SPECS = {"tiny": TINY, "13b": LLAMA2_13B, "70b": LLAMA2_70B}


def _torch_dtype(spec: ModelSpec):
    return torch.float32 if spec.dtype == "f32" else torch.bfloat16


def weight_tensor(seed: int, tensor_id: int, rows: int, cols: int, scale: float, dtype,
                  device="cpu") -> torch.Tensor:
    """[rows, cols] row-major weight: scale * 0.02 * z, rounded to dtype (RNE)."""
    z = normal_f32(seed, 1000 + tensor_id, rows * cols, device,
                   chunk=(1 << 24) if str(device) == "cpu" else (1 << 27))
    z *= 0.02
    if scale != 1.0:
        z *= scale
    return z.to(dtype).view(rows, cols)


def layer_weights(spec: ModelSpec, layer: int, seed: int = SEED, device="cpu"
                  ) -> Dict[str, torch.Tensor]:
    """Weights of target layer `layer` (0-based).  All matrices are [out, in] row-major.

    wqkv rows: q heads, then k heads, then v heads.  wgu rows: gate rows then up rows.
    """
    dt = _torch_dtype(spec)
    d, F = spec.d_model, spec.ffn_dim
    s = spec.damp if layer >= spec.n_early else 1.0
    t = layer * 16
    wg = weight_tensor(seed, t + KIND_WG, F, d, 1.0, dt, device)
    wu = weight_tensor(seed, t + KIND_WU, F, d, 1.0, dt, device)
    return {
        "g_attn": torch.ones(d, dtype=torch.float32, device=device),
        "wqkv": weight_tensor(seed, t + KIND_WQKV, spec.qkv_rows, d, 1.0, dt, device),
        "wo": weight_tensor(seed, t + KIND_WO, d, spec.q_dim, s, dt, device),
        "g_ffn": torch.ones(d, dtype=torch.float32, device=device),
        "wgu": torch.cat([wg, wu], dim=0),
        "wd": weight_tensor(seed, t + KIND_WD, d, F, s, dt, device),
    }


def embedding(spec: ModelSpec, seed: int = SEED, device="cpu") -> torch.Tensor:
    return weight_tensor(seed, TID_EMBED, spec.vocab, spec.d_model, 1.0, _torch_dtype(spec), device)


def lm_head(spec: ModelSpec, seed: int = SEED, device="cpu") -> torch.Tensor:
    return weight_tensor(seed, TID_LM_HEAD, spec.vocab, spec.d_model, 1.0, _torch_dtype(spec), device)


def exit_layer_weights(spec: ModelSpec, seed: int = SEED, device="cpu", index: int = 0, count: int = 1) -> Dict[str, torch.Tensor]:
    """The early-exit layer: a copy of the last target layer.  With `count` exit layers (the paper's
    experiment on their number) exit layer `index` is a copy of target layer L - count + index: the
    last `count` target layers in their order."""
    return layer_weights(spec, spec.n_layers - count + index, seed, device)


def accept_case(case: int, batch: int, k: int, vocab: int, sigma: float, delta: float,
                seed: int = SEED, device="cpu"):
    """Inputs of one accept/resample sweep case.

    Returns (p_logits [B,K+1,V] f32, q_logits [B,K,V] f32, u_accept [B,K], u_resample [B],
    u_draft [B,K]).  Target logits ~ N(0, sigma^2); draft logits = target logits of the same
    row + N(0, delta^2).  Draft tokens are not generated here: they are drawn from q by the
    sampler under test from u_draft.
    """
    s = seed + 7919 * (case + 1)
    p = normal_f32(s, STREAM_LOGITS, batch * (k + 1) * vocab, device).view(batch, k + 1, vocab) * sigma
    noise = normal_f32(s, STREAM_LOGITS + 100, batch * k * vocab, device).view(batch, k, vocab) * delta
    q = (p[:, :k, :] + noise).contiguous()
    u_acc = uniforms(s, STREAM_ACCEPT, batch * k, device).view(batch, k)
    u_res = uniforms(s, STREAM_RESAMPLE, batch, device)
    u_dr = uniforms(s, STREAM_DRAFT, batch * k, device).view(batch, k)
    return p.contiguous(), q, u_acc, u_res, u_dr


def generate_uniforms(max_ctx: int, n_ctrl: int, seed: int = SEED, device="cpu"):
    """Uniform streams for one generation: draft/accept/resample indexed by absolute token
    position, and a sequential stream for the controller's draws."""
    return {
        "u_draft": uniforms(seed, STREAM_DRAFT, max_ctx, device),
        "u_accept": uniforms(seed, STREAM_ACCEPT, max_ctx, device),
        "u_resample": uniforms(seed, STREAM_RESAMPLE, max_ctx, device),
        "u_ctrl": uniforms(seed, STREAM_CTRL, n_ctrl, device),
    }


STREAM_CALI = 7


def cali_weights(spec: ModelSpec, seed: int = SEED, device="cpu") -> Dict[str, torch.Tensor]:
    """Random-init weights of the calibration predictor (trained ones are not available): ten
    d x d matrices W^1..W^10 in the model's dtype and the 2 x 2d matrix W_p in fp32, N(0, 0.02^2)
    and N(0, 0.05^2)."""
    d = spec.d_model
    w = torch.stack([weight_tensor(seed, 4000 + i, d, d, 1.0, _torch_dtype(spec), device) for i in range(10)])
    wp = (normal_f32(seed, STREAM_CALI, 4 * d, device) * 0.05).view(2, 2 * d)
    return {"w": w, "wp": wp}
