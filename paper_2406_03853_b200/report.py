"""Host-side report helpers: the paper's quality metrics of a decoding run and the
max-over-ranks aggregation used when several independent replicas are benchmarked.

Nothing here is on the decode path; these are a few scalar formulas.
"""
from __future__ import annotations

from typing import Dict, Optional


def harmonic_mean_metric(v_d: float, r_d: float) -> float:
    """HM = 2 v_d r_d / (v_d + r_d) * 100 (Sec. 4.1, metrics paragraph): v_d = accepted drafts /
    drafted tokens, r_d = accepted drafts / output length."""
    return 0.0 if v_d + r_d == 0 else 200.0 * v_d * r_d / (v_d + r_d)


def modelled_speedup(v_d: float, r_d: float, alpha: float) -> float:
    """Speed-up over autoregressive decoding predicted by the paper's cost model (appendix on
    the harmonic mean): T = (r_d L / v_d) T_d + (1 - r_d) L T_t, speedup = L T_t / T
    = v_d / ((alpha - v_d) r_d + v_d) with alpha = T_d / T_t."""
    return v_d / ((alpha - v_d) * r_d + v_d)


def modelled_time(v_d: float, r_d: float, L: int, t_draft: float, t_target: float) -> float:
    """T of the same model, in the units of t_draft / t_target."""
    return r_d * L / v_d * t_draft + (1.0 - r_d) * L * t_target


def run_quality(drafted: int, accepted: int, emitted: int) -> Dict[str, float]:
    v_d = accepted / drafted if drafted else 0.0
    r_d = accepted / emitted if emitted else 0.0
    return {"v_d": v_d, "r_d": r_d, "hm": harmonic_mean_metric(v_d, r_d)}


def aggregate_replicas(local_ms: float, local_units: float, dist=None, device: Optional[str] = None):
    """Whole-job throughput of independent replicas: every rank reports the device time of its
    timed region and the units (tokens) it produced; the job's time is the MAX over ranks, the
    job's work the SUM.  `dist` is torch.distributed (initialised) or None for one process.
    Returns (max_ms, total_units, units_per_second)."""
    import torch
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return local_ms, local_units, local_units / (local_ms / 1e3)
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    u = torch.tensor([local_units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item()), float(u.item()) / (float(t.item()) / 1e3)


def time_breakdown(stats: Dict[str, float]) -> Dict[str, float]:
    """The four buckets of the paper's time-breakdown table (drafting, verification, sampling,
    others) from an eesd_stats record, in seconds, plus the prompt pass and their sum, which is
    the call's wall time (the table's rows add up to the per-instance inference time)."""
    b = {"drafting": stats["ms_draft"] / 1e3, "verification": stats["ms_verify"] / 1e3,
         "sampling": stats["ms_sampling"] / 1e3, "others": stats["ms_other"] / 1e3,
         "prefill": stats["ms_prefill"] / 1e3}
    b["total"] = sum(b.values())
    return b
