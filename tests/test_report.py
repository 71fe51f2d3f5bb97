"""Host logic: the paper's report formulas against the values it prints, and the
max-over-ranks aggregation of independent replicas on two gloo ranks."""
import os
import socket
import sys

import pytest
import torch
import torch.multiprocessing as mp

from paper_2406_03853_b200 import report

GOLD = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _rows(name):
    for line in open(os.path.join(GOLD, name)):
        if line.strip() and not line.startswith("#"):
            yield line.split()


def test_harmonic_mean_matches_printed_scores():
    for _, _, v, r, hm in _rows("hm_table10.txt"):
        # v_d, r_d are printed to two decimals: +-0.005 each moves HM by up to ~1.5 points
        assert abs(report.harmonic_mean_metric(float(v), float(r)) - float(hm)) < 1.5


def test_time_buckets_add_up_to_inference_time():
    for _, _, d, v, s, o, total in _rows("time_breakdown_table8.txt"):
        assert abs(float(d) + float(v) + float(s) + float(o) - float(total)) < 0.011


def test_speed_model_algebra():
    # speedup formula == L * T_t / T of the time model, for any parameters
    for v_d, r_d, td, tt, L in [(0.5, 0.67, 3.0, 40.0, 512), (0.9, 0.7, 20.0, 40.0, 100), (0.2, 0.3, 1.0, 9.0, 64)]:
        T = report.modelled_time(v_d, r_d, L, td, tt)
        assert abs(report.modelled_speedup(v_d, r_d, td / tt) - L * tt / T) < 1e-12
    # alpha >= v_d gives no speed-up (the paper's remark under the formula)
    assert report.modelled_speedup(0.5, 0.6, 0.5) == pytest.approx(1.0)
    assert report.modelled_speedup(0.5, 0.6, 0.7) < 1.0 < report.modelled_speedup(0.5, 0.6, 0.1)
    q = report.run_quality(drafted=100, accepted=50, emitted=75)
    assert q["v_d"] == 0.5 and abs(q["r_d"] - 2 / 3) < 1e-12 and abs(q["hm"] - 200 * 0.5 * (2 / 3) / (0.5 + 2 / 3)) < 1e-9


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _rank(rank, world, port, out):
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import torch.distributed as dist
    from paper_2406_03853_b200 import report as rep
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    ms, units, rate = rep.aggregate_replicas(100.0 * (rank + 1), 256.0, dist)
    out.put((rank, ms, units, rate))
    dist.barrier()
    dist.destroy_process_group()


def test_replica_aggregation_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    ps = [ctx.Process(target=_rank, args=(r, 2, port, q)) for r in range(2)]
    for p in ps:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in ps:
        p.join(timeout=60)
        assert p.exitcode == 0
    for _, ms, units, rate in res:
        assert ms == 200.0 and units == 512.0 and rate == pytest.approx(512.0 / 0.2)  # slowest rank sets the time
    assert report.aggregate_replicas(50.0, 10.0) == (50.0, 10.0, 200.0)


def test_time_breakdown_has_the_papers_four_buckets_and_adds_up():
    # the same bookkeeping as the time-breakdown table: its four buckets add up to the inference time
    from paper_2406_03853_b200 import report
    for line in open(os.path.join(GOLD, "time_breakdown_table8.txt")):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        d, v, s, o, total = (float(x) for x in f[2:7])
        b = report.time_breakdown({"ms_draft": d * 1e3, "ms_verify": v * 1e3, "ms_sampling": s * 1e3, "ms_other": o * 1e3,
                                   "ms_prefill": 0.0})
        assert set(b) == {"drafting", "verification", "sampling", "others", "prefill", "total"}
        assert abs(b["total"] - total) < 0.006          # the table prints three decimals, the total two
