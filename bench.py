#!/usr/bin/env python
"""EESD decode benchmark on B200.

One "step" is one full decode of `max_new` tokens by Early-exiting Speculative Decoding
(draft steps through the first N layers + exit layer + exit head, one verify pass of K+1 rows
through every layer, lossless acceptance, Thompson-sampling draft length) on a synthetic
random-init model of the named LLaMA-2 shape, batch 1.

  value  tokens/s of the decode loop (eesd_decode) with the prompt already prefilled: every
         input resident in HBM when the timed region starts.
  e2e    tokens/s of eesd_generate called with host buffers: prompt upload, prefill, uniform
         streams upload, decode, per-round result read-back, all inside the timed region.
  roofline  the dominant kernel (the skinny projection that streams the weights), timed by
         CUDA events over the layers' real weight matrices, against the measured HBM copy rate.
  cpu_baseline  the CPU oracle timed on a bounded slice of the same workload.

Multi-GPU (--gpus N under torchrun): N independent replicas, no collective on the data path.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np
import torch

import eesd_synth as synth

WORKLOADS = {
    # name: (spec, prompt length, generated tokens, damp alpha, kv cache length for the verify-pass leg)
    "13b-eesd": ("13b", 512, 256, 0.05, 1024),   # alpha 0.05: acceptance statistics of the paper's 13B rows
    "70b-eesd": ("70b", 1024, 256, 0.2, 1024),
    "tiny-eesd": ("tiny", 32, 64, 0.1, 64),
}


def profiled_traffic(spec_name):
    """DRAM bytes (read + write) of one launch of the dominant kernel from the ncu capture summarised
    under profiles/ (a line `dram_bytes_per_launch <shape> <bytes>`); None when no capture of this shape
    is on file."""
    path = os.path.join(ROOT, "profiles", "gemm_tc_gate_up_dram_traffic.txt")
    if not os.path.exists(path):
        return None, None
    for line in open(path):
        f = line.split()
        if len(f) >= 3 and f[0] == "dram_bytes_per_launch" and f[1] == spec_name:
            return int(f[2]), "profiles/gemm_tc_gate_up_dram_traffic.txt"
    return None, None


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def build_engine(wl, temperature, controller, device, n_layers=0, alpha=None, n_early=None, cali=False, tree_width=0, n_exit=1,
                 spec_edit=None, kv_seqs=1):
    from paper_2406_03853_b200 import Engine
    from paper_2406_03853_b200 import binding as b
    spec_name, n_prompt, max_new, damp, _ = WORKLOADS[wl]
    spec = synth.SPECS[spec_name].with_(damp=damp if alpha is None else alpha)
    if spec_edit:
        spec = spec.with_(**spec_edit)
    if n_early:
        spec = spec.with_(n_early=n_early)
    if n_layers:
        spec = spec.with_(n_layers=n_layers, n_early=min(spec.n_early, n_layers))
    max_ctx = max(n_prompt + max_new + 16, 1024 + 32)
    cfg = b.make_config(d_model=spec.d_model, n_heads=spec.n_heads, n_kv_heads=spec.n_kv_heads, head_dim=spec.head_dim,
                        ffn_dim=spec.ffn_dim, vocab=spec.vocab, n_layers=spec.n_layers, n_early=spec.n_early,
                        dtype=spec.dtype, tie_exit_head=spec.tie_exit_head, max_ctx=max_ctx,
                        k_cap=10 if tree_width < 2 else 15 // tree_width,
                        temperature=temperature, controller=b.CTRL_CALI_TS if cali else controller, fixed_k=5, page_tokens=16,
                        tree_width=tree_width, n_exit_layers=n_exit)
    # (kv_seqs > 1: one page pool that holds that many sequences, for batch mode)
    eng = Engine(cfg, device=device, kv_pages=None if kv_seqs == 1 else kv_seqs * (max_ctx // 16 + 2))
    # synthetic weights, generated on the device by the shared seeded generator
    for l in range(spec.n_layers):
        v = eng.layer_views(l)
        for k, t in synth.layer_weights(spec, l, synth.SEED, device).items():
            v[k].copy_(t)
    for e in range(n_exit):
        v = eng.layer_views(spec.n_layers + e)
        for k, t in synth.exit_layer_weights(spec, synth.SEED, device, e, n_exit).items():
            v[k].copy_(t)
    g = eng.global_views()
    g["embed"].copy_(synth.embedding(spec, synth.SEED, device))
    head = synth.lm_head(spec, synth.SEED, device)
    g["lm_head"].copy_(head)
    if not spec.tie_exit_head:
        g["exit_head"].copy_(head)
    g["g_final"].fill_(1.0)
    g["g_exit"].fill_(1.0)
    if cali:   # random-init predictor (trained weights are not available): times the mechanism only
        cw = synth.cali_weights(spec, synth.SEED, device)
        g["cali_w"].copy_(cw["w"])
        g["cali_wp"].copy_(cw["wp"])
    torch.cuda.synchronize(device)
    return eng, spec, n_prompt, max_new


def pass_bytes(spec, rows_ctx):
    """Algorithmic HBM bytes of one verify pass and one draft step: every weight of the layers
    used plus the vocabulary head once, plus the KV rows read (cache of rows_ctx tokens)."""
    es = 2 if spec.dtype == "bf16" else 4
    layer = spec.layer_params * es
    head = spec.vocab * spec.d_model * es
    kv_tok = 2 * spec.kv_dim * es
    verify = spec.n_layers * layer + head + spec.n_layers * rows_ctx * kv_tok
    draft = (spec.n_early + 1) * layer + head + (spec.n_early + 1) * rows_ctx * kv_tok
    return verify, draft


def time_projection(eng, spec, M, reps=3):
    """Dominant kernel as the passes launch it: the gate/up projection of every layer, back to
    back over the layers' own weights (consecutive launches never re-read a matrix from L2),
    bracketed by CUDA events on the library's stream (eesd_time_projection)."""
    ms = [eng.time_projection(2, M) for _ in range(reps)]
    return ms[0][1], statistics.median(m for m, _ in ms)


def time_verify_pass(eng, spec, ctx_len, M, reps=5):
    toks = synth.prompt_tokens(5, M, spec.vocab).numpy()
    eng.assume_context(ctx_len, int(toks[0]))
    for _ in range(2):
        eng.verify_only(toks)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ts = []
    for _ in range(reps):
        e0.record()
        eng.verify_only(toks)
        e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
    return statistics.median(ts)


def time_accept_kernel(device, batches=(1, 8, 64), ks=(4, 16), vocab=32000, reps=20):
    """The fused softmax / accept / resample kernel on the accept-sweep inputs (vocab 32000,
    sigma 1, delta 1, temperature 1).  Algorithmic bytes: every p and q logit read once, plus the
    rejected (or bonus) row pair read again for the residual draw: (2K + 3) V 4 bytes per sequence
    at most.  Inputs exceed L2 only at batch 64 x K 16 (262 MB); the smaller cases are timed from
    L2, are latency bound, and their figure includes the host's launch overhead (one call, one
    memset and one kernel, between the two events)."""
    from paper_2406_03853_b200 import binding as b
    out = {}
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for B in batches:
        for K in ks:
            p, q, ua, ur, ud = synth.accept_case(0, B, K, vocab, 1.0, 1.0, device=device)
            toks = b.sample_rows(q.view(B * K, vocab), ud.view(-1), 1.0).view(B, K)
            for _ in range(3):
                b.accept_resample(p, q, toks, ua, ur, 1.0)
            torch.cuda.synchronize()
            ts = []
            for _ in range(reps):
                e0.record()
                b.accept_resample(p, q, toks, ua, ur, 1.0)
                e1.record()
                torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1))
            ms = statistics.median(ts)
            nbytes = B * (2 * K + 3) * vocab * 4
            out[f"B{B}_K{K}"] = {"us": round(ms * 1e3, 2), "gbs": round(nbytes / (ms * 1e-3) / 1e9, 1)}
    return out


# The round both CPU legs (cpu_baseline of the default run, --impl reference) are scaled to: K drafted
# tokens and EMIT emitted tokens per round, the rounded means of the default workload under Beta-TS
# (mean K 2.5, 2.2 tokens per round).  Fixed so that both legs describe the same work.
ORACLE_ROUND_K, ORACLE_ROUND_EMIT = 3, 2.2


def _omp_threads(n=None):
    """Sets (n given) or reads the OpenMP thread count of the process the oracle runs in."""
    import ctypes
    try:
        gomp = ctypes.CDLL("libgomp.so.1")
    except OSError:
        return os.cpu_count() or 1
    if n is not None:
        gomp.omp_set_num_threads(int(n))
    return int(gomp.omp_get_max_threads())


_SLICES = {}


def _oracle_slice(spec):
    """The oracle's model for the timed slice (built once per process): one layer, the real head."""
    if spec.name not in _SLICES:
        import oracle
        L1 = spec.with_(n_layers=1, n_early=1)
        lw = {k: v for k, v in synth.layer_weights(spec, 0).items()}
        emb = np.zeros((spec.vocab, spec.d_model), np.float32)
        _SLICES[spec.name] = oracle.model_from_weights(L1, [lw], lw, emb, synth.lm_head(spec), max_ctx=640)
    return _SLICES[spec.name]


def oracle_sample(spec, budget_s=12.0):
    """CPU oracle on a bounded slice of the workload: ONE decoder layer of this shape and the real
    vocabulary head (full vocabulary), on ORACLE_ROUND_K + 1 rows (a verify pass) and on 1 row (a draft
    step) against a 512-token cache, repeated until about `budget_s` seconds of CPU work have been
    timed with all OpenMP threads, then once more single-threaded.  The medians are scaled to a whole
    round by the layer counts (all layers + head for the verify pass; early layers + exit layer + exit
    head per draft step).  Returns a dict with tokens/s (all threads and one thread) and what was timed."""
    m = _oracle_slice(spec)
    rows = ORACLE_ROUND_K + 1
    x = np.asarray(synth.normal_f32(1, 1, rows * spec.d_model).view(rows, spec.d_model), np.float64)
    m.layer_fwd(0, 0, x[:1], 512)   # touch the weights once, untimed
    m.head(x[:1])

    def one():
        t0 = time.time()
        m.layer_fwd(0, 0, x, 512)
        t1 = time.time()
        m.layer_fwd(0, 0, x[:1], 512)
        t2 = time.time()
        m.head(x)
        t3 = time.time()
        m.head(x[:1])
        t4 = time.time()
        return t1 - t0, t2 - t1, t3 - t2, t4 - t3

    def tokens_per_s(t):
        t_layer_rows, t_layer_1, t_head_rows, t_head_1 = t
        t_verify = spec.n_layers * t_layer_rows + t_head_rows
        t_draft = ORACLE_ROUND_K * ((spec.n_early + 1) * t_layer_1 + t_head_1)
        return ORACLE_ROUND_EMIT / (t_verify + t_draft)

    threads = _omp_threads()
    samples, spent = [], 0.0
    while spent < budget_s and len(samples) < 200:
        samples.append(one())
        spent += sum(samples[-1])
    med = tuple(statistics.median(c) for c in zip(*samples))
    _omp_threads(1)
    single = one()
    _omp_threads(threads)
    return {"tokens_per_s": tokens_per_s(med), "tokens_per_s_one_thread": tokens_per_s(single), "threads": threads,
            "seconds_timed": spent + sum(single), "repetitions": len(samples), "rows": rows,
            "sample": (f"one {spec.name}-shaped decoder layer and the {spec.vocab}-entry vocabulary head on {rows} rows and on 1 row "
                       f"against a 512-token cache ({len(samples)} repetitions with {threads} OpenMP threads, medians; once with 1 thread), "
                       f"scaled by layer count to a round of K={ORACLE_ROUND_K} drafts emitting {ORACLE_ROUND_EMIT} tokens "
                       f"({spec.n_layers} layers + head per verify pass, {spec.n_early + 1} layers + head per draft step); extrapolated over layers")}


def profile_pass(args, device):
    """Verify passes and draft steps between cudaProfilerStart/Stop (for the ncu recipes)."""
    from paper_2406_03853_b200 import binding as b
    eng, spec, _, _ = build_engine(args.workload, 0.0, b.CTRL_FIXED_K, device, args.layers)
    kv_len = WORKLOADS[args.workload][4]
    toks = synth.prompt_tokens(5, args.profile_pass, spec.vocab).numpy()
    eng.assume_context(kv_len, int(toks[0]))
    eng.verify_only(toks)
    torch.cuda.synchronize()
    torch.cuda.profiler.start()
    eng.verify_only(toks)
    eng.draft(1)
    torch.cuda.synchronize()
    torch.cuda.profiler.stop()
    print("profiled: 1 verify pass of %d rows + 1 draft step, %s, %d layers" % (args.profile_pass, spec.name, spec.n_layers))
    eng.close()


def profile_tree_round(args, device):
    """One greedy round with tree verification (K = 3 draft steps, width --profile-tree, so
    1 + 3 width rows in the verify pass) against a 1024-token cache, between
    cudaProfilerStart/Stop (for the ncu recipes)."""
    from paper_2406_03853_b200 import binding as b
    W = args.profile_tree
    eng, spec, _, _ = build_engine(args.workload, 0.0, b.CTRL_FIXED_K, device, args.layers, tree_width=W)
    kv_len = WORKLOADS[args.workload][4]
    eng.assume_context(kv_len, 17)
    eng.draft(3)
    eng.verify_accept()
    torch.cuda.synchronize()
    torch.cuda.profiler.start()
    eng.draft(3)
    a, y = eng.verify_accept()
    torch.cuda.synchronize()
    torch.cuda.profiler.stop()
    print("profiled: 1 round of 3 draft steps + tree verify pass of %d rows (width %d), %s, %d layers; accepted %d"
          % (1 + 3 * W, W, spec.name, spec.n_layers, a))
    eng.close()


def profile_prefill(args, device):
    """One prompt pass (eesd_prefill) between cudaProfilerStart/Stop (for the ncu recipes)."""
    from paper_2406_03853_b200 import binding as b
    eng, spec, n_prompt, _ = build_engine(args.workload, 0.0, b.CTRL_FIXED_K, device, args.layers)
    prompt = synth.prompt_tokens(synth.SEED, n_prompt, spec.vocab).numpy()
    eng.prefill(prompt)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.profiler.start()
    e0.record()
    eng.prefill(prompt)
    e1.record()
    torch.cuda.synchronize()
    torch.cuda.profiler.stop()
    print("profiled: prefill of %d tokens, %s, %d layers, %.3f ms" % (n_prompt, spec.name, spec.n_layers, e0.elapsed_time(e1)))
    eng.close()


def run_sweep(args, device):
    """Method sweeps on the synthetic model (one JSON line per setting, rank 0 only, not the
    contract line): `--sweep k` decodes with every fixed draft length K = 1..10 and with the
    Beta-TS controller (the paper's fixed-K curve against Thompson sampling); `--sweep n` rebuilds
    the model with the early exit after N = 1, 2, 3, 5, 8, 10 layers (the paper's N sweep; in the
    synthetic model the layers after N are the damped ones, so acceptance changes with N by
    construction); `--sweep tree` decodes greedily with tree verification of width 1 (the chain),
    2 and 3 at fixed draft lengths (the paper's table on tree attention: more candidates per
    position, one verification pass).  Each setting decodes `--steps` different seeded prompts."""
    from paper_2406_03853_b200 import binding as b
    from paper_2406_03853_b200 import report
    spec_name, n_prompt, max_new, damp, kv_len = WORKLOADS[args.workload]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def measure(eng, spec, label, k_schedule):
        u = {k: v.numpy() for k, v in synth.generate_uniforms(eng.cfg.max_ctx, 1 << 20).items()}
        tot = {"drafted": 0, "accepted": 0, "emitted": 0, "rounds": 0}
        ms, leaves = 0.0, 0
        for i in range(args.steps):
            eng.prefill(synth.prompt_tokens(synth.SEED + i, n_prompt, spec.vocab).numpy())
            torch.cuda.synchronize()
            e0.record()
            _, _, st = eng.decode(max_new, k_schedule=k_schedule, uniforms=u)
            e1.record()
            torch.cuda.synchronize()
            ms += e0.elapsed_time(e1)
            for k in tot:
                tot[k] += st.as_dict()[k]
            leaves += st.leaves_kept
        q = report.run_quality(tot["drafted"], tot["accepted"], tot["emitted"])
        t1 = time_verify_pass(eng, spec, kv_len, 1)
        tps = args.steps * max_new / (ms / 1e3)
        print(json.dumps({"sweep": args.sweep, "setting": label, "workload": args.workload, "tokens_per_s": round(tps, 2),
                          "speedup_vs_autoregressive": round(tps / (1e3 / t1), 4), "mean_k": round(tot["drafted"] / max(1, tot["rounds"]), 3),
                          "v_d": round(q["v_d"], 4), "r_d": round(q["r_d"], 4), "hm": round(q["hm"], 2),
                          "leaves_kept_per_round": round(leaves / max(1, tot["rounds"]), 4),
                          "early_layers": spec.n_early, "damp_alpha": spec.damp, "steps": args.steps}), flush=True)

    if args.sweep == "k":
        eng, spec, _, _ = build_engine(args.workload, args.temperature, b.CTRL_BETA_TS, device, alpha=args.alpha)
        for K in range(1, 11):
            measure(eng, spec, f"fixed K={K}", [K] * max_new)
        measure(eng, spec, "beta-ts", None)
        eng.close()
    elif args.sweep == "tree":
        for W in (1, 2, 3):
            eng, spec, _, _ = build_engine(args.workload, 0.0, b.CTRL_BETA_TS, device, alpha=args.alpha, tree_width=W)
            for K in (2, 3, 4, 5):
                measure(eng, spec, f"width {W}, fixed K={K} ({1 + K * max(W, 1)} rows per pass)", [K] * max_new)
            measure(eng, spec, f"width {W}, beta-ts (K cap {eng.cfg.k_cap})", None)
            eng.close()
            del eng
            torch.cuda.empty_cache()
    elif args.sweep == "batch":
        # Several sequences sharing every pass (an extension: the paper's batch is 1).  The rows of a pass are capped
        # at 16, so more sequences mean shorter drafts: B x (K + 1) <= 16.  One JSON line per (B, K): tokens/s summed
        # over the sequences, against single-sequence decoding with the same fixed draft length.
        edit = {"dtype": "bf16", "ffn_dim": 640} if synth.SPECS[spec_name].dtype == "f32" else None   # batch mode is bf16 only
        eng, spec, _, _ = build_engine(args.workload, args.temperature, b.CTRL_FIXED_K, device, alpha=args.alpha, spec_edit=edit, kv_seqs=8)
        u = [{k: v.numpy() for k, v in synth.generate_uniforms(eng.cfg.max_ctx, 64, seed=synth.SEED + 50 + i).items()} for i in range(8)]
        for B, K in ((1, 3), (1, 1), (2, 3), (2, 7), (4, 3), (4, 1), (8, 1)):
            ms, tot = 0.0, {"drafted": 0, "accepted": 0, "emitted": 0, "rounds": 0}
            for i in range(args.steps):
                eng.batch_begin(B)
                for q in range(B):
                    eng.batch_prefill(q, synth.prompt_tokens(synth.SEED + 8 * i + q, n_prompt, spec.vocab).numpy())
                torch.cuda.synchronize()
                e0.record()
                _, _, st = eng.batch_decode(max_new, k_schedule=[K] * (4 * max_new), uniforms=u[:B] if args.temperature else None)
                e1.record()
                torch.cuda.synchronize()
                ms += e0.elapsed_time(e1)
                for k in tot:
                    tot[k] += st.as_dict()[k]
            eng.batch_begin(0)
            q = report.run_quality(tot["drafted"], tot["accepted"], tot["emitted"])
            print(json.dumps({"sweep": "batch", "setting": f"B={B}, K={K}", "workload": args.workload, "sequences": B, "k": K,
                              "rows_per_verify_pass": B * (K + 1), "tokens_per_s": round(args.steps * B * max_new / (ms / 1e3), 2),
                              "tokens_per_s_per_sequence": round(args.steps * max_new / (ms / 1e3), 2),
                              "v_d": round(q["v_d"], 4), "r_d": round(q["r_d"], 4), "batch_rounds": tot["rounds"],
                              "steps": args.steps}), flush=True)
        eng.close()
    elif args.sweep == "exit":
        # the paper's experiment on the number of early-exit layers: a deeper draft head accepts more and costs more
        for E in (1, 2, 3):
            eng, spec, _, _ = build_engine(args.workload, args.temperature, b.CTRL_BETA_TS, device, alpha=args.alpha, n_exit=E)
            measure(eng, spec, f"{E} exit layer(s)", None)
            eng.close()
            del eng
            torch.cuda.empty_cache()
    else:
        for N in (1, 2, 3, 5, 8, 10):
            if N >= synth.SPECS[spec_name].n_layers:   # the exit must leave at least one layer to skip
                continue
            eng, spec, _, _ = build_engine(args.workload, args.temperature, b.CTRL_BETA_TS, device, alpha=args.alpha, n_early=N)
            measure(eng, spec, f"N={N}", None)
            eng.close()
            del eng
            torch.cuda.empty_cache()


def leg_70b(device, peaks, steps=2, new_tokens=64):
    """The LLaMA-2-70B-shaped configuration (80 layers, 64 / 8 heads, about 140 GB of bf16 weights, early
    exit after 10 layers, damping 0.2, 1024-token prompt) on the same GPU: verify passes of 1, 6 and 16
    rows against a 1024-token cache, and a short decode (`steps` prompts x `new_tokens` tokens, Beta-TS)."""
    from paper_2406_03853_b200 import binding as b
    from paper_2406_03853_b200 import report
    t0 = time.time()
    torch.cuda.empty_cache()
    eng, spec, n_prompt, _ = build_engine("70b-eesd", 0.0, b.CTRL_BETA_TS, device)
    t_build = time.time() - t0
    kv_len = WORKLOADS["70b-eesd"][4]
    bv, bd = pass_bytes(spec, kv_len)
    out = {"weights_gb": round(eng.sizes.weights_bytes / 1e9, 1), "verify_pass": {"kv_len": kv_len, "bytes": bv}, "draft_step_bytes": bd}
    for M in (1, 6, 16):
        ms = time_verify_pass(eng, spec, kv_len, M)
        out["verify_pass"][f"M{M}"] = {"ms": round(ms, 4), "gbs": round(bv / (ms * 1e-3) / 1e9, 1),
                                       "frac_of_measured_copy": round(bv / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 4),
                                       "frac_of_8tbs": round(bv / (ms * 1e-3) / 1e9 / 8000.0, 4)}
    u = {k: v.numpy() for k, v in synth.generate_uniforms(eng.cfg.max_ctx, 1 << 20).items()}
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ms_dec, ms_e2e, tot = 0.0, 0.0, {"drafted": 0, "accepted": 0, "emitted": 0, "rounds": 0, "ms_draft": 0.0}
    for i in range(steps):
        prompt = synth.prompt_tokens(synth.SEED + i, n_prompt, spec.vocab).numpy()
        eng.prefill(prompt)
        torch.cuda.synchronize()
        e0.record()
        _, _, st = eng.decode(new_tokens, uniforms=u)
        e1.record()
        torch.cuda.synchronize()
        ms_dec += e0.elapsed_time(e1)
        for k in tot:
            tot[k] += st.as_dict()[k]
        e0.record()
        eng.generate(prompt, new_tokens, uniforms=u)
        e1.record()
        torch.cuda.synchronize()
        ms_e2e += e0.elapsed_time(e1)
    q = report.run_quality(tot["drafted"], tot["accepted"], tot["emitted"])
    out["decode"] = {"tokens_per_s": round(steps * new_tokens / (ms_dec * 1e-3), 2), "prompts": steps, "new_tokens": new_tokens,
                     "prompt_tokens": n_prompt, "e2e_tokens_per_s": round(steps * new_tokens / (ms_e2e * 1e-3), 2),
                     "autoregressive_tokens_per_s": round(1e3 / out["verify_pass"]["M1"]["ms"], 2),
                     "ms_per_draft_step": round(tot["ms_draft"] / max(1, tot["drafted"]), 4),
                     "mean_k": round(tot["drafted"] / max(1, tot["rounds"]), 3), "v_d": round(q["v_d"], 4), "r_d": round(q["r_d"], 4),
                     "early_layers": spec.n_early, "damp_alpha": spec.damp}
    eng.close()
    del eng
    torch.cuda.empty_cache()
    out["seconds"] = {"build": round(t_build, 1), "whole_leg": round(time.time() - t0, 1)}
    return out


def run_reference(args):
    """--impl reference: the CPU oracle as it stands, timed on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    spec_name, n_prompt, max_new, damp, _ = WORKLOADS[args.workload]
    spec = synth.SPECS[spec_name].with_(damp=damp)
    vals, ms, last = [], [], None
    for i in range(args.warmup + args.steps):
        t0 = time.time()
        last = oracle_sample(spec, budget_s=8.0)
        if i >= args.warmup:
            vals.append(last["tokens_per_s"])
            ms.append((time.time() - t0) * 1e3)
    v = statistics.median(vals)
    print(json.dumps({"impl": "reference", "metric": "eesd_decode_tokens_per_s", "value": v, "unit": "tokens/s",
                      "n_gpus": 0, "steps": args.steps, "warmup": args.warmup, "ms_per_step": statistics.median(ms),
                      "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                      "config": {"workload": args.workload, "round_model": {"k": ORACLE_ROUND_K, "tokens_per_round": ORACLE_ROUND_EMIT}},
                      "cpu_baseline": {"value": v, "unit": "tokens/s", "cores": last["threads"], "kind": "oracle",
                                       "value_one_thread": last["tokens_per_s_one_thread"], "sample": last["sample"]},
                      "e2e": {"value": v, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=6)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="13b-eesd", choices=sorted(WORKLOADS))
    ap.add_argument("--temperature", type=float, default=0.0)
    ap.add_argument("--alpha", type=float, default=None,
                    help="scale of the upper layers' output projections (draft/target agreement): 0.05 high, "
                         "0.2 medium (default), 0.5 low acceptance")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-variants", action="store_true", help="skip the temperature-1 / lower-agreement legs")
    ap.add_argument("--no-tree", action="store_true", help="skip the tree-verification leg of the default run")
    ap.add_argument("--no-70b", action="store_true",
                    help="skip the LLaMA-2-70B-shaped leg of the default run (verify passes and a short decode; about a minute)")
    ap.add_argument("--profile-pass", type=int, default=0, metavar="M",
                    help="only run verify passes of M rows (and draft steps) inside a cudaProfilerStart/Stop "
                         "bracket, for ncu --profile-from-start off")
    ap.add_argument("--controller", choices=["beta", "cali"], default="beta",
                    help="draft-length controller: Beta-TS (default) or TS with calibration (random-init predictor)")
    ap.add_argument("--sweep", choices=["k", "n", "tree", "exit", "batch"], default=None,
                    help="method sweep instead of the benchmark line: fixed K = 1..10 against Beta-TS, the exit depth N, "
                         "tree verification widths, the number of early-exit layers, or the number of sequences decoded together")
    ap.add_argument("--profile-prefill", action="store_true",
                    help="only run one prompt pass inside a cudaProfilerStart/Stop region (for ncu)")
    ap.add_argument("--profile-tree", type=int, default=0, metavar="W",
                    help="only run one round with tree verification of width W inside a cudaProfilerStart/Stop bracket")
    ap.add_argument("--layers", type=int, default=0, help="with --profile-pass: keep only this many layers")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.warmup < 3:
        args.warmup = 3

    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    device = torch.device(f"cuda:{local}")
    torch.cuda.set_device(device)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    from paper_2406_03853_b200 import binding as b
    if args.profile_pass:
        return profile_pass(args, device)
    if args.profile_prefill:
        return profile_prefill(args, device)
    if args.profile_tree:
        return profile_tree_round(args, device)
    if args.sweep:
        return run_sweep(args, device) if rank == 0 else None
    from paper_2406_03853_b200 import report
    eng, spec, n_prompt, max_new = build_engine(args.workload, args.temperature, b.CTRL_BETA_TS, device, alpha=args.alpha,
                                                cali=args.controller == "cali")
    # acceptance along one greedy trajectory of a random-init model is noisy, so every step
    # decodes a different seeded prompt (the same ones on every run; ranks take disjoint seeds)
    prompts = [synth.prompt_tokens(synth.SEED + 1000 * rank + i, n_prompt, spec.vocab).numpy()
               for i in range(max(args.steps, args.warmup))]
    u = {k: v.numpy() for k, v in synth.generate_uniforms(eng.cfg.max_ctx, 1 << 20).items()}

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        torch.cuda.synchronize()

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # ---- value: decode loop only, prompt prefilled, everything resident
    for i in range(args.warmup):
        eng.prefill(prompts[i])
        eng.decode(max_new, uniforms=u)
    clocks = ClockSampler(local)
    stats, dec_ms = [], 0.0
    launches0 = eng.launch_count()
    barrier()
    clocks.start()
    for i in range(args.steps):
        eng.prefill(prompts[i])   # untimed: builds the KV cache of the prompt
        torch.cuda.synchronize()
        e0.record()
        out, trace, st = eng.decode(max_new, uniforms=u)
        e1.record()
        torch.cuda.synchronize()
        dec_ms += e0.elapsed_time(e1)
        stats.append(st.as_dict())
    clk = clocks.stop()
    barrier()
    launches = eng.launch_count() - launches0
    # independent replicas: the job's time is the slowest rank's, its work the sum over ranks
    dec_ms, _, value = report.aggregate_replicas(dec_ms, args.steps * max_new, dist, device)

    # ---- e2e: eesd_generate with host buffers (prefill and all copies inside the timed region)
    e2e_ms = 0.0
    barrier()
    d2h = 0
    for i in range(args.steps):
        e0.record()
        out2, trace2, st2 = eng.generate(prompts[i], max_new, uniforms=u)
        e1.record()
        torch.cuda.synchronize()
        e2e_ms += e0.elapsed_time(e1)
        d2h += sum(12 + 4 * k for k, _, _ in trace2)
    d2h //= args.steps
    e2e_ms, _, e2e_value = report.aggregate_replicas(e2e_ms, args.steps * max_new, dist, device)
    greedy = args.temperature == 0.0
    h2d = n_prompt * 4 + (0 if greedy else 3 * eng.cfg.max_ctx * 4)

    if rank != 0:
        return
    # ---- dominant kernel and verify pass against the HBM roofline
    peaks, peak_kind = measured_peaks()
    mean_k = sum(s["drafted"] for s in stats) / max(1, sum(s["rounds"] for s in stats))
    mean_emit = sum(s["emitted"] for s in stats) / max(1, sum(s["rounds"] for s in stats))
    M_typ = min(16, int(round(mean_k)) + 1)
    kbytes, kms = time_projection(eng, spec, M_typ)
    achieved = kbytes / (kms * 1e-3) / 1e9
    kv_len = WORKLOADS[args.workload][4]
    bv, bd = pass_bytes(spec, kv_len)
    vp = {}
    for M in sorted({1, 2, 4, 8, 16, M_typ, 6, 11}):   # 6 and 11: K = 5 (the paper's best fixed K for 13B) and K = k_cap
        ms = time_verify_pass(eng, spec, kv_len, M)
        vp[f"M{M}"] = {"ms": round(ms, 4), "ms_per_layer": round(ms / spec.n_layers, 5), "gbs": round(bv / (ms * 1e-3) / 1e9, 1),
                       "frac_of_measured_copy": round(bv / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 4),
                       "frac_of_8tbs": round(bv / (ms * 1e-3) / 1e9 / 8000.0, 4)}
    traffic, traffic_src = profiled_traffic(spec.name)
    s0 = {k: sum(st[k] for st in stats) for k in ("drafted", "accepted", "emitted", "rounds", "ms_draft", "ms_verify", "ms_sampling",
                                                  "ms_other", "ms_total")}
    qual = report.run_quality(s0["drafted"], s0["accepted"], s0["emitted"])
    v_d, r_d = qual["v_d"], qual["r_d"]
    # the paper's cost model (its appendix on the harmonic mean) with the measured draft-step and
    # verify-pass times: what speed-up over one-token-per-pass decoding these v_d, r_d predict
    t_d = s0["ms_draft"] / max(1, s0["drafted"])
    t_t = vp["M1"]["ms"]
    model_speedup = report.modelled_speedup(v_d, r_d, t_d / t_t) if v_d > 0 else None
    line = {
        "metric": "eesd_decode_tokens_per_s", "value": round(value, 3), "unit": "tokens/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(dec_ms / args.steps, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": spec.dtype, "data": "synthetic",
        "config": {"workload": args.workload, "shape": spec.name, "prompt_tokens": n_prompt, "new_tokens": max_new,
                   "batch": 1, "early_layers": spec.n_early, "damp_alpha": spec.damp,
                   "controller": "beta_ts" if args.controller == "beta" else "cali_ts (random-init predictor)",
                   "k_cap": 10, "temperature": args.temperature, "parallelism": f"replicas x{world}",
                   "prompts": "a different seeded prompt every step",
                   "l2_policy": "inputs larger than L2 (each pass streams every weight once)"},
        "e2e": {"value": round(e2e_value, 3), "unit": "tokens/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": round(e2e_ms / args.steps, 3)},
        "gpu_launches": int(launches),
        "clocks": clk,
        "roofline": {"bound": "hbm", "kernel": "skinny projection (gate/up shape, M=%d)" % M_typ,
                     "achieved": round(achieved, 1), "peak": peaks["hbm_gbs"], "peak_kind": peak_kind, "unit": "GB/s",
                     "frac": round(achieved / peaks["hbm_gbs"], 4),
                     "frac_of_8tbs": round(achieved / 8000.0, 4),
                     "note": "the denominator is a COPY rate (read + write); a read-only weight stream can exceed it, so a "
                             "fraction above 1 is not headroom.  The figure the target is set on is verify_pass_frac_of_8tbs",
                     "traffic": traffic, "traffic_source": traffic_src,
                     "bytes_per_launch": kbytes, "ms_per_launch": round(kms, 5)},
        "verify_pass_frac_of_8tbs": {spec.name: {k: v["frac_of_8tbs"] for k, v in vp.items() if k in ("M1", "M6", "M16")}},
        "verify_pass": {"kv_len": kv_len, "bytes": bv, **vp},
        "draft_step_bytes": bd,
        "accept_kernel": time_accept_kernel(device),
        "round_stats": {"rounds_per_step": round(s0["rounds"] / args.steps, 1), "mean_k": round(mean_k, 3), "v_d": round(v_d, 4), "r_d": round(r_d, 4),
                        "hm": round(qual["hm"], 2),
                        "ms_per_draft_step": round(t_d, 4), "autoregressive_tokens_per_s": round(1e3 / t_t, 2),
                        "speedup_vs_autoregressive": round(value / world / (1e3 / t_t), 4),
                        "speedup_by_cost_model": None if model_speedup is None else round(model_speedup, 4),
                        # the paper's time-breakdown buckets, per decoded sequence (decode loop only: no prompt pass)
                        "ms_draft": round(s0["ms_draft"] / args.steps, 3), "ms_verify": round(s0["ms_verify"] / args.steps, 3),
                        "ms_sampling": round(s0["ms_sampling"] / args.steps, 3), "ms_other": round(s0["ms_other"] / args.steps, 3),
                        "ms_wall": round(s0["ms_total"] / args.steps, 3),
                        "ms_prefill_e2e": round(st2.ms_prefill, 3)},
    }
    if not args.no_cpu_baseline and world == 1:
        import oracle
        oracle.build()
        o = oracle_sample(spec)
        line["cpu_baseline"] = {
            "value": round(o["tokens_per_s"], 5), "unit": "tokens/s", "cores": o["threads"], "kind": "oracle",
            "value_one_thread": round(o["tokens_per_s_one_thread"], 5), "seconds_timed": round(o["seconds_timed"], 1),
            "round_model": {"k": ORACLE_ROUND_K, "tokens_per_round": ORACLE_ROUND_EMIT}, "sample": o["sample"]}
    eng.close()
    del eng
    if world == 1 and greedy and args.controller == "beta" and not args.no_tree:
        # tree verification (the paper's tree-attention table) on the same prompts: width 2, three
        # draft steps per round (7 rows per pass), against the chain at the same draft length
        torch.cuda.empty_cache()
        tv, outs = {}, {}
        for W in (1, 2):
            eng_t, _, _, _ = build_engine(args.workload, 0.0, b.CTRL_FIXED_K, device, alpha=args.alpha, tree_width=W,
                                          kv_seqs=4 if W == 1 else 1)
            ms_t, tot = 0.0, {"drafted": 0, "accepted": 0, "rounds": 0, "leaves_kept": 0}
            for i in range(args.steps):
                eng_t.prefill(prompts[i])
                torch.cuda.synchronize()
                e0.record()
                out_t, _, st_t = eng_t.decode(max_new, k_schedule=[3] * max_new)
                outs.setdefault(W, []).append(out_t.copy())
                e1.record()
                torch.cuda.synchronize()
                ms_t += e0.elapsed_time(e1)
                for k in tot:
                    tot[k] += st_t.as_dict()[k]
            tv["chain_k3" if W == 1 else "width2_k3"] = {
                "tokens_per_s": round(args.steps * max_new / (ms_t * 1e-3), 2),
                "v_d": round(tot["accepted"] / max(1, tot["drafted"]), 4),
                "leaves_kept_per_round": round(tot["leaves_kept"] / max(1, tot["rounds"]), 4)}
            if W == 1 and spec.dtype == "bf16" and args.steps >= 4:
                # batch mode (an extension: the paper's batch is 1): the first four prompts decoded together, three
                # drafts per round (16 rows per verification pass), against the same prompts decoded one by one above
                for timed in (False, True):   # once untimed: the first launches of the batched kernels load them
                    eng_t.batch_begin(4)
                    for q in range(4):
                        eng_t.batch_prefill(q, prompts[q])
                    if not timed:
                        eng_t.batch_decode(8, k_schedule=[3] * 32)
                torch.cuda.synchronize()
                e0.record()
                out_b, _, st_b = eng_t.batch_decode(max_new, k_schedule=[3] * (4 * max_new))
                e1.record()
                torch.cuda.synchronize()
                eng_t.batch_begin(0)
                line["batch_decode"] = {"sequences": 4, "k": 3, "rows_per_verify_pass": 16,
                                        "tokens_per_s": round(4 * max_new / (e0.elapsed_time(e1) * 1e-3), 2),
                                        "v_d": round(st_b.accepted / max(1, st_b.drafted), 4),
                                        "same_tokens_as_one_by_one": all((out_b[q] == outs[1][q]).all() for q in range(4))}
            eng_t.close()
            del eng_t
            torch.cuda.empty_cache()
        # greedy decoding is lossless either way: both runs must have emitted the same tokens
        tv["same_tokens_as_chain"] = all((a == c).all() for a, c in zip(outs[2], outs[1]))
        line["tree_verification"] = tv
    if world == 1 and greedy and args.controller == "beta" and not args.no_variants and args.alpha is None:
        # the same workload at temperature 1 (stochastic acceptance and residual resampling on the device) and with
        # less agreement between draft and target (output projections of the upper layers scaled by 0.2 and 0.5
        # instead of 0.05): two prompts each, Beta-TS
        torch.cuda.empty_cache()
        var = {}
        for label, alpha_v, temp_v in (("temperature_1", None, 1.0), ("alpha_0.2", 0.2, 0.0), ("alpha_0.5", 0.5, 0.0)):
            eng_v, _, _, _ = build_engine(args.workload, temp_v, b.CTRL_BETA_TS, device, alpha=alpha_v)
            ms_v, tot = 0.0, {"drafted": 0, "accepted": 0, "emitted": 0, "rounds": 0}
            for i in range(min(2, args.steps)):
                eng_v.prefill(prompts[i])
                torch.cuda.synchronize()
                e0.record()
                _, _, st_v = eng_v.decode(max_new, uniforms=u)
                e1.record()
                torch.cuda.synchronize()
                ms_v += e0.elapsed_time(e1)
                for k in tot:
                    tot[k] += st_v.as_dict()[k]
            qv = report.run_quality(tot["drafted"], tot["accepted"], tot["emitted"])
            var[label] = {"tokens_per_s": round(tot["emitted"] / (ms_v * 1e-3), 2), "v_d": round(qv["v_d"], 4), "r_d": round(qv["r_d"], 4),
                          "mean_k": round(tot["drafted"] / max(1, tot["rounds"]), 3), "prompts": min(2, args.steps)}
            eng_v.close()
            del eng_v
            torch.cuda.empty_cache()
        line["variants"] = var
    if world == 1 and greedy and args.controller == "beta" and not args.no_70b and args.workload == "13b-eesd":
        line["shape_70b"] = leg_70b(device, peaks)
        line["verify_pass_frac_of_8tbs"]["70b"] = {k: v["frac_of_8tbs"] for k, v in line["shape_70b"]["verify_pass"].items()
                                                   if k.startswith("M")}
    print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
