#!/usr/bin/env python
"""Benchmark of the speculative-decoding verify path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl reference]

One step = one pass of the whole hot path on one sequence: n-gram draft, verify (one forward pass
over the pending token plus k drafts against the KV cache, greedy tokens, accept scan), commit.
The default workload is the Qwen2.5-1.5B-shaped decoder (random-init weights, synthetic Zipf
context of 2048 tokens prefilled in 256-token chunks, k = 8).  Several GPUs run independent
replicas of the same workload (the path does not shard: no collective).

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "generated_tokens_per_sec"
UNIT = "tokens/s"
# dram__bytes_read.sum + dram__bytes_write.sum per launch of sdv_forward_kernel, as a multiple of the
# algorithmic bytes: captured on the 0.5B-shaped workload (profiles/sdv_forward_kernel_qwen0.5b_ncu_full.md)
# and scaled to the timed workload by its algorithmic bytes (traffic grows with the bytes streamed).
# None once the kernel has changed since the capture.
NCU_TRAFFIC_RATIO = 1.0051


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 7:
                self.rows.append(parts)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_steps_per_sec(cfg, weights, ctx, n_prefill, n_steps, k):
    """The CPU oracle as it stands on a bounded sample: prefill n_prefill context tokens, then time
    n_steps verify steps of k+1 rows (n-gram draft, forward, greedy tokens, accept)."""
    from oracle import sdv_oracle as O
    m = O.OracleModel(weights)
    sub = ctx[:n_prefill]
    last = m.prefill(sub, cfg.chunk)
    T = O.argmax(last)
    hist = [int(t) for t in sub] + [T]
    L = n_prefill
    emitted_total = 0
    t0 = time.perf_counter()
    for _ in range(n_steps):
        draft = O.ngram_draft(sub, hist, cfg.ngram_n, cfg.ngram_min, k)[0].tolist()
        draft = (draft + [0] * k)[:k]            # fixed k+1 rows, as the GPU path computes
        logits = m.forward([T] + draft, L, logits_from=0)
        y = [O.argmax(logits[j]) for j in range(k + 1)]
        a = O.accept_len(draft, y)
        em = draft[:a] + [y[a]]
        hist.extend(em)
        L += len(em)
        T = em[-1]
        emitted_total += len(em)
    dt = time.perf_counter() - t0
    return emitted_total / dt, dt / n_steps, emitted_total


def aggregate_over_ranks(times_ms, counts, world, device):
    """Replicas only: the job's time is the slowest rank's (MAX), its work the sum over ranks (SUM).
    Needs an initialised process group when world > 1 (any backend); returns two lists of floats."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    c = torch.tensor(list(counts), dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return t.tolist(), c.tolist()


def run_reference(args, cfg):
    from sdv_inputs import make_context, make_weights
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = len(os.sched_getaffinity(0))
    w = make_weights(cfg, threads=max(8, cores))
    ctx = make_context(cfg)
    n_prefill = min(cfg.chunk, cfg.n_ctx)
    total = args.warmup + args.steps
    tps, s_per_step, emitted = oracle_steps_per_sec(cfg, w, ctx, n_prefill, total, cfg.k)
    sample = (f"{total} verify steps of {cfg.k + 1} rows after prefilling the first {n_prefill} context tokens "
              f"(KV length {n_prefill}+, not {cfg.n_ctx}+)")
    line = {
        "impl": "reference", "metric": METRIC, "value": tps, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": s_per_step * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: {cfg.n_layers} layers d={cfg.d_model}, k={cfg.k}", "sample": sample},
        "cpu_baseline": {"value": tps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": tps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", default="qwen1.5b")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--k", type=int, default=0)
    ap.add_argument("--sweep-k", default="", help="comma-separated draft lengths: adds verify-step us and GB/s per k "
                                                 "at the fixed KV length reached after prefill (rolled back after each step)")
    ap.add_argument("--extension", type=int, default=0, metavar="MAX_TOTAL",
                    help="adds a third timed loop with draft extension (Sec. 4.4): drafts grow to at most MAX_TOTAL "
                         "tokens by reuse of rejected drafts; reported under \"extension\"")
    ap.add_argument("--extension-life", type=int, default=32)
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    from sdv_inputs import get_config, make_context, make_weights
    cfg = get_config(args.config)
    if args.k:
        cfg = cfg.with_(k=args.k)
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    import torch.distributed as dist
    from paper_2510_15312_b200.binding import Sdv, config_from

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    k = cfg.k
    sweep = [int(x) for x in args.sweep_k.split(",") if x.strip()]
    k_max = max([k] + sweep + [args.extension])
    total = args.warmup + args.steps
    max_seq = cfg.n_ctx + 2 * total * (k + 1) + 64          # room for two timed loops at full acceptance
    if args.extension:
        max_seq += total * (args.extension + 1)
    cores = len(os.sched_getaffinity(0))
    w = make_weights(cfg, threads=max(8, cores // max(1, world)))
    ctx = make_context(cfg)
    stream = torch.cuda.Stream()
    s = Sdv(config_from(cfg, k_max=k_max, max_seq=max_seq), stream=stream)
    s.load_weights(w)
    for i in range(0, cfg.n_ctx, cfg.chunk):
        s.prefill_chunk(ctx[i:i + cfg.chunk], is_last=(i + cfg.chunk >= cfg.n_ctx))
    L0 = s.kv_len()

    def sweep_point(kk, n):
        """n verify steps of kk+1 rows at KV length L0 (nothing committed): mean forward-kernel ms."""
        draft = [int(t) for t in ctx[:kk]]
        ms = []
        for i in range(n + 3):
            s.verify(draft, fetch=False)
            s.rollback(L0)
            if i >= 3:
                ms.append(s.last_verify_ms())
        return statistics.mean(ms)

    sweep_ms = {kk: sweep_point(kk, max(10, args.steps // 4)) for kk in sweep}

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def loop(n, host_buffers):
        """n steps; returns (tokens emitted, list of forward-kernel ms)."""
        tokens, kms = 0, []
        for _ in range(n):
            if host_buffers:
                d = s.draft(k)                       # D2H: the draft
                d = (d + [0] * k)[:k]                # same k+1 rows as the device-resident loop
                s.verify(d)                          # H2D: drafts; D2H: y, accept length
            else:
                s.draft(k, fetch=False)
                s.verify(None, fetch=False)
            em, _ = s.commit()                       # D2H: emitted tokens, KV length
            tokens += len(em)
            kms.append(s.last_verify_ms())
        return tokens, kms

    # ---- device-resident loop
    loop(args.warmup, False)
    sampler = ClockSampler(local)
    launches0 = s.launch_count()
    barrier()
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    tokens, kms = loop(args.steps, False)
    ev1.record(stream)
    barrier()
    clocks = sampler.stop()
    launches = s.launch_count() - launches0
    ms_total = ev0.elapsed_time(ev1)
    L_mid = (L0 + s.kv_len()) // 2

    # ---- end-to-end loop with host buffers
    loop(args.warmup, True)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    tokens_e, _ = loop(args.steps, True)
    e1.record(stream)
    barrier()
    ms_e2e = e0.elapsed_time(e1)

    # ---- optional: device-resident loop with draft extension (every step computes MAX_TOTAL + 1 rows)
    ext = None
    if args.extension:
        def ext_loop(n):
            tokens, kms = 0, []
            for _ in range(n):
                s.draft(k, fetch=False)
                s.extend_draft(args.extension, fetch=False)
                s.verify(None, fetch=False)
                s.extension_update(args.extension_life, fetch=False)
                em, _ = s.commit()
                tokens += len(em)
                kms.append(s.last_verify_ms())
            return tokens, kms
        ext_loop(args.warmup)
        barrier()
        x0, x1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        x0.record(stream)
        tokens_x, kms_x = ext_loop(args.steps)
        x1.record(stream)
        barrier()
        ms_x = x0.elapsed_time(x1)
        ext = {"max_total": args.extension, "max_life": args.extension_life, "rows_per_verify": args.extension + 1,
               "value": tokens_x / (ms_x * 1e-3), "unit": UNIT, "ms_per_step": ms_x / args.steps,
               "verify_kernel_us": statistics.mean(kms_x) * 1e3,
               "accepted_drafts_per_step": tokens_x / args.steps - 1.0, "scope": "rank 0"}

    (ms_total, ms_e2e), (tokens_all, tokens_e_all) = aggregate_over_ranks([ms_total, ms_e2e], [tokens, tokens_e], world,
                                                                          "cuda")

    if rank == 0:
        peak, peak_kind = load_peaks()
        wbytes, kvbytes = s.step_bytes(k + 1, L_mid)
        kernel_ms = statistics.mean(kms)
        achieved = (wbytes + kvbytes) / (kernel_ms * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": tokens_all / (ms_total * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {
                "workload": (f"{cfg.name}: {cfg.n_layers} layers d={cfg.d_model} {cfg.n_q_heads}q/{cfg.n_kv_heads}kv "
                             f"hd={cfg.head_dim} ffn={cfg.d_ffn} vocab={cfg.vocab}; context {cfg.n_ctx} Zipf tokens "
                             f"with planted repeats prefilled in {cfg.chunk}-token chunks; k={k} (n-gram drafter, "
                             f"context search); KV length {L0}..{s.kv_len()}"),
                "rows_per_verify": k + 1, "replicas": world,
                "l2": "inputs larger than L2: every step streams all weights (>= 1 GB) once",
                "accepted_drafts_per_step": tokens_all / (args.steps * world) - 1.0,
            },
            "verify_kernel_us": kernel_ms * 1e3,
            "verify_kernel_us_p10_p90": [float(np.percentile(kms, 10)) * 1e3, float(np.percentile(kms, 90)) * 1e3],
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "peak_kind": f"of {peak_kind}", "bytes_per_launch": wbytes + kvbytes,
                         "traffic": None if NCU_TRAFFIC_RATIO is None else (wbytes + kvbytes) * NCU_TRAFFIC_RATIO,
                         "traffic_source": "ncu capture on the 0.5B-shaped workload, scaled by algorithmic bytes",
                         "kernel": "sdv_forward_kernel"},
            "e2e": {"value": tokens_e_all / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 4 * k + 4,
                    "d2h_bytes_per_step": 3 * 640},
            "gpu_launches": launches,
            "clocks": clocks,
        }
        if ext:
            line["extension"] = ext
        if sweep:
            line["k_sweep"] = []
            for kk in sweep:
                wb, kb = s.step_bytes(kk + 1, L0)
                gbs = (wb + kb) / (sweep_ms[kk] * 1e-3) / 1e9
                line["k_sweep"].append({"k": kk, "kv_len": L0, "verify_kernel_us": sweep_ms[kk] * 1e3, "GB/s": gbs,
                                        "frac": gbs / peak})
        if world == 1 and not args.no_cpu_baseline:
            n_prefill = min(cfg.chunk, cfg.n_ctx)
            n_steps = 48 if cfg.linear_params() < 1.0e9 else (24 if cfg.linear_params() < 4.0e9 else 8)
            tps, sps, _ = oracle_steps_per_sec(cfg, w, ctx, n_prefill, n_steps, k)
            line["cpu_baseline"] = {
                "value": tps, "unit": UNIT, "cores": cores, "kind": "oracle",
                "sample": (f"{n_steps} verify steps of {k + 1} rows after prefilling the first {n_prefill} context "
                           f"tokens; {sps * 1e3:.1f} ms per step"),
            }
        print(json.dumps(line), flush=True)
    s.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
