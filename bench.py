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
# algorithmic bytes: from an ncu capture on the 0.5B-shaped workload, scaled to the timed workload by its
# algorithmic bytes (traffic grows with the bytes streamed).  None once the kernel has changed since the
# capture.
NCU_TRAFFIC_RATIO = 1.0039


NOMINAL_HBM_GBS = 8000.0   # the "about 8 TB/s" the target is worded against


def load_tflops():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return float(p.get("bf16_tflops_sustained", p.get("bf16_tflops", 1400.0))), "measured"
    return 1400.0, "fallback"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi (read-only queries) while the timed regions
    run.  Started before the warm-up so that even a short timed region has samples; samples taken while
    the GPU was idle (before the first launch) are dropped by the caller's `mark()`."""

    REASONS = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")

    def __init__(self, index: int, period_ms: int = 20):
        self.index, self.period_ms = index, period_ms
        self.rows, self.err, self.proc, self.thread, self.t_mark = [], "", None, None, None

    def _fields(self, prefix):
        return "clocks.sm,clocks.max.sm,power.draw," + ",".join(f"{prefix}.{r}" for r in self.REASONS)

    def start(self):
        for prefix in ("clocks_event_reasons", "clocks_throttle_reasons"):   # older drivers know the second name only
            try:
                probe = subprocess.run(["nvidia-smi", f"--query-gpu={self._fields(prefix)}", "--format=csv,noheader,nounits",
                                        "-i", str(self.index)], capture_output=True, text=True, timeout=20)
            except (OSError, subprocess.TimeoutExpired) as e:
                self.err = str(e)
                return
            if probe.returncode == 0 and "not a valid field" not in probe.stdout.lower():
                break
            self.err = (probe.stderr or probe.stdout).strip()[:200]
        else:
            return
        self.err = ""
        self.proc = subprocess.Popen(
            ["nvidia-smi", f"--query-gpu={self._fields(prefix)}", "--format=csv,noheader,nounits", "-lms",
             str(self.period_ms), "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True)
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 7:
                self.rows.append((time.perf_counter(), parts))

    def mark(self):
        """Samples from here on count (the GPU is under load from now)."""
        self.t_mark = time.perf_counter()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0,
                    "error": self.err}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for t, r in self.rows:
            if self.t_mark is not None and t < self.t_mark:
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for name, v in zip(self.REASONS, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "period_ms": self.period_ms}


def workload_string(cfg, k):
    """Names the workload; the GPU arm and the CPU reference arm print the same string."""
    return (f"{cfg.name}: {cfg.n_layers} layers d={cfg.d_model} {cfg.n_q_heads}q/{cfg.n_kv_heads}kv "
            f"hd={cfg.head_dim} ffn={cfg.d_ffn} vocab={cfg.vocab}; context {cfg.n_ctx} Zipf tokens "
            f"with planted repeats prefilled in {cfg.chunk}-token chunks; k={k} (n-gram drafter, "
            f"context search); verify steps of {k + 1} rows from KV length {cfg.n_ctx}")


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


def oracle_prefill_tokens(cfg):
    """Context tokens the CPU oracle prefills before its timed steps: the whole context where that takes the
    host cores tens of seconds (the workloads up to the 1.5B shape), else the first chunk only."""
    return cfg.n_ctx if cfg.linear_params() * cfg.n_ctx <= 4.0e12 else min(cfg.chunk, cfg.n_ctx)


def oracle_sample_string(cfg, k, n_steps, n_prefill, ms_per_step=None):
    txt = f"{n_steps} verify steps of {k + 1} rows from KV length {n_prefill}"
    if n_prefill != cfg.n_ctx:
        txt += f" (the oracle prefilled only the first {n_prefill} of {cfg.n_ctx} context tokens)"
    if ms_per_step is not None:
        txt += f"; {ms_per_step:.1f} ms per step"
    return txt + "; oracle prefill not timed"


def run_reference(args, cfg):
    from sdv_inputs import make_context, make_weights
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = len(os.sched_getaffinity(0))
    w = make_weights(cfg, threads=max(8, cores))
    ctx = make_context(cfg)
    n_prefill = oracle_prefill_tokens(cfg)
    total = args.warmup + args.steps
    tps, s_per_step, emitted = oracle_steps_per_sec(cfg, w, ctx, n_prefill, total, cfg.k)
    sample = oracle_sample_string(cfg, cfg.k, total, n_prefill, s_per_step * 1e3)
    line = {
        "impl": "reference", "metric": METRIC, "value": tps, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": s_per_step * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_string(cfg, cfg.k), "rows_per_verify": cfg.k + 1, "sample": sample,
                   "same_state_as_gpu_arm": n_prefill == cfg.n_ctx},
        "cpu_baseline": {"value": tps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": tps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def phase_timeline(s, cfg, k):
    """One profiled verify step: the kernel's own per-phase, per-block timestamps (%globaltimer) as a
    table.  dur = first block in to last block out; gap = grid barrier to the next phase."""
    names = ["QKV projection", "attention", "output projection", "gate|up + SwiGLU + down"]
    nph = 2 + 4 * cfg.n_layers
    s.debug_profile(True)
    s.draft(k, fetch=False)
    s.verify(None, fetch=False)
    s.commit()
    prof_us = s.last_verify_ms() * 1e3
    p = s.debug_profile(False, nph).astype(np.int64)
    st, en = p[:, :, 0], p[:, :, 1]
    rows = {}
    for ph in range(nph):
        m = en[ph] > 0
        a, d = st[ph][m].min(), en[ph][m].max()
        nxt = st[ph + 1][en[ph + 1] > 0].min() if ph + 1 < nph else d
        nm = "embedding" if ph == 0 else ("LM head + argmax" if ph == nph - 1 else names[(ph - 1) % 4])
        r = rows.setdefault(nm, {"dur": [], "gap": [], "marks": []})
        r["dur"].append((d - a) / 1e3)
        r["gap"].append((nxt - d) / 1e3)
        marks = []
        for wd in (2, 3, 4, 5, 6):       # per-role timestamps inside the phase, relative to its start
            x = p[ph][:, wd]
            mm = (x > 0) & m
            marks.append((float((x[mm].min() - a) / 1e3), float((x[mm].max() - a) / 1e3)) if mm.any() else None)
        r["marks"].append(marks)
    out = [f"verify step of {k + 1} rows, KV length {s.kv_len()}, {cfg.name}: {prof_us:.1f} us with the per-phase stamps on",
           "", "| phase | launches of it | dur us (mean) | gap us (mean) | marks inside the phase, us after its start: first block / last block |",
           "|---|---|---|---|---|"]
    legend = {"attention": ["loads issued", "Q tile and new rows ready", "first key block in place", "key loop done", "unit done"],
              "default": ["token operand built", "tensor-core warp done issuing", "epilogue done", "reached the down projection",
                          "SwiGLU operand complete"]}
    total = 0.0
    for nm, r in rows.items():
        lg = legend.get(nm, legend["default"])
        mk = []
        for i, name in enumerate(lg):
            vals = [x[i] for x in r["marks"] if x[i] is not None]
            if vals:
                mk.append(f"{name} {np.mean([v[0] for v in vals]):.1f} / {np.mean([v[1] for v in vals]):.1f}")
        total += sum(r["dur"]) + sum(r["gap"])
        out.append(f"| {nm} | {len(r['dur'])} | {np.mean(r['dur']):.2f} | {np.mean(r['gap']):.2f} | {'; '.join(mk)} |")
    out.append("")
    out.append(f"sum of dur + gap over all phases: {total:.1f} us")
    return "\n".join(out)


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
    ap.add_argument("--phase-timeline", action="store_true",
                    help="prints the per-phase timeline of one profiled verify step (a table) instead of the JSON line")
    ap.add_argument("--no-extras", action="store_true", help="skips the history-search and forced-acceptance loops")
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
    extras = not args.no_extras and not args.phase_timeline and world == 1
    max_seq = cfg.n_ctx + 2 * total * (k + 1) + 64          # room for two timed loops at full acceptance
    if args.extension:
        max_seq += total * (args.extension + 1)
    # forced acceptance: seeded accept lengths whose mean number of emitted tokens per step lies in the range
    # the paper reports for its 1.5B model (Table "ablation on accept length": 2.5 to 5.5 tokens per step)
    rng = np.random.default_rng(20251015)
    forced_a = [int(x) for x in np.minimum(rng.geometric(1.0 / 3.6, size=total) - 1, k)] if extras else []
    stream_len = sum(forced_a) + len(forced_a) + k + 2 if extras else 0
    max_seq = max(max_seq, cfg.n_ctx + stream_len + 2 * (k + 2) + 64)
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

    if args.phase_timeline:
        loop(max(args.warmup, 25), False)
        if rank == 0:
            print(phase_timeline(s, cfg, k), flush=True)
        s.close()
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- device-resident loop: the steps are enqueued as one run (sdv_decode_steps: KV length, history and drafts
    # pass from step to step on the device; one synchronisation at the end of the run)
    def run(n):
        em, _ = s.decode_steps(k, n)
        return len(em), [float(x) for x in s.run_kernel_ms(n)]

    # the period is only as short as 20 ms when the timed regions would otherwise end before the second sample
    sampler = ClockSampler(local, period_ms=20 if 2 * total * 1.5 < 400 else 200)
    sampler.start()                      # before the warm-up: the first samples arrive while it runs
    run(args.warmup)
    launches0 = s.launch_count()
    barrier()
    sampler.mark()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    tokens, kms = run(args.steps)
    ev1.record(stream)
    barrier()
    launches = s.launch_count() - launches0
    ms_total = ev0.elapsed_time(ev1)
    kv_end = s.kv_len()
    L_mid = (L0 + kv_end) // 2

    # ---- end-to-end loop with host buffers: one sdv_step call per step.  The host passes the draft in (H2D, as launch
    # parameters) and reads the emitted tokens, the KV length and the next draft back (D2H: one copy of the state block).
    def host_loop(n, d):
        tok = 0
        for _ in range(n):
            em, nd, _ = s.step(d, k)
            d = (nd + [0] * k)[:k]                   # same k+1 rows as the device-resident loop
            tok += len(em)
        return tok, d
    d0 = (s.draft(k) + [0] * k)[:k]
    _, d0 = host_loop(args.warmup, d0)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    tokens_e, _ = host_loop(args.steps, d0)
    e1.record(stream)
    barrier()
    ms_e2e = e0.elapsed_time(e1)
    clocks = sampler.stop()              # sampled over both timed loops (and the warm-up between them)

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

    # ---- the two other labelled throughput numbers (single-GPU runs only; synthetic acceptance)
    forced = hist_mode = prefill = batched = None
    if extras and world == 1:
        # (C) forced acceptance.  The greedy continuation comes from this path's own plain decoding (one token
        # per step, no oracle involved), recorded before the timed region; each timed step then verifies a
        # draft that agrees with it for a seeded number of tokens and is wrong right after.
        # Recorded in the launch shape of the timed steps (k + 1 rows, the drafts all wrong): the work partition,
        # and with it the rounding of a row, depends on the row count, and the crowded logits of random-init
        # weights would let a one-row recording part from the k+1-row steps at the first near-tie.
        s.rollback(L0)
        greedy = []
        while len(greedy) < stream_len:
            s.verify([(greedy[-1] + 1) % cfg.vocab if greedy else 0] * k, fetch=False)
            em, _ = s.commit(max_emit=1)
            greedy += em
        s.rollback(L0)

        def forced_loop(steps_a, pos):
            toks, kms_f, hits = 0, [], 0
            for a_t in steps_a:
                d = (greedy[pos:pos + a_t] + [(greedy[pos + a_t] + 1) % cfg.vocab] * (k - a_t))[:k]
                before = s.kv_len()
                s.verify(d, fetch=False)
                em, _ = s.commit()
                toks += len(em)
                kms_f.append(s.last_verify_ms())
                if em == greedy[pos:pos + a_t + 1]:
                    hits += 1
                else:
                    # a near-tie fell the other way (fp32 reduction order differs from run to run): the step's own
                    # tokens are counted, then the sequence is put back on the recorded continuation (the KV rows
                    # the step wrote belong to the same tokens) so that the later steps keep their accept lengths
                    s.rollback(before)
                    s.debug_accept(d, greedy[pos:pos + k + 1])
                    s.commit()
                pos += a_t + 1
            return toks, kms_f, pos, hits
        _, _, pos, _ = forced_loop(forced_a[:args.warmup], 0)
        torch.cuda.synchronize()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(stream)
        toks_f, kms_f, pos, hits = forced_loop(forced_a[args.warmup:], pos)
        f1.record(stream)
        torch.cuda.synchronize()
        ms_f = f0.elapsed_time(f1)
        forced = {"label": "synthetic: drafts forced to agree with the model's own greedy continuation for a seeded "
                           "number of tokens (geometric, mean emitted 3.6 per step, the range of the paper's accept-length "
                           "table for its 1.5B model); random-init weights accept nothing on their own",
                  "value": toks_f / (ms_f * 1e-3), "unit": UNIT, "ms_per_step": ms_f / args.steps,
                  "emitted_per_step": toks_f / args.steps, "steps_with_the_forced_accept_length": hits,
                  "verify_kernel_us": statistics.mean(kms_f) * 1e3}
        # (B) the drafter also searches the generated tokens (search_history): a second context of the same model;
        # its prefill is the timed prefill number
        # chunked prefill of the whole context on a fresh context: the dense path (tokens on the tensor cores' M side)
        s.close()
        s = Sdv(config_from(cfg, k_max=k_max, max_seq=max_seq, search_history=True), stream=stream)
        s.load_weights(w)
        torch.cuda.synchronize()
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0 = s.launch_count()
        p0.record(stream)
        for i in range(0, cfg.n_ctx, cfg.chunk):
            s.prefill_chunk(ctx[i:i + cfg.chunk], is_last=(i + cfg.chunk >= cfg.n_ctx))
        p1.record(stream)
        torch.cuda.synchronize()
        ms_p = p0.elapsed_time(p1)
        lin = 2.0 * (cfg.linear_params() - cfg.vocab * cfg.d_model) * cfg.n_ctx   # the LM head runs on the last row only
        att = 4.0 * cfg.n_layers * cfg.n_q_heads * cfg.head_dim * (cfg.n_ctx * (cfg.n_ctx + 1) / 2.0)
        tf = load_tflops()
        prefill = {"label": f"chunked prefill of the {cfg.n_ctx}-token context in {cfg.chunk}-token chunks (host loop included: "
                            "one call per chunk, each synchronises)",
                   "ms": ms_p, "tokens_per_sec": cfg.n_ctx / (ms_p * 1e-3), "launches": s.launch_count() - l0,
                   "tflops_linear": lin / (ms_p * 1e-3) / 1e12, "tflops_linear_plus_attention": (lin + att) / (ms_p * 1e-3) / 1e12,
                   "bf16_peak_tflops": tf[0], "peak_kind": f"of {tf[1]} (sustained)",
                   "frac": (lin + att) / (ms_p * 1e-3) / 1e12 / tf[0]}
        run(args.warmup)
        torch.cuda.synchronize()
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record(stream)
        toks_h, kms_h = run(args.steps)
        h1.record(stream)
        torch.cuda.synchronize()
        ms_h = h0.elapsed_time(h1)
        hist_mode = {"label": "drafter searches the request context and the generated tokens (search_history)",
                     "value": toks_h / (ms_h * 1e-3), "unit": UNIT, "ms_per_step": ms_h / args.steps,
                     "emitted_per_step": toks_h / args.steps, "verify_kernel_us": statistics.mean(kms_h) * 1e3}

        # batched verify: further sequences (their own contexts, the same length) read this context's weights and
        # share every pass over them; aggregate tokens/s over the sequences of the batch
        n_seq = min(3, 32 // (k + 1))
        if n_seq >= 2:
            fols = [s.follower() for _ in range(n_seq - 1)]
            for i, fo in enumerate(fols):
                fctx = make_context(cfg, seed=cfg.seed + 1 + i)
                for j in range(0, cfg.n_ctx, cfg.chunk):
                    fo.prefill_chunk(fctx[j:j + cfg.chunk], is_last=(j + cfg.chunk >= cfg.n_ctx))
            seqs = [s] + fols

            def batch_loop(n):
                toks, kms_b = 0, []
                for _ in range(n):
                    for q in seqs:
                        q.draft(k, fetch=False)
                    Sdv.verify_batch(seqs, fetch=False)
                    for q in seqs:
                        em, _ = q.commit()
                        toks += len(em)
                    kms_b.append(s.last_verify_ms())
                return toks, kms_b
            batch_loop(args.warmup)
            torch.cuda.synchronize()
            b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            b0.record(stream)
            toks_b, kms_b = batch_loop(args.steps)
            b1.record(stream)
            torch.cuda.synchronize()
            ms_b = b0.elapsed_time(b1)
            wb_b, _ = s.step_bytes(k + 1, L0)
            kv_b = sum(q.step_bytes(k + 1, q.kv_len())[1] for q in seqs)
            gbs_b = (wb_b + kv_b) / (statistics.mean(kms_b) * 1e-3) / 1e9
            batched = {"label": f"{n_seq} sequences per verify step (sdv_verify_batch): one pass over the weights for "
                                f"{n_seq * (k + 1)} rows, each sequence its own context, KV cache and search_history drafter",
                       "sequences": n_seq, "rows_per_verify": n_seq * (k + 1),
                       "value": toks_b / (ms_b * 1e-3), "unit": UNIT, "ms_per_step": ms_b / args.steps,
                       "emitted_per_step": toks_b / args.steps, "verify_kernel_us": statistics.mean(kms_b) * 1e3,
                       "GB/s": gbs_b, "frac": gbs_b / load_peaks()[0]}
            for fo in fols:
                fo.close()

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
                "workload": workload_string(cfg, k),
                "rows_per_verify": k + 1, "replicas": world, "kv_len_range": [L0, kv_end],
                "l2": "inputs larger than L2: every step streams all weights (>= 1 GB) once",
                "accepted_drafts_per_step": tokens_all / (args.steps * world) - 1.0,
            },
            "verify_kernel_us": kernel_ms * 1e3,
            "verify_kernel_us_p10_p90": [float(np.percentile(kms, 10)) * 1e3, float(np.percentile(kms, 90)) * 1e3],
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "peak_kind": f"of {peak_kind}", "frac_nominal": achieved / NOMINAL_HBM_GBS,
                         "nominal_peak": NOMINAL_HBM_GBS, "bytes_per_launch": wbytes + kvbytes,
                         "traffic": None if NCU_TRAFFIC_RATIO is None else (wbytes + kvbytes) * NCU_TRAFFIC_RATIO,
                         "traffic_source": "ncu capture on the 0.5B-shaped workload, scaled by algorithmic bytes",
                         "kernel": "sdv_forward_kernel"},
            "e2e": {"value": tokens_e_all / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 4 * k + 4,
                    "d2h_bytes_per_step": 1280},
            "gpu_launches": launches,
            "clocks": clocks,
        }
        line["config"]["tokens_per_sec_variants"] = ("value: n-gram drafter over the request context (accepts ~0 with "
                                                     "random-init weights); history: search_history drafter; "
                                                     "forced_acceptance: synthetic accept lengths")
        if forced:
            line["forced_acceptance"] = forced
        if hist_mode:
            line["history"] = hist_mode
            line["prefill"] = prefill
        if batched:
            line["batched"] = batched
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
            n_prefill = oracle_prefill_tokens(cfg)
            n_steps = 48 if cfg.linear_params() < 1.0e9 else (24 if cfg.linear_params() < 4.0e9 else 8)
            tps, sps, _ = oracle_steps_per_sec(cfg, w, ctx, n_prefill, n_steps, k)
            line["cpu_baseline"] = {
                "value": tps, "unit": UNIT, "cores": cores, "kind": "oracle",
                "sample": oracle_sample_string(cfg, k, n_steps, n_prefill, sps * 1e3),
            }
        print(json.dumps(line), flush=True)
    s.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
