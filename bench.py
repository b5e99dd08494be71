#!/usr/bin/env python
"""Benchmark of the batched N-gram speculation step on B200.

One *step* = draft_context_ngrams -> verify_lmhead_argmax -> accept_and_commit over one batch of
synthetic sequences (hidden states are an input: the transformer body is outside this library).
The model bigram table is a one-off build and is timed separately (reported under "table_build").

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C5] [--impl ours|reference]

Prints ONE JSON line.  The headline numbers (value, ms_per_step, e2e, roofline) are those of
`--workload` (default: the long-context configuration, the largest one); the other configurations are
measured in the same run and reported as `per_config`.  With `--gpus N` and no launcher (WORLD_SIZE
unset) the script starts N ranks itself, one process per GPU; under torchrun it is one of the ranks.
`--impl reference` times the plain CPU oracle on the host cores instead.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth  # noqa: E402

METRIC = "accepted_tokens_per_s"
UNIT = "tokens/s"
RHO = 0.55  # planted acceptance: P(accepted length >= j) = RHO^j  (about 2.2 tokens per call)
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}   # NVIDIA's B200 figures (dense), for the second denominator
MIN_TIMED_S = 0.2                                      # blocks of `steps` steps are repeated until this much was timed
KERNEL_SOURCES = ["paper_2411_03786_b200/csrc/head_gemm.cu", "paper_2411_03786_b200/csrc/common.cuh",
                  "paper_2411_03786_b200/csrc/accept.cuh"]


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=d["hbm_gbs"], tc_burst=d["bf16_tflops"], tc_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]),
                    source="measured")
    return dict(hbm=6650.0, tc_burst=1590.0, tc_sustained=1400.0, source="fallback")


def kernel_source_hash():
    h = hashlib.sha256()
    for f in KERNEL_SOURCES:
        h.update(open(os.path.join(ROOT, f), "rb").read())
    return h.hexdigest()[:12]


def dram_traffic(workload, kernel):
    """DRAM bytes per launch (read + write) from the ncu captures summarised in profiles/dram_traffic.md.
    A row counts only while the kernel sources still hash to the value recorded with the capture."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.md")
    if not os.path.exists(path):
        return None
    now = kernel_source_hash()
    for line in open(path):
        cells = [x.strip().strip("`") for x in line.strip().strip("|").split("|")]
        if len(cells) >= 5 and cells[0] == workload and cells[1] == kernel:
            try:
                return float(cells[2]) if cells[4] == now else None
            except ValueError:
                return None
    return None


def bf16_bits(w):
    return synth.f32_to_bf16_bits(w) if w.dtype == np.float32 else w


class ClockSampler:
    """Samples SM clocks and throttle reasons while the timed region runs (NVML, read-only; falls back
    to nvidia-smi)."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index):
        self.index, self.rows, self._stop = index, [], threading.Event()
        self.t = threading.Thread(target=self._run, daemon=True)
        self.nvml = None
        try:
            import pynvml
            pynvml.nvmlInit()
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = int(vis.split(",")[index]) if vis and all(x.strip().isdigit() for x in vis.split(",")) else index
            self.h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.nvml = pynvml
        except Exception:
            self.nvml = None

    def _sample_nvml(self):
        n = self.nvml
        mhz = float(n.nvmlDeviceGetClockInfo(self.h, n.NVML_CLOCK_SM))
        r = int(n.nvmlDeviceGetCurrentClocksEventReasons(self.h)) if hasattr(n, "nvmlDeviceGetCurrentClocksEventReasons") \
            else int(n.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
        bits = [0x8, 0x40, 0x20, 0x4]      # hw slowdown, hw thermal, sw thermal, sw power cap
        self.rows.append([mhz, self.max_mhz] + [bool(r & b) for b in bits])

    def _sample_smi(self):
        out = subprocess.run(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                              "-i", str(self.index)], capture_output=True, text=True, timeout=5).stdout.strip()
        if out:
            f = [x.strip() for x in out.splitlines()[0].split(",")]
            self.rows.append([float(f[0]), float(f[1])] + [x.lower().startswith("active") for x in f[2:6]])

    def _run(self):
        while not self._stop.is_set():
            try:
                self._sample_nvml() if self.nvml else self._sample_smi()
            except Exception:
                pass
            self._stop.wait(0.002 if self.nvml else 0.1)

    def __enter__(self):
        self.t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self.t.join(timeout=6)

    def summary(self):
        if not self.rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        reasons = [n for i, n in enumerate(self.NAMES) if any(r[2 + i] for r in self.rows)]
        return {"sm_mhz": statistics.median(r[0] for r in self.rows), "sm_max_mhz": max(r[1] for r in self.rows),
                "reasons": reasons, "samples": len(self.rows), "source": "nvml" if self.nvml else "nvidia-smi"}


# ----------------------------------------------------------------------------------------------- CPU oracle leg
def oracle_step_time(c, hist, lens, T, H_bits, W_bits, budget_s, min_steps=1, max_steps=50):
    """Times the oracle's step as it stands.  Verification is the costly part; when a full step would
    exceed the budget the verify rows are sampled and the time is scaled to all M rows."""
    import oracle
    M = H_bits.shape[0]
    t0 = time.perf_counter()
    oracle.verify(H_bits, W_bits, rows=[0])
    per_row = time.perf_counter() - t0
    threads = oracle.num_threads()
    est_full = per_row * M / max(1, min(threads, M))
    rows = None
    scale = 1.0
    if est_full > budget_s / 2:
        n = int(max(threads, min(M, (budget_s / 2) / per_row * threads)))
        n = max(threads, n // threads * threads)
        if n < M:
            rows = np.linspace(0, M - 1, n).astype(np.int64)
            scale = M / n
    steps, total, accepted = 0, 0.0, 0
    while steps < min_steps or (total < budget_s and steps < max_steps):
        h, l = hist.copy(), lens.copy()
        t0 = time.perf_counter()
        drafts, nd, _, _ = oracle.draft_batch(h, l, c["qs"], c["topk"], c["B"], c["w"], 3, T)
        t1 = time.perf_counter()
        am, _, _ = oracle.verify(H_bits, W_bits, rows=rows)
        t2 = time.perf_counter()
        if rows is not None:
            full = np.zeros(M, np.int32)
            full[rows] = am
            am = full
        acc, _, _ = oracle.accept_commit(drafts, nd, am.reshape(c["S"], c["B"], c["w"] + 1), h, l)
        t3 = time.perf_counter()
        total += (t1 - t0) + (t2 - t1) * scale + (t3 - t2)
        accepted += int((acc + 1).sum())
        steps += 1
    sample = (f"{steps} full oracle steps (draft + verify of all {M} rows + accept)" if rows is None else
              f"{steps} oracle steps with verify on {len(rows)} of {M} rows, verify time scaled by {scale:.1f}")
    return total / steps, accepted / steps, threads, sample, rows is not None


def ev(torch):
    return torch.cuda.Event(enable_timing=True)


def scaled_streams(ctx, torch, dev, c, pk):
    """Streaming rates of the integer kernels on batches large enough to measure bandwidth (at the
    benchmark sizes they move a few KB and are launch-latency-bound)."""
    out = {}

    def timed(fn, reps):
        # warm up under the kernel's own load for 50 ms: these kernels are bound by latency and instruction issue,
        # so they follow the SM clock, and directly after a table build or a block of verify steps the clock is
        # still the power-capped one of that work
        t_warm, n_warm = time.time(), 0
        while n_warm < 3 or time.time() - t_warm < 0.05:
            fn()
            n_warm += 1
            if n_warm % 8 == 0:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        a, b = ev(torch), ev(torch)
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    # shaped like C3 (V = 32000, Zipf 1.1) and like C5 (V = 128256, Zipf 1.05); the third entry keeps the 32000-token
    # vocabulary on the long histories (more matches per sequence)
    for S, L, qs, reps, Vz, zz, tag in ((4096, 2048, (3, 2, 1), 20, 32000, 1.1, ""), (512, 131072, (3, 2), 5, 128256, 1.05, ""),
                                        (512, 131072, (3, 2), 5, 32000, 1.1, "_V32000"),
                                        # eight rounds of 148 sequences instead of 3.46: the launch's fixed costs weigh less
                                        (1184, 131072, (3, 2), 5, 128256, 1.05, "_8rounds")):
        if ctx.V < Vz:
            continue
        base, lens_b, _ = synth.zipf_histories(32, L, Vz, zz, 0.3, seed=77, cap=L + 64, name="scaled")
        hist = torch.from_numpy(np.tile(base, (S // 32, 1))).to(dev)
        lens = torch.from_numpy(np.tile(lens_b, S // 32)).to(dev)
        assert hist.shape[0] == S
        B, w, topk = 16, 8, 4
        bufs = (torch.empty((S, B, w), dtype=torch.int32, device=dev), torch.empty(S, dtype=torch.int32, device=dev),
                torch.empty((S, B), dtype=torch.int32, device=dev), torch.empty((S, B), dtype=torch.int32, device=dev))
        ms = timed(lambda: ctx.draft_context_ngrams(hist, lens, qs, topk, B, w, out=bufs), reps)
        by = 4.0 * S * L + 4.0 * S * B * (w + 2) + 8.0 * S
        ix_ms = None
        if not tag:   # the same batch drafted from the incremental context index (built once, outside the timing)
            index = ctx.context_index_build(hist, lens, qs, w)
            ix_ms = timed(lambda: ctx.draft_context_ngrams_indexed(index, hist, lens, qs, topk, B, w, out=bufs), reps)
            del index
        out[f"draft_S{S}_L{L}{tag}"] = {"qs": list(qs), "vocabulary": Vz, "zipf": zz, "ms": ms, "ms_from_context_index": ix_ms, "GB/s": by / ms / 1e6, "frac_of_hbm": by / ms / 1e6 / pk["hbm"],
                                   "frac_of_nominal_hbm": by / ms / 1e6 / NOMINAL["hbm_gbs"], "bytes": by,
                                   "l2": "larger than L2" if by > 126e6 else "L2-resident"}
        del hist, lens, bufs
    # acceptance where every byte has to be read: every draft row is accepted in full (drafts equal the
    # predictions), so no prefix comparison stops early
    S, B, w = 65536, 64, 10
    g = torch.Generator(device=dev).manual_seed(3)
    P = torch.randint(0, 1000, (S, B, w + 1), device=dev, dtype=torch.int32, generator=g)
    drafts = P[:, :, :w].contiguous()
    nd = torch.full((S,), B, dtype=torch.int32, device=dev)
    cap = 64
    hist = torch.zeros((S, cap), dtype=torch.int32, device=dev)
    lens0 = torch.full((S,), 8, dtype=torch.int32, device=dev)
    lens = lens0.clone()
    bufs = (torch.empty(S, dtype=torch.int32, device=dev), torch.empty(S, dtype=torch.int32, device=dev),
            torch.empty((S, w + 1), dtype=torch.int32, device=dev))

    def acc():
        ctx.accept_and_commit(drafts, nd, P, hist, lens, out=bufs)

    def acc_reset():
        lens.copy_(lens0)

    # the length reset is timed on its own and taken off
    ms_both = timed(lambda: (acc_reset(), acc()), 10)
    ms_reset = timed(acc_reset, 10)
    ms = ms_both - ms_reset
    assert int(bufs[0].min()) == w and int(bufs[0].max()) == w, "the full-acceptance batch was not accepted in full"
    by = 4.0 * S * B * (2 * w + 1) + 4.0 * S * (1 + 1) + 4.0 * S * (w + 1) + 4.0 * S * (w + 1) + 4.0 * S * 3
    out[f"accept_S{S}_B{B}_w{w}"] = {"ms": ms, "GB/s": by / ms / 1e6, "frac_of_hbm": by / ms / 1e6 / pk["hbm"],
                                    "frac_of_nominal_hbm": by / ms / 1e6 / NOMINAL["hbm_gbs"], "bytes": by,
                                    "workload": "every row accepted in full: all drafts and predictions are read",
                                    "l2": "larger than L2"}
    return out


# ----------------------------------------------------------------------------------------------- one configuration
class Head:
    """Weights, context and model table of one head (C2 and C3 share one, C4 and C5 the other)."""

    def __init__(self, torch, ngs, c, dev, pk, time_table):
        self.E = synth.gaussian_weights(c["V"], c["d"], c["wstd"], c["wseed"], "E", c["wdtype"])
        self.W = synth.gaussian_weights(c["V"], c["d"], c["wstd"], c["wseed"], "W", c["wdtype"])
        to_dev = (lambda w: torch.from_numpy(w).to(dev)) if c["wdtype"] == "f32" else \
            (lambda w: torch.from_numpy(w.view(np.int16)).view(torch.bfloat16).to(dev))
        self.dE, self.dW = to_dev(self.E), to_dev(self.W)
        self.ctx = ngs.SpecContext(self.dE, self.dW)
        self.W_bits = bf16_bits(self.W)
        self.k_tab = c["k_tab"]
        w_ext = 10 if c["V"] > 2048 else c["w"]
        self.tab, _, self.ext = self.ctx.build_model_ngram_tables(c["k_tab"], w_ext=w_ext)
        torch.cuda.synchronize()
        self.table = {}
        self.fp8_ready = False
        if time_table:
            reps = 3 if c["V"] <= 40000 else 2
            ts = []
            for _ in range(reps):
                a, b = ev(torch), ev(torch)
                a.record()
                self.ctx.build_model_ngram_tables(c["k_tab"], w_ext=w_ext)
                b.record()
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b))
            ms = min(ts)
            fl = 2.0 * c["V"] * c["V"] * c["d"]
            a, b = ev(torch), ev(torch)
            self.ctx.build_model_unigram(25)
            a.record()
            self.ctx.build_model_unigram(25)
            b.record()
            torch.cuda.synchronize()
            uni_ms = a.elapsed_time(b)
            tf = fl / ms / 1e9
            self.table = {"head": f"V={c['V']} d={c['d']} k_tab={c['k_tab']}", "ms": ms, "ms_all_repeats": ts, "tflops": tf,
                          "frac_of_burst_peak": tf / pk["tc_burst"], "frac_of_sustained_peak": tf / pk["tc_sustained"],
                          "frac_of_nominal_peak": tf / NOMINAL["bf16_tflops"], "target": "60 % of the bf16 tensor peak",
                          "meets_target_vs_measured_burst": tf / pk["tc_burst"] >= 0.6,
                          "meets_target_vs_nominal": tf / NOMINAL["bf16_tflops"] >= 0.6,
                          "unigram_ms": uni_ms, "unigram_tflops": fl / uni_ms / 1e9, "flops": fl, "peak_source": pk["source"],
                          "includes": "contraction with fused top-k, merge of the per-chunk lists, extension table"}


def measure_config(torch, ngs, c, head, dev, pk, args, rank, dist, headline):
    """Times one configuration.  Returns the record and what the end-to-end / CPU legs need."""
    ctx = head.ctx
    S, B, w, M = c["S"], c["B"], c["w"], c["M"]
    hist_h, lens_h, copied = synth.zipf_histories(S, c["L"], c["V"], c["zipf"], c["copy"], c["seed"], cap=c["L"] + 64,
                                                  name=f"hist/rank{rank}")
    hist, lens0 = torch.from_numpy(hist_h).to(dev), torch.from_numpy(lens_h).to(dev)
    out_d = ctx.draft_context_ngrams(hist, lens0.clone(), c["qs"], c["topk"], B, w)
    torch.cuda.synchronize()
    drafts0, nd0 = out_d[0].cpu().numpy(), out_d[1].cpu().numpy()
    targets, _, _ = synth.planted_targets(drafts0, nd0, None, c["V"], c["zipf"], RHO, seed=c["seed"] + 100 * rank)
    H_bits = synth.hidden_planted(head.W_bits, targets.reshape(-1), seed=c["seed"] + 100 * rank)
    dH = torch.from_numpy(H_bits.view(np.int16)).view(torch.bfloat16).to(dev)
    out_v = (torch.empty(M, dtype=torch.int32, device=dev), None)
    out_a = (torch.empty(S, dtype=torch.int32, device=dev), torch.empty(S, dtype=torch.int32, device=dev),
             torch.empty((S, w + 1), dtype=torch.int32, device=dev))

    # Every step sees the same history: step k of a round works on its own copy of the lengths, and one
    # small copy per round of R steps restores all of them.  (A reset before every step would sit between
    # accept and the next draft and break the dependent-launch chain that a real decode loop has there.)
    K = args.steps
    R = max(r for r in range(1, 17) if K % r == 0)
    lens_all = lens0.unsqueeze(0).repeat(R, 1).contiguous()
    lens0_all = lens_all.clone()

    def step(fused, timers=None, k=0):
        lens = lens_all[k]
        if timers:
            lens.copy_(lens0)
            timers[0].record()
        ctx.draft_context_ngrams(hist, lens, c["qs"], c["topk"], B, w, out=out_d)
        if timers:
            timers[1].record()
        if fused and not timers:   # verify + accept in one launch
            ctx.verify_accept_commit(dH, out_d[0], out_d[1], hist, lens, argmax=out_v[0], out=out_a)
            return
        ctx.verify_lmhead_argmax(dH, out=out_v)
        if timers:
            timers[2].record()
        ctx.accept_and_commit(out_d[0], out_d[1], out_v[0].view(S, B, w + 1), hist, lens, out=out_a)
        if timers:
            timers[3].record()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    side = torch.cuda.Stream()

    def make_round(fused):
        def round_of_steps():
            lens_all.copy_(lens0_all)
            for k in range(R):
                step(fused, k=k)
        with torch.cuda.stream(side):
            for _ in range(2):
                round_of_steps()
        torch.cuda.synchronize()
        if args.no_graph:
            return round_of_steps
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            round_of_steps()
        return graph.replay

    def time_blocks(run_round, min_s, clock_index=None):
        """Blocks of exactly K steps, each bracketed by events, repeated until min_s seconds were timed
        (at least 3, at most 2000 blocks).  Returns (median block ms, all block ms, clock summary)."""
        for _ in range((args.warmup + R - 1) // R):
            run_round()
        barrier()
        blocks = []
        sampler = ClockSampler(clock_index) if clock_index is not None else None
        if sampler:
            sampler.__enter__()
        barrier()
        while True:
            a, b = ev(torch), ev(torch)
            a.record()
            for _ in range(K // R):
                run_round()
            b.record()
            b.synchronize()
            blocks.append(a.elapsed_time(b))
            more = len(blocks) < 3 or (sum(blocks) < min_s * 1e3 and len(blocks) < 2000)
            if dist is not None:   # all ranks stop after the same number of blocks
                flag = torch.tensor([1.0 if more else 0.0], device=dev)
                dist.all_reduce(flag, op=dist.ReduceOp.MAX)
                more = flag.item() != 0.0
            if not more:
                break
        barrier()
        clocks = None
        if sampler:
            sampler.__exit__()
            clocks = sampler.summary()
        return statistics.median(blocks), blocks, clocks

    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    three = make_round(False)
    block_ms, blocks, clocks = time_blocks(three, MIN_TIMED_S if headline else MIN_TIMED_S / 2, local_rank if headline else None)
    acc_tokens = float((out_a[0].float() + 1).sum().item())          # tokens committed by one step of this rank
    fused = make_round(True)
    fblock_ms, fblocks, _ = time_blocks(fused, MIN_TIMED_S / 2)
    assert float((out_a[0].float() + 1).sum().item()) == acc_tokens, "the fused step committed a different number of tokens"
    fused_launches = 2 if S <= 256 else 3

    # per-phase device times, measured in a separate eager loop with events between the launches
    n_ph = 30
    timers = [[ev(torch) for _ in range(4)] for _ in range(n_ph)]
    for i in range(n_ph):
        step(False, timers[i])
    torch.cuda.synchronize()
    phase = lambda a, b: statistics.median(t[a].elapsed_time(t[b]) for t in timers)
    draft_ms, verify_ms, accept_ms = phase(0, 1), phase(1, 2), phase(2, 3)

    def back_to_back(fn, reps):
        """ms per call over `reps` calls in a row: launched eagerly, and replayed from one CUDA graph (the
        step's own launch mode, which takes the host's launch rate out of the measurement)."""
        a, b = ev(torch), ev(torch)
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        eager = a.elapsed_time(b) / reps
        if args.no_graph:
            return eager, None
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for _ in range(reps):
                    fn()
        g.replay()
        torch.cuda.synchronize()
        a.record()
        for _ in range(3):
            g.replay()
        b.record()
        torch.cuda.synchronize()
        return eager, a.elapsed_time(b) / (3 * reps)

    reps = 30 if M <= 512 else 8
    verify_eager_ms, verify_graph_ms = back_to_back(lambda: ctx.verify_lmhead_argmax(dH, out=out_v), reps)
    verify_alone_ms = verify_eager_ms if verify_graph_ms is None else min(verify_eager_ms, verify_graph_ms)

    from paper_2411_03786_b200.multigpu import reduce_max_sum
    (block_ms, fblock_ms, verify_alone_ms), (acc_total,) = reduce_max_sum([block_ms, fblock_ms, verify_alone_ms], [acc_tokens], device=dev)
    world = dist.get_world_size() if dist is not None else 1
    ms_per_step = block_ms / K

    # ---- roofline of the dominant kernel (the verify contraction), against the measured and the nominal peak
    bytes_alg = 2.0 * c["V"] * c["d"] + 2.0 * M * c["d"] + 4.0 * M
    flops = 2.0 * M * c["V"] * c["d"]
    t_hbm, t_tc = bytes_alg / (pk["hbm"] * 1e9), flops / (pk["tc_sustained"] * 1e12)
    if t_hbm >= t_tc:
        ach = bytes_alg / (verify_alone_ms / 1e3) / 1e9
        roof = {"bound": "hbm", "achieved": ach, "peak": pk["hbm"], "unit": "GB/s", "frac": ach / pk["hbm"],
                "frac_of_nominal": ach / NOMINAL["hbm_gbs"], "nominal_peak": NOMINAL["hbm_gbs"],
                "target": "70 % of HBM bandwidth", "meets_target_vs_measured": ach / pk["hbm"] >= 0.7,
                "meets_target_vs_nominal": ach / NOMINAL["hbm_gbs"] >= 0.7}
    else:
        ach = flops / (verify_alone_ms / 1e3) / 1e12
        roof = {"bound": "tensor", "achieved": ach, "peak": pk["tc_sustained"], "unit": "TFLOP/s",
                "frac": ach / pk["tc_sustained"], "frac_of_burst": ach / pk["tc_burst"],
                "frac_of_nominal": ach / NOMINAL["bf16_tflops"], "nominal_peak": NOMINAL["bf16_tflops"],
                "note": "tensor-bound: the 70 %-of-HBM target does not apply; inside a step the kernel runs under the "
                        "power cap, so the denominator is the sustained cuBLAS figure"}
    roof.update({"traffic": dram_traffic(c["name"], "head_gemm_kernel<ARGMAX>"), "kernel": "head_gemm_kernel<ARGMAX> (verify_lmhead_argmax)",
                 "ms_per_launch": verify_alone_ms, "ms_per_launch_eager": verify_eager_ms, "ms_per_launch_graph": verify_graph_ms,
                 "timing": "CUDA events around back-to-back launches on the launching stream (the faster of eager launches and one graph replay)",
                 "algorithmic_bytes": bytes_alg, "flops": flops,
                 "peak_source": pk["source"] + (" sustained" if roof["bound"] == "tensor" else " copy")})

    fp8 = None
    if args.fp8_for(c["name"], headline) and c["d"] % 16 == 0:
        if not head.fp8_ready:
            ctx.quantize_head_fp8()
            head.fp8_ready = True
        scratch8 = (torch.empty((M, c["d"]), dtype=torch.uint8, device=dev), torch.empty(M, dtype=torch.float32, device=dev))
        out8 = (torch.empty(M, dtype=torch.int32, device=dev), None)
        for _ in range(3):
            ctx.verify_lmhead_argmax_fp8(dH, scratch=scratch8, out=out8)
        e_ms, g_ms = back_to_back(lambda: ctx.verify_lmhead_argmax_fp8(dH, scratch=scratch8, out=out8), reps)
        fp8_ms = e_ms if g_ms is None else min(e_ms, g_ms)
        e2_ms, g2_ms = back_to_back(lambda: ctx.verify_lmhead_argmax_fp8(None, scratch=scratch8, out=out8), reps)
        fp8_gemm_ms = e2_ms if g2_ms is None else min(e2_ms, g2_ms)
        ctx.verify_lmhead_argmax(dH, out=out_v)
        torch.cuda.synchronize()
        bytes8 = 1.0 * c["V"] * c["d"] + 4.0 * c["V"] + 2.0 * M * c["d"] + 2.0 * M * c["d"] + 8.0 * M
        fp8 = {"ms_per_call": fp8_ms, "ms_contraction_only": fp8_gemm_ms, "launches_per_call": 2, "algorithmic_bytes": bytes8,
               "contraction_frac_of_copy_peak": (bytes8 - 4.0 * M * c["d"]) / (fp8_gemm_ms / 1e3) / 1e9 / pk["hbm"],
               "contraction_tflops": flops / fp8_gemm_ms / 1e9,
               "speedup_vs_bf16_verify": verify_alone_ms / fp8_ms,
               "argmax_agrees_with_bf16": float((out8[0] == out_v[0]).float().mean().item())}

    rec = {"workload": workload_string(c), "ms_per_step": ms_per_step, "blocks_timed": len(blocks),
           "block_ms_min_median_max": [min(blocks), statistics.median(blocks), max(blocks)],
           "value": acc_total / (ms_per_step / 1e3), "unit": UNIT, "steps_per_s": world * 1e3 / ms_per_step,
           "tokens_per_step": acc_total / world / S,
           "step_calls": "draft_context_ngrams, verify_lmhead_argmax, accept_and_commit", "launches_per_step": 3,
           "fused_step": {"step_calls": "draft_context_ngrams, verify_accept_commit", "ms_per_step": fblock_ms / K,
                          "launches_per_step": fused_launches, "value": acc_total / (fblock_ms / K / 1e3)},
           "steps_per_replay": R,
           "phase_ms": {"draft": draft_ms, "verify": verify_ms, "accept": accept_ms,
                        "note": "medians; events between eagerly launched calls: small kernels include the host's launch gap"},
           "roofline": roof, "copied_fraction": copied}
    if fp8:
        rec["fp8_verify"] = fp8
    if headline or c["name"] in ("C2", "C3"):
        rec["context_index"] = index_comparison(torch, c, head, dict(hist=hist, lens0=lens0, out_v=out_v, out_d=out_d, out_a=out_a, side=side), dev)
    extra = dict(hist_h=hist_h, lens_h=lens_h, H_bits=H_bits, hist=hist, lens0=lens0, dH=dH, out_d=out_d, out_v=out_v, out_a=out_a,
                 acc_tokens=acc_tokens, side=side, clocks=clocks, n_blocks=len(blocks), n_fblocks=len(fblocks), K=K, barrier=barrier)
    return rec, extra


def index_comparison(torch, c, head, x, dev):
    """Drafting + acceptance of consecutive decode steps with the history scanned at every step, and with the
    incremental context index (looked up by the draft, updated by the commit).  Each variant is one CUDA graph of
    `n` steps on its own copy of the histories (the steps really advance: a token or more is committed per step)."""
    ctx = head.ctx
    S, B, w, M = c["S"], c["B"], c["w"], c["M"]
    n = 24
    cap2 = (c["L"] + n * (w + 1) + 8 + 3) // 4 * 4
    hist0 = torch.full((S, cap2), -1, dtype=torch.int32, device=dev)
    hist0[:, :x["hist"].shape[1]] = x["hist"]
    lens0 = x["lens0"].clone()
    P = x["out_v"][0].view(S, B, w + 1).clone()          # the planted step's predictions, reused at every step
    out_d = tuple(torch.empty_like(t) for t in x["out_d"])
    out_a = tuple(torch.empty_like(t) for t in x["out_a"])
    res = {"steps_per_graph": n, "note": "draft + accept per step, steps advance the history; planted predictions of the first step reused"}
    side = x["side"]
    for kind in ("scan", "index"):
        hist, lens = hist0.clone(), lens0.clone()
        index = ctx.context_index_build(hist, lens, c["qs"], w) if kind == "index" else None

        def steps():
            for _ in range(n):
                if kind == "index":
                    ctx.draft_context_ngrams_indexed(index, hist, lens, c["qs"], c["topk"], B, w, out=out_d)
                    ctx.accept_and_commit_indexed(index, out_d[0], out_d[1], P, hist, lens, out=out_a)
                else:
                    ctx.draft_context_ngrams(hist, lens, c["qs"], c["topk"], B, w, out=out_d)
                    ctx.accept_and_commit(out_d[0], out_d[1], P, hist, lens, out=out_a)

        def reset():
            hist.copy_(hist0)
            lens.copy_(lens0)
            if kind == "index":
                ctx.context_index_build(hist, lens, c["qs"], w, index=index)

        with torch.cuda.stream(side):
            steps()
        torch.cuda.synchronize()
        reset()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            steps()
        ts = []
        for _ in range(5):
            reset()
            torch.cuda.synchronize()
            a, b = ev(torch), ev(torch)
            a.record()
            g.replay()
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b) / n)
        res[kind] = {"us_per_step": statistics.median(ts) * 1e3, "tokens_committed": int((lens - lens0).sum().item())}
        if kind == "index":
            t0 = ev(torch), ev(torch)
            t0[0].record()
            ctx.context_index_build(hist, lens, c["qs"], w, index=index)
            t0[1].record()
            torch.cuda.synchronize()
            res["index"]["build_ms"] = t0[0].elapsed_time(t0[1])
            res["index"]["bytes"] = int(index.numel())
    assert res["scan"]["tokens_committed"] == res["index"]["tokens_committed"], "the two variants decoded differently"
    assert ctx.get_status() == 0
    return res


def workload_string(c):
    return (f"{c['name']}: V={c['V']} d={c['d']} S={c['S']} L={c['L']} qs={list(c['qs'])} topk={c['topk']} "
            f"B={c['B']} w={c['w']} M={c['M']} k_tab={c['k_tab']} per GPU")


def end_to_end(torch, c, head, x, args, dist, rank, world):
    """The step through the public API with HOST buffers: pinned staging blobs [history | lengths] and [hidden
    states] go up, [accepted lengths | committed tokens] come back, inside the timed region, every step."""
    ctx = head.ctx
    dev = x["hist"].device
    S, B, w, M = c["S"], c["B"], c["w"], c["M"]
    hist, lens0, dH, out_d, out_v, out_a, side = x["hist"], x["lens0"], x["dH"], x["out_d"], x["out_v"], x["out_a"], x["side"]

    def carve(blob, specs):
        views, off = [], 0
        for shape, dtype in specs:
            n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
            views.append(blob[off:off + n].view(dtype).view(shape))
            off += (n + 255) // 256 * 256
        return views

    def blob_bytes(specs):
        return sum((int(np.prod(sh)) * torch.empty((), dtype=dt).element_size() + 255) // 256 * 256 for sh, dt in specs)

    tok_specs = [(tuple(hist.shape), torch.int32), ((S,), torch.int32)]
    hid_specs = [((M, c["d"]), torch.bfloat16)]
    out_specs = [((S,), torch.int32), ((S, w + 1), torch.int32)]
    pinned = lambda specs: torch.empty(blob_bytes(specs), dtype=torch.uint8).pin_memory()
    ondev = lambda specs: torch.empty(blob_bytes(specs), dtype=torch.uint8, device=dev)
    h_tok, h_hid, h_out = pinned(tok_specs), pinned(hid_specs), pinned(out_specs)
    d_tok, d_hid = ondev(tok_specs), ondev(hid_specs)
    for hv, src in zip(carve(h_tok, tok_specs) + carve(h_hid, hid_specs), (hist, lens0, dH)):
        hv.copy_(src.cpu())
    d_hist2, d_lens2 = carve(d_tok, tok_specs)
    (d_H2,) = carve(d_hid, hid_specs)
    # The step's result (accepted lengths, committed tokens) is written by the accepting kernel straight into
    # mapped pinned host memory: the device-to-host transfer is the kernel's own stores.
    out_a2 = (carve(h_out, out_specs)[0], out_a[1], carve(h_out, out_specs)[1])
    copy_stream = torch.cuda.Stream()

    def e2e_body():
        # the hidden states are not needed before the verify call: their upload overlaps the drafting
        main = torch.cuda.current_stream()
        copy_stream.wait_stream(main)
        with torch.cuda.stream(copy_stream):
            d_hid.copy_(h_hid, non_blocking=True)
        d_tok.copy_(h_tok, non_blocking=True)
        ctx.draft_context_ngrams(d_hist2, d_lens2, c["qs"], c["topk"], B, w, out=out_d)
        main.wait_stream(copy_stream)
        ctx.verify_lmhead_argmax(d_H2, out=out_v)
        ctx.accept_and_commit(out_d[0], out_d[1], out_v[0].view(S, B, w + 1), d_hist2, d_lens2, out=out_a2)

    e2e_graph = None
    if not args.no_graph:
        with torch.cuda.stream(side):
            e2e_body()
        torch.cuda.synchronize()
        e2e_graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(e2e_graph, stream=side):
            e2e_body()

    def e2e_step():
        # host -> device copies, the three kernels and the device -> host read-back, then wait for the result
        if e2e_graph is not None:
            e2e_graph.replay()
        else:
            e2e_body()
        torch.cuda.synchronize()

    for _ in range(3):
        e2e_step()
    x["barrier"]()
    blocks = []
    while len(blocks) < 3 or (sum(blocks) < MIN_TIMED_S * 1e3 / 2 and len(blocks) < 500):
        a, b = ev(torch), ev(torch)
        a.record()
        for _ in range(args.steps):
            e2e_step()
        b.record()
        b.synchronize()
        blocks.append(a.elapsed_time(b))
        if dist is not None:
            break   # several ranks: one block each, so that nobody waits at a collective the others skip
    x["barrier"]()
    e2e_ms = statistics.median(blocks) / args.steps
    h2d = h_tok.numel() + h_hid.numel()
    d2h = out_a2[0].numel() * 4 + out_a2[2].numel() * 4        # what the kernel stores into host memory per step
    assert torch.equal(out_a2[0], out_a[0].cpu()), "the host copy of the accepted lengths differs from the device run"

    # ---- the same end-to-end step, two deep: step i+1's uploads run while step i computes, and the host reads
    # step i's result while step i+1 is already queued (how a serving loop would drive it).
    pipe_ms = None
    if not args.no_graph and rank == 0 and world == 1:
        sets = []
        for bset in range(2):
            ht, hh, ho = pinned(tok_specs), pinned(hid_specs), pinned(out_specs)
            dt, dh = ondev(tok_specs), ondev(hid_specs)
            ht.copy_(h_tok); hh.copy_(h_hid)
            dhist, dlens = carve(dt, tok_specs)
            (dHb,) = carve(dh, hid_specs)
            outb = (carve(ho, out_specs)[0], out_a[1], carve(ho, out_specs)[1])

            def compute(dhist=dhist, dlens=dlens, dHb=dHb, outb=outb):
                ctx.draft_context_ngrams(dhist, dlens, c["qs"], c["topk"], B, w, out=out_d)
                ctx.verify_lmhead_argmax(dHb, out=out_v)
                ctx.accept_and_commit(out_d[0], out_d[1], out_v[0].view(S, B, w + 1), dhist, dlens, out=outb)

            with torch.cuda.stream(side):
                dt.copy_(ht); dh.copy_(hh)
                compute()
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                compute()
            sets.append(dict(ht=ht, hh=hh, ho=ho, dt=dt, dh=dh, g=g, acc=outb[0], up=torch.cuda.Event(), done=torch.cuda.Event()))
        main = torch.cuda.current_stream()

        def pipelined(n):
            tokens = 0
            for i in range(n):
                cur, prev = sets[i & 1], sets[(i & 1) ^ 1]
                if i >= 2:
                    copy_stream.wait_event(cur["done"])       # the step that used these device buffers has finished
                with torch.cuda.stream(copy_stream):
                    cur["dt"].copy_(cur["ht"], non_blocking=True)
                    cur["dh"].copy_(cur["hh"], non_blocking=True)
                    cur["up"].record(copy_stream)
                main.wait_event(cur["up"])
                cur["g"].replay()
                cur["done"].record(main)
                if i >= 1:
                    prev["done"].synchronize()
                    tokens += int(prev["acc"].sum()) + S       # the host reads the previous step's result
            sets[(n - 1) & 1]["done"].synchronize()
            return tokens + int(sets[(n - 1) & 1]["acc"].sum()) + S

        n_pipe = max(args.steps, int(min(2000, 0.1 / max(e2e_ms / 1e3, 1e-6))))
        pipelined(10)
        torch.cuda.synchronize()
        p0, p1 = ev(torch), ev(torch)
        p0.record()
        tok_pipe = pipelined(n_pipe)
        p1.record()
        torch.cuda.synchronize()
        pipe_ms = p0.elapsed_time(p1) / n_pipe
        assert tok_pipe == int(round(x["acc_tokens"])) * n_pipe, "the pipelined loop committed a different number of tokens"
    return e2e_ms, h2d, d2h, pipe_ms, len(blocks)


def spawn_ranks(args):
    """`--gpus N` without a launcher: start N ranks of this script (one process per GPU, NCCL), relay rank 0's
    JSON line to stdout and everything else (NCCL's communicator lines among it) to stderr."""
    import socket
    import torch
    n = args.gpus
    have = torch.cuda.device_count() if torch.cuda.is_available() else 0
    if have < n:
        raise SystemExit(f"bench.py --gpus {n}: this machine shows {have} CUDA device(s); refusing to run fewer ranks than asked")
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        env.setdefault("NCCL_DEBUG", "INFO")
        env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env,
                                      stdout=subprocess.PIPE, stderr=None, text=True))
    rc, line = 0, None
    for r, p in enumerate(procs):
        out, _ = p.communicate()
        for ln in out.splitlines():
            if r == 0 and ln.startswith("{") and '"metric"' in ln:
                line = ln
            else:
                print(ln, file=sys.stderr)
        rc = rc or p.returncode
    if line:
        print(line)
    return rc or (0 if line else 1)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="C5", choices=sorted(synth.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-budget", type=float, default=15.0, help="seconds of CPU work for the oracle baseline")
    ap.add_argument("--no-table", action="store_true", help="skip timing the one-off table build")
    ap.add_argument("--no-scaled", action="store_true", help="skip timing draft/accept on bandwidth-sized batches")
    ap.add_argument("--no-per-config", action="store_true", help="measure the headline workload only")
    ap.add_argument("--no-sweep", action="store_true", help="skip the sweep of verify block heights across the tile steps")
    ap.add_argument("--no-fp8", action="store_true", help="skip timing the 8-bit (E4M3) verification head (reported beside the bf16 numbers)")
    ap.add_argument("--no-graph", action="store_true", help="launch the step eagerly instead of replaying a CUDA graph")
    ap.add_argument("--scaled-only", action="store_true", help="only time draft/accept on the bandwidth-sized batches (a short run to profile those kernels)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    args.steps = max(args.steps, 1)
    args.fp8_for = lambda name, headline: (not args.no_fp8) and (headline or name == "C2")

    if "WORLD_SIZE" not in os.environ and args.gpus > 1 and args.impl == "ours":
        return spawn_ranks(args)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    c = synth.config(args.workload)
    cfg = {"workload": workload_string(c),
           "hidden_states": f"planted acceptance rho={RHO}", "l2": "verify streams the unembedding (larger than L2) every step; "
           "draft/accept inputs are at most 2 MB and stay L2-resident", "sharding": "sequences per rank, no collective"}

    if args.impl == "reference":
        if rank != 0:
            return 0
        return run_reference(args, c, cfg)

    import torch
    import paper_2411_03786_b200 as ngs
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    if world > torch.cuda.device_count():
        raise SystemExit(f"bench.py: {world} ranks but {torch.cuda.device_count()} CUDA device(s)")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)
    pk = peaks()

    if args.scaled_only:
        head = Head(torch, ngs, c, dev, pk, time_table=False)
        print(json.dumps({"scaled_streams": scaled_streams(head.ctx, torch, dev, c, pk), "workload_head": workload_string(c)}))
        head.ctx.close()
        return 0
    names = [args.workload] + ([] if args.no_per_config else [n for n in ("C2", "C3", "C4", "C5") if n != args.workload and args.workload != "C1"])
    heads, per_config, head_rec, head_x = {}, {}, None, None
    for name in names:
        cc = synth.config(name)
        key = (cc["V"], cc["d"], cc["wseed"])
        if key not in heads:
            heads[key] = Head(torch, ngs, cc, dev, pk, time_table=not args.no_table)
        rec, x = measure_config(torch, ngs, cc, heads[key], dev, pk, args, rank, dist, headline=(name == args.workload))
        if heads[key].table and name in ("C2", "C4", args.workload):
            rec["table_build"] = heads[key].table
        if name == args.workload:
            head_rec, head_x = rec, x
        else:
            per_config[name] = rec
            del x
    head = heads[(c["V"], c["d"], c["wseed"])]

    e2e_ms, h2d, d2h, pipe_ms, e2e_blocks = end_to_end(torch, c, head, head_x, args, dist, rank, world)
    from paper_2411_03786_b200.multigpu import reduce_max_sum
    (e2e_ms,), _ = reduce_max_sum([e2e_ms], [0.0], device=dev)
    acc_total = head_rec["value"] * head_rec["ms_per_step"] / 1e3
    e2e_value = acc_total / (e2e_ms / 1e3)
    status = head.ctx.get_status()

    single = rank == 0 and world == 1
    scaled = scaled_streams(head.ctx, torch, dev, c, pk) if (not args.no_scaled and single) else None
    sweep = verify_rows_sweep(torch, heads, dev, pk) if (not args.no_sweep and single and not args.no_per_config) else None
    if rank == 0:
        cpu = {}
        if args.cpu_budget > 0:
            T_h = head.tab.cpu().numpy()
            sec, acc_cpu, threads, sample, sampled = oracle_step_time(c, head_x["hist_h"], head_x["lens_h"], T_h, head_x["H_bits"],
                                                                      head.W_bits, args.cpu_budget)
            cpu = {"value": acc_cpu / sec, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample,
                   "s_per_step": sec}
            if head.table:
                # the oracle's table build on a row sample, projected to all V rows (each row costs 2 V d flop)
                import oracle
                n_rows = 2 * threads
                t0 = time.perf_counter()
                oracle.model_table(bf16_bits(head.E), head.W_bits, c["k_tab"], rows=np.linspace(0, c["V"] - 1, n_rows).astype(np.int64))
                dt = time.perf_counter() - t0
                cpu["table_build"] = {"rows_per_s": n_rows / dt, "projected_s": dt / n_rows * c["V"],
                                      "sample": f"{n_rows} of {c['V']} rows"}
        K = args.steps
        n_launch = 3 * K * head_x["n_blocks"]
        line = {"metric": METRIC, "value": head_rec["value"], "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
                "ms_per_step": head_rec["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16", "data": "synthetic", "config": cfg,
                "timing": f"blocks of exactly {K} steps, each between two CUDA events, repeated until {MIN_TIMED_S} s were timed; "
                          "ms_per_step = median block / steps; max over ranks",
                "blocks_timed": head_x["n_blocks"], "block_ms_min_median_max": head_rec["block_ms_min_median_max"],
                "step_calls": head_rec["step_calls"], "steps_per_replay": head_rec["steps_per_replay"],
                "steps_per_s": head_rec["steps_per_s"], "tokens_per_step": head_rec["tokens_per_step"],
                "fused_step": head_rec["fused_step"], "phase_ms": head_rec["phase_ms"],
                "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                        "ms_per_step": e2e_ms, "blocks_timed": e2e_blocks,
                        "mode": "one step at a time: upload, draft / verify / accept, host waits for the result",
                        "pipelined_two_deep_ms_per_step": pipe_ms},
                "gpu_launches": int(n_launch) * world,
                "gpu_launches_note": f"3 kernels per step x {K} steps x {head_x['n_blocks']} timed blocks (per block: {3 * K})",
                "launch_mode": "eager" if args.no_graph else "cuda_graph_replay", "roofline": head_rec["roofline"],
                "table_build": head_rec.get("table_build", {}), "cpu_baseline": cpu,
                "clocks": head_x["clocks"], "status_bits": status, "copied_fraction": head_rec["copied_fraction"],
                "peaks": {"measured": pk, "nominal": NOMINAL}}
        if "fp8_verify" in head_rec:
            line["fp8_verify"] = head_rec["fp8_verify"]
        if "context_index" in head_rec:
            line["context_index"] = head_rec["context_index"]
        if per_config:
            line["per_config"] = per_config
        if scaled:
            line["scaled_streams"] = scaled
        if sweep:
            line["verify_rows_sweep"] = sweep
        print(json.dumps(line))
    for h in heads.values():
        h.ctx.close()
    if dist is not None:
        dist.destroy_process_group()
    return 0


def verify_rows_sweep(torch, heads, dev, pk):
    """The memory-to-compute transition of the verification call on the 7B-shaped head: back-to-back launches
    (one graph replay) for block heights on both sides of each 128-row tile step."""
    head = next((h for (V, d, _), h in heads.items() if V == 32000), None)
    if head is None:
        return None
    V, d = head.ctx.V, head.ctx.d
    out = {"head": f"V={V} d={d}", "rows": {}}
    g = torch.Generator(device=dev).manual_seed(5)
    side = torch.cuda.Stream()
    for M in (48, 128, 129, 192, 256, 257, 320, 384, 512, 1024):
        H = torch.randn((M, d), device=dev, dtype=torch.float32, generator=g).to(torch.bfloat16)
        am = (torch.empty(M, dtype=torch.int32, device=dev), None)
        reps = 20
        for _ in range(3):
            head.ctx.verify_lmhead_argmax(H, out=am)
        torch.cuda.synchronize()
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(gr, stream=side):
                for _ in range(reps):
                    head.ctx.verify_lmhead_argmax(H, out=am)
        gr.replay()
        torch.cuda.synchronize()
        a, b = ev(torch), ev(torch)
        a.record()
        for _ in range(3):
            gr.replay()
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / (3 * reps)
        fl = 2.0 * M * V * d
        by = 2.0 * V * d + 2.0 * M * d + 4.0 * M
        out["rows"][str(M)] = {"us": ms * 1e3, "tflops": fl / ms / 1e9, "gbs": by / ms / 1e6,
                               "frac_of_roofline": max(by / (pk["hbm"] * 1e9), fl / (pk["tc_burst"] * 1e12)) / (ms / 1e3)}
    out["note"] = "frac_of_roofline = max(bytes / copy bandwidth, flops / burst bf16 peak) / measured time (measured peaks)"
    return out


def run_reference(args, c, cfg):
    """The CPU oracle, as it stands, on the host cores: same workload, metric and unit."""
    import oracle
    W = synth.gaussian_weights(c["V"], c["d"], c["wstd"], c["wseed"], "W", c["wdtype"])
    hist_h, lens_h, _ = synth.zipf_histories(c["S"], c["L"], c["V"], c["zipf"], c["copy"], c["seed"], cap=c["L"] + 64,
                                             name="hist/rank0")
    W_bits = bf16_bits(W)
    k = c["k_tab"]
    # a model table is an input of the step; which tokens it holds is irrelevant to the timing, so a
    # seeded stand-in is used instead of the (hours-long) CPU table build
    g = synth.stream(c["seed"], "ref/T")
    T = g.integers(0, c["V"], (c["V"], k)).astype(np.int32)
    drafts0, nd0, _, _ = oracle.draft_batch(hist_h, lens_h, c["qs"], c["topk"], c["B"], c["w"], 3, T)
    targets, _, _ = synth.planted_targets(drafts0, nd0, None, c["V"], c["zipf"], RHO, seed=c["seed"])
    H_bits = synth.hidden_planted(W_bits, targets.reshape(-1), seed=c["seed"])
    per_step_budget = max(2.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    for _ in range(min(args.warmup, 1)):
        oracle_step_time(c, hist_h, lens_h, T, H_bits, W_bits, per_step_budget, max_steps=1)
    secs, accs = [], []
    t_wall = time.perf_counter()
    for _ in range(args.steps):
        sec, acc, threads, sample, _ = oracle_step_time(c, hist_h, lens_h, T, H_bits, W_bits, per_step_budget, max_steps=1)
        secs.append(sec)
        accs.append(acc)
        if time.perf_counter() - t_wall > 150:
            break
    sec = statistics.mean(secs)
    value = statistics.mean(accs) / sec
    cpu = {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample}
    print(json.dumps({"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
                      "steps": len(secs), "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
                      "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": cfg,
                      "model_table": "seeded stand-in table (the CPU table build would take hours): the model-fill rows, and "
                                     "the hidden states planted on them, differ from the GPU arm's; the work per step is the same",
                      "cpu_baseline": cpu, "gpu_launches": 0,
                      "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
    return 0


if __name__ == "__main__":
    sys.exit(main())
