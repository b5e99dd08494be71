#!/usr/bin/env python
"""Benchmark of the batched N-gram speculation step on B200.

One *step* = draft_context_ngrams -> verify_lmhead_argmax -> accept_and_commit over one batch of
synthetic sequences (hidden states are an input: the transformer body is outside this library).
The model bigram table is a one-off build and is timed separately (reported under "table_build").

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C2] [--impl ours|reference]

Prints ONE JSON line.  `--impl reference` times the plain CPU oracle on the host cores instead.
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth  # noqa: E402

METRIC = "accepted_tokens_per_s"
UNIT = "tokens/s"
RHO = 0.55  # planted acceptance: P(accepted length >= j) = RHO^j  (about 2.2 tokens per call)


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=d["hbm_gbs"], tc_burst=d["bf16_tflops"], tc_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]),
                    source="measured")
    return dict(hbm=6650.0, tc_burst=1590.0, tc_sustained=1400.0, source="fallback")


def host_inputs(c, rank):
    """Seeded host-side inputs of one rank's batch (weights are shared, histories differ per rank)."""
    seed = c["seed"]
    E = synth.gaussian_weights(c["V"], c["d"], c["wstd"], c["wseed"], "E", c["wdtype"])
    W = synth.gaussian_weights(c["V"], c["d"], c["wstd"], c["wseed"], "W", c["wdtype"])
    cap = c["L"] + 64
    hist, lens, copied = synth.zipf_histories(c["S"], c["L"], c["V"], c["zipf"], c["copy"], seed, cap=cap,
                                              name=f"hist/rank{rank}")
    return E, W, hist, lens, copied


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


def scaled_streams(ctx, torch, dev, c, pk):
    """Streaming rates of the integer kernels on batches large enough to measure bandwidth (at the
    benchmark sizes they move a few KB and are launch-latency-bound)."""
    out = {}
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def timed(fn, reps):
        for _ in range(2):
            fn()
        torch.cuda.synchronize()
        a, b = ev(), ev()
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    for S, L, qs, reps in ((4096, 2048, (3, 2, 1), 20), (512, 131072, (3, 2), 5)):   # shaped like C3 / C5
        base, lens_b, _ = synth.zipf_histories(32, L, c["V"], c["zipf"], 0.3, seed=77, cap=L + 64, name="scaled")
        hist = torch.from_numpy(np.tile(base, (S // 32, 1))).to(dev)
        lens = torch.from_numpy(np.tile(lens_b, S // 32)).to(dev)
        B, w, topk = 16, 8, 4
        bufs = (torch.empty((S, B, w), dtype=torch.int32, device=dev), torch.empty(S, dtype=torch.int32, device=dev),
                torch.empty((S, B), dtype=torch.int32, device=dev), torch.empty((S, B), dtype=torch.int32, device=dev))
        ms = timed(lambda: ctx.draft_context_ngrams(hist, lens, qs, topk, B, w, out=bufs), reps)
        by = 4.0 * S * L + 4.0 * S * B * (w + 2) + 8.0 * S
        out[f"draft_S{S}_L{L}"] = {"qs": list(qs), "ms": ms, "GB/s": by / ms / 1e6, "frac_of_hbm": by / ms / 1e6 / pk["hbm"], "bytes": by,
                                   "l2": "larger than L2" if by > 126e6 else "L2-resident"}
        del hist, lens, bufs
    S, B, w = 65536, 64, 10
    g = torch.Generator(device=dev).manual_seed(3)
    drafts = torch.randint(0, 4, (S, B, w), device=dev, dtype=torch.int32, generator=g)
    P = torch.randint(0, 4, (S, B, w + 1), device=dev, dtype=torch.int32, generator=g)
    nd = torch.full((S,), B, dtype=torch.int32, device=dev)
    cap = 64
    hist = torch.zeros((S, cap), dtype=torch.int32, device=dev)
    lens0 = torch.full((S,), 8, dtype=torch.int32, device=dev)
    lens = lens0.clone()
    bufs = (torch.empty(S, dtype=torch.int32, device=dev), torch.empty(S, dtype=torch.int32, device=dev),
            torch.empty((S, w + 1), dtype=torch.int32, device=dev))

    def acc():
        lens.copy_(lens0)
        ctx.accept_and_commit(drafts, nd, P, hist, lens, out=bufs)

    ms = timed(acc, 10)
    # early exit reads only the first sector of most rows: count the bytes of every 32-byte sector touched at
    # least once, i.e. the first sector of each draft row and of each prediction row, plus the outputs
    by_full = 4.0 * S * B * (2 * w + 1) + 4.0 * S * (w + 4)
    out[f"accept_S{S}_B{B}_w{w}"] = {"ms": ms, "GB/s_if_all_bytes_read": by_full / ms / 1e6, "bytes_all": by_full,
                                    "note": "prefix comparison stops at the first mismatch, so fewer bytes are needed"}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="C2", choices=sorted(synth.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-budget", type=float, default=15.0, help="seconds of CPU work for the oracle baseline")
    ap.add_argument("--no-table", action="store_true", help="skip timing the one-off table build")
    ap.add_argument("--no-scaled", action="store_true", help="skip timing draft/accept on bandwidth-sized batches")
    ap.add_argument("--no-fuse", action="store_true",
                    help="call verify_lmhead_argmax and accept_and_commit separately instead of verify_accept_commit (one launch)")
    ap.add_argument("--fp8", action="store_true", help=argparse.SUPPRESS)      # accepted for older command lines: now the default
    ap.add_argument("--scaled", action="store_true", help=argparse.SUPPRESS)   # likewise
    ap.add_argument("--no-fp8", action="store_true", help="skip timing the 8-bit (E4M3) verification head (reported beside the bf16 numbers)")
    ap.add_argument("--no-graph", action="store_true", help="launch the step eagerly instead of replaying a CUDA graph")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    c = synth.config(args.workload)
    cfg = {"workload": f"{args.workload}: V={c['V']} d={c['d']} S={c['S']} L={c['L']} qs={list(c['qs'])} topk={c['topk']} "
                       f"B={c['B']} w={c['w']} M={c['M']} k_tab={c['k_tab']} per GPU",
           "hidden_states": f"planted acceptance rho={RHO}", "l2": "verify streams the unembedding (larger than L2) every step; "
           "draft/accept inputs are KB-sized and stay L2-resident", "sharding": "sequences per rank, no collective"}

    if args.impl == "reference":
        if rank != 0:
            return 0
        return run_reference(args, c, cfg)

    import torch
    import paper_2411_03786_b200 as ngs
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)
    pk = peaks()

    E, W, hist_h, lens_h, copied = host_inputs(c, rank)
    to_dev = (lambda w: torch.from_numpy(w).to(dev)) if c["wdtype"] == "f32" else \
        (lambda w: torch.from_numpy(w.view(np.int16)).view(torch.bfloat16).to(dev))
    dE, dW = to_dev(E), to_dev(W)
    ctx = ngs.SpecContext(dE, dW)
    W_bits = bf16_bits(W)

    # ---- one-off table build (timed on its own)
    table = {}
    ev = lambda: torch.cuda.Event(enable_timing=True)
    tab, _, ext = ctx.build_model_ngram_tables(c["k_tab"], w_ext=c["w"])
    torch.cuda.synchronize()
    if not args.no_table:
        reps = 3 if c["V"] <= 40000 else 1
        ts = []
        for _ in range(reps):
            a, b = ev(), ev()
            a.record()
            ctx.build_model_ngram_tables(c["k_tab"], w_ext=c["w"])
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        ms = min(ts)
        fl = 2.0 * c["V"] * c["V"] * c["d"]
        a, b = ev(), ev()
        ctx.build_model_unigram(25)
        a.record()
        ctx.build_model_unigram(25)
        b.record()
        torch.cuda.synchronize()
        uni_ms = a.elapsed_time(b)
        table = {"ms": ms, "tflops": fl / ms / 1e9, "unigram_ms": uni_ms, "unigram_tflops": fl / uni_ms / 1e9, "frac_of_burst_peak": fl / ms / 1e9 / pk["tc_burst"],
                 "frac_of_sustained_peak": fl / ms / 1e9 / pk["tc_sustained"], "flops": fl, "peak_source": pk["source"]}

    # ---- inputs of a step: histories, then hidden states planted on the initial drafts
    hist, lens0 = torch.from_numpy(hist_h).to(dev), torch.from_numpy(lens_h).to(dev)
    lens = lens0.clone()
    S, B, w, M = c["S"], c["B"], c["w"], c["M"]
    out_d = ctx.draft_context_ngrams(hist, lens, c["qs"], c["topk"], B, w)
    torch.cuda.synchronize()
    drafts0, nd0 = out_d[0].cpu().numpy(), out_d[1].cpu().numpy()
    targets, _, planted_a = synth.planted_targets(drafts0, nd0, None, c["V"], c["zipf"], RHO, seed=c["seed"] + 100 * rank)
    H_bits = synth.hidden_planted(W_bits, targets.reshape(-1), seed=c["seed"] + 100 * rank)
    dH = torch.from_numpy(H_bits.view(np.int16)).view(torch.bfloat16).to(dev)
    out_v = (torch.empty(M, dtype=torch.int32, device=dev), None)
    out_a = (torch.empty(S, dtype=torch.int32, device=dev), torch.empty(S, dtype=torch.int32, device=dev),
             torch.empty((S, w + 1), dtype=torch.int32, device=dev))

    fused = not args.no_fuse   # verify + accept as one launch: 1.1 us per C2 step less than the two calls (same box, same run)
    cfg["step_calls"] = "draft_context_ngrams, verify_accept_commit" if fused else "draft_context_ngrams, verify_lmhead_argmax, accept_and_commit"

    # Every step sees the same history: step k of a round works on its own copy of the lengths, and one
    # small copy per round of R steps restores all of them.  (A reset before every step would sit between
    # accept and the next draft and break the dependent-launch chain that a real decode loop has there.)
    R = max(r for r in range(1, 17) if args.steps % r == 0)
    lens_all = lens0.unsqueeze(0).repeat(R, 1).contiguous()
    lens0_all = lens_all.clone()
    cfg["steps_per_replay"] = R

    def step(timers=None, k=0):
        lens = lens_all[k]
        if timers:
            lens.copy_(lens0)
            timers[0].record()
        ctx.draft_context_ngrams(hist, lens, c["qs"], c["topk"], B, w, out=out_d)
        if timers:
            timers[1].record()
        if timers or not fused:
            ctx.verify_lmhead_argmax(dH, out=out_v)
            if timers:
                timers[2].record()
            ctx.accept_and_commit(out_d[0], out_d[1], out_v[0].view(S, B, w + 1), hist, lens, out=out_a)
            if timers:
                timers[3].record()
        else:   # verify + accept in one launch (the per-phase timing loop keeps them apart)
            ctx.verify_accept_commit(dH, out_d[0], out_d[1], hist, lens, argmax=out_v[0], out=out_a)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # The step is launch-bound at small sizes: capture it once in a CUDA graph and replay it.
    def round_of_steps():
        lens_all.copy_(lens0_all)
        for k in range(R):
            step(k=k)

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for _ in range(3):
            round_of_steps()
    torch.cuda.synchronize()
    graph = None
    if not args.no_graph:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            round_of_steps()
    run_round = graph.replay if graph is not None else round_of_steps
    launches_per_step = 2 if (fused and S <= 256) else 3   # draft, verify(+accept) (the length reset is a torch copy)

    for _ in range((args.warmup + R - 1) // R):
        run_round()
    barrier()
    t_begin, t_end = ev(), ev()
    with ClockSampler(local_rank) as clk:
        barrier()
        t_begin.record()
        for i in range(args.steps // R):
            run_round()
        t_end.record()
        barrier()
    total_ms = t_begin.elapsed_time(t_end)
    launches = launches_per_step * args.steps
    acc_mean = float((out_a[0].float() + 1).sum().item())          # tokens committed by one step of this rank
    # per-phase device times, measured in a separate eager loop with events between the launches
    n_ph = min(args.steps, 50)
    timers = [[ev() for _ in range(4)] for _ in range(n_ph)]
    for i in range(n_ph):
        step(timers[i])
    torch.cuda.synchronize()
    status = ctx.get_status()
    phase = lambda a, b: statistics.mean(t[a].elapsed_time(t[b]) for t in timers)
    draft_ms, verify_ms, accept_ms = phase(0, 1), phase(1, 2), phase(2, 3)
    # the verify kernel alone, back to back, for the roofline (same launch configuration)
    def back_to_back(fn, reps):
        """ms per call over `reps` calls in a row: launched eagerly, and replayed from one CUDA graph (the
        step's own launch mode, which takes the host's launch rate out of the measurement)."""
        a, b = ev(), ev()
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

    verify_eager_ms, verify_graph_ms = back_to_back(lambda: ctx.verify_lmhead_argmax(dH, out=out_v), n_ph)
    verify_alone_ms = verify_eager_ms if verify_graph_ms is None else min(verify_eager_ms, verify_graph_ms)

    fp8 = None
    if not args.no_fp8 and c["d"] % 16 == 0:
        # quantise the head once, then the same back-to-back timing: each call = quantise H (1 launch) + contraction
        ctx.quantize_head_fp8()
        scratch8 = (torch.empty((M, c["d"]), dtype=torch.uint8, device=dev), torch.empty(M, dtype=torch.float32, device=dev))
        out8 = (torch.empty(M, dtype=torch.int32, device=dev), None)
        for _ in range(5):
            ctx.verify_lmhead_argmax_fp8(dH, scratch=scratch8, out=out8)
        e_ms, g_ms = back_to_back(lambda: ctx.verify_lmhead_argmax_fp8(dH, scratch=scratch8, out=out8), n_ph)
        fp8_ms = e_ms if g_ms is None else min(e_ms, g_ms)
        # hidden states already quantised: the contraction alone
        e2_ms, g2_ms = back_to_back(lambda: ctx.verify_lmhead_argmax_fp8(None, scratch=scratch8, out=out8), n_ph)
        fp8_gemm_ms = e2_ms if g2_ms is None else min(e2_ms, g2_ms)
        ctx.verify_lmhead_argmax(dH, out=out_v)
        torch.cuda.synchronize()
        bytes8 = 1.0 * c["V"] * c["d"] + 4.0 * c["V"] + 2.0 * M * c["d"] + 2.0 * M * c["d"] + 8.0 * M
        fp8 = {"ms_per_call": fp8_ms, "ms_per_call_eager": e_ms, "ms_contraction_only_eager": e2_ms, "launches_per_call": 2, "algorithmic_bytes": bytes8, "ms_contraction_only": fp8_gemm_ms,
               "contraction_frac_of_copy_peak": (bytes8 - 4.0 * M * c["d"]) / (fp8_gemm_ms / 1e3) / 1e9 / pk["hbm"],
               "achieved_gbs": bytes8 / (fp8_ms / 1e3) / 1e9, "frac_of_copy_peak": bytes8 / (fp8_ms / 1e3) / 1e9 / pk["hbm"],
               "speedup_vs_bf16_verify": verify_alone_ms / fp8_ms,
               "argmax_agrees_with_bf16": float((out8[0] == out_v[0]).float().mean().item())}

    # ---- end to end through the public API with host buffers
    # Pinned staging blobs: [history | lengths] and [hidden states] in, [accepted lengths | committed tokens] out.
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
    d_tok, d_hid, d_out = ondev(tok_specs), ondev(hid_specs), ondev(out_specs)
    for hv, src in zip(carve(h_tok, tok_specs) + carve(h_hid, hid_specs), (hist, lens0, dH)):
        hv.copy_(src.cpu())
    d_hist2, d_lens2 = carve(d_tok, tok_specs)
    (d_H2,) = carve(d_hid, hid_specs)
    # The step's result (accepted lengths, committed tokens) is written by the accepting CTA straight into
    # mapped pinned host memory: the device-to-host transfer is the kernel's own stores (a copy node of 512 B
    # after the kernel measured 10 us slower).
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
        if fused:
            ctx.verify_accept_commit(d_H2, out_d[0], out_d[1], d_hist2, d_lens2, argmax=out_v[0], out=out_a2)
        else:
            ctx.verify_lmhead_argmax(d_H2, out=out_v)
            ctx.accept_and_commit(out_d[0], out_d[1], out_v[0].view(S, B, w + 1), d_hist2, d_lens2, out=out_a2)

    e2e_graph = None
    if graph is not None:
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
    barrier()
    e_begin, e_end = ev(), ev()
    e_begin.record()
    for _ in range(args.steps):
        e2e_step()
    e_end.record()
    barrier()
    e2e_ms = e_begin.elapsed_time(e_end)
    h2d = h_tok.numel() + h_hid.numel()
    d2h = out_a2[0].numel() * 4 + out_a2[2].numel() * 4        # what the kernel stores into host memory per step
    assert torch.equal(out_a2[0], out_a[0].cpu()), "the host copy of the accepted lengths differs from the device run"

    # ---- the same end-to-end step, two deep: step i+1's uploads run while step i computes, and the host reads
    # step i's result while step i+1 is already queued (how a serving loop would drive it).  Extra information:
    # the e2e value above stays the one-step-at-a-time figure.
    pipe_ms = None
    if graph is not None and rank == 0 and world == 1:
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
                if fused:
                    ctx.verify_accept_commit(dHb, out_d[0], out_d[1], dhist, dlens, argmax=out_v[0], out=outb)
                else:
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

        pipelined(20)
        torch.cuda.synchronize()
        p0, p1 = ev(), ev()
        p0.record()
        tok_pipe = pipelined(args.steps)
        p1.record()
        torch.cuda.synchronize()
        pipe_ms = p0.elapsed_time(p1) / args.steps
        assert tok_pipe == int(round(acc_mean)) * args.steps, "the pipelined loop committed a different number of tokens"

    # ---- max over ranks, totals over ranks
    from paper_2411_03786_b200.multigpu import reduce_max_sum
    (total_ms, e2e_ms, verify_ms, verify_alone_ms), (acc_total,) = reduce_max_sum(
        [total_ms, e2e_ms, verify_ms, verify_alone_ms], [acc_mean], device=dev)
    ms_per_step = total_ms / args.steps
    value = acc_total / (ms_per_step / 1e3)
    e2e_value = acc_total / (e2e_ms / args.steps / 1e3)

    # ---- roofline of the dominant kernel (the verify contraction)
    bytes_alg = 2.0 * c["V"] * c["d"] + 2.0 * M * c["d"] + 4.0 * M
    flops = 2.0 * M * c["V"] * c["d"]
    t_hbm, t_tc = bytes_alg / (pk["hbm"] * 1e9), flops / (pk["tc_sustained"] * 1e12)
    if t_hbm >= t_tc:
        ach = bytes_alg / (verify_alone_ms / 1e3) / 1e9
        roof = {"bound": "hbm", "achieved": ach, "peak": pk["hbm"], "unit": "GB/s", "frac": ach / pk["hbm"]}
    else:
        ach = flops / (verify_alone_ms / 1e3) / 1e12
        roof = {"bound": "tensor", "achieved": ach, "peak": pk["tc_sustained"], "unit": "TFLOP/s",
                "frac": ach / pk["tc_sustained"]}
    roof.update({"traffic": TRAFFIC.get(args.workload), "kernel": "head_gemm_kernel<ARGMAX> (verify_lmhead_argmax)",
                 "ms_per_launch": verify_alone_ms, "ms_per_launch_eager": verify_eager_ms, "ms_per_launch_graph": verify_graph_ms,
                 "timing": "CUDA events around back-to-back launches on the launching stream (the faster of eager launches and one graph replay)", "algorithmic_bytes": bytes_alg, "flops": flops,
                 "peak_source": pk["source"] + (" sustained" if roof["bound"] == "tensor" else " copy")})

    scaled = scaled_streams(ctx, torch, dev, c, pk) if (not args.no_scaled and rank == 0 and world == 1) else None
    line = None
    if rank == 0:
        cpu = {}
        if args.cpu_budget > 0:
            T_h = tab.cpu().numpy()
            sec, acc_cpu, threads, sample, sampled = oracle_step_time(c, hist_h, lens_h, T_h, H_bits, W_bits, args.cpu_budget)
            cpu = {"value": acc_cpu / sec, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample,
                   "s_per_step": sec}
            if table:
                # the oracle's table build on a row sample, projected to all V rows (each row costs 2 V d flop)
                import oracle
                n_rows = 2 * threads
                t0 = time.perf_counter()
                oracle.model_table(bf16_bits(E), W_bits, c["k_tab"], rows=np.linspace(0, c["V"] - 1, n_rows).astype(np.int64))
                dt = time.perf_counter() - t0
                cpu["table_build"] = {"rows_per_s": n_rows / dt, "projected_s": dt / n_rows * c["V"],
                                      "sample": f"{n_rows} of {c['V']} rows"}
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16", "data": "synthetic", "config": cfg,
                "steps_per_s": world * 1e3 / ms_per_step, "tokens_per_step": acc_total / world / S,
                "phase_ms": {"draft": draft_ms, "verify": verify_ms, "accept": accept_ms,
                             "note": "events between eagerly launched calls: small kernels include the host's launch gap"},
                "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                        "ms_per_step": e2e_ms / args.steps, "mode": "one step at a time: upload, step, host waits for the result",
                        "pipelined_two_deep_ms_per_step": pipe_ms},
                "gpu_launches": int(launches) * world, "launch_mode": "eager" if graph is None else "cuda_graph_replay", "roofline": roof, "table_build": table, "cpu_baseline": cpu,
                "clocks": clk.summary(), "status_bits": status, "copied_fraction": copied}
        if fp8:
            line["fp8_verify"] = fp8
        if scaled:
            line["scaled_streams"] = scaled
        print(json.dumps(line))
    ctx.close()
    if dist is not None:
        dist.destroy_process_group()
    return 0


# DRAM bytes per verify launch from the ncu captures summarised under profiles/ (None = not captured
# for the current kernel).
TRAFFIC = {"C2": 267.0e6, "C3": 1.688e9}


def run_reference(args, c, cfg):
    """The CPU oracle, as it stands, on the host cores: same workload, metric and unit."""
    import oracle
    E, W, hist_h, lens_h, _ = host_inputs(c, 0)
    W_bits = bf16_bits(W)
    k = c["k_tab"]
    # a model table is an input of the step; rank-order rows of it are irrelevant to the timing, so a
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
                      "cpu_baseline": cpu, "gpu_launches": 0,
                      "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
    return 0


if __name__ == "__main__":
    sys.exit(main())
