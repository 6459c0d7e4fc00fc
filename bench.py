#!/usr/bin/env python
"""Benchmark of the diffusion-forcing sampler step on B200.

`--steps K` times exactly K sampler steps AT A FULL WINDOW: the generation is restarted (prefill,
untimed), `window - 1` untimed ramp steps fill the wavefront, then K steps are timed with CUDA events
between barriers; with the fixed exit every timed step commits one token per sequence.  The timed
region is repeated (`--repeats`, default 5) and the median repeat is reported (the paper's protocol:
CUDA events, median over repeats).  `whole_generation_tok_s` is one whole generation, ramp and drain
included.

Workload (N=1): the 3.5B-shape configuration -- bf16 weights, batch 1, prompt 512 random ids,
256 tokens generated greedily, DF sampler with window 32 and one inner iteration per step, next to
the same library's AR decoder with r = 32.  A "step" is one rd_df_step: one pass of the whole hot
path (prelude, core, coda, LM head, sampling, freeze/commit) over the in-flight wavefront.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  `value` is generated tokens/s with everything resident on the device;
`e2e` is the same metric for a whole request through the C ABI with host buffers (prompt upload,
prefill, decode with a device->host read of the commit counter every step, tokens read back).
With --gpus N > 1 (under torchrun) every rank runs an independent replica of the workload: the
path has no exchange step, so there is no data-path collective.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import rd_inputs  # noqa: E402

WORKLOADS = {
    # name: shape, bf16, batch, prompt, gen, window, inner, eps, ar_r, prefill_r, temperature
    "3p5b_b1_p512_g256_W32": dict(shape=rd_inputs.SHAPE_3P5B, bf16=True, batch=1, prompt=512, gen=256, window=32,
                                  inner=1, eps=0.0, ar_r=32, prefill_r=32, temperature=0.0),
    "tiny_fp32_p32_g64_W4": dict(shape=rd_inputs.TINY, bf16=False, batch=1, prompt=32, gen=64, window=4, inner=1,
                                 eps=0.0, ar_r=8, prefill_r=8, temperature=0.0),
    "twin_b1_p512_g256_W32": dict(shape=rd_inputs.TWIN, bf16=True, batch=1, prompt=512, gen=256, window=32,
                                  inner=1, eps=0.0, ar_r=32, prefill_r=32, temperature=0.0),
    # long context (prefill is outside `value`; its recurrence is kept short so that a run stays short)
    "3p5b_b4_p8192_g1024_W32": dict(shape=rd_inputs.SHAPE_3P5B, bf16=True, batch=4, prompt=8192, gen=1024,
                                    window=32, inner=1, eps=0.0, ar_r=32, prefill_r=1, temperature=0.0),
    # batched serving: 16 sequences, ragged prompts, temperature sampling, adaptive exit
    "3p5b_b16_ragged_g512_W16": dict(shape=rd_inputs.SHAPE_3P5B, bf16=True, batch=16, prompt=(128, 2048), gen=512,
                                     window=16, inner=1, eps=1e-3, ar_r=32, prefill_r=1, temperature=1.0),
    # adaptive exit sweep point (window and inner iterations set on the command line)
    "3p5b_b1_p1024_g512_adaptive": dict(shape=rd_inputs.SHAPE_3P5B, bf16=True, batch=1, prompt=1024, gen=512,
                                        window=16, inner=1, eps=1e-3, ar_r=32, prefill_r=4, temperature=0.0),
    # same GEMM and attention shapes as the 3.5B model with 1/1/1 layers and a small vocabulary:
    # about 1.3 GB on the device, for ncu captures
    "3p5b_layers111_v8192_p512_g64_W32": dict(shape=dict(rd_inputs.SHAPE_3P5B, n_prelude=1, n_core=1, n_coda=1, vocab=8192),
                                              bf16=True, batch=1, prompt=512, gen=64, window=32, inner=1, eps=0.0,
                                              ar_r=4, prefill_r=2, temperature=0.0),
    # small cases of the two batched configurations (same kernel shapes, 1/1/1 layers), for ncu captures
    "3p5b_layers111_v8192_b16_p256_g64_W16": dict(shape=dict(rd_inputs.SHAPE_3P5B, n_prelude=1, n_core=1, n_coda=1, vocab=8192),
                                                  bf16=True, batch=16, prompt=256, gen=64, window=16, inner=1, eps=0.0,
                                                  ar_r=4, prefill_r=1, temperature=0.0),
    "3p5b_layers111_v8192_b4_p8192_g64_W32": dict(shape=dict(rd_inputs.SHAPE_3P5B, n_prelude=1, n_core=1, n_coda=1, vocab=8192),
                                                  bf16=True, batch=4, prompt=8192, gen=64, window=32, inner=1, eps=0.0,
                                                  ar_r=4, prefill_r=1, temperature=0.0),
}
DEFAULT_WORKLOAD = "3p5b_b1_p512_g256_W32"
SETTLE_STEPS = 8      # untimed full-window steps enqueued directly in front of the timed ones



def max_over_ranks_sum_tokens(total_ms, tokens, dist=None, device=None):
    """Whole-job aggregation for N independent replicas: the time is the maximum over ranks, the
    tokens are summed.  With dist None (one process) the inputs come back unchanged."""
    if dist is None:
        return float(total_ms), float(tokens)
    import torch
    tm = torch.tensor([total_ms], dtype=torch.float64, device=device)
    tk = torch.tensor([float(tokens)], dtype=torch.float64, device=device)
    dist.all_reduce(tm, op=dist.ReduceOp.MAX)
    dist.all_reduce(tk, op=dist.ReduceOp.SUM)
    return float(tm.item()), float(tk.item())


def full_window_steps(gen, window):
    """Fixed exit (Algorithm 1): rows are appended one per step, so after `window - 1` ramp steps the
    wavefront holds `window` rows and every step commits one token per sequence, until the last of the
    `gen` positions has been appended: steps window .. gen of a generation.  Returns that count."""
    return max(0, gen - window + 1)


def plan_timed_region(steps, gen, window):
    """Segments (ramp_steps, timed_steps) that time exactly `steps` sampler steps at a full window.
    Each segment restarts the generation (prefill, outside the timed region), runs `window - 1`
    untimed ramp steps and then times up to full_window_steps(gen, window) steps.  A generation
    shorter than its window never fills it: then the whole generation is the steady state there is,
    and the segment times it from its first step (ramp 0)."""
    if steps <= 0:
        return []
    full = full_window_steps(gen, window)
    ramp = window - 1
    if full <= 0:
        ramp, full = 0, gen + window - 1
    segs, left = [], steps
    while left > 0:
        n = min(left, full)
        segs.append((ramp, n))
        left -= n
    return segs


def expected_fixed_exit_tokens(segments, batch, gen, window):
    """Tokens the fixed-exit sampler commits inside the timed segments: one per sequence and step at a
    full window; for a generation that never fills its window, step t commits once t >= window."""
    full = full_window_steps(gen, window)
    tok = 0
    for ramp, n in segments:
        if full > 0:
            tok += n * batch
        else:
            tok += batch * max(0, min(n, gen + window - 1) - (window - 1))
    return tok


def ncu_traffic_per_launch(workload):
    """DRAM bytes (read + write) of one average GEMM launch from the ncu capture summarised in
    profiles/, or None when the GEMM source has changed since the capture (the summary records the
    sha256 of the kernel file it was taken with)."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "gemm_tc_kernel_bn32_3p5b_shapes_W32.md")
    src = os.path.join(ROOT, "paper_2510_14961_b200", "csrc", "rd_gemm_tc.cuh")
    if workload != DEFAULT_WORKLOAD or not (os.path.exists(path) and os.path.exists(src)):
        return None
    traffic = sha = None
    for line in open(path):
        if line.startswith("traffic_bytes_per_launch:"):
            traffic = float(line.split(":", 1)[1])
        if line.startswith("kernel_source_sha256:"):
            sha = line.split(":", 1)[1].strip()
    if traffic is None or sha is None:
        return None
    return traffic if hashlib.sha256(open(src, "rb").read()).hexdigest() == sha else None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def prefill_flops(shape, lens, r):
    """FLOPs of prefilling prompts of the given lengths (Section 3.3): rows 0..L-2 of each prompt go
    through the prelude, r simultaneous core passes (adapter included) and the coda layers; causal
    attention of row p costs 4 h (p + 1) per layer (QK^T and PV)."""
    h, I = shape["hidden"], shape["mlp_inner"]
    per_layer = 4 * h * h + 3 * h * I
    n_p, n_r, n_c = shape["n_prelude"], shape["n_core"], shape["n_coda"]
    w_elems = (n_p + n_c) * per_layer + r * (n_r * per_layer + 2 * h * h)
    layers = n_p + n_c + r * n_r
    total = 0
    for L in lens:
        n = max(int(L) - 1, 0)
        total += 2 * n * w_elems + 4 * h * layers * (n * (n + 1) // 2)
    return total


def step_bytes_flops(shape, batch, rows, ctx_sum, inner, esz):
    """Algorithmic bytes and FLOPs of one DF step: every weight matrix streamed once per pass, the
    KV prefix read once per layer per pass for the whole window, K/V of the in-flight rows written."""
    h, I, V = shape["hidden"], shape["mlp_inner"], shape["vocab"]
    per_layer = 4 * h * h + 3 * h * I
    n_p, n_r, n_c = shape["n_prelude"], shape["n_core"], shape["n_coda"]
    w_elems = (n_p + n_c) * per_layer + V * h + inner * (n_r * per_layer + 2 * h * h)
    layers = n_p + n_c + inner * n_r
    kv_read = ctx_sum * 2 * h * esz * layers
    kv_write = rows * 2 * h * esz * layers
    flops = 2 * rows * w_elems + 4 * h * layers * rows * (ctx_sum / max(batch, 1))
    return w_elems * esz + kv_read + kv_write, flops


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows, self.proc, self.index = [], None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx = float(r[1])
            except Exception:
                continue
            for name, v in zip(names, r[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def torch_weights(shape, bf16, device, seed=0, std=0.02):
    """Random-init weights generated on the device (synthetic data; values do not affect timing)."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    out = []
    for name, shp, is_gain in rd_inputs.tensor_specs(**rd_inputs.shape_args(shape)):
        if is_gain:
            out.append(torch.ones(shp, dtype=torch.float32, device=device))
        else:
            t = torch.empty(shp, dtype=torch.float32, device=device).normal_(0.0, std, generator=g)
            out.append(t.to(torch.bfloat16) if bf16 else t)
    return out


def admission_latency(rd, model, stream, shape, wl):
    """Step latency seen by three running sequences while a fourth is admitted (Appendix, "Larger Batch
    Sizes"), with the prompt prefilled in one piece (rd_prefill) and in slices (rd_prefill_sliced):
    one CUDA-event pair per step, 20 steps before the admission and 60 after it."""
    import torch
    B, W, L, r = 4, wl["window"], wl["prompt"] if not isinstance(wl["prompt"], tuple) else wl["prompt"][1], wl["prefill_r"]
    n_steps, at = 80, 20
    N = 60 + n_steps + 2 * W
    prompts = [rd_inputs.make_prompt(L, shape["vocab"], seed=117 + b) for b in range(B)]
    out = {"running_sequences": B - 1, "admitted_prompt": L, "prefill_r": r, "window": W}
    for mode in ("whole", "sliced"):
        sess = rd.Session(model, batch=B, max_context=L + N + 8, max_window=W, max_iters_per_pos=64, max_new_tokens=N,
                          seed=1, stream=stream.cuda_stream)
        for b in range(B - 1):
            sess.prefill(b, prompts[b], 1)
        for _ in range(2 * W):
            sess.df_step(W, wl["inner"], 0.0)
        sess.sync()
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(n_steps + 1)]
        with torch.cuda.stream(stream):
            evs[0].record(stream)
            for i in range(n_steps):
                if i == at:
                    (sess.prefill if mode == "whole" else sess.prefill_sliced)(B - 1, prompts[B - 1], r)
                sess.df_step(W, wl["inner"], 0.0)
                evs[i + 1].record(stream)
        sess.sync()
        ms = [evs[i].elapsed_time(evs[i + 1]) for i in range(n_steps)]
        out[mode] = {"step_ms_before": sorted(ms[:at])[at // 2], "worst_step_ms": max(ms), "total_ms": sum(ms)}
        sess.close()
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2510_14961_b200 as rd

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    wl = dict(WORKLOADS[args.workload])
    if args.prefill_r > 0:
        wl["prefill_r"] = args.prefill_r
    if args.temperature >= 0.0:
        wl["temperature"] = args.temperature
    if args.top_p > 0.0:
        wl["top_p"] = args.top_p
    if args.eps >= 0.0:
        wl["eps"] = args.eps
    if args.window > 0:
        wl["window"] = args.window
    if args.inner > 0:
        wl["inner"] = args.inner
    shape, B, N, W = wl["shape"], wl["batch"], wl["gen"], wl["window"]
    if isinstance(wl["prompt"], tuple):      # ragged batch: lengths uniform in [lo, hi]
        lens = [int(x) for x in rd_inputs.make_prompt_lengths(B, wl["prompt"][0], wl["prompt"][1], seed=4)]
    else:
        lens = [wl["prompt"]] * B
    L = max(lens)
    esz = 2 if wl["bf16"] else 4
    peaks = load_peaks()

    tensors = torch_weights(shape, wl["bf16"], dev, seed=rank)
    model = rd.Model(shape["hidden"], shape["n_heads"], shape["head_dim"], shape["mlp_inner"], shape["n_prelude"],
                     shape["n_core"], shape["n_coda"], shape["vocab"], tensors,
                     dtype=rd.RD_BF16 if wl["bf16"] else rd.RD_F32, elem_bytes=esz)
    del tensors
    torch.cuda.empty_cache()
    stream = torch.cuda.Stream(device=dev)
    max_ctx = L + N + 8
    prompts = [rd_inputs.make_prompt(lens[b], shape["vocab"], seed=17 + b) for b in range(B)]
    pinned = [torch.from_numpy(p).pin_memory() for p in prompts]

    def new_session(window, temperature=0.0):
        ses = rd.Session(model, batch=B, max_context=max_ctx, max_window=window, max_iters_per_pos=64,
                         max_new_tokens=N, temperature=temperature, seed=1234, stream=stream.cuda_stream,
                         top_p=wl.get("top_p", 0.0))
        if args.unfused_swiglu:
            ses.set_fused_swiglu(False)     # A/B: gate/up leaves partial sums, SwiGLU in a kernel of its own
        if args.attention_path >= 0:
            ses.set_attention_path(args.attention_path)   # A/B: 3 default, 2 mma.sync prefill, 1 cp.async, 0 one block per row
        if args.unchained:
            ses.set_launch_chaining(False)  # A/B: ordinary stream-ordered launches
        return ses

    def prefill(sess):
        for b in range(B):
            sess.prefill(b, pinned[b].numpy(), wl["prefill_r"])

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- DF sampler, device-resident ----------------------------------------------------------
    sess = new_session(W, wl["temperature"])
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    prefill(sess)                            # first call: also loads the kernels
    sess.sync()
    ev0.record(stream)
    prefill(sess)
    ev1.record(stream)
    sess.sync()
    prefill_s = ev0.elapsed_time(ev1) * 1e-3
    warm = max(args.warmup, 3)
    for _ in range(warm):
        sess.df_step(W, wl["inner"], wl["eps"])
    sess.sync()
    adaptive = wl["eps"] > 0
    if not adaptive:
        steps_per_gen = N + W - 1            # fixed exit: one token per step after the ramp
        K = args.steps if args.steps > 0 else (full_window_steps(N, W) or steps_per_gen)
        segments = plan_timed_region(K, N, W)
    else:
        # adaptive exit: the number of steps depends on the latents; an untimed generation with the
        # same seeds counts them (every run of the same inputs takes the same steps).  The timed
        # region starts once the oldest row can have reached the iteration cap.
        prefill(sess)
        steps_per_gen = 0
        while not all(sess.committed(b)[1] for b in range(B)) and steps_per_gen < 64 * (N + W):
            sess.df_step(W, wl["inner"], wl["eps"])
            steps_per_gen += 1
        if args.steps > 0:
            ramp = min(max(W, -(-64 // wl["inner"])) - 1, max(steps_per_gen - 1, 0))
            K = min(args.steps, steps_per_gen - ramp)
            segments = [(ramp, K)]
        else:
            K = steps_per_gen
            segments = [(0, K)]

    def run_segments(segs):
        """Times the segments' steps; returns (ms, tokens committed inside, kernel launches inside,
        algorithmic bytes and FLOPs of the timed steps as the library counted them)."""
        ms, tok, launches, work_b, work_f = 0.0, 0, 0, 0, 0
        for ramp, n in segs:
            prefill(sess)                   # restart the generation (outside the timed region)
            for _ in range(ramp):
                sess.df_step(W, wl["inner"], wl["eps"])
            st0 = sess.stats()              # (synchronises: the device is idle when the region starts)
            # full-window steps enqueued back to back in front of the timed ones, so that the timed steps
            # see a busy launch queue and settled clocks instead of the idle device the host's
            # synchronisation left; fixed exit only (every such step is like the timed ones)
            settle = SETTLE_STEPS if (not adaptive and ramp + SETTLE_STEPS + n <= N) else 0
            barrier()
            with torch.cuda.stream(stream):
                for _ in range(settle):
                    sess.df_step(W, wl["inner"], wl["eps"])
                ev0.record(stream)
                for _ in range(n):
                    sess.df_step(W, wl["inner"], wl["eps"])
                ev1.record(stream)
            barrier()
            ms += ev0.elapsed_time(ev1)
            st1 = sess.stats()
            share = n / float(n + settle)   # the settle steps are full-window steps like the timed ones
            tok += st1["tokens_committed"] - st0["tokens_committed"] - settle * B
            launches += int(round((st1["kernel_launches"] - st0["kernel_launches"]) * share))
            work_b += (st1["weight_bytes"] + st1["kv_bytes"] - st0["weight_bytes"] - st0["kv_bytes"]) * share
            work_f += (st1["flops"] - st0["flops"]) * share
        return ms, tok, launches, work_b, work_f

    clocks = ClockSampler(local)
    clocks.start()
    reps = []
    for _ in range(max(args.repeats, 1)):
        ms, tok, launches0, work_b, work_f = run_segments(segments)
        ms_max, tok_all = max_over_ranks_sum_tokens(ms, tok, dist if world > 1 else None, dev)
        reps.append((ms_max, tok_all))
    clk = clocks.stop()
    if not adaptive:
        want = expected_fixed_exit_tokens(segments, B, N, W)
        if any(t != world * want for _, t in reps):
            raise RuntimeError(f"timed region committed {[t for _, t in reps]} tokens, expected {world * want} per repeat")
    rates = sorted(t / (m / 1e3) for m, t in reps)
    if rates[len(rates) // 2] <= 0.0:
        raise RuntimeError("the timed region committed no token: time more steps (adaptive exit commits in bursts)")
    order = sorted(range(len(reps)), key=lambda i: reps[i][1] / reps[i][0])
    total_ms_max, tokens_all = reps[order[len(order) // 2]]          # the median repeat
    df_tok_s = tokens_all / (total_ms_max / 1e3)
    ms_per_step = total_ms_max / K
    timed_ctx_sum = sum(lens) + B * (sum(r + n / 2.0 for r, n in segments) / max(len(segments), 1))

    # whole generation (ramp and drain included), timed once
    prefill(sess)
    barrier()
    with torch.cuda.stream(stream):
        ev0.record(stream)
        for _ in range(steps_per_gen):
            sess.df_step(W, wl["inner"], wl["eps"])
        ev1.record(stream)
    barrier()
    gen_ms, gen_tok = max_over_ranks_sum_tokens(ev0.elapsed_time(ev1), B * N, dist if world > 1 else None, dev)
    whole_generation_tok_s = gen_tok / (gen_ms / 1e3)

    # ---- per-kernel roofline: event pairs around every GEMM / attention launch -----------------
    rows_full = B * W
    prefill(sess)
    for _ in range(W + 2):                  # reach the full window
        sess.df_step(W, wl["inner"], wl["eps"])
    sess.sync()
    sess.profile_enable(True)
    prof_steps = 20
    for _ in range(prof_steps):
        sess.df_step(W, wl["inner"], wl["eps"])
    prof = sess.profile_read()
    sess.profile_enable(False)
    gemm_gbs = prof["gemm_weight_bytes"] / (prof["gemm_ms"] * 1e-3) / 1e9 if prof["gemm_ms"] > 0 else 0.0
    # the same GEMM launches as a chain of their own (the launch mode of the timed steps: programmatic
    # dependent launches, no event between them), timed with one event pair around 20 steps' worth
    chain = None
    try:
        sess.gemm_sequence(rows_full, 2)                    # warm
        sess.sync()
        with torch.cuda.stream(stream):
            ev0.record(stream)
            chain_bytes, chain_launches = sess.gemm_sequence(rows_full, 20)
            ev1.record(stream)
        sess.sync()
        chain_ms = ev0.elapsed_time(ev1)
        chain = {"achieved": chain_bytes / (chain_ms * 1e-3) / 1e9, "launches": chain_launches,
                 "avg_us": 1e3 * chain_ms / chain_launches, "bytes_per_launch": chain_bytes / chain_launches}
    except rd.RdError:
        pass                                                # float32 configuration: no tensor-core GEMM path
    attn_gbs = prof["attn_kv_bytes"] / (prof["attn_ms"] * 1e-3) / 1e9 if prof["attn_ms"] > 0 else 0.0
    tc_launches = sess.stats()["tc_gemm_launches"]
    # step roofline for the steps that were timed: algorithmic bytes and FLOPs as the library's
    # counters (rd_stats) have them for exactly those steps -- a full window of rows, the contexts
    # they had; the formula beside it is the hand-worked one the tests pin
    step_b, step_f = work_b / K, work_f / K
    formula_b, formula_f = step_bytes_flops(shape, B, B * W, timed_ctx_sum, wl["inner"], esz)
    t_roof = max(step_b / (peaks["hbm_gbs"] * 1e9), step_f / (peaks["bf16_tflops_sustained"] * 1e12))
    lib_stats = sess.stats()
    sess.close()
    pf_flops = prefill_flops(shape, lens, wl["prefill_r"])

    # ---- AR decoder from the same library -------------------------------------------------------
    ar = new_session(1)
    prefill(ar)
    for _ in range(3):
        ar.ar_step(wl["ar_r"])
    prefill(ar)
    n_ar = min(N, args.ar_tokens)
    barrier()
    with torch.cuda.stream(stream):
        ev0.record(stream)
        for _ in range(n_ar):
            ar.ar_step(wl["ar_r"])
        ev1.record(stream)
    barrier()
    ar_ms = ev0.elapsed_time(ev1)
    ar_tok_s = B * n_ar / (ar_ms / 1e3)
    ar_b, ar_f = step_bytes_flops(shape, B, B, sum(lens) + B * (n_ar // 2), wl["ar_r"], esz)
    ar_roof = max(ar_b / (peaks["hbm_gbs"] * 1e9), ar_f / (peaks["bf16_tflops_sustained"] * 1e12))
    ar.close()

    # ---- end to end through the C ABI with host buffers ------------------------------------------
    e2e = new_session(W, wl["temperature"])
    out_tokens = [torch.empty(max_ctx + 1, dtype=torch.int32).pin_memory() for _ in range(B)]
    prefill(e2e)
    for _ in range(3):
        e2e.df_step(W, wl["inner"], wl["eps"])
    e2e.sync()
    barrier()
    t0 = time.perf_counter()
    prefill(e2e)                                            # H2D of the prompts + prefill
    e2e.sync()
    e2e_prefill_s = time.perf_counter() - t0
    n_steps_e2e, d2h = 0, 0
    poll_bytes = 4 * (4 + 2 * B)                           # status word, |y_frozen| and done flag per sequence
    pending = None
    while True:
        # every step's result (commit counters, done flags) is read back: the copy is enqueued behind
        # the step, the next step is enqueued, and only then does the host wait for the copy
        e2e.df_step(W, wl["inner"], wl["eps"])
        n_steps_e2e += 1
        ticket = e2e.poll_begin()                          # D2H behind this step
        d2h += poll_bytes
        if pending is not None:
            _, done_all = e2e.poll_end(pending)
            if done_all:
                e2e.poll_end(ticket)
                break
        pending = ticket
        if n_steps_e2e > 100000:
            break
    got = 0
    for b in range(B):
        t = e2e.tokens(b, out=out_tokens[b].numpy())       # D2H: the generated sequence
        got += len(t) - lens[b]
        d2h += 4 * len(t)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    e2e_s_max, got_all = max_over_ranks_sum_tokens(e2e_s, got, dist if world > 1 else None, dev)
    e2e_tok_s = got_all / e2e_s_max
    e2e.close()

    # Dominant kernel: the weight-streaming GEMM.  `achieved` is measured in the launch mode of the timed
    # steps (a chain of programmatic dependent launches: the 34 GEMM launches of a step back to back, 20
    # steps' worth inside one event pair); `alone` is the same launches each inside its own event pair
    # during real steps (the pair breaks the chain, so the launch gap and a cold start are included).
    alone = {"achieved": gemm_gbs, "frac": gemm_gbs / peaks["hbm_gbs"], "launches": prof["gemm_launches"],
             "avg_us": 1e3 * prof["gemm_ms"] / max(prof["gemm_launches"], 1),
             "bytes_per_launch": prof["gemm_weight_bytes"] / max(prof["gemm_launches"], 1)}
    best = chain if chain else alone
    roofline = {"bound": "hbm", "kernel": "weight-streaming GEMM (all projections of the step)",
                "achieved": best["achieved"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": best["achieved"] / peaks["hbm_gbs"], "traffic": ncu_traffic_per_launch(args.workload),
                "launches": best["launches"], "avg_us": best["avg_us"], "bytes_per_launch": best["bytes_per_launch"],
                "how": "GEMM launches of 20 steps as one chain of programmatic dependent launches, one CUDA-event pair"
                       if chain else "one CUDA-event pair around every GEMM launch of 20 steps",
                "alone": alone, "peak_source": peaks["source"]}
    line = {
        "metric": "generated tok/s at 1 B200, DF sampler vs AR recurrence; % of step roofline",
        "value": df_tok_s, "unit": "tok/s", "n_gpus": world, "steps": K, "warmup": warm,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "repeats": {"n": len(reps), "statistic": "median", "tok_s": rates, "min": rates[0], "max": rates[-1]},
        "timed_region": {"segments": [{"untimed_ramp_steps": r, "timed_steps": n} for r, n in segments],
                         "untimed_settle_steps_in_stream": 0 if adaptive else SETTLE_STEPS,
                         "what": "steps at a full window, every one committing" if not adaptive else
                                 "steps after the ramp to the iteration cap (adaptive exit commits in bursts)"},
        "whole_generation_tok_s": whole_generation_tok_s,
        "dtype": "bf16" if wl["bf16"] else "f32", "data": "synthetic",
        "config": {"workload": args.workload, "batch": B, "prompt": L if len(set(lens)) == 1 else lens, "generate": N, "window": W,
                   "steps_per_generation": steps_per_gen, "tokens_per_step": tokens_all / (world * K) if K else None,
                   "inner_iters": wl["inner"], "exit_threshold": wl["eps"], "ar_r": wl["ar_r"],
                   "temperature": wl["temperature"], "top_p": wl.get("top_p", 0.0),
                   "l2": "inputs larger than L2 (weights streamed per step: %.2f GB)" % (step_b / 1e9),
                   "multi_gpu": "replicas only (no data-path collective)",
                   "variant": {"fused_swiglu": not args.unfused_swiglu, "chained_launches": not args.unchained,
                               "attention_path": 3 if args.attention_path < 0 else args.attention_path}},
        "df_tok_s": df_tok_s, "ar_tok_s": ar_tok_s, "df_over_ar": df_tok_s / ar_tok_s if ar_tok_s else None,
        "ar_tokens_timed": n_ar, "ar_ms_per_token": ar_ms / n_ar,
        "prefill": {"seconds": prefill_s, "flops": pf_flops, "tflops": pf_flops / prefill_s / 1e12,
                    "frac_of_bf16_sustained": pf_flops / prefill_s / 1e12 / peaks["bf16_tflops_sustained"],
                    "prompts": L if len(set(lens)) == 1 else lens, "r": wl["prefill_r"], "timing": "CUDA events on the session's stream"},
        "step_roofline": {"bound": "hbm" if step_b / (peaks["hbm_gbs"] * 1e9) >= step_f / (peaks["bf16_tflops_sustained"] * 1e12) else "tensor",
                          "bytes_per_step": step_b, "flops_per_step": step_f, "t_roof_ms": t_roof * 1e3,
                          "source": "rd_stats counters over the timed steps", "formula_bytes_per_step": formula_b,
                          "df_frac": t_roof * 1e3 / ms_per_step,
                          "ar_t_roof_ms": ar_roof * 1e3, "ar_frac": ar_roof / (ar_ms / n_ar / 1e3),
                          "peak_source": peaks["source"]},
        "roofline": roofline,
        "attention": {"achieved_gbs": attn_gbs, "launches": prof["attn_launches"],
                      "avg_us": 1e3 * prof["attn_ms"] / max(prof["attn_launches"], 1)},
        "kernel_time_shares": {k: prof[k + "_ms"] / max(prof["gemm_ms"] + prof["attn_ms"] + prof["other_ms"], 1e-9)
                               for k in ("gemm", "attn", "other")},
        "gemm_share_of_step": prof["gemm_ms"] / max(prof["gemm_ms"] + prof["attn_ms"] + prof["other_ms"], 1e-9),
        "clocks": clk,
        "e2e": {"value": e2e_tok_s, "unit": "tok/s", "h2d_bytes_per_step": 4.0 * sum(lens) / n_steps_e2e,
                "d2h_bytes_per_step": d2h / n_steps_e2e, "steps": n_steps_e2e, "prefill_s": e2e_prefill_s,
                "total_s": e2e_s, "includes": "prompt upload, prefill, decode, a device-to-host read of the commit counters and done flags behind every step "
                            "(read one step late, so one step past the end is enqueued as a no-op), token readback"},
        "gpu_launches": int(launches0), "tc_gemm_launches": int(tc_launches),
        "commit_hist": lib_stats["commit_hist"],
    }
    if args.admission:
        line["admission"] = admission_latency(rd, model, stream, shape, wl)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(args.workload, budget_s=args.cpu_budget)
    if world > 1:
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line))


# ---------------------------------------------------------------------------------------------
# The oracle, timed as it stands on the host cores (reported baseline, not the target)
# ---------------------------------------------------------------------------------------------
def _oracle_weights(shape, bf16):
    """Random-init weights for the oracle.  At the 3.5B shape generating 3.5e9 normals takes about a
    minute; the values do not affect timing, so one layer's matrices are drawn and reused by every
    layer when host memory is short (stated in the result)."""
    import psutil
    specs = rd_inputs.tensor_specs(**rd_inputs.shape_args(shape))
    need = sum(int(np.prod(s)) for _, s, _ in specs) * 4
    full = psutil.virtual_memory().available > 3 * need + (8 << 30)
    rng = np.random.default_rng(0)
    w, cache = {}, {}
    for name, shp, is_gain in specs:
        if is_gain:
            w[name] = np.ones(shp, dtype=np.float32)
            continue
        key = name.split(".")[-1] if not full else name
        if key not in cache:
            a = rng.standard_normal(shp, dtype=np.float32)
            a *= np.float32(0.02)
            cache[key] = a
        w[name] = cache[key]
    return w, full


def oracle_steps(workload, n_steps, budget_s=25.0):
    """Runs the oracle's DF sampler on a bounded sample of the workload; returns per-step seconds."""
    from oracle import rd_oracle as orc
    wl = WORKLOADS[workload]
    shape = wl["shape"]
    big = shape["hidden"] >= 2048
    w, full = _oracle_weights(shape, wl["bf16"])
    cfg = orc.RDConfig(**shape)
    L = 16 if big else wl["prompt"]
    W = wl["window"]
    model = orc.RDModel(cfg, w, dtype=np.float32 if big else np.float64, contract=False, max_ctx=L + wl["gen"] + 8)
    sm = orc.Sampler(model, seed=1234, temperature=wl["temperature"], top_p=wl.get("top_p", 0.0) or 1.0)
    prompt = rd_inputs.make_prompt(L, shape["vocab"], seed=17)
    sq = sm.prefill(0, prompt, 1 if big else wl["prefill_r"], wl["gen"])
    times, t_start = [], time.perf_counter()
    ramp = 0
    while len(sq.window) < W and not sq.done:            # untimed ramp to the full window
        sm.df_step(sq, W, wl["inner"], wl["eps"])
        ramp += 1
        if time.perf_counter() - t_start > 4 * budget_s:
            break
    for _ in range(n_steps):
        if sq.done:
            break
        t0 = time.perf_counter()
        sm.df_step(sq, W, wl["inner"], wl["eps"])
        times.append(time.perf_counter() - t0)
        if sum(times) > budget_s:
            break
    import threadpoolctl
    threads = max([p.get("num_threads", 1) for p in threadpoolctl.threadpool_info()] + [1])
    sample = (f"oracle DF steps at a full window of {len(sq.window)} rows, prompt {L} tokens"
              f" (prefill r={1 if big else wl['prefill_r']}), {ramp} untimed ramp steps, {len(times)} timed steps; "
              f"dtype {'float32' if big else 'float64'}; weights {'distinct per layer' if full else 'one layer reused'}")
    return times, threads, sample, len(sq.window)


def cpu_baseline(workload, budget_s=25.0):
    times, threads, sample, rows = oracle_steps(workload, 6, budget_s)
    if not times:
        return {"value": None, "unit": "tok/s", "cores": threads, "kind": "oracle", "sample": sample}
    # steady state of the fixed-exit sampler commits one token per step
    return {"value": 1.0 / float(np.mean(times)), "unit": "tok/s", "cores": threads, "kind": "oracle",
            "sample": sample, "s_per_step": float(np.mean(times))}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    K = args.steps if args.steps > 0 else 4
    Wm = max(args.warmup, 0)
    times, threads, sample, rows = oracle_steps(args.workload, K + Wm, budget_s=120.0)
    timed = times[Wm:] if len(times) > Wm else times
    wl = WORKLOADS[args.workload]
    s_step = float(np.mean(timed))
    v = 1.0 / s_step
    print(json.dumps({
        "impl": "reference", "metric": "generated tok/s at 1 B200, DF sampler vs AR recurrence; % of step roofline",
        "value": v, "unit": "tok/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": len(timed),
        "warmup": Wm, "ms_per_step": s_step * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32" if wl["shape"]["hidden"] >= 2048 else "f64", "data": "synthetic",
        "config": {"workload": args.workload, "batch": 1, "window": wl["window"], "inner_iters": wl["inner"]},
        "cpu_baseline": {"value": v, "unit": "tok/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": "tok/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0,
                    help="timed DF steps at a full window (default: every full-window step of one generation)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--repeats", type=int, default=5, help="repeats of the timed region; the median is reported")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--ar-tokens", type=int, default=24)
    ap.add_argument("--window", type=int, default=0, help="override the workload's window (sweeps)")
    ap.add_argument("--eps", type=float, default=-1.0, help="override the workload's exit threshold (0: fixed exit)")
    ap.add_argument("--inner", type=int, default=0, help="override the workload's inner iterations per step (sweeps)")
    ap.add_argument("--prefill-r", type=int, default=0, help="override the workload's prefill recurrence (profiling aid)")
    ap.add_argument("--temperature", type=float, default=-1.0, help="override the workload's sampling temperature (sweeps)")
    ap.add_argument("--top-p", type=float, default=0.0, help="top-p of Sample (sweeps; needs a temperature > 0)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--unfused-swiglu", action="store_true", help="A/B: SwiGLU as a separate kernel")
    ap.add_argument("--attention-path", type=int, default=-1, help="A/B: 3 default (TMA ring; tcgen05 prefill), 2 without the tcgen05 prefill kernel, 1 cp.async, 0 SIMT")
    ap.add_argument("--unchained", action="store_true", help="A/B: no programmatic dependent launch")
    ap.add_argument("--admission", action="store_true",
                    help="also measure the step latency of running sequences while one more is admitted (whole vs sliced prefill)")
    ap.add_argument("--cpu-budget", type=float, default=20.0)
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
