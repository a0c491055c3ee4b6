#!/usr/bin/env python
"""Benchmark of the Mira MoE-layer hot path on B200.

    python bench.py --gpus N --steps K --warmup W [--workload mixtral|fine|tiny] [--tokens T]
    python bench.py --impl reference ...        # the CPU oracle timed on the host cores

One step = one pass of the whole hot path (router, top-k, grouping, fused dequant + up/gate,
down, combine) over one batch of T tokens of synthetic input, through the C ABI. The default
workload is the Mixtral-8x7B-shaped layer (C 4096, R 14336, 8 experts, top-2, all experts
resident) at decode batch 32. Metric: MoE-layer tokens/s.

Prints ONE JSON line. `value` is measured with inputs resident in HBM; `e2e` includes the
host->device copy of the hidden states from pinned memory and the device->host copy of the
output every step. `roofline` is for the dominant kernel (the fused dequant + up/gate stream),
timed per launch with CUDA events in a second, profiled pass over the same steps.
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

from paper_2609_38090_b200 import inputs  # noqa: E402

METRIC = "moe_layer_tokens_per_s"
UNIT = "tokens/s"
N_BATCHES = 4          # distinct hidden-state batches rotated over the steps
QUANTIZE_STATS: dict = {}        # filled by build_layer: time and rate of mira_quantize_experts


def shape_of(name: str, tokens: int | None) -> inputs.LayerShape:
    base = {"mixtral": inputs.MIXTRAL, "mixtral22": inputs.MIXTRAL22, "fine": inputs.FINE, "tiny": inputs.TINY}[name]
    return base.with_tokens(tokens if tokens else base.T)


NOMINAL_HBM_GBS = 8000.0       # the vendor's figure the benchmark spec quotes; fractions of it are reported beside the measured ones
NOMINAL_TFLOPS = 2250.0        # dense bf16 / fp16 tensor rate of the data sheet


def peaks() -> tuple[float, float, float, str]:
    """(HBM GB/s, bf16 TFLOP/s sustained, bf16 TFLOP/s burst, source) -- measured on this machine if the file exists.
    The copy rate and the cuBLAS rates were taken with torch on this machine's B200s; the sustained rate is under the
    power cap (SM clock near 1.34 GHz), the burst rate is a short run at full clock."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), float(d["bf16_tflops_sustained"]), float(d.get("bf16_tflops", d["bf16_tflops_sustained"])), "measured"
    return 6650.0, 1400.0, 1590.0, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows: list[list[str]] = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "10"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def mark(self):
        return len(self.rows)

    def wait_started(self, timeout_s: float = 3.0):
        """nvidia-smi takes a few hundred ms to print its first row: do not start the timed region before it."""
        t0 = time.perf_counter()
        while self.proc and not self.rows and time.perf_counter() - t0 < timeout_s:
            time.sleep(0.01)

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self, lo: int, hi: int | None = None) -> dict:
        rows = self.rows[lo:hi] or self.rows[-3:]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------------------------
# CPU oracle leg (cpu_baseline and --impl reference)
# --------------------------------------------------------------------------------------------
FMT = 0      # blob format of the run (--format): 0 = the paper's shared scale, 1 = per-matrix scales


def oracle_sample(sh: inputs.LayerShape, n_tokens: int, repeats: int = 1, target_seconds: float | None = None):
    """Times the oracle, as it stands, on the first n_tokens tokens of the workload's batches. Only the experts
    those tokens need are generated and compressed (untimed set-up). With target_seconds the sample is whole
    batches of the workload, one after the other, until that much CPU time has been spent (at most 16 batches)."""
    import oracle
    wr, bias = inputs.router(sh)
    n_batches = 16 if target_seconds else 1
    xs = [inputs.hidden(sh, sh.T, step=i)[:n_tokens] for i in range(n_batches)]
    blobs = [None] * (sh.E + sh.n_shared)

    def ensure(x):
        idx, _, _, _ = oracle.topk_softmax(oracle.linear_scores(x, wr, bias), sh.k)
        need = sorted(set(idx.ravel().tolist()) | set(range(sh.E, sh.E + sh.n_shared)))
        for e in need:
            if blobs[e] is None:
                blobs[e] = oracle.quantize_expert(*inputs.expert_weights(sh, e), fmt=FMT)
    cores = len(os.sched_getaffinity(0))
    times = []
    if target_seconds:
        total, used = 0.0, 0
        for x in xs:
            ensure(x)
            t0 = time.perf_counter()
            oracle.moe_layer(x, wr, bias, blobs, sh.R, sh.k, n_shared=sh.n_shared, fmt=FMT)
            dt = time.perf_counter() - t0
            times.append(dt); total += dt; used += 1
            if total >= target_seconds:
                break
        touched = sum(1 for b in blobs if b is not None)
        return times, cores, (f"{used} batches of {n_tokens} tokens ({touched} experts touched), full layer per token, "
                              f"{total:.1f} s of CPU time")
    ensure(xs[0])
    for _ in range(repeats):
        t0 = time.perf_counter()
        oracle.moe_layer(xs[0], wr, bias, blobs, sh.R, sh.k, n_shared=sh.n_shared, fmt=FMT)
        times.append(time.perf_counter() - t0)
    touched = sum(1 for b in blobs if b is not None)
    return times, cores, f"{n_tokens} of {sh.T} tokens of batch 0 ({touched} experts touched), full layer per token"


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sh = shape_of(args.workload, args.tokens)
    n_tok = max(1, min(sh.T, args.ref_tokens))
    times, cores, sample = oracle_sample(sh, n_tok, repeats=args.warmup + args.steps)
    timed = times[args.warmup:]
    ms = 1e3 * sum(timed) / len(timed)
    value = n_tok / (ms / 1e3)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(sh),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(sh: inputs.LayerShape) -> dict:
    return {"workload": f"{sh.name} layer: hidden {sh.C}, ffn {sh.R}, {sh.E} experts top-{sh.k}"
                        f"{' + %d shared' % sh.n_shared if sh.n_shared else ''}, {sh.T} tokens per step, "
                        + ("all experts resident in the per-matrix-scale INT8 format (the format variant)" if FMT else
                           "all experts resident in the paper's shared-scale INT8 format"),
            "tokens": sh.T, "hidden": sh.C, "ffn": sh.R, "experts": sh.E, "top_k": sh.k, "shared": sh.n_shared,
            "zipf_a": sh.zipf_a, "seed": sh.seed,
            "l2": "expert weights (%.2f GB) far exceed the 126 MB L2 and %d hidden batches rotate; no flush"
                  % ((sh.E + sh.n_shared) * sh.expert_bytes / 1e9, N_BATCHES)}


# --------------------------------------------------------------------------------------------
# CUDA leg
# --------------------------------------------------------------------------------------------
def build_layer(sh: inputs.LayerShape, dev, out_fp32=False):
    """Seeded synthetic layer on the device: weights drawn with torch's CUDA generator (same
    distributions as the numpy recipe of the tests) and compressed by mira_quantize_experts."""
    import torch
    from paper_2609_38090_b200 import binding
    m = binding.Mira(sh.C, sh.R, sh.E, n_shared=sh.n_shared, n_layers=32, max_tokens=sh.T, max_top_k=sh.k,
                     out_fp32=out_fp32, device=dev, fmt=FMT)
    g = torch.Generator(device=dev)
    g.manual_seed(1000 + sh.seed)
    n = sh.E + sh.n_shared
    blobs = torch.empty((n, m.expert_bytes), dtype=torch.uint8, device=dev)
    q_ms = 0.0
    qa, qb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for e in range(n):
        w1 = torch.randn((1, sh.R, sh.C), generator=g, device=dev) * 0.02
        w2 = torch.randn((1, sh.C, sh.R), generator=g, device=dev) * 0.02
        w3 = torch.randn((1, sh.R, sh.C), generator=g, device=dev) * 0.02
        qa.record()
        m.quantize_experts(w1, w2, w3, out=blobs[e:e + 1])                 # S0 (offline step, timed for the record)
        qb.record()
        qb.synchronize()
        q_ms += qa.elapsed_time(qb)
        del w1, w2, w3
    # S0 reads W2 twice (column abs-max, then codes), W1 and W3 once, and writes the blob; the per-matrix format
    # reads every matrix once
    QUANTIZE_STATS.update(ms_per_expert=q_ms / n,
                          gbs=n * ((12.0 if FMT else 16.0) * sh.R * sh.C + m.expert_bytes) / (q_ms / 1e3) / 1e9)
    wr_np, bias_np = inputs.router(sh)
    wr = torch.from_numpy(wr_np).to(torch.bfloat16).to(dev)
    bias = torch.from_numpy(bias_np).to(dev)
    xs = [torch.from_numpy(inputs.hidden(sh, sh.T, step=i)).to(torch.bfloat16) for i in range(N_BATCHES)]
    slots = binding.slot_table(blobs)
    slot_map = torch.arange(n, dtype=torch.int32, device=dev)
    torch.cuda.synchronize(dev)
    return m, blobs, slots, slot_map, wr, bias, xs


def algorithmic_bytes(sh, counts) -> tuple[int, int]:
    """(bytes of the whole layer step, bytes of the up/gate kernel) for one batch: compressed bytes of
    the experts actually hit plus activations, router and the fp16 intermediate."""
    active = int(sum(1 for c in counts if c > 0))
    pairs = int(sum(counts))
    Be = 3 * sh.R * sh.C + 2 * sh.R + (2 * sh.R + 2 * sh.C if FMT else 0)
    layer = active * Be + 2 * sh.T * sh.C * 2 + sh.E * sh.C * 2
    upgate = active * (2 * sh.R * sh.C + (4 if FMT else 2) * sh.R) + sh.T * sh.C * 2 + pairs * sh.R * 2
    return layer, upgate


def reduce_max_ms(ms: float, dev, world: int) -> float:
    """Max over ranks of an elapsed time (the only cross-rank step: the path itself has no exchange)."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_throughput(tokens: int, steps: int, world: int, ms_total: float) -> float:
    """Whole-job tokens/s of `world` independent replicas that each ran `steps` steps of `tokens` tokens."""
    return world * tokens * steps / (ms_total / 1e3)


MIN_SECONDS = 0.5      # every timed region lasts at least this long (--min-seconds; 0 = one block, for profiler runs)


def timed_blocks(fn, steps, barrier, dev, world, min_seconds=None, finish=None, max_blocks=400):
    """Times blocks of exactly `steps` steps, each bracketed by barrier + synchronize on both sides and CUDA events
    on the launching stream, repeated until the blocks together last at least `min_seconds` (so that the clock
    sampler sees the timed region). Returns the per-block times in ms (max over ranks)."""
    import torch
    if min_seconds is None:
        min_seconds = MIN_SECONDS
    blocks, total = [], 0.0
    while True:
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        a.record()
        for i in range(steps):
            fn(i)
        if finish:
            finish()                                # e.g. make the stop event wait for copies on other streams
        b.record()
        barrier()
        ms = reduce_max_ms(a.elapsed_time(b), dev, world)
        blocks.append(ms)
        total += ms
        if total >= 1e3 * min_seconds or len(blocks) >= max_blocks:
            return blocks


def block_stats(blocks, steps):
    med = statistics.median(blocks)
    return {"ms_per_step": med / steps, "ms_per_step_best": min(blocks) / steps, "blocks": len(blocks),
            "timed_seconds": sum(blocks) / 1e3}


def clock_record(sampler, lo, hi, ms_per_step):
    """Clock summary of the samples taken inside one timed region, plus time x clock (ms x MHz) so that steps timed
    at different clocks can be compared."""
    if sampler is None:
        return None
    c = sampler.summary(lo, hi) if hi > lo else sampler.summary(lo, max(sampler.mark(), lo + 1))
    c["samples_in_timed_region"] = max(hi - lo, 0)
    c["ms_per_step_x_sm_mhz"] = (ms_per_step * c["sm_mhz"]) if c.get("sm_mhz") else None
    return c


def traffic_ratio(key: str):
    """DRAM bytes of one launch relative to its algorithmic bytes, from the ncu capture summarised under profiles/
    (profiles/traffic_ratios.json, written when the capture is taken); None if no capture is on record."""
    p = os.path.join(ROOT, "profiles", "traffic_ratios.json")
    try:
        return json.load(open(p)).get(key)
    except (OSError, ValueError):
        return None


class ResidentLayer:
    """One resident MoE layer on the device (all experts in their slots), shared by the token counts timed on it."""

    def __init__(self, sh: inputs.LayerShape, dev):
        self.sh, self.dev = sh, dev
        self.m0, self.blobs, self.slots, self.slot_map, self.wr, self.bias, _ = build_layer(sh, dev)
        self.quantize = dict(QUANTIZE_STATS)

    def context(self, T):
        from paper_2609_38090_b200 import binding
        sh = self.sh
        return binding.Mira(sh.C, sh.R, sh.E, n_shared=sh.n_shared, n_layers=32, max_tokens=T, max_top_k=sh.k,
                            device=self.dev, fmt=FMT)


def measure_resident(layer: ResidentLayer, T: int, args, world, rank, sampler, barrier, e2e=True):
    """Times one token count of a resident layer: the steps with inputs in HBM (blocks of args.steps steps for at
    least half a second), the same steps end to end (H2D of the hidden states, D2H of the output, every step), and a
    per-kernel pass with CUDA events around every launch. Returns the record of this configuration."""
    import torch
    sh, dev = layer.sh.with_tokens(T), layer.dev
    m = layer.context(T)
    wr, bias, slots, slot_map = layer.wr, layer.bias, layer.slots, layer.slot_map
    xs_host = [torch.from_numpy(inputs.hidden(sh, T, step=i)).to(torch.bfloat16) for i in range(N_BATCHES)]
    xs = [x.to(dev) for x in xs_host]
    out = torch.empty((T, sh.C), dtype=torch.bfloat16, device=dev)
    counts = [m.route(x, wr, bias, sh.k)["count"].cpu().tolist() for x in xs]
    bytes_layer = [algorithmic_bytes(sh, c)[0] for c in counts]
    bytes_upgate = [algorithmic_bytes(sh, c)[1] for c in counts]

    def step(i):
        m.moe_layer(xs[i % N_BATCHES], wr, bias, slots, slot_map, sh.k, out=out)

    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()
    launches0 = m.kernel_launches
    lo = sampler.mark() if sampler else 0
    blocks = timed_blocks(step, args.steps, barrier, dev, world)
    hi = sampler.mark() if sampler else 0
    launches = (m.kernel_launches - launches0) // len(blocks)
    code, missing = m.poll_status()
    assert code == 0, f"device status {code}, missing experts {missing}"
    st = block_stats(blocks, args.steps)
    ms_step = st["ms_per_step"]
    rec = {"workload": workload_config(sh)["workload"], "tokens": T, **st,
           "tokens_per_s": replica_throughput(T, 1, world, ms_step), "gpu_launches": int(launches),
           "clocks": clock_record(sampler, lo, hi, ms_step)}

    if e2e:
        # End to end: every step copies its hidden states from pinned host memory and its output back. The copies run
        # on their own streams with two buffers each, so the copy of step i + 1 and the read-back of step i - 1
        # overlap the kernels of step i, as a serving loop would arrange it; every step still moves its own bytes.
        xs_pinned = [x.pin_memory() for x in xs_host]
        s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        s_main = torch.cuda.current_stream(dev)
        x_buf = [torch.empty((T, sh.C), dtype=torch.bfloat16, device=dev) for _ in range(2)]
        o_buf = [torch.empty_like(out) for _ in range(2)]
        o_host = [torch.empty((T, sh.C), dtype=torch.bfloat16).pin_memory() for _ in range(2)]
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_cmp = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]
        for b in range(2):
            ev_cmp[b].record(s_main); ev_out[b].record(s_main)

        def step_e2e(i):
            b = i & 1
            s_in.wait_event(ev_cmp[b])              # the kernels that read this input buffer two steps ago are done
            with torch.cuda.stream(s_in):
                x_buf[b].copy_(xs_pinned[i % N_BATCHES], non_blocking=True)
                ev_in[b].record(s_in)
            s_main.wait_event(ev_in[b])
            s_main.wait_event(ev_out[b])            # this output buffer has been read back
            m.moe_layer(x_buf[b], wr, bias, slots, slot_map, sh.k, out=o_buf[b])
            ev_cmp[b].record(s_main)
            s_out.wait_event(ev_cmp[b])
            with torch.cuda.stream(s_out):
                o_host[b].copy_(o_buf[b], non_blocking=True)
                ev_out[b].record(s_out)

        for i in range(max(args.warmup, 3)):
            step_e2e(i)
        eb = timed_blocks(step_e2e, args.steps, barrier, dev, world, finish=lambda: [s_main.wait_event(e) for e in ev_out])
        est = block_stats(eb, args.steps)
        rec["e2e"] = {"value": world * T / (est["ms_per_step"] / 1e3), "unit": UNIT, "h2d_bytes_per_step": T * sh.C * 2,
                      "d2h_bytes_per_step": T * sh.C * 2, "ms_per_step": est["ms_per_step"], "blocks": est["blocks"]}

    # per-kernel pass: the same steps with an event pair around every launch (the events switch the programmatic
    # launch overlap off, so the kernel times add up to a little more than the step)
    n_prof = max(args.steps, min(400, int(0.1e3 / max(ms_step, 1e-3)))) if MIN_SECONDS > 0 else args.steps
    m.profile(True)
    barrier()
    for i in range(n_prof):
        step(i)
    prof = m.profile_read()
    m.profile(False)
    barrier()

    hbm, tf_sus, tf_burst, src = peaks()
    tc_kernels = T >= (32 if sh.E + sh.n_shared > 16 else 56)        # up/gate on the tcgen05 grouped GEMM kernel
    pairs_avg = sum(sum(c) for c in counts) / len(counts)
    flops_step = 6.0 * sh.R * sh.C * pairs_avg
    bytes_step = sum(bytes_layer) / len(bytes_layer)
    tensor_path = tc_kernels and flops_step / (tf_sus * 1e12) > bytes_step / (hbm * 1e9)
    up_ms, up_n = prof.get("up_gate", (0.0, 0))
    up_bytes = sum(bytes_upgate) / len(bytes_upgate)
    up_us = 1e3 * up_ms / max(up_n, 1)
    total_prof_ms = sum(v[0] for v in prof.values())
    shares = {k: round(v[0] / total_prof_ms, 4) for k, v in prof.items()} if total_prof_ms else None
    avg_us = {k: round(1e3 * v[0] / v[1], 2) for k, v in prof.items() if v[1]}
    if tensor_path:
        up_flops = 4.0 * sh.R * sh.C * pairs_avg                      # up + gate projections of every pair
        ach = up_flops / (up_us / 1e6) / 1e12 if up_us > 0 else None
        rec["roofline"] = {"bound": "tensor", "kernel": "k_ffn_tc<up/gate> (tcgen05 grouped GEMM on in-register dequantized fp16 tiles, SwiGLU epilogue)",
                           "achieved": ach, "peak": tf_sus, "unit": "TFLOP/s", "frac": (ach / tf_sus) if ach else None,
                           "frac_of_burst_peak": (ach / tf_burst) if ach else None,
                           "frac_of_nominal_2250TFLOPs": (ach / NOMINAL_TFLOPS) if ach else None,
                           "peak_source": src + " (cuBLAS bf16, sustained under the power cap; fp16 has the same nominal rate)",
                           "traffic": None, "avg_launch_us": up_us, "algorithmic_flops_per_launch": up_flops,
                           "kernel_share": shares, "kernel_avg_us": avg_us}
    else:
        ach = up_bytes / (up_us / 1e6) / 1e9 if up_us > 0 else None
        key = "k_ffn_up_gate" if not tc_kernels else "k_ffn_tc_up_gate"
        tr = traffic_ratio(key)
        rec["roofline"] = {"bound": "hbm", "kernel": ("k_ffn_tc<up/gate> (tcgen05 grouped GEMM, in-register dequant, SwiGLU epilogue)" if tc_kernels
                                                      else "k_ffn<up/gate> (fused int8 unpack/dequant + up/gate GEMV/GEMM + SwiGLU)"),
                           "achieved": ach, "peak": hbm, "unit": "GB/s", "frac": (ach / hbm) if ach else None,
                           "frac_of_nominal_8TBps": (ach / NOMINAL_HBM_GBS) if ach else None, "peak_source": src,
                           "traffic": (tr["ratio"] * up_bytes) if tr else None,
                           "traffic_source": (tr["source"] if tr else "no ncu capture of this kernel on record"),
                           "avg_launch_us": up_us, "algorithmic_bytes_per_launch": up_bytes,
                           "kernel_share": shares, "kernel_avg_us": avg_us}
    layer_gbs = bytes_step / (ms_step / 1e3) / 1e9
    rec["layer_roofline"] = {"bound": "hbm", "algorithmic_bytes_per_step": bytes_step, "achieved": layer_gbs, "peak": hbm,
                             "unit": "GB/s", "frac": layer_gbs / hbm, "frac_of_nominal_8TBps": layer_gbs / NOMINAL_HBM_GBS,
                             "peak_source": src,
                             "active_experts_per_batch": [int(sum(1 for c in cs if c > 0)) for cs in counts]}
    tfl = flops_step / (ms_step / 1e3) / 1e12
    rec["layer_tensor"] = {"algorithmic_flops_per_step": flops_step, "achieved": tfl, "unit": "TFLOP/s",
                           "peak": tf_sus, "frac": tfl / tf_sus, "frac_of_burst_peak": tfl / tf_burst,
                           "frac_of_nominal_2250TFLOPs": tfl / NOMINAL_TFLOPS, "peak_source": src,
                           "binding": "tensor" if tensor_path else "hbm"}
    rec["_m"] = m
    rec["_xs"] = xs
    return rec


def run_cuda(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    sh = shape_of(args.workload, args.tokens)
    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.wait_started()
    layer = ResidentLayer(sh, dev)
    quantize = dict(layer.quantize)                      # S0 of the headline layer (later layers overwrite the global)
    head = measure_resident(layer, sh.T, args, world, rank, sampler, barrier)
    m, xs = head.pop("_m"), head.pop("_xs")
    wr, bias = layer.wr, layer.bias

    # S7 and S0 carry no target; their times are reported next to the layer's
    pw_np, pb_np = inputs.predictor(sh)
    pred_w = torch.from_numpy(pw_np).to(torch.bfloat16).to(dev)
    pred_b = torch.from_numpy(pb_np).to(dev)
    for _ in range(3):
        m.predict(0, xs[0], pred_w, pred_b, k_pred=min(2, sh.E))
    m.profile(True)
    for i in range(20):
        m.predict(0, xs[i % N_BATCHES], pred_w, pred_b, k_pred=min(2, sh.E))
    torch.cuda.synchronize(dev)
    pprof = m.profile_read()
    m.profile(False)
    predict_us = 1e3 * sum(v[0] for v in pprof.values()) / 20          # device time of its two kernels
    # MixtureHead on the routing by-products of one batch
    mh_np = inputs.mixture_head(sh)
    mh_dev = {n: (torch.from_numpy(v).to(torch.bfloat16).to(dev) if n[0] in "wg" else torch.from_numpy(np.asarray(v, np.float32)).to(dev))
              for n, v in mh_np.items() if n != "b_g"}
    mh_dev["b_g"] = float(mh_np["b_g"])
    rb = m.route(xs[0], wr, bias, sh.k)
    for _ in range(3):
        m.predict_mixture(0, xs[0], rb["logits"], rb["count"], sh.k, mh_dev, min(2, sh.E))
    m.profile(True)
    for _ in range(20):
        m.predict_mixture(0, xs[0], rb["logits"], rb["count"], sh.k, mh_dev, min(2, sh.E))
    torch.cuda.synchronize(dev)
    mprof = m.profile_read()
    m.profile(False)
    mixture_us = 1e3 * sum(v[0] for v in mprof.values()) / 20

    # The other configurations of the workload list, one record each (skipped with --headline-only, with a workload
    # or token count chosen on the command line, and on multi-GPU launches, where every rank is a replica of the
    # headline step).
    others = []
    default_run = args.workload == "mixtral" and args.tokens is None and not FMT
    if default_run and world == 1 and not args.headline_only:
        for T in (1, 8, 2048):
            r = measure_resident(layer, T, args, world, rank, sampler, barrier, e2e=False)
            r.pop("_m"); r.pop("_xs")
            others.append(r)
        del m, xs
        others.append(staged_record(args, layer, sampler, barrier, dev, world, rank))
        del layer
        torch.cuda.empty_cache()
        fine = ResidentLayer(inputs.FINE, dev)
        for T in (4, 64, 1024):
            r = measure_resident(fine, T, args, world, rank, sampler, barrier, e2e=False)
            r.pop("_m"); r.pop("_xs")
            others.append(r)
        del fine
        torch.cuda.empty_cache()
        others.append(stack_record(args, sampler, barrier, dev, world, rank, steps=max(args.steps, 8)))
    if sampler:
        sampler.stop()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    line = {
        "metric": METRIC, "value": head["tokens_per_s"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "ms_per_step_best_block": head["ms_per_step_best"],
        "timed_blocks": head["blocks"], "timed_seconds": head["timed_seconds"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "s8 weights x f16 activations, f32 accumulate",
        "data": "synthetic", "config": workload_config(sh),
        "roofline": head["roofline"], "layer_roofline": head["layer_roofline"], "layer_tensor": head["layer_tensor"],
        "e2e": head["e2e"], "gpu_launches": head["gpu_launches"], "clocks": head["clocks"],
        "timing_note": ("ms_per_step is the median over blocks of exactly --steps steps, each block bracketed by barrier + "
                        "synchronize and timed with CUDA events, repeated until the blocks last 0.5 s; gpu_launches counts one block"),
        "other_steps": {"predictor_us_per_call": predict_us,
                        "predictor_note": "device time of mira_predict on one batch: linear head, mean over tokens, top-2 (S7)",
                        "mixture_head_us_per_call": mixture_us,
                        "mixture_head_note": "device time of mira_predict_mixture (ActHead + HistHead + gate) on the routing by-products",
                        "quantize_ms_per_expert": quantize.get("ms_per_expert"),
                        "quantize_gbs": quantize.get("gbs"),
                        "quantize_note": "mira_quantize_experts (S0): fp32 W2 read twice, W1 and W3 once, blob written"},
    }
    if others:
        line["configs"] = others
    if world == 1 and not args.no_cpu_baseline:
        # whole batches of the workload until about 10 s of CPU time (large batches: a 64-token slice of each)
        n_tok = min(sh.T, 64)
        times, cores, sample = oracle_sample(sh, n_tok, target_seconds=10.0)
        line["cpu_baseline"] = {"value": n_tok * len(times) / sum(times), "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": sample, "seconds": sum(times)}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def staged_record(args, layer, sampler, barrier, dev, world, rank):
    """Prefill with the predictor and a small expert cache (the third workload): per step the predictor scores the
    tokens (S7), the router runs (S1-S3), the host reads the expert counts, the experts in the HOT slots run as the
    first wave while the side stream copies the missing experts from pinned host memory into the STAGE slots (S8),
    and the staged experts run as later waves; the last wave combines. Returns the record of the configuration."""
    import torch
    from paper_2609_38090_b200 import binding

    sh = layer.sh.with_tokens(args.tokens or 2048) if args.mode == "staged" else layer.sh.with_tokens(2048)
    n_hot, n_stage, k_pred = 4, 2, 2
    m = layer.context(sh.T)
    blobs, wr, bias = layer.blobs, layer.wr, layer.bias
    xs = [torch.from_numpy(inputs.hidden(sh, sh.T, step=i)).to(torch.bfloat16).to(dev) for i in range(N_BATCHES)]
    E = sh.E
    counts = [m.route(x, wr, bias, sh.k)["count"].cpu().tolist() for x in xs]
    popularity = np.sum(np.array(counts), axis=0)
    hot = sorted(np.argsort(-popularity, kind="stable")[:n_hot].tolist())
    cold = [e for e in range(E) if e not in hot]
    host_blobs = torch.empty((E, m.expert_bytes), dtype=torch.uint8).pin_memory()
    host_blobs.copy_(blobs)
    cache = torch.empty((n_hot + n_stage, m.expert_bytes), dtype=torch.uint8, device=dev)
    for i, e in enumerate(hot):
        cache[i].copy_(blobs[e])
    slots = binding.slot_table(cache)

    def smap(pairs):
        t = torch.full((E,), -1, dtype=torch.int32)
        for e, sl in pairs:
            t[e] = sl
        return t.to(dev)
    map_hot = smap([(e, i) for i, e in enumerate(hot)])
    stage_maps = {}                      # (expert, stage slot) pairs of one wave -> device slot map
    pw_np, pb_np = inputs.predictor(sh)
    pred_w = torch.from_numpy(pw_np).to(torch.bfloat16).to(dev)
    pred_b = torch.from_numpy(pb_np).to(dev)
    out = torch.empty((sh.T, sh.C), dtype=torch.bfloat16, device=dev)
    side = torch.cuda.Stream(device=dev)
    ready = [torch.cuda.Event() for _ in range(n_stage)]          # STAGE slot filled
    freed = [torch.cuda.Event() for _ in range(n_stage)]          # STAGE slot consumed by its wave
    for ev in freed:
        ev.record()
    main = torch.cuda.current_stream(dev)
    count_host = torch.empty(E, dtype=torch.int32).pin_memory()
    staged_bytes = [0]

    def step(i):
        x = xs[i % N_BATCHES]
        m.predict(0, x, pred_w, pred_b, k_pred=k_pred, token_scores=True)       # S7, scored per token
        r = m.route(x, wr, bias, sh.k)                                            # S1-S3
        count_host.copy_(r["count"], non_blocking=True)
        main.synchronize()                                                        # the cache manager reads the counts
        cnt = count_host.tolist()
        need_hot = [e for e in hot if cnt[e] > 0]
        need_cold = [e for e in cold if cnt[e] > 0]
        waves = [need_cold[j:j + n_stage] for j in range(0, len(need_cold), n_stage)]
        # stage the first wave's experts while the HOT wave computes
        def stage(wave):
            for sl, e in enumerate(wave):
                side.wait_event(freed[sl])
                m.stage_expert(host_blobs[e], cache[n_hot + sl], side, ready[sl])
                staged_bytes[0] += m.expert_bytes
        if waves:
            stage(waves[0])
        m.moe_experts(x, slots, map_hot, expert_ids=need_hot, final_wave=not waves, out=out)
        for wi, wave in enumerate(waves):
            for sl in range(len(wave)):
                main.wait_event(ready[sl])
            key = tuple(wave)
            if key not in stage_maps:
                stage_maps[key] = smap([(e, n_hot + sl) for sl, e in enumerate(wave)])
            m.moe_experts(x, slots, stage_maps[key], expert_ids=wave, final_wave=wi == len(waves) - 1, out=out)
            for sl in range(len(wave)):
                freed[sl].record(main)
            if wi + 1 < len(waves):
                stage(waves[wi + 1])

    # plain pinned host -> device copy rate of this machine, same size as one expert
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    scratch = torch.empty(m.expert_bytes, dtype=torch.uint8, device=dev)
    scratch.copy_(host_blobs[0], non_blocking=True)
    barrier()
    a.record()
    for e in range(4):
        scratch.copy_(host_blobs[e], non_blocking=True)
    b.record()
    barrier()
    h2d_gbs = 4 * m.expert_bytes / (a.elapsed_time(b) / 1e3) / 1e9
    del scratch
    # Scale-only staging (the paper's micro-benchmark, Section IV-B): one shared bf16 scale vector per expert
    # against the three vectors of per-matrix per-row INT8 (W1: R, W3: R, W2: C scales), each its own copy.
    sc_host = [torch.empty(n, dtype=torch.bfloat16).pin_memory() for n in (sh.R, sh.R, sh.C)]
    sc_dev = [torch.empty(n, dtype=torch.bfloat16, device=dev) for n in (sh.R, sh.R, sh.C)]

    def scale_copies(which, reps=400):
        for i in which:
            sc_dev[i].copy_(sc_host[i], non_blocking=True)
        barrier()
        a.record()
        for _ in range(reps):
            for i in which:
                sc_dev[i].copy_(sc_host[i], non_blocking=True)
        b.record()
        barrier()
        return 1e3 * a.elapsed_time(b) / reps                        # us per expert
    scale_shared_us, scale_three_us = scale_copies([0]), scale_copies([0, 1, 2])

    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()
    launches0 = m.kernel_launches
    staged_bytes[0] = 0
    lo = sampler.mark() if sampler else 0
    blocks = timed_blocks(step, args.steps, barrier, dev, world)
    hi = sampler.mark() if sampler else 0
    st = block_stats(blocks, args.steps)
    ms_step = st["ms_per_step"]
    launches = (m.kernel_launches - launches0) // len(blocks)
    bytes_staged = staged_bytes[0] / (args.steps * len(blocks))
    code, missing = m.poll_status()
    assert code == 0, f"device status {code}, missing experts {missing}"
    # compute-only time of the same waves: the part staging has to hide behind
    n_prof = min(args.steps, 5)
    m.profile(True)
    for i in range(n_prof):
        step(i)
    barrier()
    prof = m.profile_read()
    m.profile(False)
    hbm, tf_sus, tf_burst, src = peaks()
    kernel_ms = sum(v[0] for v in prof.values()) / n_prof
    up_ms, up_n = prof.get("up_gate", (0.0, 1))
    pairs = float(np.mean([sum(c) for c in counts]))
    up_flops = 4.0 * sh.R * sh.C * pairs
    ach = up_flops / (up_ms / n_prof / 1e3) / 1e12 if up_ms > 0 else None
    return {
        "workload": (f"{sh.name} layer, prefill {sh.T} tokens with the two-layers-ahead predictor scored per token; "
                     f"cache of {n_hot} HOT + {n_stage} STAGE slots for {E} experts, the other experts are staged "
                     "from pinned host memory every step and run as later waves"),
        "tokens": sh.T, **st, "tokens_per_s": world * sh.T / (ms_step / 1e3), "gpu_launches": int(launches),
        "clocks": clock_record(sampler, lo, hi, ms_step), "hot_experts": hot,
        "roofline": {"bound": "tensor", "kernel": "k_ffn_tc<up/gate>, summed over the waves of a step",
                     "achieved": ach, "peak": tf_sus, "unit": "TFLOP/s", "frac": (ach / tf_sus) if ach else None,
                     "frac_of_burst_peak": (ach / tf_burst) if ach else None,
                     "frac_of_nominal_2250TFLOPs": (ach / NOMINAL_TFLOPS) if ach else None,
                     "peak_source": src + " (cuBLAS bf16, sustained)", "traffic": None,
                     "kernel_ms_per_step": {k: round(v[0] / n_prof, 4) for k, v in prof.items()}},
        "staging": {"bytes_per_step": bytes_staged, "experts_per_step": bytes_staged / m.expert_bytes,
                    "step_gbs": bytes_staged / (ms_step / 1e3) / 1e9, "plain_h2d_gbs": h2d_gbs,
                    "frac_of_plain_h2d": bytes_staged / (ms_step / 1e3) / 1e9 / h2d_gbs,
                    "kernel_ms_per_step": kernel_ms,
                    "note": "the step is bound by the host-to-device copies; step_gbs counts the whole step, kernels included"},
        "scale_only_staging": {"shared_scale_us_per_expert": scale_shared_us, "per_matrix_scales_us_per_expert": scale_three_us,
                               "ratio": scale_three_us / scale_shared_us,
                               "note": "one bf16[R] copy against three copies (bf16[R], bf16[R], bf16[C]) from pinned host memory"},
        "e2e": {"value": world * sh.T / (ms_step / 1e3), "unit": UNIT,
                "h2d_bytes_per_step": int(bytes_staged), "d2h_bytes_per_step": E * 4,
                "note": "hidden states resident; the staged experts and the counts cross PCIe inside the timed region"},
    }


def _single_workload_setup():
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)
    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.wait_started()
    return world, rank, dev, barrier, sampler


def _print_record(rec, args, world, rank, sampler, config):
    import torch.distributed as dist
    if sampler:
        sampler.stop()
    if rank == 0:
        line = {"metric": METRIC, "value": rec["tokens_per_s"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": rec["ms_per_step"], "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "s8 weights x f16 activations, f32 accumulate", "data": "synthetic",
                "config": config}
        line.update({k: v for k, v in rec.items() if k not in ("tokens_per_s", "ms_per_step")})
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_staged(args):
    """`--mode staged`: the third workload alone. One GPU; ranks > 0 of a multi-GPU launch run the same step as
    independent replicas."""
    world, rank, dev, barrier, sampler = _single_workload_setup()
    layer = ResidentLayer(shape_of("mixtral", args.tokens or 2048), dev)
    rec = staged_record(args, layer, sampler, barrier, dev, world, rank)
    cfg = workload_config(layer.sh)
    cfg["workload"] = rec["workload"]
    _print_record(rec, args, world, rank, sampler, cfg)


def stack_record(args, sampler, barrier, dev, world, rank, steps):
    """The fifth workload: a 24-layer stack of the fine-grained layer decoded with beam search of width 4; per layer
    a cache of 12 HOT + 3 STAGE slots for the 60 routed experts (25 %) plus the 4 shared experts, predictor-driven
    and on-demand staging from pinned host memory on a side stream. One step = one decode step (24 layer steps of
    4 tokens each plus the harness glue: norm, output head, beam step). Also timed with every expert resident."""
    import torch
    from paper_2609_38090_b200.stack import MoEStack, StackConfig

    sh = inputs.FINE_STACK
    n_hot, n_stage, budget = 12, 3, None
    if args.expert_budget_gb:                # byte budget -> slots, as the cache section of the paper describes
        from paper_2609_38090_b200.cache import plan_budget
        budget = plan_budget(int(args.expert_budget_gb * 1e9), 0, sh.expert_bytes, 24, sh.E, sh.n_shared)
        n_hot, n_stage = budget.n_hot, budget.n_stage
    cfg = StackConfig(shape=sh, n_layers=24, vocab=1024, n_hot=n_hot, n_stage=n_stage, k_pred=args.k_pred, seed=1,
                      hot_init=args.hot_init, rebalance_every=args.rebalance_every, max_swaps=2,
                      native_step=not args.python_steps)
    st = MoEStack(cfg, device=dev)

    def stepper(stack, n_warm):
        """One decode step per call, continuing one beam search (the expert traffic of a search that restarts
        every step would be the same few experts over and over)."""
        hist, sc = stack.decode(n_warm)
        state = [hist[-1], sc]

        def fn(i):
            h, s_ = stack.decode(1, state[0], state[1])
            state[0], state[1] = h[-1], s_
        return fn
    step_fn = stepper(st, max(args.warmup, 3))
    barrier()
    st.reset_stats()
    launches0 = st.m.kernel_launches
    lo = sampler.mark() if sampler else 0
    blocks = timed_blocks(step_fn, steps, barrier, dev, world)
    hi = sampler.mark() if sampler else 0
    bs = block_stats(blocks, steps)
    n_steps = steps * len(blocks)
    ms_total = sum(blocks)
    launches = (st.m.kernel_launches - launches0) // len(blocks)
    code, missing = st.m.poll_status()
    assert code == 0, f"device status {code}, missing experts {missing}"
    hbm, tf_sus, tf_burst, src = peaks()
    stats = st.stats()
    cov = st.coverage()
    W, L = sh.T, cfg.n_layers
    ms_step = bs["ms_per_step"]
    layer_steps = n_steps * L
    be = st.m.expert_bytes
    # distinct experts a layer step touches (for the algorithmic bytes): the routed ones from the cache statistics
    # plus the shared ones, which every step uses
    experts_per_layer_step = (stats.experts_hot + stats.experts_stage + stats.experts_demand) / layer_steps + sh.n_shared
    alg_bytes = experts_per_layer_step * be
    layer_ms = ms_step / L
    bytes_staged, copies = st.bytes_staged, stats.copies
    rec = {
        "workload": (f"{L}-layer stack of the fine-grained layer (hidden {sh.C}, ffn {sh.R}, {sh.E} experts top-{sh.k} + "
                     f"{sh.n_shared} shared), beam width {W}, {steps} decode steps per block; per layer {cfg.n_hot} HOT + "
                     f"{cfg.n_stage} STAGE slots of {sh.E} routed experts, predictor-driven and on-demand staging from pinned host memory"),
        "tokens": W, "layers": L, **bs, "tokens_per_s": world * W * L / (ms_step / 1e3),
        "beam_tokens_per_s": world * W / (ms_step / 1e3), "gpu_launches": int(launches),
        "clocks": clock_record(sampler, lo, hi, ms_step),
        "roofline": {"bound": "hbm", "kernel": "whole layer step (route, predictor, waves of up/gate + down, combine, host read-back)",
                     "achieved": alg_bytes / (layer_ms / 1e3) / 1e9, "peak": hbm, "unit": "GB/s",
                     "frac": alg_bytes / (layer_ms / 1e3) / 1e9 / hbm,
                     "frac_of_nominal_8TBps": alg_bytes / (layer_ms / 1e3) / 1e9 / NOMINAL_HBM_GBS, "peak_source": src, "traffic": None,
                     "algorithmic_bytes_per_layer_step": alg_bytes, "us_per_layer_step": 1e3 * layer_ms,
                     "note": "latency bound: 4 tokens per layer step; the host-side cache manager reads the routing counts of every layer (a flag in host-mapped memory with the library runtime, a stream synchronisation with --python-steps)",
                     "layer_step": "mira_stack_layer_step (library runtime)" if st.native is not None else "issued from Python call by call"},
        "cache": {"shares_of_routed_pairs": stats.shares(), "experts_per_layer_step": experts_per_layer_step,
                  "copies_per_decode_step": copies / n_steps, "h2d_bytes_per_decode_step": bytes_staged / n_steps,
                  "budget": None if budget is None else {"expert_bytes_gb": args.expert_budget_gb, "mode": budget.mode,
                                                          "n_hot": budget.n_hot, "n_stage": budget.n_stage,
                                                          "share_of_routed_experts_in_slots": budget.slots_per_layer / sh.E},
                  "coverage_at_k_mean_over_source_layers": [sum(r[k] for r in cov) / max(len(cov), 1) for k in range(cfg.k_pred)],
                  "hot_init": args.hot_init, "rebalance_every_tokens": args.rebalance_every,
                  "hot_swaps": st.hot_swaps(),
                  "prefetch": {"issued": stats.prefetch_issued, "useful": stats.prefetch_useful,
                               "declined": stats.prefetch_declined, "skipped": stats.prefetch_skipped}},
        "e2e": {"value": world * W * L / (ms_step / 1e3), "unit": UNIT,
                "h2d_bytes_per_step": int(bytes_staged / n_steps), "d2h_bytes_per_step": L * (sh.E + sh.n_shared + cfg.k_pred) * 4,
                "note": "the staged experts and the per-layer counts / predicted ids cross PCIe inside the timed region"},
    }
    del st
    torch.cuda.empty_cache()
    if not args.expert_budget_gb:
        # the same stack with every expert resident: what the layer kernels and the runtime cost without copies
        full = MoEStack(StackConfig(shape=sh, n_layers=24, vocab=1024, n_hot=sh.E, n_stage=1, k_pred=0, seed=1,
                                    native_step=not args.python_steps), device=dev)
        fb = block_stats(timed_blocks(stepper(full, max(args.warmup, 3)), steps, barrier, dev, world), steps)
        rec["all_resident"] = {"ms_per_step": fb["ms_per_step"], "ms_per_step_best": fb["ms_per_step_best"],
                               "us_per_layer_step": 1e3 * fb["ms_per_step"] / L,
                               "tokens_per_s": world * W * L / (fb["ms_per_step"] / 1e3)}
        del full
        torch.cuda.empty_cache()
    return rec


def run_stack(args):
    world, rank, dev, barrier, sampler = _single_workload_setup()
    rec = stack_record(args, sampler, barrier, dev, world, rank, steps=args.steps)
    cfgj = workload_config(inputs.FINE_STACK)
    cfgj["workload"] = rec["workload"]
    cfgj["layers"] = 24
    _print_record(rec, args, world, rank, sampler, cfgj)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="mira", choices=["mira", "reference"])
    ap.add_argument("--workload", default="mixtral", choices=["mixtral", "mixtral22", "fine", "tiny", "stack"])
    ap.add_argument("--tokens", type=int, default=None)
    ap.add_argument("--ref-tokens", type=int, default=4, help="tokens of the bounded oracle sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--min-seconds", type=float, default=0.5,
                    help="repeat the block of --steps steps until the timed region lasts this long (0: one block)")
    ap.add_argument("--headline-only", action="store_true",
                    help="time the headline configuration only (the default run adds one record per other configuration)")
    ap.add_argument("--k-pred", type=int, default=4, help="stack workload: expert ids requested from each predictor head")
    ap.add_argument("--expert-budget-gb", type=float, default=0.0,
                    help="stack workload: device bytes for expert slots of all layers (default: 12 HOT + 3 STAGE per layer)")
    ap.add_argument("--python-steps", action="store_true",
                    help="stack workload: issue each layer step's calls from Python instead of mira_stack_layer_step")
    ap.add_argument("--hot-init", default="bias", choices=["bias", "random"],
                    help="stack workload: HOT sets start with the experts the router bias favours, or a random set")
    ap.add_argument("--rebalance-every", type=int, default=0,
                    help="stack workload: tokens per layer between HOT rebalancing passes (0: fixed HOT sets)")
    ap.add_argument("--format", default="shared", choices=["shared", "per-matrix"],
                    help="compressed-expert format: the paper's shared scale, or one scale per row of each matrix")
    ap.add_argument("--mode", default="resident", choices=["resident", "staged"],
                    help="staged: prefill with the predictor and a 4+2-slot expert cache fed from pinned host memory")
    args = ap.parse_args()
    global FMT, MIN_SECONDS
    FMT = 1 if args.format == "per-matrix" else 0
    MIN_SECONDS = max(0.0, args.min_seconds)
    if FMT and (args.workload == "stack" or args.mode == "staged"):
        ap.error("--format per-matrix is available for the resident layer workloads")
    if args.warmup < 3 and args.impl == "mira":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "stack":
        run_stack(args)
    elif args.mode == "staged":
        run_staged(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
