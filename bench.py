#!/usr/bin/env python
"""Benchmark of the RefreshKV decode-attention hot path.

One "step" is one decode token through the attention work of ALL layers of the workload
(default: Llama-3.1-8B attention shape, 32 layers, batch 1, L=32768, K=2048, fixed stride 10):
per layer  (every 10th token) rkv_append + rkv_full_step + rkv_gather_small, else rkv_append_small_step.
Each token's launches are replayed from a CUDA graph (one graph per kind of token).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  `value` is the amortised decode-attention time per token in microseconds
(all layers), inputs resident in HBM; `e2e` is the same with each token's q/k/v rows coming from
pinned host memory and its attention outputs copied back to the host inside the timed region.
N > 1 runs independent replicas (the path has no exchange step), one rank per GPU.
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
sys.path.insert(0, ROOT)

METRIC = "decode attention us/token (all layers, stride-10 refresh; full step and small step also reported)"
UNIT = "us/token"
STRIDE = 10


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--ctx", type=int, default=32768)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--small-min-chunk", type=int, default=0, help="override rkv_small_step chunking (0: library default)")
    ap.add_argument("--no-dependent-launch", action="store_true", help="plain stream order between kernels")
    return ap.parse_args()


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s)"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------------------------- reference arm
def oracle_period_sample(w, layer_cache_bits, qs_bits, kn_bits, vn_bits):
    """One stride period of ONE layer on the CPU oracle: 1 full step (+ rebuild) and stride-1 partial steps.

    Returns seconds taken.  Inputs are the same bf16 bytes the GPU path consumes.
    """
    from oracle import rkv_oracle as O
    kf, vf = layer_cache_bits
    st = O.SequenceState(kf, vf, w.lens[0], w.k_small[0])
    t0 = time.perf_counter()
    st.full(qs_bits[0])
    for t in range(1, STRIDE):
        st.append(kn_bits[t], vn_bits[t])
        st.small(qs_bits[t])
    return time.perf_counter() - t0


def cpu_inputs(w):
    """Host copies (uint16 bf16 bits) of one layer of the workload for the oracle."""
    import numpy as np
    import torch
    from paper_2411_05787_b200 import synth
    cache = synth.fill_layer(w, 0, torch.device("cpu"), extra_cap=STRIDE + 1)
    qs = synth.query_trajectory(synth.scaled(w, steps=STRIDE), 0)
    synth.plant_heavy(w, cache, 0, qs[0])
    kn, vn = synth.new_token_kv(synth.scaled(w, steps=STRIDE), 0)
    cap = int(cache.cap[0])
    kf = synth.to_bits(cache.k).reshape(w.n_kv_heads, cap, 128)
    vf = synth.to_bits(cache.v).reshape(w.n_kv_heads, cap, 128)
    qb = [synth.to_bits(qs[t, 0]) for t in range(STRIDE)]
    knb = [synth.to_bits(kn[t, 0]) for t in range(STRIDE)]
    vnb = [synth.to_bits(vn[t, 0]) for t in range(STRIDE)]
    return (kf, vf), qb, knb, vnb


def cpu_threads() -> int:
    try:
        import torch
        return max(1, torch.get_num_threads())
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    """The oracle, as it stands, on the host cores: each step = one stride period of one layer, scaled to
    all layers and divided by the stride to give microseconds per token."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2411_05787_b200 import synth
    w = synth.config2(n_layers=args.layers, ctx=args.ctx)
    caches, qb, knb, vnb = cpu_inputs(w)
    steps = max(1, min(args.steps, 40))          # bounded: a period costs about a second of CPU time
    warm = max(1, min(args.warmup, 2))
    for _ in range(warm):
        oracle_period_sample(w, (caches[0].copy(), caches[1].copy()), qb, knb, vnb)
    t = [oracle_period_sample(w, (caches[0].copy(), caches[1].copy()), qb, knb, vnb) for _ in range(steps)]
    per_token_us = statistics.mean(t) * w.n_layers / STRIDE * 1e6
    cores = cpu_threads()
    sample = (f"{steps} samples of one stride period (1 full step + rebuild + {STRIDE - 1} partial steps) of 1 of "
              f"{w.n_layers} layers, scaled x{w.n_layers} layers / {STRIDE} tokens")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": per_token_us, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": per_token_us / 1000.0, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, args),
        "cpu_baseline": {"value": per_token_us, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": per_token_us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def workload_config(w, args):
    return {"workload": w.name, "layers": w.n_layers, "batch": w.batch, "q_heads": w.n_q_heads,
            "kv_heads": w.n_kv_heads, "head_dim": 128, "context": w.lens[0], "k_small": w.k_small[0],
            "stride": STRIDE, "schedule": "fixed", "l2_hygiene": "inputs larger than L2: every token walks all "
            "layers' distinct caches (full 4.3 GB, small 0.27 GB)", "launch": "one CUDA graph replay per token"}


# ----------------------------------------------------------------------------------------------- our arm
def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2411_05787_b200 import build
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank == 0:
        build.build()
    if world > 1:
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    else:
        torch.cuda.set_device(0)
    from paper_2411_05787_b200 import rkv, runner, synth

    dev = torch.device("cuda", torch.cuda.current_device())
    n_tokens = args.steps + args.warmup
    w = synth.config2(n_layers=args.layers, ctx=args.ctx)
    # capacity for: warm-up + timed tokens of the main loop, the e2e loop, the always-full loop, profiling
    total_tokens = 2 * n_tokens + 2 * 30 + 2 * STRIDE + 8
    wl = synth.scaled(w, steps=total_tokens)
    L, K, Hq, Hkv = w.lens[0], w.k_small[0], w.n_q_heads, w.n_kv_heads
    max_len = L + total_tokens + 1
    ctx = rkv.Context(1, Hq, Hkv, max_len, K + STRIDE + 2)
    if args.small_min_chunk:
        ctx.set_option(rkv.OPT_SMALL_MIN_CHUNK, args.small_min_chunk)
    if args.no_dependent_launch:
        ctx.set_option(rkv.OPT_DEPENDENT_LAUNCH, 0)

    layers = []
    q0 = synth.query_trajectory(synth.scaled(w, steps=1), 0).to(dev)
    for l in range(w.n_layers):
        cache = synth.fill_layer(wl, l, dev)
        synth.plant_heavy(w, cache, l, q0[0])
        layers.append(runner.LayerState(ctx, cache, [K], STRIDE + 2, Hq, Hkv))

    # per-token inputs for all layers: [q | k_new | v_new] rows, one contiguous block per token
    row = (Hq + 2 * Hkv) * 128
    n_in = 64                                     # distinct input blocks, cycled
    g = torch.Generator(device="cpu"); g.manual_seed(1234)
    inputs_host = torch.randn((n_in, w.n_layers, row), generator=g, dtype=torch.float32).to(torch.bfloat16).pin_memory()
    inputs_dev = inputs_host.to(dev)
    stage = torch.zeros((w.n_layers, row), dtype=torch.bfloat16, device=dev)
    outs = torch.zeros((w.n_layers, Hq * 128), dtype=torch.bfloat16, device=dev)
    outs_host = torch.zeros((w.n_layers, Hq * 128), dtype=torch.bfloat16).pin_memory()
    views = []
    for l in range(w.n_layers):
        q = stage[l, : Hq * 128].view(1, Hq, 128)
        kn = stage[l, Hq * 128: (Hq + Hkv) * 128].view(1, Hkv, 128)
        vn = stage[l, (Hq + Hkv) * 128:].view(1, Hkv, 128)
        layers[l].out = outs[l].view(1, Hq, 128)
        views.append((q, kn, vn))

    def token(full: bool):
        for l, st in enumerate(layers):
            q, kn, vn = views[l]
            if full:
                st.append(kn, vn)
                st.refresh(q, max_len_hint=max_len)
            else:      # append + partial step in one call (one launch)
                st.append_partial(q, kn, vn, max_len_hint=K + STRIDE + 1)

    # initial small caches + eager warm-up of every kernel (also creates the tensor maps)
    stage.copy_(inputs_dev[0])
    for st, (q, _, _) in zip(layers, views):
        st.refresh(q, max_len_hint=max_len)
    token(False); token(True)
    torch.cuda.synchronize()

    # capture one graph per kind of token
    side = torch.cuda.Stream()
    graphs, launches_per = {}, {}
    for kind in (False, True):
        gr = torch.cuda.CUDAGraph()
        before = ctx.launch_count
        with torch.cuda.stream(side):
            with torch.cuda.graph(gr, stream=side):
                token(kind)
        launches_per[kind] = ctx.launch_count - before
        graphs[kind] = gr
    torch.cuda.synchronize()

    tok_counter = [1]

    def run_tokens(n, e2e=False, always_full=False, force_small=False):
        """Enqueue n decode tokens; returns (#full tokens, #small tokens)."""
        nf = ns = 0
        for _ in range(n):
            t = tok_counter[0]; tok_counter[0] += 1
            src = inputs_host if e2e else inputs_dev
            stage.copy_(src[t % n_in], non_blocking=True)
            full = (always_full or (t % STRIDE == 0)) and not force_small
            graphs[full].replay()
            if e2e:
                outs_host.copy_(outs, non_blocking=True)
            nf += int(full); ns += int(not full)
        return nf, ns

    def timed(n, **kw):
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        nf, ns = run_tokens(n, **kw)
        e1.record()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        ms = e0.elapsed_time(e1)
        if world > 1:
            tt = torch.tensor([ms], device=dev)
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
            ms = float(tt.item())
        return ms, nf, ns

    # ---- main measurement: inputs resident in HBM.  The token counter runs on through all phases, so a
    # refresh comes at least every STRIDE tokens and the small caches never outgrow their capacity.
    run_tokens(args.warmup)
    sampler = ClockSampler(torch.cuda.current_device() if "CUDA_VISIBLE_DEVICES" not in os.environ else 0)
    if rank == 0:
        sampler.start()
    ms, nf, ns = timed(args.steps)
    clocks = sampler.stop() if rank == 0 else {}
    us_per_token = ms * 1000.0 / (args.steps * world)
    launches = nf * launches_per[True] + ns * launches_per[False]

    # ---- end to end: inputs from pinned host memory, outputs back to the host, every token
    run_tokens(min(args.warmup, 10), e2e=True)
    ms_e2e, _, _ = timed(args.steps, e2e=True)
    e2e_us = ms_e2e * 1000.0 / (args.steps * world)

    # ---- always-full attention (the vanilla comparator) on the same caches
    run_tokens(3, always_full=True)
    ms_full, nff, _ = timed(20, always_full=True)
    full_token_us = ms_full * 1000.0 / (20 * world)
    ms_small, _, nss = timed(STRIDE - 1, force_small=True)   # right after a full token: K .. K+8 rows
    run_tokens(1, always_full=True)
    # ---- per-kernel device time: every launch bracketed by CUDA events on its stream (same schedule, two
    # periods).  A spin kernel first keeps the GPU busy while the host enqueues, so that the launches sit
    # back to back in the queue and an event pair measures the kernel, not the host's launch latency.
    torch.cuda.synchronize()
    ctx.set_profiling(True)
    ctx.get_profile()
    torch.cuda._sleep(int(8e7))
    for _ in range(2 * STRIDE):
        t = tok_counter[0]; tok_counter[0] += 1
        stage.copy_(inputs_dev[t % n_in])
        token(t % STRIDE == 0)
    torch.cuda.synchronize()
    prof = ctx.get_profile()
    ctx.set_profiling(False)
    status = ctx.device_status()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_src = load_peaks()
    len_avg = L + total_tokens / 2.0
    kv_bytes_full = len_avg * Hkv * 512.0                       # K+V bytes one full-step launch must read
    kv_bytes_small = (K + STRIDE / 2.0) * Hkv * 512.0
    kern = {}
    for name, (us, cnt) in prof.items():
        if cnt:
            kern[name] = {"launches": cnt, "avg_us": us / cnt}
    attn_us = kern["attn_full"]["avg_us"]
    achieved = kv_bytes_full / (attn_us * 1e-6) / 1e9
    small_us = kern["attn_small"]["avg_us"]
    kern["attn_full"]["gbs"] = achieved
    kern["attn_small"]["gbs"] = kv_bytes_small / (small_us * 1e-6) / 1e9
    kern["gather"]["gbs"] = 2 * K * Hkv * 512.0 / (kern["gather"]["avg_us"] * 1e-6) / 1e9
    full_step_us = attn_us + kern["select"]["avg_us"]

    result = {
        "metric": METRIC, "value": us_per_token, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 in / fp32 accumulate", "data": "synthetic",
        "config": workload_config(w, args),
        "clocks": clocks,
        "e2e": {"value": e2e_us, "unit": UNIT, "h2d_bytes_per_step": w.n_layers * row * 2,
                "d2h_bytes_per_step": w.n_layers * Hq * 128 * 2},
        "gpu_launches": launches,
        "roofline": {"bound": "hbm", "kernel": "attn_kernel<logits> (full-cache attention + score logits)",
                     "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_source": peak_src, "traffic": None,
                     "algorithmic_bytes_per_launch": kv_bytes_full},
        "detail": {
            "always_full_us_per_token": full_token_us,
            "refresh_speedup_vs_always_full": full_token_us / us_per_token,
            "small_only_us_per_token": ms_small * 1000.0 / ((STRIDE - 1) * world),
            "per_layer_kernel_us": kern,
            "full_step_attn_plus_select_us": full_step_us,
            "full_step_frac_of_8TBs": kv_bytes_full / (full_step_us * 1e-6) / 8e12,
            "small_step_frac_of_8TBs": kv_bytes_small / (small_us * 1e-6) / 8e12,
            "attn_full_frac_of_8TBs": achieved / 8000.0,
            "device_status": status,
            "graph_launches": {"full_token": launches_per[True], "small_token": launches_per[False]},
        },
    }
    if not args.no_cpu_baseline and world == 1:
        caches, qb, knb, vnb = cpu_inputs(w)
        oracle_period_sample(w, (caches[0].copy(), caches[1].copy()), qb, knb, vnb)
        n_s = 8
        t = [oracle_period_sample(w, (caches[0].copy(), caches[1].copy()), qb, knb, vnb) for _ in range(n_s)]
        per_token_us = statistics.mean(t) * w.n_layers / STRIDE * 1e6
        result["cpu_baseline"] = {
            "value": per_token_us, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
            "sample": f"{n_s} samples of one stride period (1 full + {STRIDE - 1} partial steps) of 1 of "
                      f"{w.n_layers} layers, scaled x{w.n_layers} / {STRIDE} tokens"}
    print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
