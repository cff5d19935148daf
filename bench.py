#!/usr/bin/env python
"""Benchmark of the RefreshKV decode-attention hot path.

One "step" is one decode token through the attention work of ALL layers of the workload.  Default
workload: Llama-3.1-8B attention shape, 32 layers, batch 1, L=32768, K=2048, fixed stride 10:
per layer  rkv_append_small_step  on nine tokens out of ten, and on the tenth the full step
(rkv_append_full_attention, rkv_select_topk, rkv_gather_small).  Dynamic workloads run, every QC-th
token, rkv_should_refresh and then both branches under the per-sequence masks it wrote.  Each token's
launches are replayed from a CUDA graph (one graph per kind of token).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--workload cfg1..cfg5 | lm16k_S10 | lm16k_S15 | novel128k_S10 | ...]
                  [--k-small K] [--stride S] [--qc QC] [--threshold s] [--schedule fixed|dynamic]

Prints ONE JSON line.  `value` is the amortised decode-attention time per token in microseconds
(all layers), inputs resident in HBM: the median over repeated timed regions of K steps each; `e2e`
is the same with each token's q/k/v rows coming from pinned host memory and its attention outputs
copied back to the host inside the timed region.  N > 1 runs independent replicas (the path has no
exchange step), one rank per GPU.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import re
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "decode attention us/token (all layers, refresh schedule of the workload; full step and small step also reported)"
UNIT = "us/token"
# ncu summary that holds the DRAM counters of the full-cache attention launch, and the source it was taken from
TRAFFIC_PROFILE = os.path.join(ROOT, "profiles", "attn_kernel_full_step_cfg2_L32768.md")
ATTN_SOURCE = os.path.join(ROOT, "paper_2411_05787_b200", "csrc", "rkv_attn.cu")


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2",
                    help="cfg1..cfg5 (the five stated configurations) or one of the paper's operating points: "
                         "lm16k_S10, lm16k_S15, lm16k_dyn085_qc5, lm16k_dyn085_qc10, novel128k_S10, "
                         "novel128k_dyn085_qc10, qwen16k_dyn095_qc5, qwen16k_dyn095_qc10")
    ap.add_argument("--layers", type=int, default=0, help="override the workload's layer count (0: its own)")
    ap.add_argument("--ctx", type=int, default=0, help="override the context length of cfg2 / cfg3 (0: its own)")
    ap.add_argument("--k-small", type=int, default=0, help="override the small-cache size K (0: the workload's)")
    ap.add_argument("--stride", type=int, default=0, help="override the fixed refresh stride S (0: the workload's)")
    ap.add_argument("--qc", type=int, default=0, help="override the stride of the similarity check (0: the workload's)")
    ap.add_argument("--threshold", type=float, default=-1.0, help="override the similarity threshold s (< 0: the workload's)")
    ap.add_argument("--schedule", default="", choices=["", "fixed", "dynamic"], help="override the refresh schedule")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra-workloads", action="store_true", help="skip the compact rows of the other configurations")
    ap.add_argument("--small-min-chunk", type=int, default=0, help="override rkv_small_step chunking (0: library default)")
    ap.add_argument("--no-dependent-launch", action="store_true", help="plain stream order between kernels")
    ap.add_argument("--no-small-cluster", action="store_true", help="merge partial-step splits through the workspace")
    ap.add_argument("--full-schedule", default="deferred", choices=["deferred", "overlap", "one_stream"],
                    help="full-step tokens: 'deferred' = every layer's selection and rebuild after the last attention "
                         "pass; 'overlap' = behind the layer's attention in a second stream, beside the next layers'; "
                         "'one_stream' = attention, selection and rebuild of a layer in stream order")
    ap.add_argument("--no-overlap", action="store_true", help="same as --full-schedule one_stream")
    ap.add_argument("--no-interleave", action="store_true", help="full-cache pass: one contiguous chunk per CTA")
    ap.add_argument("--select-keys-per-cta", type=int, default=0, help="override RKV_OPT_SELECT_KEYS_PER_CTA (0: default)")
    ap.add_argument("--score-slice", type=int, default=0, help="override RKV_OPT_SCORE_SLICE (0: default)")
    ap.add_argument("--deferred-keys-per-cta", type=int, default=16384,
                    help="deferred schedule with 8+ layers: RKV_OPT_SELECT_KEYS_PER_CTA of the tail's selections (0: the contexts')")
    ap.add_argument("--deferred-score-slice", type=int, default=4096,
                    help="deferred schedule with 8+ layers: RKV_OPT_SCORE_SLICE of the tail's score passes (0: the contexts')")
    ap.add_argument("--early-scores", action="store_true",
                    help="deferred schedule: every layer's score pass right behind its attention pass, in a stream of its own")
    ap.add_argument("--side-streams", type=int, default=16,
                    help="deferred schedule: streams the layers' selections and rebuilds are spread over")
    ap.add_argument("--regions", type=int, default=0,
                    help="timed regions of K steps to take (0: as many as region_repeats() says; 1 keeps a profiler run short)")
    return ap.parse_args()


def make_workload(args):
    from paper_2411_05787_b200 import synth
    name = args.workload
    if name == "cfg1":
        w = synth.config1()
    elif name in ("cfg2", "cfg5"):
        w = synth.config2(ctx=args.ctx or 32768)
    elif name == "cfg3":
        w = synth.config3(ctx=args.ctx or 65536)
    elif name == "cfg4":
        w = synth.config4(n_layers=8)      # 8 of the 32 layers (23 GB of caches) unless --layers says otherwise
    elif name in synth.PAPER_POINTS:
        w = synth.paper_point(name)
    else:
        raise SystemExit(f"unknown workload {name}")
    kw = {}
    if args.layers:
        kw["n_layers"] = args.layers
    if args.k_small:
        kw["k_small"] = [min(args.k_small, l) for l in w.lens]
    if args.schedule:
        kw["schedule"] = args.schedule
        if args.schedule == "dynamic" and w.threshold == 0.0:
            kw["threshold"] = 0.9
    if args.stride:
        kw["stride"] = args.stride
    if args.qc:
        kw["stride"] = args.qc
    if args.threshold >= 0.0:
        kw["threshold"] = args.threshold
    if kw:
        w = synth.scaled(w, **kw)
        if set(kw) - {"n_layers"}:
            w = synth.scaled(w, name=f"{w.name}|K{max(w.k_small)}_{w.schedule}{w.stride}" +
                             (f"_s{w.threshold}" if w.schedule == "dynamic" else ""))
    return w


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s)"


def attn_traffic_per_kv_byte():
    """DRAM bytes per algorithmic K/V byte of one full-cache attention launch, from the tracked ncu summary - but
    only while the kernel's source is still the one the counters were taken from (the summary records its hash)."""
    try:
        text = open(TRAFFIC_PROFILE).read()
        src = hashlib.sha256(open(ATTN_SOURCE, "rb").read()).hexdigest()
    except OSError:
        return None, "no tracked ncu summary"
    m = re.search(r"source sha256 \(rkv_attn\.cu\): ([0-9a-f]{64})", text)
    if not m:
        return None, "the tracked ncu summary names no source hash"
    if m.group(1) != src:
        return None, "rkv_attn.cu has changed since the counters were taken"
    rd = re.search(r"dram__bytes_read\.sum \| ([0-9.]+) Mbyte", text)
    wr = re.search(r"dram__bytes_write\.sum \| ([0-9.]+) Mbyte", text)
    kv = re.search(r"algorithmic K/V bytes of the captured launch: ([0-9.]+) MB", text)
    if not (rd and wr and kv):
        return None, "the tracked ncu summary lacks the DRAM counters"
    return (float(rd.group(1)) + float(wr.group(1))) / float(kv.group(1)), os.path.relpath(TRAFFIC_PROFILE, ROOT)


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
def oracle_period_sample(w, layer_cache_bits, qs_bits, kn_bits, vn_bits, stride):
    """One stride period of ONE layer and ONE sequence on the CPU oracle: 1 full step (+ rebuild) and
    stride-1 partial steps.  Returns seconds taken.  Inputs are the same kind of bf16 bytes the GPU path consumes."""
    from oracle import rkv_oracle as O
    kf, vf = layer_cache_bits
    st = O.SequenceState(kf, vf, w.lens[0], w.k_small[0])
    t0 = time.perf_counter()
    st.full(qs_bits[0])
    for t in range(1, stride):
        st.append(kn_bits[t], vn_bits[t])
        st.small(qs_bits[t])
    return time.perf_counter() - t0


def cpu_inputs(w, stride):
    """Host copies (uint16 bf16 bits) of sequence 0 of one layer of the workload for the oracle."""
    import torch
    from paper_2411_05787_b200 import synth
    w1 = synth.scaled(w, lens=[w.lens[0]], k_small=[w.k_small[0]], rho=[w.rho[0]] if w.rho else [], steps=stride)
    cache = synth.fill_layer(w1, 0, torch.device("cpu"), extra_cap=stride + 1)
    qs = synth.query_trajectory(w1, 0)
    synth.plant_heavy(w1, cache, 0, qs[0])
    kn, vn = synth.new_token_kv(w1, 0)
    cap = int(cache.cap[0])
    kf = synth.to_bits(cache.k).reshape(w.n_kv_heads, cap, 128)
    vf = synth.to_bits(cache.v).reshape(w.n_kv_heads, cap, 128)
    qb = [synth.to_bits(qs[t, 0]) for t in range(stride)]
    knb = [synth.to_bits(kn[t, 0]) for t in range(stride)]
    vnb = [synth.to_bits(vn[t, 0]) for t in range(stride)]
    return (kf, vf), qb, knb, vnb


def blas_threads() -> int:
    """Threads numpy's BLAS may use (the oracle's only source of parallelism: it is one Python process)."""
    try:
        from threadpoolctl import threadpool_info
        return max([int(p.get("num_threads", 1)) for p in threadpool_info()] or [1])
    except Exception:
        return 1


def cpu_baseline(w, n_samples, warm, budget_s=None):
    """The oracle, as it stands, on the host cores: microseconds per token for all layers and sequences,
    from samples of one stride period of one layer of sequence 0, scaled by the positions the other
    sequences and layers hold.  With budget_s, samples are taken until that much oracle time has been spent
    (at least n_samples, at most 64).  Returns (us per token, description of the sample, cores actually used:
    process CPU time / wall time over the samples, rounded up)."""
    stride = w.stride
    caches, qb, knb, vnb = cpu_inputs(w, stride)
    for _ in range(warm):
        oracle_period_sample(w, (caches[0].copy(), caches[1].copy()), qb, knb, vnb, stride)
    t = []
    cpu0, wall0 = time.process_time(), time.perf_counter()
    while len(t) < n_samples or (budget_s is not None and sum(t) < budget_s and len(t) < 64):
        t.append(oracle_period_sample(w, (caches[0].copy(), caches[1].copy()), qb, knb, vnb, stride))
    cpu_s, wall_s = time.process_time() - cpu0, time.perf_counter() - wall0
    n_samples = len(t)
    seq_scale = sum(w.lens) / float(w.lens[0])
    per_token_us = statistics.mean(t) * w.n_layers * seq_scale / stride * 1e6
    sample = (f"{n_samples} samples of one stride period (1 full step + rebuild + {stride - 1} partial steps) of sequence 0 "
              f"in 1 of {w.n_layers} layers, scaled x{w.n_layers} layers x{seq_scale:.2f} (positions of all sequences) "
              f"/ {stride} tokens")
    used = max(1, int(math.ceil(cpu_s / max(wall_s, 1e-9) - 0.05)))
    return per_token_us, sample, {"cores": used, "cpu_seconds_per_wall_second": round(cpu_s / max(wall_s, 1e-9), 2),
                                  "blas_threads_available": blas_threads(), "host_logical_cpus": os.cpu_count()}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = make_workload(args)
    steps = max(1, min(args.steps, 40))          # bounded: a period costs about a second of CPU time
    warm = max(1, min(args.warmup, 2))
    per_token_us, sample, used = cpu_baseline(w, steps, warm)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": per_token_us, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": per_token_us / 1000.0, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w),
        "cpu_baseline": dict({"value": per_token_us, "unit": UNIT, "kind": "oracle", "sample": sample}, **used),
        "e2e": {"value": per_token_us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def workload_config(w):
    full_gb = sum(w.lens) * w.n_kv_heads * 512.0 * w.n_layers / 1e9
    small_gb = sum(w.k_small) * w.n_kv_heads * 512.0 * w.n_layers / 1e9
    return {"workload": w.name, "layers": w.n_layers, "batch": w.batch, "q_heads": w.n_q_heads,
            "kv_heads": w.n_kv_heads, "head_dim": 128, "context": max(w.lens), "context_min": min(w.lens),
            "k_small": max(w.k_small), "stride": w.stride, "schedule": w.schedule,
            "threshold": w.threshold if w.schedule == "dynamic" else None,
            "l2_hygiene": f"inputs larger than L2: every token walks all layers' distinct caches "
                          f"(full {full_gb:.1f} GB, small {small_gb:.2f} GB)",
            "launch": "one CUDA graph replay per token"}


# ----------------------------------------------------------------------------------------------- our arm
def max_over_ranks(ms: float, world: int, device=None) -> float:
    """Replicas only: the job's time for a timed region is the slowest rank's (MAX all-reduce of the device time)."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    tt = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return float(tt.item())


def whole_job_us_per_token(ms: float, steps: int, world: int) -> float:
    """N replicas decode N * steps tokens in the (max-over-ranks) time: whole-job microseconds per token."""
    return ms * 1000.0 / (steps * world)


def region_repeats(first_region_ms: float) -> int:
    """How many timed regions of K steps to take: one when a region lasts half a second or more, otherwise at
    least five and as many as fit into about a quarter of a second of device time (at most 50)."""
    if first_region_ms >= 500.0:
        return 1
    return int(min(50, max(5, math.ceil(250.0 / max(first_region_ms, 1e-3)))))


def measure_workload(args, w, dev, world, steps, warmup, level):
    """All device measurements of one workload.  level "full": everything the headline line reports;
    "compact": the timed schedule, the kinds of token and the per-kernel times only (rows of the other
    configurations).  Returns a dict; frees its device memory before returning."""
    import torch
    import torch.distributed as dist
    from paper_2411_05787_b200 import rkv, runner, synth

    full_level = level == "full"
    S, B, Hq, Hkv, NL = w.stride, w.batch, w.n_q_heads, w.n_kv_heads, w.n_layers
    dynamic = w.schedule == "dynamic"
    n_prof = 2 * S
    # most tokens decoded between two resets of the cache lengths (a region, the loops of comparison tokens, profiling)
    span = max(steps, warmup, 2 * S, n_prof, 24) + S + 2
    wl = synth.scaled(w, steps=span)
    k_max = max(w.k_small)
    full_hint = max(w.lens) + span + 1
    # a sequence that never refreshes keeps growing its small cache (dynamic schedule); fixed: at most S - 1 rows
    small_extra = (span + 2) if dynamic else (S + 2)
    small_hint = k_max + small_extra
    schedule = "one_stream" if (args.no_overlap or NL == 1) else args.full_schedule
    # Contexts: a workspace holds one full step's logits.  'deferred' keeps every layer's until the end of the token
    # (one context per layer); 'overlap' needs two that alternate (a layer's selection may still be reading while the
    # next layer's attention runs); one stream needs one.
    n_ctx = NL if schedule == "deferred" else (2 if NL > 1 else 1)
    ctxs = [rkv.Context(B, Hq, Hkv, full_hint, small_hint) for _ in range(n_ctx)]
    for c in ctxs:
        if args.small_min_chunk:
            c.set_option(rkv.OPT_SMALL_MIN_CHUNK, args.small_min_chunk)
        if args.no_dependent_launch:
            c.set_option(rkv.OPT_DEPENDENT_LAUNCH, 0)
        if args.no_small_cluster:
            c.set_option(rkv.OPT_SMALL_CLUSTER, 0)
        if args.no_interleave:
            c.set_option(rkv.OPT_INTERLEAVE_TILES, 0)
        if args.select_keys_per_cta:
            c.set_option(rkv.OPT_SELECT_KEYS_PER_CTA, args.select_keys_per_cta)
        if args.score_slice:
            c.set_option(rkv.OPT_SCORE_SLICE, args.score_slice)

    # per-token inputs: one contiguous block per token = all layers' q, then all k_new, then all v_new, so that
    # one copy stages a token and the calls get contiguous views.  Queries follow the workload's AR(1) process
    # per layer and sequence (the dynamic trigger depends on it).
    n_in = min(span + 1, 320)                    # distinct tokens kept; the loop cycles through them
    win = synth.scaled(w, steps=n_in - 1)
    nq, nk = NL * B * Hq * 128, NL * B * Hkv * 128
    row = (Hq + 2 * Hkv) * 128
    inputs_host = torch.empty((n_in, nq + 2 * nk), dtype=torch.bfloat16).pin_memory()
    for l in range(NL):
        qs = synth.query_trajectory(win, l)                       # [n_in, B, Hq, 128]
        kn, vn = synth.new_token_kv(win, l)                       # [n_in, B, Hkv, 128]
        inputs_host[:, :nq].view(n_in, NL, B * Hq * 128)[:, l] = qs.reshape(n_in, -1)
        inputs_host[:, nq: nq + nk].view(n_in, NL, B * Hkv * 128)[:, l] = kn.reshape(n_in, -1)
        inputs_host[:, nq + nk:].view(n_in, NL, B * Hkv * 128)[:, l] = vn.reshape(n_in, -1)
    inputs_dev = inputs_host.to(dev)
    stage = torch.zeros((nq + 2 * nk,), dtype=torch.bfloat16, device=dev)
    q_stage = stage[:nq].view(NL, B, Hq, 128)
    k_stage = stage[nq: nq + nk].view(NL, B, Hkv, 128)
    v_stage = stage[nq + nk:].view(NL, B, Hkv, 128)
    outs = torch.zeros((NL, B, Hq * 128), dtype=torch.bfloat16, device=dev)
    outs_host = torch.zeros((NL, B, Hq * 128), dtype=torch.bfloat16).pin_memory()
    flag_total = torch.zeros((NL, B), dtype=torch.int32, device=dev)

    stage.copy_(inputs_dev[0])
    layers = []
    # all layers' full caches in one K and one V buffer (each layer works on its view of it), so that the full step
    # can also be measured as one call over layers x B sequences
    stack = synth.alloc_layer_stack(wl, dev) if (NL > 1 and full_level and not dynamic) else None
    for l in range(NL):
        cache = synth.fill_layer(wl, l, dev, into=synth.layer_view(stack, l, B) if stack is not None else None)
        synth.plant_heavy(w, cache, l, q_stage[l])
        st = runner.LayerState(ctxs[l % n_ctx], cache, list(w.k_small), small_extra, Hq, Hkv)
        st.out = outs[l].view(B, Hq, 128)
        layers.append(st)
    len0 = torch.tensor(list(w.lens), dtype=torch.int32, device=dev)
    launch_total = lambda: sum(c.launch_count for c in ctxs)

    overlapped = runner.OverlappedRefresh(layers) if schedule == "overlap" else None
    deferred = (runner.DeferredRefresh(layers, n_side=args.side_streams, select_keys_per_cta=args.deferred_keys_per_cta,
                                       score_slice=args.deferred_score_slice, early_scores=args.early_scores)
                if schedule == "deferred" else None)
    qf, kf, vf = (lambda l: q_stage[l]), (lambda l: k_stage[l]), (lambda l: v_stage[l])

    def token(kind: str):
        if kind == "full" and overlapped is not None:
            return overlapped.run(qf, kf, vf, max_len_hint=full_hint)
        if kind == "full" and deferred is not None:
            return deferred.run(qf, kf, vf, max_len_hint=full_hint)
        if kind == "check" and (overlapped is not None or deferred is not None):
            return (overlapped or deferred).run_checked(qf, kf, vf, w.threshold, small_hint=small_hint,
                                                        full_hint=full_hint,
                                                        after_trigger=lambda l, st: flag_total[l].add_(st.flag))
        for l, st in enumerate(layers):
            q, kn, vn = q_stage[l], k_stage[l], v_stage[l]
            if kind in ("full", "full_seq"):
                st.append(kn, vn)
                st.refresh(q, max_len_hint=full_hint)
            elif kind == "full_prof":  # the timed full token's kernels, one stream (per-kernel timing)
                st.append_refresh_attention(q, kn, vn, max_len_hint=full_hint)
                st.refresh_select(q)
            elif kind == "attn_only":  # the main stream of the full token alone: streaming pass + fold per layer
                st.append_refresh_attention(q, kn, vn, max_len_hint=full_hint)
            elif kind == "fs_only":    # rkv_full_step alone: attention, scores and top-K of every layer in stream order
                st.ctx.full_step(q, st.full_c, st.k_small, st.k_max, st.out, st.topk_idx, q_last_full=st.q_last_full,
                                 max_len_hint=full_hint)
            elif kind == "score":      # score-only refresh: K-only pass + top-K, rebuild, attention over the new small cache
                st.append(kn, vn)
                st.refresh_scores_only(q, max_len_hint=full_hint, small_hint=small_hint)
            elif kind == "small":      # append + partial step in one call (one launch)
                st.append_partial(q, kn, vn, max_len_hint=small_hint)
            else:                      # check: the trigger decides per sequence; both branches run under its masks
                st.check_trigger(q, w.threshold)
                st.append_partial(q, kn, vn, active=st.not_flag, max_len_hint=small_hint)
                st.refresh(q, active=st.flag, max_len_hint=full_hint)
                flag_total[l].add_(st.flag)

    # layer-batched partial step: every layer's small cache in one buffer, one launch per token
    batched = runner.LayerBatchedSmall(layers, small_hint) if (NL > 1 and not dynamic) else None
    # layer-batched full step: one rkv_full_step per token over layers x B sequences
    batched_full = (runner.LayerBatchedFull(stack, NL, list(w.k_small), Hq, Hkv, full_hint) if stack is not None else None)

    # initial small caches + eager warm-up of every kernel (also creates the tensor maps)
    for l, st in enumerate(layers):
        st.refresh(q_stage[l], max_len_hint=full_hint)
    kinds = ["small", "full"]
    if full_level:
        kinds += ["score", "fs_only"]
    if schedule != "one_stream":
        kinds += ["full_seq", "attn_only"]
    if dynamic:
        kinds.append("check")
    for kind in kinds:
        token(kind)
    if batched is not None:
        batched.sync_from_layers()
        batched.append_partial(q_stage, k_stage, v_stage, outs.view(NL, B, Hq, 128))
    if batched_full is not None:
        batched_full.full_step(q_stage)
    torch.cuda.synchronize()

    # capture one graph per kind of token
    side = torch.cuda.Stream()
    graphs, launches_per = {}, {}
    for kind in kinds:
        gr = torch.cuda.CUDAGraph()
        before = launch_total()
        with torch.cuda.stream(side):
            with torch.cuda.graph(gr, stream=side):
                token(kind)
        launches_per[kind] = launch_total() - before
        graphs[kind] = gr
    if batched is not None:
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(gr, stream=side):
                batched.append_partial(q_stage, k_stage, v_stage, outs.view(NL, B, Hq, 128))
        graphs["small_batched"], launches_per["small_batched"] = gr, 1
    if batched_full is not None:
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(gr, stream=side):
                batched_full.full_step(q_stage)
        graphs["fs_batched"], launches_per["fs_batched"] = gr, 3
    torch.cuda.synchronize()

    tok_counter = [1]

    def reset():
        """Back to the workload's starting lengths, small caches rebuilt: every timed region decodes the same tokens."""
        for st in layers:
            st.full.len.copy_(len0)
        tok_counter[0] = 1
        stage.copy_(inputs_dev[0])
        graphs["full"].replay()
        for st in layers:                        # the rebuild token appended a row: the region starts at the stated length
            st.full.len.copy_(len0)

    def kind_of(t, always_full, force_small, force_kind=None):
        if force_kind:
            return force_kind
        if force_small:
            return "small"
        if always_full:
            return "full"
        if t % S != 0:
            return "small"
        return "check" if dynamic else "full"

    readback = torch.cuda.Stream()
    ev_token, ev_read = torch.cuda.Event(), torch.cuda.Event()

    def run_tokens(n, e2e=False, always_full=False, force_small=False, force_kind=None):
        """Enqueue n decode tokens; returns the count of each kind.  e2e: every token's inputs come from pinned host
        memory and its outputs go back to the host.  The read-back runs in a stream of its own: the NEXT token's
        inputs are copied in while it is under way (the two directions have their own copy engines), but the next
        token's kernels start only when the read-back is complete (they overwrite what it reads)."""
        cnt = {k: 0 for k in graphs}
        main = torch.cuda.current_stream()
        for _ in range(n):
            t = tok_counter[0]; tok_counter[0] += 1
            src = inputs_host if e2e else inputs_dev
            stage.copy_(src[t % n_in], non_blocking=True)
            kind = kind_of(t, always_full, force_small, force_kind)
            if e2e:
                main.wait_event(ev_read)          # (the first wait finds the event unrecorded and passes)
            graphs[kind].replay()
            if e2e:
                ev_token.record(main)
                readback.wait_event(ev_token)
                with torch.cuda.stream(readback):
                    outs_host.copy_(outs, non_blocking=True)
                    ev_read.record(readback)
            cnt[kind] += 1
        if e2e:
            main.wait_event(ev_read)              # the region ends when the last token has been read back
        return cnt

    def timed(n, fresh=True, **kw):
        if fresh:
            reset()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        cnt = run_tokens(n, **kw)
        e1.record()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        return max_over_ranks(e0.elapsed_time(e1), world, dev), cnt

    def repeated(n, **kw):
        """Regions of n tokens each, every one from the same starting state; (median ms, all ms, token counts)."""
        ms0, cnt = timed(n, **kw)
        reps = args.regions if args.regions > 0 else region_repeats(ms0)
        if world > 1:                            # every rank must take the same number of regions
            tt = torch.tensor([reps], dtype=torch.int32, device=dev)
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
            reps = int(tt.item())
        all_ms = [ms0] + [timed(n, **kw)[0] for _ in range(reps - 1)]
        return statistics.median(all_ms), all_ms, cnt

    def median3(n, **kw):
        return statistics.median([timed(n, **kw)[0] for _ in range(3)])

    rank = int(os.environ.get("RANK", "0"))
    # ---- main measurement: inputs resident in HBM.  Clocks are sampled from the warm-up on (same load as the timed
    # regions, which may be shorter than one sample period).
    sampler = ClockSampler(torch.cuda.current_device() if "CUDA_VISIBLE_DEVICES" not in os.environ else 0)
    if rank == 0 and full_level:
        sampler.start()
    reset()
    run_tokens(warmup)
    torch.cuda.synchronize()
    flag_total.zero_()
    ms, all_ms, cnt = repeated(steps)
    clocks = sampler.stop() if (rank == 0 and full_level) else {}
    us_per_token = whole_job_us_per_token(ms, steps, world)
    launches = sum(cnt[k] * launches_per[k] for k in cnt)
    refreshed = (int(flag_total.sum().item()) // max(len(all_ms), 1)) if dynamic else cnt["full"] * NL * B
    checks = cnt.get("check", 0)
    res = {"us_per_token": us_per_token, "ms_per_region": ms, "regions_ms": all_ms, "clocks": clocks,
           "launches": launches, "refreshed": refreshed, "checks": checks, "schedule": schedule,
           "launches_per": launches_per}

    # ---- end to end: inputs from pinned host memory, outputs back to the host, every token
    if full_level:
        reset()
        run_tokens(min(warmup, 10), e2e=True)
        ms_e2e, all_e2e, _ = repeated(steps, e2e=True)
        res["e2e_us"] = whole_job_us_per_token(ms_e2e, steps, world)
        res["e2e_regions_ms"] = all_e2e
        res["h2d"], res["d2h"] = NL * B * row * 2, NL * B * Hq * 128 * 2

    # ---- comparison loops: always-full attention (the vanilla comparator) on the same caches, the other schedules
    # of the full token, and partial steps only
    n_cmp = 20
    per_layer = lambda ms_: ms_ * 1000.0 / (n_cmp * world) / NL
    reset()
    run_tokens(3, always_full=True)
    ms_full = median3(n_cmp, always_full=True)
    res["always_full_us_per_token"] = ms_full * 1000.0 / (n_cmp * world)
    graph_us = {"full_token": per_layer(ms_full)}
    ms_attn_only = None
    if "full_seq" in graphs:
        graph_us["full_token_one_stream"] = per_layer(median3(n_cmp, force_kind="full_seq"))
        # the streaming passes (+ folds) of all layers back to back, nothing beside them: what the pass achieves when
        # no event bracket separates it from its neighbours
        ms_attn_only = median3(n_cmp, force_kind="attn_only")
        graph_us["attention_and_fold_only"] = per_layer(ms_attn_only)
    if "fs_only" in graphs:
        graph_us["full_step_call_only"] = per_layer(median3(n_cmp, force_kind="fs_only"))
    if "score" in graphs:
        graph_us["score_only_refresh_token"] = per_layer(median3(n_cmp, force_kind="score"))
    ms_small = []
    for _ in range(3):                           # the partial tokens between two full ones: K .. K+S-2 rows
        reset()
        ms_small.append(timed(S - 1, fresh=False, force_small=True)[0])
    ms_small = statistics.median(ms_small)
    res["small_only_us_per_token"] = ms_small * 1000.0 / ((S - 1) * world)
    graph_us["small_token"] = res["small_only_us_per_token"] / NL
    if batched is not None:
        msb = []
        for _ in range(3):
            reset()
            batched.sync_from_layers()
            msb.append(timed(S - 1, fresh=False, force_kind="small_batched")[0])
        res["small_batched_us_per_token"] = statistics.median(msb) * 1000.0 / ((S - 1) * world)
    if batched_full is not None:
        res["fs_batched_us_per_token"] = median3(n_cmp, force_kind="fs_batched") * 1000.0 / (n_cmp * world)
    res["in_graph_us_per_layer"] = graph_us

    # ---- per-kernel device time: every launch bracketed by CUDA events on its stream (fixed-stride schedule,
    # two periods, every sequence active).  A spin kernel first keeps the GPU busy while the host enqueues, so
    # that the launches sit back to back in the queue and an event pair measures the kernel, not the host.
    reset()
    torch.cuda.synchronize()
    for c in ctxs:
        c.set_profiling(True)
        c.get_profile()
    torch.cuda._sleep(int(8e7))
    for i in range(n_prof):
        t = tok_counter[0]; tok_counter[0] += 1
        stage.copy_(inputs_dev[t % n_in])
        token("full_prof" if i % S == 0 else "small")
    torch.cuda.synchronize()
    prof = {}
    for c in ctxs:
        for name, (us, n) in c.get_profile().items():
            us0, n0 = prof.get(name, (0.0, 0))
            prof[name] = (us0 + us, n0 + n)
        c.set_profiling(False)
    status = 0
    for c in ctxs:
        status |= c.device_status()
    if batched is not None:
        status |= batched.ctx.device_status()
    if batched_full is not None:
        status |= batched_full.ctx.device_status()
    res["status"] = status
    kern = {name: {"launches": c, "avg_us": us / c} for name, (us, c) in prof.items() if c}
    pos_full = sum(w.lens) + B * (n_prof / 2.0)                 # positions one full-step launch streams (all sequences)
    pos_small = sum(w.k_small) + B * (S / 2.0)
    res["kv_bytes_full"] = pos_full * Hkv * 512.0               # K+V bytes one full-step launch must read
    res["kv_bytes_small"] = pos_small * Hkv * 512.0
    kern["attn_full"]["gbs"] = res["kv_bytes_full"] / (kern["attn_full"]["avg_us"] * 1e-6) / 1e9
    kern["attn_small"]["gbs"] = res["kv_bytes_small"] / (kern["attn_small"]["avg_us"] * 1e-6) / 1e9
    kern["gather"]["gbs"] = 2 * sum(w.k_small) * Hkv * 512.0 / (kern["gather"]["avg_us"] * 1e-6) / 1e9
    # the selection is two launches: the score pass (logits -> keys, histogram) and the top-K proper
    kern["score_plus_select"] = {"launches": kern["select"]["launches"],
                                 "avg_us": kern["select"]["avg_us"] + (kern["score"]["avg_us"] if "score" in kern else 0.0)}
    res["kern"] = kern

    # free everything this workload holds on the device
    del graphs, layers, overlapped, deferred, batched, batched_full, stack, ctxs, inputs_dev, stage, outs, flag_total, st, cache
    del q_stage, k_stage, v_stage
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    return res


def fractions(res, w, peak):
    """Roofline fractions of one workload's measurements (K/V bytes touched over time, against the measured copy
    peak and against the nominal 8 TB/s)."""
    NL = w.n_layers
    kern, g = res["kern"], res["in_graph_us_per_layer"]
    kvf, kvs = res["kv_bytes_full"], res["kv_bytes_small"]
    gbs = lambda nbytes, us: nbytes / (us * 1e-6) / 1e9
    out = {
        "attn_full_single_launch": {"us": kern["attn_full"]["avg_us"], "gbs": gbs(kvf, kern["attn_full"]["avg_us"])},
        "small_token_per_layer_launch_in_graph": {"us": g["small_token"], "gbs": gbs(kvs, g["small_token"])},
        "full_token_in_graph": {"us": g["full_token"], "gbs": gbs(kvf, g["full_token"])},
    }
    if g.get("attention_and_fold_only"):
        out["attention_and_fold_chained"] = {"us": g["attention_and_fold_only"], "gbs": gbs(kvf, g["attention_and_fold_only"])}
    if g.get("full_step_call_only"):
        out["full_step_call_attention_scores_topk"] = {"us": g["full_step_call_only"], "gbs": gbs(kvf, g["full_step_call_only"])}
    if "small_batched_us_per_token" in res:
        us = res["small_batched_us_per_token"]
        out["small_token_layer_batched_one_launch"] = {"us_per_token": us, "us": us / NL, "gbs": gbs(kvs * NL, us)}
    if "fs_batched_us_per_token" in res:
        us = res["fs_batched_us_per_token"]
        out["full_step_call_layer_batched_one_call"] = {"us_per_token": us, "us": us / NL, "gbs": gbs(kvf * NL, us)}
    for v in out.values():
        v["frac_of_measured"] = v["gbs"] / peak
        v["frac_of_8TBs"] = v["gbs"] / 8000.0
    return out


def compact_row(res, w, peak):
    k = res["kern"]
    return {"config": workload_config(w), "us_per_token": res["us_per_token"], "regions": len(res["regions_ms"]),
            "always_full_us_per_token": res["always_full_us_per_token"],
            "small_only_us_per_token": res["small_only_us_per_token"],
            "small_batched_us_per_token": res.get("small_batched_us_per_token"),
            "full_token_schedule": res["schedule"],
            "in_graph_us_per_layer": res["in_graph_us_per_layer"],
            "per_layer_kernel_us": {n: round(v["avg_us"], 2) for n, v in k.items()},
            "fractions": fractions(res, w, peak), "device_status": res["status"],
            "full_steps_in_timed_region": {"sequence_layer_refreshes": res["refreshed"], "check_tokens": res["checks"]}}


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
    from paper_2411_05787_b200 import synth

    dev = torch.device("cuda", torch.cuda.current_device())
    w = make_workload(args)
    res = measure_workload(args, w, dev, world, args.steps, args.warmup, "full")

    # compact rows of the other configurations: a few resident layers each, single GPU only
    rows = {}
    if world == 1 and not args.no_extra_workloads and args.workload == "cfg2" and not args.layers:
        extra = [("cfg3", synth.config3(n_layers=4)), ("cfg4", synth.config4(n_layers=2)),
                 ("cfg1", synth.config1()), ("lm16k_S15", synth.paper_point("lm16k_S15", n_layers=8)),
                 ("novel128k_S10", synth.paper_point("novel128k_S10", n_layers=4)),
                 ("qwen16k_dyn095_qc5", synth.paper_point("qwen16k_dyn095_qc5", n_layers=8))]
        peak0 = load_peaks()[0]
        for name, wx in extra:
            try:
                rows[name] = compact_row(measure_workload(args, wx, dev, 1, 20, 5, "compact"), wx, peak0)
            except Exception as e:   # a row that cannot be measured is reported as such, never silently dropped
                rows[name] = {"error": f"{type(e).__name__}: {e}"}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_src = load_peaks()
    NL = w.n_layers
    kern, g = res["kern"], res["in_graph_us_per_layer"]
    fr = fractions(res, w, peak)
    kvf = res["kv_bytes_full"]
    # The dominant kernel's average launch duration: CUDA events around regions of 20 tokens in which the attention
    # passes of all layers follow each other on one stream (each with its short fold kernel, whose time stays in the
    # figure: a lower bound for the pass itself).  Without that loop: one launch alone between two events.
    if "attention_and_fold_chained" in fr:
        achieved_main = fr["attention_and_fold_chained"]["gbs"]
        how_main = ("CUDA events around 20 tokens x %d layers of rkv_append_full_attention launched back to back on one "
                    "stream; bytes / (region / launches), the fold kernel's time included; median of 3 regions" % NL)
    else:
        achieved_main = fr["attn_full_single_launch"]["gbs"]
        how_main = "one launch alone between two CUDA events, averaged over the profiling pass"
    tpb, tsrc = attn_traffic_per_kv_byte()
    full_step = fr.get("full_step_call_attention_scores_topk", fr["full_token_in_graph"])
    small_b = fr.get("small_token_layer_batched_one_launch")
    full_b = fr.get("full_step_call_layer_batched_one_call")
    result = {
        "metric": METRIC, "value": res["us_per_token"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": res["ms_per_region"] / args.steps, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16 in / fp32 accumulate", "data": "synthetic",
        "config": workload_config(w),
        "clocks": res["clocks"],
        "e2e": {"value": res["e2e_us"], "unit": UNIT, "h2d_bytes_per_step": res["h2d"], "d2h_bytes_per_step": res["d2h"]},
        "gpu_launches": res["launches"],
        "roofline": {"bound": "hbm", "kernel": "attn_kernel<full> (full-cache attention + score logits, the token's "
                                               "append fused in)",
                     "achieved": achieved_main, "peak": peak, "unit": "GB/s", "frac": achieved_main / peak,
                     "peak_source": peak_src, "how": how_main,
                     # one launch alone between two CUDA events (carries the launch and drain latency of a kernel
                     # that nothing overlaps)
                     "achieved_single_launch": fr["attn_full_single_launch"]["gbs"],
                     "frac_single_launch": fr["attn_full_single_launch"]["frac_of_measured"],
                     "traffic": (kvf * tpb if tpb and w.name.startswith("cfg2") else None), "traffic_source": tsrc,
                     "algorithmic_bytes_per_launch": kvf,
                     # the full step (attention + scores + top-K) and the partial step as wholes, K/V bytes over the
                     # step's time, against the nominal 8 TB/s
                     "step_fractions": {
                         "full_attention_scores_topk_step_frac_of_8TBs": full_step["frac_of_8TBs"],
                         "full_attention_scores_topk_step_us_per_layer": full_step["us"],
                         "full_attention_scores_topk_step_is": "rkv_full_step of every layer in stream order inside a "
                                                               "CUDA graph (attention pass, score pass, top-K): region / launches",
                         "full_attention_scores_topk_step_layer_batched_frac_of_8TBs": full_b["frac_of_8TBs"] if full_b else None,
                         "full_attention_scores_topk_step_layer_batched_is": "all layers' full caches in one buffer, ONE "
                                                                             "rkv_full_step per token over layers x B sequences "
                                                                             "(three launches; legal only because the synthetic "
                                                                             "per-layer queries are independent)",
                         "small_step_frac_of_8TBs": fr["small_token_per_layer_launch_in_graph"]["frac_of_8TBs"],
                         "small_step_us_per_layer": fr["small_token_per_layer_launch_in_graph"]["us"],
                         "small_step_is": "rkv_append_small_step, one launch per layer inside a CUDA graph (what a decoder can do)",
                         "small_step_layer_batched_frac_of_8TBs": small_b["frac_of_8TBs"] if small_b else None,
                         "small_step_layer_batched_is": "all layers' small caches in one buffer, ONE launch per token "
                                                        "(legal only because the synthetic per-layer queries are independent)"}},
        "detail": {
            "timed_regions": {"count": len(res["regions_ms"]), "steps_each": args.steps,
                              "us_per_token_median": res["us_per_token"],
                              "us_per_token_min": min(res["regions_ms"]) * 1000.0 / (args.steps * world),
                              "us_per_token_max": max(res["regions_ms"]) * 1000.0 / (args.steps * world),
                              "each_region": "starts from the workload's stated lengths with freshly rebuilt small caches"},
            "always_full_us_per_token": res["always_full_us_per_token"],
            "refresh_speedup_vs_always_full": res["always_full_us_per_token"] / res["us_per_token"],
            "small_only_us_per_token": res["small_only_us_per_token"],
            "small_step_layer_batched": ({"us_per_token": res["small_batched_us_per_token"],
                                          "gbs": small_b["gbs"], "frac_of_measured": small_b["frac_of_measured"],
                                          "frac_of_8TBs": small_b["frac_of_8TBs"]} if small_b else None),
            "full_step_layer_batched": ({"us_per_token": res["fs_batched_us_per_token"], "gbs": full_b["gbs"],
                                         "frac_of_measured": full_b["frac_of_measured"],
                                         "frac_of_8TBs": full_b["frac_of_8TBs"]} if full_b else None),
            "full_steps_in_timed_region": {"sequence_layer_refreshes": res["refreshed"], "check_tokens": res["checks"],
                                           "of_possible": args.steps * NL * w.batch},
            "per_layer_kernel_us": kern,
            "fractions": fr,
            "in_graph_us_per_layer": g,
            "full_token_schedule": {"deferred": "the layers' attention passes follow each other; every layer's selection and "
                                                "small-cache rebuild run after the last pass, spread over %d side streams " % args.side_streams +
                                                "(one context per layer)",
                                    "overlap": "two streams: the layers' attention passes follow each other; a layer's "
                                               "selection and small-cache rebuild run behind its attention in a second stream",
                                    "one_stream": "one stream"}[res["schedule"]],
            "device_status": res["status"],
            "graph_launches": res["launches_per"],
            "workloads": rows,
        },
    }
    if not args.no_cpu_baseline and world == 1:
        per_token_us, sample, used = cpu_baseline(w, 4, 1, budget_s=12.0)    # about 12 s of oracle time
        result["cpu_baseline"] = dict({"value": per_token_us, "unit": UNIT, "kind": "oracle", "sample": sample}, **used)
    print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------------------------- end-to-end decode loop
def run_cfg5(args):
    """Random-init Llama-3.1-8B-shaped decoder, batch 1, 32768-token prompt (KV cache from an untimed torch
    prefill), greedy decoding with dynamic refresh (threshold 0.9, check every 5 tokens).  One step = one token
    through the whole model, replayed from a CUDA graph; reports tokens/s and the attention share."""
    import torch
    from paper_2411_05787_b200 import build
    build.build()
    torch.cuda.set_device(0)
    from paper_2411_05787_b200 import harness
    dev = torch.device("cuda", 0)
    shape = harness.llama8b()
    if args.layers:
        shape.n_layers = args.layers
    prompt_len, K = args.ctx or 32768, args.k_small or 2048
    QC, THR = args.qc or 5, (args.threshold if args.threshold >= 0.0 else 0.9)
    n_share = 20
    max_new = 2 * (args.steps + args.warmup) + 3 * n_share + 40
    dec = harness.LlamaDecoder(shape, prompt_len, max_new, K, QC, THR, seed=5, device=dev)
    g = torch.Generator(device="cpu"); g.manual_seed(55)
    t0 = time.perf_counter()
    dec.prefill(torch.randint(0, shape.vocab, (prompt_len,), generator=g).to(dev))
    prefill_s = time.perf_counter() - t0
    for kind in ("small", "check"):
        dec.token_step(kind)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graphs, launches_per = {}, {}
    for name, kw in (("small", {}), ("check", {}), ("small_attn", {"with_harness": False}),
                     ("check_attn", {"with_harness": False}), ("small_rest", {"with_attention": False})):
        gr = torch.cuda.CUDAGraph()
        before = dec.ctx.launch_count
        with torch.cuda.stream(side):
            with torch.cuda.graph(gr, stream=side):
                dec.token_step(name.split("_")[0], **kw)
        graphs[name], launches_per[name] = gr, dec.ctx.launch_count - before
    torch.cuda.synchronize()
    tok_host = torch.zeros((1,), dtype=torch.int32).pin_memory()
    history = torch.zeros((max_new + 8,), dtype=torch.int32, device=dev)
    counter = [3]

    def run(n, suffix="", e2e=False):
        c = {"small": 0, "check": 0}
        for _ in range(n):
            t = counter[0]; counter[0] += 1
            kind = dec.kind_of(t)
            graphs[kind + suffix].replay()
            if not suffix:
                history[t: t + 1].copy_(dec.token, non_blocking=True)
            if e2e:
                tok_host.copy_(dec.token, non_blocking=True)
                torch.cuda.current_stream().synchronize()      # the caller reads each token before the next step
            c[kind] += 1
        return c

    def timed(n, **kw):
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); c = run(n, **kw); e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1), c

    run(args.warmup)
    sampler = ClockSampler(0)
    sampler.start()
    dec.flag_total.zero_()
    ms, cnt = timed(args.steps)
    clocks = sampler.stop()
    refreshed = int(dec.flag_total.sum().item())
    run(min(args.warmup, 5), e2e=True)
    ms_e2e, _ = timed(args.steps, e2e=True)
    # attention share: the same attention calls alone (inputs as the last full token left them), and the rest alone
    ms_attn, _ = timed(n_share, suffix="_attn")
    counter[0] = ((counter[0] + QC - 1) // QC) * QC + 1          # keep the rest-only run on 'small' kinds only
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n_share):
        graphs["small_rest"].replay()
    e1.record(); torch.cuda.synchronize()
    ms_rest = e0.elapsed_time(e1)
    status = dec.ctx.device_status()
    peak, peak_src = load_peaks()
    us_token = ms * 1000.0 / args.steps
    attn_us = ms_attn * 1000.0 / n_share
    rest_us = ms_rest * 1000.0 / n_share
    wbytes = harness.weight_bytes(shape)
    result = {
        "metric": "greedy decode tokens/s, batch 1 (Llama-3.1-8B-shaped random-init model, dynamic refresh)",
        "value": 1e6 / us_token, "unit": "tokens/s", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 weights and KV, fp32 activations and accumulation", "data": "synthetic",
        "config": {"workload": "cfg5_llama8b_decode_L%d_K%d_dyn%d" % (prompt_len, K, QC), "layers": shape.n_layers,
                   "hidden": shape.hidden, "ffn": shape.ffn, "vocab": shape.vocab, "q_heads": shape.n_q,
                   "kv_heads": shape.n_kv, "context": prompt_len, "k_small": K, "threshold": THR, "stride": QC,
                   "prefill": "untimed torch set-up pass (bf16 matrix products, causal attention), %.1f s" % prefill_s,
                   "l2_hygiene": "inputs larger than L2: each token streams %.1f GB of weights" % (wbytes / 1e9),
                   "launch": "one CUDA graph replay per token"},
        "clocks": clocks,
        "e2e": {"value": 1e6 / (ms_e2e * 1000.0 / args.steps), "unit": "tokens/s", "h2d_bytes_per_step": 0,
                "d2h_bytes_per_step": 4},
        "gpu_launches": cnt["small"] * launches_per["small"] + cnt["check"] * launches_per["check"],
        "roofline": {"bound": "hbm", "kernel": "whole decode token (bf16 weights once + small-cache K/V; full-cache K/V "
                     "on refreshes not counted)", "achieved": (wbytes + shape.n_layers * K * shape.n_kv * 512.0) / (us_token * 1e-6) / 1e9,
                     "peak": peak, "unit": "GB/s", "peak_source": peak_src, "traffic": None,
                     "algorithmic_bytes_per_launch": wbytes + shape.n_layers * K * shape.n_kv * 512.0},
        "detail": {"us_per_token": us_token, "attention_only_us_per_token": attn_us, "rest_only_us_per_token": rest_us,
                   "attention_share_of_step": attn_us / us_token,
                   "layer_refreshes_in_timed_region": refreshed, "check_tokens": cnt["check"],
                   "of_possible": cnt["check"] * shape.n_layers, "device_status": status,
                   "library_launches_per_token": {k: v for k, v in launches_per.items() if "_" not in k},
                   "harness_launches_per_token": 5 * shape.n_layers + 3,
                   "first_tokens": history[3: 19].tolist()},
    }
    result["roofline"]["frac"] = result["roofline"]["achieved"] / peak
    print(json.dumps(result))


def main():
    args = parse_args()
    if args.workload == "cfg5":
        if args.impl == "reference":
            run_reference(args)             # the oracle covers the attention calls: cfg5's are cfg2's
        else:
            run_cfg5(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
