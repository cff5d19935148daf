"""Seeded synthetic inputs shaped like the paper's long-context decode workloads.

This module only *draws numbers and lays them out*; it contains none of the
method's arithmetic (no attention, no softmax, no selection, no trigger) and
is the one module that both the tests of the CPU oracle and the CUDA path may
use.  Everything is generated with a seeded torch.Generator on the requested
device and then handed, as the same bf16 bytes, to whichever side consumes it.

Cache layout (one layer): K and V are each one bf16 buffer of `n_rows` rows of
128 channels.  Sequence b, KV head g, position p lives in row
`row_offset[b] + g * cap[b] + p`, which lets ragged batches be packed.

Workload shapes follow the paper's experiment settings (Sec. 3 "Inference
settings", App. A.1, A.4): Llama-3.1-8B (32 query / 8 KV heads) and Qwen2-7B
(28 / 4) attention with head size 128, contexts of 16K-128K tokens, small
cache K = L/8 capped at a few thousand, strides 5-15, thresholds 0.85-0.95.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np
import torch

HEAD_DIM = 128
ZETA_1P1 = 10.584448464950803   # Riemann zeta(1.1), normaliser of the Zipf(1.1) law


@dataclass
class Workload:
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    lens: list            # context length per sequence
    k_small: list         # small-cache size per sequence
    steps: int            # decode steps T
    schedule: str         # "fixed" or "dynamic"
    stride: int           # S (fixed) or QC stride (dynamic)
    threshold: float = 0.0
    rho: list = field(default_factory=list)      # AR(1) coefficient per sequence (None -> random walk)
    kv_scale: float = 1.0
    heavy_frac: float = 0.01
    heavy_count: int = 0          # if > 0, overrides heavy_frac
    heavy_gain: float = 10.0      # heavy key = noise*heavy_noise + gain * u(q)
    heavy_noise: float = 1.0
    heavy_zipf: bool = False      # heavy key = noise * min(z, 16), z ~ Zipf(1.1)
    replant_every: int = 0        # move the heavy positions every this many steps
    walk_sigma: float = 0.1       # random-walk step when rho is None
    seed: int = 0

    @property
    def batch(self) -> int:
        return len(self.lens)

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


def config1() -> Workload:
    """Single layer, L=2048, K=256, S=4, 16 steps, planted heavy keys, drifting query."""
    return Workload("cfg1_L2048_K256_S4", 1, 32, 8, [2048], [256], 16, "fixed", 4,
                    rho=[None], kv_scale=1.0 / math.sqrt(HEAD_DIM), heavy_count=32,
                    heavy_gain=4.0, heavy_noise=0.0, walk_sigma=0.1, seed=0)


def config2(n_layers: int = 32, ctx: int = 32768, steps: int = 512, k_small: int = 0, stride: int = 10) -> Workload:
    """Llama-3.1-8B attention shape, batch 1, L=32768, K=2048, fixed stride 10 (k_small = 0: ctx / 16)."""
    k = k_small or ctx // 16
    return Workload(f"cfg2_llama8b_L{ctx}_K{k}_S{stride}", n_layers, 32, 8, [ctx], [k], steps,
                    "fixed", stride, rho=[0.95], replant_every=64, seed=2)


def config3(n_layers: int = 28, ctx: int = 65536, steps: int = 1024, qc: int = 5, k_small: int = 0,
            threshold: float = 0.9) -> Workload:
    """Qwen2-7B attention shape (G=7), batch 4, L=65536, K=4096, dynamic refresh at 0.9 (k_small = 0: ctx / 16)."""
    k = k_small or ctx // 16
    return Workload(f"cfg3_qwen7b_L{ctx}_K{k}_dyn{qc}", n_layers, 28, 4, [ctx] * 4, [k] * 4,
                    steps, "dynamic", qc, threshold=threshold, rho=[0.80, 0.90, 0.96, 0.99], seed=3)


# The paper's own operating points (Sec. 3 "Inference settings", Sec. 4.1 on strides, App. A.4 on thresholds):
# K = L / 8 - 16K-token language-modelling inputs with K = 2048 and 256 generated tokens, 100K+-token inputs with
# K = 4096 - fixed strides of 10 and 15, and the query-similarity trigger checked every 5 or 10 steps with
# threshold 0.85 (Llama-3.1-8B) or 0.95 (Qwen2-7B), batch 1.  Shapes only: data and weights are synthetic.
PAPER_POINTS = {
    # name: (model shape, context, K, schedule, stride or QC, threshold, decode steps)
    "lm16k_S10": ("llama", 16384, 2048, "fixed", 10, 0.0, 256),
    "lm16k_S15": ("llama", 16384, 2048, "fixed", 15, 0.0, 256),
    "lm16k_dyn085_qc5": ("llama", 16384, 2048, "dynamic", 5, 0.85, 256),
    "lm16k_dyn085_qc10": ("llama", 16384, 2048, "dynamic", 10, 0.85, 256),
    "novel128k_S10": ("llama", 131072, 4096, "fixed", 10, 0.0, 256),
    "novel128k_dyn085_qc10": ("llama", 131072, 4096, "dynamic", 10, 0.85, 256),
    "qwen16k_dyn095_qc5": ("qwen", 16384, 2048, "dynamic", 5, 0.95, 256),
    "qwen16k_dyn095_qc10": ("qwen", 16384, 2048, "dynamic", 10, 0.95, 256),
}


def paper_point(name: str, n_layers: int = 0) -> Workload:
    """One of the paper's operating points as a batch-1 workload (AR(1) queries with rho = 0.95, 1 % heavy keys)."""
    model, ctx, k, schedule, stride, thr, steps = PAPER_POINTS[name]
    n_q, n_kv, layers = (32, 8, 32) if model == "llama" else (28, 4, 28)
    return Workload(f"paper_{name}", n_layers or layers, n_q, n_kv, [ctx], [k], steps, schedule, stride,
                    threshold=thr, rho=[0.95], replant_every=64, seed=7)


def config4(n_layers: int = 32, n_seq: int = 16, lo: int = 8192, hi: int = 131072, steps: int = 256) -> Workload:
    """Ragged batch: lengths log-uniform in [lo, hi], K = min(2048, L/8), stride 10."""
    rng = np.random.default_rng(4)
    lens = [int(math.floor(math.exp(rng.uniform(math.log(lo), math.log(hi))))) for _ in range(n_seq)]
    ks = [min(2048, l // 8) for l in lens]
    return Workload(f"cfg4_ragged{n_seq}_S10", n_layers, 32, 8, lens, ks, steps, "fixed", 10,
                    rho=[0.95] * n_seq, heavy_zipf=True, seed=4)


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (used for small parity cases)."""
    d = dict(w.__dict__)
    d.update(kw)
    return Workload(**d)


# --------------------------------------------------------------------------
@dataclass
class LayerCache:
    """Packed bf16 K/V buffers of one layer plus the index tensors that describe them."""
    k: torch.Tensor           # [n_rows, 128] bf16
    v: torch.Tensor
    row_offset: torch.Tensor  # [B] int64
    cap: torch.Tensor         # [B] int32
    len: torch.Tensor         # [B] int32

    @property
    def n_rows(self) -> int:
        return self.k.shape[0]

    def head_rows(self, b: int, g: int, host_cap=None, host_off=None) -> slice:
        off = int(self.row_offset[b]) if host_off is None else host_off[b]
        cap = int(self.cap[b]) if host_cap is None else host_cap[b]
        return slice(off + g * cap, off + (g + 1) * cap)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def alloc_cache(caps: list, lens: list, n_kv_heads: int, device, fill=None) -> LayerCache:
    """Allocate one layer's packed K/V with the given per-sequence capacities."""
    offs, total = [], 0
    for c in caps:
        offs.append(total)
        total += n_kv_heads * c
    if fill is None:
        k = torch.empty((total, HEAD_DIM), dtype=torch.bfloat16, device=device)
        v = torch.empty((total, HEAD_DIM), dtype=torch.bfloat16, device=device)
    else:
        k = torch.full((total, HEAD_DIM), fill, dtype=torch.bfloat16, device=device)
        v = torch.full((total, HEAD_DIM), fill, dtype=torch.bfloat16, device=device)
    return LayerCache(k, v,
                      torch.tensor(offs, dtype=torch.int64, device=device),
                      torch.tensor(caps, dtype=torch.int32, device=device),
                      torch.tensor(lens, dtype=torch.int32, device=device))


def unit_group_mean(q: torch.Tensor, n_kv_heads: int) -> torch.Tensor:
    """Unit vector of the mean of the G query heads of every KV group: [Hkv, 128] fp32."""
    qf = q.float().reshape(n_kv_heads, -1, HEAD_DIM).mean(dim=1)
    return qf / qf.norm(dim=1, keepdim=True).clamp_min(1e-20)


def heavy_positions(w: Workload, layer: int, b: int, epoch: int, n_ctx: int, device) -> torch.Tensor:
    """Distinct planted positions per KV head: [Hkv, n_heavy] int64 (seeded per epoch)."""
    n_heavy = w.heavy_count if w.heavy_count > 0 else int(math.ceil(w.heavy_frac * n_ctx))
    g = _gen(w.seed * 1000003 + layer * 7919 + b * 104729 + epoch * 15485863 + 17, "cpu")
    rows = [torch.randperm(n_ctx, generator=g)[:n_heavy] for _ in range(w.n_kv_heads)]
    return torch.stack(rows).to(device)


def layer_view(stack: LayerCache, layer: int, batch: int) -> LayerCache:
    """One layer's sequences of a cache that holds `batch` sequences per layer for several layers in one K and one V
    buffer: the same buffers, the layer's slice of the index tensors (row offsets stay global)."""
    sl = slice(layer * batch, (layer + 1) * batch)
    return LayerCache(stack.k, stack.v, stack.row_offset[sl], stack.cap[sl], stack.len[sl])


def alloc_layer_stack(w: Workload, device, extra_cap: int | None = None) -> LayerCache:
    """All layers' full caches in ONE K and ONE V buffer: layers x batch sequences."""
    extra = w.steps + 1 if extra_cap is None else extra_cap
    caps = [l + extra for l in w.lens] * w.n_layers
    return alloc_cache(caps, list(w.lens) * w.n_layers, w.n_kv_heads, device)


def fill_layer(w: Workload, layer: int, device, extra_cap: int | None = None, into: LayerCache | None = None) -> LayerCache:
    """Random K/V for all context positions of one layer (noise part only).  into: a layer_view() to fill in place."""
    extra = w.steps + 1 if extra_cap is None else extra_cap
    caps = [l + extra for l in w.lens]
    g = _gen(w.seed * 7907 + layer * 31 + 1, device)
    if into is not None:
        r0 = int(into.row_offset[0])
        r1 = r0 + w.n_kv_heads * sum(caps)
        assert into.cap.tolist() == caps
        step = 1 << 22
        for t in (into.k, into.v):
            for a in range(r0, r1, step):
                b = min(r1, a + step)
                t[a:b] = (torch.randn((b - a, HEAD_DIM), generator=g, device=device,
                                      dtype=torch.float32) * w.kv_scale).to(torch.bfloat16)
        return into
    cache = alloc_cache(caps, list(w.lens), w.n_kv_heads, device)
    # chunked so that the fp32 temporaries stay small next to the bf16 result
    step = 1 << 22
    for t in (cache.k, cache.v):
        for r0 in range(0, t.shape[0], step):
            r1 = min(t.shape[0], r0 + step)
            t[r0:r1] = (torch.randn((r1 - r0, HEAD_DIM), generator=g, device=device,
                                    dtype=torch.float32) * w.kv_scale).to(torch.bfloat16)
    return cache


def plant_heavy(w: Workload, cache: LayerCache, layer: int, q: torch.Tensor, epoch: int = 0,
                saved: dict | None = None) -> dict:
    """Overwrite the heavy positions' keys so that they line up with the current query.

    q: [B, Hq, 128] bf16.  Returns what is needed to restore the rows later.
    """
    device = cache.k.device
    offs = cache.row_offset.tolist()
    caps = cache.cap.tolist()
    restore = {}
    for b, n_ctx in enumerate(w.lens):
        pos = heavy_positions(w, layer, b, epoch, n_ctx, device)          # [Hkv, n_heavy]
        u = unit_group_mean(q[b], w.n_kv_heads).to(device)                   # [Hkv, 128]
        g = _gen(w.seed * 92821 + layer * 613 + b * 97 + epoch * 389 + 5, device)
        for h in range(w.n_kv_heads):
            rows = offs[b] + h * caps[b] + pos[h]
            restore[(b, h)] = (rows, cache.k[rows].clone())
            n = rows.shape[0]
            noise = torch.randn((n, HEAD_DIM), generator=g, device=device, dtype=torch.float32)
            if w.heavy_zipf:
                # min(z, 16) with z ~ Zipf(1.1): weights i^-1.1 for i < 16, the whole tail mass at 16
                wts = torch.arange(1, 17, dtype=torch.float64) ** -1.1
                wts[15] = ZETA_1P1 - wts[:15].sum()
                wts = wts.float().to(device)
                z = torch.multinomial(wts, n, replacement=True, generator=g).float() + 1.0
                newk = noise * z[:, None]
            else:
                newk = noise * w.heavy_noise + w.heavy_gain * u[h][None, :]
            cache.k[rows] = newk.to(torch.bfloat16)
    return restore


def unplant(cache: LayerCache, restore: dict) -> None:
    for rows, old in restore.values():
        cache.k[rows] = old


def query_trajectory(w: Workload, layer: int) -> torch.Tensor:
    """Per-step queries [T+1, B, Hq, 128] bf16 on the host (step 0 initialises C_p).

    AR(1) with coefficient rho keeps unit variance: q_t = rho q_{t-1} + sqrt(1-rho^2) e_t.
    rho None is the random walk q_t = q_{t-1} + walk_sigma e_t.  State is fp64.
    """
    g = _gen(w.seed * 1299709 + layer * 101 + 3, "cpu")
    shape = (w.n_q_heads, HEAD_DIM)
    out = torch.empty((w.steps + 1, w.batch) + shape, dtype=torch.bfloat16)
    for b in range(w.batch):
        rho = w.rho[b] if w.rho else 0.95
        state = torch.randn(shape, generator=g, dtype=torch.float64)
        out[0, b] = state.to(torch.bfloat16)
        for t in range(1, w.steps + 1):
            e = torch.randn(shape, generator=g, dtype=torch.float64)
            if rho is None:
                state = state + w.walk_sigma * e
            else:
                state = rho * state + math.sqrt(1.0 - rho * rho) * e
            out[t, b] = state.to(torch.bfloat16)
    return out


def new_token_kv(w: Workload, layer: int) -> tuple[torch.Tensor, torch.Tensor]:
    """K/V rows of the decoded tokens: two [T+1, B, Hkv, 128] bf16 host tensors (index 0 unused)."""
    g = _gen(w.seed * 2750159 + layer * 211 + 9, "cpu")
    shape = (w.steps + 1, w.batch, w.n_kv_heads, HEAD_DIM)
    k = (torch.randn(shape, generator=g, dtype=torch.float32) * w.kv_scale).to(torch.bfloat16)
    v = (torch.randn(shape, generator=g, dtype=torch.float32) * w.kv_scale).to(torch.bfloat16)
    return k, v


def to_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 bit patterns on the host (what the CPU checker consumes)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def head_view_bits(cache: LayerCache, b: int, which: str = "k") -> np.ndarray:
    """uint16 [Hkv, cap, 128] copy of one sequence's K or V region."""
    off = int(cache.row_offset[b])
    cap = int(cache.cap[b])
    t = cache.k if which == "k" else cache.v
    n_kv = (int(cache.row_offset[b + 1]) - off) // cap if b + 1 < cache.row_offset.shape[0] else (t.shape[0] - off) // cap
    return to_bits(t[off: off + n_kv * cap]).reshape(n_kv, cap, HEAD_DIM)
