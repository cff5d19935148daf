"""End-to-end decode harness: a random-init Llama-shaped decoder whose attention is the RefreshKV library.

This is the measuring harness of the end-to-end workload (tokens/s and the attention share of a decode
step), not part of the attention library.  The decoder pieces between attention calls (RMSNorm, bf16
matrix-vector products, rotary embedding, SwiGLU, embedding lookup, argmax) are the CUDA kernels of
libllama_harness.so (include/rkv_harness.h); this module marshals their arguments, owns the weights
and sequences the calls of one decode token.  The prompt's KV cache is produced by an untimed set-up
pass written with torch matrix products (`prefill`), which is not on the measured path.

The paper (arXiv 2411.05787, Sec. 3) runs RefreshKV inside Llama-3.1-8B with greedy decoding, dynamic
refresh (threshold s, query-comparison stride QC) and a small cache initialised from the attention
scores of the last prompt token (Sec. 2.2 "Prefilling stage"); the loop below follows that outline.
"""
from __future__ import annotations

import ctypes
import math
import os
from dataclasses import dataclass

import torch

from . import rkv, runner, synth

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libllama_harness.so")
EXPORTS = ["llh_rmsnorm", "llh_gemv", "llh_gemv_swiglu", "llh_rope_split", "llh_embed", "llh_argmax"]


def _load() -> ctypes.CDLL:
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it first (python -m paper_2411_05787_b200.build)")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i32, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_float
    lib.llh_rmsnorm.argtypes = [vp, vp, f32, vp, i32, vp]
    lib.llh_gemv.argtypes = [vp, vp, i32, vp, f32, vp, vp, i32, i32, vp]
    lib.llh_gemv_swiglu.argtypes = [vp, vp, vp, f32, vp, i32, i32, vp]
    lib.llh_rope_split.argtypes = [vp, vp, f32, vp, vp, vp, i32, i32, vp]
    lib.llh_embed.argtypes = [vp, vp, vp, i32, i32, vp]
    lib.llh_argmax.argtypes = [vp, i32, vp, vp]
    for n in EXPORTS:
        getattr(lib, n).restype = i32
    return lib


lib = _load()


def _p(t):
    return None if t is None else t.data_ptr()


def _st():
    return torch.cuda.current_stream().cuda_stream


def _ck(rc, what):
    if rc != 0:
        raise RuntimeError(f"{what} failed with code {rc}")


def rmsnorm(x, w, eps, y):
    _ck(lib.llh_rmsnorm(_p(x), _p(w), eps, _p(y), x.numel(), _st()), "llh_rmsnorm")


def gemv(w, x, y, residual=None, norm_w=None, eps=1e-5):
    """y = W x' (+ residual); with norm_w the input is RMS-normalised inside the kernel."""
    n_out, n_in = w.shape
    _ck(lib.llh_gemv(_p(w), _p(x), 1 if x.dtype == torch.bfloat16 else 0, _p(norm_w), eps, _p(residual), _p(y), n_out,
                     n_in, _st()), "llh_gemv")


def gemv_swiglu(w_gate_up, x, y, norm_w=None, eps=1e-5):
    _ck(lib.llh_gemv_swiglu(_p(w_gate_up), _p(x), _p(norm_w), eps, _p(y), w_gate_up.shape[0] // 2, w_gate_up.shape[1],
                            _st()), "llh_gemv_swiglu")


def rope_split(qkv, pos, theta, q, k, v, n_q, n_kv):
    _ck(lib.llh_rope_split(_p(qkv), _p(pos), theta, _p(q), _p(k), _p(v), n_q, n_kv, _st()), "llh_rope_split")


def embed(table, token, x):
    _ck(lib.llh_embed(_p(table), _p(token), _p(x), table.shape[1], table.shape[0], _st()), "llh_embed")


def argmax(logits, token):
    _ck(lib.llh_argmax(_p(logits), logits.numel(), _p(token), _st()), "llh_argmax")


@dataclass
class LlamaShape:
    hidden: int = 4096
    n_layers: int = 32
    n_q: int = 32
    n_kv: int = 8
    ffn: int = 14336
    vocab: int = 128256
    theta: float = 500000.0
    eps: float = 1e-5

    @property
    def params(self) -> int:
        per = (self.n_q + 2 * self.n_kv) * 128 * self.hidden + self.hidden * self.n_q * 128 + 3 * self.ffn * self.hidden
        return per * self.n_layers + 2 * self.vocab * self.hidden


class LlamaDecoder:
    """Weights, caches and the per-token call sequence.  Batch 1."""

    def __init__(self, shape: LlamaShape, prompt_len: int, max_new: int, k_small: int, qc_stride: int,
                 threshold: float, seed: int = 5, device="cuda"):
        self.s, self.dev = shape, torch.device(device)
        self.prompt_len, self.max_new, self.k_small = prompt_len, max_new, k_small
        self.qc, self.threshold = qc_stride, threshold
        s, dev = shape, self.dev
        g = torch.Generator(device=dev); g.manual_seed(seed)

        def w(*shp):   # bf16 N(0, 0.02), generated in slabs so that the fp32 temporary stays small
            t = torch.empty(shp, dtype=torch.bfloat16, device=dev)
            rows = max(1, (1 << 26) // shp[1])
            for r0 in range(0, shp[0], rows):
                r1 = min(shp[0], r0 + rows)
                t[r0:r1] = (torch.randn((r1 - r0, shp[1]), generator=g, device=dev) * 0.02).to(torch.bfloat16)
            return t
        self.embed_w, self.lm_head = w(s.vocab, s.hidden), w(s.vocab, s.hidden)
        self.final_norm = torch.ones((s.hidden,), dtype=torch.bfloat16, device=dev)
        self.layers_w = []
        for _ in range(s.n_layers):
            self.layers_w.append(dict(
                norm1=torch.ones((s.hidden,), dtype=torch.bfloat16, device=dev),
                norm2=torch.ones((s.hidden,), dtype=torch.bfloat16, device=dev),
                wqkv=w((s.n_q + 2 * s.n_kv) * 128, s.hidden), wo=w(s.hidden, s.n_q * 128),
                wgu=w(2 * s.ffn, s.hidden), wd=w(s.hidden, s.ffn)))
        cap = prompt_len + max_new + 2
        small_extra = max_new + 2            # a layer that never refreshes keeps growing its small cache
        self.full_hint, self.small_hint = cap, k_small + small_extra
        self.ctx = rkv.Context(1, s.n_q, s.n_kv, cap, self.small_hint)
        self.states = []
        for _ in range(s.n_layers):
            cache = synth.alloc_cache([cap], [0], s.n_kv, dev, fill=0.0)
            self.states.append(runner.LayerState(self.ctx, cache, [k_small], small_extra, s.n_q, s.n_kv))
        f32 = dict(dtype=torch.float32, device=dev)
        self.x, self.h = torch.zeros(s.hidden, **f32), torch.zeros(s.hidden, **f32)
        self.qkv = torch.zeros((s.n_q + 2 * s.n_kv) * 128, **f32)
        self.act = torch.zeros(s.ffn, **f32)
        self.logits = torch.zeros(s.vocab, **f32)
        self.q = torch.zeros((s.n_layers, 1, s.n_q, 128), dtype=torch.bfloat16, device=dev)
        self.k = torch.zeros((s.n_layers, 1, s.n_kv, 128), dtype=torch.bfloat16, device=dev)
        self.v = torch.zeros((s.n_layers, 1, s.n_kv, 128), dtype=torch.bfloat16, device=dev)
        self.token = torch.zeros((1,), dtype=torch.int32, device=dev)
        self.flag_total = torch.zeros((s.n_layers,), dtype=torch.int32, device=dev)
        self.capture = None                   # set to (set of layers, list) to record attention calls (tests)

    # ------------------------------------------------------------------ untimed set-up (torch, not measured)
    @torch.no_grad()
    def prefill(self, prompt: torch.Tensor) -> None:
        """Run the prompt through the model with torch matrix products, fill every layer's full cache, pick the
        first generated token and initialise every small cache from the last prompt token's attention scores."""
        s, L = self.s, self.prompt_len
        assert prompt.shape == (L,)
        F = torch.nn.functional
        x = self.embed_w[prompt.long()]                                          # [L, H] bf16
        half = 64
        inv = s.theta ** (-torch.arange(half, dtype=torch.float64, device=self.dev) / half)
        ang = torch.arange(L, dtype=torch.float64, device=self.dev)[:, None] * inv[None, :]
        cs, sn = torch.cos(ang).float()[:, None, :], torch.sin(ang).float()[:, None, :]   # [L, 1, 64]

        def rot(t):   # [L, heads, 128] fp32, rotate-half pairing
            a, b = t[..., :half], t[..., half:]
            return torch.cat([a * cs - b * sn, b * cs + a * sn], dim=-1)
        q_last = []
        for l, wl in enumerate(self.layers_w):
            h = F.rms_norm(x.float(), (s.hidden,), wl["norm1"].float(), eps=s.eps).to(torch.bfloat16)
            qkv = h @ wl["wqkv"].t()
            q = rot(qkv[:, : s.n_q * 128].float().view(L, s.n_q, 128)).to(torch.bfloat16)
            k = rot(qkv[:, s.n_q * 128: (s.n_q + s.n_kv) * 128].float().view(L, s.n_kv, 128)).to(torch.bfloat16)
            v = qkv[:, (s.n_q + s.n_kv) * 128:].view(L, s.n_kv, 128)
            cache = self.states[l].full
            cap = int(cache.cap[0])
            cache.k.view(s.n_kv, cap, 128)[:, :L] = k.transpose(0, 1)
            cache.v.view(s.n_kv, cap, 128)[:, :L] = v.transpose(0, 1)
            cache.len.fill_(L)
            att = F.scaled_dot_product_attention(q.transpose(0, 1)[None], k.transpose(0, 1)[None], v.transpose(0, 1)[None],
                                                 is_causal=True, enable_gqa=True)[0]            # [Hq, L, 128]
            x = x + att.transpose(0, 1).reshape(L, s.n_q * 128) @ wl["wo"].t()
            h = F.rms_norm(x.float(), (s.hidden,), wl["norm2"].float(), eps=s.eps).to(torch.bfloat16)
            for r0 in range(0, L, 8192):                                          # FFN in slabs of rows
                hs = h[r0: r0 + 8192]
                gu = hs @ wl["wgu"].t()
                x[r0: r0 + 8192] += (F.silu(gu[:, : s.ffn].float()) * gu[:, s.ffn:].float()).to(torch.bfloat16) @ wl["wd"].t()
            q_last.append(q[-1][None].contiguous())                                # [1, Hq, 128]
        hl = F.rms_norm(x[-1].float(), (s.hidden,), self.final_norm.float(), eps=s.eps)
        self.token.fill_(int(torch.argmax(hl @ self.lm_head.float().t()).item()))
        # small caches: top-K of the last prompt token's scores (a full step on its query; the output is not used)
        for l, st in enumerate(self.states):
            st.refresh(q_last[l], max_len_hint=self.full_hint)
        torch.cuda.synchronize()

    # ------------------------------------------------------------------ one decode token (measured path)
    def attention(self, l: int, kind: str):
        st, q, k, v = self.states[l], self.q[l], self.k[l], self.v[l]
        if kind == "check":
            st.check_trigger(q, self.threshold)
            st.append_partial(q, k, v, active=st.not_flag, max_len_hint=self.small_hint)
            st.refresh(q, active=st.flag, max_len_hint=self.full_hint)
            self.flag_total[l: l + 1].add_(st.flag)
        elif kind == "full":
            st.append(k, v)
            st.refresh(q, max_len_hint=self.full_hint)
        else:
            st.append_partial(q, k, v, max_len_hint=self.small_hint)
        if self.capture is not None and l in self.capture[0]:
            torch.cuda.synchronize()
            self.capture[1].append(dict(layer=l, kind=kind, q=q.clone(), out=st.out.clone(), flag=st.flag.clone(),
                                        small_len=int(st.small.len[0]), full_len=int(st.full.len[0]),
                                        small_k=st.small.k.clone(), small_v=st.small.v.clone(),
                                        small_cap=int(st.small.cap[0]), topk=st.topk_idx.clone()))
        return st.out

    def token_step(self, kind: str, with_harness: bool = True, with_attention: bool = True):
        """kind: 'small' (partial steps everywhere), 'check' (trigger decides per layer) or 'full'."""
        s = self.s
        if with_harness:
            embed(self.embed_w, self.token, self.x)
        for l, wl in enumerate(self.layers_w):
            if with_harness:
                gemv(wl["wqkv"], self.x, self.qkv, norm_w=wl["norm1"], eps=s.eps)        # RMSNorm fused into the read of x
                rope_split(self.qkv, self.states[l].full.len, s.theta, self.q[l], self.k[l], self.v[l], s.n_q, s.n_kv)
            out = self.attention(l, kind) if with_attention else self.states[l].out
            if with_harness:
                gemv(wl["wo"], out.view(-1), self.x, residual=self.x)
                gemv_swiglu(wl["wgu"], self.x, self.act, norm_w=wl["norm2"], eps=s.eps)
                gemv(wl["wd"], self.act, self.x, residual=self.x)
        if with_harness:
            gemv(self.lm_head, self.x, self.logits, norm_w=self.final_norm, eps=s.eps)
            argmax(self.logits, self.token)

    def kind_of(self, t: int) -> str:
        return "check" if t % self.qc == 0 else "small"


def llama8b() -> LlamaShape:
    return LlamaShape()


def weight_bytes(s: LlamaShape) -> int:
    """bf16 bytes one decode token streams: every layer's matrices and the output head (the embedding is one row)."""
    per = (s.n_q + 2 * s.n_kv) * 128 * s.hidden + s.hidden * s.n_q * 128 + 3 * s.ffn * s.hidden
    return 2 * (per * s.n_layers + s.vocab * s.hidden)
