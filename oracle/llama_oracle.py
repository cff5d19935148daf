"""fp64 CPU oracle for the decoder kernels around the attention calls of the end-to-end workload.

TEST INFRASTRUCTURE ONLY (see oracle/rkv_oracle.py): plain numpy float64 statements of the standard
Llama decoder pieces that the measuring harness runs between RefreshKV attention calls - the paper
(arXiv 2411.05787, Sec. 3 "Inference settings") applies its method inside off-the-shelf
Llama-3.1-8B / Qwen2-7B and defines none of these itself, so each function follows its textbook
definition.  Shares no code with the CUDA harness.  Pinned by tests/test_oracle_llama_pins.py.
"""
from __future__ import annotations

import numpy as np


def rmsnorm(x: np.ndarray, w: np.ndarray, eps: float) -> np.ndarray:
    """y_i = x_i / sqrt(mean_j x_j^2 + eps) * w_i."""
    x = np.asarray(x, dtype=np.float64)
    return x / np.sqrt(np.mean(x * x) + eps) * np.asarray(w, dtype=np.float64)


def gemv(w: np.ndarray, x: np.ndarray, residual: np.ndarray | None = None) -> np.ndarray:
    """y = W x (+ residual), W [out, in]."""
    y = np.asarray(w, dtype=np.float64) @ np.asarray(x, dtype=np.float64)
    return y if residual is None else y + np.asarray(residual, dtype=np.float64)


def silu(t: np.ndarray) -> np.ndarray:
    return t / (1.0 + np.exp(-t))


def swiglu_in(w_gate_up: np.ndarray, x: np.ndarray) -> np.ndarray:
    """silu(W_gate x) * (W_up x) with W = [W_gate ; W_up] stacked along the output axis."""
    n_ff = w_gate_up.shape[0] // 2
    g = gemv(w_gate_up[:n_ff], x)
    u = gemv(w_gate_up[n_ff:], x)
    return silu(g) * u


def rope(head: np.ndarray, pos: int, theta: float) -> np.ndarray:
    """Rotary embedding of one head vector [d] at position pos, rotate-half pairing:
    channel c (< d/2) is paired with c + d/2 and the pair is rotated by pos * theta^(-2c/d)."""
    head = np.asarray(head, dtype=np.float64)
    d = head.shape[-1]
    half = d // 2
    c = np.arange(half, dtype=np.float64)
    ang = float(pos) * theta ** (-c / half)
    cs, sn = np.cos(ang), np.sin(ang)
    a, b = head[..., :half], head[..., half:]
    return np.concatenate([a * cs - b * sn, b * cs + a * sn], axis=-1)


def rope_split(qkv: np.ndarray, pos: int, theta: float, n_q: int, n_kv: int, d: int = 128):
    """Split a fused projection [q heads | k heads | v heads] and rotate the q and k heads."""
    qkv = np.asarray(qkv, dtype=np.float64)
    q = qkv[: n_q * d].reshape(n_q, d)
    k = qkv[n_q * d: (n_q + n_kv) * d].reshape(n_kv, d)
    v = qkv[(n_q + n_kv) * d:].reshape(n_kv, d)
    return rope(q, pos, theta), rope(k, pos, theta), v.copy()


def argmax_first(logits: np.ndarray) -> int:
    """Index of the maximum; the lowest index among equal maxima."""
    return int(np.argmax(np.asarray(logits)))
