"""Pins of the decoder-piece oracle (oracle/llama_oracle.py): closed forms, invariants and an independent
library routine, chosen so that a dropped term, a wrong sign or a wrong pairing fails one of them."""
import math

import numpy as np
import torch

from oracle import llama_oracle as L


def _rng(seed):
    return np.random.default_rng(seed)


def test_rmsnorm_closed_forms():
    w = _rng(1).normal(size=64)
    # a constant vector c has rms |c|: the output is sign(c) * w (eps = 0)
    assert np.allclose(L.rmsnorm(np.full(64, -3.0), w, 0.0), -w, atol=1e-12)
    x = _rng(2).normal(size=64)
    y = L.rmsnorm(x, np.ones(64), 0.0)
    assert abs(np.mean(y * y) - 1.0) < 1e-12            # unit mean square
    assert np.allclose(L.rmsnorm(5.0 * x, w, 0.0), L.rmsnorm(x, w, 0.0))       # scale invariance
    # eps enters under the root, next to the MEAN of squares (not the sum)
    assert np.allclose(L.rmsnorm(x, w, 0.5), x / math.sqrt(np.mean(x * x) + 0.5) * w)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (64,), torch.from_numpy(w), eps=1e-5).numpy()
    assert np.allclose(L.rmsnorm(x, w, 1e-5), ref, atol=1e-12)


def test_gemv_and_swiglu():
    r = _rng(3)
    w, x, res = r.normal(size=(6, 8)), r.normal(size=8), r.normal(size=6)
    want = np.array([sum(w[o, i] * x[i] for i in range(8)) for o in range(6)])
    assert np.allclose(L.gemv(w, x), want, atol=1e-12)
    assert np.allclose(L.gemv(w, x, res), want + res, atol=1e-12)
    assert L.silu(np.array([0.0]))[0] == 0.0 and abs(L.silu(np.array([20.0]))[0] - 20.0) < 1e-7
    assert abs(L.silu(np.array([-1.0]))[0] + 1.0 / (1.0 + math.e)) < 1e-12
    wgu = r.normal(size=(10, 8))
    g, u = wgu[:5] @ x, wgu[5:] @ x
    assert np.allclose(L.swiglu_in(wgu, x), torch.nn.functional.silu(torch.from_numpy(g)).numpy() * u, atol=1e-12)
    # gate and up are not interchangeable
    assert not np.allclose(L.swiglu_in(wgu, x), L.swiglu_in(np.concatenate([wgu[5:], wgu[:5]]), x))


def test_rope_properties():
    r = _rng(4)
    q, k = r.normal(size=128), r.normal(size=128)
    theta = 500000.0
    assert np.allclose(L.rope(q, 0, theta), q)                                   # position 0 is the identity
    assert abs(np.linalg.norm(L.rope(q, 12345, theta)) - np.linalg.norm(q)) < 1e-9   # a rotation
    # the score depends on the distance only
    a = L.rope(q, 1000, theta) @ L.rope(k, 990, theta)
    b = L.rope(q, 25, theta) @ L.rope(k, 15, theta)
    assert abs(a - b) < 1e-9
    # pairing is (c, c + 64) and channel 0 turns by exactly pos radians
    e = np.zeros(128); e[0] = 1.0
    out = L.rope(e, 1, theta)
    assert abs(out[0] - math.cos(1.0)) < 1e-12 and abs(out[64] - math.sin(1.0)) < 1e-12 and abs(out[1]) < 1e-15
    # the slowest pair turns by pos * theta^(-63/64)
    e = np.zeros(128); e[63] = 1.0
    out = L.rope(e, 1000, theta)
    assert abs(out[63] - math.cos(1000 * theta ** (-63 / 64))) < 1e-12
    # composition: rotating by m then by n equals rotating by m + n
    assert np.allclose(L.rope(L.rope(q, 7, theta), 9, theta), L.rope(q, 16, theta), atol=1e-9)


def test_rope_split_layout_and_argmax():
    r = _rng(5)
    n_q, n_kv = 4, 2
    qkv = r.normal(size=(n_q + 2 * n_kv) * 128)
    q, k, v = L.rope_split(qkv, 3, 10000.0, n_q, n_kv)
    assert q.shape == (4, 128) and k.shape == (2, 128) and v.shape == (2, 128)
    assert np.allclose(q[1], L.rope(qkv[128:256], 3, 10000.0)) and np.allclose(k[0], L.rope(qkv[512:640], 3, 10000.0))
    assert np.array_equal(v.reshape(-1), qkv[768:])                               # values are not rotated
    assert L.argmax_first(np.array([1.0, 7.0, 7.0, -2.0])) == 1
