"""rkv_small_step_noalloc: the partial step for hosts that cannot allocate device memory.

Some programs that embed this library may not call cudaMalloc where attention runs (their own arena
owns the device heap, or an allocation's implicit synchronisation is not allowed on that path), so
they cannot create an rkv_ctx.  The context-free entry point keeps its scratch in a fixed array in
the library image instead.  This test calls it through the C ABI twice in a row - the second call
finds the array as the first one left it - and checks each result against rkv_small_step on the
same inputs and against the fp64 CPU oracle, with the tolerance of the other attention tests (the
context call merges its splits inside a thread-block cluster, the context-free one through the static
array, so the two reach the answer by different routes and their sums differ in order).  The second
call must also leave the amount of free device memory unchanged: the first call on a device may load
the library's device code, later ones take nothing.  Collected last, so a run that stops at the first
failure has already covered everything else.
"""
import numpy as np
import pytest
import torch

from oracle import rkv_oracle as O

pytestmark = pytest.mark.gpu

OUT_MAX_ABS = 2e-2
OUT_REL_L2 = 5e-3


def _close(a, b, what):
    a, b = a.float().cpu().numpy().astype(np.float64), b.float().cpu().numpy().astype(np.float64)
    err = np.abs(a - b).max()
    rel = np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30)
    assert err <= OUT_MAX_ABS and rel <= OUT_REL_L2, f"{what}: max-abs {err:.3e}, rel-L2 {rel:.3e}"


def _bits(t):
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def _oracle_out(q_b, cache, b, n, n_kv):
    off, cap = int(cache.row_offset[b]), int(cache.cap[b])
    k = O.bf16_bits_to_f64(_bits(cache.k[off: off + n_kv * cap]).reshape(n_kv, cap, 128)[:, :n])
    v = O.bf16_bits_to_f64(_bits(cache.v[off: off + n_kv * cap]).reshape(n_kv, cap, 128)[:, :n])
    return O.decode_attention(O.bf16_bits_to_f64(_bits(q_b)), k, v)[0]


def test_noalloc_small_step_matches_the_context_call_twice_in_a_row():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2411_05787_b200 import rkv, synth
    dev = torch.device("cuda")
    n_q, n_kv = 32, 8
    lens = [2058, 700, 1]                      # several CTAs per head, a ragged tail, a one-row cache
    caps = [n + 6 for n in lens]
    g = torch.Generator(device=dev); g.manual_seed(41)
    small = synth.alloc_cache(caps, lens, n_kv, dev)
    small.k.copy_(torch.randn(small.k.shape, generator=g, device=dev).to(torch.bfloat16))
    small.v.copy_(torch.randn(small.v.shape, generator=g, device=dev).to(torch.bfloat16))
    small_c = rkv.cache_struct(small.k, small.v, small.row_offset, small.cap, small.len)
    ctx = rkv.Context(len(lens), n_q, n_kv, max(caps), max(caps))
    cfg = rkv.RkvConfig(len(lens), n_q, n_kv, 128, max(caps), max(caps), 0, 1, 0.0)
    status = torch.zeros((1,), dtype=torch.int32, device=dev)
    active = torch.tensor([1, 1, 1], dtype=torch.int32, device=dev)
    for call in range(2):
        q = torch.randn((len(lens), n_q, 128), generator=g, device=dev).to(torch.bfloat16)
        want = torch.zeros((len(lens), n_q, 128), dtype=torch.bfloat16, device=dev)
        got = torch.full_like(want, 7.0)
        ctx.small_step(q, small_c, want)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        rkv.small_step_noalloc(cfg, q, small_c, got, active=active if call else None, device_status=status)
        torch.cuda.synchronize()
        free_after = torch.cuda.mem_get_info()[0]
        if call:          # the first call on a device may load the library's device code; later calls take nothing
            assert free_after == free_before, (free_before, free_after)
        assert ctx.device_status() == 0 and int(status.item()) == 0
        _close(got, want, f"call {call}")
        cur = small.len.tolist()
        for b in range(len(lens)):      # and against the definition itself, sequence by sequence
            ref = torch.from_numpy(_oracle_out(q[b], small, b, cur[b], n_kv))
            _close(got[b], ref, f"call {call} seq {b} vs oracle")
        # grow the caches between the calls, as decoding does
        ctx.append(torch.randn((len(lens), n_kv, 128), generator=g, device=dev).to(torch.bfloat16),
                   torch.randn((len(lens), n_kv, 128), generator=g, device=dev).to(torch.bfloat16), None, small_c)
    # sizes beyond the static scratch are refused with a reason, before anything is launched
    big = rkv.RkvConfig(rkv.NOALLOC_MAX_PROBLEMS // n_kv + 1, n_q, n_kv, 128, 64, 64, 0, 1, 0.0)
    with pytest.raises(rkv.RkvError, match="RKV_NOALLOC_MAX_PROBLEMS"):
        rkv.small_step_noalloc(big, q, small_c, got)
    long = rkv.RkvConfig(1, n_q, n_kv, 128, 64, rkv.NOALLOC_MAX_LEN + 1, 0, 1, 0.0)
    with pytest.raises(rkv.RkvError, match="RKV_NOALLOC_MAX_LEN"):
        rkv.small_step_noalloc(long, q, small_c, got)
