"""Parity of the CUDA library (through its C ABI) with the fp64 CPU oracle, element by element.

Tolerances (bf16 inputs, fp32 accumulation, bf16 output):
  out      max-abs <= 2e-2 and relative L2 <= 5e-3
  scores   relative 1e-4 + absolute 1e-9 against the oracle probabilities
  top-K    the set must equal the oracle's except inside the 1e-5 relative band around the K-th
           largest oracle score (oracle.check_topk_set); listed in ascending position order
  gather, append, flags   bit exact
"""
import math

import numpy as np
import pytest
import torch

from oracle import rkv_oracle as O

pytestmark = pytest.mark.gpu

OUT_MAX_ABS = 2e-2
OUT_REL_L2 = 5e-3


@pytest.fixture(scope="module")
def mods():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2411_05787_b200 import rkv, runner, synth
    return rkv, runner, synth


def bits(t):
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def check_out(got_bf16, want_f64, what=""):
    got = O.bf16_bits_to_f64(bits(got_bf16)).reshape(want_f64.shape)
    err = np.abs(got - want_f64).max()
    rel = np.linalg.norm(got - want_f64) / max(np.linalg.norm(want_f64), 1e-30)
    assert err <= OUT_MAX_ABS and rel <= OUT_REL_L2, f"{what}: max-abs {err:.3e}, rel-L2 {rel:.3e}"


def host_heads(cache, b, n_kv, which):
    off = int(cache.row_offset[b]); cap = int(cache.cap[b])
    t = cache.k if which == "k" else cache.v
    return bits(t[off: off + n_kv * cap]).reshape(n_kv, cap, 128)


def make_layer(mods, lens, k_small, n_q, n_kv, extra=8, seed=0, scale=1.0, agg=0, want_scores=True, poison=False,
               pool=1):
    rkv, runner, synth = mods
    dev = torch.device("cuda")
    caps = [l + extra for l in lens]
    cache = synth.alloc_cache(caps, lens, n_kv, dev)
    g = torch.Generator(device=dev); g.manual_seed(seed)
    cache.k.copy_((torch.randn(cache.k.shape, generator=g, device=dev) * scale).to(torch.bfloat16))
    cache.v.copy_((torch.randn(cache.v.shape, generator=g, device=dev)).to(torch.bfloat16))
    if poison:   # rows past each sequence's length hold NaN patterns: they must never leak into results
        for b, n in enumerate(lens):
            for h in range(n_kv):
                r0 = int(cache.row_offset[b]) + h * caps[b]
                cache.k[r0 + n: r0 + caps[b]] = float("nan")
                cache.v[r0 + n: r0 + caps[b]] = float("nan")
    ctx = rkv.Context(len(lens), n_q, n_kv, max(caps), max(max(k_small), 1) + extra, agg=agg, pool_kernel=pool)
    st = runner.LayerState(ctx, cache, k_small, extra, n_q, n_kv, want_scores=want_scores)
    q = (torch.randn((len(lens), n_q, 128), generator=g, device=dev)).to(torch.bfloat16)
    return ctx, st, cache, q


def oracle_full(cache, b, n, q_b, n_kv, k_small, agg="max", pool=1):
    k = O.bf16_bits_to_f64(host_heads(cache, b, n_kv, "k")[:, :n])
    v = O.bf16_bits_to_f64(host_heads(cache, b, n_kv, "v")[:, :n])
    return O.full_step(O.bf16_bits_to_f64(bits(q_b)), k, v, k_small, agg=agg, pool=pool)


def check_full_against_oracle(st, cache, q, lens, k_small, n_kv, agg="max", seqs=None, pool=1):
    idx_host = st.topk_idx.cpu().numpy()
    scores = st.scores.cpu().numpy() if st.scores is not None else None
    for b in (range(len(lens)) if seqs is None else seqs):
        n = lens[b]
        out, score, idx, _ = oracle_full(cache, b, n, q[b], n_kv, k_small[b], agg, pool)
        check_out(st.out[b], out, f"seq {b}")
        take = min(k_small[b], n)
        for g in range(n_kv):
            got = idx_host[b, g]
            assert (got[take:] == -1).all(), "padding must be -1"
            sel = got[:take]
            assert (np.diff(sel) > 0).all(), "indices must be strictly ascending"
            why = O.check_topk_set(score[g], k_small[b], sel)
            assert why is None, f"seq {b} head {g}: {why}"
            if scores is not None:
                assert np.allclose(scores[b, g, :n], score[g], rtol=1e-4, atol=1e-9), f"scores seq {b} head {g}"
    return True


CASES = [
    # lens, k_small, Hq, Hkv
    ([1], [1], 4, 1),
    ([15], [4], 8, 2),
    ([63, 64, 65], [16, 16, 70], 8, 2),
    ([1000], [100], 32, 8),
    ([777, 130, 2049], [64, 200, 256], 28, 4),      # G = 7, ragged, K > L for one sequence
    ([4096 + 37], [512], 8, 1),                    # G = 8, several chunks and a ragged tail
    ([300, 5], [0, 3], 6, 6),                      # G = 1, K = 0
]


@pytest.mark.parametrize("lens,k_small,n_q,n_kv", CASES)
def test_full_step_matches_oracle(mods, lens, k_small, n_q, n_kv):
    ctx, st, cache, q = make_layer(mods, lens, k_small, n_q, n_kv, seed=len(lens) * 131 + n_q, poison=True)
    st.refresh(q)
    assert ctx.device_status() == 0
    check_full_against_oracle(st, cache, q, lens, k_small, n_kv)
    # the rebuilt small cache holds exactly the selected rows, bit for bit
    idx_host = st.topk_idx.cpu().numpy()
    lens_small = st.small.len.cpu().numpy()
    for b, n in enumerate(lens):
        take = min(k_small[b], n)
        assert lens_small[b] == take
        for which in ("k", "v"):
            full_h = host_heads(cache, b, n_kv, which)
            small_h = host_heads(st.small, b, n_kv, which)
            for g in range(n_kv):
                assert np.array_equal(small_h[g, :take], full_h[g, idx_host[b, g, :take]])


@pytest.mark.parametrize("lens,k_small,n_q,n_kv", CASES)
def test_full_step_in_two_halves_matches_oracle(mods, lens, k_small, n_q, n_kv):
    """rkv_full_attention + rkv_select_topk (+ gather): the attention kernel finishes out itself, the selection
    works from the workspace.  Same checks as the one-call full step, and the same indices and scores as it."""
    rkv, runner, synth = mods
    ctx, st, cache, q = make_layer(mods, lens, k_small, n_q, n_kv, seed=len(lens) * 131 + n_q, poison=True)
    st.out.fill_(7.0)
    st.refresh_attention(q)
    torch.cuda.synchronize()
    for b, n in enumerate(lens):          # out is final before the selection has run
        want = oracle_full(cache, b, n, q[b], n_kv, k_small[b])[0]
        check_out(st.out[b], want, f"attention half, seq {b}")
    st.refresh_select(q)
    assert ctx.device_status() == 0
    check_full_against_oracle(st, cache, q, lens, k_small, n_kv)
    idx_two, scores_two = st.topk_idx.clone(), st.scores.clone()
    small_k = st.small.k.clone()
    st.refresh(q)
    assert torch.equal(idx_two, st.topk_idx) and torch.equal(scores_two, st.scores) and torch.equal(small_k, st.small.k)
    assert torch.equal(st.q_last_full, q)


@pytest.mark.parametrize("n_full", [0, 1, 63, 64, 1000, 2047, 2048, 4159])
def test_fused_append_full_attention_equals_append_then_attention(mods, n_full):
    """rkv_append_full_attention against rkv_append + rkv_full_attention on twin caches: same rows, lengths, flags,
    output bits, and - after rkv_select_topk - the same scores and indices; the active sequences also against the
    oracle.  The new row lands at tile and chunk boundaries, in an empty cache and (third step) in a full one."""
    rkv, runner, synth = mods
    dev = torch.device("cuda")
    n_q, n_kv, B, K = 28, 4, 3, 48
    lens, caps = [n_full, n_full // 2, 5], [n_full + 2, n_full // 2 + 3, 7]
    g = torch.Generator(device=dev); g.manual_seed(900 + n_full)
    fa = synth.alloc_cache(caps, lens, n_kv, dev)
    fb = synth.alloc_cache(caps, lens, n_kv, dev)
    for t in (fa.k, fa.v):
        t.copy_(torch.randn(t.shape, generator=g, device=dev).to(torch.bfloat16))
    fb.k.copy_(fa.k); fb.v.copy_(fa.v)
    ctx_a = rkv.Context(B, n_q, n_kv, max(caps), K + 4)
    ctx_b = rkv.Context(B, n_q, n_kv, max(caps), K + 4)
    cs = lambda c: rkv.cache_struct(c.k, c.v, c.row_offset, c.cap, c.len)
    sa, sb = cs(fa), cs(fb)
    k_small = torch.tensor([K, K, 3], dtype=torch.int32, device=dev)
    active = torch.tensor([1, 0, 1], dtype=torch.int32, device=dev)
    mk = lambda: (torch.zeros((B, n_q, 128), dtype=torch.bfloat16, device=dev),
                  torch.full((B, n_kv, K), -7, dtype=torch.int32, device=dev),
                  torch.zeros((B, n_kv, max(caps)), dtype=torch.float32, device=dev))
    for step in range(3):
        q = torch.randn((B, n_q, 128), generator=g, device=dev).to(torch.bfloat16)
        kn = torch.randn((B, n_kv, 128), generator=g, device=dev).to(torch.bfloat16)
        vn = torch.randn((B, n_kv, 128), generator=g, device=dev).to(torch.bfloat16)
        (out_a, idx_a, sc_a), (out_b, idx_b, sc_b) = mk(), mk()
        out_a.fill_(3.0); out_b.fill_(3.0)
        ctx_a.append_full_attention(q, kn, vn, sa, out_a, active=active)
        ctx_a.select_topk(None, sa, k_small, K, idx_a, active=active, scores=sc_a)
        bits_a = ctx_a.device_status()
        ctx_b.append(kn, vn, sb, None)
        ctx_b.full_attention(q, sb, out_b, active=active)
        ctx_b.select_topk(None, sb, k_small, K, idx_b, active=active, scores=sc_b)
        bits_b = ctx_b.device_status()
        assert bits_a == bits_b, (step, bits_a, bits_b)
        assert fa.len.tolist() == fb.len.tolist()
        assert torch.equal(fa.k, fb.k) and torch.equal(fa.v, fb.v)
        assert torch.equal(out_a, out_b) and torch.equal(idx_a, idx_b) and torch.equal(sc_a, sc_b), f"step {step}"
        assert (out_a[1] == 3.0).all() and (idx_a[1] == -7).all()   # inactive: untouched, but its cache grew
        for b in (0, 2):
            n = int(fa.len[b])
            want = oracle_full(fa, b, n, q[b], n_kv, int(k_small[b]))[0]
            check_out(out_a[b], want, f"fused full step {step} seq {b}")
    # three appends: sequence 0 had room for two, sequence 1 for three, sequence 2 for two
    assert fa.len.tolist() == [n_full + 2, n_full // 2 + 3, 7]


def test_select_topk_needs_its_attention_pass(mods):
    rkv, runner, synth = mods
    ctx, st, cache, q = make_layer(mods, [300], [16], 8, 2)
    with pytest.raises(rkv.RkvError):
        st.refresh_select(q)                          # nothing to complete
    st.refresh_attention(q)
    other = synth.alloc_cache([310], [300], 2, torch.device("cuda"))
    with pytest.raises(rkv.RkvError):                 # another cache than the attention pass read
        ctx.select_topk(q, rkv.cache_struct(other.k, other.v, other.row_offset, other.cap, other.len), st.k_small,
                        st.k_max, st.topk_idx)
    st.refresh_select(q)                              # the right one still works
    with pytest.raises(rkv.RkvError):
        st.refresh_select(q)                          # and is used up
    assert ctx.device_status() == 0


@pytest.mark.parametrize("lens,k_small,n_q,n_kv", [([5000, 3000], [256, 100], 32, 8), ([20000], [2048], 28, 4)])
def test_full_step_in_three_launches_matches_oracle(mods, lens, k_small, n_q, n_kv):
    """rkv_full_attention, rkv_score_keys, then rkv_select_topk for the selection alone (+ gather): same indices,
    scores and q_last_full as the one call, everything against the oracle; and the order of the calls is enforced."""
    rkv, runner, synth = mods
    ctx, st, cache, q = make_layer(mods, lens, k_small, n_q, n_kv, seed=41)
    with pytest.raises(rkv.RkvError):
        st.refresh_score_keys(q)                      # no attention pass to take the logits from
    st.refresh(q)
    one = (st.topk_idx.clone(), st.scores.clone(), st.small.k.clone(), st.q_last_full.clone())
    st.topk_idx.fill_(-7); st.scores.fill_(0.0); st.small.k.fill_(0.0); st.q_last_full.fill_(0.0)
    st.refresh_attention(q)
    st.refresh_score_keys(q)
    assert torch.equal(one[1], st.scores) and torch.equal(one[3], st.q_last_full)
    with pytest.raises(rkv.RkvError):                 # scores and q_last_full belong to the score pass
        ctx.select_topk(q, st.full_c, st.k_small, st.k_max, st.topk_idx, scores=st.scores)
    with pytest.raises(rkv.RkvError):                 # another k_max than the score pass was given
        ctx.select_topk(None, st.full_c, st.k_small, st.k_max - 1, st.topk_idx)
    st.refresh_select_only()
    assert torch.equal(one[0], st.topk_idx) and torch.equal(one[2], st.small.k)
    with pytest.raises(rkv.RkvError):
        st.refresh_select_only()                      # used up
    check_full_against_oracle(st, cache, q, lens, k_small, n_kv)
    # a score pass whose selection never ran leaves its histogram behind: the next full step must not see it
    st.refresh_attention(q)
    st.refresh_score_keys(q)
    st.refresh(q)
    assert torch.equal(one[0], st.topk_idx) and torch.equal(one[1], st.scores)
    assert ctx.device_status() == 0


@pytest.mark.parametrize("agg,name", [(1, "mean"), (2, "first")])
def test_aggregation_modes(mods, agg, name):
    lens, k_small = [500, 129], [50, 20]
    ctx, st, cache, q = make_layer(mods, lens, k_small, 16, 4, seed=5, agg=agg)
    st.refresh(q)
    check_full_against_oracle(st, cache, q, lens, k_small, 4, agg=name)


@pytest.mark.parametrize("pool,agg,name", [(7, 0, "max"), (3, 0, "max"), (7, 1, "mean"), (31, 0, "max")])
@pytest.mark.parametrize("lens,k_small,n_q,n_kv", [([1], [1], 4, 1), ([5, 64, 2049], [2, 16, 300], 28, 4),
                                                  ([4096 + 37], [512], 8, 1), ([1000, 33], [100, 40], 32, 8)])
def test_full_step_with_neighbour_max_pooling(mods, lens, k_small, n_q, n_kv, pool, agg, name):
    """Scores max-pooled over `pool` neighbouring positions before the top-K (the paper's kernel size is 7):
    windows clipped at both ends of the sequence and reaching across the slices of the selection cluster."""
    ctx, st, cache, q = make_layer(mods, lens, k_small, n_q, n_kv, seed=7 * pool + n_q, agg=agg, pool=pool, poison=True)
    st.refresh(q)
    assert ctx.device_status() == 0
    check_full_against_oracle(st, cache, q, lens, k_small, n_kv, agg=name, pool=pool)


@pytest.mark.parametrize("cluster", [1, 0])
def test_small_step_and_K_equals_L_invariant(mods, cluster):
    lens = [640, 200]
    ctx, st, cache, q = make_layer(mods, lens, list(lens), 8, 2, seed=9)
    ctx.set_option(mods[0].OPT_SMALL_CLUSTER, cluster)   # both ways of merging the splits
    full_out = st.refresh(q).clone()
    small_out = st.partial(q).clone()
    assert ctx.device_status() == 0
    # K = L: the small cache is the whole context, so both steps are the same attention
    for b, n in enumerate(lens):
        out, _, _, _ = oracle_full(cache, b, n, q[b], 2, n)
        check_out(small_out[b], out, "small step, K = L")
        check_out(full_out[b], out, "full step")


@pytest.mark.parametrize("cluster,n_q,n_kv", [(1, 32, 8), (0, 32, 8), (1, 28, 4), (1, 8, 1)])
def test_small_step_on_a_selected_subset(mods, cluster, n_q, n_kv):
    lens, k_small = [3000, 1111], [300, 64]
    ctx, st, cache, q = make_layer(mods, lens, k_small, n_q, n_kv, seed=10)
    ctx.set_option(mods[0].OPT_SMALL_CLUSTER, cluster)
    st.refresh(q)
    g = torch.Generator(device="cuda"); g.manual_seed(77)
    q2 = torch.randn(q.shape, generator=g, device="cuda").to(torch.bfloat16)
    small_out = st.partial(q2).clone()
    idx_host = st.topk_idx.cpu().numpy()
    for b, n in enumerate(lens):
        kf, vf = host_heads(cache, b, n_kv, "k"), host_heads(cache, b, n_kv, "v")
        sel = [idx_host[b, h, : k_small[b]] for h in range(n_kv)]
        ks = O.bf16_bits_to_f64(np.stack(O.gather_rows(kf, sel)))
        vs = O.bf16_bits_to_f64(np.stack(O.gather_rows(vf, sel)))
        out, _, _ = O.decode_attention(O.bf16_bits_to_f64(bits(q2[b])), ks, vs)
        check_out(small_out[b], out, f"small step seq {b}")


@pytest.mark.parametrize("n_small", [1, 64, 65, 130, 200, 321, 700])
def test_small_step_every_cluster_shape(mods, n_small):
    """Small caches from one tile to several per CTA: 1, 2, 4 and 8 CTAs per head, some of them idle."""
    lens = [n_small, max(1, n_small // 3)]
    ctx, st, cache, q = make_layer(mods, lens, list(lens), 28, 4, seed=100 + n_small, poison=True)
    st.refresh(q)
    out = st.partial(q).clone()
    assert ctx.device_status() == 0
    for b, n in enumerate(lens):
        want, _, _, _ = oracle_full(cache, b, n, q[b], 4, n)
        check_out(out[b], want, f"small step n={n}")


@pytest.mark.parametrize("n_small,n_q,n_kv", [(2560, 32, 8), (3073, 32, 8), (4096 + 9, 32, 8), (8000, 32, 8),
                                              (5000, 28, 4), (8180, 8, 1)])
def test_small_step_long_small_cache_one_sequence(mods, n_small, n_q, n_kv):
    """One sequence, few KV heads: the latency-bound form of the clustered step (one CTA per SM, groups of MMA warps
    on alternate tiles) with chunks longer than its ring, so every stage is used more than once; plain and with
    the append fused in, against the oracle."""
    rkv, runner, synth = mods
    ctx, st, cache, q = make_layer(mods, [n_small], [n_small], n_q, n_kv, seed=300 + n_small, poison=True)
    st.refresh(q)                                   # K = L: the small cache is the whole cache
    out = st.partial(q).clone()
    want, _, _, _ = oracle_full(cache, 0, n_small, q[0], n_kv, n_small)
    check_out(out[0], want, f"small step n={n_small}")
    g = torch.Generator(device=q.device); g.manual_seed(n_small)
    for step in range(2):
        q2 = torch.randn(q.shape, generator=g, device=q.device).to(torch.bfloat16)
        kn = torch.randn((1, n_kv, 128), generator=g, device=q.device).to(torch.bfloat16)
        vn = torch.randn((1, n_kv, 128), generator=g, device=q.device).to(torch.bfloat16)
        out2 = st.append_partial(q2, kn, vn).clone()
        n = int(st.small.len[0])
        assert n == n_small + step + 1
        k = O.bf16_bits_to_f64(host_heads(st.small, 0, n_kv, "k")[:, :n])
        v = O.bf16_bits_to_f64(host_heads(st.small, 0, n_kv, "v")[:, :n])
        want2, _, _ = O.decode_attention(O.bf16_bits_to_f64(bits(q2[0])), k, v)
        check_out(out2[0], want2, f"fused step {step} n={n}")
    assert ctx.device_status() == 0


@pytest.mark.parametrize("n_small", [0, 1, 63, 64, 127, 128, 320, 639, 640, 2047])
def test_fused_append_small_step_equals_append_then_small_step(mods, n_small):
    """rkv_append_small_step against the two separate calls on twin caches: same rows, lengths, flags, output.

    The new row lands at tile and chunk boundaries, in an empty cache, and (third step) in a full one."""
    rkv, runner, synth = mods
    dev = torch.device("cuda")
    n_q, n_kv, B = 28, 4, 3
    lens_s, caps_s = [n_small, n_small // 2, 5], [n_small + 3, n_small // 2 + 2, 9]
    lens_f, caps_f = [100, 40, 7], [102, 50, 9]
    g = torch.Generator(device=dev); g.manual_seed(500 + n_small)

    def twin():
        sm = synth.alloc_cache(caps_s, lens_s, n_kv, dev)
        fu = synth.alloc_cache(caps_f, lens_f, n_kv, dev)
        return sm, fu
    sm_a, fu_a = twin()
    for t in (sm_a.k, sm_a.v, fu_a.k, fu_a.v):
        t.copy_(torch.randn(t.shape, generator=g, device=dev).to(torch.bfloat16))
    sm_b, fu_b = twin()
    for x, y in ((sm_a, sm_b), (fu_a, fu_b)):
        y.k.copy_(x.k); y.v.copy_(x.v)
    ctx = rkv.Context(B, n_q, n_kv, max(caps_f), max(caps_s))
    cs = lambda c: rkv.cache_struct(c.k, c.v, c.row_offset, c.cap, c.len)
    sa, fa, sb, fb = cs(sm_a), cs(fu_a), cs(sm_b), cs(fu_b)
    out_a = torch.zeros((B, n_q, 128), dtype=torch.bfloat16, device=dev)
    out_b = torch.zeros_like(out_a)
    active = torch.tensor([1, 0, 1], dtype=torch.int32, device=dev)
    for step in range(3):
        q = torch.randn((B, n_q, 128), generator=g, device=dev).to(torch.bfloat16)
        kn = torch.randn((B, n_kv, 128), generator=g, device=dev).to(torch.bfloat16)
        vn = torch.randn((B, n_kv, 128), generator=g, device=dev).to(torch.bfloat16)
        out_a.fill_(3.0); out_b.fill_(3.0)
        ctx.append_small_step(q, kn, vn, fa, sa, out_a, active=active)
        bits_a = ctx.device_status()
        ctx.append(kn, vn, fb, sb)
        ctx.small_step(q, sb, out_b, active=active)
        bits_b = ctx.device_status()
        assert bits_a == bits_b, (step, bits_a, bits_b)
        assert sm_a.len.tolist() == sm_b.len.tolist() and fu_a.len.tolist() == fu_b.len.tolist()
        for x, y in ((sm_a, sm_b), (fu_a, fu_b)):
            assert torch.equal(x.k, y.k) and torch.equal(x.v, y.v)
        assert torch.equal(out_a, out_b), f"step {step}"
        assert (out_a[1] == 3.0).all()      # inactive sequence: output untouched, but its caches grew
        # and against the oracle, on the bytes now in the cache
        for b in (0, 2):
            n = int(sm_a.len[b])
            k = O.bf16_bits_to_f64(host_heads(sm_a, b, n_kv, "k")[:, :n])
            v = O.bf16_bits_to_f64(host_heads(sm_a, b, n_kv, "v")[:, :n])
            want, _, _ = O.decode_attention(O.bf16_bits_to_f64(bits(q[b])), k, v)
            check_out(out_a[b], want, f"fused step {step} seq {b}")
    # the third step found sequence 0's full cache and sequence 2's caches at capacity
    assert fu_a.len.tolist() == [102, 43, 9] and sm_a.len.tolist() == [n_small + 3, n_small // 2 + 2, 8]


def test_early_cache_read_changes_nothing(mods):
    """The clustered partial step may request its cache rows before its stream dependency has resolved when the
    launch before it wrote none of them.  A mix of calls where that is allowed (another cache's step before it)
    and where it is not (the same cache's step, an append, a gather directly before it) must give the same bits as
    the same calls with the option off, and match the oracle."""
    rkv, runner, synth = mods
    dev = torch.device("cuda")
    n_q, n_kv, B, n0 = 32, 8, 1, 700
    g = torch.Generator(device=dev); g.manual_seed(77)

    def make(n_caches):
        out = []
        for _ in range(n_caches):
            c = synth.alloc_cache([n0 + 40], [n0], n_kv, dev)
            out.append(c)
        return out
    on, off = make(3), make(3)
    for x, y in zip(on, off):
        x.k.copy_(torch.randn(x.k.shape, generator=g, device=dev).to(torch.bfloat16))
        x.v.copy_(torch.randn(x.v.shape, generator=g, device=dev).to(torch.bfloat16))
        y.k.copy_(x.k); y.v.copy_(x.v)
    ctx_on = rkv.Context(B, n_q, n_kv, n0 + 40, n0 + 40)
    ctx_off = rkv.Context(B, n_q, n_kv, n0 + 40, n0 + 40)
    ctx_off.set_option(rkv.OPT_EARLY_CACHE_READ, 0)
    cs = lambda c: rkv.cache_struct(c.k, c.v, c.row_offset, c.cap, c.len)
    order = [0, 1, 2, 0, 0, 1, 1, 2, 0, 2, 2, 1]          # neighbours equal: the predecessor wrote the same cache
    outs = {}
    for name, ctx, caches in (("on", ctx_on, on), ("off", ctx_off, off)):
        gg = torch.Generator(device=dev); gg.manual_seed(78)
        structs = [cs(c) for c in caches]
        res = []
        ins = [(torch.randn((B, n_q, 128), generator=gg, device=dev).to(torch.bfloat16),
                torch.randn((B, n_kv, 128), generator=gg, device=dev).to(torch.bfloat16),
                torch.randn((B, n_kv, 128), generator=gg, device=dev).to(torch.bfloat16),
                torch.zeros((B, n_q, 128), dtype=torch.bfloat16, device=dev)) for _ in order]
        torch.cuda.synchronize()
        for step, i in enumerate(order):                   # nothing but the library's launches in the stream
            q, kn, vn, o = ins[step]
            if step % 5 == 4:                              # a plain append, then the step on the cache just written
                ctx.append(kn, vn, None, structs[i])
                ctx.small_step(q, structs[i], o)
            else:
                ctx.append_small_step(q, kn, vn, None, structs[i], o)
            res.append((i, q, o))
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        outs[name] = res
    for (i, q, a), (_, _, b) in zip(outs["on"], outs["off"]):
        assert torch.equal(a, b)
    for x, y in zip(on, off):
        assert torch.equal(x.k, y.k) and torch.equal(x.v, y.v) and x.len.tolist() == y.len.tolist()
    # the last step on every cache against the oracle, on the bytes now in the cache
    seen = set()
    for i, q, o in reversed(outs["on"]):
        if i in seen:
            continue
        seen.add(i)
        n = int(on[i].len[0])
        k = O.bf16_bits_to_f64(host_heads(on[i], 0, n_kv, "k")[:, :n])
        v = O.bf16_bits_to_f64(host_heads(on[i], 0, n_kv, "v")[:, :n])
        want, _, _ = O.decode_attention(O.bf16_bits_to_f64(bits(q[0])), k, v)
        check_out(o[0], want, f"cache {i}")


@pytest.mark.parametrize("lens,k_small,n_q,n_kv", [([3000, 70], [300, 64], 32, 8), ([4096 + 37, 1], [512, 1], 28, 4)])
def test_score_only_refresh_step(mods, lens, k_small, n_q, n_kv):
    """rkv_score_step (K only) selects exactly what rkv_full_step selects; followed by the rebuild and a partial
    step it gives the oracle's "w/o full attention" output."""
    ctx, st, cache, q = make_layer(mods, lens, k_small, n_q, n_kv, seed=21, poison=True)
    st.refresh(q)
    idx_full, sc_full = st.topk_idx.clone(), st.scores.clone()
    st.topk_idx.fill_(-9); st.scores.fill_(-1.0); st.out.fill_(5.0); st.q_last_full.fill_(0.0)
    out = st.refresh_scores_only(q).clone()
    assert ctx.device_status() == 0
    assert torch.equal(st.topk_idx, idx_full) and torch.equal(st.q_last_full, q)
    for b, n in enumerate(lens):
        assert torch.equal(st.scores[b, :, :n], sc_full[b, :, :n])
        k = O.bf16_bits_to_f64(host_heads(cache, b, n_kv, "k")[:, :n])
        v = O.bf16_bits_to_f64(host_heads(cache, b, n_kv, "v")[:, :n])
        # the oracle's output on the GPU's own (validated) selection, so that ties cannot differ
        want_out, score, _ = O.score_only_step(O.bf16_bits_to_f64(bits(q[b])), k, v, k_small[b])
        take = min(k_small[b], n)
        sel = [st.topk_idx[b, g, :take].cpu().numpy().astype(np.int64) for g in range(n_kv)]
        for g in range(n_kv):
            assert O.check_topk_set(score[g], k_small[b], sel[g]) is None
        ks = np.stack([k[g, sel[g]] for g in range(n_kv)]); vs = np.stack([v[g, sel[g]] for g in range(n_kv)])
        want, _, _ = O.decode_attention(O.bf16_bits_to_f64(bits(q[b])), ks, vs)
        check_out(out[b], want, f"score-only step seq {b}")


def test_append_and_overflow_flag(mods):
    rkv, runner, synth = mods
    lens, k_small = [40, 9], [8, 4]
    ctx, st, cache, q = make_layer(mods, lens, k_small, 8, 2, extra=2, seed=11)
    st.refresh(q)
    g = torch.Generator(device="cuda"); g.manual_seed(3)
    before_k = cache.k.clone()
    rows = []
    for t in range(2):
        kn = torch.randn((2, 2, 128), generator=g, device="cuda").to(torch.bfloat16)
        vn = torch.randn((2, 2, 128), generator=g, device="cuda").to(torch.bfloat16)
        st.append(kn, vn)
        rows.append((kn, vn))
    assert ctx.device_status() == 0
    assert cache.len.tolist() == [42, 11] and st.small.len.tolist() == [10, 6]
    for b in range(2):
        fk, fv = host_heads(cache, b, 2, "k"), host_heads(cache, b, 2, "v")
        sk = host_heads(st.small, b, 2, "k")
        for t, (kn, vn) in enumerate(rows):
            assert np.array_equal(fk[:, lens[b] + t], bits(kn[b]))
            assert np.array_equal(fv[:, lens[b] + t], bits(vn[b]))
            assert np.array_equal(sk[:, k_small[b] + t], bits(kn[b]))
    # nothing but the appended rows changed
    changed = (cache.k != before_k).any(dim=1).sum().item()
    assert changed <= 2 * 2 * 2
    # a third append exceeds both capacities: flagged, lengths unchanged, nothing written
    snap = cache.k.clone()
    st.append(rows[0][0], rows[0][1])
    assert ctx.device_status() & rkv.DEV_APPEND_OVERFLOW
    assert cache.len.tolist() == [42, 11] and torch.equal(cache.k, snap)


def test_trigger_flags_and_similarity(mods):
    rkv, runner, synth = mods
    n_seq, n_q = 64, 28
    ctx = rkv.Context(n_seq, n_q, 4, 256, 64)
    g = torch.Generator(device="cuda"); g.manual_seed(12)
    last = torch.randn((n_seq, n_q, 128), generator=g, device="cuda").to(torch.bfloat16)
    mix = torch.linspace(0.0, 1.0, n_seq, device="cuda")[:, None, None]
    now = (mix * last.float() + (1 - mix) * torch.randn(last.shape, generator=g, device="cuda")).to(torch.bfloat16)
    now[3] = 0          # zero mean query -> NaN similarity -> refresh
    now[5] = last[5]    # identical -> similarity 1
    flag = torch.full((n_seq,), -7, dtype=torch.int32, device="cuda")
    sim = torch.zeros((n_seq,), dtype=torch.float32, device="cuda")
    thr = 0.9
    keep = torch.full((n_seq,), -7, dtype=torch.int32, device="cuda")
    ctx.should_refresh(now, last, thr, flag, sim, keep=keep)
    assert torch.equal(keep, 1 - flag)
    flag_h, sim_h = flag.cpu().numpy(), sim.cpu().numpy()
    near = 0
    for b in range(n_seq):
        want_flag, cos = O.should_refresh(O.bf16_bits_to_f64(bits(now[b])), O.bf16_bits_to_f64(bits(last[b])), thr)
        if not math.isnan(cos):
            assert abs(sim_h[b] - cos) < 1e-5
            if abs(cos - thr) < 1e-4:
                near += 1
                continue
        assert flag_h[b] == want_flag, (b, cos)
    assert flag_h[3] == 1 and flag_h[5] == 0 and near <= 2
    # equality is not "higher": threshold 1.0 against an identical query refreshes
    ctx.should_refresh(last, last, 1.0000001, flag)
    assert flag.cpu().numpy().all()


def test_active_mask_leaves_inactive_sequences_untouched(mods):
    lens, k_small = [500, 400, 300], [32, 32, 32]
    ctx, st, cache, q = make_layer(mods, lens, k_small, 8, 2, seed=13)
    st.out.fill_(7.0); st.topk_idx.fill_(-5); st.scores.fill_(-3.0); st.q_last_full.fill_(9.0)
    st.small.len.fill_(0)
    active = torch.tensor([1, 0, 1], dtype=torch.int32, device="cuda")
    st.refresh(q, active=active)
    assert ctx.device_status() == 0
    assert (st.out[1] == 7.0).all() and (st.topk_idx[1] == -5).all() and (st.scores[1] == -3.0).all()
    assert (st.q_last_full[1] == 9.0).all() and st.small.len.tolist() == [32, 0, 32]
    assert torch.equal(st.q_last_full[0], q[0]) and torch.equal(st.q_last_full[2], q[2])
    check_full_against_oracle(st, cache, q, lens, k_small, 2, seqs=[0, 2])
    st.out.fill_(7.0)
    st.partial(q, active=torch.tensor([0, 0, 1], dtype=torch.int32, device="cuda"))
    assert (st.out[0] == 7.0).all() and (st.out[1] == 7.0).all() and not (st.out[2] == 7.0).all()


def test_ties_go_to_the_lower_position(mods):
    """Identical keys give identical scores: the K lowest positions must be chosen."""
    rkv, runner, synth = mods
    lens, k_small = [900], [37]
    ctx, st, cache, q = make_layer(mods, lens, k_small, 4, 1, seed=14)
    cache.k[:] = cache.k[0:1]          # every key row identical
    st.refresh(q)
    assert st.topk_idx[0, 0, :37].tolist() == list(range(37))
    # two distinct key values: the larger-score class first (all of it), then the lowest positions of the other
    cache.k[:] = 0
    hot = [5, 400, 899]
    cache.k[hot] = (q[0].float().mean(dim=0) * 0.5).to(torch.bfloat16)
    st.refresh(q)
    got = st.topk_idx[0, 0, :37].tolist()
    assert got == sorted(hot + [i for i in range(40) if i not in hot][:34])


def test_many_near_equal_scores_take_the_refinement_path(mods):
    """Thousands of distinct scores inside one histogram bin (keys that differ by a small perturbation): the
    selection has to narrow the bin down with its finer histograms before it can resolve the threshold."""
    rkv, runner, synth = mods
    for lens, k_small, n_q, n_kv in (([3000], [700], 4, 1), ([9000, 5000], [1500, 4000], 8, 2), ([40000], [9000], 4, 1)):
        ctx, st, cache, q = make_layer(mods, lens, k_small, n_q, n_kv, seed=23 + len(lens))
        g = torch.Generator(device="cuda"); g.manual_seed(77)
        base = torch.randn((1, 128), generator=g, device="cuda")
        cache.k.copy_((base + 0.004 * torch.randn(cache.k.shape, generator=g, device="cuda")).to(torch.bfloat16))
        st.refresh(q)
        assert ctx.device_status() == 0
        check_full_against_oracle(st, cache, q, lens, k_small, n_kv)
        a = st.topk_idx.clone()
        st.refresh(q)                       # the histogram was left clean: the same answer again
        assert torch.equal(a, st.topk_idx)


@pytest.mark.parametrize("scale,k_small", [(30.0, [600, 40]), (1.0, [3990, 1495]), (30.0, [3990, 1495]), (0.0, [100, 7])])
def test_threshold_outside_the_histogram_window(mods, scale, k_small):
    """The selection's fine histogram covers a window of 32 nats placed below the log-sum-exp.  Logits of very
    large spread put the K-th score below the window (first bin), a K close to the length puts it above (last,
    open-ended bin), all-zero keys put every score into one bin: each time the finer passes must take over."""
    lens = [4000, 1500]
    ctx, st, cache, q = make_layer(mods, lens, k_small, 16, 4, seed=61, scale=scale)
    st.refresh(q)
    assert ctx.device_status() == 0
    check_full_against_oracle(st, cache, q, lens, k_small, 4)


def test_gather_flags_indices_outside_the_cache(mods):
    """rkv_gather_small: -1 is padding and is skipped silently; any other index outside [0, len) is skipped
    and raises RKV_DEV_BAD_INDEX; the rows of valid indices are still copied."""
    rkv, runner, synth = mods
    lens, k_small = [200], [8]
    ctx, st, cache, q = make_layer(mods, lens, k_small, 4, 2, seed=31)
    for bad in (200, 10 ** 6, -2, -(2 ** 31)):
        idx = torch.tensor([[[3, 5, bad, 9, 11, -1, 20, 21], [0, 1, 2, 3, 4, 5, 6, 7]]], dtype=torch.int32, device="cuda")
        st.small.k.fill_(0.0); st.small.v.fill_(0.0)
        ctx.gather_small(idx, st.k_small, 8, st.full_c, st.small_c)
        assert ctx.device_status() == rkv.DEV_BAD_INDEX, bad
        fk, sk = host_heads(cache, 0, 2, "k"), host_heads(st.small, 0, 2, "k")
        for r, j in enumerate([3, 5, None, 9, 11, None, 20, 21]):
            if j is None:
                assert not sk[0, r].any()
            else:
                assert np.array_equal(sk[0, r], fk[0, j])
        assert np.array_equal(sk[1, :8], fk[1, :8])
    idx = torch.tensor([[[3, 5, -1, 9, 11, -1, 20, 21], [0, 1, 2, 3, 4, 5, 6, 7]]], dtype=torch.int32, device="cuda")
    ctx.gather_small(idx, st.k_small, 8, st.full_c, st.small_c)
    assert ctx.device_status() == 0


def test_gather_tiles_with_and_without_skipped_rows(mods):
    """rkv_gather_small moves 64 output rows per CTA: whole tiles leave with one bulk store per cache, a tile with
    a skipped row (padding or a flagged index) row by row, the last tile is ragged, rows at and beyond
    min(k_small, len) stay untouched, inactive sequences too; both sequences and both heads bit for bit."""
    rkv, runner, synth = mods
    lens, k_small = [5000, 700], [200, 150]
    ctx, st, cache, q = make_layer(mods, lens, k_small, 4, 2, seed=33)
    g = torch.Generator().manual_seed(5)
    k_max = 200
    idx = torch.full((2, 2, k_max), -1, dtype=torch.int32)
    for b in range(2):
        for h in range(2):
            idx[b, h, : k_small[b]] = torch.randperm(lens[b], generator=g)[: k_small[b]].to(torch.int32)
    idx[0, 0, 70] = 5000          # flagged, tile 1 of (0, 0)
    idx[0, 1, 130] = -1           # padding inside the range, tile 2 of (0, 1)
    idx[1, 0, 149] = 10 ** 6      # flagged, in the ragged last tile of (1, 0)
    idx = idx.cuda()
    for active in (None, torch.tensor([1, 0], dtype=torch.int32, device="cuda")):
        st.small.k.fill_(7.0); st.small.v.fill_(7.0); st.small.len.fill_(0)
        ctx.gather_small(idx, st.k_small, k_max, st.full_c, st.small_c, active=active)
        assert ctx.device_status() == rkv.DEV_BAD_INDEX
        host_idx = idx.cpu().numpy()
        for b in range(2):
            fk, fv = host_heads(cache, b, 2, "k"), host_heads(cache, b, 2, "v")
            sk, sv = host_heads(st.small, b, 2, "k"), host_heads(st.small, b, 2, "v")
            on = active is None or int(active[b]) == 1
            assert int(st.small.len[b]) == (k_small[b] if on else 0)
            seven = bits(torch.tensor([7.0], dtype=torch.bfloat16))[0]
            for h in range(2):
                for r in range(st.small.cap[b].item()):
                    j = host_idx[b, h, r] if r < k_small[b] else -1
                    if on and 0 <= j < lens[b]:
                        assert np.array_equal(sk[h, r], fk[h, j]) and np.array_equal(sv[h, r], fv[h, j]), (b, h, r)
                    else:
                        assert (sk[h, r] == seven).all() and (sv[h, r] == seven).all(), (b, h, r)


def test_deterministic_bits(mods):
    lens, k_small = [5000, 3000], [256, 100]
    ctx, st, cache, q = make_layer(mods, lens, k_small, 32, 8, seed=15)
    st.refresh(q)
    a = (st.out.clone(), st.topk_idx.clone(), st.scores.clone(), st.small.k.clone())
    for _ in range(3):
        st.refresh(q)
        assert torch.equal(a[0], st.out) and torch.equal(a[1], st.topk_idx)
        assert torch.equal(a[2], st.scores) and torch.equal(a[3], st.small.k)


def test_launch_shape_options_change_nothing(mods):
    """RKV_OPT_SCORE_SLICE and RKV_OPT_SELECT_KEYS_PER_CTA only change how the score pass and the top-K are cut
    into CTAs: scores, indices and the rebuilt small cache keep their bits, the output agrees with the oracle, and
    rkv_get_option returns what was set."""
    rkv, runner, synth = mods
    lens, k_small = [20000, 7001], [2048, 300]
    ctx, st, cache, q = make_layer(mods, lens, k_small, 16, 4, seed=23)
    assert ctx.get_option(rkv.OPT_SCORE_SLICE) == 0 and ctx.get_option(rkv.OPT_SELECT_KEYS_PER_CTA) == 4096
    st.refresh(q)
    check_full_against_oracle(st, cache, q, lens, k_small, 4)
    a = (st.out.clone(), st.topk_idx.clone(), st.scores.clone(), st.small.k.clone(), st.small.v.clone())
    for slice_, per_cta in ((1024, 512), (2048, 16384), (4096, 40960), (8192, 4096), (0, 8192)):
        ctx.set_option(rkv.OPT_SCORE_SLICE, slice_)
        ctx.set_option(rkv.OPT_SELECT_KEYS_PER_CTA, per_cta)
        assert ctx.get_option(rkv.OPT_SCORE_SLICE) == slice_ and ctx.get_option(rkv.OPT_SELECT_KEYS_PER_CTA) == per_cta
        st.small.k.fill_(0.0); st.small.v.fill_(0.0)
        st.refresh(q)
        assert torch.equal(a[0], st.out) and torch.equal(a[1], st.topk_idx), (slice_, per_cta)
        assert torch.equal(a[2], st.scores) and torch.equal(a[3], st.small.k) and torch.equal(a[4], st.small.v)
    with pytest.raises(rkv.RkvError):
        ctx.set_option(rkv.OPT_SCORE_SLICE, 3000)
    with pytest.raises(rkv.RkvError):
        ctx.get_option(99)
    assert ctx.device_status() == 0


def test_length_above_hint_is_clamped_and_flagged(mods):
    rkv, runner, synth = mods
    lens, k_small = [600], [16]
    ctx, st, cache, q = make_layer(mods, lens, k_small, 8, 2, seed=16)
    st.refresh(q, max_len_hint=512)
    assert ctx.device_status() & rkv.DEV_LEN_CLAMPED
    assert int(st.topk_idx.max()) < 512


def test_host_side_argument_errors(mods):
    rkv, runner, synth = mods
    ctx, st, cache, q = make_layer(mods, [100], [8], 8, 2, seed=17)
    with pytest.raises(rkv.RkvError):
        ctx.full_step(q, st.full_c, st.k_small, 10 ** 6, st.out, st.topk_idx)           # k_max too large
    with pytest.raises(rkv.RkvError):
        ctx.full_step(q, st.full_c, st.k_small, st.k_max, st.out, st.topk_idx, max_len_hint=10 ** 7)
    with pytest.raises(rkv.RkvError):
        rkv.Context(1, 8, 2, 100, 10, pool_kernel=4)
    with pytest.raises(rkv.RkvError):
        rkv.Context(1, 8, 2, 100, 10, pool_kernel=33)
    with pytest.raises(rkv.RkvError):
        rkv.Context(1, 8, 2, 8 * 40960 + 1, 10, pool_kernel=7)   # the length limit, with or without pooling
    # bf16 tensors start on a 16-byte boundary: a query (or output) view that begins 2 bytes in is refused
    skew = torch.zeros(q.numel() + 8, dtype=torch.bfloat16, device=q.device)
    q_off = skew[1: 1 + q.numel()].view_as(q)
    out_off = skew[1: 1 + st.out.numel()].view_as(st.out)
    with pytest.raises(rkv.RkvError):
        ctx.full_step(q_off, st.full_c, st.k_small, st.k_max, st.out, st.topk_idx)
    with pytest.raises(rkv.RkvError):
        ctx.small_step(q, st.small_c, out_off)
    st.refresh(q)                                            # the context is still usable
    assert ctx.device_status() == 0


# ----------------------------------------------------------------------------- the five workload configs
NEAR_THRESHOLD = {"checks": 0, "excluded": 0}      # flag comparisons made / left out because |cos - s| < 1e-4


def run_trajectory(mods, w, layer, seqs=None, check_every=1, fused=False, evict=0, overlapped=False, deferred=False):
    """Run workload `w` for one layer on the GPU and step the oracle beside it on the same bytes.

    overlapped: full-step and check tokens go through runner.OverlappedRefresh (attention in the calling stream,
    selection and rebuild behind it in a second one), the way bench.py launches them."""
    rkv, runner, synth = mods
    dev = torch.device("cuda")
    cache = synth.fill_layer(w, layer, dev)
    qs = synth.query_trajectory(w, layer).to(dev)
    kn, vn = synth.new_token_kv(w, layer)
    kn, vn = kn.to(dev), vn.to(dev)
    restore = synth.plant_heavy(w, cache, layer, qs[0], epoch=0)
    max_len = max(w.lens) + w.steps + 1
    ctx = rkv.Context(w.batch, w.n_q_heads, w.n_kv_heads, max_len, max(w.k_small) + w.steps + 1)
    st = runner.LayerState(ctx, cache, list(w.k_small), w.steps + 1, w.n_q_heads, w.n_kv_heads, want_scores=False)
    if evict:       # fixed-size small cache: new tokens replace the lowest-scoring survivors
        st.enable_eviction(evict)
        st.refresh, st.append_partial = st.refresh_evict, st.append_partial_evict
        fused = True
    ov = runner.OverlappedRefresh([st]) if overlapped else (runner.DeferredRefresh([st]) if deferred else None)
    seqs = list(range(w.batch)) if seqs is None else seqs
    checks = excluded = 0
    # oracle state per checked sequence, on copies of the same bytes
    states = {}
    for b in seqs:
        states[b] = O.SequenceState(host_heads(cache, b, w.n_kv_heads, "k").copy(),
                                    host_heads(cache, b, w.n_kv_heads, "v").copy(), w.lens[b], w.k_small[b],
                                    evict=bool(evict))
    st.refresh(qs[0])
    for b in seqs:
        o_out, o_score, o_idx = states[b].full(bits(qs[0, b]))
        check_out(st.out[b], o_out, f"init seq {b}")
        follow_gpu_selection(st, states[b], b, o_score, w)
    n_full = {b: 0 for b in seqs}
    for t in range(1, w.steps + 1):
        if w.replant_every and t % w.replant_every == 0:
            synth.unplant(cache, restore)
            restore = synth.plant_heavy(w, cache, layer, qs[t], epoch=t // w.replant_every)
            for b in seqs:      # the oracle's copy of C_f follows the replanted rows
                states[b].k_full[:, : w.lens[b]] = host_heads(cache, b, w.n_kv_heads, "k")[:, : w.lens[b]]
        for b in seqs:
            states[b].append(bits(kn[t, b]), bits(vn[t, b]))
        if w.schedule == "fixed":
            full_now = [O.fixed_stride_is_full(t, w.stride)] * w.batch
            if full_now[0] and ov is not None:
                ov.run(lambda l: qs[t], lambda l: kn[t], lambda l: vn[t])
            elif full_now[0]:
                st.append(kn[t], vn[t])
                st.refresh(qs[t])
            elif fused:
                st.append_partial(qs[t], kn[t], vn[t])
            else:
                st.append(kn[t], vn[t])
                st.partial(qs[t])
        else:
            full_now = [False] * w.batch
            if t % w.stride == 0:
                if ov is not None:      # trigger, both branches under its masks, selection in the second stream
                    ov.run_checked(lambda l: qs[t], lambda l: kn[t], lambda l: vn[t], w.threshold)
                    torch.cuda.synchronize()
                    flags = st.flag.cpu().numpy()
                else:
                    st.check_trigger(qs[t], w.threshold)
                    flags = st.flag.cpu().numpy()
                    if fused:      # appends for every sequence, attends for those that keep the partial cache
                        st.append_partial(qs[t], kn[t], vn[t], active=st.not_flag)
                        st.refresh(qs[t], active=st.flag)
                    else:
                        st.append(kn[t], vn[t])
                        st.refresh(qs[t], active=st.flag)
                        st.partial(qs[t], active=st.not_flag)
                assert torch.equal(st.not_flag, 1 - st.flag)      # the trigger wrote both masks
                full_now = [bool(f) for f in flags]
                for b in seqs:
                    want, cos = O.should_refresh(O.bf16_bits_to_f64(bits(qs[t, b])), states[b].q_last_full, w.threshold)
                    checks += 1
                    if abs(cos - w.threshold) >= 1e-4:
                        assert flags[b] == want, (t, b, cos)
                    else:       # too close to the threshold for fp32 against fp64: counted, and bounded below
                        excluded += 1
                    full_now[b] = bool(flags[b])
            elif fused:
                st.append_partial(qs[t], kn[t], vn[t])
            else:
                st.append(kn[t], vn[t])
                st.partial(qs[t])
        for b in seqs:
            if full_now[b]:
                o_out, o_score, o_idx = states[b].full(bits(qs[t, b]))
                n_full[b] += 1
                check_out(st.out[b], o_out, f"full step t={t} seq {b}")
                follow_gpu_selection(st, states[b], b, o_score, w)
            elif t % check_every == 0:
                o_out = states[b].small(bits(qs[t, b]))
                check_out(st.out[b], o_out, f"small step t={t} seq {b}")
    assert ctx.device_status() == 0
    assert cache.len.tolist() == [l + w.steps for l in w.lens]
    # cases left out of the flag comparison are counted, never silently passed: they must stay rare
    NEAR_THRESHOLD["checks"] += checks
    NEAR_THRESHOLD["excluded"] += excluded
    assert excluded <= max(1, checks // 20), (excluded, checks)
    return n_full


def follow_gpu_selection(st, state, b, o_score, w):
    """Validate the GPU's top-K set against the oracle's scores, then make the oracle's small cache
    hold the same rows in the same (ascending) order so that later small steps compare like with like."""
    n = state.len_full
    idx = st.topk_idx[b].cpu().numpy()
    take = min(w.k_small[b], n)
    sel = []
    for g in range(w.n_kv_heads):
        got = idx[g, :take]
        assert (np.diff(got) > 0).all()
        why = O.check_topk_set(o_score[g], w.k_small[b], got)
        assert why is None, f"seq {b} head {g}: {why}"
        sel.append(got.astype(np.int64))
    state.k_small = O.gather_rows(state.k_full, sel)
    state.v_small = O.gather_rows(state.v_full, sel)
    state.small_pos = [x.copy() for x in sel]
    state.len_small = take
    if state.evict:
        # the eviction order the GPU derived: scores must not decrease along it (within the selection band), nothing
        # left behind may score clearly lower than the last listed victim; the oracle then follows the same order
        order = st.evict_order[b].cpu().numpy()
        assert int(st.evict_count[b]) == 0
        state.evict_queue = []
        for g in range(w.n_kv_heads):
            e = order[g][order[g] >= 0]
            assert len(e) == min(order.shape[1], take) and len(set(e.tolist())) == len(e) and e.max() < take
            sc = o_score[g][sel[g][e]]
            assert (sc[:-1] <= sc[1:] * (1 + 1e-5)).all(), "victims must come lowest score first"
            rest = np.ones(take, dtype=bool); rest[e] = False
            if rest.any():
                assert o_score[g][sel[g][rest]].min() >= sc[-1] * (1 - 1e-5)
            state.evict_queue.append(e.tolist())
    # gathered rows on the GPU are bit-exact copies
    for which, small in (("k", state.k_small), ("v", state.v_small)):
        gpu_small = host_heads(st.small, b, w.n_kv_heads, which)
        for g in range(w.n_kv_heads):
            assert np.array_equal(gpu_small[g, :take], small[g])


@pytest.mark.parametrize("fused,overlapped", [(False, False), (True, False), (True, True)])
def test_config1_every_step_every_head(mods, fused, overlapped):
    rkv, runner, synth = mods
    w = synth.config1()
    n_full = run_trajectory(mods, w, 0, fused=fused, overlapped=overlapped)
    assert n_full[0] == 4      # full steps at t = 4, 8, 12, 16


def test_config1_fixed_size_small_cache_with_eviction(mods):
    """Config 1 with the paper's fixed-size partial cache: every partial step attends over exactly K rows."""
    rkv, runner, synth = mods
    n_full = run_trajectory(mods, synth.config1(), 0, evict=8)
    assert n_full[0] == 4


def test_config3_shape_dynamic_with_eviction(mods):
    rkv, runner, synth = mods
    w = synth.scaled(synth.config3(n_layers=1, ctx=8192), steps=40)
    n_full = run_trajectory(mods, w, 0, evict=64)
    assert n_full[0] >= 1


def test_eviction_runs_out_of_slots_and_short_caches_grow(mods):
    rkv, runner, synth = mods
    lens, k_small = [300, 20], [16, 32]            # sequence 1 is shorter than its K: its small cache grows instead
    ctx, st, cache, q = make_layer(mods, lens, k_small, 8, 2, extra=8, seed=31)
    st.enable_eviction(2)
    st.refresh_evict(q)
    assert st.small.len.tolist() == [16, 20] and st.evict_count.tolist() == [0, 0]
    assert (st.evict_order[0] >= 0).all() and (st.evict_order[1] >= 0).all()
    g = torch.Generator(device="cuda"); g.manual_seed(32)
    for step in range(3):
        kn = torch.randn((2, 2, 128), generator=g, device="cuda").to(torch.bfloat16)
        vn = torch.randn((2, 2, 128), generator=g, device="cuda").to(torch.bfloat16)
        before = st.small.k.clone()
        victims = st.evict_order[0, :, min(step, 1)].tolist()
        st.append_partial_evict(q, kn, vn)
        bits_now = ctx.device_status()
        assert st.small.len.tolist() == [16, 21 + step] and cache.len.tolist() == [301 + step, 21 + step]
        sk = host_heads(st.small, 0, 2, "k")
        if step < 2:
            assert bits_now == 0 and st.evict_count.tolist()[0] == step + 1
            for h in range(2):
                assert np.array_equal(sk[h, victims[h]], bits(kn[0, h]))
        else:                                      # third new token, two eviction slots: flagged, small cache of seq 0 untouched
            assert bits_now & rkv.DEV_APPEND_OVERFLOW
            cap0 = int(st.small.cap[0])
            assert torch.equal(st.small.k[: 2 * cap0], before[: 2 * cap0]) and st.evict_count.tolist()[0] == 2
        # attention of sequence 0 runs over exactly the 16 rows now in the cache
        k = O.bf16_bits_to_f64(host_heads(st.small, 0, 2, "k")[:, :16])
        v = O.bf16_bits_to_f64(host_heads(st.small, 0, 2, "v")[:, :16])
        want, _, _ = O.decode_attention(O.bf16_bits_to_f64(bits(q[0])), k, v)
        check_out(st.out[0], want, f"evicting step {step}")


def test_config1_planted_positions_are_selected(mods):
    rkv, runner, synth = mods
    w = synth.config1()
    dev = torch.device("cuda")
    cache = synth.fill_layer(w, 0, dev)
    qs = synth.query_trajectory(w, 0).to(dev)
    synth.plant_heavy(w, cache, 0, qs[0])
    ctx = rkv.Context(1, 32, 8, int(cache.cap.max()), 256 + 32)
    st = runner.LayerState(ctx, cache, [256], 32, 32, 8, want_scores=True)
    st.refresh(qs[0])
    heavy = synth.heavy_positions(w, 0, 0, 0, 2048, "cpu").numpy()
    idx = st.topk_idx[0].cpu().numpy()
    sc = st.scores[0].cpu().numpy()
    for g in range(8):
        assert set(heavy[g].tolist()) <= set(idx[g].tolist())
        assert sc[g, heavy[g]].sum() > 0.05       # the planted keys carry a visible share of the mass


def test_config2_shape_one_layer_full_size(mods):
    """Llama-3.1-8B shape at L=32768, K=2048: a short trajectory (one stride period + a replant) at full size."""
    rkv, runner, synth = mods
    w = synth.scaled(synth.config2(n_layers=1), steps=12, replant_every=6)
    n_full = run_trajectory(mods, w, 0)
    assert n_full[0] == 1


@pytest.mark.parametrize("fused,overlapped", [(False, False), (True, False), (True, True)])
def test_config3_shape_dynamic_flags(mods, fused, overlapped):
    """Qwen2-7B shape (G=7), batch 4, dynamic refresh; reduced context for the per-step oracle, full K ratio."""
    rkv, runner, synth = mods
    w = synth.scaled(synth.config3(n_layers=1, ctx=8192), steps=40)
    n_full = run_trajectory(mods, w, 0, fused=fused, overlapped=overlapped)
    # fast-drifting sequences refresh more often than slow ones
    assert n_full[0] >= n_full[3]
    assert n_full[0] >= 1


@pytest.mark.parametrize("layer", [0, 31])
def test_config2_full_size_two_replants(mods, layer):
    """Config 2 as stated (L=32768, K=2048, stride 10, heavy positions moved every 64 steps) for 130 steps of the
    first and the last layer: 13 full steps, two replants; every full step and every fifth partial step against the
    oracle.  Full-step tokens run the way bench.py launches them (selection and rebuild after the attention pass,
    from a context of the layer's own)."""
    rkv, runner, synth = mods
    w = synth.scaled(synth.config2(n_layers=32), steps=130)
    n_full = run_trajectory(mods, w, layer, check_every=5, fused=True, deferred=True)
    assert n_full[0] == 13


def test_config3_full_size_dynamic_all_drift_rates(mods):
    """Config 3 at its stated size (G=7, four sequences of 65536 tokens, K=4096, threshold 0.9, check every 5
    tokens) for 20 steps: every check of every sequence against the oracle's flag, every refresh and every fifth
    partial step against its outputs; the sequences that drift fast refresh, the slow one does not."""
    rkv, runner, synth = mods
    w = synth.scaled(synth.config3(n_layers=1), steps=20)
    n_full = run_trajectory(mods, w, 0, check_every=5, fused=True, deferred=True)
    assert n_full[0] >= 3 and n_full[0] >= n_full[3]


PAPER_CASES = [("lm16k_S10", 4096), ("lm16k_S15", 4096), ("lm16k_dyn085_qc5", 4096), ("lm16k_dyn085_qc10", 4096),
               ("novel128k_S10", 16384), ("novel128k_dyn085_qc10", 16384), ("qwen16k_dyn095_qc5", 4096),
               ("qwen16k_dyn095_qc10", 4096)]


@pytest.mark.parametrize("name,ctx", PAPER_CASES)
def test_paper_operating_points_reduced_length(mods, name, ctx):
    """The paper's own operating points (K = L / 8, capped at 4096 for 100K+ inputs; fixed strides 10 and 15; the
    similarity trigger every 5 or 10 steps at threshold 0.85 or 0.95; both model shapes) at a reduced context with the
    point's own K / L, 31 steps each, every step checked."""
    rkv, runner, synth = mods
    full = synth.paper_point(name, n_layers=1)
    w = synth.scaled(full, lens=[ctx], k_small=[ctx * full.k_small[0] // full.lens[0]], steps=31, replant_every=16)
    assert w.k_small[0] * full.lens[0] == ctx * full.k_small[0]      # the point's own K / L (1/8; 1/32 for 100K+ inputs)
    n_full = run_trajectory(mods, w, 0, fused=True, deferred=True)
    if w.schedule == "fixed":
        assert n_full[0] == 31 // w.stride
    else:
        assert n_full[0] <= 31 // w.stride


def test_layer_batched_partial_step_every_layer_and_sequence(mods):
    """The partial step of all layers in one launch (bench.py's layer-batched measurement): the small caches of
    three layers x two sequences in one buffer, one rkv_append_small_step per token; every (layer, sequence)
    against the oracle on the rows its own layer's refresh selected, for three tokens."""
    rkv, runner, synth = mods
    dev = torch.device("cuda")
    n_q, n_kv, NL = 32, 8, 3
    lens, k_small = [1500, 700], [200, 64]
    layers = []
    for l in range(NL):
        ctx, st, cache, q = make_layer(mods, lens, k_small, n_q, n_kv, extra=8, seed=70 + l, want_scores=False)
        st.refresh(q)
        layers.append((ctx, st, cache))
    hint = max(k_small) + 8
    lb = runner.LayerBatchedSmall([st for _, st, _ in layers], hint)
    lb.sync_from_layers()
    g = torch.Generator(device=dev); g.manual_seed(99)
    small_bits = {}
    for l, (_, st, _) in enumerate(layers):
        for b in range(2):
            small_bits[(l, b)] = [host_heads(st.small, b, n_kv, "k").copy(), host_heads(st.small, b, n_kv, "v").copy(),
                                  k_small[b]]
    for step in range(3):
        q_all = torch.randn((NL, 2, n_q, 128), generator=g, device=dev).to(torch.bfloat16)
        k_all = torch.randn((NL, 2, n_kv, 128), generator=g, device=dev).to(torch.bfloat16)
        v_all = torch.randn((NL, 2, n_kv, 128), generator=g, device=dev).to(torch.bfloat16)
        out_all = torch.zeros((NL, 2, n_q, 128), dtype=torch.bfloat16, device=dev)
        lb.append_partial(q_all, k_all, v_all, out_all)
        assert lb.ctx.device_status() == 0
        assert lb.cache.len.tolist() == [k + step + 1 for _ in range(NL) for k in k_small]
        for l in range(NL):
            for b in range(2):
                kb, vb, n = small_bits[(l, b)]
                kb[:, n], vb[:, n] = bits(k_all[l, b]), bits(v_all[l, b])        # the oracle's copy takes the new row too
                small_bits[(l, b)][2] = n + 1
                want, _, _ = O.decode_attention(O.bf16_bits_to_f64(bits(q_all[l, b])), O.bf16_bits_to_f64(kb[:, : n + 1]),
                                                O.bf16_bits_to_f64(vb[:, : n + 1]))
                check_out(out_all[l, b], want, f"token {step} layer {l} seq {b}")
    # the rows the batched cache holds are the layers' own, bit for bit
    offs = lb.cache.row_offset.tolist()
    for l, (_, st, _) in enumerate(layers):
        cap0 = int(st.small.cap[0])
        assert torch.equal(lb.cache.k[offs[2 * l]: offs[2 * l] + 200], st.small.k[:200])
        assert torch.equal(lb.cache.k[offs[2 * l] + cap0: offs[2 * l] + cap0 + 200], st.small.k[cap0: cap0 + 200])


def test_layer_batched_full_step_every_layer_and_sequence(mods):
    """rkv_full_step of all layers in one call (bench.py's layer-batched measurement): the full caches of three
    layers x two ragged sequences in one K and one V buffer, one context that sees six sequences; outputs and top-K
    sets of every (layer, sequence) against the oracle (the per-layer calls on the layers' views of the same buffers
    split the caches differently, so their log-sum-exps - and with them keys one ulp apart - may differ in the last
    bit: both are held to the oracle, not to each other)."""
    rkv, runner, synth = mods
    dev = torch.device("cuda")
    w = synth.Workload("stack", 3, 28, 4, [3000, 700], [300, 64], 4, "fixed", 10, rho=[0.9, 0.9], seed=11)
    stack = synth.alloc_layer_stack(w, dev)
    qs = []
    per_layer = []
    for l in range(w.n_layers):
        view = synth.fill_layer(w, l, dev, into=synth.layer_view(stack, l, w.batch))
        q = synth.query_trajectory(w, l)[0].to(dev)
        synth.plant_heavy(w, view, l, q)
        qs.append(q)
        ctx = rkv.Context(w.batch, w.n_q_heads, w.n_kv_heads, max(w.lens) + 8, max(w.k_small) + 8)
        st = runner.LayerState(ctx, view, list(w.k_small), 8, w.n_q_heads, w.n_kv_heads, want_scores=False)
        st.refresh(q)
        assert ctx.device_status() == 0
        per_layer.append((ctx, st, view))
    q_all = torch.stack(qs)                                       # [layers, B, Hq, 128]
    lb = runner.LayerBatchedFull(stack, w.n_layers, list(w.k_small), w.n_q_heads, w.n_kv_heads, max(w.lens) + 8)
    out = lb.full_step(q_all).view(w.n_layers, w.batch, w.n_q_heads, 128)
    assert lb.ctx.device_status() == 0
    idx = lb.topk_idx.view(w.n_layers, w.batch, w.n_kv_heads, -1)
    for l, (ctx, st, view) in enumerate(per_layer):
        for b, n in enumerate(w.lens):
            o_out, o_score, o_idx, _ = oracle_full(view, b, n, q_all[l, b], w.n_kv_heads, w.k_small[b])
            check_out(out[l, b], o_out, f"layer {l} seq {b}")
            for g in range(w.n_kv_heads):
                why = O.check_topk_set(o_score[g], w.k_small[b], idx[l, b, g, : w.k_small[b]].cpu().numpy())
                assert why is None, f"layer {l} seq {b} head {g}: {why}"


def test_config3_full_size_single_step(mods):
    rkv, runner, synth = mods
    w = synth.scaled(synth.config3(n_layers=1), steps=2, stride=1)
    run_trajectory(mods, w, 0, seqs=[0, 3])


@pytest.mark.parametrize("fused,overlapped", [(False, False), (True, True)])
def test_config4_ragged_sampled_sequences(mods, fused, overlapped):
    """Ragged batch of 16 (lengths 8K..128K): shortest, median and longest sequence against the oracle; the second
    variant in the calls bench.py makes (append fused into the partial step - two CTAs per (sequence, KV head) at
    this batch size - and the full step in two halves on two streams)."""
    rkv, runner, synth = mods
    w = synth.scaled(synth.config4(n_layers=1), steps=11)
    order = np.argsort(w.lens)
    seqs = [int(order[0]), int(order[len(order) // 2]), int(order[-1])]
    n_full = run_trajectory(mods, w, 0, seqs=seqs, fused=fused, overlapped=overlapped)
    assert all(v == 1 for v in n_full.values())


def test_largest_supported_length(mods):
    """One sequence close to the selection kernel's limit (8 CTAs x 40960 keys): 300000 positions, top-4096."""
    lens, k_small = [300000], [4096]
    ctx, st, cache, q = make_layer(mods, lens, k_small, 2, 1, seed=41, want_scores=True)
    st.refresh(q)
    assert ctx.device_status() == 0
    check_full_against_oracle(st, cache, q, lens, k_small, 1)
    out = st.partial(q).clone()
    n = 300000
    kf, vf = host_heads(cache, 0, 1, "k"), host_heads(cache, 0, 1, "v")
    sel = [st.topk_idx[0, 0, :4096].cpu().numpy().astype(np.int64)]
    want, _, _ = O.decode_attention(O.bf16_bits_to_f64(bits(q[0])), O.bf16_bits_to_f64(np.stack(O.gather_rows(kf, sel))),
                                    O.bf16_bits_to_f64(np.stack(O.gather_rows(vf, sel))))
    check_out(out[0], want, "partial step on 4096 of 300000")
    rkv = mods[0]
    with pytest.raises(rkv.RkvError):
        rkv.Context(1, 2, 1, 8 * 40960 + 1, 64)            # beyond the limit: refused at creation


@pytest.mark.parametrize("pool", [7, 31])
def test_pooling_on_a_long_sequence(mods, pool):
    """Neighbour max-pooling at a length where the selection runs with its largest slices (163840 positions)."""
    lens, k_small = [163840], [4096]
    ctx, st, cache, q = make_layer(mods, lens, k_small, 2, 1, seed=43 + pool, want_scores=True, pool=pool)
    st.refresh(q)
    assert ctx.device_status() == 0
    check_full_against_oracle(st, cache, q, lens, k_small, 1, pool=pool)


def test_bench_configuration_graph_replay_shared_context(mods):
    """The launch configuration bench.py times, at config 2's full size: the layers alternate between two
    contexts, a token's calls are replayed from CUDA graphs with the inputs staged in a device buffer.  Partial
    tokens: one rkv_append_small_step per layer (the early cache read is live: the launch before each is another
    layer's).  Full-step tokens: rkv_append + rkv_full_attention in the capturing stream, rkv_select_topk +
    rkv_gather_small behind them in a second stream (runner.OverlappedRefresh).  Every layer's output of every
    token is compared with the oracle."""
    rkv, runner, synth = mods
    dev = torch.device("cuda")
    NL, S, T = 3, 10, 21
    w = synth.scaled(synth.config2(n_layers=NL), steps=T)
    L, K, Hq, Hkv = w.lens[0], w.k_small[0], w.n_q_heads, w.n_kv_heads
    full_hint, small_hint = L + T + 1, K + S + 2
    ctxs = [rkv.Context(1, Hq, Hkv, full_hint, small_hint) for _ in range(2)]
    q_stage = torch.zeros((NL, 1, Hq, 128), dtype=torch.bfloat16, device=dev)
    k_stage = torch.zeros((NL, 1, Hkv, 128), dtype=torch.bfloat16, device=dev)
    v_stage = torch.zeros((NL, 1, Hkv, 128), dtype=torch.bfloat16, device=dev)
    layers, states, inputs = [], [], []
    for l in range(NL):
        cache = synth.fill_layer(w, l, dev)
        qs = synth.query_trajectory(w, l).to(dev)
        kn, vn = synth.new_token_kv(w, l)
        synth.plant_heavy(w, cache, l, qs[0])
        st = runner.LayerState(ctxs[l % 2], cache, [K], S + 2, Hq, Hkv)
        layers.append(st)
        inputs.append((qs, kn.to(dev), vn.to(dev)))
        states.append(O.SequenceState(host_heads(cache, 0, Hkv, "k").copy(), host_heads(cache, 0, Hkv, "v").copy(), L, K))

    def stage(t):
        for l in range(NL):
            q_stage[l].copy_(inputs[l][0][t]); k_stage[l].copy_(inputs[l][1][t]); v_stage[l].copy_(inputs[l][2][t])

    overlapped = runner.OverlappedRefresh(layers)

    def token(kind):
        if kind == "full":
            return overlapped.run(lambda l: q_stage[l], lambda l: k_stage[l], lambda l: v_stage[l],
                                  max_len_hint=full_hint)
        for l, st in enumerate(layers):
            st.append_partial(q_stage[l], k_stage[l], v_stage[l], max_len_hint=small_hint)

    class W1:      # what follow_gpu_selection needs to know about the workload
        n_kv_heads, k_small = Hkv, [K]
    stage(0)
    for l, st in enumerate(layers):          # initial small caches (eager; also builds the tensor maps)
        st.refresh(q_stage[l], max_len_hint=full_hint)
        o_out, o_score, _ = states[l].full(bits(inputs[l][0][0, 0]))
        check_out(st.out[0], o_out, f"init layer {l}")
        follow_gpu_selection(st, states[l], 0, o_score, W1)
    # warm both kinds eagerly on throw-away copies?  No: capture directly; capture does not execute
    torch.cuda.synchronize()
    graphs, side = {}, torch.cuda.Stream()
    for kind in ("small", "full"):
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(gr, stream=side):
                token(kind)
        graphs[kind] = gr
    for t in range(1, T + 1):
        stage(t)
        kind = "full" if t % S == 0 else "small"
        graphs[kind].replay()
        torch.cuda.synchronize()
        for l, st in enumerate(layers):
            states[l].append(bits(inputs[l][1][t, 0]), bits(inputs[l][2][t, 0]))
            if kind == "full":
                o_out, o_score, _ = states[l].full(bits(inputs[l][0][t, 0]))
                check_out(st.out[0], o_out, f"full token {t} layer {l}")
                follow_gpu_selection(st, states[l], 0, o_score, W1)
            else:
                check_out(st.out[0], states[l].small(bits(inputs[l][0][t, 0])), f"partial token {t} layer {l}")
    assert all(c.device_status() == 0 for c in ctxs)
    assert all(int(st.full.len[0]) == L + T and int(st.small.len[0]) == K + 1 for st in layers)


@pytest.mark.parametrize("early_scores", [False, True])
def test_bench_configuration_deferred_tail_eight_layers(mods, early_scores):
    """(early_scores: every layer's score pass right behind its attention pass in a stream of its own, rkv_score_keys.)
    The schedule bench.py times by default (runner.DeferredRefresh), with the eight layers from which on it runs
    its tail in the throughput shape (large score-pass slices, few large top-K CTAs, set around the calls and
    restored): config-2 shape at a reduced context, one context per layer, tokens replayed from CUDA graphs.  Every
    layer's output of every token against the oracle, the selected sets validated, the options back at their defaults."""
    rkv, runner, synth = mods
    dev = torch.device("cuda")
    NL, S, T = 8, 10, 21
    w = synth.scaled(synth.config2(n_layers=NL, ctx=6144), steps=T)
    L, K, Hq, Hkv = w.lens[0], w.k_small[0], w.n_q_heads, w.n_kv_heads
    full_hint, small_hint = L + T + 1, K + S + 2
    ctxs = [rkv.Context(1, Hq, Hkv, full_hint, small_hint) for _ in range(NL)]
    q_stage = torch.zeros((NL, 1, Hq, 128), dtype=torch.bfloat16, device=dev)
    k_stage = torch.zeros((NL, 1, Hkv, 128), dtype=torch.bfloat16, device=dev)
    v_stage = torch.zeros((NL, 1, Hkv, 128), dtype=torch.bfloat16, device=dev)
    layers, states, inputs = [], [], []
    for l in range(NL):
        cache = synth.fill_layer(w, l, dev)
        qs = synth.query_trajectory(w, l).to(dev)
        kn, vn = synth.new_token_kv(w, l)
        synth.plant_heavy(w, cache, l, qs[0])
        layers.append(runner.LayerState(ctxs[l], cache, [K], S + 2, Hq, Hkv))
        inputs.append((qs, kn.to(dev), vn.to(dev)))
        states.append(O.SequenceState(host_heads(cache, 0, Hkv, "k").copy(), host_heads(cache, 0, Hkv, "v").copy(), L, K))

    def stage(t):
        for l in range(NL):
            q_stage[l].copy_(inputs[l][0][t]); k_stage[l].copy_(inputs[l][1][t]); v_stage[l].copy_(inputs[l][2][t])

    deferred = runner.DeferredRefresh(layers, early_scores=early_scores)
    assert all(val for _, val in deferred.tuning)          # eight layers: the tail runs in its throughput shape

    def token(kind):
        if kind == "full":
            return deferred.run(lambda l: q_stage[l], lambda l: k_stage[l], lambda l: v_stage[l], max_len_hint=full_hint)
        for l, st in enumerate(layers):
            st.append_partial(q_stage[l], k_stage[l], v_stage[l], max_len_hint=small_hint)

    class W1:
        n_kv_heads, k_small = Hkv, [K]
    stage(0)
    for l, st in enumerate(layers):
        st.refresh(q_stage[l], max_len_hint=full_hint)
        o_out, o_score, _ = states[l].full(bits(inputs[l][0][0, 0]))
        check_out(st.out[0], o_out, f"init layer {l}")
        follow_gpu_selection(st, states[l], 0, o_score, W1)
    torch.cuda.synchronize()
    graphs, side = {}, torch.cuda.Stream()
    for kind in ("small", "full"):
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(gr, stream=side):
                token(kind)
        graphs[kind] = gr
    for c in ctxs:      # the tail's settings were put back after the calls were captured
        assert c.get_option(rkv.OPT_SELECT_KEYS_PER_CTA) == 4096 and c.get_option(rkv.OPT_SCORE_SLICE) == 0
    for t in range(1, T + 1):
        stage(t)
        kind = "full" if t % S == 0 else "small"
        graphs[kind].replay()
        torch.cuda.synchronize()
        for l, st in enumerate(layers):
            states[l].append(bits(inputs[l][1][t, 0]), bits(inputs[l][2][t, 0]))
            if kind == "full":
                o_out, o_score, _ = states[l].full(bits(inputs[l][0][t, 0]))
                check_out(st.out[0], o_out, f"full token {t} layer {l}")
                follow_gpu_selection(st, states[l], 0, o_score, W1)
            else:
                check_out(st.out[0], states[l].small(bits(inputs[l][0][t, 0])), f"partial token {t} layer {l}")
    assert all(c.device_status() == 0 for c in ctxs)
    assert all(int(st.full.len[0]) == L + T and int(st.small.len[0]) == K + 1 for st in layers)


def test_bench_configuration_dynamic_schedule_graph_replay(mods):
    """The dynamic schedule as bench.py launches it (config-3 shape, reduced context): three layers that alternate
    between two contexts; plain tokens = one rkv_append_small_step per layer; every fifth token the trigger, both
    branches under its masks and the selection in the second stream (runner.OverlappedRefresh.run_checked); both
    kinds replayed from CUDA graphs with the inputs staged in a device buffer.  Every layer, sequence and token
    against the oracle."""
    rkv, runner, synth = mods
    dev = torch.device("cuda")
    NL, T = 3, 16
    w = synth.scaled(synth.config3(n_layers=NL, ctx=4096), steps=T)
    B, Hq, Hkv, QC = w.batch, w.n_q_heads, w.n_kv_heads, w.stride
    full_hint, small_hint = max(w.lens) + T + 1, max(w.k_small) + T + 2
    ctxs = [rkv.Context(B, Hq, Hkv, full_hint, small_hint) for _ in range(2)]
    q_stage = torch.zeros((NL, B, Hq, 128), dtype=torch.bfloat16, device=dev)
    k_stage = torch.zeros((NL, B, Hkv, 128), dtype=torch.bfloat16, device=dev)
    v_stage = torch.zeros((NL, B, Hkv, 128), dtype=torch.bfloat16, device=dev)
    layers, inputs, states = [], [], []
    for l in range(NL):
        cache = synth.fill_layer(w, l, dev)
        qs = synth.query_trajectory(w, l).to(dev)
        kn, vn = synth.new_token_kv(w, l)
        synth.plant_heavy(w, cache, l, qs[0])
        layers.append(runner.LayerState(ctxs[l % 2], cache, list(w.k_small), T + 2, Hq, Hkv))
        inputs.append((qs, kn.to(dev), vn.to(dev)))
        states.append([O.SequenceState(host_heads(cache, b, Hkv, "k").copy(), host_heads(cache, b, Hkv, "v").copy(),
                                       w.lens[b], w.k_small[b]) for b in range(B)])

    def stage(t):
        for l in range(NL):
            q_stage[l].copy_(inputs[l][0][t]); k_stage[l].copy_(inputs[l][1][t]); v_stage[l].copy_(inputs[l][2][t])

    overlapped = runner.OverlappedRefresh(layers)

    def token(kind):
        if kind == "check":
            return overlapped.run_checked(lambda l: q_stage[l], lambda l: k_stage[l], lambda l: v_stage[l], w.threshold,
                                          small_hint=small_hint, full_hint=full_hint)
        for l, st in enumerate(layers):
            st.append_partial(q_stage[l], k_stage[l], v_stage[l], max_len_hint=small_hint)

    stage(0)
    for l, st in enumerate(layers):          # initial small caches (eager; also builds the tensor maps)
        st.refresh(q_stage[l], max_len_hint=full_hint)
        for b in range(B):
            o_out, o_score, _ = states[l][b].full(bits(inputs[l][0][0, b]))
            check_out(st.out[b], o_out, f"init layer {l} seq {b}")
            follow_gpu_selection(st, states[l][b], b, o_score, w)
    torch.cuda.synchronize()
    graphs, side = {}, torch.cuda.Stream()
    for kind in ("small", "check"):
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(gr, stream=side):
                token(kind)
        graphs[kind] = gr
    n_full = 0
    for t in range(1, T + 1):
        stage(t)
        kind = "check" if t % QC == 0 else "small"
        graphs[kind].replay()
        torch.cuda.synchronize()
        for l, st in enumerate(layers):
            flags = st.flag.cpu().numpy()
            for b in range(B):
                state = states[l][b]
                state.append(bits(inputs[l][1][t, b]), bits(inputs[l][2][t, b]))
                qb = bits(inputs[l][0][t, b])
                full_now = False
                if kind == "check":
                    want, cos = O.should_refresh(O.bf16_bits_to_f64(qb), state.q_last_full, w.threshold)
                    if abs(cos - w.threshold) >= 1e-4:
                        assert flags[b] == want, (t, l, b, cos)
                    full_now = bool(flags[b])
                if full_now:
                    o_out, o_score, _ = state.full(qb)
                    check_out(st.out[b], o_out, f"full step t={t} layer {l} seq {b}")
                    follow_gpu_selection(st, state, b, o_score, w)
                    n_full += 1
                else:
                    check_out(st.out[b], state.small(qb), f"partial step t={t} layer {l} seq {b}")
    assert all(c.device_status() == 0 for c in ctxs)
    assert n_full >= 1
    for st in layers:
        assert st.full.len.tolist() == [n + T for n in w.lens]

