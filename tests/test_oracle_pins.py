"""Pins for the fp64 CPU oracle: every function is tied to something other than itself.

Closed forms, hand-worked fixtures (tests/golden), an independent library routine
(torch scaled_dot_product_attention on fp64 CPU tensors), brute force on tiny inputs,
and invariants the method's definition fixes.  No GPU needed.
"""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import rkv_oracle as O


def _rng(seed):
    return np.random.default_rng(seed)


def _rand_case(seed, n_q=8, n_kv=2, n=37, d=16):
    r = _rng(seed)
    return r.normal(size=(n_q, d)), r.normal(size=(n_kv, n, d)), r.normal(size=(n_kv, n, d))


# ------------------------------------------------------------------ number formats
def test_bf16_widening_matches_torch():
    bits = np.arange(0, 65536, dtype=np.uint32).astype(np.uint16)
    ours = O.bf16_bits_to_f64(bits)
    ref = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    finite = np.isfinite(ref)
    assert np.array_equal(ours[finite], ref[finite])
    assert np.array_equal(np.isnan(ours), np.isnan(ref))


def test_bf16_rounding_matches_torch():
    x = _rng(1).normal(size=4096) * np.exp(_rng(2).uniform(-20, 20, size=4096))
    ours = O.f64_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, ref)
    # exact ties round to even: 1 + 2^-8 lies half-way between 1.0 and the next bf16
    assert O.f64_to_bf16_bits(np.array([1.0 + 2.0 ** -8]))[0] == 0x3F80
    assert O.f64_to_bf16_bits(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 0x3F82


# ------------------------------------------------------------------ softmax / attention
def test_softmax_rows_sum_to_one_and_lse():
    q, k, v = _rand_case(3)
    out, p, lse = O.decode_attention(q, k, v)
    assert np.allclose(p.sum(axis=1), 1.0, atol=1e-12)
    s = O.attention_logits(q, k)
    assert np.allclose(lse, np.log(np.exp(s).sum(axis=1)), atol=1e-12)
    assert np.allclose(p, np.exp(s - lse[:, None]), atol=1e-14)


def test_uniform_keys_give_mean_of_values():
    r = _rng(4)
    q = r.normal(size=(4, 16))
    k = np.tile(r.normal(size=(2, 1, 16)), (1, 29, 1))
    v = r.normal(size=(2, 29, 16))
    out, p, _ = O.decode_attention(q, k, v)
    assert np.allclose(p, 1.0 / 29, atol=1e-14)
    for h in range(4):
        assert np.allclose(out[h], v[h // 2].mean(axis=0), atol=1e-13)


def test_one_hot_key_selects_its_value():
    r = _rng(5)
    d = 16
    q = np.zeros((2, d))
    q[:, 0] = 1.0
    k = np.zeros((1, 11, d))
    k[0, 7, 0] = 50.0 * math.sqrt(d)       # logit +50 over the rest
    v = r.normal(size=(1, 11, d))
    out, p, _ = O.decode_attention(q, k, v)
    # the other ten positions carry exp(-50) each
    assert abs((1.0 - p[0, 7]) - 10 * math.exp(-50.0)) < 1e-24 or p[0, 7] == 1.0
    assert np.allclose(p[0, :7], math.exp(-50.0), rtol=1e-12)
    assert np.allclose(out[0], v[0, 7], atol=1e-15)


def test_against_torch_sdpa_fp64():
    """Independent library routine: softmax(QK^T/sqrt(d))V with KV heads repeated G times."""
    q, k, v = _rand_case(6, n_q=12, n_kv=3, n=53, d=128)
    out, _, _ = O.decode_attention(q, k, v)
    tq = torch.from_numpy(q)[None, :, None, :]                       # [1, Hq, 1, d]
    tk = torch.from_numpy(k).repeat_interleave(4, dim=0)[None]      # [1, Hq, n, d]
    tv = torch.from_numpy(v).repeat_interleave(4, dim=0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv)[0, :, 0, :].numpy()
    assert np.allclose(out, ref, atol=1e-12, rtol=1e-12)


def test_head_grouping_is_contiguous():
    """Heads gG..gG+G-1 read KV head g: changing KV head 1 must move only heads 2 and 3."""
    q, k, v = _rand_case(7, n_q=4, n_kv=2)
    base, _, _ = O.decode_attention(q, k, v)
    k2 = k.copy()
    k2[1] = _rng(70).normal(size=k2[1].shape)
    moved, _, _ = O.decode_attention(q, k2, v)
    assert np.array_equal(base[:2], moved[:2])
    assert not np.allclose(base[2], moved[2]) and not np.allclose(base[3], moved[3])


def test_default_scale_is_inverse_sqrt_d():
    q, k, v = _rand_case(8, d=64)
    assert np.allclose(O.attention_logits(q, k), O.attention_logits(q, k, scale=0.125))


# ------------------------------------------------------------------ GQA aggregation (golden, hand-worked)
def _read_fixture(path):
    rows = {}
    with open(path) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, vals = line.split("|")
            rows[name.strip()] = vals.split()
    return rows


def test_gqa_hand_example(golden_dir):
    fx = _read_fixture(os.path.join(golden_dir, "gqa_hand_example.txt"))
    w = np.array([[float(x) for x in fx[f"weights_head{h}"]] for h in range(4)])
    # one channel, scale 1, q = 1, k = ln(w): logits are ln(w) and p = w / sum(w)
    q = np.ones((4, 1))
    for mode in ("max", "mean", "first"):
        score = np.empty((2, 3))
        for g in range(2):
            # each group gets its own key rows, so build per-head logits through two single-head calls
            p_heads = []
            for h in (2 * g, 2 * g + 1):
                k = np.log(w[h])[None, :, None]
                _, p, _ = O.decode_attention(q[h:h + 1], k, np.zeros((1, 3, 1)), scale=1.0)
                p_heads.append(p[0])
            score[g] = O.aggregate_scores(np.stack(p_heads), 1, mode)[0]
            want = np.array([float(Fraction(x)) for x in fx[f"{mode}_group{g}"]])
            assert np.allclose(score[g], want, atol=1e-15), (mode, g)
        if mode == "max":
            for g in range(2):
                want_idx = [int(x) for x in fx[f"top2_max_group{g}"]]
                assert O.top_k_positions(score[g], 2).tolist() == want_idx


def test_aggregation_orderings_and_identity():
    _, p, _ = O.decode_attention(*_rand_case(9, n_q=8, n_kv=2))
    mx, mean, first = (O.aggregate_scores(p, 2, m) for m in ("max", "mean", "first"))
    assert (mx >= mean - 1e-18).all() and (mx >= first).all()
    assert (mean >= p.reshape(2, 4, -1).min(axis=1) - 1e-18).all()
    # G = 1: aggregation is the identity for every mode
    for m in ("max", "mean", "first"):
        assert np.array_equal(O.aggregate_scores(p, 8, m), p)


# ------------------------------------------------------------------ pooling
def test_pool_max_properties():
    x = _rng(10).random((3, 41))
    assert np.array_equal(O.pool_max(x, 1), x)
    p7 = O.pool_max(x, 7)
    assert (p7 >= x).all()
    # against torch's max_pool1d with -inf padding (independent routine)
    ref = torch.nn.functional.max_pool1d(torch.from_numpy(x)[None], 7, stride=1, padding=3)[0].numpy()
    assert np.array_equal(p7, ref)
    c = np.full((1, 9), 0.25)
    assert np.array_equal(O.pool_max(c, 7), c)
    # a single spike spreads to exactly its 7-neighbourhood
    s = np.zeros((1, 20)); s[0, 10] = 1.0
    assert np.nonzero(O.pool_max(s, 7)[0])[0].tolist() == list(range(7, 14))


# ------------------------------------------------------------------ top-K
@pytest.mark.parametrize("n", list(range(1, 13)) + [16])
def test_topk_brute_force_maximises_total_score(n):
    r = _rng(100 + n)
    score = r.random(n)
    ks = range(0, n + 2) if n <= 12 else (1, 3, 8, 13, 16)
    for k in ks:
        got = O.top_k_positions(score, k)
        take = min(k, n)
        assert len(got) == take and len(set(got.tolist())) == take
        best = max((sum(score[list(c)]) for c in itertools.combinations(range(n), take)), default=0.0)
        assert abs(score[got].sum() - best) <= 1e-12
        # rank order: non-increasing scores
        assert (np.diff(score[got]) <= 0).all()


def test_topk_matches_library_on_tie_free_input():
    score = _rng(11).permutation(5000).astype(np.float64)
    got = O.top_k_positions(score, 777)
    ref = torch.topk(torch.from_numpy(score), 777).indices.numpy()
    assert np.array_equal(got, ref)


def test_topk_ties_prefer_lower_index():
    assert O.top_k_positions(np.full(9, 0.5), 4).tolist() == [0, 1, 2, 3]
    s = np.array([0.1, 0.7, 0.7, 0.2, 0.7])
    assert O.top_k_positions(s, 2).tolist() == [1, 2]
    assert O.top_k_positions(s, 10).tolist() == [1, 2, 4, 3, 0]


def test_check_topk_set_rule():
    s = np.array([0.5, 0.4, 0.3, 0.3 * (1 + 5e-6), 0.1])
    assert O.check_topk_set(s, 3, [0, 1, 3]) is None
    assert O.check_topk_set(s, 3, [0, 1, 2]) is None            # inside the 1e-5 band
    assert O.check_topk_set(s, 3, [0, 1, 4]) is not None        # clearly below tau
    assert O.check_topk_set(s, 3, [0, 2, 3]) is not None        # misses a clear winner
    assert O.check_topk_set(s, 3, [0, 0, 1]) is not None
    assert O.check_topk_set(s, 3, [0, 1]) is not None
    assert O.check_topk_set(s, 9, [4, 3, 2, 1, 0]) is None


# ------------------------------------------------------------------ gather + small step
def test_small_step_equals_full_step_when_K_is_L():
    q, k, v = _rand_case(12, n_q=8, n_kv=2, n=64, d=128)
    out, score, idx, _ = O.full_step(q, k, v, 64)
    ks = np.stack(O.gather_rows(k, idx))
    vs = np.stack(O.gather_rows(v, idx))
    out_small, _, _ = O.decode_attention(q, ks, vs)
    assert np.allclose(out, out_small, atol=1e-12)
    for g in range(2):
        assert sorted(idx[g].tolist()) == list(range(64))


def test_attention_is_permutation_invariant_over_rows():
    q, k, v = _rand_case(13)
    perm = _rng(14).permutation(k.shape[1])
    a, _, _ = O.decode_attention(q, k, v)
    b, _, _ = O.decode_attention(q, k[:, perm], v[:, perm])
    assert np.allclose(a, b, atol=1e-13)


def test_gather_is_a_row_copy():
    cache = _rng(15).integers(0, 65536, size=(2, 10, 4)).astype(np.uint16)
    idx = [np.array([9, 0, 3]), np.array([5, 5 - 4, 2])]
    small = O.gather_rows(cache, idx)
    for g in range(2):
        for r, j in enumerate(idx[g]):
            assert np.array_equal(small[g][r], cache[g, j])


def test_small_cache_mass_dominates_when_topk_holds_the_heavy_positions():
    """Planted structure: keys aligned with the query must all be selected."""
    r = _rng(16)
    d, n, n_heavy = 128, 512, 8
    q = r.normal(size=(4, d))
    k = r.normal(size=(1, n, d)) / math.sqrt(d)
    v = r.normal(size=(1, n, d))
    u = q.mean(axis=0); u /= np.linalg.norm(u)
    heavy = r.choice(n, n_heavy, replace=False)
    k[0, heavy] = 4.0 * u
    _, score, idx, _ = O.full_step(q, k, v, 64)
    assert set(heavy.tolist()) <= set(idx[0].tolist())
    assert set(idx[0][:n_heavy].tolist()) == set(heavy.tolist())      # they rank first


# ------------------------------------------------------------------ trigger
def test_cosine_closed_forms():
    r = _rng(17)
    q = r.normal(size=(4, 8))
    assert abs(O.cosine_similarity(q, q) - 1.0) < 1e-15
    assert abs(O.cosine_similarity(q, -q) + 1.0) < 1e-15
    assert abs(O.cosine_similarity(3.0 * q, 0.25 * q) - 1.0) < 1e-15
    a = np.zeros((2, 4)); a[:, 0] = 1
    b = np.zeros((2, 4)); b[:, 1] = 2
    assert O.cosine_similarity(a, b) == 0.0
    # the mean over heads is taken BEFORE the cosine: two heads that cancel leave the other direction
    c = np.array([[1.0, 0, 0, 0], [-1.0, 0, 0, 0], [0, 3.0, 0, 0]])
    dvec = np.array([[0, 1.0, 0, 0]] * 3)
    assert abs(O.cosine_similarity(c, dvec) - 1.0) < 1e-15
    # 45 degrees
    e = np.array([[1.0, 1.0, 0, 0]])
    f = np.array([[1.0, 0, 0, 0]])
    assert abs(O.cosine_similarity(e, f) - math.sqrt(0.5)) < 1e-15


def test_trigger_direction_and_edge_cases():
    e = np.array([[1.0, 1.0, 0, 0]])
    f = np.array([[1.0, 0, 0, 0]])           # cos = 0.7071
    assert O.should_refresh(e, f, 0.5)[0] == 0     # similarity higher than s -> partial step
    assert O.should_refresh(e, f, 0.9)[0] == 1     # otherwise -> full step
    assert O.should_refresh(f, f, 1.0)[0] == 1     # equality is not "higher"
    assert O.should_refresh(np.zeros((1, 4)), f, 0.5)[0] == 1    # zero mean query -> NaN -> refresh


# ------------------------------------------------------------------ schedule + cost model (golden)
def test_fig1_schedule(golden_dir):
    with open(os.path.join(golden_dir, "fig1_schedule.txt")) as f:
        line = [l for l in f if l.strip() and not l.startswith("#")][0]
    left, right = line.split("|")
    L, K, S, n = (int(x) for x in left.split())
    want = right.split()
    got = ["F" if O.fixed_stride_is_full(t, S) else "P" for t in range(1, n + 1)]
    assert got == want


def test_cost_model_closed_forms(golden_dir):
    with open(os.path.join(golden_dir, "cost_model.txt")) as f:
        for line in f:
            if not line.strip() or line.startswith("#"):
                continue
            a, b, c = line.split("|")
            T, L, K, S = (int(x) for x in a.split())
            vanilla, refresh = (float(x) for x in b.split())
            assert O.attention_cost_vanilla(T, L) == vanilla
            assert abs(O.attention_cost_refreshkv(T, L, K, S) - refresh) < 1e-9
            assert L + K == int(c)


def _tiny_state(seed, n_kv=2, group=2, ctx=24, k_small=6, steps=9, d=128):
    r = _rng(seed)
    cap = ctx + steps + 1
    kf = O.f64_to_bf16_bits(r.normal(size=(n_kv, cap, d)))
    vf = O.f64_to_bf16_bits(r.normal(size=(n_kv, cap, d)))
    qs = [O.f64_to_bf16_bits(r.normal(size=(n_kv * group, d))) for _ in range(steps + 1)]
    kn = [O.f64_to_bf16_bits(r.normal(size=(n_kv, d))) for _ in range(steps + 1)]
    vn = [O.f64_to_bf16_bits(r.normal(size=(n_kv, d))) for _ in range(steps + 1)]
    return O.SequenceState(kf, vf, ctx, k_small), qs, kn, vn


def test_driver_positions_touched_match_cost_model():
    """Counter invariant behind Table 5: T/S full passes over the context + the rest over K (+ appended tokens)."""
    ctx, k_small, steps, S = 24, 6, 9, 3
    st, qs, kn, vn = _tiny_state(18, ctx=ctx, k_small=k_small, steps=steps)
    trace = O.run_fixed_stride(st, qs, kn, vn, S)
    kinds = [k for k, _ in trace]
    assert kinds == ["small", "small", "full"] * 3
    assert st.n_full_steps == 1 + steps // S and st.n_small_steps == steps - steps // S
    # exact count: init pass over ctx; full step at t sees ctx+t rows; small step at t sees K + (t mod S) rows
    want = ctx + sum(ctx + t for t in range(1, steps + 1) if t % S == 0) \
               + sum(k_small + (t % S) for t in range(1, steps + 1) if t % S)
    assert st.positions_touched == want
    # and this is the paper's T*L/S + T*K up to the appended-token terms
    model = O.attention_cost_refreshkv(steps, ctx, k_small, S)
    assert abs((st.positions_touched - ctx) - model) <= steps * S + steps


def test_append_writes_rows_and_bumps_lengths():
    st, qs, kn, vn = _tiny_state(19)
    st.full(qs[0])
    l0, s0 = st.len_full, st.len_small
    for t in range(1, 4):
        st.append(kn[t], vn[t])
    assert st.len_full == l0 + 3 and st.len_small == s0 + 3
    for t in range(1, 4):
        assert np.array_equal(st.k_full[:, l0 + t - 1], kn[t])
        assert np.array_equal(st.v_full[:, l0 + t - 1], vn[t])
        for g in range(2):
            assert np.array_equal(st.k_small[g][s0 + t - 1], kn[t][g])
            assert st.small_pos[g][s0 + t - 1] == l0 + t - 1


def test_never_refreshing_keeps_the_context_part_fixed():
    """Without refresh the context part of C_p stays what the first selection chose (the SnapKV case)."""
    st, qs, kn, vn = _tiny_state(20, steps=5)
    st.full(qs[0])
    first = [p.copy() for p in st.small_pos]
    for t in range(1, 6):
        st.append(kn[t], vn[t])
        st.small(qs[t])
    for g in range(2):
        assert np.array_equal(st.small_pos[g][: len(first[g])], first[g])
        assert st.small_pos[g][len(first[g]):].tolist() == list(range(24, 29))


def test_generated_tokens_compete_in_later_selections():
    st, qs, kn, vn = _tiny_state(21, ctx=8, k_small=8, steps=4)
    trace = O.run_fixed_stride(st, qs, kn, vn, 4)
    assert trace[-1][0] == "full"
    # K = 8 of 12 positions: make sure appended positions (>= 8) can be selected at all
    allpos = np.concatenate(st.small_pos)
    assert allpos.max() < 12 and st.len_small == 8


def test_dynamic_schedule_follows_the_trigger():
    st, qs, kn, vn = _tiny_state(22, steps=6)
    # identical queries: cos = 1 > s -> never refresh after the initial step
    same = [qs[0]] * 7
    kinds = [k for k, _ in O.run_dynamic(st, same, kn, vn, 2, 0.9)]
    assert kinds == ["small"] * 6
    # independent random queries: cos ~ 0 < s -> refresh at every check step (t even), never in between
    st2, qs2, kn2, vn2 = _tiny_state(23, steps=6)
    kinds = [k for k, _ in O.run_dynamic(st2, qs2, kn2, vn2, 2, 0.9)]
    assert kinds == ["small", "full"] * 3


# ------------------------------------------------------------------ mutation checks: the pins bite
def test_pins_catch_planted_mistakes():
    """Plant plausible mistakes in a copy of the oracle's steps and check that a pin above notices."""
    q, k, v = _rand_case(24, n_q=4, n_kv=2, n=31, d=128)
    good, p, _ = O.decode_attention(q, k, v)
    # (1) dropped scale
    bad, _, _ = O.decode_attention(q, k, v, scale=1.0)
    assert not np.allclose(good, bad, atol=1e-6)
    # (2) wrong grouping (interleaved instead of contiguous)
    tk = torch.from_numpy(k).repeat(2, 1, 1)[None]
    tv = torch.from_numpy(v).repeat(2, 1, 1)[None]
    inter = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(q)[None, :, None, :], tk, tv)[0, :, 0].numpy()
    assert not np.allclose(good, inter, atol=1e-6)
    # (3) ascending instead of descending selection loses total score
    score = O.aggregate_scores(p, 2)[0]
    assert score[np.argsort(score)[:5]].sum() < score[O.top_k_positions(score, 5)].sum()
    # (4) cosine of per-head vectors averaged afterwards differs from cosine of the averaged vector
    r = _rng(25)
    a, b = r.normal(size=(4, 8)), r.normal(size=(4, 8))
    per_head = np.mean([a[h] @ b[h] / np.linalg.norm(a[h]) / np.linalg.norm(b[h]) for h in range(4)])
    assert abs(per_head - O.cosine_similarity(a, b)) > 1e-3


def test_score_only_step_pins():
    """Sec. 4.2 "w/o full attention": same selection as the full step; output = attention over the selected rows.
    With K = L it is the full step; with one dominant key the two outputs nearly coincide."""
    q, k, v = _rand_case(31, n_q=4, n_kv=2, n=40, d=128)
    full_out, score, idx, _ = O.full_step(q, k, v, 9)
    out, score2, idx2 = O.score_only_step(q, k, v, 9)
    assert all(np.array_equal(a, b) for a, b in zip(idx, idx2)) and np.array_equal(score, score2)
    assert not np.allclose(out, full_out, atol=1e-6)          # 9 of 40 positions: a different softmax
    out_all, _, _ = O.score_only_step(q, k, v, 40)
    assert np.allclose(out_all, full_out, atol=1e-12)
    # renormalised probabilities over the kept set: by hand for head 0
    p = O.softmax_rows(O.attention_logits(q, k))[0][0]
    keep = idx[0]
    want = (p[keep] / p[keep].sum()) @ v[0, keep]
    assert np.allclose(out[0], want, atol=1e-12)


def test_fixed_size_small_cache_evicts_the_lowest_score_first():
    """Sec. 2.2 "Decoding with partial cache": |C_p| stays K; each new token replaces the entry with the lowest
    score of the last full step.  Hand-checkable case: one head, keys aligned with the query by known amounts."""
    d = 128
    q = np.zeros((1, d)); q[0, 0] = math.sqrt(d)                 # logit of position j = k[j, 0]
    levels = [0.0, 3.0, 1.0, 5.0, 2.0, 4.0]                      # scores order: pos 3 > 5 > 1 > 4 > 2 > 0
    k = np.zeros((1, 8, d)); k[0, :6, 0] = levels
    v = np.zeros((1, 8, d)); v[0, :6, 1] = np.arange(6)
    st = O.SequenceState(O.f64_to_bf16_bits(k), O.f64_to_bf16_bits(v), 6, 3, evict=True)
    st.full(O.f64_to_bf16_bits(q))
    assert st.small_pos[0].tolist() == [3, 5, 1] and st.len_small == 3
    new_k, new_v = O.f64_to_bf16_bits(np.ones((1, d))), O.f64_to_bf16_bits(np.full((1, d), 9.0))
    st.append(new_k, new_v)                                       # victim: position 1 (lowest of the three)
    assert st.len_small == 3 and sorted(st.small_pos[0].tolist()) == [3, 5, 6]
    st.append(new_k, new_v)                                       # next victim: position 5, never the new token
    assert st.len_small == 3 and sorted(st.small_pos[0].tolist()) == [3, 6, 7] and st.len_full == 8
    assert np.array_equal(st.k_small[0][st.small_pos[0].tolist().index(6)], new_k[0])
    # without eviction the same two appends grow the cache
    st2 = O.SequenceState(O.f64_to_bf16_bits(k), O.f64_to_bf16_bits(v), 6, 3)
    st2.full(O.f64_to_bf16_bits(q)); st2.append(new_k, new_v); st2.append(new_k, new_v)
    assert st2.len_small == 5
    # equal scores: the later position is dropped first
    k3 = np.zeros((1, 6, d)); k3[0, :4, 0] = [2.0, 2.0, 2.0, 0.0]
    st3 = O.SequenceState(O.f64_to_bf16_bits(k3), O.f64_to_bf16_bits(np.zeros((1, 6, d))), 4, 3, evict=True)
    st3.full(O.f64_to_bf16_bits(q)); st3.append(new_k, new_v)
    assert sorted(st3.small_pos[0].tolist()) == [0, 1, 4]


def test_fixed_size_cache_matches_the_cost_model_exactly(golden_dir):
    """With eviction a partial step touches exactly K positions: T steps at stride S cost
    (T/S) full steps over the context plus K per partial step - the T*L/S + T*K form of App. A.2 without the
    growth term of the growing cache."""
    T, L, K, S = 12, 40, 6, 4
    q, k, v = _rand_case(41, n_q=2, n_kv=1, n=L + T + 1, d=128)
    kb, vb = O.f64_to_bf16_bits(k), O.f64_to_bf16_bits(v)
    st = O.SequenceState(kb.copy(), vb.copy(), L, K, evict=True)
    qs = [O.f64_to_bf16_bits(q + 0.01 * t) for t in range(T + 1)]
    O.run_fixed_stride(st, qs, [kb[:, L + t] for t in range(T + 1)], [vb[:, L + t] for t in range(T + 1)], S)
    n_full, n_small = T // S, T - T // S
    assert st.n_full_steps == n_full + 1 and st.n_small_steps == n_small and st.len_small == K
    full_part = L + sum(L + t for t in range(1, T + 1) if t % S == 0)
    assert st.positions_touched == full_part + n_small * K
