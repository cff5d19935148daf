"""fp64 CPU oracle for the RefreshKV decode-attention hot path.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, obviously-correct
statement of what the CUDA library must compute.  It shares no code, tables
or helpers with the CUDA path and is imported only by the tests, by the smoke
check and by the CPU-baseline leg of the benchmark.  Nothing in the product
path may call it.

Everything is float64 numpy.  bf16 inputs arrive as uint16 bit patterns and
are widened exactly (bf16 -> fp64 is lossless), so the oracle sees the very
numbers the GPU kernels read.

Paper passages followed (arXiv 2411.05787, "RefreshKV"):
  * Sec. 2.1  - decode step: the model attends to the tokens in the KV cache
                and then adds the current token's key/value to the cache.
  * Sec. 2.2 "Prefilling stage" + its footnote - attention scores a_L of the
                current token; for grouped-query attention the scores of all
                query heads of a group are aggregated by max (mean / first
                head are the ablation modes of App. A.3, Table 6); optional
                max-pooling over neighbouring positions (kernel 7, App. A.1).
  * Sec. 2.2 "Decoding with full cache"   - attend over C_f, take a_L, rebuild
                C_p from the top-K positions of a_L.
  * Sec. 2.2 "Decoding with partial cache" - attend over C_p, append the new
                token's K/V to C_p.
  * Sec. 2.2 "Deciding when to decode with full cache" - fixed stride S, or
                cosine similarity of the head-averaged query against the one
                of the latest full step, compared with threshold s every
                QC-th step: similarity higher than s -> partial step,
                otherwise full step.
  * App. A.2, Table 5 - attention cost T*L/S + T*K, cache memory L + K.

Parity pins: every function below is pinned by tests/test_oracle_*.py
(closed forms, an independent library routine, brute force on tiny inputs,
hand-worked fixtures under tests/golden/).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

HEAD_DIM = 128


# --------------------------------------------------------------------------
# number formats
# --------------------------------------------------------------------------
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to float64, exactly.

    A bf16 value is the upper half of an IEEE binary32, so placing the 16
    bits in the high half of a uint32 and reinterpreting gives the value.
    """
    bits = np.asarray(bits)
    if bits.dtype != np.uint16:
        raise TypeError("bf16 tensors are passed to the oracle as uint16 bit patterns")
    as_f32 = (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)
    with np.errstate(invalid="ignore"):      # signalling-NaN patterns widen to NaN silently
        return as_f32.astype(np.float64)


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float64 to bf16 (round-to-nearest-even), return uint16 bits.

    Used only to build inputs inside oracle-side tests; finite inputs only.
    """
    f32 = np.asarray(x, dtype=np.float64).astype(np.float32)
    u = f32.view(np.uint32).astype(np.uint64)
    rounded = u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))
    return (rounded >> np.uint64(16)).astype(np.uint16)


# --------------------------------------------------------------------------
# attention over one sequence (Sec. 2.1; Sec. 2.2 full / partial decoding)
# --------------------------------------------------------------------------
def attention_logits(q: np.ndarray, k: np.ndarray, scale: float | None = None) -> np.ndarray:
    """s[h, j] = scale * sum_c q[h, c] * k[g(h), j, c],  g(h) = h // G.

    q: [Hq, d] float64, k: [Hkv, n, d] float64.  Query heads gG..gG+G-1 share
    KV head g (contiguous grouping).  scale defaults to 1/sqrt(d).
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    n_q, d = q.shape
    n_kv, n, d2 = k.shape
    if d != d2 or n_q % n_kv != 0:
        raise ValueError("shape mismatch")
    group = n_q // n_kv
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    s = np.empty((n_q, n), dtype=np.float64)
    for h in range(n_q):
        s[h] = scale * (k[h // group] @ q[h])
    return s


def softmax_rows(s: np.ndarray) -> tuple[np.ndarray, np.ndarray]:
    """p[h, j] = exp(s[h, j] - m_h) / Z_h and LSE_h = m_h + ln Z_h."""
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    z = e.sum(axis=1, keepdims=True)
    return e / z, (m + np.log(z))[:, 0]


def decode_attention(q, k, v, scale=None):
    """One decode step of softmax attention over n cached positions.

    Returns (out [Hq, d], p [Hq, n], lse [Hq]);  out[h] = sum_j p[h, j] v[g(h), j].
    """
    v = np.asarray(v, dtype=np.float64)
    s = attention_logits(q, k, scale)
    p, lse = softmax_rows(s)
    n_q = p.shape[0]
    group = n_q // v.shape[0]
    out = np.empty((n_q, v.shape[2]), dtype=np.float64)
    for h in range(n_q):
        out[h] = p[h] @ v[h // group]
    return out, p, lse


# --------------------------------------------------------------------------
# score aggregation, pooling, top-K (Sec. 2.2 prefilling stage + footnote)
# --------------------------------------------------------------------------
def aggregate_scores(p: np.ndarray, n_kv: int, mode: str = "max") -> np.ndarray:
    """Collapse the G query heads of each KV group: [Hq, n] -> [Hkv, n].

    mode "max" is the paper's rule; "mean" and "first" are its ablations.
    """
    n_q, n = p.shape
    group = n_q // n_kv
    grouped = p.reshape(n_kv, group, n)
    if mode == "max":
        return grouped.max(axis=1)
    if mode == "mean":
        return grouped.mean(axis=1)
    if mode == "first":
        return grouped[:, 0, :].copy()
    raise ValueError(mode)


def pool_max(score: np.ndarray, width: int) -> np.ndarray:
    """1-D max-pool along positions, odd window `width`, window clipped at the ends.

    pooled[j] = max over i with |i - j| <= (width - 1) / 2 and 0 <= i < n.
    width = 1 is the identity.
    """
    if width < 1 or width % 2 == 0:
        raise ValueError("pool width must be odd and positive")
    half = (width - 1) // 2
    n = score.shape[-1]
    pooled = np.empty_like(score)
    for j in range(n):
        lo = max(0, j - half)
        hi = min(n, j + half + 1)
        pooled[..., j] = score[..., lo:hi].max(axis=-1)
    return pooled


def top_k_positions(score_row: np.ndarray, k: int) -> np.ndarray:
    """The min(k, n) positions of largest score; ties go to the lower index.

    Returned in rank order (score descending, index ascending).
    """
    n = score_row.shape[0]
    take = max(0, min(int(k), n))
    # sort by score descending; a stable sort keeps lower indices first among ties
    order = np.argsort(-score_row, kind="stable")
    return order[:take].astype(np.int64)


def full_step(q, k, v, k_small_size, *, agg="max", pool=1, scale=None):
    """Full-cache step: out, aggregated (pooled) scores [Hkv, n], top-K per KV head."""
    out, p, lse = decode_attention(q, k, v, scale)
    score = aggregate_scores(p, k.shape[0], agg)
    if pool > 1:
        score = pool_max(score, pool)
    idx = [top_k_positions(score[g], k_small_size) for g in range(k.shape[0])]
    return out, score, idx, lse


def score_only_step(q, k, v, k_small_size, *, agg="max", pool=1, scale=None):
    """The "w/o full attention" refresh of Sec. 4.2: scores over the whole cache pick the top-K positions,
    and the step's output is attention over those K positions only.  Returns (out, score, idx)."""
    _, score, idx, _ = full_step(q, k, v, k_small_size, agg=agg, pool=pool, scale=scale)
    v = np.asarray(v, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    ks = np.stack([k[g, idx[g]] for g in range(k.shape[0])])
    vs = np.stack([v[g, idx[g]] for g in range(k.shape[0])])
    out, _, _ = decode_attention(q, ks, vs, scale)
    return out, score, idx


def gather_rows(cache: np.ndarray, idx: list[np.ndarray]) -> list[np.ndarray]:
    """small[g][r] = cache[g, idx[g][r]] (bit copy; works on uint16 or float arrays)."""
    return [cache[g, idx[g]] for g in range(cache.shape[0])]


# --------------------------------------------------------------------------
# refresh trigger and schedule (Sec. 2.2 "Deciding when ...", Fig. 1 caption)
# --------------------------------------------------------------------------
def mean_query(q: np.ndarray) -> np.ndarray:
    return np.asarray(q, dtype=np.float64).mean(axis=0)


def cosine_similarity(q_now: np.ndarray, q_last_full: np.ndarray) -> float:
    """cos between the head-averaged query now and at the latest full step."""
    a = mean_query(q_now)
    b = mean_query(q_last_full)
    na = math.sqrt(float(a @ a))
    nb = math.sqrt(float(b @ b))
    if na == 0.0 or nb == 0.0:
        return float("nan")
    return float(a @ b) / (na * nb)


def should_refresh(q_now, q_last_full, threshold: float) -> tuple[int, float]:
    """flag = 1 (take a full step) unless the similarity is higher than the threshold.

    Equality and NaN (a zero mean query) both give 1.
    """
    cos = cosine_similarity(q_now, q_last_full)
    return (0 if cos > threshold else 1), cos


def fixed_stride_is_full(t: int, stride: int) -> bool:
    """Decode steps are counted from 1; every stride-th step is a full step."""
    return t % stride == 0


# --------------------------------------------------------------------------
# per-sequence state machine: both caches of one layer of one sequence
# --------------------------------------------------------------------------
@dataclass
class SequenceState:
    """C_f and C_p of one (layer, sequence).  K/V kept as bf16 bit patterns.

    k_full, v_full: uint16 [Hkv, cap, d]; len_full positions valid.
    k_small, v_small: per KV head uint16 [cap_small, d]; len_small rows valid.
    By default the small cache grows by one row per appended token until the
    next refresh.  With evict=True it keeps the paper's fixed size (Sec. 2.2
    "Decoding with partial cache"): once it holds k_small_size rows, each new
    token replaces the surviving entry that had the lowest attention score in
    the last full step (among equal scores the later position goes first);
    tokens appended since that step carry no score and are never the victim.
    """
    k_full: np.ndarray
    v_full: np.ndarray
    len_full: int
    k_small_size: int
    agg: str = "max"
    pool: int = 1
    evict: bool = False
    evict_queue: list = field(default_factory=list)   # per KV head: small-cache rows in eviction order
    k_small: list = field(default_factory=list)
    v_small: list = field(default_factory=list)
    small_pos: list = field(default_factory=list)   # position in C_f of every small row
    len_small: int = 0
    q_last_full: np.ndarray | None = None
    positions_touched: int = 0
    n_full_steps: int = 0
    n_small_steps: int = 0

    def append(self, k_new: np.ndarray, v_new: np.ndarray, to_small: bool = True):
        """Write the new token's K/V (uint16 [Hkv, d]) at the end of both caches."""
        if self.len_full >= self.k_full.shape[1]:
            raise IndexError("full cache capacity exceeded")
        self.k_full[:, self.len_full] = k_new
        self.v_full[:, self.len_full] = v_new
        if to_small and self.k_small and self.evict and self.len_small >= self.k_small_size > 0:
            for g in range(self.k_full.shape[0]):
                slot = self.evict_queue[g].pop(0)          # lowest-scoring survivor of the last full step
                self.k_small[g][slot] = k_new[g]
                self.v_small[g][slot] = v_new[g]
                self.small_pos[g][slot] = self.len_full
        elif to_small and self.k_small:
            for g in range(self.k_full.shape[0]):
                self.k_small[g] = np.concatenate([self.k_small[g], k_new[g][None]], axis=0)
                self.v_small[g] = np.concatenate([self.v_small[g], v_new[g][None]], axis=0)
                self.small_pos[g] = np.concatenate([self.small_pos[g], [self.len_full]])
            self.len_small += 1
        self.len_full += 1

    def full(self, q_bits: np.ndarray):
        """Full step on the current query (uint16 [Hq, d]); rebuilds C_p."""
        q = bf16_bits_to_f64(q_bits)
        k = bf16_bits_to_f64(self.k_full[:, : self.len_full])
        v = bf16_bits_to_f64(self.v_full[:, : self.len_full])
        out, score, idx, lse = full_step(q, k, v, self.k_small_size, agg=self.agg, pool=self.pool)
        self.k_small = gather_rows(self.k_full, idx)
        self.v_small = gather_rows(self.v_full, idx)
        self.small_pos = [i.copy() for i in idx]
        self.len_small = len(idx[0])
        # rows are in rank order (score descending, position ascending): the victims come from the back
        self.evict_queue = [list(range(len(i) - 1, -1, -1)) for i in idx]
        self.q_last_full = q
        self.positions_touched += self.len_full
        self.n_full_steps += 1
        return out, score, idx

    def small(self, q_bits: np.ndarray):
        """Partial step: attention over C_p only."""
        q = bf16_bits_to_f64(q_bits)
        k = bf16_bits_to_f64(np.stack(self.k_small))
        v = bf16_bits_to_f64(np.stack(self.v_small))
        out, _, _ = decode_attention(q, k, v)
        self.positions_touched += self.len_small
        self.n_small_steps += 1
        return out


def run_fixed_stride(state: SequenceState, q_steps, k_steps, v_steps, stride: int):
    """Drive one sequence for T steps with a fixed stride.

    q_steps[0] initialises C_p by a full step at t = 0 (stand-in for the
    prefill initialisation); then for t = 1..T: append the token's K/V,
    full step iff t % stride == 0, else partial step.  Returns the list of
    (kind, out) per step t >= 1.
    """
    state.full(q_steps[0])
    trace = []
    for t in range(1, len(q_steps)):
        state.append(k_steps[t], v_steps[t])
        if fixed_stride_is_full(t, stride):
            out, _, _ = state.full(q_steps[t])
            trace.append(("full", out))
        else:
            trace.append(("small", state.small(q_steps[t])))
    return trace


def run_dynamic(state: SequenceState, q_steps, k_steps, v_steps, qc_stride: int, threshold: float):
    """Dynamic schedule: at every qc_stride-th step evaluate the trigger."""
    state.full(q_steps[0])
    trace = []
    for t in range(1, len(q_steps)):
        state.append(k_steps[t], v_steps[t])
        flag = 0
        if t % qc_stride == 0:
            flag, _ = should_refresh(bf16_bits_to_f64(q_steps[t]), state.q_last_full, threshold)
        if flag:
            out, _, _ = state.full(q_steps[t])
            trace.append(("full", out))
        else:
            trace.append(("small", state.small(q_steps[t])))
    return trace


# --------------------------------------------------------------------------
# cost model (App. A.2, Table 5)
# --------------------------------------------------------------------------
def attention_cost_refreshkv(t_new: int, ctx_len: int, k_small: int, stride: int) -> float:
    return t_new * ctx_len / stride + t_new * k_small


def attention_cost_vanilla(t_new: int, ctx_len: int) -> float:
    return float(t_new * ctx_len)


# --------------------------------------------------------------------------
# acceptance rule for a top-K set that need not equal the oracle's exactly
# --------------------------------------------------------------------------
def check_topk_set(score_row: np.ndarray, k: int, got: np.ndarray, rel_band: float = 1e-5) -> str | None:
    """Return None if `got` is an acceptable top-k set for `score_row`, else why not.

    Acceptable: min(k, n) distinct in-range indices; contains every position
    whose score exceeds tau*(1+band); contains no position whose score is
    below tau*(1-band); tau = the k-th largest oracle score.
    """
    n = score_row.shape[0]
    take = min(int(k), n)
    got = np.asarray(got).astype(np.int64)
    if got.shape[0] != take:
        return f"expected {take} indices, got {got.shape[0]}"
    if take == 0:
        return None
    if got.min() < 0 or got.max() >= n:
        return "index out of range"
    if np.unique(got).shape[0] != take:
        return "duplicate indices"
    ref = top_k_positions(score_row, take)
    tau = score_row[ref[-1]]
    must = np.nonzero(score_row > tau * (1.0 + rel_band))[0]
    chosen = np.zeros(n, dtype=bool)
    chosen[got] = True
    if not chosen[must].all():
        return f"missing {int((~chosen[must]).sum())} positions that are clearly above the threshold"
    low = score_row[got] < tau * (1.0 - rel_band)
    if low.any():
        return f"{int(low.sum())} chosen positions are clearly below the threshold"
    return None
