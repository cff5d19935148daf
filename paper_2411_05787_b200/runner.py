"""Per-layer decode state on the GPU: both caches of a layer plus the buffers the calls write.

A convenience wrapper over the C-ABI calls (rkv.Context).  It allocates device
tensors with torch and sequences the calls of one decode step; every
computation happens inside librkv.
"""
from __future__ import annotations

import torch

from . import rkv
from .synth import HEAD_DIM, LayerCache, alloc_cache


class LayerState:
    """C_f and C_p of one layer for a batch of sequences, and the step calls on them."""

    def __init__(self, ctx: rkv.Context, full: LayerCache, k_small: list, small_extra: int, n_q_heads: int,
                 n_kv_heads: int, want_scores: bool = False):
        dev = full.k.device
        self.ctx, self.full = ctx, full
        self.n_seq, self.n_q, self.n_kv = len(k_small), n_q_heads, n_kv_heads
        self.k_max = max(max(k_small), 1)
        self.k_small = torch.tensor(k_small, dtype=torch.int32, device=dev)
        self.small = alloc_cache([k + small_extra for k in k_small], [0] * self.n_seq, n_kv_heads, dev, fill=0.0)
        self.full_c = rkv.cache_struct(full.k, full.v, full.row_offset, full.cap, full.len)
        self.small_c = rkv.cache_struct(self.small.k, self.small.v, self.small.row_offset, self.small.cap,
                                        self.small.len)
        self.out = torch.zeros((self.n_seq, n_q_heads, HEAD_DIM), dtype=torch.bfloat16, device=dev)
        self.topk_idx = torch.full((self.n_seq, n_kv_heads, self.k_max), -2, dtype=torch.int32, device=dev)
        self.q_last_full = torch.zeros((self.n_seq, n_q_heads, HEAD_DIM), dtype=torch.bfloat16, device=dev)
        self.flag = torch.zeros((self.n_seq,), dtype=torch.int32, device=dev)
        self.not_flag = torch.zeros((self.n_seq,), dtype=torch.int32, device=dev)
        self.sim = torch.zeros((self.n_seq,), dtype=torch.float32, device=dev)
        self.scores = None
        if want_scores:
            stride = int(full.cap.max().item())
            self.scores = torch.zeros((self.n_seq, n_kv_heads, stride), dtype=torch.float32, device=dev)

    def enable_eviction(self, max_evict: int):
        """Fixed-size small cache: allocate the eviction order and counter that the *_evict calls keep."""
        dev = self.out.device
        self.evict_order = torch.full((self.n_seq, self.n_kv, max_evict), -1, dtype=torch.int32, device=dev)
        self.evict_count = torch.zeros((self.n_seq,), dtype=torch.int32, device=dev)

    def refresh_evict(self, q, active=None, max_len_hint=0):
        """Full step, rebuild of the small cache and its eviction order."""
        self.ctx.full_step(q, self.full_c, self.k_small, self.k_max, self.out, self.topk_idx, active=active,
                           scores=self.scores, q_last_full=self.q_last_full, max_len_hint=max_len_hint)
        self.ctx.gather_small_evict(self.topk_idx, self.k_small, self.k_max, self.full_c, self.small_c,
                                    self.evict_order, self.evict_count, active=active)
        return self.out

    def append_partial_evict(self, q, k_new, v_new, active=None, max_len_hint=0):
        self.ctx.append_small_step_evict(q, k_new, v_new, self.full_c, self.small_c, self.k_small, self.out,
                                         self.evict_order, self.evict_count, active=active, max_len_hint=max_len_hint)
        return self.out

    def refresh(self, q, active=None, max_len_hint=0):
        """Full step followed by the rebuild of the small cache."""
        self.ctx.full_step(q, self.full_c, self.k_small, self.k_max, self.out, self.topk_idx, active=active,
                           scores=self.scores, q_last_full=self.q_last_full, max_len_hint=max_len_hint)
        self.ctx.gather_small(self.topk_idx, self.k_small, self.k_max, self.full_c, self.small_c, active=active)
        return self.out

    def refresh_attention(self, q, active=None, max_len_hint=0, stream=None):
        """First half of a refresh: attention over the full cache; out is final when this call's kernel ends."""
        self.ctx.full_attention(q, self.full_c, self.out, active=active, max_len_hint=max_len_hint, stream=stream)
        return self.out

    def append_refresh_attention(self, q, k_new, v_new, active=None, max_len_hint=0, stream=None):
        """Append to the full cache and attend over it, one launch (the refresh rebuilds the small cache anyway)."""
        self.ctx.append_full_attention(q, k_new, v_new, self.full_c, self.out, active=active,
                                       max_len_hint=max_len_hint, stream=stream)
        return self.out

    def refresh_select(self, q, active=None, stream=None):
        """Second half: scores, top-K and the rebuild of the small cache from what refresh_attention left."""
        self.ctx.select_topk(q, self.full_c, self.k_small, self.k_max, self.topk_idx, active=active,
                             scores=self.scores, q_last_full=self.q_last_full, stream=stream)
        self.ctx.gather_small(self.topk_idx, self.k_small, self.k_max, self.full_c, self.small_c, active=active,
                              stream=stream)

    def refresh_score_keys(self, q, active=None, stream=None):
        """Second half, first launch: scores, keys and histogram (and q_last_full) from the logits of refresh_attention."""
        self.ctx.score_keys(q, self.full_c, self.k_small, self.k_max, active=active, scores=self.scores,
                            q_last_full=self.q_last_full, stream=stream)

    def refresh_select_only(self, active=None, stream=None):
        """Second half, second launch after refresh_score_keys: top-K, then the rebuild of the small cache."""
        self.ctx.select_topk(None, self.full_c, self.k_small, self.k_max, self.topk_idx, active=active, stream=stream)
        self.ctx.gather_small(self.topk_idx, self.k_small, self.k_max, self.full_c, self.small_c, active=active,
                              stream=stream)

    def refresh_scores_only(self, q, active=None, max_len_hint=0, small_hint=0):
        """Score-only refresh: scores and top-K from K alone, rebuild of the small cache, attention over the new one."""
        self.ctx.score_step(q, self.full_c, self.k_small, self.k_max, self.topk_idx, active=active, scores=self.scores,
                            q_last_full=self.q_last_full, max_len_hint=max_len_hint)
        self.ctx.gather_small(self.topk_idx, self.k_small, self.k_max, self.full_c, self.small_c, active=active)
        self.ctx.small_step(q, self.small_c, self.out, active=active, max_len_hint=small_hint)
        return self.out

    def partial(self, q, active=None, max_len_hint=0):
        self.ctx.small_step(q, self.small_c, self.out, active=active, max_len_hint=max_len_hint)
        return self.out

    def append_partial(self, q, k_new, v_new, active=None, max_len_hint=0):
        """Append to both caches and attend over the small cache, in one call."""
        self.ctx.append_small_step(q, k_new, v_new, self.full_c, self.small_c, self.out, active=active,
                                   max_len_hint=max_len_hint)
        return self.out

    def append(self, k_new, v_new):
        self.ctx.append(k_new, v_new, self.full_c, self.small_c)

    def check_trigger(self, q, threshold):
        self.ctx.should_refresh(q, self.q_last_full, threshold, self.flag, self.sim, keep=self.not_flag)
        return self.flag


class OverlappedRefresh:
    """Full-step token over a stack of layers with the selection off the layers' critical path.

    What layer l + 1 needs from layer l is its attention output, which is final when rkv_full_attention's kernel
    ends; the selection and the rebuild of the small cache are first needed by the NEXT token.  The attention
    passes of all layers follow each other in the calling stream; each layer's selection and rebuild run in a
    second stream behind its attention and overlap the next layers' attention.  Consecutive layers must use
    different contexts (a context's workspace holds one attention pass): with two contexts that alternate, a
    workspace is reused two layers later, after an event has said that the selection reading it has ended."""

    def __init__(self, layers, priority=0):
        self.layers = layers
        for a, b in zip(layers, layers[1:]):
            if a.ctx is b.ctx:
                raise ValueError("consecutive layers must not share a context")
        for a, c in zip(layers, layers[2:]):
            if a.ctx is not c.ctx:
                raise ValueError("layers two apart must share a context (two contexts, alternating)")
        self.side = torch.cuda.Stream(priority=priority)
        self.ev_attn = [torch.cuda.Event() for _ in layers]
        self.ev_sel = [torch.cuda.Event() for _ in layers]

    def run(self, q_of, k_new_of, v_new_of, max_len_hint=0):
        """q_of(l), k_new_of(l), v_new_of(l): the layer's inputs.  Appends, attends, selects, rebuilds."""
        main = torch.cuda.current_stream()
        n = len(self.layers)
        for l, st in enumerate(self.layers):
            if l >= 2:
                main.wait_event(self.ev_sel[l - 2])
            st.append_refresh_attention(q_of(l), k_new_of(l), v_new_of(l), max_len_hint=max_len_hint)
            self.ev_attn[l].record(main)
            self.side.wait_event(self.ev_attn[l])
            with torch.cuda.stream(self.side):
                st.refresh_select(q_of(l))
                self.ev_sel[l].record(self.side)
        for l in range(max(n - 2, 0), n):
            main.wait_event(self.ev_sel[l])

    def run_checked(self, q_of, k_new_of, v_new_of, threshold, small_hint=0, full_hint=0, after_trigger=None):
        """Token of the dynamic schedule at a check position: per layer the trigger, then both branches under its
        device masks - the partial step (which appends to both caches for every sequence) for the sequences that
        keep their small cache, the full step for those that refresh - with the full step's selection and rebuild
        behind the attention in the second stream, as in run()."""
        main = torch.cuda.current_stream()
        n = len(self.layers)
        for l, st in enumerate(self.layers):
            if l >= 2:
                main.wait_event(self.ev_sel[l - 2])
            st.check_trigger(q_of(l), threshold)
            if after_trigger is not None:
                after_trigger(l, st)
            st.append_partial(q_of(l), k_new_of(l), v_new_of(l), active=st.not_flag, max_len_hint=small_hint)
            st.refresh_attention(q_of(l), active=st.flag, max_len_hint=full_hint)
            self.ev_attn[l].record(main)
            self.side.wait_event(self.ev_attn[l])
            with torch.cuda.stream(self.side):
                st.refresh_select(q_of(l), active=st.flag)
                self.ev_sel[l].record(self.side)
        for l in range(max(n - 2, 0), n):
            main.wait_event(self.ev_sel[l])



class DeferredRefresh:
    """Full-step token over a stack of layers with every layer's selection and rebuild AFTER the last attention pass.

    The refreshed small cache of a layer is first read by the NEXT token's partial step, so nothing forces the
    selection to run beside the following layers' attention, where its CTAs displace attention CTAs and unbalance
    their single wave.  Here the attention passes of all layers follow each other undisturbed in the calling stream;
    then the layers' selections and rebuilds run, spread over a few side streams so that several of these short,
    latency-bound kernel chains are in flight at once.  Every layer needs a context of its own: its logits stay in
    the context's workspace until its selection runs."""

    def __init__(self, layers, n_side=16, select_keys_per_cta=16384, score_slice=4096, early_scores=False):
        self.layers = layers
        # early_scores: every layer's score pass runs right behind its attention pass, in a stream of its own beside
        # the next layer's attention (its logits are then still in L2); only top-K and rebuild wait for the tail
        self.early_scores = early_scores
        self.score_stream = torch.cuda.Stream() if early_scores else None
        self.ev_layer = [torch.cuda.Event() for _ in layers] if early_scores else None
        self.ev_scores = torch.cuda.Event() if early_scores else None
        ctxs = [id(st.ctx) for st in layers]
        if len(set(ctxs)) != len(ctxs):
            raise ValueError("every layer needs its own context (the workspace holds its logits until the token's end)")
        self.sides = [torch.cuda.Stream() for _ in range(max(1, min(n_side, len(layers))))]
        self.ev_attn = torch.cuda.Event()
        self.ev_done = [torch.cuda.Event() for _ in self.sides]
        # With many layers, many selections run side by side, and what counts is the SM time each takes, not the
        # length of its own chain: few large CTAs per score pass and per top-K cluster (0: leave the contexts'
        # settings alone, as is done for a handful of layers, whose selections are still latency-bound).
        many = len(layers) >= 8
        self.tuning = [(rkv.OPT_SELECT_KEYS_PER_CTA, select_keys_per_cta if many else 0),
                       (rkv.OPT_SCORE_SLICE, score_slice if many else 0)]

    def _set_tuning(self):
        saved = {}
        for st in self.layers:
            saved[id(st.ctx)] = [(opt, st.ctx.get_option(opt)) for opt, val in self.tuning if val]
            for opt, val in self.tuning:
                if val:
                    st.ctx.set_option(opt, val)
        return saved

    def _restore_tuning(self, saved):
        for st in self.layers:
            for opt, val in saved[id(st.ctx)]:
                st.ctx.set_option(opt, val)

    def _tail(self, main, select_of, wait_for=()):
        """After the attention passes: every layer's selection and rebuild, dealt out to the side streams."""
        self.ev_attn.record(main)
        for i, side in enumerate(self.sides):
            side.wait_event(self.ev_attn)
            for ev in wait_for:
                side.wait_event(ev)
            with torch.cuda.stream(side):
                for l in range(i, len(self.layers), len(self.sides)):
                    select_of(l, self.layers[l])
                self.ev_done[i].record(side)
        for ev in self.ev_done:
            main.wait_event(ev)

    def run(self, q_of, k_new_of, v_new_of, max_len_hint=0):
        """q_of(l), k_new_of(l), v_new_of(l): the layer's inputs.  Appends, attends; then selects and rebuilds."""
        main = torch.cuda.current_stream()
        saved = self._set_tuning()
        if not self.early_scores:
            for l, st in enumerate(self.layers):
                st.append_refresh_attention(q_of(l), k_new_of(l), v_new_of(l), max_len_hint=max_len_hint)
            self._tail(main, lambda l, st: st.refresh_select(q_of(l)))
        else:
            for l, st in enumerate(self.layers):
                st.append_refresh_attention(q_of(l), k_new_of(l), v_new_of(l), max_len_hint=max_len_hint)
                self.ev_layer[l].record(main)
                self.score_stream.wait_event(self.ev_layer[l])
                st.refresh_score_keys(q_of(l), stream=self.score_stream)
            self.ev_scores.record(self.score_stream)
            self._tail(main, lambda l, st: st.refresh_select_only(), wait_for=(self.ev_scores,))
        self._restore_tuning(saved)

    def run_checked(self, q_of, k_new_of, v_new_of, threshold, small_hint=0, full_hint=0, after_trigger=None):
        """Token of the dynamic schedule at a check position: per layer the trigger, then both branches under its
        device masks (the partial step, which appends to both caches for every sequence, for the sequences that keep
        their small cache; the full step's attention for those that refresh); the selections and rebuilds of the
        refreshing sequences follow after the last layer, as in run()."""
        main = torch.cuda.current_stream()
        for l, st in enumerate(self.layers):
            st.check_trigger(q_of(l), threshold)
            if after_trigger is not None:
                after_trigger(l, st)
            st.append_partial(q_of(l), k_new_of(l), v_new_of(l), active=st.not_flag, max_len_hint=small_hint)
            st.refresh_attention(q_of(l), active=st.flag, max_len_hint=full_hint)
        saved = self._set_tuning()
        self._tail(main, lambda l, st: st.refresh_select(q_of(l), active=st.flag))
        self._restore_tuning(saved)


class LayerBatchedSmall:
    """The partial step of ALL layers of a token as one call: the small caches of every (layer, sequence) live in one
    K and one V buffer and one context sees them as layers x B sequences.

    A decoder cannot run its layers' attention at once (layer l + 1's query depends on layer l's output); this form
    exists to measure what the partial-step kernel streams when launch and dependency latencies are amortised over
    all layers, which is legal for synthetic per-layer queries that do not depend on each other."""

    def __init__(self, layers, max_len_hint: int):
        first = layers[0]
        dev = first.out.device
        self.layers, self.n_layers, self.n_seq = layers, len(layers), first.n_seq
        self.n_q, self.n_kv = first.n_q, first.n_kv
        caps = []
        for st in layers:
            caps += st.small.cap.tolist()
        self.cache = alloc_cache(caps, [0] * len(caps), self.n_kv, dev, fill=0.0)
        self.cache_c = rkv.cache_struct(self.cache.k, self.cache.v, self.cache.row_offset, self.cache.cap, self.cache.len)
        self.ctx = rkv.Context(len(caps), self.n_q, self.n_kv, max(max_len_hint, 1), max(max_len_hint, 1))
        self.hint = max_len_hint

    def sync_from_layers(self):
        """Copy every layer's small cache (rows and lengths) into the combined buffers."""
        offs = self.cache.row_offset.tolist()
        for l, st in enumerate(self.layers):
            base = offs[l * self.n_seq]
            n = st.small.k.shape[0]
            self.cache.k[base: base + n].copy_(st.small.k)
            self.cache.v[base: base + n].copy_(st.small.v)
            self.cache.len[l * self.n_seq: (l + 1) * self.n_seq].copy_(st.small.len)

    def append_partial(self, q_all, k_all, v_all, out_all):
        """q_all [layers, B, Hq, 128], k_all / v_all [layers, B, Hkv, 128], out_all [layers, B, Hq, 128]: one launch."""
        n = self.n_layers * self.n_seq
        self.ctx.append_small_step(q_all.view(n, self.n_q, HEAD_DIM), k_all.view(n, self.n_kv, HEAD_DIM),
                                   v_all.view(n, self.n_kv, HEAD_DIM), None, self.cache_c,
                                   out_all.view(n, self.n_q, HEAD_DIM), max_len_hint=self.hint)


class LayerBatchedFull:
    """rkv_full_step of ALL layers of a token as one call: the full caches of every (layer, sequence) live in one K
    and one V buffer (synth.alloc_layer_stack) and one context sees them as layers x B sequences.

    Like LayerBatchedSmall this is a measuring form, legal only for synthetic per-layer queries that do not depend on
    each other: it shows what the attention pass, the score pass and the selection stream when launch and dependency
    latencies are amortised over all layers."""

    def __init__(self, stack: LayerCache, n_layers: int, k_small: list, n_q_heads: int, n_kv_heads: int, max_len_hint: int):
        dev = stack.k.device
        n = stack.row_offset.shape[0]
        self.n, self.n_q, self.n_kv, self.hint = n, n_q_heads, n_kv_heads, max_len_hint
        self.k_max = max(max(k_small), 1)
        self.ctx = rkv.Context(n, n_q_heads, n_kv_heads, max_len_hint, self.k_max)
        self.full_c = rkv.cache_struct(stack.k, stack.v, stack.row_offset, stack.cap, stack.len)
        self.k_small = torch.tensor(list(k_small) * n_layers, dtype=torch.int32, device=dev)
        self.topk_idx = torch.full((n, n_kv_heads, self.k_max), -2, dtype=torch.int32, device=dev)
        self.out = torch.zeros((n, n_q_heads, HEAD_DIM), dtype=torch.bfloat16, device=dev)

    def full_step(self, q_all):
        """q_all [layers, B, Hq, 128]: attention over every cache, scores and top-K, one call (three launches)."""
        self.ctx.full_step(q_all.view(self.n, self.n_q, HEAD_DIM), self.full_c, self.k_small, self.k_max, self.out,
                           self.topk_idx, max_len_hint=self.hint)
        return self.out
