"""Host-side checks of the seeded input generators (no method arithmetic lives there; these pin the layouts)."""
import torch

from paper_2411_05787_b200 import synth


def test_layer_stack_holds_the_same_bytes_as_separate_layers():
    """All layers' caches in one K and one V buffer (the layer-batched measurements) are, layer by layer, the very
    bytes the per-layer generator produces; the views keep global row offsets and share the stack's lengths."""
    w = synth.Workload("t", 3, 8, 2, [70, 33], [8, 4], 5, "fixed", 10, rho=[0.9, 0.9], seed=5)
    dev = torch.device("cpu")
    stack = synth.alloc_layer_stack(w, dev)
    assert stack.row_offset.shape[0] == w.n_layers * w.batch
    caps = [l + w.steps + 1 for l in w.lens]
    per_layer_rows = w.n_kv_heads * sum(caps)
    assert stack.k.shape[0] == w.n_layers * per_layer_rows
    for l in range(w.n_layers):
        view = synth.fill_layer(w, l, dev, into=synth.layer_view(stack, l, w.batch))
        alone = synth.fill_layer(w, l, dev)
        assert view.k.data_ptr() == stack.k.data_ptr()                        # a view, not a copy
        assert view.row_offset.tolist() == [l * per_layer_rows + o for o in alone.row_offset.tolist()]
        assert view.cap.tolist() == alone.cap.tolist() and view.len.tolist() == alone.len.tolist()
        r0 = int(view.row_offset[0])
        assert torch.equal(stack.k[r0: r0 + per_layer_rows], alone.k)
        assert torch.equal(stack.v[r0: r0 + per_layer_rows], alone.v)
        view.len[0] += 1                                                      # lengths are shared with the stack
        assert int(stack.len[l * w.batch]) == w.lens[0] + 1


def test_paper_points_have_the_stated_ratios():
    """K = L / 8 for the 16K-token points, K = 4096 for the 100K+ ones; strides, thresholds and shapes as named."""
    for name, (model, ctx, k, schedule, stride, thr, steps) in synth.PAPER_POINTS.items():
        w = synth.paper_point(name)
        assert w.lens == [ctx] and w.k_small == [k] and w.schedule == schedule and w.stride == stride
        assert (w.n_q_heads, w.n_kv_heads) == ((32, 8) if model == "llama" else (28, 4))
        assert k == (ctx // 8 if ctx <= 16384 else 4096)
        assert (w.threshold == thr) and steps == 256
