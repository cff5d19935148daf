"""The decoder kernels of the end-to-end workload against their fp64 oracle, and the attention calls made
inside a (reduced-size) decode loop against the attention oracle on the inputs captured at the call."""
import numpy as np
import pytest
import torch

from oracle import llama_oracle as LO
from oracle import rkv_oracle as O

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def H():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2411_05787_b200 import harness
    return harness


def f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def bits(t):
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def gen(seed):
    g = torch.Generator(device="cuda"); g.manual_seed(seed)
    return g


def test_rmsnorm_gemv_swiglu(H):
    g = gen(1)
    for n_in, n_out in ((512, 384), (4096, 1031), (14336, 640)):
        x = torch.randn(n_in, generator=g, device="cuda")
        wn = (1.0 + 0.1 * torch.randn(n_in, generator=g, device="cuda")).to(torch.bfloat16)
        y = torch.empty_like(x)
        H.rmsnorm(x, wn, 1e-5, y)
        assert np.allclose(f64(y), LO.rmsnorm(f64(x), f64(wn), 1e-5), rtol=2e-5, atol=2e-6)
        w = (torch.randn((n_out, n_in), generator=g, device="cuda") * 0.05).to(torch.bfloat16)
        res = torch.randn(n_out, generator=g, device="cuda")
        out = torch.empty(n_out, device="cuda")
        H.gemv(w, x, out)
        want = LO.gemv(f64(w), f64(x))
        scale = np.abs(f64(w)) @ np.abs(f64(x))            # fp32 accumulation error scales with the sum of magnitudes
        assert (np.abs(f64(out) - want) <= 1e-5 * scale + 1e-6).all()
        H.gemv(w, x, out, residual=res)
        assert (np.abs(f64(out) - (want + f64(res))) <= 1e-5 * scale + 1e-5).all()
        H.gemv(w, x, out, norm_w=wn, eps=1e-5)              # RMSNorm fused into the read of x
        xn = LO.rmsnorm(f64(x), f64(wn), 1e-5)
        assert (np.abs(f64(out) - LO.gemv(f64(w), xn)) <= 2e-5 * (np.abs(f64(w)) @ np.abs(xn)) + 1e-6).all()
        xb = x.to(torch.bfloat16)                           # bf16 input vector (the attention output)
        H.gemv(w, xb, out)
        assert (np.abs(f64(out) - LO.gemv(f64(w), f64(xb))) <= 1e-5 * scale + 1e-6).all()
        res2 = res.clone()
        H.gemv(w, x, res2, residual=res2)                   # in place on the residual stream
        assert (np.abs(f64(res2) - (want + f64(res))) <= 1e-5 * scale + 1e-5).all()
    x = torch.randn(1024, generator=g, device="cuda")
    wgu = (torch.randn((2 * 777, 1024), generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    act = torch.empty(777, device="cuda")
    H.gemv_swiglu(wgu, x, act)
    assert np.allclose(f64(act), LO.swiglu_in(f64(wgu), f64(x)), rtol=1e-4, atol=1e-5)
    wn = (1.0 + 0.1 * torch.randn(1024, generator=g, device="cuda")).to(torch.bfloat16)
    H.gemv_swiglu(wgu, x, act, norm_w=wn, eps=1e-5)
    assert np.allclose(f64(act), LO.swiglu_in(f64(wgu), LO.rmsnorm(f64(x), f64(wn), 1e-5)), rtol=2e-4, atol=2e-5)


@pytest.mark.parametrize("pos", [0, 1, 777, 33791])
def test_rope_split(H, pos):
    g = gen(2 + pos)
    n_q, n_kv = 28, 4
    qkv = torch.randn((n_q + 2 * n_kv) * 128, generator=g, device="cuda")
    p = torch.tensor([pos], dtype=torch.int32, device="cuda")
    q = torch.zeros((n_q, 128), dtype=torch.bfloat16, device="cuda")
    k = torch.zeros((n_kv, 128), dtype=torch.bfloat16, device="cuda")
    v = torch.zeros((n_kv, 128), dtype=torch.bfloat16, device="cuda")
    H.rope_split(qkv, p, 500000.0, q, k, v, n_q, n_kv)
    wq, wk, wv = LO.rope_split(f64(qkv), pos, 500000.0, n_q, n_kv)
    # the kernel rounds to bf16: half an ulp of the value (2^-9 relative) plus fp32 rounding of the products
    for got, want in ((q, wq), (k, wk), (v, wv)):
        assert (np.abs(f64(got) - want) <= np.abs(want) * 2.0 ** -8 + 1e-6).all()


def test_embed_and_argmax(H):
    g = gen(3)
    table = torch.randn((300, 512), generator=g, device="cuda").to(torch.bfloat16)
    x = torch.empty(512, device="cuda")
    for tok, row in ((7, 7), (299, 299), (5000, 299), (-3, 0)):           # out-of-range ids are clamped
        H.embed(table, torch.tensor([tok], dtype=torch.int32, device="cuda"), x)
        assert torch.equal(x, table[row].float())
    logits = torch.randn(128256, generator=g, device="cuda")
    out = torch.zeros(1, dtype=torch.int32, device="cuda")
    H.argmax(logits, out)
    assert int(out) == LO.argmax_first(f64(logits))
    logits[[90001, 17, 4000]] = 99.0                                       # equal maxima: the lowest index wins
    H.argmax(logits, out)
    assert int(out) == 17
    H.argmax(logits[:1].contiguous(), out)
    assert int(out) == 0


def test_decode_loop_attention_calls_match_the_oracle(H):
    """Reduced-size decoder (3 layers, hidden 512, 4 q / 2 kv heads), 1500-token prompt, dynamic refresh.
    Every attention call of two layers is captured with its inputs and compared with the attention oracle;
    the greedy token stream itself is not gated (random weights make it chaotic)."""
    shape = H.LlamaShape(hidden=512, n_layers=3, n_q=4, n_kv=2, ffn=1024, vocab=1000)
    dec = H.LlamaDecoder(shape, prompt_len=1500, max_new=24, k_small=128, qc_stride=4, threshold=0.9, seed=11)
    g = torch.Generator(device="cpu"); g.manual_seed(12)
    dec.prefill(torch.randint(0, shape.vocab, (1500,), generator=g).to("cuda"))
    assert all(int(st.full.len[0]) == 1500 and int(st.small.len[0]) == 128 for st in dec.states)
    # the prefill wrote rotated keys: the cached key of position p is a rotation, so its norm equals the norm of
    # the unrotated projection; spot-check one layer through the library's own full step instead:
    # the small cache must hold exactly the rows its index list names
    st0 = dec.states[0]
    idx = st0.topk_idx[0].cpu().numpy()
    cap_f, cap_s = int(st0.full.cap[0]), int(st0.small.cap[0])
    kf = bits(st0.full.k).reshape(2, cap_f, 128)
    ks = bits(st0.small.k).reshape(2, cap_s, 128)
    for h in range(2):
        assert np.array_equal(ks[h, :128], kf[h, idx[h, :128]])
    records = []
    dec.capture = ({0, 2}, records)
    kinds = []
    for t in range(1, 21):
        kind = dec.kind_of(t)
        kinds.append(kind)
        # snapshot of the full caches of the captured layers before the step is not needed: rows only get appended
        dec.token_step(kind)
    torch.cuda.synchronize()
    assert dec.ctx.device_status() == 0
    assert kinds.count("check") == 5 and len(records) == 40
    assert all(int(st.full.len[0]) == 1520 for st in dec.states)
    n_full = 0
    for r in records:
        st = dec.states[r["layer"]]
        q = O.bf16_bits_to_f64(bits(r["q"][0]))
        if r["kind"] == "check" and int(r["flag"][0]) == 1:               # this layer refreshed: attention over C_f
            n_full += 1
            n = r["full_len"]
            k = O.bf16_bits_to_f64(bits(st.full.k).reshape(2, cap_f, 128)[:, :n])
            v = O.bf16_bits_to_f64(bits(st.full.v).reshape(2, cap_f, 128)[:, :n])
            want, score, _, _ = O.full_step(q, k, v, 128)
            got_idx = r["topk"][0].cpu().numpy()
            for h in range(2):
                assert O.check_topk_set(score[h], 128, got_idx[h, :128]) is None
        else:
            n = r["small_len"]
            k = O.bf16_bits_to_f64(bits(r["small_k"]).reshape(2, r["small_cap"], 128)[:, :n])
            v = O.bf16_bits_to_f64(bits(r["small_v"]).reshape(2, r["small_cap"], 128)[:, :n])
            want, _, _ = O.decode_attention(q, k, v)
        got = O.bf16_bits_to_f64(bits(r["out"][0]))
        err = np.abs(got - want).max()
        rel = np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30)
        assert err <= 2e-2 and rel <= 5e-3, (r["layer"], r["kind"], err, rel)
    assert int(dec.flag_total.sum()) >= n_full
    # the loop is graph-capturable: replaying a captured token advances every cache by one row
    dec.capture = None
    side = torch.cuda.Stream()
    gr = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(gr, stream=side):
            dec.token_step("small")
    gr.replay(); gr.replay()
    torch.cuda.synchronize()
    assert all(int(st.full.len[0]) == 1522 for st in dec.states) and dec.ctx.device_status() == 0
    assert 0 <= int(dec.token) < shape.vocab
