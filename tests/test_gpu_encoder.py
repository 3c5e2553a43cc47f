"""Encoder-level checks: the FP32 support kernels against the oracle, and whole encoder forwards.

A forward chains ~50-100 quantised layers, and layer k+1 quantises what layer k computed in fp32,
so an ulp of difference upstream can flip a nearest-integer decision downstream.  Bit-exactness is
therefore checked per call with the call's own input: for every q8_linear inside the forward the CPU
oracle is given the same fp32 input bytes that the layer received (and its own quantisation of the
seeded weights) and must reproduce the Int8 activation, the Int32 accumulator and the fp32 output of
that call.  On top of that a small model is run end to end in the oracle from the seeded inputs alone."""
import numpy as np
import pytest
import torch

from oracle import q8_oracle as o
from paper_1910_06188_b200 import binding as q8
from paper_1910_06188_b200 import encoder as enc_mod
from paper_1910_06188_b200 import synth
from tests.gpu_util import REL_TOL, assert_close_fp, dev

pytestmark = pytest.mark.gpu


# ------------------------------------------------------------------ support kernels
@pytest.mark.parametrize("rows,H", [(1, 4), (37, 96), (300, 768), (64, 1024), (5, 1000)])
def test_add_layernorm(rows, H):
    x = synth.activation(rows, H, 3000 + H)
    r1 = synth.activation(rows, H, 3001 + H)
    r2 = synth.normal((rows, H), 0.5, 3002 + H)
    g = synth.normal((H,), 1.0, 3003 + H)
    b = synth.normal((H,), 1.0, 3004 + H)
    assert_close_fp(q8.q8_add_layernorm(dev(x), dev(r1), dev(r2), dev(g), dev(b)).cpu().numpy(),
                    o.add_layernorm(x, r1, r2, g, b), "LN(x+r1+r2)")
    assert_close_fp(q8.q8_add_layernorm(dev(x), dev(r1)).cpu().numpy(), o.add_layernorm(x, r1), "LN(x+r1)")
    assert_close_fp(q8.q8_add_layernorm(dev(x)).cpu().numpy(), o.add_layernorm(x), "LN(x)")
    xd = dev(x)
    q8.q8_add_layernorm(xd, dev(r1), out=xd)                       # in place
    assert_close_fp(xd.cpu().numpy(), o.add_layernorm(x, r1), "LN in place")


@pytest.mark.parametrize("B,S,heads", [(1, 1, 1), (2, 9, 3), (3, 64, 2), (2, 70, 2), (2, 128, 12), (1, 384, 4)])
def test_attention(B, S, heads):
    qkv = synth.normal((B * S, 3 * heads * 64), 1.0, 3100 + S)
    got = q8.q8_attention(dev(qkv), B, S, heads).cpu().numpy()
    assert_close_fp(got, o.attention(qkv, B, S, heads), "attention")


@pytest.mark.parametrize("B,S,heads", [(2, 100, 2), (1, 384, 2), (1, 448, 1), (1, 500, 1)])
def test_attention_tensor_core_and_cuda_core_kernels_both_match_the_oracle(B, S, heads):
    """S <= 448 runs on the tensor cores (split TF32 products), longer sequences and q8_tune_attention(0)
    on the CUDA-core kernel; both must meet the fp32 tolerance."""
    qkv = synth.normal((B * S, 3 * heads * 64), 1.0, 3150 + S)
    ref = o.attention(qkv, B, S, heads)
    try:
        for tensor_cores in (True, False):
            q8.q8_tune_attention(tensor_cores)
            got = q8.q8_attention(dev(qkv), B, S, heads).cpu().numpy()
            assert q8.q8_attention_status() == (q8.Q8_OK, 0)
            assert_close_fp(got, ref, f"attention (tensor cores {tensor_cores})")
    finally:
        q8.q8_tune_attention(True)


def test_attention_large_logits_stay_finite():
    B, S, heads = 1, 130, 1
    qkv = synth.normal((B * S, 3 * 64), 6.0, 3150)             # logits of several hundred
    got = q8.q8_attention(dev(qkv), B, S, heads).cpu().numpy()
    assert np.isfinite(got).all()
    # fp32 logits of magnitude ~500 carry an absolute rounding error of ~500 * 2^-24 = 3e-5, which the
    # exponential turns into the same relative error of the weights: bound the output error accordingly
    ref = o.attention(qkv, B, S, heads)
    assert np.abs(got - ref).max() <= 1e-4 * np.abs(ref).max()


# ------------------------------------------------------------------ whole forwards
def _oracle_weights(enc):
    w = {}
    for name, t in enc.fp32.items():
        if name.startswith("b."):
            w[name] = t
        else:
            w[name] = o.quantize_weight(t)[:2]        # (W_q, S_w) from the seeded fp32 tensor
    return w


def _teacher_forced_hook(enc, w, T, slabs, record):
    """Checks each quantised FC of a forward against the oracle on the rows in `slabs`."""
    def hook(l, name, X, Y, p, S_x, Xq, acc):
        Wq_ref, S_w_ref = w[f"W.{l}.{name}"]
        b = w[f"b.{l}.{name}"]
        assert p["S_w"].item() == S_w_ref
        sx = np.float32(S_x.item())
        for lo, hi in slabs:
            Xs = X[lo:hi].cpu().numpy()
            ref = o.linear(Xs, Wq_ref, S_w_ref, sx, b, p["act"])
            assert np.array_equal(Xq[lo:hi].cpu().numpy(), ref["xq"]), f"layer {l} {name}: X_q rows {lo}:{hi}"
            assert np.array_equal(acc[lo:hi].cpu().numpy(), ref["acc"]), f"layer {l} {name}: Int32 rows {lo}:{hi}"
            err = np.abs(Y[lo:hi].cpu().numpy() - ref["y"]).max()
            assert err <= REL_TOL * max(np.abs(ref["y"]).max(), 1e-30), f"layer {l} {name}: fp32 rows {lo}:{hi}"
        record.append((l, name, float(sx)))
    return hook


def _oracle_forward(enc, w, ids, B, S):
    """The same forward, every step in the oracle, from the seeded inputs alone (dynamic scales)."""
    f32 = lambda a: np.asarray(a, dtype=np.float32)
    T = B * S
    pos = np.tile(np.arange(S, dtype=np.int32), B)
    typ = np.zeros(T, np.int32)
    ew = o.embedding(ids, *w["word"])[1]
    ep = o.embedding(pos, *w["pos"])[1]
    et = o.embedding(typ, *w["typ"])[1]
    h = f32(o.add_layernorm(f32(ew), f32(ep), f32(et), eps=enc_mod.LN_EPS))
    lin = lambda l, name, X, act: f32(o.linear(X, *w[f"W.{l}.{name}"], None, w[f"b.{l}.{name}"], act)["y"])
    for l in range(enc.L):
        qkv = lin(l, "qkv", h, 0)
        ctx = f32(o.attention(qkv, B, S, enc.heads))
        ao = lin(l, "attn_out", ctx, 0)
        h1 = f32(o.add_layernorm(ao, h, eps=enc_mod.LN_EPS))
        f = lin(l, "ffn1", h1, 1)
        f2 = lin(l, "ffn2", f, 0)
        h = f32(o.add_layernorm(f2, h1, eps=enc_mod.LN_EPS))
    return h


def test_small_encoder_teacher_forced_and_end_to_end():
    dims = dict(hidden=128, ffn=512, heads=2, layers=3, vocab=500, max_pos=96)
    B, S = 3, 70
    enc = enc_mod.Q8BertEncoder(dims, config=30, keep_fp32=True)
    w = _oracle_weights(enc)
    ids_h = synth.token_ids(B * S, dims["vocab"], synth.seed_for(30, 90))
    ids = torch.from_numpy(ids_h).cuda()
    rec = []
    out = enc.forward(ids, B, S, scales="dynamic", debug=True,
                      hook=_teacher_forced_hook(enc, w, B * S, [(0, B * S)], rec)).cpu().numpy()
    assert len(rec) == 4 * dims["layers"] and enc.poll() == ((q8.Q8_OK, 0), (q8.Q8_OK, 0))
    want = _oracle_forward(enc, w, ids_h, B, S)
    # end to end a nearest-integer flip may occur somewhere; outputs are LayerNorm-ed (unit scale)
    diff = np.abs(out - want)
    assert diff.max() < 5e-2 and np.median(diff) < 1e-4, (diff.max(), np.median(diff))


def _run_model_case(dims, config, B, S, scales, calib_batches, layers=None):
    enc = enc_mod.Q8BertEncoder(dims, config=config, keep_fp32=True, layers=layers)
    w = _oracle_weights(enc)
    T = B * S
    V = dims["vocab"]
    if scales == "static":
        refs = {}
        for c in range(calib_batches):
            cid = torch.from_numpy(synth.token_ids(T, V, synth.seed_for(config, 300 + c))).cuda()

            def cal_hook(l, name, X, Y, p, S_x, Xq, acc):
                if l == 0:                      # follow the EMA of the first layer's four quantisers in the oracle
                    refs.setdefault(name, o.EmaState()).update(o.absmax(X.cpu().numpy()), 0.9999)
            enc.forward(cid, B, S, scales="calibrate", decay=0.9999, hook=cal_hook)
        for name, st in refs.items():
            got = q8.calibrate_S_x(enc.layers[0][name]["state"]).item()
            assert np.float32(got) == st.S_x, f"Eq. 4 scale of layer 0 {name}"
            assert enc.layers[0][name]["state"][2].item() == calib_batches
    ids = enc_mod.random_ids(T, V, config)
    mid = (T // 2 // 256) * 256
    slabs = [(0, 24), (mid - 12, mid + 12), (T - 24, T)]
    rec = []
    out = enc.forward(ids, B, S, scales=scales, debug=True, hook=_teacher_forced_hook(enc, w, T, slabs, rec))
    assert len(rec) == 4 * enc.L
    assert enc.poll() == ((q8.Q8_OK, 0), (q8.Q8_OK, 0))
    o_np = out.cpu().numpy()
    assert np.isfinite(o_np).all()
    assert np.allclose(o_np.mean(1), 0, atol=1e-4) and np.allclose(o_np.var(1), 1, atol=1e-3)   # LayerNorm-ed rows
    # int8 weights are a quarter of the fp32 bytes
    fp32_bytes = 4 * sum(t.size for n, t in enc.fp32.items() if not n.startswith("b."))
    assert enc.memory_bytes_int8() * 4 == fp32_bytes


def test_bert_base_encoder_forward():
    """BERT-Base encoder, batch 32 x seq 128: int8 embeddings, all FC layers quantised, static scales from
    one seeded calibration batch."""
    _run_model_case(synth.BERT_BASE, config=3, B=32, S=128, scales="static", calib_batches=1)


def test_bert_large_encoder_forward():
    """BERT-Large encoder, batch 64 x seq 384, EMA scales (decay 0.9999) over 16 seeded batches."""
    _run_model_case(synth.BERT_LARGE, config=5, B=64, S=384, scales="static", calib_batches=16)


# ------------------------------------------------------------------ fused re-quantisation
def test_requantising_outputs_equal_quantising_the_fp32_output():
    """Each producer's Int8 output must be Eq. 1 applied to exactly the fp32 value it would have stored."""
    S_q = dev(np.array([9.5], np.float32))
    # LayerNorm
    x, r1 = synth.activation(300, 768, 4000), synth.activation(300, 768, 4001)
    out = torch.empty((300, 768), device="cuda")
    oq = q8.q8_add_layernorm_quant(dev(x), dev(r1), None, S_q, out=out)
    assert_close_fp(out.cpu().numpy(), o.add_layernorm(x, r1), "LN fp32")
    assert np.array_equal(oq.cpu().numpy(), o.quantize(out.cpu().numpy(), 9.5))
    assert torch.equal(q8.q8_add_layernorm_quant(dev(x), dev(r1), None, S_q), oq)          # Int8 only
    # attention
    B, S, heads = 2, 70, 3
    qkv = synth.normal((B * S, 3 * heads * 64), 1.0, 4010)
    ctx = torch.empty((B * S, heads * 64), device="cuda")
    cq = q8.q8_attention_quant(dev(qkv), B, S, heads, S_q, ctx=ctx)
    assert_close_fp(ctx.cpu().numpy(), o.attention(qkv, B, S, heads), "attention fp32")
    assert np.array_equal(cq.cpu().numpy(), o.quantize(ctx.cpu().numpy(), 9.5))
    assert torch.equal(q8.q8_attention_quant(dev(qkv), B, S, heads, S_q), cq)
    # quantised FC, fp32 in and Int8 in, with and without GELU, tensor-core and generic kernels
    for (M, N, K, act) in [(515, 1040, 272, 1), (300, 208, 400, 0), (64, 50, 33, 1)]:
        X, W, b = synth.activation(M, K, 4020 + M), synth.weight(N, K, 4021 + M), synth.bias(N, 4022 + M)
        Wq_ref, S_w_ref, _ = o.quantize_weight(W)
        S_x = np.float32(20.0)
        ref = o.linear(X, Wq_ref, S_w_ref, S_x, b, act)
        Wq, S_w = q8.q8_quantize_weight(dev(W))
        Sx_d = dev(np.array([S_x], np.float32))
        S_y = dev(np.array([31.0], np.float32))
        Y = torch.empty((M, N), device="cuda")
        Yq = q8.q8_linear_requant(dev(X), Wq, S_w, Sx_d, dev(b), act, S_y, Y=Y)
        assert_close_fp(Y.cpu().numpy(), ref["y"], "requant fp32 copy")
        want_q = o.quantize(Y.cpu().numpy(), 31.0)
        assert np.array_equal(Yq.cpu().numpy(), want_q)
        assert torch.equal(q8.q8_linear_requant(dev(X), Wq, S_w, Sx_d, dev(b), act, S_y), Yq)   # Int8 only
        Xq, _ = q8.q8_quantize_activation(dev(X), Sx_d)
        assert torch.equal(q8.q8_linear_q_requant(Xq, Sx_d, Wq, S_w, dev(b), act, S_y), Yq)
        # against the oracle's own fp64 output the Int8 values may differ by one step only where y * S_y
        # sits within fp32 rounding of a tie
        exact = o.quantize(ref["y"].astype(np.float32), 31.0).astype(np.int32)
        d = np.abs(exact - Yq.cpu().numpy().astype(np.int32))
        assert d.max() <= 1 and (d != 0).mean() < 1e-3


def test_fused_forward_is_bit_identical_to_the_unfused_one():
    dims = dict(hidden=128, ffn=512, heads=2, layers=3, vocab=500, max_pos=96)
    for dims_, cfg, B, S in [(dims, 31, 3, 70), (synth.BERT_BASE, 3, 32, 128)]:
        enc = enc_mod.Q8BertEncoder(dims_, config=cfg)
        ids = enc_mod.random_ids(B * S, dims_["vocab"], cfg)
        enc.forward(ids, B, S, scales="calibrate")
        want = enc.forward(ids, B, S, scales="static").clone()
        got = enc.forward_fused(ids, B, S)
        assert enc.poll() == ((q8.Q8_OK, 0), (q8.Q8_OK, 0))
        assert torch.equal(got, want)
        # and replayed from a CUDA graph, also after the token ids change in place
        graph, out = enc.capture(ids, B, S)
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, want)
        ids.copy_(torch.flip(ids, dims=[0]))
        graph.replay()
        torch.cuda.synchronize()
        replayed = out.clone()
        assert torch.equal(replayed, enc.forward(ids, B, S, scales="static"))


# ------------------------------------------------------------------ dynamic quantisation with fused abs-max (Sec. 4.1)
def _word():
    return torch.zeros(1, dtype=torch.int32, device="cuda")


def _bits_of_absmax(t: torch.Tensor) -> int:
    """IEEE bits of the oracle's max|.| over the tensor the GPU actually stored."""
    return int(np.float32(o.absmax(t.cpu().numpy())).view(np.uint32))


@pytest.mark.parametrize("rows,H", [(37, 96), (300, 768), (5, 1000), (3, 2048), (3, 1001), (2000, 1024)])
def test_layernorm_folds_the_absmax_of_what_it_stores(rows, H):
    x = synth.activation(rows, H, 3400 + H)
    r1 = synth.activation(rows, H, 3401 + H)
    w = _word()
    out = q8.q8_add_layernorm_absmax(dev(x), w, dev(r1))
    assert torch.equal(out, q8.q8_add_layernorm(dev(x), dev(r1)))           # same values as the plain call
    assert (w.item() & 0xFFFFFFFF) == _bits_of_absmax(out)
    # the word only ever rises: a second producer with smaller values leaves it, one with larger values raises it
    before = w.item()
    q8.q8_add_layernorm_absmax(dev(x), w, dev(r1), gamma=dev(np.full(H, 0.5, np.float32)))
    assert w.item() == before
    big = q8.q8_add_layernorm_absmax(dev(x), w, dev(r1), gamma=dev(np.full(H, 3.0, np.float32)))
    assert (w.item() & 0xFFFFFFFF) == _bits_of_absmax(big)


@pytest.mark.parametrize("B,S,heads,tensor_cores", [(2, 100, 2, True), (1, 384, 4, True), (2, 70, 2, False), (1, 500, 1, True)])
def test_attention_folds_the_absmax_of_what_it_stores(B, S, heads, tensor_cores):
    qkv = dev(synth.normal((B * S, 3 * heads * 64), 1.0, 3450 + S))
    try:
        q8.q8_tune_attention(tensor_cores)
        w = _word()
        ctx = q8.q8_attention_absmax(qkv, B, S, heads, w)
        assert torch.equal(ctx, q8.q8_attention(qkv, B, S, heads))
        assert (w.item() & 0xFFFFFFFF) == _bits_of_absmax(ctx)
    finally:
        q8.q8_tune_attention(True)


@pytest.mark.parametrize("M,N,K,act", [(300, 200, 400, 1), (515, 1030, 144, 0), (4096, 768, 768, 1), (100, 52, 50, 1),
                                       (20000, 1000, 128, 1)])
def test_linear_dyn_takes_its_scale_from_a_word_and_reports_its_own_output_absmax(M, N, K, act):
    """q8_linear_dyn with max|X| supplied by the producer equals q8_linear with its own abs-max pass, bit for bit
    (and therefore the oracle, which check_linear compares q8_linear with), in two kernels instead of four
    operations; its y_absmax word is the oracle's max|.| of the stored output."""
    X = synth.activation(M, K, 3500 + M)
    Wq, S_w = q8.q8_quantize_weight(dev(synth.weight(N, K, 3501 + M)))
    b = dev(synth.bias(N, 3502 + M))
    Xd = dev(X)
    xw = _word()
    # the producer here is a LayerNorm that reproduces X: fold max|X| with the library's own abs-max kernel instead
    _, S_dyn = q8.q8_quantize_activation(Xd)                       # S = 127 / max|X|
    xw.copy_(torch.from_numpy(np.array([np.float32(o.absmax(X))]).view(np.int32)))
    ws0, ws1 = q8.new_workspace(M, N, K), q8.new_workspace(M, N, K)
    xq0, xq1 = (torch.empty((M, K), dtype=torch.int8, device="cuda") for _ in range(2))
    a0, a1 = (torch.empty((M, N), dtype=torch.int32, device="cuda") for _ in range(2))
    Y0 = q8.q8_linear(Xd, Wq, S_w, None, b, act, workspace=ws0, dbg_Xq=xq0, dbg_acc=a0)
    launches_plain = q8.q8_last_launch_info()["launches"]
    yw = _word()
    Y1 = q8.q8_linear_dyn(Xd, xw, Wq, S_w, b, act, y_absmax=yw, workspace=ws1, dbg_Xq=xq1, dbg_acc=a1)
    # q8_linear itself needs a memset-free single quantise launch only for small activations (one cluster holds them)
    assert q8.q8_last_launch_info()["launches"] == 2 and launches_plain == (2 if M * K <= 196608 and M * K % 4 == 0 else 3)
    assert q8.q8_poll_status(ws1) == (q8.Q8_OK, 0)
    assert torch.equal(xq0, xq1) and torch.equal(a0, a1) and torch.equal(Y0, Y1)
    assert ws1[4:8].view(torch.float32).item() == S_dyn.item() == ws0[4:8].view(torch.float32).item()
    assert (yw.item() & 0xFFFFFFFF) == _bits_of_absmax(Y1)
    ref = o.linear(X, Wq.cpu().numpy(), S_w.item(), None, b.cpu().numpy(), act)
    assert np.array_equal(xq1.cpu().numpy(), ref["xq"]) and np.array_equal(a1.cpu().numpy(), ref["acc"])
    assert_close_fp(Y1.cpu().numpy(), ref["y"], "Y")
    # a word that is still zero (producer never ran) is reported, not divided by
    q8.q8_linear_dyn(Xd, _word(), Wq, S_w, b, act, workspace=ws1)
    assert q8.q8_poll_status(ws1)[0] == q8.Q8_ERR_SCALE


def test_dynamic_forward_without_absmax_passes_equals_the_unfused_dynamic_forward():
    """Sec. 4.1 end to end: the forward whose producers fold max|y| (no stand-alone abs-max pass, no memset per FC)
    gives the same bits as the forward in which every q8_linear computes its own dynamic scale."""
    dims = dict(synth.BERT_BASE, layers=3)
    enc = enc_mod.Q8BertEncoder(dims, config=3)
    B, S = 4, 128
    ids = enc_mod.random_ids(B * S, dims["vocab"], 3)
    want = enc.forward(ids, B, S, scales="dynamic").clone()
    got = enc.forward_dynamic_fused(ids, B, S)
    assert torch.equal(got, want)
    assert enc.poll() == ((q8.Q8_OK, 0), (q8.Q8_OK, 0))
    assert enc.launches_per_forward("dynamic", fused=True) < enc.launches_per_forward("dynamic")
