"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Integers (X_q, W_q, Int32 accumulators, scales' bits) must match exactly; fp32 outputs
within 1e-5 of the output magnitude."""
import numpy as np
import pytest
import torch

from oracle import q8_oracle as o
from paper_1910_06188_b200 import binding as q8
from paper_1910_06188_b200 import synth
from tests.gpu_util import REL_TOL, assert_close_fp, check_linear, dev

pytestmark = pytest.mark.gpu


# ------------------------------------------------------------------ quantiser (Eq. 1, Eq. 3, Sec. 4.1)
@pytest.mark.parametrize("n", [1, 3, 4, 5, 15, 16, 17, 1023, 4096, 100_003, 1 << 20])
def test_quantize_dynamic_bit_exact(n):
    x = synth.activation(1, n, seed=100 + n).reshape(-1)
    xq, S = q8.q8_quantize_activation(dev(x))
    S_ref, _ = o.scale_from_absmax(o.absmax(x))
    assert S.cpu().numpy()[0] == S_ref
    assert np.array_equal(xq.cpu().numpy(), o.quantize(x, S_ref))


def test_quantize_static_scale_ties_clamp_and_nonfinite():
    x = np.concatenate([
        np.arange(-300, 301, dtype=np.float32) * 0.5,
        np.array([np.nan, np.inf, -np.inf, 1e30, -1e30, 0.0, -0.0], np.float32),
        synth.activation(1, 5000, seed=5).reshape(-1) * 20,
    ]).astype(np.float32)
    for S in (1.0, 0.5, 3.1875, float(np.float32(1) / np.float32(3))):
        Sd = dev(np.array([S], np.float32))
        xq, _ = q8.q8_quantize_activation(dev(x), Sd)
        got = xq.cpu().numpy()
        assert np.array_equal(got, o.quantize(x, S))
        assert got.min() >= -127


def test_quantize_unaligned_pointer_uses_scalar_kernel():
    x = synth.activation(1, 1000, seed=9).reshape(-1)
    buf = torch.zeros(1001, dtype=torch.float32, device="cuda")
    buf[1:] = dev(x)
    xq, S = q8.q8_quantize_activation(buf[1:])
    S_ref, _ = o.scale_from_absmax(o.absmax(x))
    assert S.cpu().numpy()[0] == S_ref
    assert np.array_equal(xq.cpu().numpy(), o.quantize(x, S_ref))


def test_zero_tensor_flags_scale():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    x = torch.zeros(1000, dtype=torch.float32, device="cuda")
    xq, S = q8.q8_quantize_activation(x, dev_status=status)
    code, bits = q8.q8_poll_status(status)
    assert code == q8.Q8_ERR_SCALE and bits == 1 << q8.Q8_ERR_SCALE
    assert S.cpu().numpy()[0] == 1.0 and not xq.any()
    assert q8.q8_poll_status(status) == (q8.Q8_OK, 0)  # polling clears the word


@pytest.mark.parametrize("shape", [(1, 1), (7, 13), (768, 768), (3072, 768)])
def test_quantize_weight(shape):
    W = synth.weight(shape[0], shape[1], seed=200 + shape[0])
    Wq, S_w = q8.q8_quantize_weight(dev(W))
    Wq_ref, S_ref, _ = o.quantize_weight(W)
    assert S_w.cpu().numpy()[0] == S_ref
    assert np.array_equal(Wq.cpu().numpy(), Wq_ref)


# ------------------------------------------------------------------ Eq. 4
def test_calibrate_matches_oracle_ema():
    state = q8.new_calibrate_state()
    ref = o.EmaState()
    decay = 0.9999
    for i in range(6):
        x = synth.activation(64, 96, seed=300 + i) * np.float32(1.0 + 0.3 * i)
        q8.q8_calibrate(dev(x), decay, state)
        ref.update(o.absmax(x), decay)
        words = state.cpu()
        ema, S_x = words.view(torch.float32)[0].item(), words.view(torch.float32)[1].item()
        assert np.float32(ema) == ref.ema[0] and np.float32(S_x) == ref.S_x
        assert words[2].item() == i + 1 and words[4].item() == 0
    assert q8.calibrate_S_x(state).cpu().numpy()[0] == ref.S_x


def test_calibrate_decay_zero_is_dynamic_and_zero_batch_flags():
    state = q8.new_calibrate_state()
    ref = o.EmaState()
    for i, g in enumerate((3.0, 0.5, 7.0)):
        x = synth.activation(8, 40, seed=310 + i) * np.float32(g)
        q8.q8_calibrate(dev(x), 0.0, state)
        ref.update_batch(x, 0.0)
        got = state.view(torch.float32)[1].item()
        # decay 0 keeps no history: exactly the dynamic scale of Sec. 4.1 for this batch
        assert np.float32(got) == ref.S_x == np.float32(127.0) / o.absmax(x)
    # an empty batch is no observation: state (ema, S_x, n_batches) unchanged, nothing launched
    before = state.clone()
    q8.q8_calibrate(torch.empty(0, device="cuda"), 0.5, state)
    assert q8.q8_last_launch_info()["launches"] == 0 and torch.equal(state, before)
    assert ref.update_batch(np.zeros(0, np.float32), 0.5) == np.float32(state.view(torch.float32)[1].item())
    state = q8.new_calibrate_state()
    q8.q8_calibrate(torch.zeros(100, device="cuda"), 0.9, state)
    assert state[4].item() == 1 << q8.Q8_ERR_SCALE and state.view(torch.float32)[1].item() == 1.0


# ------------------------------------------------------------------ quantised FC, small / ragged / tile-boundary shapes
SHAPES = [
    (1, 8, 16), (1, 1, 16), (5, 3, 32), (128, 128, 128), (129, 130, 144), (127, 255, 48), (256, 64, 16),
    (300, 200, 400), (33, 257, 272), (260, 520, 1040), (1000, 96, 2064),
]


@pytest.mark.parametrize("M,N,K", SHAPES)
@pytest.mark.parametrize("mode", ["dynamic", "static"])
def test_linear_small_shapes(M, N, K, mode):
    X = synth.activation(M, K, seed=400 + M + N + K)
    W = synth.weight(N, K, seed=401 + M + N + K)
    b = synth.bias(N, seed=402 + M + N + K)
    S_x = None if mode == "dynamic" else float(np.float32(127.0) / np.float32(6.0))  # clamps the x8 outliers
    info = check_linear(X, W, b, act=(M + N) % 2, S_x=S_x)
    assert info["gemm_kernel"] == 1, "K % 16 == 0 shapes must run the tcgen05 kernel"


@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (3, 5, 7), (64, 64, 100), (130, 70, 33), (17, 200, 1001)])
def test_linear_generic_shapes(M, N, K):
    X = synth.activation(M, K, seed=500 + M)
    W = synth.weight(N, K, seed=501 + M)
    b = synth.bias(N, seed=502 + M)
    info = check_linear(X, W, b, act=1)
    assert info["gemm_kernel"] == 2, "K % 16 != 0 must fall back to the generic kernel"


def test_linear_no_bias_and_forced_generic_agree():
    X = synth.activation(200, 256, seed=600)
    W = synth.weight(300, 256, seed=601)
    check_linear(X, W, None, act=0)
    check_linear(X, W, None, act=1, fn=q8.q8_linear_generic)


def test_linear_integer_inputs_reduce_to_exact_matmul():
    rng = np.random.default_rng(5)
    M, N, K = 150, 90, 160
    X = rng.integers(-127, 128, size=(M, K)).astype(np.float32)
    Wq = rng.integers(-127, 128, size=(N, K), dtype=np.int8)
    b = rng.integers(-1000, 1000, size=N).astype(np.float32)
    one = dev(np.ones(1, np.float32))
    acc = torch.empty((M, N), dtype=torch.int32, device="cuda")
    Y = q8.q8_linear(dev(X), dev(Wq), one, one, dev(b), 0, dbg_acc=acc)
    want = X.astype(np.int64) @ Wq.astype(np.int64).T + b.astype(np.int64)
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), want)
    assert np.array_equal(Y.cpu().numpy().astype(np.float64), want.astype(np.float64))


def test_linear_saturated_accumulator():
    # all-127 rows: acc = 16129 * K, the largest value the path can produce for this K
    M, N, K = 128, 64, 4096
    X = np.full((M, K), 127.0, np.float32)
    X[1::2] *= -1
    Wq = np.full((N, K), 127, np.int8)
    one = dev(np.ones(1, np.float32))
    acc = torch.empty((M, N), dtype=torch.int32, device="cuda")
    q8.q8_linear(dev(X), dev(Wq), one, one, None, 0, dbg_acc=acc)
    got = acc.cpu().numpy()
    assert np.all(got[0::2] == 66064384) and np.all(got[1::2] == -66064384)


def test_linear_q_matches_linear():
    M, N, K = 256, 384, 512
    X = synth.activation(M, K, seed=700)
    W = synth.weight(N, K, seed=701)
    b = synth.bias(N, seed=702)
    Wq, S_w = q8.q8_quantize_weight(dev(W))
    Xq, S_x = q8.q8_quantize_activation(dev(X))
    Y1 = q8.q8_linear_q(Xq, S_x, Wq, S_w, dev(b), 1)
    Y2 = q8.q8_linear(dev(X), Wq, S_w, None, dev(b), 1)
    assert torch.equal(Y1, Y2)


def test_linear_is_deterministic():
    X, W, b = synth.activation(512, 768, 800), synth.weight(768, 768, 801), synth.bias(768, 802)
    Wq, S_w = q8.q8_quantize_weight(dev(W))
    Xd, bd = dev(X), dev(b)
    Y1 = q8.q8_linear(Xd, Wq, S_w, None, bd, 1).clone()
    Y2 = q8.q8_linear(Xd, Wq, S_w, None, bd, 1)
    assert torch.equal(Y1, Y2)


def test_device_side_errors_are_returned_as_codes():
    X = torch.zeros((8, 16), device="cuda")
    Wq = torch.ones((4, 16), dtype=torch.int8, device="cuda")
    S_w = torch.ones(1, device="cuda")
    ws = q8.new_workspace(8, 4, 16)
    Y = q8.q8_linear(X, Wq, S_w, None, None, 0, workspace=ws)      # max|X| == 0
    assert q8.q8_poll_status(ws)[0] == q8.Q8_ERR_SCALE and not Y.any()
    # a caller-supplied static scale that is zero, negative, NaN or infinite is reported the same way
    Xr = torch.randn((8, 16), device="cuda")
    for bad in (0.0, -3.0, float("nan"), float("inf")):
        q8.q8_linear(Xr, Wq, S_w, torch.full((1,), bad, device="cuda"), None, 0, workspace=ws)
        assert q8.q8_poll_status(ws)[0] == q8.Q8_ERR_SCALE, bad
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        q8.q8_quantize_activation(Xr, torch.full((1,), bad, device="cuda"), dev_status=st)
        assert q8.q8_poll_status(st)[0] == q8.Q8_ERR_SCALE, bad
    q8.q8_linear(Xr, Wq, S_w, torch.full((1,), 2.5, device="cuda"), None, 0, workspace=ws)
    assert q8.q8_poll_status(ws) == (q8.Q8_OK, 0)
    with pytest.raises(q8.Q8Error) as e:
        q8.q8_linear(X, Wq, S_w, None, None, 0, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.status == q8.Q8_ERR_WORKSPACE
    with pytest.raises(q8.Q8Error) as e:
        q8.q8_linear(X, Wq, S_w, None, None, 3)
    assert e.value.status == q8.Q8_ERR_ARG


@pytest.mark.parametrize("M,K,N", [(128, 768, 768), (256, 768, 96), (1, 16, 8), (37, 96, 40), (4, 48, 32), (255, 768, 64)])
def test_small_dynamic_layer_is_two_launches_and_matches_the_oracle(M, K, N):
    """A small activation (up to 256 x 768 values) is abs-maxed, scaled and quantised by one cluster in one launch
    (Sec. 4.1 + Eq. 1), so the whole dynamic layer is two kernels; same bits as the oracle, call after call."""
    X = synth.activation(M, K, seed=700 + M)
    W = synth.weight(N, K, seed=701 + M)
    b = synth.bias(N, seed=702 + M)
    for _ in range(2):
        info = check_linear(X, W, b, act=1)
        assert info["launches"] == 2
    # all-zero and non-finite activations: scale forced to 1, flagged, no NaN in the Int8 tensor
    Wq, S_w = q8.q8_quantize_weight(dev(W))
    ws = q8.new_workspace(M, N, K)
    xq = torch.empty((M, K), dtype=torch.int8, device="cuda")
    q8.q8_linear(torch.zeros((M, K), device="cuda"), Wq, S_w, None, dev(b), 0, workspace=ws, dbg_Xq=xq)
    assert q8.q8_poll_status(ws)[0] == q8.Q8_ERR_SCALE and not xq.any()
    Xi = dev(X).clone()
    Xi[0, 0] = float("inf")
    Xi[0, 1] = float("nan")
    q8.q8_linear(Xi, Wq, S_w, None, dev(b), 0, workspace=ws, dbg_Xq=xq)
    assert q8.q8_poll_status(ws)[0] == q8.Q8_ERR_SCALE
    assert np.array_equal(xq.cpu().numpy(), o.quantize(Xi.cpu().numpy(), 1.0))
    q8.q8_linear(dev(X), Wq, S_w, None, dev(b), 0, workspace=ws)        # and the next call starts clean
    assert q8.q8_poll_status(ws) == (q8.Q8_OK, 0)


# ------------------------------------------------------------------ the paper-shaped configurations
def test_config_single_layer_dynamic():
    """X [128 x 768] with x8 outliers, W [768 x 768], bias; dynamic S_x (Sec. 4.1)."""
    X = synth.activation(128, 768, synth.seed_for(1, 0))
    W = synth.weight(768, 768, synth.seed_for(1, 1))
    b = synth.bias(768, synth.seed_for(1, 2))
    info = check_linear(X, W, b, act=0)
    assert info["gemm_kernel"] == 1


@pytest.mark.parametrize("name,K,N,act", synth.fc_set(768, 3072))
def test_config_bert_base_fc_set(name, K, N, act):
    """BERT-Base FC set at 32 x 128 tokens, S_x from one seeded calibration batch (Eq. 4)."""
    M = 4096
    idx = [n for n, *_ in synth.fc_set(768, 3072)].index(name)
    X = synth.activation(M, K, synth.seed_for(2, 10 * idx))
    calib = synth.activation(M, K, synth.seed_for(2, 10 * idx + 1))
    W = synth.weight(N, K, synth.seed_for(2, 10 * idx + 2))
    b = synth.bias(N, synth.seed_for(2, 10 * idx + 3))
    state = q8.new_calibrate_state()
    q8.q8_calibrate(dev(calib), 0.9999, state)
    ref = o.EmaState()
    S_x = ref.update(o.absmax(calib), 0.9999)
    assert q8.calibrate_S_x(state).cpu().numpy()[0] == S_x
    info = check_linear(X, W, b, act=act, S_x=float(S_x), canary=False)
    assert info["gemm_kernel"] == 1


# ------------------------------------------------------------------ embedding (Sec. 3)
@pytest.mark.parametrize("V,H,T", [(50, 24, 31), (1000, 768, 4096), (77, 10, 200), (30522, 1024, 3000)])
def test_embedding(V, H, T):
    E = synth.embedding_table(V, H, seed=900 + H)
    ids = synth.token_ids(T, V, seed=901 + H)
    Eq, S_e = q8.q8_quantize_weight(dev(E))
    Eq_ref, S_ref, _ = o.quantize_weight(E)
    assert np.array_equal(Eq.cpu().numpy(), Eq_ref) and S_e.cpu().numpy()[0] == S_ref
    rows = torch.empty((T, H), dtype=torch.int8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = q8.q8_embedding(dev(ids), Eq, S_e, rows_q=rows, dev_status=status)
    rows_ref, out_ref, bad = o.embedding(ids, Eq_ref, S_ref)
    assert bad == 0 and q8.q8_poll_status(status) == (q8.Q8_OK, 0)
    assert np.array_equal(rows.cpu().numpy(), rows_ref)
    assert_close_fp(out.cpu().numpy(), out_ref, "embedding")


def test_embedding_bad_ids_are_flagged_and_zeroed():
    V, H, T = 40, 32, 20
    E = synth.embedding_table(V, H, seed=950)
    ids = synth.token_ids(T, V, seed=951)
    ids[3], ids[11] = -1, V
    Eq, S_e = q8.q8_quantize_weight(dev(E))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = q8.q8_embedding(dev(ids), Eq, S_e, dev_status=status)
    assert q8.q8_poll_status(status)[0] == q8.Q8_ERR_INDEX
    rows_ref, out_ref, bad = o.embedding(ids, Eq.cpu().numpy(), S_e.cpu().numpy()[0])
    assert bad == 2
    got = out.cpu().numpy()
    assert not got[3].any() and not got[11].any()
    assert_close_fp(got, out_ref, "embedding with bad ids")


# ------------------------------------------------------------------ training-mode pieces (Sec. 2.2, Eq. 5)
@pytest.mark.parametrize("n", [1, 7, 4096, 100_003])
def test_fake_quantize_and_ste(n):
    x = synth.activation(1, n, seed=1300 + n).reshape(-1)
    state = q8.new_calibrate_state()
    q8.q8_calibrate(dev(x), 0.9, state)                       # the EMA update training does on every forward
    S = q8.calibrate_S_x(state)
    xh = q8.q8_fake_quantize(dev(x), S).cpu().numpy()
    S_ref, _ = o.scale_from_absmax(o.absmax(x))
    assert S.item() == S_ref
    ref = o.fake_quantize(x, S_ref)
    assert np.abs(xh - ref).max() <= 1e-6 * max(np.abs(ref).max(), 1e-30)
    # the fake-quantised values sit exactly on the Int8 grid of the real quantiser
    assert np.array_equal(np.rint(xh.astype(np.float64) * float(S_ref)).astype(np.int8), o.quantize(x, S_ref))
    g = synth.normal((n,), 1.0, 1400 + n)
    assert np.array_equal(q8.q8_ste_backward(dev(g)).cpu().numpy(), g)
    gd = dev(g)
    assert q8.q8_ste_backward(gd, gd).data_ptr() == gd.data_ptr()


# ------------------------------------------------------------------ one weight scale per fused layer (Eq. 3 per layer)
@pytest.mark.parametrize("M,H,seg,act", [(300, 128, 128, 0), (515, 256, 256, 1), (64, 40, 40, 0)])
def test_fused_projection_with_per_layer_scales_equals_separate_layers(M, H, seg, act):
    """Q, K and V stored as one [3H, H] matrix with one S_w per block of H rows must give what three separate
    quantised FC layers give (the paper's model has three layers, each with its own Eq. 3 scale)."""
    X = synth.activation(M, H, seed=1500 + M)
    Ws = [synth.normal((H, H), 0.02 * (1 + 2 * i), 1501 + M + i) for i in range(3)]   # different ranges per layer
    bs = [synth.bias(H, 1510 + M + i) for i in range(3)]
    W, b = np.concatenate(Ws), np.concatenate(bs)
    Wq, S_w = q8.q8_quantize_weight_segments(dev(W), seg)
    acc = torch.empty((M, 3 * H), dtype=torch.int32, device="cuda")
    Y = q8.q8_linear_wseg(dev(X), Wq, S_w, seg, None, dev(b), act, dbg_acc=acc)
    info = q8.q8_last_launch_info()
    assert info["gemm_kernel"] == (1 if seg % 32 == 0 else 2)
    for i in range(3):
        Wq_ref, S_ref, _ = o.quantize_weight(Ws[i])
        assert S_w[i].item() == S_ref and np.array_equal(Wq[i * H:(i + 1) * H].cpu().numpy(), Wq_ref)
        ref = o.linear(X, Wq_ref, S_ref, None, bs[i], act)
        assert np.array_equal(acc[:, i * H:(i + 1) * H].cpu().numpy(), ref["acc"])
        assert_close_fp(Y[:, i * H:(i + 1) * H].cpu().numpy(), ref["y"], f"segment {i}")
    Xq, S_x = q8.q8_quantize_activation(dev(X))
    assert torch.equal(q8.q8_linear_q_wseg(Xq, S_x, Wq, S_w, seg, dev(b), act), Y)
