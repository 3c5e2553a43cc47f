"""Parity at the benchmark's full size and launch configuration: the BERT-Large FC set at
M = 24576 tokens with static scales, automatic tile choice (CTA pairs on 256 x 256 tiles).

The CPU oracle computes every one of the 24576 rows of each layer (a few seconds per layer on a
multi-core host), so the whole quantised activation, the whole Int32 matrix and the whole fp32
output are compared with it, element by element.  The generic CUDA-core kernel is compared as well,
but only as a secondary, on-device cross-check: it is part of the same library, not a reference."""
import numpy as np
import pytest
import torch

from oracle import q8_oracle as o
from paper_1910_06188_b200 import binding as q8
from paper_1910_06188_b200 import synth
from tests.gpu_util import REL_TOL, dev

pytestmark = pytest.mark.gpu

M = synth.BERT_LARGE["batch"] * synth.BERT_LARGE["seq"]
LAYERS = synth.fc_set(synth.BERT_LARGE["hidden"], synth.BERT_LARGE["ffn"])


@pytest.mark.parametrize("name,K,N,act", LAYERS)
def test_bert_large_fc_full_size(name, K, N, act):
    idx = [n for n, *_ in LAYERS].index(name)
    X = synth.activation(M, K, synth.seed_for(4, 10 * idx))
    calib = synth.activation(4096, K, synth.seed_for(4, 10 * idx + 1))
    W = synth.weight(N, K, synth.seed_for(4, 10 * idx + 2))
    b = synth.bias(N, synth.seed_for(4, 10 * idx + 3))

    state = q8.new_calibrate_state()
    q8.q8_calibrate(dev(calib), 0.9999, state)
    S_x_dev = q8.calibrate_S_x(state).clone()
    S_x = o.EmaState().update(o.absmax(calib), 0.9999)
    assert S_x_dev.item() == S_x
    Wq, S_w = q8.q8_quantize_weight(dev(W))
    Wq_ref, S_w_ref, _ = o.quantize_weight(W)
    assert np.array_equal(Wq.cpu().numpy(), Wq_ref) and S_w.item() == S_w_ref

    Xd, bd = dev(X), dev(b)
    xq = torch.empty((M, K), dtype=torch.int8, device="cuda")
    acc = torch.empty((M, N), dtype=torch.int32, device="cuda")
    ws = q8.new_workspace(M, N, K)
    Y = q8.q8_linear(Xd, Wq, S_w, S_x_dev, bd, act, workspace=ws, dbg_Xq=xq, dbg_acc=acc)
    info = q8.q8_last_launch_info()
    assert q8.q8_poll_status(ws) == (q8.Q8_OK, 0)
    assert info["gemm_kernel"] == 1 and info["ctas"] == 2 and info["block_n"] == 256  # what bench.py times

    # the oracle on all M rows: X_q, acc + b_q and Y, whole matrices
    ref = o.linear(X, Wq_ref, S_w_ref, S_x, b, act)
    assert ref["flags"] == 0
    assert np.array_equal(xq.cpu().numpy(), ref["xq"]), f"{name}: X_q"
    assert np.array_equal(acc.cpu().numpy(), ref["acc"]), f"{name}: Int32 matrix"
    Yh = Y.cpu().numpy()
    scale = np.abs(ref["y"]).max()
    worst = 0.0
    for lo in range(0, M, 4096):   # in slabs, to keep the fp64 temporaries small
        worst = max(worst, float(np.abs(Yh[lo:lo + 4096] - ref["y"][lo:lo + 4096]).max()))
    assert worst <= REL_TOL * scale, f"{name}: max |Y - oracle| {worst:.3e} vs {REL_TOL} * {scale:.3e}"
    del ref, Yh

    # secondary, on-device: the generic kernel of this library gives the same Int32 matrix
    acc2 = torch.empty_like(acc)
    Y2 = q8.q8_linear_generic(Xd, Wq, S_w, S_x_dev, bd, act, workspace=ws, dbg_acc=acc2)
    assert q8.q8_last_launch_info()["gemm_kernel"] == 2
    assert torch.equal(acc, acc2)
    assert (Y - Y2).abs().max().item() <= REL_TOL * Y2.abs().max().item()


@pytest.mark.parametrize("block_n,ctas", [(32, 1), (64, 1), (128, 1), (256, 1), (256, 2)])
def test_every_tile_shape_matches_the_oracle(block_n, ctas):
    """Each instantiation of the tcgen05 kernel, forced through the tuning hook, on ragged shapes."""
    from tests.gpu_util import check_linear
    try:
        q8.q8_tune_gemm_tile(block_n, ctas)
        for (Mm, Nn, Kk, act) in [(300, 200, 400, 1), (1000, 520, 272, 0), (515, 1030, 144, 1)]:
            X = synth.activation(Mm, Kk, seed=1100 + Mm)
            W = synth.weight(Nn, Kk, seed=1101 + Mm)
            bb = synth.bias(Nn, seed=1102 + Mm)
            info = check_linear(X, W, bb, act=act)
            assert (info["block_n"], info["ctas"]) == (block_n, ctas)
    finally:
        q8.q8_tune_gemm_tile(0, 0)
    with pytest.raises(q8.Q8Error):
        q8.q8_tune_gemm_tile(48, 1)


@pytest.mark.parametrize("M,N,K,act", [(20000, 1000, 128, 1), (19463, 1088, 160, 0), (21000, 520, 144, 1)])
def test_split_tail_of_the_pair_schedule_matches_the_oracle(M, N, K, act):
    """Shapes whose 256 x 256 tiles do not fill the last round over the SM pairs: the tail is cut into
    narrower tiles (ragged in M, N and K here), and the result is the oracle's either way."""
    from tests.gpu_util import check_linear
    X = synth.activation(M, K, seed=1200 + N)
    W = synth.weight(N, K, seed=1201 + N)
    bb = synth.bias(N, seed=1202 + N)
    tiles = -(-M // 256) * -(-N // 256)
    try:
        q8.q8_tune_gemm_tile(256, 2)
        info = check_linear(X, W, bb, act=act)
        assert (info["block_n"], info["ctas"]) == (256, 2)
        units = info["grid"] // 2  # SM pairs the launch ran on
        rest = tiles % units
        expect = 1 if (tiles <= units or rest == 0) else (4 if rest * 4 <= units else (2 if rest * 2 <= units else 1))
        assert q8.q8_last_launch_tail_split() == expect
        q8.q8_tune_gemm_tail_split(False)
        check_linear(X, W, bb, act=act)
        assert q8.q8_last_launch_tail_split() == 1
    finally:
        q8.q8_tune_gemm_tail_split(True)
        q8.q8_tune_gemm_tile(0, 0)


@pytest.mark.parametrize("warps", [8, 16])
def test_both_epilogue_widths_of_the_pair_kernel_match_the_oracle(warps):
    from tests.gpu_util import check_linear
    try:
        q8.q8_tune_gemm_tile(256, 2)
        q8.q8_tune_gemm_epilogue_warps(warps)
        for (Mm, Nn, Kk, act) in [(700, 520, 272, 1), (515, 1030, 144, 0)]:
            X = synth.activation(Mm, Kk, seed=1300 + Mm)
            W = synth.weight(Nn, Kk, seed=1301 + Mm)
            bb = synth.bias(Nn, seed=1302 + Mm)
            info = check_linear(X, W, bb, act=act)
            assert (info["block_n"], info["ctas"]) == (256, 2)
    finally:
        q8.q8_tune_gemm_epilogue_warps(0)
        q8.q8_tune_gemm_tile(0, 0)
    with pytest.raises(q8.Q8Error):
        q8.q8_tune_gemm_epilogue_warps(12)


@pytest.mark.parametrize("block_n,ctas,warps", [(32, 1, 0), (64, 1, 0), (128, 1, 0), (256, 1, 0), (256, 2, 8), (256, 2, 16)])
def test_int8_only_output_of_every_tile_shape(block_n, ctas, warps):
    """The Int8-only output (no fp32 Y; what FFN1 hands to FFN2) leaves full-width tiles through staged TMA
    stores and narrow or ragged ones lane by lane: either way it must be Eq. 1 applied to exactly the fp32
    value the plain call stores, and nothing may be written outside the matrix."""
    shapes = [(515, 1040, 272, 1), (700, 528, 144, 0), (100, 16, 64, 1)]
    if ctas == 2:
        shapes.append((20000, 1008, 128, 1))  # partial last round: tail tiles cut into narrower ones
    S_y = dev(np.array([23.0], np.float32))
    try:
        q8.q8_tune_gemm_tile(block_n, ctas)
        q8.q8_tune_gemm_epilogue_warps(warps)
        for (Mm, Nn, Kk, act) in shapes:
            Xq = dev((synth.token_ids(Mm * Kk, 255, seed=1600 + Mm) - 127).astype(np.int8).reshape(Mm, Kk))
            Wq, S_w = q8.q8_quantize_weight(dev(synth.weight(Nn, Kk, seed=1601 + Mm)))
            bb = dev(synth.bias(Nn, seed=1602 + Mm))
            S_x = dev(np.array([6.0], np.float32))
            Y = q8.q8_linear_q(Xq, S_x, Wq, S_w, bb, act)
            assert (q8.q8_last_launch_info()["block_n"], q8.q8_last_launch_info()["ctas"]) == (block_n, ctas)
            buf = torch.full((Mm * Nn + 256,), 77, dtype=torch.int8, device="cuda")
            Yq = buf[128: 128 + Mm * Nn].view(Mm, Nn)
            st = torch.zeros(1, dtype=torch.int32, device="cuda")
            q8.q8_linear_q_requant(Xq, S_x, Wq, S_w, bb, act, S_y, Yq=Yq, dev_status=st)
            assert q8.q8_poll_status(st) == (q8.Q8_OK, 0)
            assert np.array_equal(Yq.cpu().numpy(), o.quantize(Y.cpu().numpy(), 23.0)), (Mm, Nn, Kk)
            assert torch.all(buf[:128] == 77) and torch.all(buf[128 + Mm * Nn:] == 77)
    finally:
        q8.q8_tune_gemm_epilogue_warps(0)
        q8.q8_tune_gemm_tile(0, 0)


def test_int8_only_output_at_full_size():
    """FFN1 of BERT-Large handing its GELU output to FFN2 as Int8 (M = 24576, automatic tile choice: CTA pairs,
    staged TMA stores): equal to Eq. 1 applied to the fp32 output of the plain call, everywhere."""
    K, N, act = 1024, 4096, 1
    Xq = dev((synth.token_ids(M * K, 255, seed=1700) - 127).astype(np.int8).reshape(M, K))
    Wq, S_w = q8.q8_quantize_weight(dev(synth.weight(N, K, seed=1701)))
    bb = dev(synth.bias(N, seed=1702))
    S_x = dev(np.array([4.25], np.float32))
    S_y = dev(np.array([37.5], np.float32))
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    Y = q8.q8_linear_q(Xq, S_x, Wq, S_w, bb, act, dev_status=st)
    Yq = q8.q8_linear_q_requant(Xq, S_x, Wq, S_w, bb, act, S_y, dev_status=st)
    info = q8.q8_last_launch_info()
    assert q8.q8_poll_status(st) == (q8.Q8_OK, 0)
    assert (info["gemm_kernel"], info["block_n"], info["ctas"]) == (1, 256, 2)
    # the fp32 output of the plain call against the oracle's steps on all rows (Int8 GEMM, Int32 bias, dequantise,
    # GELU), then the Int8 output against the oracle's Eq. 1 applied to that fp32 output, everywhere
    Wq_h, S_w_h = Wq.cpu().numpy(), S_w.item()
    acc_ref, bad = o.gemm_s8(Xq.cpu().numpy(), Wq_h)
    acc_ref, bad2 = o.add_bias(acc_ref, o.quantize_bias(bb.cpu().numpy(), 4.25, S_w_h))
    assert bad == 0 and bad2 == 0
    y_ref = o.gelu(o.dequantize(acc_ref, 4.25, S_w_h))
    del acc_ref
    Yh = Y.cpu().numpy()
    assert np.abs(Yh - y_ref).max() <= REL_TOL * np.abs(y_ref).max()
    Yq_h = Yq.cpu().numpy()
    assert np.array_equal(Yq_h, o.quantize(Yh, 37.5))
    # against the oracle's own fp64 output the Int8 value may differ by one step, and only where y * S_y sits
    # within fp32 rounding of a tie
    d = np.abs(Yq_h.astype(np.int16) - o.quantize(y_ref.astype(np.float32), 37.5).astype(np.int16))
    assert d.max() <= 1 and (d != 0).mean() < 1e-3
    del y_ref, Yh, Yq_h, d
    # secondary, on the device: Eq. 1 in plain torch ops (one rounded fp32 multiply, nearest-even, symmetric clamp)
    assert torch.equal(Yq, torch.clamp(torch.round(Y * 37.5), -127, 127).to(torch.int8))


def test_fused_qkv_with_per_layer_scales_at_full_size():
    """BERT-Large Q, K and V as one [3072, 1024] matrix with one Eq. 3 scale per 1024-row layer, M = 24576, in the
    benchmark's launch configuration (CTA pairs): the whole output equals three separate oracle layers."""
    H = 1024
    X = synth.activation(M, H, seed=1800)
    Ws = [synth.normal((H, H), 0.02 * (1 + i), 1801 + i) for i in range(3)]
    bs = [synth.bias(H, 1810 + i) for i in range(3)]
    Wq, S_w = q8.q8_quantize_weight_segments(dev(np.concatenate(Ws)), H)
    S_x = np.float32(4.5)
    acc = torch.empty((M, 3 * H), dtype=torch.int32, device="cuda")
    Y = q8.q8_linear_wseg(dev(X), Wq, S_w, H, dev(np.array([S_x], np.float32)), dev(np.concatenate(bs)), 0, dbg_acc=acc)
    info = q8.q8_last_launch_info()
    assert (info["gemm_kernel"], info["block_n"], info["ctas"]) == (1, 256, 2)
    acc_h, Yh = acc.cpu().numpy(), Y.cpu().numpy()
    for i in range(3):
        Wq_ref, S_ref, _ = o.quantize_weight(Ws[i])
        assert S_w[i].item() == S_ref and np.array_equal(Wq[i * H:(i + 1) * H].cpu().numpy(), Wq_ref)
        ref = o.linear(X, Wq_ref, S_ref, S_x, bs[i], 0)       # all M rows of this layer
        assert np.array_equal(acc_h[:, i * H:(i + 1) * H], ref["acc"]), i
        err = np.abs(Yh[:, i * H:(i + 1) * H] - ref["y"]).max()
        assert err <= REL_TOL * np.abs(ref["y"]).max(), (i, err)


def test_every_tile_shape_gives_the_same_bits():
    """The epilogue arithmetic of an output element does not depend on the tile it falls in: the fp32 output is
    bit-identical across every instantiation of the tcgen05 kernel and the generic kernel's Int32 matrix."""
    Mm, Nn, Kk = 1000, 520, 272
    Xq = dev((synth.token_ids(Mm * Kk, 255, seed=1900) - 127).astype(np.int8).reshape(Mm, Kk))
    Wq, S_w = q8.q8_quantize_weight(dev(synth.weight(Nn, Kk, seed=1901)))
    bb = dev(synth.bias(Nn, seed=1902))
    S_x = dev(np.array([5.5], np.float32))
    outs = []
    try:
        for (bn, ctas, warps) in [(32, 1, 0), (64, 1, 0), (128, 1, 0), (256, 1, 0), (256, 2, 8), (256, 2, 16)]:
            q8.q8_tune_gemm_tile(bn, ctas)
            q8.q8_tune_gemm_epilogue_warps(warps)
            for act in (0, 1):
                acc = torch.empty((Mm, Nn), dtype=torch.int32, device="cuda")
                outs.append((act, q8.q8_linear_q(Xq, S_x, Wq, S_w, bb, act, dbg_acc=acc), acc))
    finally:
        q8.q8_tune_gemm_epilogue_warps(0)
        q8.q8_tune_gemm_tile(0, 0)
    for act, Y, acc in outs[2:]:
        assert torch.equal(Y, outs[act][1]) and torch.equal(acc, outs[act][2])


def test_hbm_peak_probe_runs_and_is_plausible():
    buf = torch.empty(1 << 29, dtype=torch.uint8, device="cuda")
    w = q8.q8_measure_hbm_peak(buf, store=True, repeats=5)
    r = q8.q8_measure_hbm_peak(buf, store=False, repeats=5)
    assert 500.0 < w["gbs"] < 12000.0 and 500.0 < r["gbs"] < 12000.0
    assert buf[:16].cpu().numpy().tolist() != [0] * 16  # the store pass did write
    with pytest.raises(q8.Q8Error):
        q8.q8_measure_hbm_peak(buf[1:], store=True)  # misaligned
    with pytest.raises(q8.Q8Error):
        q8.q8_measure_hbm_peak(buf, store=True, repeats=0)


def test_int8_mma_issue_peak_probe_runs_and_is_plausible():
    """The measurement aid reports a rate between what the GEMM reaches and the datasheet's dense Int8 figure."""
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    for ctas in (1, 2):
        r = q8.q8_measure_int8_mma_peak(ctas, 0.01, dev_status=st)
        assert st.item() == 0
        assert r["sms_used"] == torch.cuda.get_device_properties(0).multi_processor_count // ctas * ctas
        assert 1500.0 < r["tops"] < 6000.0, r
    with pytest.raises(q8.Q8Error):
        q8.q8_measure_int8_mma_peak(3, 0.01)
    with pytest.raises(q8.Q8Error):
        q8.q8_measure_int8_mma_peak(2, 100.0)


def test_empty_problem_is_a_noop():
    Wq = torch.ones((8, 16), dtype=torch.int8, device="cuda")
    S = torch.ones(1, device="cuda")
    X = torch.empty((0, 16), device="cuda")
    Y = q8.q8_linear(X, Wq, S, S, None, 0)
    assert Y.shape == (0, 8)
    assert q8.q8_last_launch_info()["launches"] == 0
    xq, _ = q8.q8_quantize_activation(torch.empty(0, device="cuda"), S)
    assert xq.numel() == 0
    out = q8.q8_embedding(torch.empty(0, dtype=torch.int32, device="cuda"), Wq, S)
    assert out.shape == (0, 16)


@pytest.mark.parametrize("direct", [False, True])
@pytest.mark.parametrize("warps", [8, 16])
def test_both_output_store_paths_of_the_pair_kernel_match_the_oracle(direct, warps):
    """fp32 output staged in shared memory and TMA-stored, or stored straight from the 16 x 256 bit accumulator
    fragments: the oracle's values either way (ragged M, N, K; odd tails; with and without GELU).  A call that also
    wants the debug accumulator takes the staged path whatever the hook says."""
    from tests.gpu_util import check_linear, assert_close_fp, dev
    try:
        q8.q8_tune_gemm_tile(256, 2)
        q8.q8_tune_gemm_epilogue_warps(warps)
        q8.q8_tune_gemm_direct_store(direct)
        for (Mm, Nn, Kk, act) in [(700, 520, 272, 1), (515, 1030, 144, 0), (300, 130, 256, 0), (129, 34, 64, 1)]:
            X = synth.activation(Mm, Kk, seed=1400 + Mm)
            W = synth.weight(Nn, Kk, seed=1401 + Mm)
            bb = synth.bias(Nn, seed=1402 + Mm)
            info = check_linear(X, W, bb, act=act)  # with dbg_Xq / dbg_acc
            assert (info["block_n"], info["ctas"]) == (256, 2)
            staged = 1 if Nn % 4 == 0 else 0  # a TMA store needs a 16-byte row pitch
            assert q8.q8_last_launch_store_mode() == staged
            # the plain call: Y only
            Wq_ref, S_w_ref, _ = o.quantize_weight(W)
            ref = o.linear(X, Wq_ref, S_w_ref, None, bb, act)
            Wq, S_w = q8.q8_quantize_weight(dev(W))
            Ybuf = torch.full((Mm * Nn + 64,), 12345.0, dtype=torch.float32, device="cuda")
            Y = Ybuf[: Mm * Nn].view(Mm, Nn)
            q8.q8_linear(dev(X), Wq, S_w, None, dev(bb), act, Y=Y)
            assert q8.q8_last_launch_store_mode() == (2 if direct else staged)
            assert_close_fp(Y.cpu().numpy(), ref["y"], "Y")
            assert torch.all(Ybuf[Mm * Nn:] == 12345.0)  # nothing stored past the matrix
    finally:
        q8.q8_tune_gemm_direct_store(None)
        q8.q8_tune_gemm_epilogue_warps(0)
        q8.q8_tune_gemm_tile(0, 0)


def test_l2_operand_probe_runs_and_rejects_bad_arguments():
    buf = torch.zeros((1024, 1024), dtype=torch.int8, device="cuda")
    r = q8.q8_measure_l2_operand_peak(buf, 1024, 1024, boxes_per_sm=256, sms_used=4, producers=2)
    assert r["gbs"] > 0 and r["elapsed_ms"] > 0
    for bad in [dict(rows=100), dict(K=100), dict(producers=5), dict(sms_used=100000)]:
        kw = dict(rows=1024, K=1024, boxes_per_sm=16, sms_used=1, producers=1)
        kw.update(bad)
        with pytest.raises(q8.Q8Error):
            q8.q8_measure_l2_operand_peak(buf, **kw)
