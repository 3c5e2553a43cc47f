"""Pins the CPU oracle to values and properties fixed by the paper and by arithmetic.

Nothing here touches the CUDA library.  Expected values come from tests/golden/q8_pins.json
(hand-worked, each with its citation), from closed forms, or from numpy routines that the
oracle itself does not use (int64 matmul, float64 algebra).
"""
import math

import numpy as np
import pytest

from oracle import q8_oracle as o


# ---------------------------------------------------------------- Eq. 2
def test_M_values(pins):
    for b, m in pins["M"]["cases"]:
        assert o.M_of(b) == m


# ---------------------------------------------------------------- Eq. 1 + Eq. 3 hand example
def test_dynamic_scale_hand_example(pins):
    g = pins["dynamic_scale_example"]
    x = np.array(g["x"], np.float32)
    a = o.absmax(x)
    assert a == np.float32(2.0)
    S, flag = o.scale_from_absmax(a)
    assert flag == 0 and S == np.float32(g["S"])
    xq = o.quantize(x, S)
    assert xq.dtype == np.int8 and xq.tolist() == g["xq"]
    deq = xq.astype(np.float64) / float(S)
    assert np.allclose(deq, g["dequant"], rtol=0, atol=1e-15)
    assert np.all(np.abs(deq - x.astype(np.float64)) <= g["bound"] + 1e-15)


def test_ties_round_half_to_even(pins):
    g = pins["ties_half_even"]
    xq = o.quantize(np.array(g["x"], np.float32), g["S"])
    assert xq.tolist() == g["xq"]
    assert xq.tolist() != g["xq_if_half_away"]


def test_clamp_range(pins):
    g = pins["clamp"]
    assert o.quantize(np.array(g["x"], np.float32), g["S"]).tolist() == g["xq"]
    rng = np.random.default_rng(7)
    x = (rng.standard_normal(1_000_000) * 100).astype(np.float32)
    xq = o.quantize(x, 1.7)
    assert xq.min() == -127 and xq.max() == 127  # both ends reached, -128 never
    assert not np.any(xq == -128)


def test_product_is_one_fp32_multiply(pins):
    g = pins["fp32_product"]
    S = np.float32(float.fromhex(g["S_hex"]))
    assert o.quantize(np.array(g["x"], np.float32), S).tolist() == g["xq"]


def test_nonfinite_inputs_are_defined():
    x = np.array([np.nan, np.inf, -np.inf, 1.0], np.float32)
    assert o.quantize(x, 2.0).tolist() == [0, 127, -127, 2]
    assert o.absmax(np.array([np.nan, -3.0, 2.0], np.float32)) == np.float32(3.0)
    assert o.scale_from_absmax(0.0) == (np.float32(1.0), 1)
    assert o.scale_from_absmax(np.inf) == (np.float32(1.0), 1)
    wq, S, flag = o.quantize_weight(np.zeros((3, 4), np.float32))
    assert flag == 1 and S == 1.0 and not wq.any()


def test_symmetry_q_of_minus_x():
    rng = np.random.default_rng(11)
    x = np.concatenate([
        rng.standard_normal(200_000).astype(np.float32) * 40,
        np.arange(-300, 301, dtype=np.float32) * 0.5,       # every tie and the clamp region
    ])
    for S in (1.0, 0.5, 3.1875, 63.5):
        assert np.array_equal(o.quantize(-x, S).astype(np.int32), -o.quantize(x, S).astype(np.int32))


def test_round_trip_error_bound():
    rng = np.random.default_rng(13)
    x = (rng.standard_normal(500_000) * 3).astype(np.float32)
    S, _ = o.scale_from_absmax(o.absmax(x))
    xq = o.quantize(x, S)
    # With the dynamic scale nothing is clamped, so |x - xq/S| <= 0.5/S up to fp32 rounding of x*S.
    err = np.abs(x.astype(np.float64) - xq.astype(np.float64) / float(S))
    slack = 127.0 * 2.0 ** -24 / float(S)
    assert err.max() <= 0.5 / float(S) + slack
    assert err.max() > 0.45 / float(S)      # the bound is nearly attained: it is not vacuous
    assert np.abs(xq).max() == 127          # the largest element maps to +-M exactly (Eq. 3)


def test_quantize_matches_float64_rounding_away_from_ties():
    # Away from ties and from the clamp, Eq. 1 in exact arithmetic gives the same integer.
    rng = np.random.default_rng(17)
    x = (rng.standard_normal(300_000) * 2).astype(np.float32)
    S = np.float32(21.337)
    p = x.astype(np.float64) * float(S)
    frac = np.abs(p - np.floor(p) - 0.5)
    keep = (frac > 1e-4) & (np.abs(p) < 126)
    want = np.rint(p[keep]).astype(np.int8)
    assert np.array_equal(o.quantize(x, S)[keep], want)


def test_weight_scale_is_M_over_max():
    rng = np.random.default_rng(19)
    w = (rng.standard_normal((37, 53)) * 0.02).astype(np.float32)
    wq, S_w, flag = o.quantize_weight(w)
    assert flag == 0
    assert S_w == np.float32(127.0) / np.abs(w).max()
    assert np.abs(wq).max() == 127
    i = np.unravel_index(np.argmax(np.abs(w)), w.shape)
    assert wq[i] == 127 * np.sign(w[i])


# ---------------------------------------------------------------- Int8 GEMM
def test_tiny_gemm_by_hand(pins):
    for key in ("tiny_gemm", "tiny_gemm_rect"):
        g = pins[key]
        acc, bad = o.gemm_s8(np.array(g["xq"], np.int8), np.array(g["wq"], np.int8))
        assert bad == 0 and acc.tolist() == g["acc"]


def test_saturated_dot_products(pins):
    g = pins["saturated_dot"]
    for K, want in g["cases"]:
        a = np.full((1, K), 127, np.int8)
        acc, bad = o.gemm_s8(a, a)
        assert bad == 0 and acc[0, 0] == want
        acc, bad = o.gemm_s8(a, -a)
        assert bad == 0 and acc[0, 0] == -want
    K = g["max_K_without_overflow"] + 1
    a = np.full((1, K), 127, np.int8)
    _, bad = o.gemm_s8(a, a)
    assert bad == 1      # one more term and the Int32 accumulator no longer holds the sum


def test_gemm_against_int64_matmul():
    rng = np.random.default_rng(23)
    for (M, N, K) in [(1, 1, 1), (3, 5, 7), (8, 8, 8), (17, 9, 130), (5, 33, 64)]:
        xq = rng.integers(-127, 128, size=(M, K), dtype=np.int8)
        wq = rng.integers(-127, 128, size=(N, K), dtype=np.int8)
        acc, bad = o.gemm_s8(xq, wq)
        want = xq.astype(np.int64) @ wq.astype(np.int64).T
        assert bad == 0 and np.array_equal(acc.astype(np.int64), want)


# ---------------------------------------------------------------- Eq. 4
def test_ema_hand_example(pins):
    g = pins["ema"]
    st = o.EmaState()
    for m, want in zip(g["maxima"], g["ema"]):
        S = st.update(m, g["decay"])
        assert abs(float(st.ema[0]) - want) <= g["rel_tol"] * want
    assert abs(float(S) - g["S_final"]) <= g["rel_tol"] * g["S_final"]
    assert int(st.n[0]) == 3


def test_ema_fixed_point_and_dynamic_limit():
    st = o.EmaState()
    for _ in range(50):
        st.update(np.float32(3.3), 0.9999)
    assert st.ema[0] == np.float32(3.3)                       # constant sequence: exact fixed point
    assert st.S_x == np.float32(127.0) / np.float32(3.3)
    st = o.EmaState()
    for m in (5.0, 0.25, 9.0):
        st.update(m, 0.0)                                     # decay 0: the EMA is the last maximum
    assert st.ema[0] == np.float32(9.0)
    # ... exactly, also where ema + 1*(m - ema) would not give m back in fp32 (Sec. 4.1: the dynamic scale)
    st = o.EmaState()
    for m in (np.float32(1e8), np.float32(0.3), np.float32(3.0000002), np.float32(1.1)):
        S = st.update(m, 0.0)
        assert st.ema[0] == m and S == np.float32(127.0) / m
    assert np.float32(1e8) + (np.float32(0.3) - np.float32(1e8)) != np.float32(0.3)   # the update formula would give 0
    st = o.EmaState()
    st.update(4.0, 0.9999)
    st.update(8.0, 0.9999)
    assert 4.0 < st.ema[0] < 4.001                            # moves towards the new maximum, slowly


def test_empty_calibration_batch_changes_nothing():
    st = o.EmaState()
    assert st.update_batch(np.zeros(0, np.float32), 0.9) == np.float32(1.0) and int(st.n[0]) == 0 and st.flag == 0
    x = np.array([0.5, -4.0, 1.0], np.float32)
    S = st.update_batch(x, 0.9)
    assert S == np.float32(127.0) / np.float32(4.0) and int(st.n[0]) == 1
    assert st.update_batch(np.zeros(0, np.float32), 0.9) == S and int(st.n[0]) == 1 and st.ema[0] == np.float32(4.0)
    assert st.update_batch(np.array([2.0], np.float32), 0.5) == np.float32(127.0) / np.float32(3.0)


# ---------------------------------------------------------------- bias, dequantise, GELU
def test_bias_hand_example(pins):
    g = pins["bias"]
    bq = o.quantize_bias(np.array([g["b"]], np.float32), g["S_x"], g["S_w"])
    assert bq.tolist() == [g["bq"]]
    acc, bad = o.add_bias(np.array([[g["acc"]]], np.int32), bq)
    assert bad == 0 and acc[0, 0] == g["sum"]
    y = o.dequantize(acc, g["S_x"], g["S_w"])
    assert abs(y[0, 0] - g["y"]) < 1e-15


def test_bias_clamps_at_int32_M():
    bq = o.quantize_bias(np.array([1e30, -1e30, 0.0], np.float32), 4.0, 1000.0)
    assert bq.tolist() == [2 ** 31 - 1, -(2 ** 31 - 1), 0]


def test_bias_ties_round_half_to_even(pins):
    g = pins["bias_ties"]
    bq = o.quantize_bias(np.array(g["b"], np.float32), g["S_x"], g["S_w"])
    assert bq.tolist() == g["bq"]
    assert bq.tolist() != g["bq_if_half_away"]


def test_bias_scale_product_is_rounded_to_fp32_first(pins):
    g = pins["bias_product_fp32"]
    bq = o.quantize_bias(np.array([g["b"], -g["b"]], np.float32), g["S_x"], g["S_w"])
    assert bq.tolist() == [g["bq"], -g["bq"]]
    assert g["bq"] != g["bq_if_product_unrounded"]


def test_bias_add_wraps_and_counts(pins):
    g = pins["bias_add_wraps"]
    acc, bad = o.add_bias(np.array(g["acc"], np.int32), np.array(g["bq"], np.int32))
    assert acc.tolist() == g["sum"] and bad == g["overflows"]
    # the whole layer reports the same condition: a saturated K = 133144 row plus a bias that tips it over
    K = 133144
    X = np.full((1, K), 127.0, np.float32)
    Wq = np.full((1, K), 127, np.int8)
    r = o.linear(X, Wq, 1.0, 1.0, np.array([5000.0], np.float32), 0)
    assert r["flags"] & 2 and r["acc"][0, 0] == 16129 * K + 5000 - 2 ** 32
    r = o.linear(X, Wq, 1.0, 1.0, np.array([4000.0], np.float32), 0)
    assert r["flags"] == 0 and r["acc"][0, 0] == 16129 * K + 4000


def test_gelu_textbook_values(pins):
    g = pins["gelu"]
    got = o.gelu(np.array(g["y"], np.float64))
    assert np.allclose(got, g["gelu"], rtol=0, atol=1e-15)


def test_gelu_minus_identity_is_odd():
    # y*Phi(y) - y*Phi(-y)... the identity gelu(y) - gelu(-y) = y holds for the erf form.
    y = np.linspace(-8, 8, 4001)
    assert np.allclose(o.gelu(y) - o.gelu(-y), y, rtol=0, atol=1e-14)


# ---------------------------------------------------------------- whole layer
def _fake_quant_layer(X, W, b, S_x, S_w):
    """Training-mode FC of Sec. 3 in float64: fake-quantised input times fake-quantised weight."""
    Xh = np.clip(np.rint((X * np.float32(S_x)).astype(np.float64)), -127, 127) / float(S_x)
    Wh = np.clip(np.rint((W * np.float32(S_w)).astype(np.float64)), -127, 127) / float(S_w)
    return Xh @ Wh.T, Xh, Wh


def test_int_path_equals_fake_quant_path():
    rng = np.random.default_rng(29)
    M, N, K = 19, 23, 96
    X = rng.standard_normal((M, K)).astype(np.float32)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    b = (rng.standard_normal(N) * 0.02).astype(np.float32)
    Wq, S_w, _ = o.quantize_weight(W)
    r = o.linear(X, Wq, S_w, None, b, act=0)
    S_x = r["S_x"]
    assert S_x == np.float32(127.0) / np.abs(X).max()
    fq, Xh, Wh = _fake_quant_layer(X, W, b, S_x, S_w)
    bq = np.rint(np.float64(b * (np.float32(S_x) * np.float32(S_w))))
    want = fq + bq / (float(S_x) * float(S_w))
    assert np.allclose(r["y"], want, rtol=1e-12, atol=1e-12)
    # and it approximates the unquantised layer within the propagated rounding bound
    exact = X.astype(np.float64) @ W.astype(np.float64).T + b
    ex, ew = 0.5 / float(S_x), 0.5 / float(S_w)
    bound = (np.abs(X).astype(np.float64).sum(1)[:, None] * ew
             + np.abs(W).astype(np.float64).sum(1)[None, :] * ex
             + K * ex * ew + 0.5 / (float(S_x) * float(S_w)))
    assert np.all(np.abs(r["y"] - exact) <= bound * (1 + 1e-6))
    assert np.abs(r["y"] - exact).max() > 0      # it is a quantised result, not the exact one


def test_linear_reduces_to_integer_matmul():
    rng = np.random.default_rng(31)
    M, N, K = 7, 11, 40
    X = rng.integers(-127, 128, size=(M, K)).astype(np.float32)
    Wq = rng.integers(-127, 128, size=(N, K), dtype=np.int8)
    b = rng.integers(-1000, 1000, size=N).astype(np.float32)
    r = o.linear(X, Wq, 1.0, 1.0, b, act=0)
    want = X.astype(np.int64) @ Wq.astype(np.int64).T + b.astype(np.int64)
    assert np.array_equal(r["xq"].astype(np.float32), X)
    assert np.array_equal(r["acc"].astype(np.int64), want)
    assert np.array_equal(r["y"], want.astype(np.float64))


def test_linear_static_scale_clamps_and_gelu():
    rng = np.random.default_rng(37)
    M, N, K = 9, 6, 32
    X = rng.standard_normal((M, K)).astype(np.float32) * 5
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    Wq, S_w, _ = o.quantize_weight(W)
    S_x = np.float32(20.0)                       # static scale smaller range than the data: clamps
    r0 = o.linear(X, Wq, S_w, S_x, None, act=0)
    r1 = o.linear(X, Wq, S_w, S_x, None, act=1)
    assert np.abs(r0["xq"]).max() == 127 and (np.abs(X * S_x) > 127.5).any()
    want = np.clip(np.rint((X * S_x).astype(np.float64)), -127, 127).astype(np.int64) @ Wq.astype(np.int64).T
    assert np.array_equal(r0["acc"].astype(np.int64), want)
    y = want / (float(S_x) * float(S_w))
    phi = np.array([0.5 * (1 + math.erf(v / math.sqrt(2))) for v in y.ravel()]).reshape(y.shape)
    assert np.allclose(r1["y"], y * phi, rtol=1e-13, atol=1e-15)
    assert np.array_equal(r0["acc"], r1["acc"])


def test_linear_entry_matches_full():
    rng = np.random.default_rng(41)
    xq = rng.integers(-127, 128, size=(4, 50), dtype=np.int8)
    wq = rng.integers(-127, 128, size=(3, 50), dtype=np.int8)
    full = xq.astype(np.int64) @ wq.astype(np.int64).T
    for m in range(4):
        for n in range(3):
            assert o.linear_entry(xq[m], wq[n], 17) == full[m, n] + 17


# ---------------------------------------------------------------- embedding
def test_embedding_gather_and_bound():
    rng = np.random.default_rng(43)
    V, H, T = 50, 24, 31
    E = (rng.standard_normal((V, H)) * 0.02).astype(np.float32)
    Eq, S_e, _ = o.quantize_weight(E)
    ids = rng.integers(0, V, size=T).astype(np.int32)
    rows, out, bad = o.embedding(ids, Eq, S_e)
    assert bad == 0
    assert np.array_equal(rows, Eq[ids])                        # the layer returns Int8 rows of its table
    assert np.array_equal(out, Eq[ids].astype(np.float64) / float(S_e))
    assert np.abs(out - E[ids]).max() <= 0.5 / float(S_e) * (1 + 1e-5)
    ids[3], ids[7] = -1, V
    rows, out, bad = o.embedding(ids, Eq, S_e)
    assert bad == 2 and not rows[3].any() and not out[7].any()


# ---------------------------------------------------------------- FP32-kept encoder operations (Sec. 3)
def test_layernorm_hand_example_and_moments():
    # x = [1,2,3,4]: mean 2.5, biased variance 1.25 -> (x - 2.5) / sqrt(1.25)
    x = np.array([[1.0, 2.0, 3.0, 4.0]], np.float32)
    want = (np.array([1.0, 2.0, 3.0, 4.0]) - 2.5) / math.sqrt(1.25)
    assert np.allclose(o.add_layernorm(x, eps=0.0), want, rtol=0, atol=1e-15)
    rng = np.random.default_rng(51)
    x = rng.standard_normal((7, 96)).astype(np.float32) * 3 + 1
    r1 = rng.standard_normal((7, 96)).astype(np.float32)
    g = rng.standard_normal(96).astype(np.float32)
    b = rng.standard_normal(96).astype(np.float32)
    y = o.add_layernorm(x, r1)
    assert np.allclose(y.mean(1), 0, atol=1e-12) and np.allclose(y.var(1), 1, atol=1e-9)
    z = o.add_layernorm(x, r1, None, g, b)
    assert np.allclose(z, y * g.astype(np.float64) + b.astype(np.float64), atol=1e-12)
    # the residual really is added before normalising
    assert np.allclose(o.add_layernorm(x, r1), o.add_layernorm((x.astype(np.float64) + r1).astype(np.float32)), atol=1e-5)
    assert not np.allclose(o.add_layernorm(x, r1), o.add_layernorm(x))


def test_attention_special_cases_and_numpy():
    rng = np.random.default_rng(53)
    B, S, heads, d = 2, 9, 3, 64
    H = heads * d
    qkv = rng.standard_normal((B * S, 3 * H)).astype(np.float32)
    got = o.attention(qkv, B, S, heads)
    # independent numpy evaluation of softmax(q k^T / sqrt d) v
    q = qkv[:, :H].reshape(B, S, heads, d).astype(np.float64)
    k = qkv[:, H:2 * H].reshape(B, S, heads, d).astype(np.float64)
    v = qkv[:, 2 * H:].reshape(B, S, heads, d).astype(np.float64)
    sc = np.einsum("bihd,bjhd->bhij", q, k) / 8.0
    p = np.exp(sc - sc.max(-1, keepdims=True))
    p /= p.sum(-1, keepdims=True)
    want = np.einsum("bhij,bjhd->bihd", p, v).reshape(B * S, H)
    assert np.allclose(got, want, rtol=1e-12, atol=1e-12)
    # identical keys -> uniform weights -> every output is the mean value of its sequence and head
    same = qkv.copy()
    same[:, H:2 * H] = same[0, H:2 * H]
    got = o.attention(same, B, S, heads)
    vmean = same[:, 2 * H:].reshape(B, S, H).astype(np.float64).mean(1)
    assert np.allclose(got.reshape(B, S, H), vmean[:, None, :], atol=1e-12)
    # a single token attends to itself only
    one = rng.standard_normal((3, 3 * H)).astype(np.float32)
    assert np.allclose(o.attention(one, 3, 1, heads), one[:, 2 * H:], atol=0)


# ---------------------------------------------------------------- training mode (Sec. 2.2, Eq. 5)
def test_fake_quantize_grid_bound_and_idempotence(pins):
    g = pins["dynamic_scale_example"]
    xh = o.fake_quantize(np.array(g["x"], np.float32), g["S"])
    assert np.allclose(xh, g["dequant"], rtol=0, atol=1e-15)            # the hand-worked dequantised values
    rng = np.random.default_rng(61)
    x = (rng.standard_normal(100_000) * 2).astype(np.float32)
    S, _ = o.scale_from_absmax(o.absmax(x))
    xh = o.fake_quantize(x, S)
    assert np.abs(xh - x).max() <= 0.5 / float(S) * (1 + 1e-5)           # rounding error bound of Eq. 1
    k = xh * float(S)
    assert np.allclose(k, np.rint(k), atol=1e-9) and np.abs(np.rint(k)).max() == 127   # values sit on the Int8 grid
    assert np.array_equal(o.fake_quantize(xh.astype(np.float32), S), xh)  # quantising a grid value changes nothing
    assert np.array_equal(o.fake_quantize(-x, S), -xh)


def test_straight_through_estimator_is_identity():
    g = np.random.default_rng(63).standard_normal(1000).astype(np.float32)
    assert np.array_equal(o.ste_backward(g), g.astype(np.float64))       # Eq. 5: gradient passes unchanged
