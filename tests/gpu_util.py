"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI, run the oracle on
the same seeded inputs, and compare in the classes the method fixes (integers bit-exact, fp32
outputs within 1e-5 of the output magnitude)."""
import numpy as np
import torch

from oracle import q8_oracle as o
from paper_1910_06188_b200 import binding as q8

REL_TOL = 1e-5  # max |Y_gpu - Y_oracle| <= REL_TOL * max |Y_oracle|


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def assert_close_fp(y_gpu: np.ndarray, y_ref: np.ndarray, what=""):
    scale = float(np.abs(y_ref).max())
    err = float(np.abs(y_gpu.astype(np.float64) - y_ref).max())
    assert err <= REL_TOL * max(scale, 1e-30), f"{what}: max abs err {err:.3e} vs {REL_TOL}*{scale:.3e}"


def check_linear(X, W, b, act, S_x=None, fn=None, canary=True):
    """Runs q8_linear (or `fn`) on device copies of the numpy inputs and compares every output class
    with the oracle.  Returns the launch info of the call."""
    fn = fn or q8.q8_linear
    M, K = X.shape
    N = W.shape[0]
    Wq_ref, S_w_ref, _ = o.quantize_weight(W)
    ref = o.linear(X, Wq_ref, S_w_ref, S_x, b, act)

    Wq, S_w = q8.q8_quantize_weight(dev(W))
    assert np.array_equal(Wq.cpu().numpy(), Wq_ref), "W_q differs"
    assert S_w.cpu().numpy()[0] == S_w_ref, "S_w differs"

    Xd = dev(X)
    bd = dev(b) if b is not None else None
    Sx_d = dev(np.array([S_x], np.float32)) if S_x is not None else None
    # canary rows after Y and dbg buffers catch out-of-bounds stores
    pad = 64 if canary else 0
    Ybuf = torch.full((M * N + pad,), 12345.0, dtype=torch.float32, device="cuda")
    Abuf = torch.full((M * N + pad,), -777, dtype=torch.int32, device="cuda")
    Qbuf = torch.full((M * K + pad,), 99, dtype=torch.int8, device="cuda")
    Y = Ybuf[: M * N].view(M, N)
    dbg_acc = Abuf[: M * N].view(M, N)
    dbg_Xq = Qbuf[: M * K].view(M, K)
    ws = q8.new_workspace(M, N, K)
    fn(Xd, Wq, S_w, Sx_d, bd, act, Y=Y, workspace=ws, dbg_Xq=dbg_Xq, dbg_acc=dbg_acc)
    info = q8.q8_last_launch_info()
    code, bits = q8.q8_poll_status(ws)
    assert code == q8.Q8_OK, f"device status {code} bits {bits:#x}"
    assert np.array_equal(dbg_Xq.cpu().numpy(), ref["xq"]), "X_q differs"
    assert np.array_equal(dbg_acc.cpu().numpy(), ref["acc"]), "Int32 accumulator differs"
    assert_close_fp(Y.cpu().numpy(), ref["y"], "Y")
    if S_x is None:
        sx_gpu = ws[4:8].view(torch.float32).cpu().numpy()[0]
        assert sx_gpu == ref["S_x"], "dynamic S_x differs"
    if canary:
        assert torch.all(Ybuf[M * N:] == 12345.0) and torch.all(Abuf[M * N:] == -777) and torch.all(Qbuf[M * K:] == 99)
    return info
