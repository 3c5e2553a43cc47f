"""q8_linear_noalloc: the layer for callers that are not allowed to allocate device memory (an engine
plugin, a serving loop with pre-partitioned memory).  Its scratch is a fixed array inside the library,
so its results must equal q8_linear's on the same inputs, call after call, although every call reuses
the same scratch.  Collected last on purpose: a failure here never hides another test."""
import numpy as np
import pytest
import torch

from oracle import q8_oracle as o
from paper_1910_06188_b200 import binding as q8
from paper_1910_06188_b200 import synth

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _case(M, N, K, act, seed, static_scale):
    X = _dev(synth.activation(M, K, seed))
    Wq, S_w = q8.q8_quantize_weight(_dev(synth.weight(N, K, seed + 1)))
    b = _dev(synth.bias(N, seed + 2))
    S_x = torch.full((1,), 21.0, device="cuda") if static_scale else None
    return X, Wq, S_w, S_x, b, act


def _oracle(X, Wq, S_w, S_x, b, act):
    """The CPU oracle on the same inputs (the weight is the library's own Eq. 3 result, checked elsewhere)."""
    return o.linear(X.cpu().numpy(), Wq.cpu().numpy(), S_w.item(), None if S_x is None else S_x.item(),
                    b.cpu().numpy(), act)


def test_noalloc_matches_q8_linear_on_two_calls_in_a_row():
    # two different problems back to back: the second must not see anything of the first in the scratch
    cases = [_case(640, 384, 512, 1, 2001, static_scale=False), _case(300, 200, 272, 0, 2011, static_scale=True)]
    for X, Wq, S_w, S_x, b, act in cases:
        M, K = X.shape
        N = Wq.shape[0]
        want_acc = torch.empty((M, N), dtype=torch.int32, device="cuda")
        want = q8.q8_linear(X, Wq, S_w, S_x, b, act, dbg_acc=want_acc)
        got_acc = torch.empty((M, N), dtype=torch.int32, device="cuda")
        got_xq = torch.empty((M, K), dtype=torch.int8, device="cuda")
        Y = torch.full((M, N), float("nan"), device="cuda")       # caller-owned output, as such callers have it
        got, word = q8.q8_linear_noalloc(X, Wq, S_w, S_x, b, act, Y=Y, dbg_Xq=got_xq, dbg_acc=got_acc)
        assert got.data_ptr() == Y.data_ptr() and word
        assert q8.q8_poll_status_at(word) == (q8.Q8_OK, 0)
        assert torch.equal(got_acc, want_acc)
        tol = 1e-5 * want.abs().max().item()
        assert (got - want).abs().max().item() <= tol
        want_xq, _ = q8.q8_quantize_activation(X, S_x)
        assert torch.equal(got_xq, want_xq)
        # ... and against the CPU oracle: integers bit for bit, fp32 within 1e-5 of the output magnitude
        ref = _oracle(X, Wq, S_w, S_x, b, act)
        assert np.array_equal(got_xq.cpu().numpy(), ref["xq"]) and np.array_equal(got_acc.cpu().numpy(), ref["acc"])
        assert np.abs(got.cpu().numpy() - ref["y"]).max() <= 1e-5 * np.abs(ref["y"]).max()


def test_noalloc_call_leaves_device_memory_as_it_found_it():
    """After a warm-up call, a call with caller-owned outputs takes no device memory: neither the driver's free
    byte count nor torch's allocator statistics move across it."""
    X, Wq, S_w, S_x, b, act = _case(512, 256, 384, 1, 2021, static_scale=True)
    Y = torch.empty((512, 256), device="cuda")
    q8.q8_linear_noalloc(X, Wq, S_w, S_x, b, act, Y=Y)      # warm-up: kernels and the scratch array get loaded
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    got, _ = q8.q8_linear_noalloc(X, Wq, S_w, S_x, b, act, Y=Y)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == (alloc0, reserved0)
    ref = _oracle(X, Wq, S_w, S_x, b, act)
    assert np.abs(got.cpu().numpy() - ref["y"]).max() <= 1e-5 * np.abs(ref["y"]).max()


def test_noalloc_refuses_activations_beyond_its_fixed_scratch():
    Wq = torch.ones((8, 16), dtype=torch.int8, device="cuda")
    S = torch.ones(1, device="cuda")
    M = q8.Q8_NOALLOC_MAX_MK // 16 + 1
    X = torch.zeros((M, 16), device="cuda")
    with pytest.raises(q8.Q8Error) as e:
        q8.q8_linear_noalloc(X, Wq, S, S, None, 0)
    assert e.value.status == q8.Q8_ERR_WORKSPACE
    # the largest accepted size still works (and flags the all-zero activation through the status word)
    X = torch.zeros((M - 1, 16), device="cuda")
    Y, word = q8.q8_linear_noalloc(X, Wq, S, None, None, 0)
    assert q8.q8_poll_status_at(word)[0] == q8.Q8_ERR_SCALE and not Y.any()
