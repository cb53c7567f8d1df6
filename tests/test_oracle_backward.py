"""Pins for the oracle's backward pass (CPU only).

The paper fine-tunes through its kernel (Sec. 4.1) without printing the
backward formulas, so the oracle writes out the derivative of its own forward
definition.  What fixes it from outside: central finite differences of the
oracle's forward, PyTorch's autograd on an independently assembled masked
softmax in float64, and two identities that hold for any mask with all-ones
diagonal (a uniform shift of every key leaves the softmax unchanged, and the
softmax weights of a row sum to one).
"""
import numpy as np
import pytest
import torch

from oracle import attn_c
from oracle import hilberta_oracle as ho


def _case(seed, H, W, tile, offset, shared, n_text, heads=2, D=8):
    rng = np.random.default_rng(seed)
    S = n_text + H * W
    q, k, v, do = (rng.standard_normal((1, heads, S, D)) for _ in range(4))
    M = ho.mask(H, W, tile, offset, shared, n_text)
    return q, k, v, do, M


CASES = [(4, 4, 4, 1, 2, 3), (8, 8, 16, 4, 2, 0), (4, 8, 8, 3, 2, 5), (8, 8, 64, 0, 0, 0)]


@pytest.mark.parametrize("H,W,tile,offset,shared,n_text", CASES)
def test_backward_matches_finite_differences(H, W, tile, offset, shared, n_text):
    q, k, v, do, M = _case(1, H, W, tile, offset, shared, n_text, heads=1, D=4)
    dq, dk, dv = ho.attention_backward(q, k, v, M, do)
    loss = lambda a, b, c: float((ho.attention(a, b, c, M) * do).sum())
    rng = np.random.default_rng(7)
    eps = 1e-5
    for name, x, g in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        for _ in range(12):
            idx = tuple(rng.integers(0, n) for n in x.shape)
            xp, xm = x.copy(), x.copy()
            xp[idx] += eps
            xm[idx] -= eps
            args_p = {"q": (xp, k, v), "k": (q, xp, v), "v": (q, k, xp)}[name]
            args_m = {"q": (xm, k, v), "k": (q, xm, v), "v": (q, k, xm)}[name]
            fd = (loss(*args_p) - loss(*args_m)) / (2 * eps)
            assert abs(fd - g[idx]) <= 1e-7 * max(1.0, abs(fd)), (name, idx, fd, g[idx])


@pytest.mark.parametrize("H,W,tile,offset,shared,n_text", CASES)
def test_backward_matches_torch_autograd(H, W, tile, offset, shared, n_text):
    q, k, v, do, M = _case(2, H, W, tile, offset, shared, n_text)
    tq, tk, tv = (torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in (q, k, v))
    bias = torch.zeros(M.shape, dtype=torch.float64).masked_fill(~torch.tensor(M), float("-inf"))
    out = torch.softmax(tq @ tk.transpose(-1, -2) / np.sqrt(q.shape[-1]) + bias, dim=-1) @ tv
    (out * torch.tensor(do)).sum().backward()
    dq, dk, dv = ho.attention_backward(q, k, v, M, do)
    for got, ref in ((dq, tq.grad), (dk, tk.grad), (dv, tv.grad)):
        assert np.max(np.abs(got - ref.numpy())) < 1e-12


def test_backward_identities():
    q, k, v, do, M = _case(3, 8, 8, 16, 5, 2, 4)
    dq, dk, dv = ho.attention_backward(q, k, v, M, do)
    # shifting every key by the same vector changes no softmax weight
    assert np.max(np.abs(dk.sum(axis=2))) < 1e-12
    # every row's weights sum to one
    assert np.max(np.abs(dv.sum(axis=2) - do.sum(axis=2))) < 1e-12
    # scaling q by a and k by 1/a leaves the output unchanged: <q, dq> = <k, dk> per head
    assert np.allclose((q * dq).sum(axis=(2, 3)), (k * dk).sum(axis=(2, 3)), rtol=0, atol=1e-11)


def test_backward_dense_mask_is_textbook():
    q, k, v, do, _ = _case(4, 4, 4, 16, 0, 0, 0)
    M = np.ones((16, 16), dtype=bool)
    tq, tk, tv = (torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in (q, k, v))
    out = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv)
    (out * torch.tensor(do)).sum().backward()
    dq, dk, dv = ho.attention_backward(q, k, v, M, do)
    for got, ref in ((dq, tq.grad), (dk, tk.grad), (dv, tv.grad)):
        assert np.max(np.abs(got - ref.numpy())) < 1e-12


@pytest.mark.parametrize("H,W,tile,offset,shared,n_text", CASES[:3])
def test_c_backward_matches_numpy_backward(H, W, tile, offset, shared, n_text):
    q, k, v, do, M = _case(5, H, W, tile, offset, shared, n_text, heads=3, D=16)
    q, k, v, do = (x.astype(np.float32) for x in (q, k, v, do))
    is_global, group = ho.token_classes(H, W, tile, offset, shared, n_text)
    dq, dk, dv = ho.attention_backward(q, k, v, M, do)
    cq, ck, cv = attn_c.attention_backward(q, k, v, do, is_global, group)
    for got, ref in ((cq, dq), (ck, dk), (cv, dv)):
        assert np.max(np.abs(got - ref)) < 1e-12
    rows = np.array([0, 5, q.shape[2] - 1], dtype=np.int32)
    cols = np.array([1, q.shape[2] - 2], dtype=np.int32)
    sq, sk, sv = attn_c.attention_backward(q, k, v, do, is_global, group, rows=rows, cols=cols)
    assert np.array_equal(sq, cq[:, :, rows]) and np.array_equal(sk, ck[:, :, cols])
    assert np.array_equal(sv, cv[:, :, cols])


def test_c_backward_matches_torch_autograd_compact_tiling():
    H = W = 8
    groups, offset, shared, n_text = 3, 7, 2, 3
    is_global, group = ho.token_classes_compact(H, W, groups, offset, shared, n_text)
    M = ho.mask_compact(H, W, groups, offset, shared, n_text)
    rng = np.random.default_rng(6)
    S = n_text + H * W
    q, k, v, do = (rng.standard_normal((1, 2, S, 8)).astype(np.float32) for _ in range(4))
    tq, tk, tv = (torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in (q, k, v))
    bias = torch.zeros(M.shape, dtype=torch.float64).masked_fill(~torch.tensor(M), float("-inf"))
    out = torch.softmax(tq @ tk.transpose(-1, -2) / np.sqrt(8) + bias, dim=-1) @ tv
    (out * torch.tensor(do, dtype=torch.float64)).sum().backward()
    cq, ck, cv = attn_c.attention_backward(q, k, v, do, is_global, group)
    for got, ref in ((cq, tq.grad), (ck, tk.grad), (cv, tv.grad)):
        assert np.max(np.abs(got - ref.numpy())) < 1e-12
