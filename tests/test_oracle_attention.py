"""Pins for the oracle's masked attention (Algorithm 1's result) -- CPU only."""
import numpy as np
import pytest
import torch

from oracle import attn_c
from oracle import hilberta_oracle as orc


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def test_dense_reduction_matches_sdpa_fp64():
    """tile = HW and no shared region is plain dense attention for any offset."""
    H, nt, D, heads = 4, 3, 8, 2
    S = nt + H * H
    q, k, v = (_rand((1, heads, S, D), s) for s in (1, 2, 3))
    for o in (0, 5):
        M = orc.mask(H, H, H * H, o, 0, nt)
        assert M.all()
        out = orc.attention(q, k, v, M)
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v)).numpy()
        assert np.max(np.abs(out - ref)) < 1e-12


def test_all_image_tokens_shared_is_dense():
    H, D = 4, 8
    q, k, v = (_rand((1, 1, H * H, D), s) for s in (4, 5, 6))
    M = orc.mask(H, H, 4, 1, H, 0)
    assert M.all()
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v)).numpy()
    assert np.max(np.abs(orc.attention(q, k, v, M) - ref)) < 1e-12


def test_masked_matches_sdpa_with_bool_mask_and_scale():
    H, nt, D, heads = 8, 5, 16, 2
    S = nt + H * H
    q, k, v = (_rand((2, heads, S, D), s) for s in (7, 8, 9))
    M = orc.mask(H, H, 16, 4, 2, nt)
    out = orc.attention(q, k, v, M, scale=0.37)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v),
        attn_mask=torch.from_numpy(M), scale=0.37).numpy()
    assert np.max(np.abs(out - ref)) < 1e-12


def test_block_diagonal_is_independent_dense_attentions():
    """o = 0, no text, no shared region: T separate dense attentions on
    contiguous Hilbert chunks."""
    H, tile, D = 8, 16, 8
    HW = H * H
    q, k, v = (_rand((1, 1, HW, D), s) for s in (10, 11, 12))
    out = orc.attention(q, k, v, orc.mask(H, H, tile, 0, 0, 0))
    d2t = orc.hilbert_d2t(H, H)
    for t in range(HW // tile):
        idx = d2t[t * tile:(t + 1) * tile]
        qq, kk, vv = (torch.from_numpy(x[:, :, idx]) for x in (q, k, v))
        ref = torch.nn.functional.scaled_dot_product_attention(qq, kk, vv).numpy()
        assert np.max(np.abs(out[:, :, idx] - ref)) < 1e-12


def test_closed_forms():
    H, nt, D = 8, 2, 4
    S = nt + H * H
    M = orc.mask(H, H, 16, 3, 2, nt)
    k, v = _rand((1, 1, S, D), 13), _rand((1, 1, S, D), 14)
    # q = 0: uniform weights, output = mean of V over the allowed keys
    out, lse = orc.attention(np.zeros((1, 1, S, D)), k, v, M, return_lse=True)
    for i in range(S):
        assert np.allclose(out[0, 0, i], v[0, 0, M[i]].mean(axis=0), atol=1e-13)
        assert np.isclose(lse[0, 0, i], np.log(M[i].sum()))
    # V = identity columns: outputs are the probabilities, rows sum to one and
    # vanish exactly outside the mask
    q = _rand((1, 1, S, D), 15)
    Dv = S
    out = orc.attention(np.pad(q, ((0, 0),) * 3 + ((0, Dv - D),)), np.pad(k, ((0, 0),) * 3 + ((0, Dv - D),)),
                        np.eye(S)[None, None], M, scale=0.5)
    assert np.allclose(out[0, 0].sum(axis=1), 1.0)
    assert np.all(out[0, 0][~M] == 0.0)
    logits = 0.5 * q[0, 0] @ k[0, 0].T
    i = 17
    p = np.exp(logits[i][M[i]])
    assert np.allclose(out[0, 0, i][M[i]], p / p.sum())
    # a huge scale picks the best allowed key
    out = orc.attention(q, k, v, M, scale=1e4)
    best = np.where(M, q[0, 0] @ k[0, 0].T, -np.inf).argmax(axis=1)
    assert np.allclose(out[0, 0], v[0, 0, best])


def test_rows_form_and_c_oracle_agree_with_full():
    H, nt, D, heads = 8, 5, 16, 3
    S = nt + H * H
    q, k, v = (_rand((2, heads, S, D), s).astype(np.float32) for s in (16, 17, 18))
    M = orc.mask(H, H, 16, 4, 2, nt)
    ig, grp = orc.token_classes(H, H, 16, 4, 2, nt)
    full, lse = orc.attention(q, k, v, M, return_lse=True)
    rows = [0, 4, 5, 30, 68]
    part = orc.attention_rows(q, k, v, ig, grp, rows)
    assert np.max(np.abs(part - full[:, :, rows])) < 1e-12
    c_full, c_lse = attn_c.attention_rows(q, k, v, ig, grp, return_lse=True)
    assert np.max(np.abs(c_full - full)) < 1e-12
    assert np.max(np.abs(c_lse - lse)) < 1e-12
    c_part = attn_c.attention_rows(q, k, v, ig, grp, rows=rows, scale=0.2)
    assert np.max(np.abs(c_part - orc.attention(q, k, v, M, scale=0.2)[:, :, rows])) < 1e-12


def test_c_oracle_dense_vs_sdpa():
    """The C oracle pinned directly to a library routine, not via the numpy one."""
    S, D = 37, 24
    q, k, v = (_rand((1, 2, S, D), s).astype(np.float32) for s in (19, 20, 21))
    ig = np.ones(S, dtype=np.uint8)
    grp = np.full(S, -1, dtype=np.int32)
    out = attn_c.attention_rows(q, k, v, ig, grp)
    ref = torch.nn.functional.scaled_dot_product_attention(
        *(torch.from_numpy(x).double() for x in (q, k, v))).numpy()
    assert np.max(np.abs(out - ref)) < 1e-12


def test_metrics():
    a = np.array([1.0, 2.0, 2.0])
    b = np.array([1.0, 2.0, 5.0])
    assert orc.max_abs_err(b, a) == 3.0
    assert np.isclose(orc.rel_l2_err(b, a), 1.0)
