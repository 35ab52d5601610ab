"""Pins for the oracle's backward pass (Section 4.4, gradients of Eq. 7): finite
differences of the oracle's own forward (which the forward pins hold to the
paper), a library autograd on the dense special case, closed forms, and the
structure that the mask of Eq. 1-3 forces on the gradients (the Eq. 10 remark).
No GPU is involved.
"""

import numpy as np
import pytest
import torch

import oracle
from oracle import loma_oracle as lo


def _rand(shape, seed, std=1.0):
    return np.random.default_rng(seed).normal(0.0, std, size=shape)


GEOMS = [(3, 2, 2, 0, 0), (2, 4, 4, 5, 0), (3, 2, 2, 1, 1), (2, 3, 1, 0, 0), (2, 2, 2, 3, 2), (2, 2, 2, 0, 3), (0, 2, 0, 9, 0)]


def _loss(q, k, v, w, n, c, t, tail, flags, scale):
    O, _ = oracle.masked_attn_fwd(q, k, v, n, c, t, tail, flags, scale)
    return float((O * w).sum())


@pytest.mark.parametrize("n,c,t,tail,flags", GEOMS)
def test_gradients_match_central_differences_of_the_forward(n, c, t, tail, flags):
    """dLoss/dx for Loss = sum(O * W) equals the backward's output for dO = W."""
    S, D = oracle.seq_len(n, c, t, tail, flags), 4
    q, k, v, w = (_rand((1, 1, S, D), 10 + i) for i in range(4))
    scale = 0.37
    dq, dk, dv = oracle.masked_attn_bwd(q, k, v, w, n, c, t, tail, flags, scale)
    rng = np.random.default_rng(99)
    eps = 1e-6
    for name, x, g in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        for _ in range(25):
            i, d = int(rng.integers(S)), int(rng.integers(D))
            x0 = x[0, 0, i, d]
            x[0, 0, i, d] = x0 + eps
            up = _loss(q, k, v, w, n, c, t, tail, flags, scale)
            x[0, 0, i, d] = x0 - eps
            dn = _loss(q, k, v, w, n, c, t, tail, flags, scale)
            x[0, 0, i, d] = x0
            fd = (up - dn) / (2 * eps)
            assert abs(fd - g[0, 0, i, d]) < 1e-7 * max(1.0, abs(fd)), (name, i, d, fd, g[0, 0, i, d])


@pytest.mark.parametrize("n,c,t,tail,flags", GEOMS[:5])
def test_gradients_match_library_autograd_on_the_dense_mask(n, c, t, tail, flags):
    S, D = oracle.seq_len(n, c, t, tail, flags), 8
    q, k, v, w = (_rand((2, 2, S, D), 20 + i) for i in range(4))
    M = torch.from_numpy(oracle.dense_mask(n, c, t, tail, flags))
    tq, tk, tv = (torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in (q, k, v))
    A = (tq @ tk.transpose(-1, -2)) / np.sqrt(D)
    O = torch.softmax(A.masked_fill(~M, float("-inf")), dim=-1) @ tv
    (O * torch.from_numpy(w)).sum().backward()
    dq, dk, dv = oracle.masked_attn_bwd(q, k, v, w, n, c, t, tail, flags)
    for got, want in ((dq, tq.grad), (dk, tk.grad), (dv, tv.grad)):
        assert np.abs(got - want.numpy()).max() < 1e-12


def test_single_key_rows_have_zero_score_gradient_and_pass_dO_to_v():
    """A row whose mask allows exactly one key has P = 1 there whatever the scores are:
    dQ of that row is 0 and dV of the key receives dO unchanged (closed form)."""
    # t = 0: causal attention; row 0 sees only key 0
    S, D = 6, 4
    q, k, v, w = (_rand((1, 1, S, D), 30 + i) for i in range(4))
    dq, dk, dv = oracle.masked_attn_bwd(q, k, v, w, 0, 2, 0, S)
    assert np.abs(dq[0, 0, 0]).max() == 0.0
    # the last key is seen only by the last row: dV_last = P[last,last] * dO_last
    _, _, P = oracle.masked_attn_fwd(q, k, v, 0, 2, 0, S, return_p=True)
    assert np.allclose(dv[0, 0, -1], P[0, 0, -1, -1] * w[0, 0, -1], atol=1e-15)


def test_two_key_closed_form():
    """One query, two keys, D = 1: p = sigmoid(scale*q*(k0-k1)); every derivative by hand."""
    qv, k0, k1, v0, v1, g, sc = 0.7, -0.3, 1.1, 2.0, -1.5, 0.9, 0.5
    q = np.array([[qv]]); k = np.array([[k0], [k1]]); v = np.array([[v0], [v1]]); d_o = np.array([[g]])
    dq, dk, dv = oracle.masked_softmax_attention_bwd(q, k, v, d_o, np.ones((1, 2), bool), sc)
    p = 1.0 / (1.0 + np.exp(-sc * qv * (k0 - k1)))
    dp = p * (1 - p)                       # d p / d (a0 - a1)
    assert np.isclose(dv[0, 0], g * p) and np.isclose(dv[1, 0], g * (1 - p))
    assert np.isclose(dq[0, 0], g * (v0 - v1) * dp * sc * (k0 - k1))
    assert np.isclose(dk[0, 0], g * (v0 - v1) * dp * sc * qv)
    assert np.isclose(dk[1, 0], -g * (v0 - v1) * dp * sc * qv)


@pytest.mark.parametrize("n,c,t,tail,flags", GEOMS[:4])
def test_sum_rules(n, c, t, tail, flags):
    """Rows of P sum to one, hence sum_j dV_j = sum_i dO_i; and a softmax is shift invariant,
    hence the score gradients of a row sum to zero: sum_j dK_j = scale * sum_i (sum_j dA_ij) q_i = 0
    when all q_i are equal."""
    S, D = oracle.seq_len(n, c, t, tail, flags), 4
    q, k, v, w = (_rand((1, 1, S, D), 40 + i) for i in range(4))
    dq, dk, dv = oracle.masked_attn_bwd(q, k, v, w, n, c, t, tail, flags)
    assert np.allclose(dv.sum(axis=2), w.sum(axis=2), atol=1e-12)
    q_same = np.broadcast_to(q[:, :, :1, :], q.shape).copy()
    _, dk2, _ = oracle.masked_attn_bwd(q_same, k, v, w, n, c, t, tail, flags)
    assert np.abs(dk2.sum(axis=2)).max() < 1e-12


def test_gradient_support_follows_the_mask_and_reaches_the_memory_zone():
    """Eq. 10 remark: a loss on repetition rows of chunk y reaches k_m, v_m of chunk y -- and,
    by the zero blocks of Eq. 1 and Eq. 3, nothing else but those rows' own q, k, v."""
    n, c, t = 3, 2, 2
    tc, s = c * t, 2 * c * t + t
    S, D = n * s, 4
    q, k, v = (_rand((1, 1, S, D), 50 + i) for i in range(3))
    y = 1
    rep = np.arange(y * s + tc + t, (y + 1) * s)
    mem = np.arange(y * s + tc, y * s + tc + t)
    w = np.zeros((1, 1, S, D)); w[0, 0, rep] = _rand((len(rep), D), 53)
    dq, dk, dv = oracle.masked_attn_bwd(q, k, v, w, n, c, t)
    touched_kv = np.zeros(S, bool); touched_kv[rep] = True; touched_kv[mem] = True
    touched_q = np.zeros(S, bool); touched_q[rep] = True
    assert np.abs(dk[0, 0, ~touched_kv]).max() == 0 and np.abs(dv[0, 0, ~touched_kv]).max() == 0
    assert np.abs(dq[0, 0, ~touched_q]).max() == 0
    assert np.abs(dk[0, 0, mem]).min() > 0 and np.abs(dv[0, 0, mem]).min() > 0
    # a loss on reading rows of the last chunk reaches every earlier memory zone, no repetition key, no later row
    w = np.zeros((1, 1, S, D)); read = np.arange(2 * s, 2 * s + tc); w[0, 0, read] = _rand((tc, D), 54)
    dq, dk, dv = oracle.masked_attn_bwd(q, k, v, w, n, c, t)
    zone = oracle.layout_index(n, c, t)[1]
    chunk = oracle.layout_index(n, c, t)[0]
    assert np.abs(dk[0, 0, zone == 2]).max() == 0 and np.abs(dv[0, 0, zone == 2]).max() == 0
    earlier_mem = (zone == 1) & (chunk < 2)
    assert np.abs(dv[0, 0, earlier_mem]).min() > 0
    own_mem = (zone == 1) & (chunk == 2)
    assert np.abs(dv[0, 0, own_mem]).max() == 0        # reading rows never see their own chunk's memory zone
    assert np.abs(dk[0, 0, (zone == 0) & (chunk < 2)]).max() == 0


@pytest.mark.parametrize("n,c,t,tail,flags", [(3, 2, 2, 1, 0), (2, 4, 4, 5, 1), (3, 2, 4, 0, 2)])
def test_sampled_rows_and_keys_equal_the_full_backward(n, c, t, tail, flags):
    S, D = oracle.seq_len(n, c, t, tail, flags), 8
    q, k, v, w = (_rand((1, 2, S, D), 60 + i) for i in range(4))
    dq, dk, dv = oracle.masked_attn_bwd(q, k, v, w, n, c, t, tail, flags)
    rng = np.random.default_rng(3)
    rows = np.sort(rng.choice(S, min(S, 11), replace=False))
    cols = np.sort(rng.choice(S, min(S, 9), replace=False))
    assert np.abs(oracle.masked_attn_bwd_dq_rows(q, k, v, w, rows, n, c, t, tail, flags) - dq[:, :, rows]).max() < 1e-12
    gk, gv = oracle.masked_attn_bwd_dkv_cols(q, k, v, w, cols, n, c, t, tail, flags, block=7)
    assert np.abs(gk - dk[:, :, cols]).max() < 1e-12 and np.abs(gv - dv[:, :, cols]).max() < 1e-12


def test_planted_mistakes_in_the_backward_are_caught(monkeypatch):
    orig = lo.masked_softmax_attention_bwd

    def no_row_term(q, k, v, d_o, mask, scale=None):     # Jacobian of the softmax without its rank-one part
        q_, k_, v_, g = (np.asarray(a, float) for a in (q, k, v, d_o))
        sc = 1.0 / np.sqrt(q_.shape[-1]) if scale is None else scale
        _, P, _ = lo.masked_softmax_attention(q_, k_, v_, mask, sc)
        dA = P * (g @ v_.T)
        return sc * dA @ k_, sc * dA.T @ q_, P.T @ g

    def scale_forgotten_in_dk(q, k, v, d_o, mask, scale=None):
        dq, dk, dv = orig(q, k, v, d_o, mask, scale)
        sc = 1.0 / np.sqrt(np.asarray(q).shape[-1]) if scale is None else scale
        return dq, dk / sc, dv

    def dk_from_untransposed_scores(q, k, v, d_o, mask, scale=None):   # dA Q in place of dA^T Q (square case)
        q_, k_, v_, g = (np.asarray(a, float) for a in (q, k, v, d_o))
        sc = 1.0 / np.sqrt(q_.shape[-1]) if scale is None else scale
        _, P, _ = lo.masked_softmax_attention(q_, k_, v_, mask, sc)
        dP = g @ v_.T
        dA = P * (dP - (P * dP).sum(1, keepdims=True))
        return sc * dA @ k_, sc * dA @ q_, P.T @ g

    for fn in (no_row_term, scale_forgotten_in_dk, dk_from_untransposed_scores):
        with monkeypatch.context() as m:
            m.setattr(lo, "masked_softmax_attention_bwd", fn)
            with pytest.raises(AssertionError):
                test_gradients_match_central_differences_of_the_forward(3, 2, 2, 0, 0)
