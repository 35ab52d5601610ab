"""Pins for the oracle's rotary embedding and position-id variants: the rotation against complex
multiplication (a library routine), closed forms, the properties that define a rotary embedding
(norms kept, scores depend on the position difference only), and the ids against the paper's
Eq. 14 statements and the generator listing's two position types.  No GPU is involved."""

import numpy as np
import pytest

import oracle


def _rand(shape, seed):
    return np.random.default_rng(seed).normal(size=shape)


def test_rotation_equals_complex_multiplication():
    S, D = 9, 8
    x = _rand((2, S, D), 1)
    pos = np.array([0, 1, 2, 5, 7, 100, 101, 4095, 32767])
    got = oracle.rope_rotate(x, pos, 10000.0)
    z = x[..., : D // 2] + 1j * x[..., D // 2:]
    w = np.exp(1j * pos[:, None] * 10000.0 ** (-2.0 * np.arange(D // 2) / D)[None, :])
    want = z * w
    assert np.allclose(got[..., : D // 2], want.real, atol=1e-12) and np.allclose(got[..., D // 2:], want.imag, atol=1e-12)


def test_two_features_is_the_plane_rotation_by_the_position():
    x = np.array([[[1.0, 0.0]], [[0.0, 1.0]]])            # D = 2: theta_0 = 1, the angle is the position itself
    for p in (0, 1, 3):
        got = oracle.rope_rotate(x, np.array([p]))
        assert np.allclose(got[0, 0], [np.cos(p), np.sin(p)]) and np.allclose(got[1, 0], [-np.sin(p), np.cos(p)])


def test_norms_are_kept_and_scores_depend_on_the_position_difference_only():
    D = 16
    q, k = _rand((1, D), 2), _rand((1, D), 3)
    base = None
    for m, n in ((5, 2), (105, 102), (4003, 4000)):
        qm, kn = oracle.rope_rotate(q, np.array([m])), oracle.rope_rotate(k, np.array([n]))
        assert np.isclose(np.linalg.norm(qm), np.linalg.norm(q)) and np.isclose(np.linalg.norm(kn), np.linalg.norm(k))
        s = float((qm * kn).sum())
        base = s if base is None else base
        assert np.isclose(s, base, atol=1e-9)
    assert np.allclose(oracle.rope_rotate(q, np.array([0])), q)
    twice = oracle.rope_rotate(oracle.rope_rotate(q, np.array([7])), np.array([11]))
    assert np.allclose(twice, oracle.rope_rotate(q, np.array([18])))


@pytest.mark.parametrize("n,c,t,tail", [(3, 2, 2, 1), (2, 4, 4, 0), (4, 8, 16, 5)])
def test_position_ids_follow_eq14_and_the_listing(n, c, t, tail):
    tc = c * t
    chunk, zone, offset, _, _ = oracle.layout_index(n, c, t, tail)
    inter = oracle.position_ids(n, c, t, tail)
    cont = oracle.position_ids(n, c, t, tail, position_type="contiguous")
    for y in range(n):
        mem = (chunk == y) & (zone == 1)
        # the listing at the moment chunk y is compressed: cursor = (y+1)*tc, read_len = tc, mem_cursor = y*t
        cursor, mem_cursor = (y + 1) * tc, y * t
        assert inter[mem].tolist() == list(range(cursor - tc + c - 1, cursor, c))
        assert cont[mem].tolist() == list(range(mem_cursor, mem_cursor + t))
        # Eq. 14's two purposes: reading ids are the original ones; the last memory id is one below the next chunk's first
        read = (chunk == y) & (zone == 0)
        assert inter[read].tolist() == list(range(y * tc, (y + 1) * tc))
        assert inter[mem][-1] + 1 == (y + 1) * tc
    other = zone != 1
    assert np.array_equal(inter[other], cont[other])


def test_rope_apply_uses_the_layout_ids():
    n, c, t, tail = 2, 2, 2, 1
    S = oracle.seq_len(n, c, t, tail)
    q, k = _rand((1, 2, S, 8), 4), _rand((1, 2, S, 8), 5)
    for ptype in ("intermittent", "contiguous"):
        gq, gk = oracle.rope_apply(q, k, n, c, t, tail, position_type=ptype)
        pos = oracle.position_ids(n, c, t, tail, 0, ptype)
        for i in range(S):
            assert np.allclose(gq[0, 1, i], oracle.rope_rotate(q[0, 1, i:i + 1], pos[i:i + 1])[0])
            assert np.allclose(gk[0, 0, i], oracle.rope_rotate(k[0, 0, i:i + 1], pos[i:i + 1])[0])


def test_planted_mistakes_are_caught(monkeypatch):
    from oracle import loma_oracle as lo
    orig = lo.rope_rotate

    def wrong_sign(x, pos, theta_base=10000.0):
        return orig(x, -np.asarray(pos), theta_base)

    def interleaved_pairs(x, pos, theta_base=10000.0):
        x = np.asarray(x, float)
        D = x.shape[-1]
        perm = np.concatenate([np.arange(0, D, 2), np.arange(1, D, 2)])
        return orig(x[..., perm], pos, theta_base)[..., np.argsort(perm)]

    def wrong_exponent(x, pos, theta_base=10000.0):
        return orig(x, pos, theta_base ** 2)

    for fn in (wrong_sign, interleaved_pairs, wrong_exponent):
        with monkeypatch.context() as m:
            m.setattr(lo, "rope_rotate", fn)
            m.setattr(oracle, "rope_rotate", fn)
            with pytest.raises(AssertionError):
                test_rotation_equals_complex_multiplication()
