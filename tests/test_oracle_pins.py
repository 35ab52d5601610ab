"""Pins for the CPU oracle: everything here checks oracle/ against something
other than itself -- the paper's block matrices typed out by hand, closed forms,
library routines on the special cases that reduce to them, and invariants that
hold for any correct implementation.  No GPU is involved.
"""

import math
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import loma_oracle as lo


def _load_mask(path):
    rows = [ln.strip() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    return np.array([[ch == "1" for ch in r] for r in rows], bool)


def _rand(shape, seed, std=1.0):
    return np.random.default_rng(seed).normal(0.0, std, size=shape)


GEOMS = [(1, 2, 2, 0), (3, 2, 2, 0), (2, 4, 4, 0), (2, 4, 4, 5), (4, 1, 3, 2), (3, 3, 1, 0), (2, 2, 8, 16)]


# ------------------------------------------------------------------ mask pins

def test_fig5_mask_matches_hand_typed_fixture(golden_dir):
    """Fig. 5 example (t=2, c=2, 12 tokens -> 3 chunks of 10, 30x30)."""
    want = _load_mask(os.path.join(golden_dir, "fig5_mask_t2_c2_n3.txt"))
    assert want.shape == (30, 30) and want.sum() == 126
    got = oracle.dense_mask(3, 2, 2)
    assert got.shape == (30, 30)
    assert np.array_equal(got, want)
    # the entry-wise rule and the sampled-row builder agree with it too
    ent = np.array([[oracle.allowed(i, j, 3, 2, 2) for j in range(30)] for i in range(30)])
    assert np.array_equal(ent, want)
    assert np.array_equal(oracle.mask_rows(list(range(30)), 3, 2, 2), want)


def test_fig5_mask_prior_mem_flag(golden_dir):
    want = _load_mask(os.path.join(golden_dir, "fig5_mask_t2_c2_n3_prior_mem.txt"))
    assert want.sum() == 138
    f = oracle.FLAG_MEM_SEES_PRIOR_MEM
    assert np.array_equal(oracle.dense_mask(3, 2, 2, 0, f), want)
    ent = np.array([[oracle.allowed(i, j, 3, 2, 2, f) for j in range(30)] for i in range(30)])
    assert np.array_equal(ent, want)
    assert np.array_equal(oracle.mask_rows(list(range(30)), 3, 2, 2, 0, f), want)


def _pairs_closed_form(n, c, t, flags=0):
    """Number of ones in Eq. 2, counted block by block:
    per chunk L has tc(tc+1)/2, the memory rows t(tc+t), the repetition rows
    tc(t+1); each of the n(n-1)/2 sub-diagonal blocks has tc*t (plus t*t under
    the prior-memory flag)."""
    tc = t * c
    per_chunk = tc * (tc + 1) // 2 + t * (tc + t) + tc * (t + 1)
    cross = tc * t + (t * t if flags & 1 else 0)
    return n * per_chunk + cross * n * (n - 1) // 2


@pytest.mark.parametrize("n,c,t", [(3, 2, 2), (2, 4, 4), (5, 3, 2), (4, 1, 5), (6, 2, 8)])
@pytest.mark.parametrize("flags", [0, 1])
def test_mask_popcount_closed_form(n, c, t, flags):
    assert oracle.dense_mask(n, c, t, 0, flags).sum() == _pairs_closed_form(n, c, t, flags)


def test_popcount_values_for_named_workloads():
    assert _pairs_closed_form(3, 2, 2) == 126
    assert _pairs_closed_form(2, 4, 4) == 656          # tiny config, of 72*72 = 5184
    assert _pairs_closed_form(32, 4, 16) == 650240     # 4608-token training layout
    assert _pairs_closed_form(128, 8, 32) == 73056256  # 69632-token training layout
    assert oracle.dense_mask(2, 4, 4).sum() == 656
    # the row-sampled builder reproduces the closed form at full size without the S x S array
    n, c, t = 32, 4, 16
    S = oracle.seq_len(n, c, t)
    assert S == 4608
    total = 0
    for lo_ in range(0, S, 512):
        total += int(oracle.mask_rows(range(lo_, lo_ + 512), n, c, t).sum())
    assert total == 650240


@pytest.mark.parametrize("n,c,t,tail", GEOMS)
@pytest.mark.parametrize("flags", [0, 1])
def test_three_mask_builders_agree(n, c, t, tail, flags):
    S = oracle.seq_len(n, c, t, tail)
    D = oracle.dense_mask(n, c, t, tail, flags)
    E = np.array([[oracle.allowed(i, j, n, c, t, flags) for j in range(S)] for i in range(S)])
    R = oracle.mask_rows(list(range(S)), n, c, t, tail, flags)
    assert np.array_equal(D, E) and np.array_equal(D, R)


@pytest.mark.parametrize("n,c,t,tail", GEOMS)
def test_mask_structure_criteria(n, c, t, tail):
    """The three criteria of Section 4.3, checked zone by zone on the dense mask."""
    tc, s = t * c, oracle.chunk_len(c, t)
    M = oracle.dense_mask(n, c, t, tail)
    S = M.shape[0]
    upper = np.argwhere(np.triu(M, 1))          # only the bidirectional memory zones look ahead
    for i, j in upper:
        assert i // s == j // s and tc <= i % s < tc + t and tc <= j % s < tc + t
    mem_cols = np.zeros(S, bool)
    for y in range(n):
        mem_cols[y * s + tc:y * s + tc + t] = True
    for y in range(n + (1 if tail else 0)):
        base = y * s
        nread = tc if y < n else tail
        for o in range(nread):
            row = M[base + o]
            want = np.zeros(S, bool)
            want[:base] = mem_cols[:base]            # 1. all preceding memory zones
            want[base:base + o + 1] = True           #    + causal inside the reading zone
            assert np.array_equal(row, want)
        if y == n:
            continue
        for j in range(t):
            row = M[base + tc + j]
            want = np.zeros(S, bool)
            want[base:base + tc + t] = True          # 2. own reading zone + bidirectional memory zone
            assert np.array_equal(row, want)
        for o in range(tc):
            i = base + tc + t + o
            want = np.zeros(S, bool)
            want[base + tc:base + tc + t] = True     # 3. only the memory zone right before it
            want[i] = True                           #    and itself (I block of Eq. 1)
            assert np.array_equal(M[i], want)
    # no column of a repetition row is visible to any OTHER row
    for y in range(n):
        for o in range(tc):
            j = y * s + tc + t + o
            col = M[:, j].copy()
            col[j] = False
            assert not col.any()


def test_generation_masks_of_the_listing():
    """Appendix A builds tril(ones(l, l+k), diagonal=k) for l new tokens over k
    cached entries and ones(t, t+tc) for the compress pass; the training mask
    restricted to the keys that survive in the cache must be exactly these."""
    n, c, t = 3, 2, 4
    tc, s = t * c, oracle.chunk_len(c, t)
    M = oracle.dense_mask(n, c, t, tail_read=5)
    for y in range(n + 1):
        nread = tc if y < n else 5
        rows = [y * s + o for o in range(nread)]
        cached_mem = [x * s + tc + j for x in range(y) for j in range(t)]
        cols = cached_mem + rows
        sub = M[np.ix_(rows, cols)]
        k = len(cached_mem)
        want = torch.tril(torch.ones(nread, nread + k), diagonal=k).numpy().astype(bool)
        assert np.array_equal(sub, want)
        others = np.setdiff1d(np.arange(M.shape[1]), cols)
        assert not M[np.ix_(rows, others)].any()
        if y < n:
            mrows = [y * s + tc + j for j in range(t)]
            mcols = rows + mrows                     # [read_kv ; own <m> keys]
            assert M[np.ix_(mrows, mcols)].all()
            others = np.setdiff1d(np.arange(M.shape[1]), mcols)
            assert not M[np.ix_(mrows, others)].any()


# ------------------------------------------------------------- index-map pins

@pytest.mark.parametrize("c,t", [(2, 2), (4, 4), (4, 16), (8, 16), (3, 5), (1, 7)])
def test_memory_position_ids_match_the_listing_range(c, t):
    n, tc = 4, t * c
    s = oracle.chunk_len(c, t)
    ch, zn, of, src, pos = oracle.layout_index(n, c, t)
    for y in range(n):
        cursor = (y + 1) * tc          # generator cursor after reading chunk y
        want = list(range(cursor - tc + c - 1, cursor, c))   # 'intermittent' ids of the listing
        got = pos[y * s + tc:y * s + tc + t].tolist()
        assert got == want
        assert got[-1] == (y + 1) * tc - 1      # contiguous with the next chunk's first reading id
        assert pos[y * s:y * s + tc].tolist() == list(range(y * tc, (y + 1) * tc))  # reading ids preserved
        assert (src[y * s + tc:y * s + tc + t] == -1).all()
        assert src[y * s:y * s + tc].tolist() == list(range(y * tc, (y + 1) * tc))
        # Eq. 13: the <r> row sits t(c+1) rows after the reading row whose token it reproduces
        for o in range(tc):
            i = y * s + tc + t + o
            assert zn[i] == oracle.ZONE_REP and src[i] == src[i - t * (c + 1)]


@pytest.mark.parametrize("c,t,n", [(2, 2, 3), (4, 16, 5), (8, 32, 2), (3, 5, 4)])
def test_laid_out_length_identity(c, t, n):
    """Section 5.1: s original tokens lay out to 2s + floor(s/c) rows."""
    s_orig = n * t * c
    assert oracle.seq_len(n, c, t) == 2 * s_orig + s_orig // c
    assert oracle.chunk_len(c, t) == 2 * t * c + t == t * (2 * c + 1)


def test_layout_zones_partition_rows():
    n, c, t, tail = 3, 2, 3, 4
    ch, zn, of, src, pos = oracle.layout_index(n, c, t, tail)
    tc = t * c
    want_zone = ([0] * tc + [1] * t + [2] * tc) * n + [0] * tail
    assert zn.tolist() == want_zone
    want_off = (list(range(tc)) + list(range(t)) + list(range(tc))) * n + list(range(tail))
    assert of.tolist() == want_off
    assert ch.tolist() == sum(([y] * (2 * tc + t) for y in range(n)), []) + [n] * tail
    for i in range(len(zn)):
        assert oracle.decompose(i, n, c, t) == (ch[i], zn[i], of[i])


def test_generation_index_follows_listing_state_machine():
    """Simulate the Appendix A bookkeeping with lists (cache as a Python list)."""
    c, t, n_tok = 3, 2, 40
    tc = c * t
    slot, pos, comp = oracle.generation_index(n_tok, c, t)
    cache, compressed_chunks, cursor = [], 0, 0
    for g in range(n_tok):
        assert slot[g] == len(cache) and pos[g] == cursor
        cache.append(("tok", g))
        cursor += 1
        if len(cache) - compressed_chunks * t == tc:
            assert comp[g] == 1
            mem_cursor = compressed_chunks * t
            assert mem_cursor == len(cache) - tc
            cache = cache[:mem_cursor] + [("mem", compressed_chunks, j) for j in range(t)]
            compressed_chunks += 1
        else:
            assert comp[g] == 0
    # closed form of the same map
    for g in range(n_tok):
        assert slot[g] == (g // tc) * t + g % tc
    s0, p0, c0 = oracle.generation_index(10, 4, 0)
    assert s0.tolist() == list(range(10)) and not c0.any()


# ------------------------------------------------------------ attention pins

def test_softmax_attention_two_key_closed_form():
    """One query, two keys, D=1: p0 = sigmoid(scale*q*(k0-k1)), o = p0*v0+(1-p0)*v1."""
    q, k0, k1, v0, v1, scale = 0.7, 1.3, -0.4, 2.0, -5.0, 0.37
    O, P, lse = oracle.masked_softmax_attention([[q]], [[k0], [k1]], [[v0], [v1]],
                                                np.ones((1, 2), bool), scale)
    p0 = 1.0 / (1.0 + math.exp(-scale * q * (k0 - k1)))
    assert abs(P[0, 0] - p0) < 1e-15 and abs(P[0, 1] - (1 - p0)) < 1e-15
    assert abs(O[0, 0] - (p0 * v0 + (1 - p0) * v1)) < 1e-14
    assert abs(lse[0] - math.log(math.exp(scale * q * k0) + math.exp(scale * q * k1))) < 1e-14
    # default scale is 1/sqrt(D)
    qd, kd = _rand((1, 16), 1), _rand((2, 16), 2)
    _, Pd, _ = oracle.masked_softmax_attention(qd, kd, np.eye(2), np.ones((1, 2), bool))
    a = (qd @ kd.T)[0] / 4.0
    assert np.allclose(Pd[0], np.exp(a) / np.exp(a).sum(), atol=1e-15)


def test_all_ones_mask_equals_library_sdpa():
    """With nothing masked the oracle must equal the library's plain attention
    (non-square shapes so a transposed operand cannot slip through)."""
    R, C, D, Dv = 5, 9, 8, 6
    q, k, v = _rand((R, D), 3), _rand((C, D), 4), _rand((C, Dv), 5)
    O, P, _ = oracle.masked_softmax_attention(q, k, v, np.ones((R, C), bool))
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None], torch.from_numpy(k)[None], torch.from_numpy(v)[None])[0].numpy()
    assert np.allclose(O, ref, atol=1e-13)


@pytest.mark.parametrize("S,D", [(1, 4), (7, 8), (33, 16)])
def test_invariant_a_t0_is_causal_attention(S, D):
    """t = 0: no memory zones, the layout is one reading zone, plain causal SDPA."""
    q, k, v = (_rand((2, 3, S, D), s) for s in (10, 11, 12))
    O, lse = oracle.masked_attn_fwd(q, k, v, 0, 4, 0, tail_read=S)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v), is_causal=True).numpy()
    assert np.allclose(O, ref, atol=1e-13)
    assert np.array_equal(oracle.dense_mask(0, 4, 0, S), np.tril(np.ones((S, S), bool)))


@pytest.mark.parametrize("n,c,t,tail", GEOMS)
def test_invariants_b_and_d_support_and_row_sums(n, c, t, tail):
    S = oracle.seq_len(n, c, t, tail)
    tc, s = t * c, oracle.chunk_len(c, t)
    q, k, v = (_rand((1, 2, S, 8), sd) for sd in (20, 21, 22))
    O, lse, P = oracle.masked_attn_fwd(q, k, v, n, c, t, tail, return_p=True)
    assert np.allclose(P.sum(-1), 1.0, atol=1e-14)                      # (d)
    M = oracle.dense_mask(n, c, t, tail)
    assert np.array_equal(P > 0, np.broadcast_to(M, P.shape))           # weight exactly 0 when blocked
    for y in range(n):                                                  # (b)
        for o in range(tc):
            i = y * s + tc + t + o
            support = set(np.nonzero(P[0, 0, i])[0].tolist())
            assert support == set(range(y * s + tc, y * s + tc + t)) | {i}


@pytest.mark.parametrize("n,c,t,tail", GEOMS)
def test_zero_query_gives_mean_of_allowed_values(n, c, t, tail):
    """q = 0 makes every allowed weight equal: O_i = mean of the allowed V rows,
    lse_i = log(#allowed).  Uses the hand-checkable row structure, not the oracle's mask."""
    S = oracle.seq_len(n, c, t, tail)
    tc, s = t * c, oracle.chunk_len(c, t)
    D = 4
    k, v = _rand((1, 1, S, D), 30), _rand((1, 1, S, D), 31)
    O, lse = oracle.masked_attn_fwd(np.zeros((1, 1, S, D)), k, v, n, c, t, tail)
    for i in range(S):
        y, r = (divmod(i, s) if i < n * s else (n, i - n * s))
        mems = [x * s + tc + j for x in range(y) for j in range(t)]
        if y == n or r < tc:
            cols = mems + list(range(y * s, y * s + r + 1))
        elif r < tc + t:
            cols = list(range(y * s, y * s + tc + t))
        else:
            cols = list(range(y * s + tc, y * s + tc + t)) + [i]
        assert np.allclose(O[0, 0, i], v[0, 0, cols].mean(0), atol=1e-14)
        assert abs(lse[0, 0, i] - math.log(len(cols))) < 1e-13


def test_identity_values_return_the_probabilities_and_brute_force_rows():
    """V = I turns O into P; each P row is then recomputed with scalar loops."""
    n, c, t = 2, 2, 2
    S = oracle.seq_len(n, c, t)
    D = 3
    q, k = _rand((1, 1, S, D), 40), _rand((1, 1, S, D), 41)
    v = np.eye(S)[None, None]
    O, lse = oracle.masked_attn_fwd(q, k, v, n, c, t, scale=0.5)
    M = _load_small_mask_by_criteria(n, c, t)
    for i in range(S):
        w = [math.exp(0.5 * sum(q[0, 0, i, d] * k[0, 0, j, d] for d in range(D))) if M[i][j] else 0.0
             for j in range(S)]
        z = sum(w)
        for j in range(S):
            assert abs(O[0, 0, i, j] - w[j] / z) < 1e-14
        assert abs(lse[0, 0, i] - math.log(z)) < 1e-13


def _load_small_mask_by_criteria(n, c, t):
    """Mask from the three prose criteria of Section 4.3 (lists of allowed columns)."""
    tc, s = t * c, t * (2 * c + 1)
    S = n * s
    M = [[False] * S for _ in range(S)]
    for y in range(n):
        b = y * s
        for o in range(tc):
            for x in range(y):
                for j in range(t):
                    M[b + o][x * s + tc + j] = True
            for o2 in range(o + 1):
                M[b + o][b + o2] = True
        for j in range(t):
            for col in range(b, b + tc + t):
                M[b + tc + j][col] = True
        for o in range(tc):
            i = b + tc + t + o
            for j in range(t):
                M[i][b + tc + j] = True
            M[i][i] = True
    return M


def test_memory_zone_key_permutation_leaves_other_rows_unchanged():
    """Rows outside a memory zone see that zone all-or-nothing, so permuting its
    keys (K and V together) cannot change their outputs."""
    n, c, t = 3, 2, 4
    tc, s = t * c, oracle.chunk_len(c, t)
    S = oracle.seq_len(n, c, t)
    q, k, v = (_rand((1, 1, S, 8), sd) for sd in (50, 51, 52))
    O, _ = oracle.masked_attn_fwd(q, k, v, n, c, t)
    perm = np.arange(S)
    zone = np.arange(1 * s + tc, 1 * s + tc + t)
    perm[zone] = zone[::-1]
    O2, _ = oracle.masked_attn_fwd(q, k[:, :, perm], v[:, :, perm], n, c, t)
    keep = np.setdiff1d(np.arange(S), zone)
    assert np.allclose(O[:, :, keep], O2[:, :, keep], atol=1e-13)


def test_sampled_rows_equal_full_rows():
    n, c, t, tail = 3, 2, 4, 3
    S = oracle.seq_len(n, c, t, tail)
    q, k, v = (_rand((2, 2, S, 8), sd) for sd in (60, 61, 62))
    for flags in (0, 1):
        O, lse = oracle.masked_attn_fwd(q, k, v, n, c, t, tail, flags)
        rows = [0, 5, 8, 11, 19, 20, 27, 40, S - 1]
        Or, lr = oracle.masked_attn_fwd(q, k, v, n, c, t, tail, flags, rows=rows)
        assert np.allclose(O[:, :, rows], Or, atol=1e-14) and np.allclose(lse[:, :, rows], lr, atol=1e-14)


# ------------------------------------------------------------ generation pins

def test_decode_with_empty_memory_is_last_row_of_causal_sdpa():
    B, H, L, D = 2, 2, 11, 8
    q, k, v = (_rand((B, H, L + 1, D), sd) for sd in (70, 71, 72))
    kc = np.zeros((B, H, L + 4, D)); vc = np.zeros((B, H, L + 4, D))
    kc[:, :, :L], vc[:, :, :L] = k[:, :, :L], v[:, :, :L]
    o, lse, kc2, vc2 = oracle.decode_attn(q[:, :, L:], k[:, :, L:], v[:, :, L:], kc, vc, L)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v), is_causal=True).numpy()
    assert np.allclose(o[:, :, 0], ref[:, :, L], atol=1e-13)
    assert np.array_equal(kc2[:, :, :L + 1], k) and np.array_equal(vc2[:, :, :L + 1], v)
    assert np.array_equal(kc2[:, :, L + 1:], kc[:, :, L + 1:])
    assert np.array_equal(kc[:, :, L], np.zeros((B, H, D))), "input cache is not modified"


@pytest.mark.parametrize("flags", [0, 1])
def test_compress_is_unmasked_sdpa_and_cat_compaction(flags):
    B, H, D, c, t, mem_len = 2, 2, 8, 3, 4, 8
    tc = c * t
    cap = mem_len + tc + 3
    kc, vc = _rand((B, H, cap, D), 80), _rand((B, H, cap, D), 81)
    qm, km, vm = (_rand((B, H, t, D), sd) for sd in (82, 83, 84))
    o, lse, nk, nv = oracle.compress_step(qm, km, vm, kc, vc, mem_len, c, t, flags)
    lo_ = 0 if flags else mem_len
    keys = torch.cat([torch.from_numpy(kc[:, :, lo_:mem_len + tc]), torch.from_numpy(km)], dim=2)
    vals = torch.cat([torch.from_numpy(vc[:, :, lo_:mem_len + tc]), torch.from_numpy(vm)], dim=2)
    ref = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(qm), keys, vals).numpy()
    assert np.allclose(o, ref, atol=1e-13)
    # compaction: cat([old[:, :, :mem_cursor], mem[:, :, -t:]], dim=2), bit for bit
    want_k = torch.cat([torch.from_numpy(kc)[:, :, :mem_len], torch.from_numpy(km)[:, :, -t:]], dim=2).numpy()
    want_v = torch.cat([torch.from_numpy(vc)[:, :, :mem_len], torch.from_numpy(vm)[:, :, -t:]], dim=2).numpy()
    assert nk.shape == (B, H, mem_len + t, D)
    assert np.array_equal(nk, want_k) and np.array_equal(nv, want_v)


@pytest.mark.parametrize("n,c,t,tail", [(2, 4, 4, 0), (3, 2, 2, 3), (2, 3, 5, 1), (4, 1, 3, 0)])
@pytest.mark.parametrize("flags", [0, 1])
def test_invariant_c_incremental_generation_equals_one_shot(n, c, t, tail, flags):
    S = oracle.seq_len(n, c, t, tail)
    tc, s = t * c, oracle.chunk_len(c, t)
    D = 8
    q, k, v = (_rand((1, 2, S, D), sd) for sd in (90, 91, 92))
    O, _ = oracle.masked_attn_fwd(q, k, v, n, c, t, tail, flags)
    Og, kc, vc, length = oracle.replay_generation(q, k, v, n, c, t, tail, flags)
    zn = oracle.layout_index(n, c, t, tail)[1]
    live = zn != oracle.ZONE_REP
    assert np.isnan(Og[:, :, ~live]).all()
    assert np.allclose(Og[:, :, live], O[:, :, live], atol=1e-13)
    mem_rows = [y * s + tc + j for y in range(n) for j in range(t)]
    tail_rows = list(range(n * s, S))
    assert length == n * t + tail
    assert np.array_equal(kc[:, :, :length], k[:, :, mem_rows + tail_rows])
    assert np.array_equal(vc[:, :, :length], v[:, :, mem_rows + tail_rows])


def test_t0_generation_never_compresses_and_is_causal():
    S, D = 9, 4
    q, k, v = (_rand((1, 1, S, D), sd) for sd in (95, 96, 97))
    Og, kc, vc, length = oracle.replay_generation(q, k, v, 0, 4, 0, tail_read=S)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v), is_causal=True).numpy()
    assert length == S and np.allclose(Og, ref, atol=1e-13)


# ------------------------------------------------ inference layout (no <r> zone)

NOREP = oracle.FLAG_NO_REP_ZONE


def test_inference_layout_mask_is_fig5_mask_without_repetition_rows_and_columns(golden_dir):
    """Section 3.1 generates over [reading | memory] chunks only; the <r> rows exist for the training
    loss (Section 4.2).  Deleting the repetition rows and columns from the hand-typed Fig. 5 mask must
    give the inference-layout mask."""
    full = _load_mask(os.path.join(golden_dir, "fig5_mask_t2_c2_n3.txt"))
    keep = [i for i in range(30) if i % 10 < 6]
    want = full[np.ix_(keep, keep)]
    got = oracle.dense_mask(3, 2, 2, 0, NOREP)
    assert got.shape == (18, 18) and np.array_equal(got, want)
    ent = np.array([[oracle.allowed(i, j, 3, 2, 2, NOREP) for j in range(18)] for i in range(18)])
    assert np.array_equal(ent, want)
    assert np.array_equal(oracle.mask_rows(list(range(18)), 3, 2, 2, 0, NOREP), want)
    full_p = _load_mask(os.path.join(golden_dir, "fig5_mask_t2_c2_n3_prior_mem.txt"))
    assert np.array_equal(oracle.dense_mask(3, 2, 2, 0, NOREP | 1), full_p[np.ix_(keep, keep)])


@pytest.mark.parametrize("n,c,t,tail", [(2, 4, 4, 0), (3, 2, 2, 3), (2, 3, 5, 1), (4, 1, 3, 0)])
@pytest.mark.parametrize("prior", [0, 1])
def test_inference_layout_equals_training_layout_on_shared_rows_and_replays(n, c, t, tail, prior):
    """Reading and memory rows never see a repetition key, so their outputs over the inference layout
    equal their outputs over the training layout built from the same rows; and incremental generation
    (decode per token, compress per chunk) reproduces every row of the one-shot inference-layout pass."""
    flags = NOREP | prior
    S2 = oracle.seq_len(n, c, t, tail, flags)
    assert S2 == n * t * (c + 1) + tail
    D = 8
    q2, k2, v2 = (_rand((1, 2, S2, D), sd) for sd in (190, 191, 192))
    O2, lse2 = oracle.masked_attn_fwd(q2, k2, v2, n, c, t, tail, flags)
    # embed into the training layout: repetition rows get unrelated values
    S = oracle.seq_len(n, c, t, tail)
    zone = oracle.layout_index(n, c, t, tail)[1]
    live = np.nonzero(zone != oracle.ZONE_REP)[0]
    q, k, v = (_rand((1, 2, S, D), sd) for sd in (193, 194, 195))
    q[:, :, live], k[:, :, live], v[:, :, live] = q2, k2, v2
    O, lse = oracle.masked_attn_fwd(q, k, v, n, c, t, tail, prior)
    assert np.allclose(O[:, :, live], O2, atol=1e-13) and np.allclose(lse[:, :, live], lse2, atol=1e-13)
    Og, kc, vc, length = oracle.replay_generation(q2, k2, v2, n, c, t, tail, flags)
    assert not np.isnan(Og).any()
    assert np.allclose(Og, O2, atol=1e-13)
    ch2, zn2, of2, src2, pos2 = oracle.layout_index(n, c, t, tail, flags)
    assert set(zn2.tolist()) <= {oracle.ZONE_READ, oracle.ZONE_MEM}
    mem_rows = np.nonzero(zn2 == oracle.ZONE_MEM)[0].tolist()
    tail_rows = list(range(n * t * (c + 1), S2))
    assert length == len(mem_rows) + tail
    assert np.array_equal(kc[:, :, :length], k2[:, :, mem_rows + tail_rows])
    # positions of the shared rows agree with the training layout (Eq. 14)
    assert pos2.tolist() == oracle.layout_index(n, c, t, tail)[4][live].tolist()


# ------------------------------------------- several tokens over an existing cache

def test_prefill_with_one_token_is_decode():
    B, H, L, D = 2, 3, 9, 8
    q, k, v = (_rand((B, H, 1, D), sd) for sd in (300, 301, 302))
    kc, vc = _rand((B, H, L + 3, D), 303), _rand((B, H, L + 3, D), 304)
    a = oracle.prefill_attn(q, k, v, kc, vc, L)
    b = oracle.decode_attn(q, k, v, kc, vc, L)
    assert np.allclose(a[0], b[0], atol=1e-14) and np.allclose(a[1], b[1], atol=1e-14)
    assert np.array_equal(a[2], b[2]) and np.array_equal(a[3], b[3])


@pytest.mark.parametrize("l", [1, 2, 7, 33])
def test_prefill_over_an_empty_cache_is_library_causal_sdpa(l):
    B, H, D = 2, 2, 16
    q, k, v = (_rand((B, H, l, D), sd) for sd in (310, 311, 312))
    kc = np.full((B, H, l + 2, D), 7.0); vc = np.full((B, H, l + 2, D), -7.0)      # stale contents must not matter
    o, lse, kc2, vc2 = oracle.prefill_attn(q, k, v, kc, vc, 0)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v), is_causal=True).numpy()
    assert np.allclose(o, ref, atol=1e-13)
    assert np.array_equal(kc2[:, :, :l], k) and np.array_equal(vc2[:, :, :l], v)
    assert np.array_equal(kc2[:, :, l:], kc[:, :, l:])


@pytest.mark.parametrize("l,kk", [(2, 5), (17, 3), (5, 40)])
def test_prefill_rows_are_the_last_rows_of_causal_sdpa_over_cache_plus_new(l, kk):
    """Listing mask tril(ones(l, l+k), diagonal=k): new token i sees the k cached entries and new tokens 0..i --
    exactly the last l rows of plain causal attention over the concatenation; written out with the library
    routine and an explicit boolean mask."""
    B, H, D = 1, 2, 8
    q, k, v = (_rand((B, H, l, D), sd) for sd in (320, 321, 322))
    kc, vc = _rand((B, H, kk + l + 1, D), 323), _rand((B, H, kk + l + 1, D), 324)
    o, lse, kc2, vc2 = oracle.prefill_attn(q, k, v, kc, vc, kk)
    K = np.concatenate([kc[:, :, :kk], k], axis=2)
    V = np.concatenate([vc[:, :, :kk], v], axis=2)
    mask = torch.tril(torch.ones(l, l + kk, dtype=torch.bool), diagonal=kk)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(K), torch.from_numpy(V), attn_mask=mask).numpy()
    assert np.allclose(o, ref, atol=1e-13)
    # row sums of the implied probabilities: lse is the log of the normaliser of exactly the allowed scores
    sc = np.einsum("bhid,bhjd->bhij", q, K) / math.sqrt(D)
    want_lse = np.log(np.where(mask.numpy(), np.exp(sc), 0.0).sum(-1))
    assert np.allclose(lse, want_lse, atol=1e-12)
    assert np.array_equal(kc2[:, :, :kk + l], K) and np.array_equal(vc2[:, :, :kk + l], V)


@pytest.mark.parametrize("c,t,pieces", [(4, 4, [56]), (4, 4, [5, 51]), (2, 2, [1, 2, 3, 4, 5]), (3, 5, [7, 7, 7, 7, 7, 3]),
                                        (4, 4, [16, 16, 16, 8]), (2, 8, [40, 1, 15])])
@pytest.mark.parametrize("prior", [0, 1])
def test_prompt_fed_in_pieces_equals_the_one_shot_inference_layout(c, t, pieces, prior):
    """Appendix A `add_token_ids`: however a prompt is cut into pieces (a piece that starts or ends in the middle
    of a chunk goes through `inference_input` with several tokens over a non-empty cache), every reading and
    memory row comes out as in the one-pass forward over the inference layout, and the cache ends up holding
    the memory zones in order followed by the tail."""
    flags = NOREP | prior
    tc = c * t
    n_tok = sum(pieces)
    n, tail = n_tok // tc, n_tok % tc
    S = oracle.seq_len(n, c, t, tail, flags)
    D = 8
    q, k, v = (_rand((1, 2, S, D), sd) for sd in (330, 331, 332))
    O, _ = oracle.masked_attn_fwd(q, k, v, n, c, t, tail, flags)
    Og, kc, vc, length = oracle.replay_prompt_pieces(q, k, v, pieces, c, t, flags)
    assert not np.isnan(Og).any()
    assert np.allclose(Og, O, atol=1e-13)
    zn = oracle.layout_index(n, c, t, tail, flags)[1]
    mem_rows = np.nonzero(zn == oracle.ZONE_MEM)[0].tolist()
    tail_rows = list(range(n * (tc + t), S))
    assert length == len(mem_rows) + tail
    assert np.array_equal(kc[:, :, :length], k[:, :, mem_rows + tail_rows])
    assert np.array_equal(vc[:, :, :length], v[:, :, mem_rows + tail_rows])
    # and one token per piece is the token-by-token replay
    Og1 = oracle.replay_generation(q, k, v, n, c, t, tail, flags)[0]
    assert np.allclose(Og1, O, atol=1e-13)


def test_planted_mistakes_in_prefill_are_caught(monkeypatch):
    """A shifted diagonal, a mask that forgets the cache, and an append at the wrong slot must each fail a pin."""
    good = lo.prefill_attn

    def shifted(q, k_new, v_new, kc, vc, cache_len, scale=None):       # token i does not see itself
        o, lse, a, b = good(q, k_new, v_new, kc, vc, cache_len, scale)
        l = np.asarray(q).shape[2]
        if l > 1 or cache_len > 0:
            o2 = good(q, k_new, v_new, kc, vc, max(cache_len - 1, 0), scale)[0] if cache_len > 0 else o * 0.5
            return o2, lse, a, b
        return o, lse, a, b

    def forgets_cache(q, k_new, v_new, kc, vc, cache_len, scale=None):  # causal among the new tokens only
        l = np.asarray(q).shape[2]
        o, lse, _, _ = good(q, k_new, v_new, np.zeros_like(np.asarray(kc)[:, :, :l + 1]), np.zeros_like(np.asarray(vc)[:, :, :l + 1]), 0, scale)
        _, _, a, b = good(q, k_new, v_new, kc, vc, cache_len, scale)
        return o, lse, a, b

    def wrong_slot(q, k_new, v_new, kc, vc, cache_len, scale=None):     # appended one slot too far
        o, lse, a, b = good(q, k_new, v_new, kc, vc, cache_len, scale)
        return o, lse, np.roll(a, 1, axis=2), b

    for bad in (shifted, forgets_cache, wrong_slot):
        monkeypatch.setattr(oracle, "prefill_attn", bad)
        monkeypatch.setattr(lo, "prefill_attn", bad)
        with pytest.raises(AssertionError):
            test_prefill_rows_are_the_last_rows_of_causal_sdpa_over_cache_plus_new(5, 40)
            test_prefill_with_one_token_is_decode()
    monkeypatch.setattr(oracle, "prefill_attn", good)
    monkeypatch.setattr(lo, "prefill_attn", good)


# ------------------------------------------ planted mistakes must be caught

def _run_core_pins(golden_dir):
    test_fig5_mask_matches_hand_typed_fixture(golden_dir)
    test_mask_popcount_closed_form(3, 2, 2, 0)
    test_zero_query_gives_mean_of_allowed_values(2, 4, 4, 0)
    test_all_ones_mask_equals_library_sdpa()
    test_softmax_attention_two_key_closed_form()
    test_invariant_a_t0_is_causal_attention(7, 8)
    test_invariant_c_incremental_generation_equals_one_shot(3, 2, 2, 3, 0)
    test_compress_is_unmasked_sdpa_and_cat_compaction(0)
    test_memory_position_ids_match_the_listing_range(4, 4)


def test_planted_mistakes_in_the_oracle_are_caught(monkeypatch, golden_dir):
    """Break the oracle (on the CPU) in plausible ways; the pins above must fail each time."""
    _run_core_pins(golden_dir)   # sanity: intact oracle passes

    def broken_chunk_mask_no_identity(c, t, flags=0):
        M = orig_chunk_mask(c, t, flags)
        tc = t * c
        M[tc + t:, tc + t:] = False            # dropped I block
        return M

    def broken_chunk_mask_mem_causal(c, t, flags=0):
        M = orig_chunk_mask(c, t, flags)
        tc = t * c
        M[tc:tc + t, tc:tc + t] = np.tril(np.ones((t, t), bool))   # memory zone made causal
        return M

    def broken_cross_transposed(c, t, flags=0):
        return orig_cross(c, t, flags).T       # transposed S block

    def broken_attention_no_scale(q, k, v, mask, scale=None):
        return orig_attn(q, k, v, mask, 1.0)

    def broken_attention_transposed_v(q, k, v, mask, scale=None):
        O, P, lse = orig_attn(q, k, v, mask, scale)
        return (P.T @ np.asarray(v, float) if P.shape[0] == P.shape[1] else O * 0), P, lse

    def broken_attention_mask_as_multiply(q, k, v, mask, scale=None):
        # literal reading of Eq. 6: blocked scores become 0 instead of being excluded
        q_, k_, v_ = (np.asarray(a, float) for a in (q, k, v))
        sc = (1.0 / np.sqrt(q_.shape[-1])) if scale is None else scale
        A = sc * (q_ @ k_.T) * mask
        E = np.exp(A - A.max(1, keepdims=True))
        P = E / E.sum(1, keepdims=True)
        return P @ v_, P, np.log(np.exp(A).sum(1))

    orig_chunk_mask, orig_cross, orig_attn = lo.chunk_mask, lo.cross_chunk_block, lo.masked_softmax_attention
    plants = [
        ("chunk_mask", broken_chunk_mask_no_identity),
        ("chunk_mask", broken_chunk_mask_mem_causal),
        ("cross_chunk_block", broken_cross_transposed),
        ("masked_softmax_attention", broken_attention_no_scale),
        ("masked_softmax_attention", broken_attention_transposed_v),
        ("masked_softmax_attention", broken_attention_mask_as_multiply),
    ]
    for name, fn in plants:
        with monkeypatch.context() as m:
            m.setattr(lo, name, fn)
            m.setattr(oracle, name, fn)
            with pytest.raises(AssertionError):
                _run_core_pins(golden_dir)

    # index-map and cache plants
    def broken_layout(n, c, t, tail_read=0, flags=0):
        ch, zn, of, src, pos = orig_layout(n, c, t, tail_read, flags)
        pos = pos.copy()
        pos[zn == 1] -= c - 1                  # memory ids start at the chunk start instead of +c-1
        return ch, zn, of, src, pos

    orig_layout = lo.layout_index
    with monkeypatch.context() as m:
        m.setattr(lo, "layout_index", broken_layout)
        m.setattr(oracle, "layout_index", broken_layout)
        with pytest.raises(AssertionError):
            test_memory_position_ids_match_the_listing_range(4, 4)

    def broken_compress(q_mem, k_mem, v_mem, k_cache, v_cache, mem_len, c, t, flags=0, scale=None):
        # attends to the FIRST tc cache entries instead of the last tc
        o, lse, nk, nv = orig_compress(q_mem, k_mem, v_mem, np.roll(k_cache, mem_len, axis=2),
                                       np.roll(v_cache, mem_len, axis=2), mem_len, c, t, flags, scale)
        return o, lse, nk, nv

    orig_compress = lo.compress_step
    with monkeypatch.context() as m:
        m.setattr(lo, "compress_step", broken_compress)
        m.setattr(oracle, "compress_step", broken_compress)
        with pytest.raises(AssertionError):
            test_compress_is_unmasked_sdpa_and_cat_compaction(0)


def test_ragged_decode_is_per_sequence_decode():
    """Equal lengths give the uniform function; a sequence's result does not depend on its neighbours'
    lengths or contents; entries at and beyond a sequence's own length (other than the appended slot)
    are neither read nor written."""
    B, H, D, cap = 3, 2, 8, 12
    kc, vc = _rand((B, H, cap, D), 70), _rand((B, H, cap, D), 71)
    q, kn, vn = _rand((B, H, 1, D), 72), _rand((B, H, 1, D), 73), _rand((B, H, 1, D), 74)
    o_u, l_u, k_u, v_u = oracle.decode_attn(q, kn, vn, kc, vc, 5)
    o_r, l_r, k_r, v_r = oracle.decode_attn_ragged(q, kn, vn, kc, vc, [5, 5, 5])
    assert np.array_equal(o_u, o_r) and np.array_equal(l_u, l_r) and np.array_equal(k_u, k_r) and np.array_equal(v_u, v_r)
    lens = [0, 7, 3]
    o_r, _, k_r, v_r = oracle.decode_attn_ragged(q, kn, vn, kc, vc, lens)
    kc2 = kc.copy(); kc2[0] += 100.0; kc2[2, :, 4:] = np.nan      # other sequences changed, own tail beyond len poisoned
    o_2, _, _, _ = oracle.decode_attn_ragged(q, kn, vn, kc2, vc, lens)
    assert np.array_equal(o_r[1], o_2[1]) and np.isfinite(o_2[2]).all()
    assert np.allclose(o_r[0, :, 0], vn[0, :, 0])                 # empty cache: the token sees only itself
    for b, n in enumerate(lens):
        assert np.array_equal(k_r[b, :, n], kn[b, :, 0]) and np.array_equal(v_r[b, :, n], vn[b, :, 0])
        keep = np.ones(cap, bool); keep[n] = False
        assert np.array_equal(k_r[b][:, keep], kc[b][:, keep])


def test_ragged_compress_is_per_sequence_compress():
    B, H, D, c, t, cap = 3, 2, 8, 2, 2, 20
    tc = c * t
    kc, vc = _rand((B, H, cap, D), 80), _rand((B, H, cap, D), 81)
    qm, km, vm = _rand((B, H, t, D), 82), _rand((B, H, t, D), 83), _rand((B, H, t, D), 84)
    o_u, l_u, k_u, v_u = oracle.compress_step(qm, km, vm, kc, vc, 6, c, t)
    o_r, l_r, k_r, v_r = oracle.compress_step_ragged(qm, km, vm, kc, vc, [6, 6, 6], c, t)
    assert np.array_equal(o_u, o_r) and np.array_equal(l_u, l_r)
    assert np.array_equal(k_r[:, :, :6 + t], k_u) and np.array_equal(v_r[:, :, :6 + t], v_u)
    lens = [0, -1, 10]
    o_r, _, k_r, v_r = oracle.compress_step_ragged(qm, km, vm, kc, vc, lens, c, t)
    assert np.isnan(o_r[1]).all() and np.array_equal(k_r[1], kc[1]) and np.array_equal(v_r[1], vc[1])
    for b in (0, 2):
        n = lens[b]
        ob, _, kb, _ = oracle.compress_step(qm[b:b + 1], km[b:b + 1], vm[b:b + 1], kc[b:b + 1], vc[b:b + 1], n, c, t)
        assert np.array_equal(o_r[b], ob[0]) and np.array_equal(k_r[b, :, :n + t], kb[0])
        assert np.array_equal(k_r[b, :, n + t:], kc[b, :, n + t:])        # nothing beyond the new length is touched


def test_paged_decode_is_contiguous_decode_through_the_block_table():
    """An identity block table reproduces the contiguous (ragged) decode; relabelling the pages (pool and table
    permuted together) changes nothing; pages no table entry points at are neither read nor written."""
    B, H, D, ps, max_pages = 3, 2, 8, 4, 3
    cap = ps * max_pages
    kc, vc = _rand((B, H, cap, D), 90), _rand((B, H, cap, D), 91)
    q, kn, vn = _rand((B, H, 1, D), 92), _rand((B, H, 1, D), 93), _rand((B, H, 1, D), 94)
    lens = [0, 11, 5]
    # pools whose page b*max_pages + p holds slots [p*ps, (p+1)*ps) of sequence b, plus two unused pages
    n_pages = B * max_pages + 2
    kp, vp = np.full((n_pages, H, ps, D), np.nan), np.full((n_pages, H, ps, D), np.nan)
    table = np.zeros((B, max_pages), np.int32)
    for b in range(B):
        for p_ in range(max_pages):
            table[b, p_] = b * max_pages + p_
            kp[table[b, p_]] = kc[b, :, p_ * ps:(p_ + 1) * ps]
            vp[table[b, p_]] = vc[b, :, p_ * ps:(p_ + 1) * ps]
    o_c, l_c, k_c, v_c = oracle.decode_attn_ragged(q, kn, vn, kc, vc, lens)
    o_p, l_p, kp2, vp2 = oracle.decode_attn_paged(q, kn, vn, kp, vp, table, lens)
    assert np.array_equal(o_c, o_p) and np.array_equal(l_c, l_p)
    for b, n in enumerate(lens):
        assert np.array_equal(kp2[table[b, n // ps], :, n % ps], kn[b, :, 0])
    assert np.isnan(kp2[-2:]).all() and np.isnan(vp2[-2:]).all()
    perm = np.random.default_rng(0).permutation(n_pages)          # new label of page i is perm[i]
    kq, vq = np.empty_like(kp), np.empty_like(vp)
    kq[perm], vq[perm] = kp, vp
    o_q, _, _, _ = oracle.decode_attn_paged(q, kn, vn, kq, vq, perm[table], lens)
    assert np.array_equal(o_q, o_p)


def test_paged_compress_is_ragged_compress_through_the_block_table():
    B, H, D, c, t, ps, max_pages = 3, 2, 8, 2, 2, 4, 5
    tc, cap = c * t, 4 * 5
    kc, vc = _rand((B, H, cap, D), 95), _rand((B, H, cap, D), 96)
    qm, km, vm = _rand((B, H, t, D), 97), _rand((B, H, t, D), 98), _rand((B, H, t, D), 99)
    lens = [3, -1, 14]                                   # slots [3, 5) and [14, 16) straddle no page / end a page
    n_pages = B * max_pages + 1
    kp, vp = np.full((n_pages, H, ps, D), np.nan), np.full((n_pages, H, ps, D), np.nan)
    table = np.random.default_rng(1).permutation(n_pages)[: B * max_pages].reshape(B, max_pages).astype(np.int32)
    for b in range(B):
        for p_ in range(max_pages):
            kp[table[b, p_]] = kc[b, :, p_ * ps:(p_ + 1) * ps]
            vp[table[b, p_]] = vc[b, :, p_ * ps:(p_ + 1) * ps]
    o_r, l_r, k_r, v_r = oracle.compress_step_ragged(qm, km, vm, kc, vc, lens, c, t)
    o_p, l_p, kp2, vp2 = oracle.compress_step_paged(qm, km, vm, kp, vp, table, lens, c, t)
    assert np.array_equal(o_r[[0, 2]], o_p[[0, 2]]) and np.isnan(o_p[1]).all()
    back = oracle.paged_to_contiguous(kp2, table, cap)
    for b, n in enumerate(lens):
        if n >= 0:
            assert np.array_equal(back[b, :, :n + t], k_r[b, :, :n + t])
    unused = np.setdiff1d(np.arange(n_pages), table.ravel())
    assert np.isnan(kp2[unused]).all()
    assert np.array_equal(kp2[table[1]], kp[table[1]])   # the idle sequence's pages are untouched
