"""Plain fp64 NumPy oracle for LoMA's attention hot path.

TEST INFRASTRUCTURE ONLY.  Nothing here is tuned, tiled, fused or reordered:
each function takes the paper's definition and writes it out, so a reader can
hold it against the paper by eye.  Floating point is float64 throughout
(inputs are upcast exactly from whatever precision they were stored in).

Notation (Section 3.1, Section 4.3):
    c   compression ratio
    t   memory-zone length (number of <m> tokens per chunk)
    tc  = t*c, reading-zone length = repetition-zone length
    s   = t*(2c+1) = 2*tc + t, length of one training chunk
    n   number of complete chunks
    tail_read  extra reading rows after the last complete chunk (the
        uncompressed tail of an unfinished chunk; with t == 0 the whole
        sequence is such a tail, i.e. ordinary causal attention)

Readings of the paper taken here (each is listed with its evidence in the
repository's design notes):
  * a mask value of 0 removes the key from the softmax (weight exactly 0),
    following the Fig. 5 caption rather than the literal product of Eq. 6;
  * the softmax scale that Section 4.4 drops "without loss of generality" is an
    explicit argument, default 1/sqrt(D);
  * memory rows see only their own reading zone and their own memory zone
    (Eq. 3 has zero memory rows; criterion 2 of Section 4.3; Appendix A slices
    the last read_len cache entries).  FLAG_MEM_SEES_PRIOR_MEM switches on the
    other reading, in which memory rows also see every earlier memory zone;
  * memory position ids of chunk y are y*tc + (j+1)*c - 1 (Eq. 14 read together
    with the generator listing, whose chunk start is y*tc);
  * repetition-zone position ids repeat those of the reading token each row
    reproduces.  The paper is silent on this one: PARITY UNPINNED for that
    single output column of layout_index (pos_id on repetition rows).
"""

from __future__ import annotations

import numpy as np

FLAG_MEM_SEES_PRIOR_MEM = 1
# Inference layout: chunks are [tc reading | t memory] with no repetition zone, i.e. the sequence the
# generator of Section 3.1 / Appendix A actually feeds the model (the <r> rows exist only for the
# training loss, Section 4.2).  The mask is Eq. 2 with the repetition rows and columns deleted.
FLAG_NO_REP_ZONE = 2

ZONE_READ = 0
ZONE_MEM = 1
ZONE_REP = 2


# --------------------------------------------------------------------------
# Layout (Section 4.1) and index maps (Eq. 14, Appendix A)
# --------------------------------------------------------------------------

def chunk_len(c: int, t: int, flags: int = 0) -> int:
    """s = t(2c+1): reading zone + memory zone + repetition zone (Section 4.3);
    t(c+1) in the inference layout, which has no repetition zone."""
    if flags & FLAG_NO_REP_ZONE:
        return t * (c + 1)
    return t * (2 * c + 1)


def seq_len(n_chunks: int, c: int, t: int, tail_read: int = 0, flags: int = 0) -> int:
    """Length of the laid-out sequence: n complete chunks plus a reading tail."""
    return n_chunks * chunk_len(c, t, flags) + tail_read


def decompose(i: int, n_chunks: int, c: int, t: int, flags: int = 0):
    """Row index -> (chunk y, zone z, offset o inside the zone) (Section 4.1).

    Rows past the last complete chunk form the reading zone of chunk n_chunks.
    """
    tc = t * c
    s = chunk_len(c, t, flags)
    if s == 0 or i >= n_chunks * s:
        return n_chunks, ZONE_READ, i - n_chunks * s
    y, r = divmod(i, s)
    if r < tc:
        return y, ZONE_READ, r
    if r < tc + t:
        return y, ZONE_MEM, r - tc
    return y, ZONE_REP, r - tc - t


def layout_index(n_chunks: int, c: int, t: int, tail_read: int = 0, flags: int = 0):
    """Integer maps over the rows of the laid-out sequence.

    Returns int32 arrays (chunk, zone, offset, src_token, pos_id), each [S].
      src_token: index into the original token sequence that the row carries
                 (reading rows) or must reproduce (repetition rows); -1 for <m>
                 rows (Section 4.1, Eq. 13).
      pos_id:    reading rows keep their original position y*tc+o; memory row j
                 of chunk y gets y*tc+(j+1)c-1 (Eq. 14); repetition rows repeat
                 the reading position (paper silent, unpinned).
    """
    tc = t * c
    S = seq_len(n_chunks, c, t, tail_read, flags)
    chunk = np.zeros(S, np.int32)
    zone = np.zeros(S, np.int32)
    offset = np.zeros(S, np.int32)
    src = np.zeros(S, np.int32)
    pos = np.zeros(S, np.int32)
    for i in range(S):
        y, z, o = decompose(i, n_chunks, c, t, flags)
        chunk[i], zone[i], offset[i] = y, z, o
        if z == ZONE_MEM:
            src[i] = -1
            pos[i] = y * tc + (o + 1) * c - 1
        else:
            src[i] = y * tc + o
            pos[i] = y * tc + o
    return chunk, zone, offset, src, pos


def generation_index(n_tokens: int, c: int, t: int):
    """Per generated token g: where its KV lands and what the cache looks like.

    Section 3.1 steps 1-3 with the Appendix A bookkeeping: the cache holds
    compressed_chunks*t memory entries followed by the uncompressed tail, and a
    compress pass fires as soon as the tail reaches tc entries.

    Returns int32 arrays [n_tokens]:
      slot            cache index the token's K/V is appended at
                      (= entries in the cache before the token)
      pos_id          the generator's `cursor` value for the token (= g)
      compress_after  1 if a compress pass runs right after this token
    With t == 0 nothing is ever compressed (`while self.mem_len > 0`).
    """
    tc = t * c
    slot = np.zeros(n_tokens, np.int32)
    pos = np.zeros(n_tokens, np.int32)
    comp = np.zeros(n_tokens, np.int32)
    compressed_chunks = 0
    tail = 0
    for g in range(n_tokens):
        slot[g] = compressed_chunks * t + tail
        pos[g] = g
        tail += 1
        if t > 0 and tail == tc:
            comp[g] = 1
            compressed_chunks += 1
            tail = 0
    return slot, pos, comp


# --------------------------------------------------------------------------
# Mask (Eq. 1-3)
# --------------------------------------------------------------------------

def chunk_mask(c: int, t: int, flags: int = 0) -> np.ndarray:
    """Eq. 1: the s x s mask of one training chunk, as a boolean array.

        [ L  0  0 ]   reading rows: causal inside the reading zone
        [ 1  1  0 ]   memory rows: whole reading zone + whole memory zone
        [ 0  1  I ]   repetition rows: whole memory zone + the row itself
    """
    tc = t * c
    L = np.tril(np.ones((tc, tc), bool))
    I = np.eye(tc, dtype=bool)
    Z = lambda a, b: np.zeros((a, b), bool)
    O = lambda a, b: np.ones((a, b), bool)
    M = np.block([
        [L,         Z(tc, t), Z(tc, tc)],
        [O(t, tc),  O(t, t),  Z(t, tc)],
        [Z(tc, tc), O(tc, t), I],
    ])
    if flags & FLAG_NO_REP_ZONE:      # inference layout: the third block row and column do not exist
        M = M[:tc + t, :tc + t]
    return M


def cross_chunk_block(c: int, t: int, flags: int = 0) -> np.ndarray:
    """Eq. 3: the s x s block linking a chunk (rows) to an EARLIER chunk (cols).

    Only reading rows x memory columns are 1.  Under FLAG_MEM_SEES_PRIOR_MEM the
    memory rows x memory columns block is 1 as well.
    """
    tc = t * c
    s = chunk_len(c, t)
    S = np.zeros((s, s), bool)
    S[0:tc, tc:tc + t] = True
    if flags & FLAG_MEM_SEES_PRIOR_MEM:
        S[tc:tc + t, tc:tc + t] = True
    if flags & FLAG_NO_REP_ZONE:
        S = S[:tc + t, :tc + t]
    return S


def dense_mask(n_chunks: int, c: int, t: int, tail_read: int = 0, flags: int = 0) -> np.ndarray:
    """Eq. 2: the whole-sample mask, block lower triangular in chunks.

    Diagonal blocks are Eq. 1, blocks below the diagonal are Eq. 3, blocks above
    are zero.  A reading tail (an unfinished chunk) contributes the leading
    tail_read rows/cols of one more chunk row: reading rows of Eq. 3 towards
    every earlier chunk and the leading corner of L on the diagonal.
    """
    s = chunk_len(c, t, flags)
    S = seq_len(n_chunks, c, t, tail_read, flags)
    M = np.zeros((S, S), bool)
    if n_chunks > 0:
        Mc = chunk_mask(c, t, flags)
        Sc = cross_chunk_block(c, t, flags)
        for y in range(n_chunks):
            for x in range(y):
                M[y * s:(y + 1) * s, x * s:(x + 1) * s] = Sc
            M[y * s:(y + 1) * s, y * s:(y + 1) * s] = Mc
        if tail_read:
            for x in range(n_chunks):
                M[n_chunks * s:, x * s:(x + 1) * s] = Sc[:tail_read, :]
    if tail_read:
        M[n_chunks * s:, n_chunks * s:] = np.tril(np.ones((tail_read, tail_read), bool))
    return M


def allowed(i: int, j: int, n_chunks: int, c: int, t: int, flags: int = 0) -> bool:
    """May row i attend to column j?  Eq. 1-3 read entry by entry."""
    yi, zi, oi = decompose(i, n_chunks, c, t, flags)
    yj, zj, oj = decompose(j, n_chunks, c, t, flags)
    if yj > yi:
        return False                       # Eq. 2: zero above the block diagonal
    if yj == yi:                           # Eq. 1
        if zi == ZONE_READ:
            return zj == ZONE_READ and oj <= oi
        if zi == ZONE_MEM:
            return zj in (ZONE_READ, ZONE_MEM)
        return zj == ZONE_MEM or j == i
    # yj < yi: Eq. 3
    if zi == ZONE_READ and zj == ZONE_MEM:
        return True
    if (flags & FLAG_MEM_SEES_PRIOR_MEM) and zi == ZONE_MEM and zj == ZONE_MEM:
        return True
    return False


def mask_rows(rows, n_chunks: int, c: int, t: int, tail_read: int = 0, flags: int = 0) -> np.ndarray:
    """Selected rows of the Eq. 2 mask, built from the entry-wise rule.

    For sequences whose full S x S mask does not fit in memory.  Returns a
    boolean [len(rows), S].
    """
    S = seq_len(n_chunks, c, t, tail_read, flags)
    ch, zn, of, _, _ = layout_index(n_chunks, c, t, tail_read, flags)
    cols = np.arange(S)
    out = np.zeros((len(rows), S), bool)
    for r, i in enumerate(rows):
        yi, zi, oi = int(ch[i]), int(zn[i]), int(of[i])
        same = ch == yi
        earlier = ch < yi
        if zi == ZONE_READ:
            row = (same & (zn == ZONE_READ) & (of <= oi)) | (earlier & (zn == ZONE_MEM))
        elif zi == ZONE_MEM:
            row = same & ((zn == ZONE_READ) | (zn == ZONE_MEM))
            if flags & FLAG_MEM_SEES_PRIOR_MEM:
                row = row | (earlier & (zn == ZONE_MEM))
        else:
            row = (same & (zn == ZONE_MEM)) | (cols == i)
        out[r] = row
    return out


# --------------------------------------------------------------------------
# Attention (Eq. 5-7)
# --------------------------------------------------------------------------

def _f64(x) -> np.ndarray:
    return np.asarray(x, dtype=np.float64)


def masked_softmax_attention(q, k, v, mask, scale=None):
    """O = Softmax(A) V with A = scale * Q K^T restricted to mask (Eq. 5-7).

    q [R, D], k [C, D], v [C, Dv], mask boolean [R, C] (True = attend).
    Masked keys get weight exactly 0.  Every row must have at least one True.
    Returns (O [R, Dv], P [R, C], lse [R]) in float64; lse is the natural-log
    normaliser log(sum_j exp(A_ij)) over the allowed keys.
    """
    q, k, v = _f64(q), _f64(k), _f64(v)
    if scale is None:
        scale = 1.0 / np.sqrt(q.shape[-1])
    A = scale * (q @ k.T)
    A = np.where(mask, A, -np.inf)
    m = A.max(axis=1, keepdims=True)
    E = np.exp(A - m)
    l = E.sum(axis=1, keepdims=True)
    P = E / l
    O = P @ v
    lse = (m + np.log(l))[:, 0]
    return O, P, lse


def masked_attn_fwd(q, k, v, n_chunks, c, t, tail_read=0, flags=0, scale=None,
                    rows=None, return_p=False):
    """Zone-masked attention over the laid-out sequence.

    q, k, v: [B, H, S, D] with S = n_chunks*s + tail_read.
    rows: optional list of row indices; if given only those rows are computed
          (against all S keys) and the outputs have len(rows) in place of S.
    Returns (O [B,H,R,D], lse [B,H,R]) and, with return_p, also P [B,H,R,S].
    """
    q, k, v = _f64(q), _f64(k), _f64(v)
    B, H, S, D = q.shape
    assert S == seq_len(n_chunks, c, t, tail_read, flags)
    if rows is None:
        rows = np.arange(S)
        M = dense_mask(n_chunks, c, t, tail_read, flags)
    else:
        rows = np.asarray(rows)
        M = mask_rows(rows, n_chunks, c, t, tail_read, flags)
    R = len(rows)
    O = np.zeros((B, H, R, v.shape[-1]))
    LSE = np.zeros((B, H, R))
    P = np.zeros((B, H, R, S)) if return_p else None
    for b in range(B):
        for h in range(H):
            o, p, lse = masked_softmax_attention(q[b, h][rows], k[b, h], v[b, h], M, scale)
            O[b, h], LSE[b, h] = o, lse
            if return_p:
                P[b, h] = p
    if return_p:
        return O, LSE, P
    return O, LSE


# --------------------------------------------------------------------------
# Backward of the masked attention (Section 4.4: gradient propagation, Eq. 10)
# --------------------------------------------------------------------------

def masked_softmax_attention_bwd(q, k, v, d_o, mask, scale=None):
    """Gradients of O = Softmax(A) V (Eq. 7), A = scale * Q K^T on the mask.

    Given dO = dLoss/dO this is the chain rule written out term by term:
      * O is linear in V:                      dV = P^T dO
      * O is linear in P:                      dP = dO V^T
      * row i of P is a softmax of row i of A (blocked entries have P = 0 and
        take no part), whose Jacobian is diag(P_i) - P_i P_i^T:
                                               dA_ij = P_ij (dP_ij - sum_k P_ik dP_ik)
      * A = scale * Q K^T:                     dQ = scale * dA K,  dK = scale * dA^T Q
    Section 4.4 follows exactly these paths when it argues (Eq. 10) that the
    repetition loss reaches k_m and v_m; here nothing is dropped.

    q [R, D], k [C, D], v [C, Dv], d_o [R, Dv], mask boolean [R, C].
    Returns (dQ [R, D], dK [C, D], dV [C, Dv]) in float64.
    """
    q, k, v, d_o = _f64(q), _f64(k), _f64(v), _f64(d_o)
    if scale is None:
        scale = 1.0 / np.sqrt(q.shape[-1])
    _, P, _ = masked_softmax_attention(q, k, v, mask, scale)
    dV = P.T @ d_o
    dP = d_o @ v.T
    row_dot = (P * dP).sum(axis=1, keepdims=True)
    dA = P * (dP - row_dot)
    dQ = scale * (dA @ k)
    dK = scale * (dA.T @ q)
    return dQ, dK, dV


def masked_attn_bwd(q, k, v, d_o, n_chunks, c, t, tail_read=0, flags=0, scale=None):
    """Gradients of masked_attn_fwd with respect to q, k and v, all rows.

    q, k, v, d_o: [B, H, S, D].  Returns (dQ, dK, dV), each [B, H, S, D] float64.
    """
    q, k, v, d_o = _f64(q), _f64(k), _f64(v), _f64(d_o)
    B, H, S, D = q.shape
    assert S == seq_len(n_chunks, c, t, tail_read, flags)
    M = dense_mask(n_chunks, c, t, tail_read, flags)
    dQ, dK, dV = np.zeros_like(q), np.zeros_like(k), np.zeros_like(v)
    for b in range(B):
        for h in range(H):
            dQ[b, h], dK[b, h], dV[b, h] = masked_softmax_attention_bwd(q[b, h], k[b, h], v[b, h], d_o[b, h], M, scale)
    return dQ, dK, dV


def masked_attn_bwd_dq_rows(q, k, v, d_o, rows, n_chunks, c, t, tail_read=0, flags=0, scale=None):
    """dQ of the sampled rows only: a row's dQ depends on that row of the mask and of dO alone.
    Returns [B, H, len(rows), D]."""
    q, k, v, d_o = _f64(q), _f64(k), _f64(v), _f64(d_o)
    rows = np.asarray(rows)
    B, H, S, D = q.shape
    M = mask_rows(rows, n_chunks, c, t, tail_read, flags)
    out = np.zeros((B, H, len(rows), D))
    for b in range(B):
        for h in range(H):
            out[b, h] = masked_softmax_attention_bwd(q[b, h][rows], k[b, h], v[b, h], d_o[b, h][rows], M, scale)[0]
    return out


def masked_attn_bwd_dkv_cols(q, k, v, d_o, cols, n_chunks, c, t, tail_read=0, flags=0, scale=None, block=2048):
    """dK and dV of the sampled keys only.  A key's gradients sum over the rows that see it, and each
    such row needs its whole softmax, so: find the rows whose mask row allows one of `cols`
    (block by block, the mask is never held whole), run those rows in full, keep the sampled columns.
    Returns (dK [B, H, len(cols), D], dV [B, H, len(cols), D])."""
    q, k, v, d_o = _f64(q), _f64(k), _f64(v), _f64(d_o)
    cols = np.asarray(cols)
    B, H, S, D = q.shape
    need = []
    for lo in range(0, S, block):
        r = np.arange(lo, min(S, lo + block))
        hit = mask_rows(r, n_chunks, c, t, tail_read, flags)[:, cols].any(axis=1)
        need.append(r[hit])
    rows = np.concatenate(need)
    M = mask_rows(rows, n_chunks, c, t, tail_read, flags)
    dK = np.zeros((B, H, len(cols), D))
    dV = np.zeros((B, H, len(cols), D))
    sc = (1.0 / np.sqrt(D)) if scale is None else scale
    for b in range(B):
        for h in range(H):
            _, P, _ = masked_softmax_attention(q[b, h][rows], k[b, h], v[b, h], M, sc)
            g = d_o[b, h][rows]
            dP = g @ v[b, h].T
            dA = P * (dP - (P * dP).sum(axis=1, keepdims=True))
            dK[b, h] = sc * (dA[:, cols].T @ q[b, h][rows])
            dV[b, h] = P[:, cols].T @ g
    return dK, dV


# --------------------------------------------------------------------------
# Rotary embedding at LoMA's position ids (Section 4.5; the rotation is Llama-2's)
# --------------------------------------------------------------------------

def position_ids(n_chunks, c, t, tail_read=0, flags=0, position_type="intermittent"):
    """Position id of every row.  'intermittent' is Eq. 14 (layout_index's pos_id); 'contiguous' is the
    generator's other setting (Appendix A, compress_last_chunk): memory row j of chunk y gets
    mem_cursor + j with mem_cursor = y*t, everything else unchanged."""
    chunk, zone, offset, _, pos = layout_index(n_chunks, c, t, tail_read, flags)
    if position_type == "intermittent":
        return pos.astype(np.int64)
    assert position_type == "contiguous"
    pos = pos.astype(np.int64).copy()
    mem = zone == ZONE_MEM
    pos[mem] = chunk[mem].astype(np.int64) * t + offset[mem]
    return pos


def rope_rotate(x, pos, theta_base=10000.0):
    """Rotary position embedding as Llama-2 applies it (the model the paper fine-tunes; the paper only
    supplies the ids).  x [..., S, D], pos [S].  Feature d of the first half is paired with feature
    d + D/2; the pair is rotated by the angle pos * theta_base**(-2d/D)."""
    x = _f64(x)
    D = x.shape[-1]
    half = D // 2
    theta = theta_base ** (-2.0 * np.arange(half) / D)
    ang = np.asarray(pos, dtype=np.float64)[:, None] * theta[None, :]      # [S, half]
    cs, sn = np.cos(ang), np.sin(ang)
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * cs - b * sn, b * cs + a * sn], axis=-1)


def rope_apply(q, k, n_chunks, c, t, tail_read=0, flags=0, theta_base=10000.0, position_type="intermittent"):
    """q and k [B, H, S, D] rotated at the layout's position ids.  Returns (q', k') in float64."""
    pos = position_ids(n_chunks, c, t, tail_read, flags, position_type)
    return rope_rotate(q, pos, theta_base), rope_rotate(k, pos, theta_base)


# --------------------------------------------------------------------------
# Generation (Section 3.1, Appendix A)
# --------------------------------------------------------------------------

def decode_attn(q, k_new, v_new, k_cache, v_cache, cache_len, scale=None):
    """One decode step: a single new token over the whole cache plus itself.

    Appendix A `inference_input` with one input token: the mask row is all ones
    over the cache_len cached entries and the token's own column
    (tril(..., diagonal=cache_len)), and the token's K/V is appended.

    q, k_new, v_new: [B, H, 1, D]; k_cache, v_cache: [B, H, cap, D] of which the
    first cache_len entries are valid.
    Returns (o [B,H,1,D], lse [B,H,1], k_cache', v_cache') where the primed
    caches are copies with entry cache_len filled in.
    """
    q = _f64(q)
    B, H, _, D = q.shape
    kc = np.array(k_cache, copy=True)
    vc = np.array(v_cache, copy=True)
    kc[:, :, cache_len, :] = np.asarray(k_new)[:, :, 0, :]
    vc[:, :, cache_len, :] = np.asarray(v_new)[:, :, 0, :]
    o = np.zeros((B, H, 1, D))
    lse = np.zeros((B, H, 1))
    ones = np.ones((1, cache_len + 1), bool)
    for b in range(B):
        for h in range(H):
            keys = kc[b, h, :cache_len + 1]
            vals = vc[b, h, :cache_len + 1]
            o[b, h], _, lse[b, h] = masked_softmax_attention(q[b, h], keys, vals, ones, scale)
    return o, lse, kc, vc


def prefill_attn(q, k_new, v_new, k_cache, v_cache, cache_len, scale=None):
    """Several new tokens at once over an existing cache (Appendix A, `inference_input`).

    The l new tokens see every one of the cache_len cached entries and, among
    themselves, are causal: the mask is tril(ones(l, l + cache_len), diagonal=cache_len),
    row i allowing columns 0 .. cache_len + i.  Their K/V are appended to the cache.

    q, k_new, v_new: [B, H, l, D]; k_cache, v_cache: [B, H, cap, D] with the first
    cache_len entries valid.  Returns (o [B,H,l,D], lse [B,H,l], k_cache', v_cache')
    where the primed caches are copies with entries cache_len .. cache_len+l-1 filled in.
    """
    q = _f64(q)
    B, H, l, D = q.shape
    kc = np.array(k_cache, copy=True)
    vc = np.array(v_cache, copy=True)
    kc[:, :, cache_len:cache_len + l, :] = np.asarray(k_new)
    vc[:, :, cache_len:cache_len + l, :] = np.asarray(v_new)
    mask = np.tril(np.ones((l, l + cache_len), bool), k=cache_len)
    o = np.zeros((B, H, l, D))
    lse = np.zeros((B, H, l))
    for b in range(B):
        for h in range(H):
            o[b, h], _, lse[b, h] = masked_softmax_attention(q[b, h], kc[b, h, :cache_len + l], vc[b, h, :cache_len + l],
                                                            mask, scale)
    return o, lse, kc, vc


def replay_prompt_pieces(q, k, v, pieces, c, t, flags=0, scale=None):
    """Feed a prompt to the generation path in arbitrary pieces, the way Appendix A's
    `add_token_ids` does: tokens are buffered; whenever the uncompressed tail can be filled
    up to tc entries, exactly that many tokens go through `inference_input` (one
    prefill_attn call) and the chunk is compressed; what is left at the end of a piece goes
    through `inference_input` as it is.

    q, k, v: [B, H, S, D] in the inference layout (chunks of [tc reading | t memory], no
    repetition zones, then a reading tail), so that row numbers of the one-shot forward
    with FLAG_NO_REP_ZONE apply.  pieces: lengths of the token pieces; their sum is the
    number of reading rows.  Returns (O [B,H,S,D], k_cache, v_cache, length).
    """
    q, k, v = np.asarray(q), np.asarray(k), np.asarray(v)
    B, H, S, D = q.shape
    tc = t * c
    s = tc + t
    n_tokens = int(sum(pieces))
    n_chunks, tail = (n_tokens // tc, n_tokens % tc) if tc > 0 else (0, n_tokens)
    assert S == n_chunks * s + tail
    row_of_token = lambda g: (g // tc) * s + g % tc if tc > 0 else g
    cap = n_chunks * t + max(tc, tail) + 1
    kc = np.zeros((B, H, cap, D), dtype=k.dtype)
    vc = np.zeros((B, H, cap, D), dtype=v.dtype)
    O = np.full((B, H, S, D), np.nan)
    length, done, chunks = 0, 0, 0          # cache entries, tokens processed, chunks compressed
    fed = 0
    for piece in pieces:
        fed += int(piece)
        while done < fed:
            uncompressed = length - chunks * t
            take = fed - done
            fills = tc > 0 and uncompressed + take >= tc
            if fills:
                take = tc - uncompressed
            rows = [row_of_token(g) for g in range(done, done + take)]
            out, _, kc, vc = prefill_attn(q[:, :, rows], k[:, :, rows], v[:, :, rows], kc, vc, length, scale)
            O[:, :, rows] = out
            length += take
            done += take
            if fills:
                m0 = chunks * s + tc
                mem_len = chunks * t
                out, _, nk, nv = compress_step(q[:, :, m0:m0 + t], k[:, :, m0:m0 + t], v[:, :, m0:m0 + t],
                                               kc, vc, mem_len, c, t, flags & FLAG_MEM_SEES_PRIOR_MEM, scale)
                O[:, :, m0:m0 + t] = out
                chunks += 1
                length = mem_len + t
                kc[:, :, :length] = nk
                vc[:, :, :length] = nv
    return O, kc, vc, length


def decode_attn_ragged(q, k_new, v_new, k_cache, v_cache, cache_lens, scale=None):
    """decode_attn for a batch whose sequences have their own cache lengths: sequence b is an
    independent run of the generator (Appendix A handles one sequence at a time), so this is
    decode_attn applied to each b with cache_lens[b].  Same return values as decode_attn."""
    q = _f64(q)
    B, H, _, D = q.shape
    o = np.zeros((B, H, 1, D))
    lse = np.zeros((B, H, 1))
    kc = np.array(k_cache, copy=True)
    vc = np.array(v_cache, copy=True)
    for b in range(B):
        ob, lb, kb, vb = decode_attn(q[b:b + 1], np.asarray(k_new)[b:b + 1], np.asarray(v_new)[b:b + 1],
                                     np.asarray(k_cache)[b:b + 1], np.asarray(v_cache)[b:b + 1], int(cache_lens[b]), scale)
        o[b], lse[b], kc[b], vc[b] = ob[0], lb[0], kb[0], vb[0]
    return o, lse, kc, vc


def paged_to_contiguous(pool, block_table, cap):
    """The logical cache [B, H, cap, D] that a pool [n_pages, H, page_size, D] and a block table [B, max_pages]
    describe: slot j of sequence b is row j % page_size of page block_table[b][j // page_size]."""
    pool = np.asarray(pool)
    n_pages, H, ps, D = pool.shape
    B = len(block_table)
    out = np.zeros((B, H, cap, D), dtype=pool.dtype)
    for b in range(B):
        for j in range(cap):
            out[b, :, j] = pool[int(block_table[b][j // ps]), :, j % ps]
    return out


def decode_attn_paged(q, k_new, v_new, k_pool, v_pool, block_table, cache_lens, scale=None):
    """decode_attn_ragged over a paged cache: read every sequence's logical cache out of the pools, run the
    per-sequence decode, and write the appended entry back into its page.  Returns (o, lse, k_pool', v_pool')."""
    k_pool, v_pool = np.asarray(k_pool), np.asarray(v_pool)
    ps = k_pool.shape[2]
    cap = max(int(n) for n in cache_lens) + 1
    kc = paged_to_contiguous(k_pool, block_table, cap)
    vc = paged_to_contiguous(v_pool, block_table, cap)
    o, lse, kc2, vc2 = decode_attn_ragged(q, k_new, v_new, kc, vc, cache_lens, scale)
    kp, vp = k_pool.copy(), v_pool.copy()
    for b, n in enumerate(cache_lens):
        n = int(n)
        page = int(block_table[b][n // ps])
        kp[page, :, n % ps] = kc2[b, :, n]
        vp[page, :, n % ps] = vc2[b, :, n]
    return o, lse, kp, vp


def compress_step(q_mem, k_mem, v_mem, k_cache, v_cache, mem_len, c, t, flags=0, scale=None):
    """Compress pass + compaction (Section 3.1 steps 2-3; Appendix A
    `compress_last_chunk`).

    Before: the cache holds mem_len memory entries followed by exactly tc tail
    entries (the listing asserts this).  The t <m> queries attend, with an
    all-ones mask, to the tc tail entries and to their own t keys.  Under
    FLAG_MEM_SEES_PRIOR_MEM the mem_len earlier memory entries are visible too.
    After: cache' = concatenate(cache[:mem_len], k_mem), valid length mem_len+t.

    q_mem, k_mem, v_mem: [B, H, t, D]; caches [B, H, cap, D].
    Returns (o_mem [B,H,t,D], lse [B,H,t], k_cache' [B,H,mem_len+t,D], v_cache').
    """
    tc = t * c
    q_mem = _f64(q_mem)
    k_cache = np.asarray(k_cache)
    v_cache = np.asarray(v_cache)
    k_mem_a = np.asarray(k_mem)
    v_mem_a = np.asarray(v_mem)
    B, H, _, D = q_mem.shape
    lo = 0 if (flags & FLAG_MEM_SEES_PRIOR_MEM) else mem_len
    o = np.zeros((B, H, t, D))
    lse = np.zeros((B, H, t))
    for b in range(B):
        for h in range(H):
            keys = np.concatenate([_f64(k_cache[b, h, lo:mem_len + tc]), _f64(k_mem_a[b, h])], axis=0)
            vals = np.concatenate([_f64(v_cache[b, h, lo:mem_len + tc]), _f64(v_mem_a[b, h])], axis=0)
            ones = np.ones((t, keys.shape[0]), bool)
            o[b, h], _, lse[b, h] = masked_softmax_attention(q_mem[b, h], keys, vals, ones, scale)
    # Compaction by explicit copies into fresh arrays.
    new_k = np.empty((B, H, mem_len + t, D), dtype=k_cache.dtype)
    new_v = np.empty((B, H, mem_len + t, D), dtype=v_cache.dtype)
    for b in range(B):
        for h in range(H):
            for e in range(mem_len):
                new_k[b, h, e] = k_cache[b, h, e]
                new_v[b, h, e] = v_cache[b, h, e]
            for j in range(t):
                new_k[b, h, mem_len + j] = k_mem_a[b, h, j]
                new_v[b, h, mem_len + j] = v_mem_a[b, h, j]
    return o, lse, new_k, new_v


def compress_step_ragged(q_mem, k_mem, v_mem, k_cache, v_cache, mem_lens, c, t, scale=None):
    """compress_step for a batch whose sequences finish their chunks at different times: sequence b
    is compressed with its own mem_lens[b] when that is >= 0 and left alone otherwise (each sequence
    is its own run of the generator).  Returns (o_mem [B,H,t,D] with NaN rows for untouched
    sequences, lse likewise, k_cache', v_cache')."""
    q_mem = _f64(q_mem)
    B, H, _, D = q_mem.shape
    o = np.full((B, H, t, D), np.nan)
    lse = np.full((B, H, t), np.nan)
    kc = np.array(k_cache, copy=True)
    vc = np.array(v_cache, copy=True)
    for b in range(B):
        n = int(mem_lens[b])
        if n < 0:
            continue
        ob, lb, kb, vb = compress_step(q_mem[b:b + 1], np.asarray(k_mem)[b:b + 1], np.asarray(v_mem)[b:b + 1],
                                       np.asarray(k_cache)[b:b + 1], np.asarray(v_cache)[b:b + 1], n, c, t, 0, scale)
        o[b], lse[b] = ob[0], lb[0]
        kc[b, :, :n + t] = kb[0]
        vc[b, :, :n + t] = vb[0]
    return o, lse, kc, vc


def compress_step_paged(q_mem, k_mem, v_mem, k_pool, v_pool, block_table, mem_lens, c, t, scale=None):
    """compress_step_ragged over a paged cache: read the logical caches out of the pools, compress per sequence,
    write the t new memory entries of every compressing sequence back into their pages.
    Returns (o_mem, lse, k_pool', v_pool')."""
    k_pool, v_pool = np.asarray(k_pool), np.asarray(v_pool)
    ps = k_pool.shape[2]
    cap = max(int(n) for n in mem_lens) + c * t
    kc = paged_to_contiguous(k_pool, block_table, cap)
    vc = paged_to_contiguous(v_pool, block_table, cap)
    o, lse, kc2, vc2 = compress_step_ragged(q_mem, k_mem, v_mem, kc, vc, mem_lens, c, t, scale)
    kp, vp = k_pool.copy(), v_pool.copy()
    for b, n in enumerate(mem_lens):
        n = int(n)
        if n < 0:
            continue
        for j in range(n, n + t):
            page = int(block_table[b][j // ps])
            kp[page, :, j % ps] = kc2[b, :, j]
            vp[page, :, j % ps] = vc2[b, :, j]
    return o, lse, kp, vp


def replay_generation(q, k, v, n_chunks, c, t, tail_read=0, flags=0, scale=None):
    """Run the laid-out sequence through the generation path chunk by chunk.

    For chunk y: the tc reading rows are decoded one token at a time, then the t
    memory rows run as one compress pass and the cache is compacted.  Repetition
    rows have no counterpart at generation time and are left as NaN.  A reading
    tail is decoded after the last compress.

    Returns (O [B,H,S,D] with NaN on repetition rows, k_cache, v_cache, length):
    the final cache arrays [B,H,cap,D] and their valid length.
    """
    q, k, v = np.asarray(q), np.asarray(k), np.asarray(v)
    B, H, S, D = q.shape
    tc = t * c
    s = chunk_len(c, t, flags)
    cap = n_chunks * t + max(tc, tail_read) + 1
    kc = np.zeros((B, H, cap, D), dtype=k.dtype)
    vc = np.zeros((B, H, cap, D), dtype=v.dtype)
    O = np.full((B, H, S, D), np.nan)
    length = 0
    for y in range(n_chunks):
        base = y * s
        for o_ in range(tc):
            i = base + o_
            out, _, kc, vc = decode_attn(q[:, :, i:i + 1], k[:, :, i:i + 1], v[:, :, i:i + 1],
                                         kc, vc, length, scale)
            O[:, :, i] = out[:, :, 0]
            length += 1
        m0 = base + tc
        mem_len = y * t
        assert length == mem_len + tc
        out, _, nk, nv = compress_step(q[:, :, m0:m0 + t], k[:, :, m0:m0 + t], v[:, :, m0:m0 + t],
                                       kc, vc, mem_len, c, t, flags, scale)
        O[:, :, m0:m0 + t] = out
        length = mem_len + t
        kc[:, :, :length] = nk
        vc[:, :, :length] = nv
    for o_ in range(tail_read):
        i = n_chunks * s + o_
        out, _, kc, vc = decode_attn(q[:, :, i:i + 1], k[:, :, i:i + 1], v[:, :, i:i + 1],
                                     kc, vc, length, scale)
        O[:, :, i] = out[:, :, 0]
        length += 1
    return O, kc, vc, length
