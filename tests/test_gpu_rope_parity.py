"""Parity of loma_rope_apply (through the C ABI) with the oracle's rotary embedding at the
layout's position ids.  fp32: max |delta| <= 1e-5 * max(1, max |x|) (a rotation keeps sizes);
bf16: the rotated values are rounded once to bf16, max |delta| <= 2e-2 and mean <= 2e-3 on N(0,1)."""

import numpy as np
import pytest
import torch

import oracle
from paper_2401_09486_b200 import binding as L
from paper_2401_09486_b200 import build, synthetic

pytestmark = pytest.mark.gpu
NOREP = L.LOMA_FLAG_NO_REP_ZONE
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _library():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    build.build_library()
    L.lib()
    torch.cuda.set_device(0)
    yield
    assert L.loma_device_status() == 0


def npf(x):
    return x.detach().to("cpu").to(torch.float64).numpy()


def check(got, want, dtype):
    d = np.abs(npf(got) - want)
    if dtype == torch.float32:
        assert d.max() <= 1e-5 * max(1.0, np.abs(want).max()), d.max()
    else:
        assert d.max() <= 2e-2 and d.mean() <= 2e-3, (d.max(), d.mean())


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("ptype", [0, 1])
@pytest.mark.parametrize("B,H,D,n,c,t,tail,flags", [(1, 1, 64, 2, 4, 4, 0, 0), (2, 3, 128, 5, 4, 16, 37, 0),
                                                    (1, 2, 128, 128, 8, 32, 0, 0),       # ids up to 32767
                                                    (2, 2, 64, 4, 1, 5, 2, 0), (1, 2, 128, 0, 4, 0, 301, 0),
                                                    (2, 2, 128, 3, 8, 32, 100, NOREP)])
def test_rope_matches_oracle(B, H, D, n, c, t, tail, flags, ptype, dtype):
    S = oracle.seq_len(n, c, t, tail, flags)
    q, k, _ = synthetic.qkv(B, H, S, D, seed=21, std=1.0, dtype=dtype)
    wq, wk = oracle.rope_apply(npf(q), npf(k), n, c, t, tail, flags, 10000.0, "contiguous" if ptype else "intermittent")
    gq, gk = q.to(DEV), k.to(DEV)
    L.loma_rope_apply(gq, gk, n, c, t, tail, flags, 0.0, ptype)
    torch.cuda.synchronize()
    check(gq, wq, dtype)
    check(gk, wk, dtype)


def test_rope_strided_views_single_tensor_and_custom_base():
    B, H, D, n, c, t = 2, 3, 128, 3, 4, 16
    S = oracle.seq_len(n, c, t)
    buf = synthetic.normal_tensor((B, S, 2, H, D), 31, 1.0, torch.float32).to(DEV)
    q, k = (buf[:, :, i].permute(0, 2, 1, 3) for i in range(2))
    q0, k0 = npf(q), npf(k)
    L.loma_rope_apply(q, None, n, c, t, 0, 0, 500000.0)
    torch.cuda.synchronize()
    wq, _ = oracle.rope_apply(q0, k0, n, c, t, theta_base=500000.0)
    check(q, wq, torch.float32)
    assert np.array_equal(npf(k), k0)          # untouched


def test_rotated_scores_see_positions_only_through_their_difference():
    """Rotating q and k on the device and taking q.k of a reading row with a memory key gives the score
    of the unrotated pair rotated by the id difference that Eq. 14 sets up (an end-to-end use of the ids)."""
    B, H, D, n, c, t = 1, 1, 128, 3, 4, 4
    S = oracle.seq_len(n, c, t)
    q, k, _ = synthetic.qkv(B, H, S, D, seed=33, dtype=torch.float32)
    gq, gk = q.to(DEV), k.to(DEV)
    L.loma_rope_apply(gq, gk, n, c, t)
    torch.cuda.synchronize()
    pos = oracle.position_ids(n, c, t)
    i, j = 2 * (2 * 16 + 4) + 3, 16 + 2                   # reading row of chunk 2, memory key of chunk 0
    got = float((gq[0, 0, i].double() * gk[0, 0, j].double()).sum())
    want = float((oracle.rope_rotate(npf(q)[0, 0, i:i + 1], np.array([pos[i] - pos[j]]))[0] * npf(k)[0, 0, j]).sum())
    assert abs(got - want) < 1e-4


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_inverse_rotation_undoes_the_rotation_and_matches_the_oracle_at_negated_positions(dtype):
    B, H, D, n, c, t, tail = 2, 2, 128, 5, 4, 16, 9
    S = oracle.seq_len(n, c, t, tail)
    q, k, _ = synthetic.qkv(B, H, S, D, seed=25, dtype=dtype)
    gq, gk = q.to(DEV), k.to(DEV)
    L.loma_rope_apply(gq, gk, n, c, t, tail, 0, 0.0, L.LOMA_ROPE_INVERSE)
    torch.cuda.synchronize()
    pos = oracle.position_ids(n, c, t, tail)
    check(gq, oracle.rope_rotate(npf(q), -pos), dtype)
    check(gk, oracle.rope_rotate(npf(k), -pos), dtype)
    L.loma_rope_apply(gq, gk, n, c, t, tail)                       # forward rotation of the inverse: back to the start
    torch.cuda.synchronize()
    tol = 1e-5 if dtype == torch.float32 else 3e-2
    assert float((gq.float().cpu() - q.float()).abs().max()) <= tol * max(1.0, float(q.float().abs().max()))


def test_differentiable_rope_then_attention_against_torch_autograd():
    """rope -> masked attention as torch ops built on the library, against torch's own autograd of the same
    composition in fp64 (rotation written with cos/sin tables from the oracle's position ids)."""
    from paper_2401_09486_b200.autograd import loma_masked_attention, loma_rope
    B, H, D, n, c, t = 1, 2, 64, 3, 2, 8
    S = oracle.seq_len(n, c, t)
    q, k, v = (x.to(DEV).requires_grad_(True) for x in synthetic.qkv(B, H, S, D, seed=27, dtype=torch.float32))
    w = synthetic.normal_tensor((B, H, S, D), 28, 1.0, torch.float32).to(DEV)
    rq, rk = loma_rope(q, k, n, c, t)
    (loma_masked_attention(rq, rk, v, n, c, t) * w).sum().backward()
    pos = torch.from_numpy(oracle.position_ids(n, c, t)).double().to(DEV)
    theta = 10000.0 ** (-2.0 * torch.arange(D // 2, dtype=torch.float64, device=DEV) / D)
    ang = pos[:, None] * theta[None, :]
    cs, sn = torch.cos(ang), torch.sin(ang)
    def rot(x):
        a, b = x[..., : D // 2], x[..., D // 2:]
        return torch.cat([a * cs - b * sn, b * cs + a * sn], dim=-1)
    q2, k2, v2 = (x.detach().double().requires_grad_(True) for x in (q, k, v))
    M = torch.from_numpy(oracle.dense_mask(n, c, t)).to(DEV)
    A = (rot(q2) @ rot(k2).transpose(-1, -2)) / D ** 0.5
    ((torch.softmax(A.masked_fill(~M, float("-inf")), dim=-1) @ v2) * w.double()).sum().backward()
    torch.cuda.synchronize()
    for g, g2 in ((q.grad, q2.grad), (k.grad, k2.grad), (v.grad, v2.grad)):
        assert float((g.double() - g2).abs().max()) <= 2e-5 * max(1.0, float(g2.abs().max()))


# ------------------------------------------------- rotation fused into the generation steps

def _round_to(x64, dtype):
    """fp64 array -> rounded once to the storage type -> fp64."""
    return torch.from_numpy(x64).to(dtype).to(torch.float64).numpy()


def _ulp_close(got, want64, dtype):
    """The appended keys are rotated in fp32 on the device and rounded to the storage type: equal to the fp64
    rotation rounded the same way, up to one unit in the last place where a rounding tie falls differently."""
    g = npf(got)
    if dtype == torch.float32:
        assert np.abs(g - want64).max() <= 2e-6          # fp32 arithmetic on values of size about one
    else:
        tol = 2.0 ** -7 * np.maximum(np.abs(want64), 2.0 ** -6)
        assert (np.abs(g - _round_to(want64, dtype)) <= tol).all()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("flags", [0, L.LOMA_FLAG_FORCE_GENERIC])
@pytest.mark.parametrize("B,H,D,cap,cache_len,pos", [(1, 1, 64, 4, 0, 0), (2, 3, 128, 40, 17, 5), (2, 2, 128, 700, 613, 2500),
                                                      (1, 4, 64, 9000, 8300, 32767), (3, 2, 128, 5000, 4999, 20001)])
def test_decode_with_fused_rotation_matches_oracle(B, H, D, cap, cache_len, pos, flags, dtype):
    kc = synthetic.normal_tensor((B, H, cap, D), 71, 1.0, dtype)
    vc = synthetic.normal_tensor((B, H, cap, D), 72, 1.0, dtype)
    q, kn, vn = synthetic.qkv(B, H, 1, D, seed=73, std=1.0, dtype=dtype)
    q_rot = oracle.rope_rotate(npf(q), [pos])
    k_rot = oracle.rope_rotate(npf(kn), [pos])
    want_o, want_lse, _, _ = oracle.decode_attn(q_rot, _round_to(k_rot, dtype), npf(vn), npf(kc), npf(vc), cache_len)
    kcd, vcd = kc.to(DEV), vc.to(DEV)
    o = torch.full((B, H, 1, D), float("nan"), dtype=dtype, device=DEV)
    lse = torch.full((B, H), float("nan"), dtype=torch.float32, device=DEV)
    ws = torch.empty(max(16, L.loma_decode_workspace_bytes(B, H, D, cache_len)), dtype=torch.uint8, device=DEV)
    L.loma_decode_attn_rope(q.to(DEV), kn.to(DEV), vn.to(DEV), kcd, vcd, o, lse, cache_len, pos, ws, flags)
    torch.cuda.synchronize()
    check(o, want_o, dtype)
    assert np.abs(npf(lse) - want_lse.reshape(B, H)).max() <= (1e-5 if dtype == torch.float32 else 2e-2)
    # the cache: the rotated key and the value appended at cache_len, nothing else touched
    keep = [j for j in range(cap) if j != cache_len]
    assert torch.equal(kcd[:, :, keep].cpu(), kc[:, :, keep]) and torch.equal(vcd[:, :, keep].cpu(), vc[:, :, keep])
    assert torch.equal(vcd[:, :, cache_len].cpu(), vn[:, :, 0])
    _ulp_close(kcd[:, :, cache_len], k_rot[:, :, 0], dtype)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("flags", [0, L.LOMA_FLAG_MEM_SEES_PRIOR_MEM, L.LOMA_FLAG_FORCE_GENERIC])
@pytest.mark.parametrize("B,H,D,c,t,mem_len,pos0,stride", [(1, 1, 64, 4, 4, 0, 3, 4), (2, 2, 128, 4, 16, 48, 3 * 64 + 3, 4),
                                                            (2, 3, 128, 8, 16, 1024, 64 * 128 + 7, 8), (1, 2, 128, 4, 16, 512, 512, 1),
                                                            (1, 2, 64, 2, 40, 80, 2 * 80 + 1, 2)])
def test_compress_with_fused_rotation_matches_oracle(B, H, D, c, t, mem_len, pos0, stride, flags, dtype):
    tc = c * t
    cap = mem_len + tc + 3
    kc = synthetic.normal_tensor((B, H, cap, D), 81, 1.0, dtype)
    vc = synthetic.normal_tensor((B, H, cap, D), 82, 1.0, dtype)
    qm, km, vm = synthetic.qkv(B, H, t, D, seed=83, std=1.0, dtype=dtype)
    pos = [pos0 + j * stride for j in range(t)]
    q_rot = oracle.rope_rotate(npf(qm), pos)
    k_rot = oracle.rope_rotate(npf(km), pos)
    prior = flags & L.LOMA_FLAG_MEM_SEES_PRIOR_MEM
    want_o, _, want_k, want_v = oracle.compress_step(q_rot, _round_to(k_rot, dtype), npf(vm), npf(kc), npf(vc), mem_len, c, t, prior)
    kcd, vcd = kc.to(DEV), vc.to(DEV)
    om = torch.full((B, H, t, D), float("nan"), dtype=dtype, device=DEV)
    ws = torch.empty(max(16, L.loma_compress_workspace_bytes(B, H, D, t, mem_len, prior)), dtype=torch.uint8, device=DEV)
    L.loma_compress_step_rope(qm.to(DEV), km.to(DEV), vm.to(DEV), kcd, vcd, om, None, mem_len, c, t, pos0, stride, ws, flags)
    torch.cuda.synchronize()
    check(om, want_o, dtype)
    assert torch.equal(kcd[:, :, :mem_len].cpu(), kc[:, :, :mem_len]) and torch.equal(vcd[:, :, :mem_len].cpu(), vc[:, :, :mem_len])
    assert torch.equal(vcd[:, :, mem_len:mem_len + t].cpu(), vm)
    _ulp_close(kcd[:, :, mem_len:mem_len + t], k_rot, dtype)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("ptype", [0, 1])
def test_generation_with_fused_rotation_equals_rotated_one_shot_forward(ptype, dtype):
    """Decode every reading token at its id and compress every chunk at the memory ids (Eq. 14, or the
    generator's contiguous ids) with the rotation fused into the steps: every reading and memory row equals the
    one-shot forward over Q and K rotated at the layout's position ids."""
    B, H, D, n, c, t, tail = 1, 2, 128, 3, 4, 16, 9
    tc, s = c * t, oracle.chunk_len(c, t)
    S = oracle.seq_len(n, c, t, tail)
    q, k, v = synthetic.qkv(B, H, S, D, seed=91, std=1.0, dtype=dtype)
    wq, wk = oracle.rope_apply(npf(q), npf(k), n, c, t, tail, 0, 10000.0, "contiguous" if ptype else "intermittent")
    want_o, _ = oracle.masked_attn_fwd(wq, wk, npf(v), n, c, t, tail)
    pos = oracle.position_ids(n, c, t, tail, 0, "contiguous" if ptype else "intermittent")
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    cap = n * t + tc + 4
    kc = torch.zeros((B, H, cap, D), dtype=dtype, device=DEV)
    vc = torch.zeros_like(kc)
    got = torch.full_like(qd, float("nan"))
    ws = torch.empty(max(16, L.loma_decode_workspace_bytes(B, H, D, cap)), dtype=torch.uint8, device=DEV)
    length = 0
    rows = lambda a, b: slice(a, b)
    for y in range(n + 1):
        nread = tc if y < n else tail
        for o_ in range(nread):
            i = y * s + o_
            o1 = torch.empty((B, H, 1, D), dtype=dtype, device=DEV)
            L.loma_decode_attn_rope(qd[:, :, i:i + 1].contiguous(), kd[:, :, i:i + 1].contiguous(), vd[:, :, i:i + 1].contiguous(),
                                    kc, vc, o1, None, length, int(pos[i]), ws)
            got[:, :, i] = o1[:, :, 0]
            length += 1
        if y < n:
            m0 = y * s + tc
            om = torch.empty((B, H, t, D), dtype=dtype, device=DEV)
            p0 = int(pos[m0]); st = int(pos[m0 + 1] - pos[m0])
            L.loma_compress_step_rope(qd[:, :, m0:m0 + t].contiguous(), kd[:, :, m0:m0 + t].contiguous(),
                                      vd[:, :, m0:m0 + t].contiguous(), kc, vc, om, None, y * t, c, t, p0, st, None)
            got[:, :, m0:m0 + t] = om
            length = (y + 1) * t
    torch.cuda.synchronize()
    zone = oracle.layout_index(n, c, t, tail)[1]
    live = zone != oracle.ZONE_REP
    check(got[:, :, torch.from_numpy(live).to(DEV)], want_o[:, :, live], dtype)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("flags", [0, L.LOMA_FLAG_FORCE_GENERIC])
def test_ragged_steps_with_fused_rotation_match_the_oracle_per_sequence(flags, dtype):
    """One cache length, one position (decode) or one first memory id (compress) per sequence."""
    B, H, D, c, t = 4, 2, 128, 4, 16
    tc = c * t
    cap = 700
    lens = [0, 17, 613, 250]
    poss = [0, 90, 20001, 1234]
    kc = synthetic.normal_tensor((B, H, cap, D), 101, 1.0, dtype)
    vc = synthetic.normal_tensor((B, H, cap, D), 102, 1.0, dtype)
    q, kn, vn = synthetic.qkv(B, H, 1, D, seed=103, std=1.0, dtype=dtype)
    kcd, vcd = kc.to(DEV), vc.to(DEV)
    o = torch.full((B, H, 1, D), float("nan"), dtype=dtype, device=DEV)
    ws = torch.empty(max(16, L.loma_decode_workspace_bytes(B, H, D, max(lens))), dtype=torch.uint8, device=DEV)
    L.loma_decode_attn_ragged_rope(q.to(DEV), kn.to(DEV), vn.to(DEV), kcd, vcd, o, None,
                                   torch.tensor(lens, dtype=torch.int32, device=DEV), max(lens),
                                   torch.tensor(poss, dtype=torch.int32, device=DEV), ws, flags)
    torch.cuda.synchronize()
    for b in range(B):
        sl = slice(b, b + 1)
        q_rot = oracle.rope_rotate(npf(q[sl]), [poss[b]])
        k_rot = oracle.rope_rotate(npf(kn[sl]), [poss[b]])
        want, _, _, _ = oracle.decode_attn(q_rot, _round_to(k_rot, dtype), npf(vn[sl]), npf(kc[sl]), npf(vc[sl]), lens[b])
        check(o[sl], want, dtype)
        _ulp_close(kcd[sl, :, lens[b]], k_rot[:, :, 0], dtype)
        assert torch.equal(vcd[b, :, lens[b]].cpu(), vn[b, :, 0])
    # compress: sequences 0 and 2 compress now, 1 and 3 do not
    mem_lens = [32, -1, 160, -1]
    pos0s = [2 * tc + c - 1, 0, 10 * tc + c - 1, 0]
    kc2 = synthetic.normal_tensor((B, H, cap, D), 104, 1.0, dtype)
    vc2 = synthetic.normal_tensor((B, H, cap, D), 105, 1.0, dtype)
    qm, km, vm = synthetic.qkv(B, H, t, D, seed=106, std=1.0, dtype=dtype)
    kcd, vcd = kc2.to(DEV), vc2.to(DEV)
    om = torch.full((B, H, t, D), float("nan"), dtype=dtype, device=DEV)
    L.loma_compress_step_ragged_rope(qm.to(DEV), km.to(DEV), vm.to(DEV), kcd, vcd, om, None,
                                     torch.tensor(mem_lens, dtype=torch.int32, device=DEV), max(mem_lens), c, t,
                                     torch.tensor(pos0s, dtype=torch.int32, device=DEV), c, flags)
    torch.cuda.synchronize()
    for b in range(B):
        sl = slice(b, b + 1)
        if mem_lens[b] < 0:
            assert torch.equal(kcd[sl].cpu(), kc2[sl]) and torch.equal(vcd[sl].cpu(), vc2[sl])     # left alone
            continue
        pos = [pos0s[b] + j * c for j in range(t)]
        q_rot, k_rot = oracle.rope_rotate(npf(qm[sl]), pos), oracle.rope_rotate(npf(km[sl]), pos)
        want, _, _, _ = oracle.compress_step(q_rot, _round_to(k_rot, dtype), npf(vm[sl]), npf(kc2[sl]), npf(vc2[sl]), mem_lens[b], c, t)
        check(om[sl], want, dtype)
        _ulp_close(kcd[sl, :, mem_lens[b]:mem_lens[b] + t], k_rot, dtype)
        assert torch.equal(vcd[sl, :, mem_lens[b]:mem_lens[b] + t].cpu(), vm[sl])
        assert torch.equal(kcd[sl, :, :mem_lens[b]].cpu(), kc2[sl, :, :mem_lens[b]])


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_staggered_sequences_over_a_paged_cache_with_fused_rotation(dtype):
    """Three sequences that started 0, 5 and 11 tokens apart share one pool of pages; every step decodes one token of
    every sequence at that sequence's own position id and a sequence compresses (memory ids of Eq. 14) as soon as its
    tail is full: every reading and memory row equals the one-shot forward over Q and K rotated at the layout's ids."""
    H, D, n, c, t, tail, ps = 2, 128, 3, 2, 8, 5, 16
    tc, s = c * t, oracle.chunk_len(c, t)
    S = oracle.seq_len(n, c, t, tail)
    B, starts = 3, [0, 5, 11]
    q, k, v = synthetic.qkv(B, H, S, D, seed=111, std=1.0, dtype=dtype)
    wq, wk = oracle.rope_apply(npf(q), npf(k), n, c, t, tail)
    want_o, _ = oracle.masked_attn_fwd(wq, wk, npf(v), n, c, t, tail)
    ids = oracle.position_ids(n, c, t, tail)
    zone = oracle.layout_index(n, c, t, tail)[1]
    gen_rows = [i for i in range(S) if zone[i] == oracle.ZONE_READ]
    max_pages = (n * t + tc + ps - 1) // ps + 1
    n_pages = B * max_pages
    table = np.random.default_rng(4).permutation(n_pages).reshape(B, max_pages).astype(np.int32)
    kpool = torch.zeros((n_pages, H, ps, D), dtype=dtype, device=DEV)
    vpool = torch.zeros_like(kpool)
    table_d = torch.from_numpy(table).to(DEV)
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    got = torch.full((B, H, S, D), float("nan"), dtype=dtype, device=DEV)
    ws = torch.empty(max(16, L.loma_decode_workspace_bytes(B, H, D, n * t + tc)), dtype=torch.uint8, device=DEV)
    i32 = lambda xs: torch.tensor(xs, dtype=torch.int32, device=DEV)
    nxt, lens, chunks, step = [0] * B, [0] * B, [0] * B, 0
    while any(p_ < len(gen_rows) for p_ in nxt):
        active = [step >= starts[b] and nxt[b] < len(gen_rows) for b in range(B)]
        rows = [gen_rows[min(nxt[b], len(gen_rows) - 1)] for b in range(B)]
        take = lambda x: torch.stack([x[b, :, rows[b]:rows[b] + 1] for b in range(B)]).contiguous()
        o1 = torch.empty((B, H, 1, D), dtype=dtype, device=DEV)
        # idle sequences decode a throw-away token into a spare slot of their own pages (their length does not advance)
        L.loma_decode_attn_paged_rope(take(qd), take(kd), take(vd), kpool, vpool, table_d, o1, None, i32(lens), max(lens),
                                      i32([int(ids[r]) for r in rows]), ws)
        for b in range(B):
            if active[b]:
                got[b, :, rows[b]] = o1[b, :, 0]
                nxt[b] += 1
                lens[b] += 1
        mem_lens = [chunks[b] * t if (lens[b] == chunks[b] * t + tc and chunks[b] < n) else -1 for b in range(B)]
        if any(m >= 0 for m in mem_lens):
            m_rows = [chunks[b] * s + tc for b in range(B)]
            takem = lambda x: torch.stack([x[b, :, m_rows[b]:m_rows[b] + t] if mem_lens[b] >= 0 else x[b, :, :t]
                                           for b in range(B)]).contiguous()
            om = torch.empty((B, H, t, D), dtype=dtype, device=DEV)
            L.loma_compress_step_paged_rope(takem(qd), takem(kd), takem(vd), kpool, vpool, table_d, om, None, i32(mem_lens),
                                            max(mem_lens), c, t, i32([int(ids[min(m_rows[b], S - 1)]) for b in range(B)]), c)
            for b in range(B):
                if mem_lens[b] >= 0:
                    got[b, :, m_rows[b]:m_rows[b] + t] = om[b]
                    chunks[b] += 1
                    lens[b] = chunks[b] * t
        step += 1
    torch.cuda.synchronize()
    live = zone != oracle.ZONE_REP
    check(got[:, :, torch.from_numpy(live).to(DEV)], want_o[:, :, live], dtype)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("flags", [0, L.LOMA_FLAG_FORCE_GENERIC])
@pytest.mark.parametrize("l,cache_len,pos0", [(1, 5, 5), (17, 100, 4000), (200, 333, 30000), (64, 0, 0)])
def test_prompt_piece_with_fused_rotation_matches_oracle(l, cache_len, pos0, flags, dtype):
    """Appendix A `inference_input` with l tokens and position_ids cursor .. cursor + l - 1: the step equals
    rotate-then-attend in the oracle, the cache receives the rotated keys (rounded once), the caller's q is untouched."""
    B, H, D = 2, 2, 128
    cap = cache_len + l + 3
    kc = synthetic.normal_tensor((B, H, cap, D), 171, 1.0, dtype)
    vc = synthetic.normal_tensor((B, H, cap, D), 172, 1.0, dtype)
    q, kn, vn = synthetic.qkv(B, H, l, D, seed=173, std=1.0, dtype=dtype)
    pos = [pos0 + i for i in range(l)]
    q_rot = oracle.rope_rotate(npf(q), pos)
    k_rot = oracle.rope_rotate(npf(kn), pos)
    want_o, want_lse, _, _ = oracle.prefill_attn(q_rot, _round_to(k_rot, dtype), npf(vn), npf(kc), npf(vc), cache_len)
    kcd, vcd, qd = kc.to(DEV), vc.to(DEV), q.to(DEV)
    o = torch.full((B, H, l, D), float("nan"), dtype=dtype, device=DEV)
    lse = torch.full((B, H, l), float("nan"), dtype=torch.float32, device=DEV)
    L.loma_prefill_attn_rope(qd, kn.to(DEV), vn.to(DEV), kcd, vcd, o, lse, cache_len, pos0, flags)
    torch.cuda.synchronize()
    check(o, want_o, dtype)
    assert np.abs(npf(lse) - want_lse).max() <= (1e-5 if dtype == torch.float32 else 2e-2)
    assert torch.equal(qd.cpu(), q)
    assert torch.equal(kcd[:, :, :cache_len].cpu(), kc[:, :, :cache_len]) and torch.equal(vcd[:, :, :cache_len].cpu(), vc[:, :, :cache_len])
    assert torch.equal(vcd[:, :, cache_len:cache_len + l].cpu(), vn)
    _ulp_close(kcd[:, :, cache_len:cache_len + l], k_rot, dtype)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("paged", [False, True])
def test_ragged_and_paged_prompt_pieces_with_fused_rotation(paged, dtype):
    """One position and one cache length per sequence; contiguous cache and 128-row pages."""
    B, H, D, l, ps = 3, 2, 128, 40, 128
    lens, poss = [100, 0, 300], [1000, 0, 20000]
    max_len = max(lens)
    q, kn, vn = synthetic.qkv(B, H, l, D, seed=181, std=1.0, dtype=dtype)
    mp = (max_len + l + ps - 1) // ps
    cap = mp * ps
    kc = synthetic.normal_tensor((B, H, cap, D), 182, 1.0, dtype)
    vc = synthetic.normal_tensor((B, H, cap, D), 183, 1.0, dtype)
    o = torch.full((B, H, l, D), float("nan"), dtype=dtype, device=DEV)
    lens_d = torch.tensor(lens, dtype=torch.int32, device=DEV)
    pos_d = torch.tensor(poss, dtype=torch.int32, device=DEV)
    if paged:
        g = torch.Generator().manual_seed(184)
        table = torch.randperm(B * mp, generator=g).to(torch.int32).view(B, mp)
        kpool = torch.empty((B * mp, H, ps, D), dtype=dtype)
        vpool = torch.empty_like(kpool)
        for b in range(B):
            for pi in range(mp):
                kpool[int(table[b, pi])] = kc[b, :, pi * ps:(pi + 1) * ps]
                vpool[int(table[b, pi])] = vc[b, :, pi * ps:(pi + 1) * ps]
        kpd, vpd = kpool.to(DEV), vpool.to(DEV)
        L.loma_prefill_attn_paged_rope(q.to(DEV), kn.to(DEV), vn.to(DEV), kpd, vpd, table.to(DEV), o, None, lens_d, max_len, pos_d)
        torch.cuda.synchronize()
        kc_after = torch.stack([torch.cat([kpd[int(table[b, pi])].cpu() for pi in range(mp)], dim=1) for b in range(B)])
    else:
        kcd, vcd = kc.to(DEV), vc.to(DEV)
        L.loma_prefill_attn_ragged_rope(q.to(DEV), kn.to(DEV), vn.to(DEV), kcd, vcd, o, None, lens_d, max_len, pos_d)
        torch.cuda.synchronize()
        kc_after = kcd.cpu()
    for b, (n, p0) in enumerate(zip(lens, poss)):
        sl = slice(b, b + 1)
        pos = [p0 + i for i in range(l)]
        q_rot = oracle.rope_rotate(npf(q[sl]), pos)
        k_rot = oracle.rope_rotate(npf(kn[sl]), pos)
        want_o, _, _, _ = oracle.prefill_attn(q_rot, _round_to(k_rot, dtype), npf(vn[sl]), npf(kc[sl, :, :n + l]),
                                              npf(vc[sl, :, :n + l]), n)
        check(o[sl], want_o, dtype)
        _ulp_close(kc_after[sl, :, n:n + l], k_rot, dtype)
        assert torch.equal(kc_after[b, :, :n], kc[b, :, :n])
    assert L.loma_device_status() == 0
