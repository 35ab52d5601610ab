"""Parity of the CUDA library (through the C ABI) with the CPU oracle, element by
element on the same seeded inputs.

Tolerances: integer maps and cache contents are bit-exact.  fp32 attention
outputs: max |delta| <= 1e-5.  bf16 (fp32 accumulation) on N(0,1) inputs:
max |delta| <= 2e-2 and mean |delta| <= 2e-3.
"""

import numpy as np
import pytest
import torch

import oracle
from paper_2401_09486_b200 import binding as L
from paper_2401_09486_b200 import build, synthetic

pytestmark = pytest.mark.gpu

PRIOR = L.LOMA_FLAG_MEM_SEES_PRIOR_MEM
NOREP = L.LOMA_FLAG_NO_REP_ZONE
GENERIC = L.LOMA_FLAG_FORCE_GENERIC
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


def npf(x: torch.Tensor) -> np.ndarray:
    return x.detach().to("cpu").to(torch.float64).numpy()


def bits(x: torch.Tensor) -> np.ndarray:
    return x.detach().cpu().contiguous().view(torch.int16 if x.dtype == torch.bfloat16 else torch.int32).numpy()


def check_close(got: torch.Tensor, want: np.ndarray, dtype):
    g = npf(got)
    assert g.shape == want.shape
    assert np.isfinite(g).all()
    d = np.abs(g - want)
    if dtype == torch.float32:
        assert d.max() <= 1e-5, f"fp32 max |delta| {d.max():.3e}"
    else:
        assert d.max() <= 2e-2, f"bf16 max |delta| {d.max():.3e}"
        assert d.mean() <= 2e-3, f"bf16 mean |delta| {d.mean():.3e}"


def run_fwd(q, k, v, n, c, t, tail=0, flags=0, scale=0.0, want_lse=True):
    o = torch.full_like(q, float("nan"))
    lse = torch.full(q.shape[:3], float("nan"), dtype=torch.float32, device=q.device) if want_lse else None
    L.loma_masked_attn_fwd(q, k, v, o, lse, n, c, t, tail, flags, scale)
    torch.cuda.synchronize()
    return o, lse


def workspace(nbytes):
    return torch.empty(max(16, nbytes), dtype=torch.uint8, device=DEV)


# ----------------------------------------------------------------- index maps

@pytest.mark.parametrize("n,c,t,tail", [(0, 4, 0, 9), (3, 2, 2, 0), (2, 4, 4, 3), (32, 4, 16, 0), (128, 8, 32, 0),
                                        (5, 3, 7, 21)])
def test_device_layout_index_bit_exact(n, c, t, tail):
    got = L.loma_layout_index(n, c, t, tail, device=DEV)
    torch.cuda.synchronize()
    for g, w in zip(got, oracle.layout_index(n, c, t, tail)):
        assert np.array_equal(g.cpu().numpy(), w)


@pytest.mark.parametrize("n_tok,c,t", [(1, 4, 4), (1000, 4, 16), (777, 8, 16), (50, 3, 0)])
def test_device_generation_index_bit_exact(n_tok, c, t):
    got = L.loma_generation_index(n_tok, c, t, device=DEV)
    torch.cuda.synchronize()
    for g, w in zip(got, oracle.generation_index(n_tok, c, t)):
        assert np.array_equal(g.cpu().numpy(), w)


# ------------------------------------------------------- masked forward, small

FWD_CASES = [
    # B, H, D, n, c, t, tail
    (1, 1, 64, 2, 4, 4, 0),       # the tiny configuration (72 rows)
    (2, 3, 64, 3, 2, 2, 3),
    (1, 2, 128, 2, 4, 16, 0),     # one 64|16|64 chunk pair
    (2, 2, 128, 5, 4, 16, 37),    # several tiles and a ragged reading tail
    (1, 2, 128, 3, 8, 16, 0),     # tc = 128
    (1, 1, 128, 3, 8, 32, 200),   # tc = 256 with a tail
    (1, 2, 64, 4, 1, 5, 2),       # c = 1, odd t
    (1, 1, 128, 2, 3, 7, 0),      # nothing is a power of two
    (1, 2, 128, 0, 4, 0, 301),    # t = 0: plain causal attention
    (1, 1, 64, 1, 2, 64, 0),      # t = 64
    (1, 1, 128, 9, 2, 8, 16),     # t = 8
]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("flags", [0, PRIOR, GENERIC, GENERIC | PRIOR])
@pytest.mark.parametrize("B,H,D,n,c,t,tail", FWD_CASES)
def test_masked_fwd_matches_oracle(B, H, D, n, c, t, tail, flags, dtype):
    S = oracle.seq_len(n, c, t, tail)
    q, k, v = synthetic.qkv(B, H, S, D, seed=7, std=1.0, dtype=dtype)
    want_o, want_lse = oracle.masked_attn_fwd(npf(q), npf(k), npf(v), n, c, t, tail, flags & PRIOR)
    o, lse = run_fwd(q.to(DEV), k.to(DEV), v.to(DEV), n, c, t, tail, flags)
    check_close(o, want_o, dtype)
    lse_tol = 1e-5 if dtype == torch.float32 else 2e-2
    assert np.abs(npf(lse) - want_lse).max() <= lse_tol


def test_masked_fwd_strided_views_and_explicit_scale():
    """Q/K/V/O given as views into a packed [B, S, 3+1, H, D]-style buffer."""
    B, H, D, n, c, t = 2, 3, 128, 3, 4, 16
    S = oracle.seq_len(n, c, t)
    buf = synthetic.normal_tensor((B, S, 4, H, D), 9, 1.0, torch.bfloat16).to(DEV)
    q, k, v, o = (buf[:, :, i].permute(0, 2, 1, 3) for i in range(4))      # [B, H, S, D] strided
    want_o, _ = oracle.masked_attn_fwd(npf(q), npf(k), npf(v), n, c, t, scale=0.05)
    L.loma_masked_attn_fwd(q, k, v, o, None, n, c, t, 0, 0, 0.05)
    torch.cuda.synchronize()
    check_close(o, want_o, torch.bfloat16)


def test_same_tensors_with_and_without_repetition_zones_do_not_share_descriptors():
    """Two bf16 calls on the same addresses with the same strides, B, H, D, n, c, t, once in the training
    layout and once in the layout without repetition zones: the second call must not reuse the TMA
    descriptors of the first (their chunk stride and zone views differ)."""
    B, H, D, n, c, t = 2, 3, 128, 3, 4, 16
    S_full = oracle.seq_len(n, c, t)
    S_norep = oracle.seq_len(n, c, t, 0, NOREP)
    buf = synthetic.normal_tensor((B, S_full, 4, H, D), 19, 1.0, torch.bfloat16).to(DEV)
    q, k, v, o = (buf[:, :, i].permute(0, 2, 1, 3) for i in range(4))      # [B, H, S, D] strided views
    for _ in range(2):                                                       # full, norep, full, norep
        for flags, S in ((0, S_full), (NOREP, S_norep)):
            qs, ks, vs, os_ = (x[:, :, :S] for x in (q, k, v, o))
            assert qs.data_ptr() == q.data_ptr() and qs.stride() == q.stride()
            want_o, _ = oracle.masked_attn_fwd(npf(qs), npf(ks), npf(vs), n, c, t, 0, flags)
            os_.fill_(float("nan"))
            L.loma_masked_attn_fwd(qs, ks, vs, os_, None, n, c, t, 0, flags, 0.0)
            torch.cuda.synchronize()
            check_close(os_, want_o, torch.bfloat16)


# ----------------------------------------- inference layout (no repetition zones)

@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("flags", [NOREP, NOREP | PRIOR, NOREP | GENERIC])
@pytest.mark.parametrize("B,H,D,n,c,t,tail", [(1, 2, 64, 3, 2, 4, 3), (2, 2, 128, 5, 4, 16, 37), (1, 2, 128, 3, 8, 32, 100),
                                              (1, 1, 128, 2, 3, 7, 0), (1, 2, 128, 20, 4, 16, 0)])
def test_prefill_one_pass_matches_oracle_and_fills_the_cache(B, H, D, n, c, t, tail, flags, dtype):
    """One pass over a prompt laid out as [reading | memory] chunks: outputs match the oracle, and
    loma_prefill_cache leaves exactly the cache that token-by-token ingestion would (bit for bit)."""
    of = (flags & PRIOR) | oracle.FLAG_NO_REP_ZONE
    S = oracle.seq_len(n, c, t, tail, of)
    q, k, v = synthetic.qkv(B, H, S, D, seed=17, std=1.0, dtype=dtype)
    want_o, want_lse = oracle.masked_attn_fwd(npf(q), npf(k), npf(v), n, c, t, tail, of)
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    o, lse = run_fwd(qd, kd, vd, n, c, t, tail, flags)
    check_close(o, want_o, dtype)
    assert np.abs(npf(lse) - want_lse).max() <= (1e-5 if dtype == torch.float32 else 2e-2)
    got = L.loma_layout_index(n, c, t, tail, device=DEV, flags=NOREP)
    torch.cuda.synchronize()
    for g, w in zip(got, oracle.layout_index(n, c, t, tail, oracle.FLAG_NO_REP_ZONE)):
        assert np.array_equal(g.cpu().numpy(), w)
    # cache after the prompt = what the oracle's incremental replay leaves
    _, ref_k, ref_v, ref_len = oracle.replay_generation(bits(q) * 0.0, bits(k), bits(v), n, c, t, tail, of, scale=0.0)
    cap = n * t + tail + 5
    kc = torch.full((B, H, cap, D), 7.0, dtype=dtype, device=DEV)
    vc = torch.full((B, H, cap, D), 7.0, dtype=dtype, device=DEV)
    length = L.loma_prefill_cache(kd, vd, kc, vc, n, c, t, tail, NOREP)
    torch.cuda.synchronize()
    assert length == ref_len == n * t + tail
    assert np.array_equal(bits(kc[:, :, :length]), ref_k[:, :, :length])
    assert np.array_equal(bits(vc[:, :, :length]), ref_v[:, :, :length])
    assert (kc[:, :, length:] == 7.0).all() and (vc[:, :, length:] == 7.0).all()      # nothing else is touched


def replay_on_gpu(q, k, v, n, c, t, tail, flags):
    """Drive loma_decode_attn / loma_compress_step over a laid-out sequence the
    way the generator would (host logic only; all arithmetic in the library)."""
    B, H, S, D = q.shape
    tc, s = c * t, oracle.chunk_len(c, t)
    cap = n * t + max(tc, tail) + 1
    kc = torch.zeros(B, H, cap, D, dtype=q.dtype, device=q.device)
    vc = torch.zeros_like(kc)
    out = torch.full_like(q, float("nan"))
    ws = workspace(max(L.loma_decode_workspace_bytes(B, H, D, cap),
                       L.loma_compress_workspace_bytes(B, H, D, max(t, 1), n * t, flags)))
    length = 0

    def decode(i):
        nonlocal length
        o1 = torch.empty(B, H, 1, D, dtype=q.dtype, device=q.device)
        L.loma_decode_attn(q[:, :, i:i + 1].contiguous(), k[:, :, i:i + 1].contiguous(),
                           v[:, :, i:i + 1].contiguous(), kc, vc, o1, None, length, ws, flags)
        out[:, :, i] = o1[:, :, 0]
        length += 1

    for y in range(n):
        for o_ in range(tc):
            decode(y * s + o_)
        m0 = y * s + tc
        om = torch.empty(B, H, t, D, dtype=q.dtype, device=q.device)
        L.loma_compress_step(q[:, :, m0:m0 + t].contiguous(), k[:, :, m0:m0 + t].contiguous(),
                             v[:, :, m0:m0 + t].contiguous(), kc, vc, om, None, y * t, c, t, ws, flags)
        out[:, :, m0:m0 + t] = om
        length = y * t + t
    for o_ in range(tail):
        decode(n * s + o_)
    torch.cuda.synchronize()
    return out, kc, vc, length


def test_tiny_config_fp32_forward_then_incremental_replay():
    """B1 H1 D64 fp32, c=4, t=4, two chunks [16|4|16] = 72 rows, N(0,1) from
    seed 0.  Forward, then the same rows replayed as generation with one compress
    step per chunk; caches compared bit for bit."""
    B, H, D, n, c, t = 1, 1, 64, 2, 4, 4
    tc, s = c * t, oracle.chunk_len(c, t)
    S = n * s
    q, k, v = synthetic.qkv(B, H, S, D, seed=0, std=1.0, dtype=torch.float32)
    want_o, _ = oracle.masked_attn_fwd(npf(q), npf(k), npf(v), n, c, t)
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    o, _ = run_fwd(qd, kd, vd, n, c, t)
    check_close(o, want_o, torch.float32)

    got_o, kc, vc, length = replay_on_gpu(qd, kd, vd, n, c, t, 0, 0)
    zone = oracle.layout_index(n, c, t)[1]
    live = zone != oracle.ZONE_REP
    assert np.abs(npf(got_o)[:, :, live] - want_o[:, :, live]).max() <= 1e-5      # invariant (c)
    ref_o, ref_k, ref_v, ref_len = oracle.replay_generation(q.numpy(), k.numpy(), v.numpy(), n, c, t)
    assert length == ref_len == n * t
    assert np.array_equal(kc[:, :, :length].cpu().numpy(), ref_k[:, :, :length])
    assert np.array_equal(vc[:, :, :length].cpu().numpy(), ref_v[:, :, :length])
    slot, _, comp = L.loma_generation_index(n * tc, c, t, device="cpu")
    assert comp.sum().item() == n


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("flags", [0, PRIOR, GENERIC, GENERIC | PRIOR])
@pytest.mark.parametrize("B,H,D,n,c,t,tail", [(1, 2, 64, 3, 2, 4, 3), (2, 2, 128, 3, 4, 16, 10),
                                              (1, 1, 128, 2, 8, 16, 0), (1, 2, 128, 2, 3, 5, 1)])
def test_incremental_generation_equals_one_shot(B, H, D, n, c, t, tail, flags, dtype):
    """Invariant (c) on the GPU path, and bit-exact compaction."""
    S = oracle.seq_len(n, c, t, tail)
    q, k, v = synthetic.qkv(B, H, S, D, seed=11, std=1.0, dtype=dtype)
    want_o, _ = oracle.masked_attn_fwd(npf(q), npf(k), npf(v), n, c, t, tail, flags & PRIOR)
    got_o, kc, vc, length = replay_on_gpu(q.to(DEV), k.to(DEV), v.to(DEV), n, c, t, tail, flags)
    zone = oracle.layout_index(n, c, t, tail)[1]
    live = zone != oracle.ZONE_REP
    check_close(got_o[:, :, torch.from_numpy(live).to(DEV)], want_o[:, :, live], dtype)
    tc, s = c * t, oracle.chunk_len(c, t)
    rows = [y * s + tc + j for y in range(n) for j in range(t)] + list(range(n * s, S))
    assert length == len(rows)
    assert torch.equal(kc[:, :, :length].cpu(), k[:, :, rows])        # bit for bit
    assert torch.equal(vc[:, :, :length].cpu(), v[:, :, rows])


# ------------------------------------------- several new tokens over an existing cache

@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("flags", [0, GENERIC])
@pytest.mark.parametrize("l", [1, 2, 8, 17, 64, 200, 300])
@pytest.mark.parametrize("cache_len", [0, 16, 100, 8192])
def test_prefill_over_a_cache_matches_oracle_and_appends_bit_exact(l, cache_len, flags, dtype):
    """Appendix A `inference_input` with l tokens: mask tril(ones(l, l + k), diagonal = k), K/V appended."""
    B, H, D = (1, 2, 128) if cache_len > 1000 else (2, 3, 128 if l != 17 else 64)
    cap = cache_len + l + 5
    kc = synthetic.normal_tensor((B, H, cap, D), 41, 1.0, dtype)
    vc = synthetic.normal_tensor((B, H, cap, D), 42, 1.0, dtype)
    q, kn, vn = synthetic.qkv(B, H, l, D, seed=43, std=1.0, dtype=dtype)
    want_o, want_lse, want_kc, want_vc = oracle.prefill_attn(npf(q), npf(kn), npf(vn), npf(kc), npf(vc), cache_len)
    kcd, vcd = kc.to(DEV), vc.to(DEV)
    o = torch.full((B, H, l, D), float("nan"), dtype=dtype, device=DEV)
    lse = torch.full((B, H, l), float("nan"), dtype=torch.float32, device=DEV)
    L.loma_prefill_attn(q.to(DEV), kn.to(DEV), vn.to(DEV), kcd, vcd, o, lse, cache_len, flags)
    torch.cuda.synchronize()
    check_close(o, want_o, dtype)
    assert np.abs(npf(lse) - want_lse).max() <= (1e-5 if dtype == torch.float32 else 2e-2)
    # the cache: new rows appended bit for bit, everything else untouched
    exp_k, exp_v = kc.clone(), vc.clone()
    exp_k[:, :, cache_len:cache_len + l] = kn
    exp_v[:, :, cache_len:cache_len + l] = vn
    assert np.array_equal(bits(kcd), bits(exp_k)) and np.array_equal(bits(vcd), bits(exp_v))
    assert np.array_equal(npf(kcd), want_kc) and np.array_equal(npf(vcd), want_vc)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("flags", [0, GENERIC])
@pytest.mark.parametrize("l,lens", [(1, [0, 5, 130]), (17, [16, 0, 300, 129]), (64, [100, 1000, 0]), (200, [513, 37, 1024, 256])])
def test_ragged_prefill_matches_the_oracle_per_sequence(l, lens, flags, dtype):
    """One run of Appendix A `inference_input` with l tokens per sequence, every sequence over its own number of
    cached entries.  The cache rows past every sequence's end start out as NaN: nothing of them may reach an
    output, and the entries below each sequence's own length stay untouched."""
    B, H, D = len(lens), 2, 128
    max_len = max(lens)
    cap = max_len + l + 130
    kc = synthetic.normal_tensor((B, H, cap, D), 71, 1.0, dtype)
    vc = synthetic.normal_tensor((B, H, cap, D), 72, 1.0, dtype)
    for b, n in enumerate(lens):
        kc[b, :, n:] = float("nan")
        vc[b, :, n:] = float("nan")
    q, kn, vn = synthetic.qkv(B, H, l, D, seed=73, std=1.0, dtype=dtype)
    kcd, vcd = kc.to(DEV), vc.to(DEV)
    o = torch.full((B, H, l, D), float("nan"), dtype=dtype, device=DEV)
    lse = torch.full((B, H, l), float("nan"), dtype=torch.float32, device=DEV)
    lens_d = torch.tensor(lens, dtype=torch.int32, device=DEV)
    L.loma_prefill_attn_ragged(q.to(DEV), kn.to(DEV), vn.to(DEV), kcd, vcd, o, lse, lens_d, max_len, flags)
    torch.cuda.synchronize()
    for b, n in enumerate(lens):
        sl = slice(b, b + 1)
        want_o, want_lse, _, _ = oracle.prefill_attn(npf(q[sl]), npf(kn[sl]), npf(vn[sl]), npf(kc[sl, :, :n + l].nan_to_num()),
                                                     npf(vc[sl, :, :n + l].nan_to_num()), n)
        check_close(o[sl], want_o, dtype)
        assert np.abs(npf(lse[sl]) - want_lse).max() <= (1e-5 if dtype == torch.float32 else 2e-2)
        assert np.array_equal(bits(kcd[b, :, :n]), bits(kc[b, :, :n])) and np.array_equal(bits(vcd[b, :, :n]), bits(vc[b, :, :n]))
        assert np.array_equal(bits(kcd[b, :, n:n + l]), bits(kn[b])) and np.array_equal(bits(vcd[b, :, n:n + l]), bits(vn[b]))
    assert L.loma_device_status() == 0


def test_ragged_prefill_with_equal_lengths_equals_the_uniform_call_bit_for_bit():
    B, H, D, l, n = 3, 2, 128, 150, 333
    cap = n + l + 7
    kc = synthetic.normal_tensor((B, H, cap, D), 75, 1.0, torch.bfloat16).to(DEV)
    vc = synthetic.normal_tensor((B, H, cap, D), 76, 1.0, torch.bfloat16).to(DEV)
    q, kn, vn = (x.to(DEV) for x in synthetic.qkv(B, H, l, D, seed=77, std=1.0, dtype=torch.bfloat16))
    o_u, o_r = torch.empty_like(q), torch.empty_like(q)
    kc2, vc2 = kc.clone(), vc.clone()
    L.loma_prefill_attn(q, kn, vn, kc, vc, o_u, None, n)
    L.loma_prefill_attn_ragged(q, kn, vn, kc2, vc2, o_r, None, torch.full((B,), n, dtype=torch.int32, device=DEV), n)
    torch.cuda.synchronize()
    assert torch.equal(o_u, o_r)
    assert torch.equal(kc[:, :, :n + l], kc2[:, :, :n + l]) and torch.equal(vc[:, :, :n + l], vc2[:, :, :n + l])


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("l,ps,lens", [(1, 16, [0, 5, 130]), (17, 16, [16, 0, 300]), (70, 64, [100, 513, 0, 64]),
                                       (70, 128, [100, 513, 0, 64]), (200, 256, [300, 5, 1000]), (8, 128, [127, 128, 121]),
                                       (43, 128, [0]), (81, 128, [1])])      # key view shorter than one 128-row tile
def test_paged_prefill_matches_the_oracle_per_sequence(l, ps, lens, dtype):
    """The same step over a paged cache: pages scattered over the pool by a seeded permutation; the new rows
    land in the pages the block table names, bit for bit.  (bf16 with pages of 128 rows or more runs on the
    tensor-core kernel.)  Every pool row that is not one of a sequence's first cache_lens[b] entries starts out as
    NaN: none of them may reach an output."""
    B, H, D = len(lens), 2, 128
    max_len = max(lens)
    mp = (max_len + l + ps - 1) // ps + 1
    n_pages = B * mp + 3
    g = torch.Generator().manual_seed(79)
    table = torch.randperm(n_pages, generator=g)[:B * mp].to(torch.int32).view(B, mp)
    kpool = synthetic.normal_tensor((n_pages, H, ps, D), 81, 1.0, dtype)
    vpool = synthetic.normal_tensor((n_pages, H, ps, D), 82, 1.0, dtype)
    q, kn, vn = synthetic.qkv(B, H, l, D, seed=83, std=1.0, dtype=dtype)
    owned = torch.zeros((n_pages, ps), dtype=torch.bool)
    for b, n in enumerate(lens):
        for j in range(n):
            owned[int(table[b, j // ps]), j % ps] = True
    kpool[~owned[:, None, :].expand(n_pages, H, ps)] = float("nan")
    vpool[~owned[:, None, :].expand(n_pages, H, ps)] = float("nan")

    def gather(pool, b, n):   # the first n entries of sequence b as [1, H, n, D]
        rows = [pool[int(table[b, j // ps]), :, j % ps] for j in range(n)]
        return torch.stack(rows, dim=1).unsqueeze(0) if rows else pool.new_zeros((1, H, 0, D))

    kpd, vpd = kpool.to(DEV), vpool.to(DEV)
    o = torch.full((B, H, l, D), float("nan"), dtype=dtype, device=DEV)
    lse = torch.full((B, H, l), float("nan"), dtype=torch.float32, device=DEV)
    fallbacks = L.loma_fallback_count()
    L.loma_prefill_attn_paged(q.to(DEV), kn.to(DEV), vn.to(DEV), kpd, vpd, table.to(DEV), o, lse,
                              torch.tensor(lens, dtype=torch.int32, device=DEV), max_len)
    torch.cuda.synchronize()
    assert L.loma_fallback_count() == fallbacks       # a tensor-core call did not end up on CUDA cores
    assert L.loma_device_status() == 0
    kp_after, vp_after = kpd.cpu(), vpd.cpu()
    for b, n in enumerate(lens):
        sl = slice(b, b + 1)
        kc_b = torch.cat([gather(kpool, b, n), torch.zeros((1, H, l, D), dtype=dtype)], dim=2)
        vc_b = torch.cat([gather(vpool, b, n), torch.zeros((1, H, l, D), dtype=dtype)], dim=2)
        want_o, want_lse, _, _ = oracle.prefill_attn(npf(q[sl]), npf(kn[sl]), npf(vn[sl]), npf(kc_b), npf(vc_b), n)
        check_close(o[sl], want_o, dtype)
        assert np.abs(npf(lse[sl]) - want_lse).max() <= (1e-5 if dtype == torch.float32 else 2e-2)
        assert np.array_equal(bits(gather(kp_after, b, n + l)[0, :, n:]), bits(kn[b]))
        assert np.array_equal(bits(gather(vp_after, b, n + l)[0, :, n:]), bits(vn[b]))
        assert np.array_equal(bits(gather(kp_after, b, n)), bits(gather(kpool, b, n)))


@pytest.mark.parametrize("seed", range(16))
def test_ragged_and_paged_prompt_pieces_on_seeded_random_shapes(seed):
    """Shapes nobody picked by hand (batch, heads, head size, piece length, cache lengths around the tile and page
    boundaries, page size; odd seeds paged): bf16 tensor-core path against the oracle, sequence by sequence."""
    import random
    rnd = random.Random(1000 + seed)
    B, H, D = rnd.randint(1, 4), rnd.randint(1, 2), rnd.choice([64, 128])
    l = rnd.randint(8, 200)
    lens = [rnd.choice([0, 1, 127, 128, 129, rnd.randint(0, 700)]) for _ in range(B)]
    max_len = max(lens) + rnd.randint(0, 3)
    paged = seed % 2 == 1
    ps = rnd.choice([128, 256])
    mp = (max_len + l + ps - 1) // ps + 1
    cap = mp * ps
    dtype = torch.bfloat16
    kc = synthetic.normal_tensor((B, H, cap, D), 2000 + seed, 1.0, dtype)
    vc = synthetic.normal_tensor((B, H, cap, D), 2100 + seed, 1.0, dtype)
    q, kn, vn = synthetic.qkv(B, H, l, D, seed=2200 + seed, std=1.0, dtype=dtype)
    o = torch.full((B, H, l, D), float("nan"), dtype=dtype, device=DEV)
    lse = torch.full((B, H, l), float("nan"), dtype=torch.float32, device=DEV)
    lens_d = torch.tensor(lens, dtype=torch.int32, device=DEV)
    if paged:
        g = torch.Generator().manual_seed(2300 + seed)
        table = torch.randperm(B * mp, generator=g).to(torch.int32).view(B, mp)
        kpool = torch.empty((B * mp, H, ps, D), dtype=dtype)
        vpool = torch.empty_like(kpool)
        for b in range(B):
            for pi in range(mp):
                kpool[int(table[b, pi])] = kc[b, :, pi * ps:(pi + 1) * ps]
                vpool[int(table[b, pi])] = vc[b, :, pi * ps:(pi + 1) * ps]
        L.loma_prefill_attn_paged(q.to(DEV), kn.to(DEV), vn.to(DEV), kpool.to(DEV), vpool.to(DEV), table.to(DEV), o, lse,
                                  lens_d, max_len)
    else:
        L.loma_prefill_attn_ragged(q.to(DEV), kn.to(DEV), vn.to(DEV), kc.to(DEV), vc.to(DEV), o, lse, lens_d, max_len)
    torch.cuda.synchronize()
    assert L.loma_device_status() == 0
    for b, n in enumerate(lens):
        sl = slice(b, b + 1)
        want_o, want_lse, _, _ = oracle.prefill_attn(npf(q[sl]), npf(kn[sl]), npf(vn[sl]), npf(kc[sl, :, :n + l]),
                                                     npf(vc[sl, :, :n + l]), n)
        check_close(o[sl], want_o, dtype)
        assert np.abs(npf(lse[sl]) - want_lse).max() <= 2e-2


def test_prefill_with_rows_already_in_the_cache_and_repeatable():
    """k_new = v_new = NULL: the new rows are read where they already lie; two calls give the same bits."""
    B, H, D, l, cache_len = 2, 2, 128, 150, 333
    cap = cache_len + l
    kc = synthetic.normal_tensor((B, H, cap, D), 51, 1.0, torch.bfloat16).to(DEV)
    vc = synthetic.normal_tensor((B, H, cap, D), 52, 1.0, torch.bfloat16).to(DEV)
    q = synthetic.normal_tensor((B, H, l, D), 53, 1.0, torch.bfloat16).to(DEV)
    want_o, _, _, _ = oracle.prefill_attn(npf(q), npf(kc[:, :, cache_len:]), npf(vc[:, :, cache_len:]), npf(kc), npf(vc), cache_len)
    o1, o2 = torch.empty_like(q), torch.empty_like(q)
    L.loma_prefill_attn(q, None, None, kc, vc, o1, None, cache_len)
    L.loma_prefill_attn(q, None, None, kc, vc, o2, None, cache_len)
    torch.cuda.synchronize()
    check_close(o1, want_o, torch.bfloat16)
    assert torch.equal(o1, o2)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("c,t,pieces", [(4, 16, [150, 74]), (8, 16, [70, 200, 178]), (2, 8, [5, 51])])
def test_prompt_ingested_in_pieces_equals_the_one_shot_inference_layout(c, t, pieces, dtype):
    """Appendix A `add_token_ids` on the GPU path: a prompt of 3.5 chunks arrives in pieces that start and end in
    the middle of chunks; every piece goes through loma_prefill_attn over the cache as it stands (exactly the
    tokens that fill the tail up to tc, then loma_compress_step), and every reading and memory row equals the
    one-pass forward over the inference layout; the cache ends as memory zones in order plus the tail."""
    B, H, D = 1, 2, 128
    tc = c * t
    n_tok = sum(pieces)
    n, tail = n_tok // tc, n_tok % tc
    s = tc + t
    S = oracle.seq_len(n, c, t, tail, NOREP)
    q, k, v = synthetic.qkv(B, H, S, D, seed=61, std=1.0, dtype=dtype)
    want_o, _ = oracle.masked_attn_fwd(npf(q), npf(k), npf(v), n, c, t, tail, NOREP)
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    cap = n * t + tc + 8
    kc = torch.zeros((B, H, cap, D), dtype=dtype, device=DEV)
    vc = torch.zeros_like(kc)
    got = torch.full_like(qd, float("nan"))
    ws = workspace(L.loma_compress_workspace_bytes(B, H, D, t, n * t, 0))
    row_of = lambda g: (g // tc) * s + g % tc
    length = done = chunks = fed = 0
    for piece in pieces:
        fed += piece
        while done < fed:
            take = fed - done
            fills = (length - chunks * t) + take >= tc
            if fills:
                take = tc - (length - chunks * t)
            rows = torch.tensor([row_of(g) for g in range(done, done + take)], device=DEV)
            o = torch.empty((B, H, take, D), dtype=dtype, device=DEV)
            L.loma_prefill_attn(qd[:, :, rows].contiguous(), kd[:, :, rows].contiguous(), vd[:, :, rows].contiguous(), kc, vc, o,
                                None, length)
            got[:, :, rows] = o
            length += take
            done += take
            if fills:
                m0 = chunks * s + tc
                om = torch.empty((B, H, t, D), dtype=dtype, device=DEV)
                L.loma_compress_step(qd[:, :, m0:m0 + t].contiguous(), kd[:, :, m0:m0 + t].contiguous(),
                                     vd[:, :, m0:m0 + t].contiguous(), kc, vc, om, None, chunks * t, c, t, ws)
                got[:, :, m0:m0 + t] = om
                chunks += 1
                length = chunks * t
    torch.cuda.synchronize()
    check_close(got, want_o, dtype)
    rows = [y * s + tc + j for y in range(n) for j in range(t)] + list(range(n * s, S))
    assert length == len(rows)
    assert torch.equal(kc[:, :, :length].cpu(), k[:, :, rows]) and torch.equal(vc[:, :, :length].cpu(), v[:, :, rows])


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_staggered_sequences_over_a_paged_cache_equal_the_one_shot_forward(dtype):
    """Invariant (c) through the ragged and paged entry points: three sequences that started 0, 5 and 11 tokens
    apart share one pool of pages; every step decodes one token of every sequence that still has tokens, and a
    sequence compresses as soon as its tail holds tc tokens, whatever the others are doing.  Every live row of the
    one-shot forward of each sequence is reproduced."""
    H, D, n, c, t, tail, ps = 2, 128, 3, 2, 8, 5, 16
    tc, s = c * t, oracle.chunk_len(c, t)
    S = oracle.seq_len(n, c, t, tail)
    B, starts = 3, [0, 5, 11]
    q, k, v = synthetic.qkv(B, H, S, D, seed=91, std=1.0, dtype=dtype)
    want_o, _ = oracle.masked_attn_fwd(npf(q), npf(k), npf(v), n, c, t, tail)
    zone = oracle.layout_index(n, c, t, tail)[1]
    gen_rows = [i for i in range(S) if zone[i] == oracle.ZONE_READ]          # tokens decoded one at a time, in order
    max_pages = (n * t + tc + ps - 1) // ps + 1
    n_pages = B * max_pages
    table = np.random.default_rng(3).permutation(n_pages).reshape(B, max_pages).astype(np.int32)
    kpool = torch.zeros((n_pages, H, ps, D), dtype=dtype, device=DEV)
    vpool = torch.zeros_like(kpool)
    table_d = torch.from_numpy(table).to(DEV)
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    got = torch.full((B, H, S, D), float("nan"), dtype=dtype, device=DEV)
    ws = workspace(L.loma_decode_workspace_bytes(B, H, D, n * t + tc))
    pos = [0] * B            # next entry of gen_rows per sequence
    lens = [0] * B           # cache entries per sequence
    chunks = [0] * B
    step = 0
    while any(p_ < len(gen_rows) for p_ in pos):
        active = [step >= starts[b] and pos[b] < len(gen_rows) for b in range(B)]
        rows = [gen_rows[min(pos[b], len(gen_rows) - 1)] for b in range(B)]
        take = lambda x: torch.stack([x[b, :, rows[b]:rows[b] + 1] for b in range(B)]).contiguous()
        o1 = torch.empty((B, H, 1, D), dtype=dtype, device=DEV)
        # idle sequences decode a throw-away token into a spare slot of their own pages (their length does not advance)
        lens_d = torch.tensor(lens, dtype=torch.int32, device=DEV)
        L.loma_decode_attn_paged(take(qd), take(kd), take(vd), kpool, vpool, table_d, o1, None, lens_d, max(lens), ws)
        for b in range(B):
            if active[b]:
                got[b, :, rows[b]] = o1[b, :, 0]
                pos[b] += 1
                lens[b] += 1
        # compress every sequence whose tail is full
        mem_lens = [chunks[b] * t if (lens[b] == chunks[b] * t + tc and chunks[b] < n) else -1 for b in range(B)]
        if any(m >= 0 for m in mem_lens):
            m_rows = [chunks[b] * s + tc for b in range(B)]
            takem = lambda x: torch.stack([x[b, :, m_rows[b]:m_rows[b] + t] if mem_lens[b] >= 0 else x[b, :, :t]
                                           for b in range(B)]).contiguous()
            om = torch.empty((B, H, t, D), dtype=dtype, device=DEV)
            L.loma_compress_step_paged(takem(qd), takem(kd), takem(vd), kpool, vpool, table_d, om, None,
                                       torch.tensor(mem_lens, dtype=torch.int32, device=DEV), max(mem_lens), c, t)
            for b in range(B):
                if mem_lens[b] >= 0:
                    got[b, :, m_rows[b]:m_rows[b] + t] = om[b]
                    chunks[b] += 1
                    lens[b] = chunks[b] * t
        step += 1
    torch.cuda.synchronize()
    live = torch.from_numpy(zone != oracle.ZONE_REP).to(DEV)
    check_close(got[:, :, live], want_o[:, :, zone != oracle.ZONE_REP], dtype)


# ------------------------------------------------------------- decode, compress

@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("flags", [0, GENERIC])
@pytest.mark.parametrize("B,H,D,cap,cache_len", [(1, 1, 64, 4, 0), (2, 3, 128, 40, 1), (2, 2, 128, 700, 613),
                                                 (1, 4, 128, 3000, 2999), (3, 2, 64, 1100, 1024),
                                                 (2, 2, 128, 5000, 4133)])
def test_decode_matches_oracle(B, H, D, cap, cache_len, flags, dtype):
    kc = synthetic.normal_tensor((B, H, cap, D), 21, 1.0, dtype)
    vc = synthetic.normal_tensor((B, H, cap, D), 22, 1.0, dtype)
    q, kn, vn = synthetic.qkv(B, H, 1, D, seed=23, std=1.0, dtype=dtype)
    want_o, want_lse, _, _ = oracle.decode_attn(npf(q), npf(kn), npf(vn), npf(kc), npf(vc), cache_len)
    kcd, vcd = kc.to(DEV), vc.to(DEV)
    o = torch.full((B, H, 1, D), float("nan"), dtype=dtype, device=DEV)
    lse = torch.full((B, H), float("nan"), dtype=torch.float32, device=DEV)
    ws = workspace(L.loma_decode_workspace_bytes(B, H, D, cache_len))
    L.loma_decode_attn(q.to(DEV), kn.to(DEV), vn.to(DEV), kcd, vcd, o, lse, cache_len, ws, flags)
    torch.cuda.synchronize()
    check_close(o, want_o, dtype)
    assert np.abs(npf(lse) - want_lse[:, :, 0]).max() <= (1e-5 if dtype == torch.float32 else 2e-2)
    # append is a bit-exact copy into slot cache_len and touches nothing else
    exp_k, exp_v = kc.clone(), vc.clone()
    exp_k[:, :, cache_len] = kn[:, :, 0]
    exp_v[:, :, cache_len] = vn[:, :, 0]
    assert np.array_equal(bits(kcd), bits(exp_k)) and np.array_equal(bits(vcd), bits(exp_v))
    # the same step with the token already in the cache (k_new = v_new = NULL)
    o2 = torch.empty_like(o)
    L.loma_decode_attn(q.to(DEV), None, None, kcd, vcd, o2, None, cache_len, ws, flags)
    torch.cuda.synchronize()
    assert torch.equal(o2, o)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("flags", [0, GENERIC])
@pytest.mark.parametrize("H,D,cap,lens", [(2, 64, 40, [0, 1, 39, 17]), (3, 128, 3000, [2999, 0, 1500, 257, 256, 255]),
                                          (2, 128, 5000, [4133, 4133]), (4, 128, 9000, [8193, 100, 8256, 4097, 1])])
def test_ragged_decode_matches_oracle(H, D, cap, lens, flags, dtype):
    """Sequences at different points of their chunks: each attends to its own prefix of its cache."""
    B = len(lens)
    kc = synthetic.normal_tensor((B, H, cap, D), 31, 1.0, dtype)
    vc = synthetic.normal_tensor((B, H, cap, D), 32, 1.0, dtype)
    q, kn, vn = synthetic.qkv(B, H, 1, D, seed=33, std=1.0, dtype=dtype)
    want_o, want_lse, _, _ = oracle.decode_attn_ragged(npf(q), npf(kn), npf(vn), npf(kc), npf(vc), lens)
    kcd, vcd = kc.to(DEV), vc.to(DEV)
    o = torch.full((B, H, 1, D), float("nan"), dtype=dtype, device=DEV)
    lse = torch.full((B, H), float("nan"), dtype=torch.float32, device=DEV)
    max_len = max(lens)
    ws = workspace(L.loma_decode_workspace_bytes(B, H, D, max_len))
    lens_d = torch.tensor(lens, dtype=torch.int32, device=DEV)
    L.loma_decode_attn_ragged(q.to(DEV), kn.to(DEV), vn.to(DEV), kcd, vcd, o, lse, lens_d, max_len, ws, flags)
    torch.cuda.synchronize()
    check_close(o, want_o, dtype)
    assert np.abs(npf(lse) - want_lse[:, :, 0]).max() <= (1e-5 if dtype == torch.float32 else 2e-2)
    exp_k, exp_v = kc.clone(), vc.clone()
    for b, n in enumerate(lens):
        exp_k[b, :, n] = kn[b, :, 0]
        exp_v[b, :, n] = vn[b, :, 0]
    assert np.array_equal(bits(kcd), bits(exp_k)) and np.array_equal(bits(vcd), bits(exp_v))
    # equal lengths reproduce the uniform entry point bit for bit
    o_u, o_r = torch.empty_like(o), torch.empty_like(o)
    same = torch.full((B,), max_len, dtype=torch.int32, device=DEV)
    L.loma_decode_attn(q.to(DEV), None, None, kcd, vcd, o_u, None, max_len, ws, flags)
    L.loma_decode_attn_ragged(q.to(DEV), None, None, kcd, vcd, o_r, None, same, max_len, ws, flags)
    torch.cuda.synchronize()
    assert torch.equal(o_u, o_r)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("flags", [0, PRIOR, GENERIC, GENERIC | PRIOR])
@pytest.mark.parametrize("B,H,D,c,t,mem_len,extra", [(1, 1, 64, 4, 4, 0, 0), (2, 2, 128, 4, 16, 48, 5),
                                                     (2, 3, 128, 8, 16, 1024, 0), (1, 2, 128, 3, 5, 35, 2),
                                                     (1, 2, 128, 8, 32, 640, 7), (1, 1, 64, 1, 1, 3, 0),
                                                     (2, 2, 128, 4, 16, 2000, 1), (1, 2, 128, 2, 64, 128, 3),
                                                     (1, 1, 64, 2, 100, 1300, 0), (2, 1, 128, 1, 17, 51, 0)])
def test_compress_matches_oracle_and_compacts_bit_exact(B, H, D, c, t, mem_len, extra, flags, dtype):
    tc = c * t
    cap = mem_len + tc + extra
    kc = synthetic.normal_tensor((B, H, cap, D), 31, 1.0, dtype)
    vc = synthetic.normal_tensor((B, H, cap, D), 32, 1.0, dtype)
    qm, km, vm = synthetic.qkv(B, H, t, D, seed=33, std=1.0, dtype=dtype)
    want_o, want_lse, _, _ = oracle.compress_step(npf(qm), npf(km), npf(vm), npf(kc), npf(vc), mem_len, c, t,
                                                  flags & PRIOR)
    kcd, vcd = kc.to(DEV), vc.to(DEV)
    om = torch.full((B, H, t, D), float("nan"), dtype=dtype, device=DEV)
    lse = torch.full((B, H, t), float("nan"), dtype=torch.float32, device=DEV)
    ws = workspace(L.loma_compress_workspace_bytes(B, H, D, t, mem_len, flags))
    L.loma_compress_step(qm.to(DEV), km.to(DEV), vm.to(DEV), kcd, vcd, om, lse, mem_len, c, t, ws, flags)
    torch.cuda.synchronize()
    check_close(om, want_o, dtype)
    assert np.abs(npf(lse) - want_lse).max() <= (1e-5 if dtype == torch.float32 else 2e-2)
    # compaction == cat(cache[:mem_len], k_mem): the oracle's explicit copies run on the raw bit patterns
    _, _, nk, nv = oracle.compress_step(np.zeros((B, H, t, D)), bits(km), bits(vm), bits(kc), bits(vc), mem_len,
                                        c, t, flags & PRIOR, scale=0.0)
    assert np.array_equal(bits(kcd[:, :, :mem_len + t]), nk)
    assert np.array_equal(bits(vcd[:, :, :mem_len + t]), nv)
    assert np.array_equal(bits(kcd[:, :, :mem_len]), bits(kc[:, :, :mem_len]))


# ------------------------------------------------------- failure detection

@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("flags", [0, GENERIC])
@pytest.mark.parametrize("H,D,c,t,lens", [(2, 64, 4, 4, [0, 16, -1, 8]), (2, 128, 4, 16, [48, -1, 1024, 0, 512]),
                                          (1, 128, 2, 64, [128, 64, -1]), (2, 128, 8, 16, [8192, 4096, -1, 16])])
def test_ragged_compress_matches_oracle_and_leaves_idle_sequences_alone(H, D, c, t, lens, flags, dtype):
    B, tc = len(lens), c * t
    max_len = max(lens)
    cap = max_len + tc + 3
    kc = synthetic.normal_tensor((B, H, cap, D), 41, 1.0, dtype)
    vc = synthetic.normal_tensor((B, H, cap, D), 42, 1.0, dtype)
    qm, km, vm = synthetic.qkv(B, H, t, D, seed=43, std=1.0, dtype=dtype)
    want_o, want_lse, want_k, want_v = oracle.compress_step_ragged(npf(qm), npf(km), npf(vm), npf(kc), npf(vc), lens, c, t)
    kcd, vcd = kc.to(DEV), vc.to(DEV)
    om = torch.full((B, H, t, D), 7.0, dtype=dtype, device=DEV)
    lse = torch.full((B, H, t), 7.0, dtype=torch.float32, device=DEV)
    lens_d = torch.tensor(lens, dtype=torch.int32, device=DEV)
    L.loma_compress_step_ragged(qm.to(DEV), km.to(DEV), vm.to(DEV), kcd, vcd, om, lse, lens_d, max_len, c, t, flags)
    torch.cuda.synchronize()
    for b, n in enumerate(lens):
        if n < 0:
            assert float((om[b].float() - 7.0).abs().max()) == 0.0 and float((lse[b] - 7.0).abs().max()) == 0.0
            assert torch.equal(kcd[b].cpu(), kc[b]) and torch.equal(vcd[b].cpu(), vc[b])
            continue
        check_close(om[b:b + 1], want_o[b:b + 1], dtype)
        assert np.abs(npf(lse[b]) - want_lse[b]).max() <= (1e-5 if dtype == torch.float32 else 2e-2)
        assert np.array_equal(npf(kcd[b, :, :n + t]), want_k[b, :, :n + t]) and np.array_equal(npf(vcd[b, :, :n + t]), want_v[b, :, :n + t])
        assert torch.equal(kcd[b, :, n + t:].cpu(), kc[b, :, n + t:])      # slots beyond the rewritten ones keep their contents


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("flags", [0, GENERIC])
@pytest.mark.parametrize("H,D,ps,lens", [(2, 64, 16, [0, 1, 39, 17]), (3, 128, 64, [2999, 0, 1500, 257, 256, 255]),
                                         (4, 128, 256, [8193, 100, 8256, 4097, 1]), (2, 128, 16, [4133, 4133])])
def test_paged_decode_matches_oracle(H, D, ps, lens, flags, dtype):
    """Sequences scattered over a shuffled pool of pages: each attends to its own slots through the block table."""
    B = len(lens)
    max_len = max(lens)
    max_pages = max_len // ps + 1
    n_pages = B * max_pages + 3
    rng = np.random.default_rng(7)
    perm = rng.permutation(n_pages)[: B * max_pages].reshape(B, max_pages).astype(np.int32)
    kp = synthetic.normal_tensor((n_pages, H, ps, D), 51, 1.0, dtype)
    vp = synthetic.normal_tensor((n_pages, H, ps, D), 52, 1.0, dtype)
    q, kn, vn = synthetic.qkv(B, H, 1, D, seed=53, std=1.0, dtype=dtype)
    want_o, want_lse, want_k, want_v = oracle.decode_attn_paged(npf(q), npf(kn), npf(vn), npf(kp), npf(vp), perm, lens)
    kpd, vpd = kp.to(DEV), vp.to(DEV)
    o = torch.full((B, H, 1, D), float("nan"), dtype=dtype, device=DEV)
    lse = torch.full((B, H), float("nan"), dtype=torch.float32, device=DEV)
    ws = workspace(L.loma_decode_workspace_bytes(B, H, D, max_len))
    table_d = torch.from_numpy(perm).to(DEV)
    lens_d = torch.tensor(lens, dtype=torch.int32, device=DEV)
    L.loma_decode_attn_paged(q.to(DEV), kn.to(DEV), vn.to(DEV), kpd, vpd, table_d, o, lse, lens_d, max_len, ws, flags)
    torch.cuda.synchronize()
    check_close(o, want_o, dtype)
    assert np.abs(npf(lse) - want_lse[:, :, 0]).max() <= (1e-5 if dtype == torch.float32 else 2e-2)
    # the pools changed in exactly the appended slots
    assert np.array_equal(npf(kpd), want_k) and np.array_equal(npf(vpd), want_v)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("flags", [0, GENERIC])
@pytest.mark.parametrize("H,D,c,t,ps,lens", [(2, 64, 4, 4, 16, [0, 16, -1, 8]), (2, 128, 4, 16, 64, [48, -1, 1024, 0, 500]),
                                             (1, 128, 2, 64, 32, [128, 70, -1]), (2, 128, 8, 16, 256, [8192, 4090, -1, 16])])
def test_paged_compress_matches_oracle(H, D, c, t, ps, lens, flags, dtype):
    """Tails and rewritten slots that straddle pages of a shuffled pool; idle sequences and unused pages untouched."""
    B, tc = len(lens), c * t
    max_len = max(lens)
    max_pages = (max_len + tc + ps - 1) // ps
    n_pages = B * max_pages + 2
    table = np.random.default_rng(9).permutation(n_pages)[: B * max_pages].reshape(B, max_pages).astype(np.int32)
    kp = synthetic.normal_tensor((n_pages, H, ps, D), 61, 1.0, dtype)
    vp = synthetic.normal_tensor((n_pages, H, ps, D), 62, 1.0, dtype)
    qm, km, vm = synthetic.qkv(B, H, t, D, seed=63, std=1.0, dtype=dtype)
    want_o, want_lse, want_k, want_v = oracle.compress_step_paged(npf(qm), npf(km), npf(vm), npf(kp), npf(vp), table, lens, c, t)
    kpd, vpd = kp.to(DEV), vp.to(DEV)
    om = torch.full((B, H, t, D), 7.0, dtype=dtype, device=DEV)
    lse = torch.full((B, H, t), 7.0, dtype=torch.float32, device=DEV)
    L.loma_compress_step_paged(qm.to(DEV), km.to(DEV), vm.to(DEV), kpd, vpd, torch.from_numpy(table).to(DEV), om, lse,
                               torch.tensor(lens, dtype=torch.int32, device=DEV), max_len, c, t, flags)
    torch.cuda.synchronize()
    for b, n in enumerate(lens):
        if n < 0:
            assert float((om[b].float() - 7.0).abs().max()) == 0.0
            continue
        check_close(om[b:b + 1], want_o[b:b + 1], dtype)
        assert np.abs(npf(lse[b]) - want_lse[b]).max() <= (1e-5 if dtype == torch.float32 else 2e-2)
    assert np.array_equal(npf(kpd), want_k) and np.array_equal(npf(vpd), want_v)      # pools differ in the rewritten slots only


def test_bounded_wait_times_out_and_leaves_the_context_usable():
    """A device-side wait that can never be satisfied gives up after its limit,
    reports LOMA_ERR_TIMEOUT through the status word, and later launches work."""
    assert L.loma_device_status() == 0
    L.loma_selftest_bounded_wait()
    assert L.loma_device_status() == -7          # LOMA_ERR_TIMEOUT, reported once
    assert L.loma_device_status() == 0           # cleared by the read
    q, k, v = (x.to(DEV) for x in synthetic.qkv(1, 1, 144, 128, seed=3, dtype=torch.bfloat16))
    o, _ = run_fwd(q, k, v, 1, 4, 16)
    want, _ = oracle.masked_attn_fwd(npf(q), npf(k), npf(v), 1, 4, 16)
    check_close(o, want, torch.bfloat16)


# ----------------------------------------------------------- repeatability

def test_results_are_bitwise_repeatable():
    B, H, D, n, c, t = 1, 2, 128, 4, 4, 16
    S = oracle.seq_len(n, c, t)
    q, k, v = (x.to(DEV) for x in synthetic.qkv(B, H, S, D, seed=5, dtype=torch.bfloat16))
    o1, l1 = run_fwd(q, k, v, n, c, t)
    o2, l2 = run_fwd(q, k, v, n, c, t)
    assert torch.equal(o1, o2) and torch.equal(l1, l2)
    kc = synthetic.normal_tensor((2, 4, 3000, 128), 1, 1.0, torch.bfloat16).to(DEV)
    vc = synthetic.normal_tensor((2, 4, 3000, 128), 2, 1.0, torch.bfloat16).to(DEV)
    q1 = synthetic.normal_tensor((2, 4, 1, 128), 3, 1.0, torch.bfloat16).to(DEV)
    ws = workspace(L.loma_decode_workspace_bytes(2, 4, 128, 2900))
    outs = []
    for _ in range(2):
        o = torch.empty_like(q1)
        L.loma_decode_attn(q1, None, None, kc, vc, o, None, 2900, ws)
        torch.cuda.synchronize()
        outs.append(o)
    assert torch.equal(outs[0], outs[1])


# ------------------------------------- named workloads at full size (sampled)

def test_training_layout_4608_tokens_sampled_heads():
    """B4 H32 D128 bf16, c=4, t=16, 32 chunks of [64|16|64] = 4608 rows, N(0,1):
    the launch covers the full tensor, the oracle checks two (b,h) pairs in full."""
    B, H, D, n, c, t = 4, 32, 128, 32, 4, 16
    S = oracle.seq_len(n, c, t)
    assert S == 4608
    q = synthetic.big_normal_(torch.empty(B, H, S, D, dtype=torch.bfloat16, device=DEV), 100)
    k = synthetic.big_normal_(torch.empty(B, H, S, D, dtype=torch.bfloat16, device=DEV), 101)
    v = synthetic.big_normal_(torch.empty(B, H, S, D, dtype=torch.bfloat16, device=DEV), 102)
    for flags in (0, PRIOR):
        o, lse = run_fwd(q, k, v, n, c, t, 0, flags)
        for b, h in [(0, 0), (3, 17)]:
            want_o, want_lse = oracle.masked_attn_fwd(npf(q[b:b + 1, h:h + 1]), npf(k[b:b + 1, h:h + 1]),
                                                      npf(v[b:b + 1, h:h + 1]), n, c, t, 0, flags)
            check_close(o[b:b + 1, h:h + 1], want_o, torch.bfloat16)
            assert np.abs(npf(lse[b:b + 1, h:h + 1]) - want_lse).max() <= 2e-2
        assert torch.isfinite(o.float()).all()


def test_long_training_layout_69632_tokens_sampled_rows():
    """B1 H32 D128 bf16, c=8, t=32, 128 chunks of [256|32|256] = 69632 rows: the
    full launch, checked on a seeded sample of rows of every zone type."""
    B, H, D, n, c, t = 1, 32, 128, 128, 8, 32
    S = oracle.seq_len(n, c, t)
    assert S == 69632
    q = synthetic.big_normal_(torch.empty(B, H, S, D, dtype=torch.bfloat16, device=DEV), 110)
    k = synthetic.big_normal_(torch.empty(B, H, S, D, dtype=torch.bfloat16, device=DEV), 111)
    v = synthetic.big_normal_(torch.empty(B, H, S, D, dtype=torch.bfloat16, device=DEV), 112)
    o, lse = run_fwd(q, k, v, n, c, t)
    zone = oracle.layout_index(n, c, t)[1]
    rng = np.random.default_rng(0)
    rows = np.concatenate([rng.choice(np.nonzero(zone == z)[0], 96, replace=False) for z in (0, 1, 2)]
                          + [np.array([0, 255, 256, 287, 288, 543, 544, S - 1, S - 257, S - 545])])
    rows = np.unique(rows)
    idx = torch.from_numpy(rows).to(DEV)
    for h in (0, 13, 31):
        want_o, want_lse = oracle.masked_attn_fwd(npf(q[:, h:h + 1]), npf(k[:, h:h + 1]), npf(v[:, h:h + 1]),
                                                  n, c, t, rows=rows)
        check_close(o[:, h:h + 1][:, :, idx], want_o, torch.bfloat16)
        assert np.abs(npf(lse[:, h:h + 1][:, :, idx]) - want_lse).max() <= 2e-2
    assert torch.isfinite(o.float()).all()


@pytest.mark.parametrize("B,H,c,t,mem_len,steps", [(32, 32, 4, 16, 8192, (0, 1, 37, 63)),
                                                   (64, 32, 8, 16, 16384, (0, 127))])
def test_generation_workloads_sampled_heads(B, H, c, t, mem_len, steps):
    """Generation shapes (D128 bf16): a cache of mem_len memory entries plus a
    growing tail; decode at several tail lengths, then the compress step.  The
    launch covers every (b,h); the oracle checks three of them in full."""
    D, tc = 128, c * t
    cap = mem_len + tc + t
    kc = synthetic.big_normal_(torch.empty(B, H, cap, D, dtype=torch.bfloat16, device=DEV), 120)
    vc = synthetic.big_normal_(torch.empty(B, H, cap, D, dtype=torch.bfloat16, device=DEV), 121)
    ws = workspace(max(L.loma_decode_workspace_bytes(B, H, D, cap),
                       L.loma_compress_workspace_bytes(B, H, D, t, mem_len, PRIOR)))
    picks = [(0, 0), (B // 2, 5), (B - 1, H - 1)]
    for j in steps:
        cache_len = mem_len + j
        q, kn, vn = (x.to(DEV) for x in synthetic.qkv(B, H, 1, D, seed=200 + j, dtype=torch.bfloat16))
        before_k = [kc[b, h].clone() for b, h in picks]
        before_v = [vc[b, h].clone() for b, h in picks]
        o = torch.empty(B, H, 1, D, dtype=torch.bfloat16, device=DEV)
        lse = torch.empty(B, H, dtype=torch.float32, device=DEV)
        L.loma_decode_attn(q, kn, vn, kc, vc, o, lse, cache_len, ws)
        torch.cuda.synchronize()
        for (b, h), bk, bv in zip(picks, before_k, before_v):
            want_o, want_lse, wk, wv = oracle.decode_attn(npf(q[b:b + 1, h:h + 1]), npf(kn[b:b + 1, h:h + 1]),
                                                          npf(vn[b:b + 1, h:h + 1]), npf(bk[None, None]),
                                                          npf(bv[None, None]), cache_len)
            check_close(o[b:b + 1, h:h + 1], want_o, torch.bfloat16)
            assert abs(float(lse[b, h]) - want_lse[0, 0, 0]) <= 2e-2
            assert np.array_equal(npf(kc[b, h]), wk[0, 0]) and np.array_equal(npf(vc[b, h]), wv[0, 0])
    for flags in (0, PRIOR):
        kc2, vc2 = kc.clone(), vc.clone()
        qm, km, vm = (x.to(DEV) for x in synthetic.qkv(B, H, t, D, seed=300, dtype=torch.bfloat16))
        om = torch.empty(B, H, t, D, dtype=torch.bfloat16, device=DEV)
        L.loma_compress_step(qm, km, vm, kc2, vc2, om, None, mem_len, c, t, ws, flags)
        torch.cuda.synchronize()
        for b, h in picks:
            want_o, _, nk, nv = oracle.compress_step(npf(qm[b:b + 1, h:h + 1]), npf(km[b:b + 1, h:h + 1]),
                                                     npf(vm[b:b + 1, h:h + 1]), npf(kc[b:b + 1, h:h + 1]),
                                                     npf(vc[b:b + 1, h:h + 1]), mem_len, c, t, flags)
            check_close(om[b:b + 1, h:h + 1], want_o, torch.bfloat16)
            assert np.array_equal(npf(kc2[b, h, :mem_len + t]), nk[0, 0])
            assert np.array_equal(npf(vc2[b, h, :mem_len + t]), nv[0, 0])
        del kc2, vc2


def test_layer_loop_equals_layer_by_layer_calls_and_the_oracle():
    """Appendix A loops over the layers' caches; the *_layers entry points do that loop inside one call: same bits
    as one call per layer, the oracle checked on one layer."""
    B, H, D, c, t, mem_len, nl = 2, 3, 128, 4, 16, 320, 3
    tc = c * t
    cap = mem_len + tc + 4
    dt = torch.bfloat16
    mk = lambda shape, seed: [synthetic.normal_tensor(shape, seed + 10 * i, 1.0, dt).to(DEV) for i in range(nl)]
    kc, vc = mk((B, H, cap, D), 400), mk((B, H, cap, D), 401)
    kc2, vc2 = [x.clone() for x in kc], [x.clone() for x in vc]
    ws = workspace(max(L.loma_decode_workspace_bytes(B, H, D, cap), L.loma_compress_workspace_bytes(B, H, D, t, mem_len, 0)))
    for j in range(tc):                                   # a whole chunk: tc decodes ...
        q, kn, vn = mk((B, H, 1, D), 500 + j), mk((B, H, 1, D), 600 + j), mk((B, H, 1, D), 700 + j)
        o = [torch.empty((B, H, 1, D), dtype=dt, device=DEV) for _ in range(nl)]
        o2 = [torch.empty_like(x) for x in o]
        if j == tc - 1:
            want_o, _, _, _ = oracle.decode_attn(npf(q[1]), npf(kn[1]), npf(vn[1]), npf(kc[1]), npf(vc[1]), mem_len + j)
        L.loma_decode_attn_layers(q, kn, vn, kc, vc, o, None, mem_len + j, ws)
        for i in range(nl):
            L.loma_decode_attn(q[i], kn[i], vn[i], kc2[i], vc2[i], o2[i], None, mem_len + j, ws)
        torch.cuda.synchronize()
        for i in range(nl):
            assert torch.equal(o[i], o2[i])
    check_close(o[1], want_o, dt)
    qm, km, vm = mk((B, H, t, D), 800), mk((B, H, t, D), 801), mk((B, H, t, D), 802)
    om = [torch.empty((B, H, t, D), dtype=dt, device=DEV) for _ in range(nl)]
    om2 = [torch.empty_like(x) for x in om]
    want_om, _, nk, nv = oracle.compress_step(npf(qm[2]), npf(km[2]), npf(vm[2]), npf(kc[2]), npf(vc[2]), mem_len, c, t)
    L.loma_compress_step_layers(qm, km, vm, kc, vc, om, None, mem_len, c, t, ws)     # ... then the compress step
    for i in range(nl):
        L.loma_compress_step(qm[i], km[i], vm[i], kc2[i], vc2[i], om2[i], None, mem_len, c, t, ws)
    torch.cuda.synchronize()
    for i in range(nl):
        assert torch.equal(om[i], om2[i])
        assert torch.equal(kc[i][:, :, :mem_len + t], kc2[i][:, :, :mem_len + t]) and torch.equal(vc[i][:, :, :mem_len + t], vc2[i][:, :, :mem_len + t])
    check_close(om[2], want_om, dt)
    assert np.array_equal(npf(kc[2][:, :, :mem_len + t]), nk) and np.array_equal(npf(vc[2][:, :, :mem_len + t]), nv)


def test_generation_cycle_replays_from_a_cuda_graph():
    """After one eager call of each entry point (first calls look up device symbols and set kernel attributes),
    a tail of decode steps plus the compress step is captured into a CUDA graph and replayed: the replay equals
    the eager run bit for bit, outputs and caches."""
    B, H, D, c, t, mem_len = 2, 4, 128, 4, 16, 256
    tc = c * t
    cap = mem_len + tc + t
    dtype = torch.bfloat16
    kc0 = synthetic.normal_tensor((B, H, cap, D), 61, 1.0, dtype).to(DEV)
    vc0 = synthetic.normal_tensor((B, H, cap, D), 62, 1.0, dtype).to(DEV)
    steps = 5
    qs, ks, vs = (synthetic.normal_tensor((steps, B, H, 1, D), 63 + i, 1.0, dtype).to(DEV) for i in range(3))
    qm, km, vm = (x.to(DEV) for x in synthetic.qkv(B, H, t, D, seed=66, dtype=dtype))
    ws = workspace(max(L.loma_decode_workspace_bytes(B, H, D, cap), L.loma_compress_workspace_bytes(B, H, D, t, mem_len, 0)))

    def cycle(kc, vc, outs, om, stream=None):
        for j in range(steps):
            L.loma_decode_attn(qs[j], ks[j], vs[j], kc, vc, outs[j], None, mem_len + tc - steps + j, ws, 0, 0.0, stream)
        L.loma_compress_step(qm, km, vm, kc, vc, om, None, mem_len, c, t, ws, 0, 0.0, stream)

    kc_e, vc_e = kc0.clone(), vc0.clone()
    outs_e, om_e = torch.zeros((steps, B, H, 1, D), dtype=dtype, device=DEV), torch.zeros((B, H, t, D), dtype=dtype, device=DEV)
    cycle(kc_e, vc_e, outs_e, om_e)
    torch.cuda.synchronize()

    kc_g, vc_g = kc0.clone(), vc0.clone()
    outs_g, om_g = torch.zeros_like(outs_e), torch.zeros_like(om_e)
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            cycle(kc_g, vc_g, outs_g, om_g, side)
    torch.cuda.synchronize()
    for _ in range(2):
        kc_g.copy_(kc0); vc_g.copy_(vc0); outs_g.zero_(); om_g.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(outs_g, outs_e) and torch.equal(om_g, om_e)
        assert torch.equal(kc_g[:, :, :mem_len + t], kc_e[:, :, :mem_len + t]) and torch.equal(vc_g[:, :, :mem_len + t], vc_e[:, :, :mem_len + t])


def test_forwards_on_two_streams_at_once_do_not_disturb_each_other():
    """The forward hands out tiles from a counter that belongs to the launch's stream (a captured launch gets
    one of its own), so launches in flight on different streams -- many more than there were counters when
    they were dealt round robin -- and a graph replay next to eager launches must each produce exactly what
    they produce alone."""
    B, H, D, n, c, t = 2, 8, 128, 12, 4, 16
    S = oracle.seq_len(n, c, t)
    a = [x.to(DEV) for x in synthetic.qkv(B, H, S, D, seed=101, dtype=torch.bfloat16)]
    b = [x.to(DEV) for x in synthetic.qkv(B, H, S, D, seed=102, dtype=torch.bfloat16)]
    alone_a, _ = run_fwd(*a, n, c, t)
    alone_b, _ = run_fwd(*b, n, c, t)
    s1, s2, s3 = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    # a captured forward (replayed below on a third stream while the eager ones run)
    og = torch.empty_like(a[0])
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s3):
        L.loma_masked_attn_fwd(*a, og, None, n, c, t, 0, 0, 0.0, s3)      # set-up call before the capture
        s3.synchronize()
        with torch.cuda.graph(graph, stream=s3):
            L.loma_masked_attn_fwd(*a, og, None, n, c, t, 0, 0, 0.0, torch.cuda.current_stream())
    og.fill_(float("nan"))
    torch.cuda.synchronize()
    reps = 70                                        # > 64 launches outstanding per stream
    oa = [torch.empty_like(a[0]) for _ in range(4)]
    ob = [torch.empty_like(b[0]) for _ in range(4)]
    for i in range(reps):
        L.loma_masked_attn_fwd(*a, oa[i % 4], None, n, c, t, 0, 0, 0.0, s1)
        L.loma_masked_attn_fwd(*b, ob[i % 4], None, n, c, t, 0, 0, 0.0, s2)
        if i % 10 == 5:
            with torch.cuda.stream(s3):
                graph.replay()
    torch.cuda.synchronize()
    for i in range(4):
        assert torch.equal(oa[i], alone_a) and torch.equal(ob[i], alone_b)
    assert torch.equal(og, alone_a)
